// lop_run_whole_static: whole-tensor execution of a chain for callers that must not allocate.
//
// Every other execution entry point wants a caller-allocated workspace and, on its first call,
// creates a side stream, events and device tables.  A caller that lives inside someone else's
// memory budget -- a plug-in of a host application that forbids cudaMalloc after start-up, a
// real-time loop that must not take the allocator's lock, a process whose device memory is
// fully pre-assigned -- cannot do either.  For them the scratch (status word, channel-padded
// input and first-layer weights, the intermediate tensors between layers) lives in one
// fixed-size array in the library's own device image, and the layers are launched one kernel
// after the other with nothing created, cached or freed.
//
// The array exists once per device that loads the library and is shared by every call: a call
// overwrites whatever the previous one left, so everything that has to start from a known value
// (the status word, the padded weights, the padded input) is rewritten by each call, and two calls
// whose kernels may overlap on the GPU (different streams, different threads) corrupt each other.
#include <cuda_runtime.h>

#include <mutex>

#include "lop_internal.h"
#include "lop_kernels.cuh"

namespace lop {
namespace {

// In host code this name is only a handle for cudaGetSymbolAddress; it is not a device address.
static __device__ __align__(256) unsigned char g_static_scratch[LOP_STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
unsigned char *g_scratch_addr[MAX_DEVICES];      // per device ordinal: device address of the array, once resolved
std::mutex g_scratch_mutex;

#define ST_CUDA(call)                                                                   \
    do {                                                                                \
        cudaError_t e__ = (call);                                                       \
        if (e__ != cudaSuccess) {                                                       \
            set_error("%s failed: %s", #call, cudaGetErrorString(e__));                 \
            return LOP_ECUDA;                                                           \
        }                                                                               \
    } while (0)

// Device address of the scratch array on the CURRENT device (resolved once per device).
int scratch_for_current_device(unsigned char **out)
{
    int dev = 0;
    ST_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MAX_DEVICES) { set_error("device ordinal %d is not supported", dev); return LOP_EUNSUPPORTED; }
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        unsigned char *p = nullptr;
        ST_CUDA(cudaGetSymbolAddress(reinterpret_cast<void **>(&p), g_static_scratch));
        if (!p) { set_error("cudaGetSymbolAddress returned a null address"); return LOP_ECUDA; }
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return LOP_OK;
}

const void *tensor_at(const lop_plan_t *pl, int idx, const void *in, void *out, unsigned char *ws)
{
    if (idx == LOP_INPUT) return in;
    if (idx == (int)pl->layers.size() - 1) return out;
    return ws + pl->layers[idx].out_off;
}

}  // namespace
}  // namespace lop

using namespace lop;

extern "C" int lop_run_whole_static(lop_plan_t *pl, const void *in, void *out, unsigned *status_dev, void *stream)
{
    if (!pl) { set_error("plan is NULL"); return LOP_EINVAL; }
    if (pl->ws_bytes > (size_t)LOP_STATIC_SCRATCH_BYTES) {
        set_error("lop_run_whole_static: this plan needs %zu bytes of scratch, the built-in scratch holds %zu "
                  "(use lop_run_whole with a workspace of your own)", pl->ws_bytes, (size_t)LOP_STATIC_SCRATCH_BYTES);
        return LOP_EUNSUPPORTED;
    }
    if (!in || !out) { set_error("input/output pointer is NULL"); return LOP_EINVAL; }
    if ((reinterpret_cast<uintptr_t>(in) & 15u) || (reinterpret_cast<uintptr_t>(out) & 15u) ||
        (reinterpret_cast<uintptr_t>(status_dev) & 3u)) {
        set_error("input/output tensors must be 16-byte aligned, the status word 4-byte aligned");
        return LOP_EINVAL;
    }
    const int L = (int)pl->layers.size();
    for (int i = 0; i < L; ++i)
        if (pl->layers[i].l.op == LOP_CONV2D && !pl->layers[i].l.weight) {
            set_error("layer %d has no weight pointer (lop_plan_set_params)", i);
            return LOP_EINVAL;
        }
    unsigned char *ws = nullptr;
    int rc = scratch_for_current_device(&ws);
    if (rc != LOP_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    // the previous call's leftovers: the status word must read 0 before any kernel can raise it
    unsigned *status = status_dev ? status_dev : reinterpret_cast<unsigned *>(ws + pl->status_off);
    ST_CUDA(cudaMemsetAsync(status, 0, sizeof(unsigned), s));
    if (pl->Cpad)
        ST_CUDA(launch_pad_channels(in, ws + pl->padin_off, pl->N, pl->H, pl->W, pl->C, pl->Cpad, 0, pl->H, s));
    for (int i = 0; i < L; ++i) {
        const LayerInfo &li = pl->layers[i];
        const lop_layer &l = li.l;
        void *y = const_cast<void *>(tensor_at(pl, i, in, out, ws));
        if (l.op == LOP_MAXPOOL2D) {
            PoolArgs a;
            a.x = tensor_at(pl, l.input_from, in, out, ws);
            a.y = y;
            a.N = pl->N; a.Hin = li.Hin; a.Win = li.Win; a.C = l.cin; a.Ho = li.Ho; a.Wo = li.Wo;
            a.kh = l.kh; a.kw = l.kw; a.sh = l.sh; a.sw = l.sw; a.ph = l.ph; a.pw = l.pw; a.dh = l.dh; a.dw = l.dw;
            a.oh_lo = 0; a.oh_hi = li.Ho;
            ST_CUDA(launch_maxpool(a, pl->dtype, s));
            continue;
        }
        ConvArgs a;
        a.x = tensor_at(pl, l.input_from, in, out, ws);
        a.w = l.weight;
        a.scale = l.scale; a.shift = l.shift;
        a.res = l.residual_from == LOP_NO_RESIDUAL ? nullptr : tensor_at(pl, l.residual_from, in, out, ws);
        a.y = y;
        a.N = pl->N; a.Hin = li.Hin; a.Win = li.Win; a.Cin = l.cin; a.Ho = li.Ho; a.Wo = li.Wo; a.Cout = l.cout;
        a.kh = l.kh; a.kw = l.kw; a.sh = l.sh; a.sw = l.sw; a.ph = l.ph; a.pw = l.pw; a.dh = l.dh; a.dw = l.dw;
        a.act = l.act; a.res_pos = a.res ? l.residual_pos : LOP_RES_NONE;
        a.oh_lo = 0; a.oh_hi = li.Ho;
        if (li.kernel != K_CONV_TC) {
            ST_CUDA(launch_conv_simt(a, pl->dtype, s));
            continue;
        }
        if (li.reads_padded_input) {
            // another plan may have used the array since: the padded weights are rebuilt by every call
            ST_CUDA(launch_pad_weights(l.weight, ws + li.wpad_off, (long long)l.cout * l.kh * l.kw, l.cin, li.cin_eff, s));
            a.x = ws + pl->padin_off;
            a.w = ws + li.wpad_off;
        }
        a.Cin = li.cin_eff;
        const ConvTcGeom g = conv_tc_geometry(a, li.Ho);
        ConvTcMaps maps;                                   // encoded on the stack: nothing is cached between calls
        rc = conv_tc_encode(a, g, &maps);
        if (rc != LOP_OK) { set_error("layer %d: tensor-map encoding failed", i); return rc; }
        ST_CUDA(launch_conv_tc(a, g, maps, status, s));
    }
    return LOP_OK;
}
