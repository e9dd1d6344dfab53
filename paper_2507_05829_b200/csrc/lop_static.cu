// lop_run_whole_static: whole-tensor execution of a chain for callers that must not allocate.
//
// Every other execution entry point wants a caller-allocated workspace and, on its first call,
// creates a side stream, events and device tables.  A caller that lives inside someone else's
// memory budget -- a plug-in of a host application that forbids cudaMalloc after start-up, a
// real-time loop that must not take the allocator's lock, a process whose device memory is
// fully pre-assigned -- cannot do either.  For them the scratch (status word, the stem's patch
// tensor and zero-padded weights, the intermediate tensors between layers) lives in one
// fixed-size array in the library's own device image, and the layers are launched one kernel
// after the other with nothing created, cached or freed.
//
// The array exists once per device that loads the library and is shared by every call: a call
// overwrites whatever the previous one left, so everything that has to start from a known value
// (the status word, the padded weights, the stem patches) is rewritten by each call, and two calls
// whose kernels may overlap on the GPU (different streams, different threads) corrupt each other.
#include <cuda_runtime.h>

#include <mutex>

#include "lop_internal.h"
#include "lop_kernels.cuh"
#include "lop_layerargs.h"

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
        if ((pl->layers[i].l.op == LOP_CONV2D || pl->layers[i].l.op == LOP_DWCONV2D) && !pl->layers[i].l.weight) {
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
    for (int i = 0; i < L; ++i) {
        const LayerInfo &li = pl->layers[i];
        const lop_layer &l = li.l;
        if (l.op == LOP_MAXPOOL2D) {
            PoolArgs pa = pool_args(pl, i, in, out, ws, 0, li.Ho);
            if (pa.dbg) pa.dbg = status;                   // checked execution reports into the word this call was given
            ST_CUDA(launch_maxpool(pa, pl->dtype, s));
            continue;
        }
        ConvArgs a = conv_args(pl, i, in, out, ws, 0, li.Ho);
        if (a.dbg) a.dbg = status;
        if (li.kernel == K_DWCONV) {
            const void *w_taps = nullptr;
            if (li.dw_transposed) {                    // rebuilt by every call, like the padded stem weights
                ST_CUDA(launch_dw_transpose(l.weight, ws + li.wpad_off, l.cin, l.kh * l.kw, s));
                w_taps = ws + li.wpad_off;
            }
            ST_CUDA(launch_dwconv(a, pl->dtype, w_taps, s));
            continue;
        }
        if (li.kernel == K_LAYERNORM) { ST_CUDA(launch_layernorm(a, pl->dtype, s)); continue; }
        if (li.kernel == K_CONCAT) { ST_CUDA(launch_concat(a, pl->dtype, s)); continue; }
        if (li.kernel != K_CONV_TC) {
            ST_CUDA(launch_conv_simt(a, pl->dtype, s));
            continue;
        }
        if (li.stem_gather) {
            // another plan may have used the array since: padded weights and patches are rebuilt by every call
            ST_CUDA(launch_pad_weights(l.weight, ws + li.wpad_off, l.cout, l.kh * l.kw * l.cin, li.cin_eff, s));
            ST_CUDA(launch_stem_gather(in, ws + pl->col_off, gather_geom(pl, i), 0, li.Ho, s, a.dbg));
        }
        const ConvTcGeom g = conv_tc_geometry(a, li.Ho);
        ConvTcMaps maps;                                   // encoded on the stack: nothing is cached between calls
        rc = conv_tc_encode(a, g, &maps);
        if (rc != LOP_OK) { set_error("layer %d: tensor-map encoding failed", i); return rc; }
        ST_CUDA(launch_conv_tc(a, g, maps, status, s));
    }
    return LOP_OK;
}
