/*
 * lop.h -- C ABI of the band-wise local-operator library for NVIDIA B200 (sm_100a).
 *
 * The library executes a chain of LOCAL operators in the sense of Sec. IV-A of the
 * Intra-DP paper (arxiv 2507.05829): block-wise operators (2-D convolution, max pooling),
 * element-wise operators (ReLU, SiLU, folded batch-norm scale/shift) and the residual
 * addition.  Following the paper's local-operation parallelism (Sec. IV-B), the rows of the
 * chain's output are cut into contiguous bands; every band carries the halo rows its
 * receptive field needs, so the input of band i+1 can still be in flight while band i is
 * being computed, and the stitched result equals whole-tensor execution.
 *
 * Conventions
 *   - Every function returns LOP_OK (0) or a negative lop_status; nothing throws or aborts.
 *     A human-readable message for the calling thread's last failure: lop_last_error().
 *   - "host" / "device" / "pinned host" say where a pointer must live.  The caller owns every
 *     buffer and the stream; the library owns the opaque plan and what hangs off it (one side
 *     stream, events, tensor maps and small device-side program tables it allocates on the first
 *     execution call for a given set of buffers), all released by lop_plan_destroy().
 *   - Activations are NHWC, contiguous; weights are [cout][kh][kw][cin] (KRSC), contiguous,
 *     in the plan's storage dtype; scale/shift are float32 [cout].  Accumulation is float32.
 *   - Row ranges are half-open [lo, hi); the empty range is {0, 0}.
 *   - A plan may be used by one thread at a time.  Work is enqueued on the caller's stream and
 *     ordered after earlier and before later work on that stream; no function synchronises the
 *     device unless its comment says so.
 */
#ifndef LOP_H
#define LOP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    LOP_OK = 0,
    LOP_EINVAL = -1,        /* NULL pointer, index out of range, bad enum value                 */
    LOP_ESHAPE = -2,        /* layer list does not type-check (channels, empty output, ...)     */
    LOP_EUNSUPPORTED = -3,  /* valid request this build has no kernel for                        */
    LOP_ENOMEM = -4,        /* host allocation failed                                           */
    LOP_ECUDA = -5,         /* a CUDA call failed; lop_last_error() carries the CUDA string      */
    LOP_EWORKSPACE = -6,    /* caller-provided scratch is NULL or misaligned                    */
    LOP_EDEVICE = -7        /* a kernel reported a bounded wait that ran out (status word)      */
} lop_status;

enum { LOP_F32 = 0, LOP_BF16 = 1 };                         /* storage dtype                     */
enum { LOP_CONV2D = 0, LOP_MAXPOOL2D = 1, LOP_LINEAR = 2, LOP_DWCONV2D = 3, LOP_LAYERNORM = 4, LOP_CONCAT = 5 };
enum { LOP_ACT_NONE = 0, LOP_ACT_RELU = 1, LOP_ACT_SILU = 2, LOP_ACT_GELU = 3 };   /* GELU: t * Phi(t), erf form */
enum { LOP_RES_NONE = 0, LOP_RES_PRE_ACT = 1, LOP_RES_POST_ACT = 2 };
enum { LOP_INPUT = -1, LOP_NO_RESIDUAL = -2 };              /* special layer indices             */
enum {
    LOP_FLAG_REUSE_HALO = 1u,     /* bands run in ascending order and compute only rows no earlier
                                     band produced (Sec. IV-C, data dependency: rows that are already
                                     there are not moved again); otherwise every band recomputes its halo and is
                                     independent of the others (operation replication, Sec. IV-C) */
    LOP_FLAG_TIME_LAYERS = 2u,    /* record a CUDA event pair around every (band, layer) launch    */
    LOP_FLAG_FORCE_SIMT = 4u,     /* never use the tensor-core convolution (second on-GPU opinion) */
    LOP_FLAG_PER_LAYER = 8u,      /* one kernel launch per (band, layer) instead of one persistent
                                     wavefront launch per call / per band                          */
    LOP_FLAG_COPY_ENGINE = 16u,   /* pipelined runs always move the bands with copy-engine copies on
                                     a side stream, also when the kernel could fetch them itself  */
    LOP_FLAG_DEBUG_BOUNDS = 32u   /* checked execution: every layer runs as a kernel of its own (as with
                                     LOP_FLAG_PER_LAYER) and the CUDA-core kernels -- fp32 / fall-back convolution,
                                     pooling, patch gather, depth-wise convolution, layer normalisation,
                                     concatenation -- test every element offset they load from or store to
                                     against the tensor it belongs to and every output row against the rows of the
                                     launch.  A violation never traps: the access is skipped, bit 0x100 of the
                                     plan's status word is set and lop_plan_check_device returns LOP_EDEVICE.  The
                                     tensor-core kernel's operand loads are TMA copies, clipped by the hardware    */
};

/*
 * One local operator (Sec. IV-A).  Convolution:
 *   acc[n,oh,ow,co] = sum_{a,b,ci} x[n, oh*sh-ph+a*dh, ow*sw-pw+b*dw, ci] * weight[co,a,b,ci]
 *   t = scale[co]*acc + shift[co];  RES_PRE_ACT: t += r;  t = act(t);  RES_POST_ACT: t += r
 * with taps outside the input contributing zero.  Max pooling takes the maximum over the
 * in-bounds taps (padding never wins); cout must equal cin; act/residual are ignored.
 * LOP_LINEAR is the row-wise operator of Sec. IV-A (Eq. 1): Y = X * W^T with the parameter matrix shared by every
 * row; here every pixel's channel vector is a row of X, weight is [cout][cin], the epilogue is the convolution's,
 * and a band's rows depend on the same rows of the input and on nothing else.  Its window fields must be
 * kh = kw = sh = sw = dh = dw = 1, ph = pw = 0.
 * LOP_DWCONV2D is the depth-wise convolution (a block-wise operator, Sec. IV-A): channel c is filtered by its own
 * kernel,  acc[n,oh,ow,c] = sum_{a,b} x[n, oh*sh-ph+a*dh, ow*sw-pw+b*dw, c] * weight[c,a,b]  (weight [cout][kh][kw][1],
 * cout == cin), followed by the convolution's epilogue (scale, shift, residual, activation).
 * LOP_LAYERNORM normalises every pixel's channel vector (row-wise: a row depends on that row alone):
 *   y[c] = scale[c] * (x[c] - mean) / sqrt(var + 1e-6) + shift[c],  mean and biased variance over the cin channels,
 * scale / shift the learned gain and offset (NULL => 1 / 0); no window, no weight, act and residual ignored.
 * LOP_CONCAT joins two tensors of the same height and width along the channels: the main input's cin channels
 * first, then the cout - cin channels of the tensor residual_from names (residual_pos is ignored); no window, no
 * parameters.  A band's rows depend on the same rows of both inputs.
 * input_from / residual_from name an earlier layer of the same list, or LOP_INPUT for the
 * chain input; residual_from == LOP_NO_RESIDUAL means none.  The list order is topological.
 * The three pointers are DEVICE pointers; they are stored, never dereferenced on the host,
 * and may be NULL at planning time (set them later with lop_plan_set_params).
 */
typedef struct {
    int32_t op, cin, cout;
    int32_t kh, kw, sh, sw, ph, pw, dh, dw;
    int32_t act;
    int32_t input_from;
    int32_t residual_from, residual_pos;
    int32_t reserved;
    const void  *weight;   /* device, KRSC, storage dtype; NULL for pooling                       */
    const float *scale;    /* device, [cout]; NULL => 1                                           */
    const float *shift;    /* device, [cout]; NULL => 0                                           */
} lop_layer;

/*
 * What one band does at one layer.  [out_lo,out_hi): output rows of this layer the band
 * depends on; [in_lo,in_hi): rows of the layer's main input those outputs read (rows that
 * exist and are touched by a tap; the inverse of the paper's child(.) relation);
 * pad_top/pad_bot: how many rows above/below the input the taps reach; new_lo: first row of
 * [out_lo,out_hi) that no earlier band has produced (reuse-halo mode computes [new_lo,out_hi)).
 */
typedef struct {
    int32_t out_lo, out_hi, in_lo, in_hi, pad_top, pad_bot, new_lo, reserved;
} lop_range;

/* Times of the last lop_run_pipelined call, in milliseconds (see lop_plan_last_timing). */
typedef struct {
    float total_ms;        /* first enqueued operation to last, on the caller's stream            */
    float copy_ms;         /* sum of the band copies' own durations (copy-stream events); 0 unless
                              the plan has LOP_FLAG_TIME_LAYERS: timing events on the side stream
                              cost more than a small band's copy, so the fast path records none  */
    float first_copy_ms;   /* duration of band 0's copy (it can never be hidden); 0 likewise       */
    int32_t n_copies;
    int32_t reserved;
} lop_timing;

typedef struct lop_plan lop_plan_t;

/* ---- planning: HOST ONLY, needs no GPU, dereferences no device pointer -------------------
 * Validates the layer list, derives every layer's output shape (floor rounding), cuts the last
 * layer's output rows into n_bands bands  [floor(i*H/B), floor((i+1)*H/B))  (bands may be empty
 * when n_bands exceeds the row count) and back-propagates each band through every layer's
 * kernel, stride, padding and dilation (Sec. IV-A block-wise operators; dependency rule of
 * Sec. IV-B).  N,H,W,C: shape of the chain input.  On success *out owns the plan. */
int lop_plan(const lop_layer *layers, int n_layers, int N, int H, int W, int C, int dtype,
             int n_bands, unsigned flags, lop_plan_t **out);
void lop_plan_destroy(lop_plan_t *plan);                       /* NULL is accepted              */
int lop_plan_num_bands(const lop_plan_t *plan);                /* <0 on NULL                    */
int lop_plan_num_layers(const lop_plan_t *plan);
/* layer in [0, n_layers) or LOP_INPUT: for the chain input, out_* is the row range the band
 * needs, new_lo the first row not already transferred for an earlier band, in_* and pad_* 0. */
int lop_plan_get_range(const lop_plan_t *plan, int band, int layer, lop_range *out);
int lop_plan_out_shape(const lop_plan_t *plan, int layer, int *H, int *W, int *C);
/* Re-point a layer's device parameters (any may be NULL as in lop_layer). */
int lop_plan_set_params(lop_plan_t *plan, int layer, const void *weight, const float *scale,
                        const float *shift);
/* Device scratch, in bytes, that every lop_run_* call must be given (256-byte aligned):
 * full-size intermediate tensors, and for a thin (image) input the first layer's gathered
 * receptive patches and zero-padded weights, which the tensor-core kernel consumes. */
size_t lop_plan_workspace_bytes(const lop_plan_t *plan);
/* Size of the device-side input tensor N*H*W*C in storage dtype (staging for pipelined runs). */
size_t lop_plan_staging_bytes(const lop_plan_t *plan);
/* 2 * multiply-accumulates of the unpartitioned convolutions of the chain. */
double lop_plan_flops(const lop_plan_t *plan);

/* ---- execution: every pointer below is a DEVICE pointer unless it says otherwise ----------
 * in_dev and out_dev are FULL-SIZE tensors (chain input N*H*W*C, last layer's output); bands
 * address row ranges inside them.  stream is a cudaStream_t passed as void* (NULL = legacy
 * default stream).  The first execution call on a plan for a given (input, output, workspace)
 * triple creates the side stream, events and program tables (cudaMalloc + synchronous uploads):
 * make it outside any stream capture; later calls with the same buffers allocate nothing.
 * out_dev (the LAST plan's, for a chain) may also be page-locked host memory that the device can
 * address (cudaHostAlloc / cudaHostRegister): nothing reads the output tensor back, so the last
 * layer's kernels then store the result rows straight to host memory as they are finished --
 * the result's transfer overlaps the computation and no device-to-host copy is needed. */

/* Whole-tensor execution: every layer over all its rows (the unpartitioned reference order). */
int lop_run_whole(lop_plan_t *plan, const void *in_dev, void *out_dev, void *workspace, void *stream);
/* One band (Sec. IV-B: the band's operations at every layer, in dependency order).  Rows
 * [out_lo,out_hi) of the chain-input range must be present in in_dev; exactly the band's rows
 * of the last layer are written to out_dev.  Without LOP_FLAG_REUSE_HALO bands may run in any
 * order; with it, bands 0..band-1 must have run on the same workspace before. */
int lop_run_band(lop_plan_t *plan, int band, const void *in_dev, void *out_dev, void *workspace,
                 void *stream);
/* All bands in ascending order from a device-resident input (no transfers). */
int lop_run_banded(lop_plan_t *plan, const void *in_dev, void *out_dev, void *workspace, void *stream);
/* The transfer step of one band (the paper's transmission, Sec. IV-B): asynchronously copies
 * the chain-input rows the band needs and no earlier band has brought, for all N images, from
 * in_host_pinned (PINNED HOST, full-size tensor) to the same rows of staging_dev. */
int lop_copy_band(lop_plan_t *plan, int band, const void *in_host_pinned, void *staging_dev, void *stream);
/* Rows [row_lo, row_hi) of ONE layer: the operator-level step of the paper's runtime loop (Sec. IV-D, Alg. 1 / 2: for
 * each layer, compute its local operations, then send / receive rows along its edges).  One kernel launch of the
 * per-layer kernels; the layer's input (and residual) rows it reads must be present in the tensors the other calls
 * use (in_dev, the workspace, out_dev for the last layer).  The building block of the halo-exchange form of band
 * sharding, where neighbouring devices trade halo rows between layers instead of recomputing them. */
int lop_run_layer(lop_plan_t *plan, int layer, int row_lo, int row_hi, const void *in_dev, void *out_dev, void *workspace,
                  void *stream);
/* ---- band sharding over several devices (Sec. IV-C: operation replication) ---------------------
 * Bands that carry their halo are independent units: device `rank` of `world` takes the contiguous
 * block of bands  [floor(rank*B/world), floor((rank+1)*B/world)), runs it with lop_run_shard on its own
 * copy of the parameters, and the devices exchange the produced output rows once per plan (an
 * all-gather; the Python package's shard module does it with torch.distributed). */
/* HOST ONLY.  The block of bands of device `rank`, the rows [row_lo,row_hi) of the LAST layer's output
 * it produces and the rows [in_lo,in_hi) of the chain input it reads (empty ranges have lo == hi). */
int lop_plan_shard(const lop_plan_t *plan, int rank, int world, int *band_lo, int *band_hi, int *row_lo,
                   int *row_hi, int *in_lo, int *in_hi);
/* Runs bands [band_lo, band_hi) in ascending order as one unit.  Only rows [in_lo,in_hi) of in_dev need
 * to be present and only rows [row_lo,row_hi) of out_dev are written.  With LOP_FLAG_REUSE_HALO a
 * band computes what the BLOCK has not produced yet (no earlier band has run on this device, so the
 * block's first band computes its whole halo); the output rows are bit-identical to those of
 * lop_run_banded on one device. */
int lop_run_shard(lop_plan_t *plan, int band_lo, int band_hi, const void *in_dev, void *out_dev,
                  void *workspace, void *stream);
/* The same transfer step done by the persistent kernel's fetch warps instead of the copy engine (see lop_run_pipelined:
 * the "fetched" transport), by itself: band >= 0 brings that band's new rows, band == -1 every band's, from
 * in_host_pinned -- which must be mapped into the device's address space and agree with staging_dev modulo 16 bytes,
 * else LOP_EUNSUPPORTED -- to staging_dev.  One launch, no operator runs.  For timing the transmission a pipelined run
 * has to hide; workspace as for the lop_run_* calls. */
int lop_fetch_band(lop_plan_t *plan, int band, const void *in_host_pinned, void *staging_dev, void *workspace, void *stream);
/* Band pipeline (Sec. IV-B computation/transmission overlap): band i+1's rows come in while band i is
 * computed.  Two transports:
 *   - fetched (default when in_host_pinned is mapped into the device's address space, as cudaHostAlloc /
 *     cudaHostRegister memory is): the persistent kernel itself reads each band's rows from host memory
 *     and stores them to staging_dev -- fetch stages that precede the band's first operator in the
 *     dependency graph, spread over the SMs -- so the whole request is ONE launch on the caller's stream
 *     with no copy, event or flag command at all;
 *   - copy engine (LOP_FLAG_COPY_ENGINE, unmapped host memory, or plans the persistent kernel does not
 *     take): one asynchronous copy per band on the plan's side stream, forked and joined by CUDA events;
 *     a band's arrival is a 4-byte stream-ordered write behind its copy that the persistent kernel polls
 *     (per-layer launches wait on one event per band instead).
 * Both leave the input in staging_dev and give the same output bits.  Returns after enqueueing; the
 * host buffer must stay unchanged until the stream has passed the call.  staging_dev:
 * lop_plan_staging_bytes() bytes. */
int lop_run_pipelined(lop_plan_t *plan, const void *in_host_pinned, void *staging_dev, void *out_dev,
                      void *workspace, void *stream);
/* ---- several plans as one chain (Sec. III-A: later operators start as soon as the rows they
 * depend on exist) ---------------------------------------------------------------------------
 * A long network is planned in pieces (one plan per stage of the network, each with its own bands);
 * plan s+1 reads the full-size output tensor of plan s.  Run one after the other with the
 * functions above, each plan waits for the whole previous one.  These two functions run all plans
 * in ONE persistent launch with dependencies tracked per row group across plan boundaries, so a
 * band of plan s+1 starts as soon as the rows of plan s it reads are written.
 * plans[0..n_plans): HOST array; outs_dev[i], workspaces[i]: DEVICE, plan i's output tensor and
 * workspace (HOST arrays of pointers).  Requirements: every plan runs on the tensor-core kernels
 * (bf16, every convolution served by them), plan i+1's input shape equals plan i's output shape,
 * all plans agree in N, dtype and LOP_FLAG_REUSE_HALO; otherwise LOP_EUNSUPPORTED / LOP_ESHAPE is
 * returned before anything is enqueued and the caller runs the plans one by one.  The device status
 * word of the launch is plan 0's (lop_plan_check_device(plans[0], workspaces[0])). */
/* All bands of all plans from a device-resident input. */
int lop_run_chain_banded(lop_plan_t *const *plans, int n_plans, const void *in_dev, void *const *outs_dev,
                         void *const *workspaces, void *stream);
/* Band pipeline over the whole chain: plan 0's input bands stream from PINNED HOST memory as in
 * lop_run_pipelined while the rows already there flow through every plan. */
int lop_run_chain_pipelined(lop_plan_t *const *plans, int n_plans, const void *in_host_pinned, void *staging_dev,
                            void *const *outs_dev, void *const *workspaces, void *stream);

/* Event times of the last lop_run_pipelined call of a plan made with LOP_FLAG_TIME_LAYERS (other plans
 * record no events -- each would be one more command on the stream -- and get LOP_EINVAL).
 * SYNCHRONISES with that call's completion. */
int lop_plan_last_timing(lop_plan_t *plan, lop_timing *out);
/* With LOP_FLAG_TIME_LAYERS (implies per-layer launches): device time in ms of the (band, layer) launch of the last
 * lop_run_band / banded / pipelined call (band = -1: last lop_run_whole).  SYNCHRONISES.
 * *ms = 0 when that band had nothing to do at that layer. */
int lop_plan_layer_time(lop_plan_t *plan, int band, int layer, float *ms);
/* Which kernel family serves a layer: 0 = pooling, 1 = CUDA-core convolution,
 * 2 = tcgen05 tensor-core convolution.  <0 on error. */
int lop_plan_layer_kernel(const lop_plan_t *plan, int layer);
/* Where the full-size output tensor of an intermediate layer (0 <= layer < n_layers - 1) lives: byte offset into the
 * workspace given to the lop_run_* calls; its shape is lop_plan_out_shape(layer), NHWC in the storage dtype.  The rows a
 * call has computed are there when the call's stream work is done (for inspection and tests; the last layer's tensor is
 * the caller's out_dev). */
int lop_plan_layer_offset(const lop_plan_t *plan, int layer, size_t *offset);
/* 1 if executions of this plan write the layer's output tensor, 0 if they never do: the persistent kernel folds a 2x2
 * stride-2 max pooling that is a convolution's only reader into that convolution's epilogue (Sec. IV-A: both are local
 * operators), and only the pooled tensor exists.  <0 on error. */
int lop_plan_layer_stored(const lop_plan_t *plan, int layer);
/* Number of kernels (this library's own) and of async copies the last execution call enqueued. */
int lop_plan_last_launches(const lop_plan_t *plan);
int lop_plan_last_copies(const lop_plan_t *plan);
/* Reads the plan's device status word (0 = no kernel gave up on a bounded wait or failed a bounds check).  SYNCHRONISES
 * the stream of the last execution call.  On LOP_EDEVICE the outputs of that call are invalid; the
 * library drops its cached device tables and clears the word, so the plan can be used again.
 * lop_last_error() then shows the word; its bits name the role of the persistent kernel whose wait
 * ran out: 0x1 loader (ring slot), 0x2 MMA issuer (operands), 0x4 epilogue / pooling / gather
 * (accumulator, dependencies), 0x8 publisher, 0x10 loader (dependencies of a tile), 0x20 fetch warp
 * (window of the in-kernel input transfer).  0x100: a kernel of a LOP_FLAG_DEBUG_BOUNDS plan computed an
 * address outside its tensor (the access was skipped). */
int lop_plan_check_device(lop_plan_t *plan, void *workspace);

/* ---- the device-side waits and their failure path ----------------------------------------------
 * Every wait inside the persistent kernel (for a producer's rows, a band's arrival, a ring slot) is bounded: when it
 * runs out the kernel raises the plan's status word, tells every CTA to stop and returns; the outputs of that call are
 * invalid and lop_plan_check_device() reports LOP_EDEVICE and readies the plan for the next call.  The paper names the
 * failure of one unit as a risk of fine-grained partitioning (Sec. I) and answers it by tracking dependencies; this is
 * what happens here when a dependency is never satisfied.
 * lop_plan_set_wait_limit: polls (of some tens of nanoseconds each) a wait for rows or for an arrival may take; 0
 * restores the default (about four million).  Applies to the plan's later launches (for a chain: the first plan's). */
int lop_plan_set_wait_limit(lop_plan_t *plan, unsigned polls);
/* lop_run_pipelined with the copy-engine transport, except that band `band` never arrives: neither its copy nor its
 * arrival write is enqueued.  Exists to exercise the failure path above without faulting anything: the kernel's wait
 * for that band runs out after the plan's wait limit -- which must have been set, to at most 65536 polls, a few
 * milliseconds -- and the call's stream work ends normally with the status word raised (bit 0x10). */
int lop_run_pipelined_withheld(lop_plan_t *plan, int band, const void *in_host_pinned, void *staging_dev, void *out_dev,
                               void *workspace, void *stream);

/* ---- execution without any allocation --------------------------------------------------------
 * (The paper has no counterpart: this entry point exists for how the library is deployed.)
 * Some callers are not allowed to allocate: a plug-in running inside an application that forbids
 * cudaMalloc once it has started, a control loop that must never wait on the allocator, a process
 * whose device memory was handed out in full beforehand.  They cannot provide a workspace, and the
 * other lop_run_* functions would also create a stream, events and device tables on first use.
 *
 * lop_run_whole_static computes what lop_run_whole computes (every layer over all its rows, one
 * kernel launch per layer, the same kernels and therefore the same bits), but takes its scratch
 * -- status word, the first layer's gathered patches and padded weights, the tensors between layers --
 * from one array of LOP_STATIC_SCRATCH_BYTES bytes built into the library's device image.  It
 * calls no cudaMalloc / cudaFree / cudaHostAlloc, creates no stream or event and caches nothing;
 * the plan is only read.  in_dev, out_dev: DEVICE, full-size tensors as for lop_run_whole, owned
 * by the caller.  status_dev: DEVICE, 4 bytes, may be NULL; when given it is cleared at the start
 * of the call and afterwards holds 0, or a non-zero mask if a tensor-core kernel gave up on a
 * bounded wait (read it after synchronising the stream).  stream: cudaStream_t as void*.
 *
 * Limits and rules:
 *   - A plan with lop_plan_workspace_bytes() > LOP_STATIC_SCRATCH_BYTES is refused with
 *     LOP_EUNSUPPORTED before anything is enqueued (16 MiB holds e.g. a 224x224 image through two
 *     64-channel layers).  Every GPU on which the library is loaded holds the array until exit.
 *   - The first call on each device looks the array's device address up (with that device
 *     current); make that first call outside any stream capture.
 *   - All calls on a device share the array.  Each call rewrites what it needs, so calls one
 *     after the other on one stream are fine; calls whose kernels can overlap on the GPU (two
 *     streams, two threads) race on the array and give wrong results. */
#define LOP_STATIC_SCRATCH_BYTES (16u << 20)
int lop_run_whole_static(lop_plan_t *plan, const void *in_dev, void *out_dev, unsigned *status_dev,
                         void *stream);

const char *lop_strerror(int status);
const char *lop_last_error(void);       /* thread-local; valid until the next failing call */

#ifdef __cplusplus
}
#endif
#endif /* LOP_H */
