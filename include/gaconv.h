/*
 * gaconv -- filter-gradient (dW) convolution of a conv layer's backward pass on one NVIDIA B200
 * (sm_100a), exact and in the approximated forms of "Accelerated CNN Training Through Gradient
 * Approximation" (arXiv 1908.05460), Section 2.
 *
 * Notation.  X[n,c,h,w] input activations (paper: I), dY[n,k,p,q] output gradient (paper: dO),
 * dW[k,c,r,s] filter gradient (paper: df); paper symbols K = r = s, C_i = c, C_o = k (Section 2.4).
 *   P = (H + 2*pad_h - R)/stride_h + 1,  Q = (W + 2*pad_w - S)/stride_w + 1.
 *
 * Conventions of every entry point
 *   - Plain C ABI: status codes only, nothing throws, nothing aborts.
 *   - Every pointer named x, dy, dw, idx, sum, dy_sparse, workspace or *_dev is DEVICE memory on the
 *     current CUDA device, allocated and freed by the caller, 16-byte aligned.  Pointers named *_host
 *     are host memory (pinned for true asynchrony).  The library allocates no device memory and keeps
 *     no reference to any buffer after the call returns (the work itself is asynchronous, see below).
 *   - `stream` is a cudaStream_t passed as void*.  All work is enqueued on it; no entry point
 *     synchronises the host except gaconv_poll_async_status and gaconv_dw_from_host's final wait
 *     (gaconv_dw_from_host_async has none).
 *   - Validation errors are returned at once and enqueue nothing.
 *   - dw is overwritten (no accumulate-into).  It is always fp32.
 *   - Same inputs, descriptor and seed give bitwise identical outputs from run to run: every
 *     reduction has a fixed order.
 */
#ifndef GACONV_H
#define GACONV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    GACONV_OK = 0,
    GACONV_ERR_NULL_POINTER = 1,
    GACONV_ERR_BAD_DESC = 2,          /* non-positive size, P or Q < 1, unknown enum, wrong struct_size */
    GACONV_ERR_UNSUPPORTED = 3,       /* valid request this build has no kernel for                      */
    GACONV_ERR_MISALIGNED = 4,        /* a device pointer is not 16-byte aligned                          */
    GACONV_ERR_WORKSPACE_TOO_SMALL = 5,
    GACONV_ERR_CUDA = 6,              /* a CUDA runtime call failed; see cudaGetLastError                 */
    GACONV_ERR_TIMEOUT = 7            /* a bounded device-side wait gave up (read by the poll call)       */
} gaconv_status_t;

typedef enum { GACONV_F32 = 0, GACONV_BF16 = 1 } gaconv_dtype_t;            /* of x and dy            */
typedef enum { GACONV_X_NHWC = 0, GACONV_X_NCHW = 1 } gaconv_x_layout_t;    /* NHWC: Section 2.4; NCHW is transposed once
                                                                               into the workspace where a fast kernel applies */
typedef enum { GACONV_DY_NKPQ = 0, GACONV_DY_NPQK = 1 } gaconv_dy_layout_t;  /* NKPQ = N C_o H W (Section 2.4); NPQK (channels
                                                                               last) is transposed once into the workspace.
                                                                               The selection-only entry points take NKPQ only */
/* KRSC = C_o K K C_i (the layout of the paper's kernel, Section 2.4), KCRS = the frameworks' filter
 * layout, RSCK = K K C_i C_o (the order in which Section 2.4 first writes df) */
typedef enum { GACONV_DW_KRSC = 0, GACONV_DW_KCRS = 1, GACONV_DW_RSCK = 2 } gaconv_dw_layout_t;
typedef enum { GACONV_METHOD_EXACT = -1, GACONV_METHOD_ZERO = 0, GACONV_METHOD_RANDOM = 1,
               GACONV_METHOD_TOP1 = 2, GACONV_METHOD_TOPK = 3 } gaconv_method_t;
/* arithmetic of the exact contraction */
typedef enum {
    GACONV_MATH_DEFAULT = 0,   /* bf16 inputs: bf16 tensor cores, fp32 accumulate; fp32 inputs: fp32-accurate
                                  (three TF32 tensor-core passes on split operands, or the FP32 pipes)          */
    GACONV_MATH_TF32 = 1       /* fp32 inputs only: one TF32 tensor-core pass (operands cut to 10 mantissa bits);
                                  GACONV_ERR_UNSUPPORTED for shapes without a tensor-core kernel                 */
} gaconv_math_t;
/* kernel family; AUTO picks the fastest that supports the shape */
typedef enum { GACONV_ALGO_AUTO = 0, GACONV_ALGO_DIRECT = 1, GACONV_ALGO_TENSOR = 2 } gaconv_algo_t;

/* Problem statement of one layer (Section 2.4: the input activations I and the output gradient dO). */
typedef struct gaconv_conv_desc {
    uint32_t struct_size;              /* = sizeof(gaconv_conv_desc_t); versions the struct               */
    int32_t  n, c, h, w;               /* X is n x c x h x w                                              */
    int32_t  k, r, s;                  /* k filters of r x s (dilation 1, one group)                      */
    int32_t  stride_h, stride_w, pad_h, pad_w;
    int32_t  in_dtype;                 /* gaconv_dtype_t of x and dy                                      */
    int32_t  x_layout, dy_layout, dw_layout;
    int32_t  math;                     /* gaconv_math_t                                                   */
    int32_t  algo;                     /* gaconv_algo_t                                                   */
    int32_t  topk;                     /* GACONV_METHOD_TOPK: entries retained per map, 1..GACONV_MAX_TOPK (else ignored) */
    int32_t  sm_budget;                /* 0: size every launch for the whole GPU (lowest latency of a single layer);
                                          n > 0: size it for about n SMs, so that layers running next to one another
                                          (gaconv_schedule_run_step with several lanes) share the GPU instead of
                                          queueing for it.  Part of the problem statement: it changes how the
                                          reduction is split, hence the rounding, never the exact value             */
    float    alpha;                    /* dw = alpha * (...); 1 for parity, 1/128 in the paper's runs (Section 2.3) */
    float    rand_std;                 /* METHOD_RANDOM: standard deviation; the paper uses 1/128 (Section 2.2)     */
    void    *workspace;                /* device scratch prepared by gaconv_workspace_init                */
    size_t   workspace_bytes;
} gaconv_conv_desc_t;

#define GACONV_MAX_TOPK 16

const char *gaconv_status_string(gaconv_status_t status);

/* Number of kernels this library has enqueued since it was loaded (all threads).  Bookkeeping for
 * benchmarks; no counterpart in the paper. */
uint64_t gaconv_launch_count(void);

/* Device scratch one call needs for `method` (GACONV_METHOD_EXACT for the exact path) with this
 * descriptor (its workspace fields are ignored).  Never fails for a valid descriptor; *bytes > 0. */
gaconv_status_t gaconv_workspace_size(const gaconv_conv_desc_t *desc, int32_t method, size_t *bytes);

/* Prepare a workspace once after allocating it (zero-fills its control words).  Afterwards the
 * workspace may be reused by any number of calls that do not overlap on the GPU; each call leaves the
 * control words as it found them.  Two calls running concurrently must use two workspaces. */
gaconv_status_t gaconv_workspace_init(void *workspace, size_t bytes, void *stream);

/* Exact filter gradient (the operation marked in the paper's Figure 1; Section 2.4):
 *   dw[k,c,r,s] = alpha * sum_{n,p,q} Xz[n,c,p*stride_h+r-pad_h,q*stride_w+s-pad_w] * dy[n,k,p,q]
 * with Xz = x, zero outside the image; cross-correlation, no filter flip.
 * x: n*c*h*w elements of in_dtype in x_layout; dy: n*k*p*q elements in dy_layout; dw: k*c*r*s floats
 * in dw_layout (written).  Errors: NULL_POINTER, BAD_DESC, MISALIGNED, UNSUPPORTED,
 * WORKSPACE_TOO_SMALL, CUDA. */
gaconv_status_t gaconv_dw_exact(const void *x, const void *dy, float *dw,
                                const gaconv_conv_desc_t *desc, void *stream);

/* gaconv_dw_exact for callers that cannot allocate device memory (no counterpart in the paper).
 * Some callers cannot give the library a workspace because they may not call cudaMalloc where they
 * run: a host framework's plugin that is handed only its inputs and outputs, a loop that was promised
 * "no allocation after warm-up", a process whose device memory pool belongs to someone else.  This
 * variant computes exactly what gaconv_dw_exact computes, with the same kernels, but keeps the scratch
 * (split partial sums, control words) in a fixed array inside the library: gaconv_static_scratch_bytes()
 * bytes (8 MiB) that every GPU loading the library holds until the process exits.  desc->workspace and
 * desc->workspace_bytes are ignored.  The call allocates nothing (no cudaMalloc, cudaFree or
 * allocating library routine).
 *   - Limit: a problem whose gaconv_workspace_size(desc, GACONV_METHOD_EXACT) exceeds
 *     gaconv_static_scratch_bytes() is rejected with GACONV_ERR_WORKSPACE_TOO_SMALL and nothing is
 *     enqueued; use gaconv_dw_exact with a caller-owned workspace for those.
 *   - The first call on each device resolves the array's device address and clears its control words
 *     on `stream`; make that first call before any stream capture begins.
 *   - All calls on a device share the one array, which keeps the previous call's contents (each call
 *     overwrites what it later reads).  Calls that can overlap on the GPU (different streams without
 *     ordering between them) race on it: serialise them, or use gaconv_dw_exact with separate
 *     workspaces.
 * Other errors as gaconv_dw_exact. */
gaconv_status_t gaconv_dw_exact_static(const void *x, const void *dy, float *dw,
                                       const gaconv_conv_desc_t *desc, void *stream);
size_t gaconv_static_scratch_bytes(void);
/* gaconv_poll_async_status for the built-in array of gaconv_dw_exact_static on the current device (the
 * paper has no counterpart): waits for `stream`, then GACONV_ERR_TIMEOUT if a kernel launched through
 * gaconv_dw_exact_static gave up on a bounded wait since the last poll (clears the flag), else GACONV_OK.
 * Before the first gaconv_dw_exact_static call on the device it returns GACONV_OK.  Allocates nothing. */
gaconv_status_t gaconv_poll_async_status_static(void *stream);

/* Approximated filter gradient, Section 2:
 *   GACONV_METHOD_ZERO   (2.1)  dw = +0.
 *   GACONV_METHOD_RANDOM (2.2)  dw[i] = rand_std * z_i, z_i independent standard normals drawn from
 *        Philox-4x32-10 keyed by `seed` (counter j gives elements 4j..4j+3 by Box-Muller; i runs over
 *        the logical [k][c][r][s] order whatever dw_layout is).  Pass a new seed per layer and batch:
 *        the paper regenerates the values every batch.  x and dy may be NULL.
 *   GACONV_METHOD_TOP1   (2.3, Algorithm 1)  for every (n,k): keep only the largest-magnitude entry of
 *        dy[n,k,:,:] (lowest p*Q+q among equals), replace it by the signed sum of the map, and take
 *        the exact filter gradient of that sparse tensor.
 *   GACONV_METHOD_TOPK   (2.3 notes that more than one entry per map may be kept, i.e. the k largest magnitudes, with an
 *        adjusted scale that the paper leaves open)  keep the desc->topk largest-magnitude entries of every
 *        map (equal magnitudes: lower p*Q+q first), give each of them sum/topk, and take the exact filter
 *        gradient of that sparse tensor.  topk = 1 is TOP1; topk is clamped to P*Q.
 * `seed` is ignored by ZERO, TOP1 and TOPK. */
gaconv_status_t gaconv_dw_approx(int32_t method, const void *x, const void *dy, float *dw,
                                 const gaconv_conv_desc_t *desc, uint64_t seed, void *stream);

/* Selection step of Algorithm 1 alone (its arg-max-of-magnitude and sum statements), for inspection:
 *   idx[n*K+k] = p*Q+q of the retained entry, sum[n*K+k] = signed sum of dy[n,k,:,:] (fp32).
 * dy_sparse (may be NULL) receives the dense sparse tensor in dy's dtype and layout: the sum, rounded
 * to in_dtype, at the retained position and zero elsewhere.  Needs no workspace. */
gaconv_status_t gaconv_approx_select(const void *dy, int32_t *idx, float *sum, void *dy_sparse,
                                     const gaconv_conv_desc_t *desc, void *stream);

/* Selection step of the top-k variant, for inspection: idx[(n*K+k)*t + i] = position of the i-th retained
 * entry of dy[n,k,:,:] in order of selection (t = min(desc->topk, P*Q)), sum[n*K+k] = signed sum of the map. */
gaconv_status_t gaconv_approx_select_topk(const void *dy, int32_t *idx, float *sum,
                                          const gaconv_conv_desc_t *desc, void *stream);

/* Same operation as gaconv_dw_exact / gaconv_dw_approx (method as above, GACONV_METHOD_EXACT for
 * exact) with HOST inputs and output: copies x_host and dy_host into the caller's device staging
 * buffers x_dev and dy_dev, runs, copies dw_dev back into dw_host, and waits for the stream.  The
 * host-to-device and device-to-host transfers are part of the call.  The paper's operator has the
 * same shape: activations and gradients in, filter gradient out (Section 2.4).  x_host and dy_host may
 * both be NULL: x_dev and dy_dev are then used as they are (a step that takes several gradients of one
 * layer -- say the exact one and an approximation -- copies the layer's inputs once). */
gaconv_status_t gaconv_dw_from_host(int32_t method, const void *x_host, const void *dy_host, float *dw_host,
                                    void *x_dev, void *dy_dev, float *dw_dev,
                                    const gaconv_conv_desc_t *desc, uint64_t seed, void *stream);

/* The same without the final wait: the three transfers and the kernels are enqueued on `stream` and the call
 * returns; dw_host holds the result once the caller has synchronised with the stream.  Layers enqueued on different
 * streams overlap their transfers in the two directions of the host link. */
gaconv_status_t gaconv_dw_from_host_async(int32_t method, const void *x_host, const void *dy_host, float *dw_host,
                                    void *x_dev, void *dy_dev, float *dw_dev,
                                    const gaconv_conv_desc_t *desc, uint64_t seed, void *stream);

/* Waits for `stream`, then reports GACONV_ERR_TIMEOUT if a kernel that used desc->workspace gave up
 * on a bounded wait since the last poll (and clears the flag), GACONV_OK otherwise. */
gaconv_status_t gaconv_poll_async_status(const gaconv_conv_desc_t *desc, void *stream);

/* ---- approximation schedules (Section 2.5): which method each layer uses at each training batch ---- */
typedef struct gaconv_schedule gaconv_schedule_t;   /* host object, owned by the caller via create/destroy */
typedef enum {
    GACONV_SCHED_EVERY_4TH_LAYER = 0,            /* Section 3: every 4th conv from the 2nd, every batch      */
    GACONV_SCHED_ALT_LAYER_ALT_BATCH = 1,        /* Section 3.4 schedule 2: even layers on odd steps         */
    GACONV_SCHED_ALL_LAYERS_EVERY_4TH_BATCH = 2, /* Section 3.4 schedule 3: all layers when step % 4 == 3    */
    GACONV_SCHED_LAYER2_ALT_BATCH = 3,           /* Section 3, two-layer CNN: conv 2 on odd steps            */
    GACONV_SCHED_SEEDED_FRACTION_ALT_BATCH = 4   /* round(fraction*L) layers with the lowest
                                                    splitmix64(seed+layer), approximated on odd steps       */
} gaconv_sched_kind_t;

gaconv_status_t gaconv_schedule_create(gaconv_schedule_t **out, int32_t num_layers, int32_t kind,
                                       int32_t method, double fraction, uint64_t seed);
/* Method of `layer` (0-based) at training step `step` (0-based): GACONV_METHOD_EXACT or the
 * schedule's approximation method; -2 on bad arguments. */
int32_t gaconv_schedule_method(const gaconv_schedule_t *sched, int32_t layer, int64_t step);
/* Decide and dispatch one layer of one step: gaconv_dw_exact or gaconv_dw_approx(method) on `stream`;
 * the random method is seeded with a mix of (schedule seed, step, layer) so values change every batch. */
gaconv_status_t gaconv_schedule_run_layer(const gaconv_schedule_t *sched, int32_t layer, int64_t step,
                                          const void *x, const void *dy, float *dw,
                                          const gaconv_conv_desc_t *desc, void *stream);
/* One training step (Sections 2.5 and 3: at every batch the schedule picks, layer by layer, the exact or an
 * approximated filter gradient): gaconv_schedule_run_layer for layers 0..num_layers-1, layer l on lane
 * l % lanes.  Lane 0 is `stream`; the other lanes are streams the library owns (created on first use, one set
 * per device), forked from `stream` when the call starts and joined back into it before it returns, so for the
 * caller the whole step is ordered like one operation on `stream` -- also inside a stream capture.  Layers of
 * different lanes overlap on the GPU, which hides the start-up and reduction latency of small layers; every
 * layer's result is bit for bit that of gaconv_schedule_run_layer with the same descriptor.  lanes in 1..16; with lanes > 1 the
 * descriptors must carry distinct workspaces (GACONV_ERR_BAD_DESC otherwise).  x, dy, dw, descs: host arrays
 * of num_layers device pointers / descriptor pointers.  Calls on one device share the lanes: enqueueing from
 * several host threads is serialised. */
gaconv_status_t gaconv_schedule_run_step(const gaconv_schedule_t *sched, int64_t step, int32_t num_layers,
                                         const void *const *x, const void *const *dy, float *const *dw,
                                         const gaconv_conv_desc_t *const *descs, int32_t lanes, void *stream);
void gaconv_schedule_destroy(gaconv_schedule_t *sched);

#ifdef __cplusplus
}
#endif
#endif /* GACONV_H */
