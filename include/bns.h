/*
 * bns.h - C ABI of the Batch Normalization Sampling library for NVIDIA B200 (sm_100a).
 *
 * One BN layer over a dense NCHW activation tensor whose per-channel mean and variance are
 * estimated from a sampled subset S of the activations (arXiv 1810.10962, "Batch Normalization
 * Sampling"), while normalise+affine and its gradient still cover the whole tensor.
 *
 * Conventions that hold for every entry point
 *  - DEVICE pointers unless a comment says HOST.  The caller owns every buffer; the library
 *    allocates no memory, keeps no state between calls (except the optional profiling hooks at
 *    the end of this file) and never synchronises the host: all work is enqueued on `cuda_stream`
 *    (a cudaStream_t passed as void*; NULL is the default stream).
 *  - x, y, dy, dx share one shape and element type (`bns_shape`), are dense NCHW and 16-byte
 *    aligned.  gamma, beta, mean, invstd, dgamma, dbeta are float[C].  Statistics and parameter
 *    gradients are always fp32; bf16 tensors are rounded to nearest-even on store.
 *  - Outputs must not alias inputs.
 *  - Arguments are validated on the host before anything is launched; a negative status means
 *    that nothing was enqueued.  No exception crosses this boundary.
 *  - Results are a deterministic function of the inputs: no floating-point atomics are used and
 *    every cross-block combine runs in a fixed order, so two runs give identical bits.
 *  - `workspace` is scratch of at least bns_workspace_bytes() bytes, 256-byte aligned; its contents
 *    need no initialisation.  Calls that overlap in time on the GPU need distinct workspaces.
 */
#ifndef BNS_H
#define BNS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    BNS_OK = 0,
    BNS_ERR_NULL = -1,       /* a required pointer is NULL                                   */
    BNS_ERR_SHAPE = -2,      /* non-positive or overflowing dimension, eps <= 0              */
    BNS_ERR_RULE = -3,       /* unknown rule / offset mode, or a rule field out of range     */
    BNS_ERR_INDEX = -4,      /* sample index or patch offset outside the tensor, or repeated */
    BNS_ERR_DTYPE = -5,      /* unknown element type                                         */
    BNS_ERR_ALIGN = -6,      /* a tensor pointer is not 16-byte aligned                      */
    BNS_ERR_WORKSPACE = -7,  /* workspace NULL, misaligned or too small                      */
    BNS_ERR_CUDA = -8        /* a CUDA runtime call failed (launch, copy)                    */
} bns_status;

typedef enum { BNS_F32 = 0, BNS_BF16 = 1 } bns_dtype;

/* How the sampled set S is chosen (Sec. 4.1, Sec. 4.2 and Algorithms 1-3 of the paper). */
typedef enum {
    BNS_RULE_FULL = 0,     /* S = every element: ordinary BN (Eq. 2)                            */
    BNS_RULE_BATCH = 1,    /* Batch Sampling: all elements of k chosen samples (Algorithm 1);   */
                           /* Naive Sampling is the same rule with indices 0..k-1               */
    BNS_RULE_FEATURE = 2,  /* Feature Sampling: one ph x pw patch of every feature map (Alg. 2) */
    BNS_RULE_VIRTUAL = 3   /* Virtual Dataset Normalization: statistics from nv virtual samples */
                           /* only (Algorithm 3); they are passed as a separate tensor xv       */
} bns_rule;

typedef enum {
    BNS_OFF_SHARED = 0,      /* one (oh,ow) for the whole layer: the paper's rule (Sec. 4.1)  */
    BNS_OFF_PER_SAMPLE = 1,  /* one (oh,ow) per sample n                                      */
    BNS_OFF_PER_MAP = 2      /* one (oh,ow) per feature map (n,c), index n*C + c              */
} bns_offset_mode;

typedef struct {
    int rule;                   /* bns_rule                                                       */
    /* BATCH */
    int k;                      /* number of sampled samples, 1..N                                */
    const int32_t* sample_idx;  /* HOST, k distinct values in [0,N), any order; copied during the */
                                /* call, so it may be reused as soon as the call returns.  A list */
                                /* begin..begin+k-1 (the paper's rule) needs no copy; any other   */
                                /* list is sent with cudaMemcpyAsync, so pin it if the stream is  */
                                /* being captured into a graph                                    */
    /* FEATURE */
    int ph, pw;                 /* patch size, 1..H and 1..W                                      */
    int offset_mode;            /* bns_offset_mode                                                */
    const int32_t* offsets;     /* (oh,ow) int32 pairs, oh in [0,H-ph], ow in [0,W-pw]:           */
                                /* SHARED: HOST, 1 pair (validated on the host);                  */
                                /* PER_SAMPLE: DEVICE, N pairs; PER_MAP: DEVICE, N*C pairs - the  */
                                /* caller guarantees that many: the kernels index the array by    */
                                /* sample (and channel) and cannot check its length.              */
                                /* Device-resident pairs are checked by the kernels: a pair out   */
                                /* of range is clamped into range and BNS_FLAG_BAD_OFFSET is set  */
                                /* in the workspace status word (see bns_workspace_status)        */
    /* VIRTUAL */
    int nv;                     /* number of virtual samples, >= 1                                */
    int xv_dtype;               /* bns_dtype of xv, yv, dyv, dxv                                  */
    const void* xv;             /* [nv,C,H,W], 16-byte aligned                                    */
    void* yv;                   /* forward: normalised virtual samples, may be NULL               */
    const void* dyv;            /* backward: gradient reaching yv, may be NULL (treated as zeros) */
    void* dxv;                  /* backward: gradient of xv, may be NULL                          */
} bns_sampling;

typedef struct {
    int N, C, H, W;
    int dtype;                  /* bns_dtype of x, y, dy, dx */
} bns_shape;

/* Scratch size that serves bns_forward, bns_backward and bns_full_bn for this shape and rule.
 * Returns 0 if the arguments are invalid. */
size_t bns_workspace_bytes(const bns_shape* shape, const bns_sampling* sampling);

/*
 * Forward (Eq. 1 with the sampled statistics of Eq. 3).
 *   mean_c   = (1/s) sum_{i in S_c} x_i
 *   var_c    = (1/s) sum_{i in S_c} (x_i - mean_c)^2            (biased)
 *   invstd_c = 1 / sqrt(var_c + eps)
 *   y_i      = gamma_c (x_i - mean_c) invstd_c + beta_c          for EVERY element of x
 * VIRTUAL: S_c is all of xv[:,c,:,:]; yv (if not NULL) receives the same map applied to xv.
 * Writes y, mean[C], invstd[C] (the statistics that the backward call needs).
 */
bns_status bns_forward(const bns_shape* shape, const void* x, const float* gamma, const float* beta,
                       float eps, const bns_sampling* sampling, void* y, float* mean, float* invstd,
                       void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Backward (Eq. 5 with the modification of Eq. 6).  mean and invstd are the forward's outputs.
 *   dbeta_c  = sum_i dy_i                      dgamma_c = sum_i dy_i xhat_i
 * where both sums run over every element that was normalised with these statistics (all
 * N*H*W real points, plus the virtual rows when dyv is given) - they keep their full length
 * (Appendix C.1, "Speedup in the Backward Pass"), and
 *   dx_i = gamma_c invstd_c ( dy_i - [i in S_c] (dbeta_c + xhat_i dgamma_c) / s )
 * which is Eq. 6 with dl/dE and dl/dVar of Eq. 5 substituted.  VIRTUAL: no real element is in S;
 * dxv (if not NULL) gets the upper branch for every virtual element.  rule FULL gives the
 * ordinary BN backward.
 */
bns_status bns_backward(const bns_shape* shape, const void* x, const void* dy, const float* gamma,
                        const float* mean, const float* invstd, const bns_sampling* sampling,
                        void* dx, float* dgamma, float* dbeta,
                        void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Ordinary BN forward (Eq. 1 with Eq. 2): the in-library comparison.  Same as bns_forward with
 * rule FULL; its backward is bns_backward with rule FULL. */
bns_status bns_full_bn(const bns_shape* shape, const void* x, const float* gamma, const float* beta,
                       float eps, void* y, float* mean, float* invstd,
                       void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Virtual Dataset Normalization combined with a sampling rule (Eq. 4 of the paper, its most accurate
 * variant, "FS+VDN"):   X = mix X[x_v] + (1 - mix) X[x_s]   for X in {E, Var},
 * where x_s is the sampled set of the real batch (`sampling->rule` BATCH or FEATURE) and x_v the nv
 * virtual samples `sampling->xv` (the VIRTUAL fields of bns_sampling are used as well); each variance
 * is taken about its own mean (Eq. 3 on each set).  The paper uses mix = 0.5.  x and, if yv is given,
 * xv are normalised with the mixed statistics (Eq. 1).
 * Forward writes y, mean[C] and invstd[C] (mixed) and the two means mean_s[C], mean_v[C], which the
 * backward needs.  The paper derives no gradient for Eq. 4; by the chain rule through it,
 *   dx_i  = gamma invstd dy_i   - [i in S] (1-mix) gamma invstd (dbeta + invstd (x_i - mean_s) dgamma) / s_s
 *   dxv_i = gamma invstd dyv_i  -             mix  gamma invstd (dbeta + invstd (xv_i - mean_v) dgamma) / s_v
 * with dbeta, dgamma the full-length sums of Eq. 5 over the real batch and (if dyv is given) the
 * virtual rows.  Workspace: bns_workspace_bytes_mixed().  mix must lie in [0,1].
 */
size_t bns_workspace_bytes_mixed(const bns_shape* shape, const bns_sampling* sampling);
bns_status bns_forward_mixed(const bns_shape* shape, const void* x, const float* gamma, const float* beta,
                             float eps, float mix, const bns_sampling* sampling, void* y, float* mean,
                             float* invstd, float* mean_s, float* mean_v,
                             void* workspace, size_t workspace_bytes, void* cuda_stream);
bns_status bns_backward_mixed(const bns_shape* shape, const void* x, const void* dy, const float* gamma,
                              const float* mean, const float* invstd, const float* mean_s, const float* mean_v,
                              float mix, const bns_sampling* sampling, void* dx, float* dgamma, float* dbeta,
                              void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Moving average of the statistics for validation (Appendix D, Eq. 8):
 *   X_ma = X at the first iteration,  alpha X + (1 - alpha) X_ma afterwards,  X in {E, Var}
 * (alpha weights the NEW value, as Eq. 8 and Eq. 9 state it; the paper finds 0.7 best for
 * BS-1/128).  mean and invstd are a forward call's outputs; Var is recovered as 1/invstd^2 - eps.
 * mean_ma[C], var_ma[C] are updated in place (read only when first_iteration == 0).
 */
bns_status bns_update_moving_average(int C, const float* mean, const float* invstd, float eps, float alpha,
                                     int first_iteration, float* mean_ma, float* var_ma, void* cuda_stream);

/*
 * bns_forward with the moving-average update of Eq. 8 done inside it: the thread that finishes a channel's
 * sampled statistics also updates mean_ma[c] and var_ma[c] (Var taken directly as the biased variance of
 * the sampled set, not recovered from invstd), so a training step needs no separate C-length launch.
 * Same arguments, outputs and workspace as bns_forward, plus alpha, first_iteration, mean_ma, var_ma as
 * in bns_update_moving_average.
 */
bns_status bns_forward_training(const bns_shape* shape, const void* x, const float* gamma, const float* beta,
                                float eps, const bns_sampling* sampling, float alpha, int first_iteration,
                                float* mean_ma, float* var_ma, void* y, float* mean, float* invstd,
                                void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Validation-time forward (Appendix D): Eq. 1 with E and Var replaced by the recorded moving
 * averages, y = gamma (x - mean_ma) / sqrt(var_ma + eps) + beta.  Workspace as for bns_full_bn.
 */
bns_status bns_inference_forward(const bns_shape* shape, const void* x, const float* gamma, const float* beta,
                                 float eps, const float* mean_ma, const float* var_ma, void* y,
                                 void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Statistics shared by several GPUs (Sec. 4.3 "Micro-BN": Sync-BN with Feature or Batch Sampling).
 * Each rank holds its own slice of the batch; the sampled statistics are those of the union of the
 * ranks' sampled sets, so the result equals one big batch normalised with Eq. 1/3 and Eq. 5/6.  The
 * exchange itself (an all-gather of 3C floats forward, an all-reduce of 2C floats backward) is the
 * caller's, e.g. NCCL through torch.distributed; these calls are the per-rank pieces around it:
 *
 *   bns_sync_local_moments   this rank's sampled set -> moments[3][C] = (count, mean, M2) rows
 *   (all-gather the 3C floats of every rank into [ranks][3][C])
 *   bns_sync_merge_moments   merges the ranks' rows in rank order (same bits on every rank) -> mean, invstd
 *                            and, if count is not NULL, count[C] = sampled points per channel over all ranks
 *   bns_sync_normalize       Eq. 1 on this rank's x with the shared statistics
 *   bns_sync_backward_sums   sums[2][C] = (sum dy, sum dy xhat) over this rank's elements, and
 *                            dx = gamma invstd dy for every element (lower branch of Eq. 6);
 *                            the two rows are also this rank's share of dbeta and dgamma
 *   (all-reduce the 2C floats)
 *   bns_sync_backward_apply  upper branch of Eq. 6 on this rank's sampled elements with the summed
 *                            rows and the merged count (DEVICE float[C]: the count never visits the host)
 *
 * The three variants of the paper's list are all expressible: (1) every rank samples its slice by the
 * same rule (FULL, BATCH or FEATURE); (2) only a fraction of the ranks contributes statistics - the
 * others pass sampling = NULL to _local_moments (a count of zero, which the merge passes over) and to
 * _backward_apply (nothing to correct); (3) the virtual samples are fed to one rank - that rank passes
 * a VIRTUAL rule (xv, optionally dyv / dxv) to _local_moments, to _backward_sums as `virtual_rows` (their
 * gradient joins its sums when dyv is given) and to _backward_apply (which writes dxv), the others NULL.
 * Workspace as for bns_forward with the same shape and rule (FULL where sampling is NULL).
 */
bns_status bns_sync_local_moments(const bns_shape* shape, const void* x, const bns_sampling* sampling, float eps,
                                  float* moments, void* workspace, size_t workspace_bytes, void* cuda_stream);
bns_status bns_sync_merge_moments(int C, int ranks, const float* moments, float eps, float* mean, float* invstd,
                                  float* count, void* cuda_stream);
bns_status bns_sync_normalize(const bns_shape* shape, const void* x, const float* gamma, const float* beta,
                              const float* mean, const float* invstd, void* y, void* cuda_stream);
bns_status bns_sync_backward_sums(const bns_shape* shape, const void* x, const void* dy, const float* gamma,
                                  const float* mean, const float* invstd, const bns_sampling* virtual_rows,
                                  void* dx, float* sums, void* workspace, size_t workspace_bytes, void* cuda_stream);
bns_status bns_sync_backward_apply(const bns_shape* shape, const void* x, const void* dy, const float* gamma,
                                   const float* mean, const float* invstd, const bns_sampling* sampling,
                                   const float* sums, const float* count, void* dx,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * BN with sampled statistics followed by a residual add and a ReLU, fused:
 *   forward   y = max(0, gamma xhat + beta + residual)
 *   backward  g = dy where gamma xhat + beta + residual > 0, else 0;  dresidual = g;  then bns_backward
 *             with g in place of dy (sums, dx, statistics terms on S).
 * This is not an equation of the paper: it is the step that follows every BN layer of the residual
 * networks it trains (Table 1); fusing it saves writing and re-reading the pre-activation tensor.  The
 * mask is recomputed from x and residual, nothing is stored for it, so the backward call needs beta and
 * the same residual.  residual and dresidual may be NULL (plain BN + ReLU; dresidual may also be NULL
 * when only dx is wanted).  rule FULL, BATCH or FEATURE; workspace as for bns_forward.
 */
bns_status bns_forward_relu(const bns_shape* shape, const void* x, const void* residual, const float* gamma,
                            const float* beta, float eps, const bns_sampling* sampling, void* y, float* mean,
                            float* invstd, void* workspace, size_t workspace_bytes, void* cuda_stream);
bns_status bns_backward_relu(const bns_shape* shape, const void* x, const void* residual, const void* dy,
                             const float* gamma, const float* beta, const float* mean, const float* invstd,
                             const bns_sampling* sampling, void* dx, void* dresidual, float* dgamma, float* dbeta,
                             void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Channels-last tensors: x, y, dy, dx (and xv, yv, dyv, dxv) are dense [N,H,W,C] - the layout the paper
 * itself works in (Appendix A: statistics reduce dims 0,1,2 of B in R^{N x H x W x C}).  Same
 * arithmetic, arguments and results as bns_forward / bns_backward; `shape` still names N, C, H, W.
 * All rules are supported; Feature Sampling takes a shared or per-sample patch location (a per-map
 * location would give every channel of a pixel a different patch: BNS_ERR_RULE).  A sampled pixel is a
 * contiguous vector of C channels in this layout, so the patch passes read whole cache lines.
 * Workspace: bns_workspace_bytes_nhwc().
 */
size_t bns_workspace_bytes_nhwc(const bns_shape* shape, const bns_sampling* sampling);
bns_status bns_forward_nhwc(const bns_shape* shape, const void* x, const float* gamma, const float* beta,
                            float eps, const bns_sampling* sampling, void* y, float* mean, float* invstd,
                            void* workspace, size_t workspace_bytes, void* cuda_stream);
bns_status bns_backward_nhwc(const bns_shape* shape, const void* x, const void* dy, const float* gamma,
                             const float* mean, const float* invstd, const bns_sampling* sampling,
                             void* dx, float* dgamma, float* dbeta,
                             void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * bns_forward for callers that cannot provide scratch memory.  (The paper has no counterpart; this
 * is a packaging variant of bns_forward: same kernels, same results.)
 *
 * Some hosts of this library are not allowed to allocate on the device: a plug-in inside an
 * inference server or framework that has handed all device memory to its own pool, code that runs
 * where cudaMalloc is forbidden because it synchronises the whole device under other tenants'
 * streams, or a component that ships with a fixed memory map.  Such a caller has its input and
 * output tensors (the host application gave them to it) but no workspace.  This entry point uses
 * scratch that is built into the library image instead: a 4 MiB array in device memory
 * (bns_static_workspace_bytes()), which every GPU that loads the library holds until the process
 * exits.  It calls no cudaMalloc/cudaFree and no allocating routine of any library.
 *
 *  - Arguments and results are those of bns_forward, minus the workspace pair.
 *  - A shape/rule whose bns_workspace_bytes() exceeds bns_static_workspace_bytes() is rejected with
 *    BNS_ERR_WORKSPACE before anything is launched (the ResNet-50 layers at N=256 need up to 2.6 MB).
 *  - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 *    that device current) and keeps it for the life of the process (the device's primary context is
 *    assumed to live that long; after a cudaDeviceReset the kept address is stale).  Host threads may
 *    make that first call at the same time.  Make it before any stream capture begins.
 *  - All calls on a device share the one array, which keeps whatever the previous call left in it.
 *    Nothing in it needs to start at zero (the status word is cleared by the call when it is used),
 *    but two calls that overlap in time on the same GPU - different streams, or different host
 *    threads - would overwrite each other's partial sums: run them one after the other.
 *  - bns_workspace_status() cannot read this scratch: device-resident patch offsets are still
 *    clamped into range, but the flag is not retrievable through this entry point.
 */
size_t bns_static_workspace_bytes(void);
bns_status bns_forward_static(const bns_shape* shape, const void* x, const float* gamma, const float* beta,
                              float eps, const bns_sampling* sampling, void* y, float* mean, float* invstd,
                              void* cuda_stream);

/*
 * Forward and backward of one layer with HOST buffers for the large tensors: copies x and dy to
 * the device, runs bns_forward and bns_backward, copies y, dx, mean, invstd, dgamma, dbeta back.
 * x, dy, y, dx, gamma, beta and the six outputs are HOST pointers (pinned memory lets the copies
 * run asynchronously); pointers inside `sampling` keep the meaning documented above.
 * `arena` is DEVICE scratch of at least bns_host_arena_bytes() bytes, 256-byte aligned.
 * Everything is enqueued on `cuda_stream`; downloads run on a helper stream of the library so that
 * the two directions of the link work at once, and the helper joins `cuda_stream` again before the call
 * returns its last copies; synchronise `cuda_stream` before reading the outputs.  With Batch Sampling
 * over a contiguous range or Feature Sampling at a shared location, and N >= 32, the call is pipelined
 * by row chunks: the sampled set goes up first, then chunks of x go up while normalised chunks of y come
 * down, chunks of dy go up while chunks of dx come down, and the sampled elements of dx are sent again
 * after their statistics terms are in (one cudaMemcpyAsync or cudaMemcpy3DAsync per piece; 20.0 ms
 * instead of 23.3 ms per step of the default benchmark, the floor being 15.6 ms of link time).  Other
 * rules copy tensor by tensor (y down while dy goes up).  The helper stream and a few events are created
 * on the first call on a device and kept: the one exception to "keeps no state".
 * The paper has no counterpart (its measurements include input pipelines only as a whole).
 */
size_t bns_host_arena_bytes(const bns_shape* shape, const bns_sampling* sampling);
bns_status bns_forward_backward_host(const bns_shape* shape, const void* x, const void* dy,
                                     const float* gamma, const float* beta, float eps,
                                     const bns_sampling* sampling, void* y, void* dx, float* mean,
                                     float* invstd, float* dgamma, float* dbeta,
                                     void* arena, size_t arena_bytes, void* cuda_stream);

/* Test aid for the selection rule (Algorithms 1-3): writes 1 where the real element is in S and 0
 * elsewhere; mask is uint8 [N,C,H,W] (all zeros for VIRTUAL).  Needs the same workspace. */
bns_status bns_debug_selection_mask(const bns_shape* shape, const bns_sampling* sampling, uint8_t* mask,
                                    void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Status word that kernels set in a workspace: synchronises the stream and copies it to *flags
 * (HOST).  Every forward/backward/mask call clears the word first. */
#define BNS_FLAG_BAD_OFFSET 1u /* a device-resident patch offset was outside [0,H-ph] x [0,W-pw] */
bns_status bns_workspace_status(const void* workspace, uint32_t* flags, void* cuda_stream);

/*
 * The one-launch path.  A layer whose per-channel data (N*H*W elements, twice that in the backward),
 * split over the up to 8 blocks of a thread-block cluster, fits their shared memory runs its whole
 * forward, and its whole backward, as one kernel each: the tensor is read from HBM once and written
 * once, the sampled statistics (Eq. 3) and the sums of Eq. 5 are taken from the on-chip copy and
 * combined across the cluster in a fixed order.  bns_forward, bns_backward and bns_full_bn choose it
 * by themselves; results obey the same definition and tolerances as the streaming path.
 * bns_slab_plan reports the choice for a shape and rule: returns 1 and fills plan[0..5] = channels
 * per cluster, blocks per cluster, samples per block, shared-memory bytes per block, blocks per
 * launch, row lanes - or returns 0 when the streaming path is used.  (HOST pointer.)
 * Those kernels wait for their bulk copies with a bounded number of polls; bns_wait_timeouts
 * synchronises the stream and returns in *count (HOST) how many such waits have run out on the
 * current device since the library was loaded.  Anything but 0 means results were computed from
 * incomplete data.
 */
int bns_slab_plan(const bns_shape* shape, const bns_sampling* sampling, int backward, int32_t* plan);
bns_status bns_wait_timeouts(uint32_t* count, void* cuda_stream);

const char* bns_status_string(bns_status status);

/* ---- measurement hooks (process-wide, not thread-safe; off by default) ---------------------- */
typedef enum {
    BNS_KERNEL_COL_MOMENTS = 0,   /* statistics over whole samples (FULL, BATCH, VIRTUAL)       */
    BNS_KERNEL_PATCH_MOMENTS = 1, /* statistics over patches (FEATURE)                          */
    BNS_KERNEL_FINALIZE_STATS = 2,
    BNS_KERNEL_NORMALIZE = 3,     /* y = a x + b over the whole tensor                          */
    BNS_KERNEL_BWD_REDUCE = 4,    /* reads dy, x; writes dx = gamma invstd dy; partial sums     */
    BNS_KERNEL_FINALIZE_BWD = 5,
    BNS_KERNEL_COL_FIXUP = 6,     /* gradient with the statistics terms over whole samples      */
    BNS_KERNEL_PATCH_FIXUP = 7,   /* the same over patches                                      */
    BNS_KERNEL_MASK = 8,
    BNS_KERNEL_DIRECT_MOMENTS = 9, /* statistics of a small sampled set, one block per channel    */
    BNS_KERNEL_DIRECT_FIXUP = 10,  /* backward sums combined + statistics terms, small sampled set */
    BNS_KERNEL_VECTOR = 11,        /* C-length kernels: mixing of statistics, moving average          */
    BNS_KERNEL_SLAB_FORWARD = 12,  /* whole forward of a layer whose channel data fits on chip        */
    BNS_KERNEL_SLAB_BACKWARD = 13, /* whole backward of such a layer                                   */
    BNS_KERNEL_KINDS = 14
} bns_kernel_kind;

/* Number of kernels this library has launched in this process since load (or since reset). */
uint64_t bns_launch_count(void);
void bns_launch_count_reset(void);
/* With profiling on, every launch is bracketed by CUDA events on its own stream (up to a fixed
 * pool; later launches go untimed).  bns_profile_read synchronises the recorded events and returns
 * the launches and the summed device time of one kernel kind since the last bns_profile_enable. */
void bns_profile_enable(int on);
bns_status bns_profile_read(int kernel_kind, int* launches, float* total_ms);
const char* bns_kernel_name(int kernel_kind);

/* Launch-shape knobs (process-wide; change them only while no call is in flight, and recompute
 * bns_workspace_bytes afterwards).  "target_blocks" / "min_chunk": blocks per launch and least rows
 * per block of the streaming kernels (0 = a multiple of the SM count); "full_min_chunk": least rows per block for rule FULL on tensors of
 * 32 MiB and more; "stat_target_blocks" / "stat_min_chunk": the same for the
 * statistics kernels; "direct_max": sampled elements per channel up to which one block per channel computes the
 * statistics (and, in the backward, combines the sums and applies the statistics terms) without
 * partial sums, 0 = never (the channels-last entry points have the same kind of path, one block per narrow strip
 * of channels, for sampled sets of up to min(direct_max, 2048) pixel rows); "nhwc_blocks": blocks per launch of the channels-last kernels (each block leaves one partial per
 * channel); "slab": 0/1 use the one-launch path where it applies, "slab_cta_kb": preferred shared memory per block of
 * that path in KiB, "slab_min_ctas": grow its clusters while a launch has fewer blocks (0 = two per SM), "slab_max_mb":
 * tensors above this many MiB keep the streaming path (default 6: measured on B200, larger tensors run faster through
 * the streaming kernels), "slab_small_sets": 0/1 take that path also when the sampled set is small (default 0: the
 * streaming path is then two short kernels per direction and measured faster), "slab_cluster_max": largest cluster (1..8);
 * "per_channel_min_hw": map size H*W from which backward pass 1 keeps its sums per channel instead of per position;
 * "host_pipeline": 0/1 row-chunk pipelining of bns_forward_backward_host; "fold_finalize": 0/1 let the second
 * backward pass over a sampled set finish the sums of Eq. 5 itself; "pdl": 0/1 programmatic dependent launch; "l2_order": 0/1 visit rows in an
 * order that lets a kernel find in L2 what the previous one read.  Returns BNS_OK,
 * BNS_ERR_RULE for an unknown name or BNS_ERR_SHAPE for a value < 1. */
int bns_set_tuning(const char* name, int value);

#ifdef __cplusplus
}
#endif
#endif /* BNS_H */
