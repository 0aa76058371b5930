/* resist.h -- C boundary of the ResIST sub-ResNet training library (CUDA, sm_100a).
 *
 * The calls follow the protocol of Algorithm 1 of "ResIST: Layer-Wise Decomposition of ResNets for
 * Distributed Training" (arXiv 2107.00961): per synchronisation round, subResNets(.) partitions the
 * residual blocks of a global pre-activation ResNet among S shallow sub-ResNets (Sec. 2.2), each
 * sub-ResNet takes l local SGD steps (Algorithm 1, inner loops), and aggregate(.) sets every global
 * parameter to its mean over the sub-ResNets that held it (Sec. 2.3; Appendix B).  Here the S
 * "workers" are S independent problems on ONE GPU; nothing crosses a link.
 *
 * Conventions
 *  - Every function returns 0 (RESIST_OK) or a negative resist_status; nothing throws or aborts.
 *    resist_last_error() gives a human-readable reason for the last failure on that context.
 *  - "dev" pointers are CUDA device pointers owned by the caller; "host" pointers are ordinary memory.
 *  - Activations are NHWC, convolution weights [Cout][kh][kw][Cin], both contiguous.
 *  - The library owns parameters, momentum, gradients, activations and scratch; it obtains device
 *    memory only through the resist_allocator given at init (or cudaMalloc when that is NULL).
 *  - Work is enqueued on the given stream; calls that return host data synchronise that stream.
 *  - State machine: init -> partition -> (local_step)* -> aggregate -> partition ...; a call out of
 *    order (a local step before the first partition, or after aggregate without a new partition)
 *    returns RESIST_ESTATE.
 *
 * Flat parameter order (all fp32 on the boundary): stem conv; stem BN gamma, beta (if any); per block in
 * network order: basic = bn1 g,b | conv1 3x3 | bn2 g,b | conv2 3x3 | projection 1x1 (if any);
 * bottleneck = bn1 g,b | conv1 1x1 | bn2 g,b | conv2 3x3 | bn3 g,b | conv3 1x1 | projection (if any);
 * final BN g,b; head weight [classes][C]; head bias.  Buffers: per BN in that order, running mean then
 * running variance.
 */
#ifndef RESIST_H
#define RESIST_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    RESIST_OK = 0,
    RESIST_EINVAL = -1,       /* bad argument */
    RESIST_ESTATE = -2,       /* call out of order */
    RESIST_ENOMEM = -3,       /* the allocator returned NULL */
    RESIST_ECUDA = -4,        /* a CUDA call failed; see resist_last_error */
    RESIST_ETIMEOUT = -5,     /* a bounded device-side wait gave up */
    RESIST_EUNSUPPORTED = -6
} resist_status;

enum { RESIST_BASIC = 0, RESIST_BOTTLENECK = 1 };
enum { RESIST_F32 = 0, RESIST_BF16 = 1 };
enum { RESIST_MOMENTUM_RESTART = 0, RESIST_MOMENTUM_KEEP = 1 };
enum { RESIST_CONV_AUTO = 0, RESIST_CONV_CUDA_CORES = 1, RESIST_CONV_TCGEN05 = 2, RESIST_CONV_WARP_MMA = 3,
       RESIST_CONV_WARP_MMA_UNFUSED = 4 };
#define RESIST_MAX_SUBNETS 32

typedef struct resist_ctx resist_ctx;
typedef void* resist_stream;                 /* a cudaStream_t */

/* One residual block (Sec. 2.1, pre-activation order BN -> ReLU -> conv).  `partitionable` marks the blocks
 * that subResNets(.) deals out (Sec. 2.2: the non-strided blocks of the third section); all others are
 * held by every sub-ResNet. */
typedef struct {
    int32_t kind;            /* RESIST_BASIC (3x3,3x3) or RESIST_BOTTLENECK (1x1,3x3,1x1; stride on the 3x3) */
    int32_t stage;
    int32_t cin, cmid, cout; /* basic: cmid = cout */
    int32_t stride;          /* 1 or 2 */
    int32_t has_projection;  /* 1x1 strided conv on the skip path, reading relu(bn1(x)) */
    int32_t partitionable;
} resist_block;

typedef struct {
    int32_t in_h, in_w, in_c, classes;
    int32_t stem_k, stem_stride, stem_cout;
    int32_t stem_bn_relu;    /* stem conv followed by BN + ReLU */
    int32_t stem_maxpool;    /* then a 3x3 stride-2 max-pool, padding 1 */
    int32_t num_blocks;
    const resist_block* blocks;   /* host, num_blocks entries, copied at init */
} resist_arch;

typedef struct {
    int32_t dtype;           /* RESIST_F32: everything fp32 on CUDA cores.  RESIST_BF16: activations, activation
                                gradients and the convolutions' weight copy are bf16, accumulation and all
                                parameters, statistics and gradients of parameters fp32 */
    float momentum;          /* SGD momentum mu: v = mu*v + g; w -= lr*v */
    float weight_decay;      /* g += wd*w */
    float bn_eps;
    float bn_momentum;       /* running = (1-m)*running + m*batch (variance unbiased) */
    int32_t min_depth;       /* >0: top sub-ResNets up to this many partitioned blocks (Sec. 2.6) */
    int32_t momentum_policy; /* RESIST_MOMENTUM_RESTART: zero the momentum at every partition */
    int32_t conv_backend;    /* RESIST_CONV_AUTO: warp-level MMA for narrow layers (<= 64 channels), tcgen05 for wide ones,
                                CUDA cores for the rest; _CUDA_CORES: never tensor cores; _TCGEN05 / _WARP_MMA: only that
                                tensor-core family where the shape allows, CUDA cores elsewhere.  With _AUTO and _WARP_MMA
                                the BN+ReLU (forward or backward) that consumes a warp-MMA convolution's output runs inside
                                that convolution's launch; _WARP_MMA_UNFUSED keeps BN in launches of its own */
    int32_t bn_stat_period;  /* 0 or 1: resist_aggregate averages the BN running statistics at every call; k > 1: only at every k-th
                                call (Sec. 5, ImageNet settings: statistics aggregated once per many synchronisation rounds); in
                                between, the global statistics keep their last aggregated values */
} resist_opts;

/* Device-memory source.  alloc returns a device pointer aligned to >= 256 bytes or NULL; release frees it.
 * Both are called on the host from inside resist_* calls (never from another thread). */
typedef struct {
    void* (*alloc)(void* user, size_t bytes);
    void (*release)(void* user, void* dev_ptr);
    void* user;
} resist_allocator;

/* Creates a context holding the global ResNet h(W) with random initial weights (Algorithm 1, input): He-normal
 * conv and head weights drawn from a splitmix64 stream seeded with `seed`, gamma 1, beta 0, bias 0, running
 * mean 0, running var 1.  arch, opts: host.  alloc may be NULL.  *out receives the context. */
int resist_init(const resist_arch* arch, const resist_opts* opts, uint64_t seed, const resist_allocator* alloc,
                resist_ctx** out);
int resist_destroy(resist_ctx* ctx);

/* subResNets(h(W), S) of Algorithm 1 (Sec. 2.2): permutes the partitionable block indices with Fisher-Yates
 * driven by splitmix64(round_seed) (i from P-1 down to 1, j = next() mod (i+1)), deals position j of the
 * permutation to sub-ResNet j mod S, gives every other block to all S; then copies the global parameters into
 * the S working copies (the step of Algorithm 1 that hands every sub-ResNet to its worker) and restarts their momentum.
 * member_mask: host, [num_blocks], bit s set = block is in sub-ResNet s (may be NULL).
 * Errors: S < 1 or S > 32, or S > P with min_depth == 0 -> RESIST_EINVAL. */
int resist_partition(resist_ctx* ctx, uint64_t round_seed, int32_t S, uint32_t* member_mask, resist_stream stream);

/* One local SGD iteration of sub-ResNet `subnet` (Algorithm 1: W_s = W_s - eta dL/dW_s): forward and backward
 * of its blocks on one minibatch (batch-statistics BN, mean softmax cross-entropy), then the momentum update.
 * images: dev, [B][in_h][in_w][in_c], fp32 or bf16 according to opts.dtype.  labels: dev int32 [B].
 * loss_out: dev float[1] or NULL.  B >= 2. */
int resist_local_step(resist_ctx* ctx, int32_t subnet, const void* images, const int32_t* labels, int32_t B,
                      float lr, float* loss_out, resist_stream stream);

/* The same iteration for all S sub-ResNets at once: each layer slot is one launch over the S problems.
 * images, labels: host arrays of S dev pointers.  loss_out: dev float[S] or NULL. */
int resist_local_step_grouped(resist_ctx* ctx, const void* const* images, const int32_t* const* labels, int32_t B,
                              float lr, float* loss_out, resist_stream stream);

/* aggregate({h_s(W_s)}) of Algorithm 1 (Sec. 2.3; Appendix B): every global parameter and BN running statistic
 * becomes the mean over the sub-ResNets that held it, evaluated in fp32 as first + (sum_s (w_s - first))/count
 * with owners in ascending order; a single owner is copied bit for bit. */
int resist_aggregate(resist_ctx* ctx, resist_stream stream);

/* Evaluates the global network (Sec. 2.6): all blocks, BN with running statistics, the residual branch of every
 * partitionable block scaled by 1/S (S of the last partition; 1 before any).  logits_out: dev float
 * [B][classes] or NULL; loss_out: dev float[1] or NULL; correct_out: dev int32[1] (top-1 hits) or NULL. */
int resist_eval(resist_ctx* ctx, const void* images, const int32_t* labels, int32_t B, float* logits_out,
                float* loss_out, int32_t* correct_out, resist_stream stream);

/* Parity and checkpoint taps (host buffers, fp32, flat order above; they synchronise the device). */
int resist_param_count(resist_ctx* ctx, int64_t* n_params, int64_t* n_buffers);
int resist_get_params(resist_ctx* ctx, int32_t subnet /* -1 = global */, float* host_params, float* host_buffers);
int resist_set_params(resist_ctx* ctx, const float* host_params, const float* host_buffers);   /* global */
int resist_get_grads(resist_ctx* ctx, int32_t subnet, float* host_grads);    /* last step's dL/dW; absent blocks 0 */
int resist_get_logits(resist_ctx* ctx, int32_t subnet, float* host_logits);  /* last step's [B][classes] */
/* bf16 mode: the convolutions' copy of sub-ResNet `subnet`'s parameters (bf16 bit patterns, flat order): after every
 * update it is the fp32 working copy rounded to nearest even (Algorithm 1's W_s, as the tensor cores read it). */
int resist_get_shadow(resist_ctx* ctx, int32_t subnet, uint16_t* host_bf16);

/* Work counters of the last local step call (grouped or single). */
typedef struct {
    int64_t kernel_launches;   /* kernels enqueued */
    int64_t conv_flops;        /* 2*M*N*K summed over forward, dgrad and wgrad convolutions */
    int64_t tensor_core_convs; /* convolution problems run on a tensor-core family: tcgen05 or warp-level MMA */
    int64_t cuda_core_convs;   /* convolution problems run on CUDA cores */
    int64_t workspace_bytes;   /* device memory held for activations and scratch */
} resist_step_info;
int resist_get_step_info(resist_ctx* ctx, resist_step_info* out);

/* ---- Layer-level entry points: one layer on caller-owned device tensors, run by the kernels of the local step.
 * They allocate their own scratch with cudaMalloc, synchronise the stream before returning, and report
 * failures through resist_layer_last_error().  dtype: RESIST_F32 or RESIST_BF16 for activations and weights.
 *
 * resist_conv2d: a k x k convolution with zero padding (k-1)/2 and stride 1 or 2, the building block of the
 * residual blocks of Sec. 2.1.  Geometry is always that of the forward convolution: a [N,H,W,C], w [K,k,k,C],
 * y [N,P,Q,K] with P = (H + 2*pad - k)/stride + 1.
 *   mode 0 (forward): act = a, wgt = w, out = y = scale * conv(a, w) + add      (add: y-shaped or NULL)
 *   mode 1 (dgrad):   act = dy, wgt = w, out = da = conv^T(dy, w) + add         (add: a-shaped or NULL)
 *   mode 2 (wgrad):   act = a, wgt = dy, out = dw, fp32 [K,k,k,C]
 * backend: one of RESIST_CONV_*; *used_backend (host, may be NULL) receives 0 (CUDA cores), 1 (tcgen05) or
 * 2 (warp-level MMA). */
int resist_conv2d(int32_t mode, int32_t dtype, int32_t backend, const void* act, const void* wgt, const void* add, void* out,
                  int32_t N, int32_t H, int32_t W, int32_t C, int32_t K, int32_t ksz, int32_t stride, float scale,
                  int32_t* used_backend, resist_stream stream);

/* BN (batch statistics over the m rows of x [m, C], biased variance) followed by ReLU, the pre-activation of
 * Sec. 2.1.  stat: dev float [4*C], receives mean and 1/sqrt(var+eps) (and, in backward, the two reduction
 * sums); run_mean/run_var: dev, updated when non-NULL.  Backward returns dx (+ add), dgamma, dbeta. */
int resist_bn_relu_forward(int32_t dtype, const void* x, const float* gamma, const float* beta, void* a, float* stat,
                           float* run_mean, float* run_var, int64_t m, int32_t C, float eps, float momentum,
                           resist_stream stream);
int resist_bn_relu_backward(int32_t dtype, const void* x, const void* da, const float* gamma, const float* beta, float* stat,
                            const void* add, void* dx, float* dgamma, float* dbeta, int64_t m, int32_t C,
                            resist_stream stream);
/* A convolution together with the BN+ReLU that consumes its output (Sec. 2.1: every convolution of a pre-activation
 * block feeds a BN -> ReLU), launched the way the local step launches the pair, bf16 only:
 *   mode 0: y = scale * conv(a, w) + add  [out];  a_out = relu(bn(y)) with batch statistics  [bn_out]; stat as in
 *           resist_bn_relu_forward; run_mean / run_var updated when non-NULL.  x, bn_add, dgamma, dbeta unused.
 *   mode 1: da = conv^T(dy, w) + add  [out];  dx = backward of the BN+ReLU with input x (a-shaped) and output gradient da,
 *           plus bn_add when non-NULL  [bn_out]; dgamma, dbeta; stat must hold that BN's mean and 1/sqrt(var+eps).
 * Layers of up to 64 channels run the BN inside the warp-MMA convolution's launch; wider ones take the statistics from
 * the per-tile sums of the tcgen05 convolution's epilogue (forward) or run the BN launch behind the dgrad.
 * *used_backend: 1 tcgen05, 2 warp-level MMA.  RESIST_EUNSUPPORTED when no tensor-core family takes the pair. */
int resist_conv2d_bn_relu(int32_t mode, int32_t backend, const void* act, const void* wgt, const void* add, void* out,
                          int32_t N, int32_t H, int32_t W, int32_t C, int32_t K, int32_t ksz, int32_t stride, float scale,
                          const void* x, const float* gamma, const float* beta, float* stat, float* run_mean, float* run_var,
                          const void* bn_add, void* bn_out, float* dgamma, float* dbeta, float eps, float momentum,
                          int32_t* used_backend, resist_stream stream);
const char* resist_layer_last_error(void);

/* resist_bn_relu_forward for callers that cannot allocate device memory (the paper has no counterpart: this is a
 * property of the library, not of the method).  Who needs it: code running inside a fixed memory pool, loops
 * that cannot afford the stall an allocation or a free can cause, hosts whose framework owns all device memory.
 * Same arguments and the same result, bit for bit, as resist_bn_relu_forward, but it calls no cudaMalloc,
 * cudaFree or other allocating routine: the per-chunk partial sums (chunks x 2 x C doubles) and the problem
 * descriptor live in a 4 MiB array built into the library, which every GPU that loads the library holds until
 * the process ends.
 *  - Limit: chunks * C <= 262144, where chunks (the number of row chunks reduced by one CTA each) never exceeds
 *    1024: any m with C <= 256 fits.  Larger problems return RESIST_EUNSUPPORTED with the sizes in the message.
 *  - The first call on each device looks up the array's device address (one cudaGetSymbolAddress, with that
 *    device current); later calls on that device reuse it.
 *  - All calls share the one array, and it keeps what the last call left there.  Nothing has to be cleared between
 *    calls (each call writes every slot before reading it), but two calls that overlap on the GPU (different
 *    streams, or different host threads without ordering) race on it: keep them on one stream or order them.
 *  - Asynchronous: work is enqueued on `stream`, nothing is synchronised.  Errors: resist_noalloc_last_error(). */
int resist_bn_relu_forward_noalloc(int32_t dtype, const void* x, const float* gamma, const float* beta, void* a, float* stat,
                                   float* run_mean, float* run_var, int64_t m, int32_t C, float eps, float momentum,
                                   resist_stream stream);
const char* resist_noalloc_last_error(void);

/* Per-kernel timing.  With profiling on, every launch of a local step, partition or aggregate is bracketed by
 * CUDA events on the call's stream and the call synchronises before returning; times, launch counts and the
 * algorithmic bytes and FLOPs of the work launched accumulate per kernel family until read.
 * A family's launches are reported in two entries: those whose algorithmic work has an arithmetic intensity above
 * 250 FLOP per byte (where the bf16 tensor peak of a B200 meets its HBM bandwidth) under "<name>@tensor", the
 * others under "<name>": the first are held against the tensor peak, the second against HBM bandwidth.
 * resist_get_profile copies up to `cap` entries to host memory, returns the number of entries in *n (may
 * exceed cap) and clears the counters. */
typedef struct {
    char name[32];
    int64_t launches;        /* kernel launches (a family may issue two kernels per operation) */
    int64_t operations;      /* bracketed operations */
    double ms;               /* summed device time */
    double bytes;            /* algorithmic bytes: each operand read once, each result written once */
    double flops;            /* algorithmic FLOPs (convolutions: 2*M*N*K) */
} resist_profile_entry;
int resist_set_profiling(resist_ctx* ctx, int32_t on);
int resist_get_profile(resist_ctx* ctx, resist_profile_entry* out, int32_t cap, int32_t* n);

/* The library's own splitmix64 (the stream that drives the partition), for cross-checking: host out[n]. */
void resist_splitmix64(uint64_t seed, int64_t n, uint64_t* out);

const char* resist_last_error(resist_ctx* ctx);   /* ctx may be NULL: the last init failure */

/* Micro-benchmark behind the tile shapes of the tensor-core kernels (the paper has no counterpart: a property of the device): every
 * SM issues `reps` tcgen05 MMAs of shape 128 x n x 16 (bf16 -> fp32) back to back and waits for them; *cycles_per_mma (host)
 * receives SM clocks per MMA, first issue to completion.  layout: 0 K-major operands without swizzle, 1 K-major with the 128-byte
 * swizzle (the four 32-byte steps of a row in turn), 2 the same reading one step only, 3 MN-major with the 128-byte swizzle.
 * issuers: 1 or 2 issuing threads; alternate: 1 = consecutive MMAs accumulate into two different accumulators.  Operand values are
 * whatever the shared memory holds.  Synchronises the device. */
int resist_micro_mma_rate(int32_t n, int32_t layout, int32_t reps, int32_t issuers, int32_t alternate, double* cycles_per_mma);

/* Test hook: stores `code` in the device status word that a kernel's bounded wait writes when it gives up, so that the next
 * call that synchronises (resist_aggregate, a parity tap, a layer-level call) returns RESIST_ETIMEOUT and clears the word.
 * No kernel has to time out for the reporting path to be tested. */
int resist_debug_set_wait_status(int32_t code);

#ifdef __cplusplus
}
#endif
#endif /* RESIST_H */
