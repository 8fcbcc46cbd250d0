/*
 * caat.h - C ABI of the B200 (sm_100a) row-parallel linear layer with partial
 * channel-reduce, residual add and per-rank norm (the hot path of CAAT-Net,
 * "Tensor-Parallelism with Partially Synchronized Activations").
 *
 * The t tensor-parallel ranks are simulated as a leading batch dimension on ONE
 * GPU ("logical devices", Section 3.2): every per-rank tensor carries a leading
 * index m = 0..t-1 and the partial channel-reduce is a sum over that index,
 * restricted to the shared channels.
 *
 * Symbols
 *   t      tensor-parallel ranks                         (paper: r; rank index m)
 *   T      tokens = batch x sequence                     (argument `tokens`)
 *   h      hidden size
 *   K      contraction width of the layer: h for the attention output projection,
 *          ffn for the MLP down-projection;  K_r = K / t is one rank's shard
 *   S      shared channels = floor(h * p)                (Eq. A3)
 *   alpha  private-channel scale, sqrt(t) (default) or 1 (Section 4)
 *
 * Conventions (all entry points)
 *   Layout     row-major, last index fastest, densely packed, no padding.
 *   Pointers   every tensor argument is a DEVICE pointer, 16-byte aligned, owned by
 *              the caller; the library keeps none of them after the call returns.
 *              `workspace` is caller-owned device scratch of at least
 *              caat_workspace_bytes(); its contents are undefined on return.
 *   Streams    all work is enqueued on `cuda_stream` (a cudaStream_t cast to void*;
 *              NULL is the default stream); calls do not synchronise.
 *   dtype      CAAT_BF16: bf16 storage, fp32 accumulation and statistics, round to
 *              nearest even on store.  CAAT_F32: fp32 throughout.
 *   Errors     a caat_status is returned; argument errors are found on the host
 *              before any launch and leave all outputs untouched.  There is no CPU
 *              fallback: without a usable CUDA device calls return CAAT_ECUDA.
 *   Determinism  same inputs, same device: bit-identical outputs (no floating-point
 *              atomics; rank sums run m = 0..t-1).
 *   Aliasing   Hn may alias R (in-place residual update); dR may alias dHn; nothing
 *              else may overlap.
 *   Threads    compute calls may be made from several host threads at once (each with its
 *              own stream and its own workspace; a context is read-only while calls run
 *              on it and must not be reconfigured with caat_set_option meanwhile).  The
 *              library's host-side caches are filled under a lock.  Two things are
 *              process-wide and therefore NOT per thread or per stream: the device status
 *              word behind caat_last_device_status (a time-out on any stream of the device
 *              sets it; the call that reads it clears it) and the caat_profile_* benchmark
 *              aid (one recording at a time, not thread-safe).
 *   Limits     h must be a multiple of 8 and at most 16384 (bf16) or 8192 (fp32) channels,
 *              t * tokens at most 2e9 (CAAT_EUNSUPPORTED otherwise); t divides h and ffn.  The tensor-core GEMM is used for CAAT_BF16 when K_r and S
 *              are multiples of 8; other shapes run a slower CUDA-core GEMM.
 */
#ifndef CAAT_H_
#define CAAT_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct caat_ctx caat_ctx; /* opaque; immutable between set_option calls */

typedef enum { CAAT_F32 = 0, CAAT_BF16 = 1 } caat_dtype;

/* Which row-parallel layer: K = h (attention output projection, Eq. A5) or
 * K = ffn (MLP down-projection, Eq. A3). */
typedef enum { CAAT_ATTN_OUT = 0, CAAT_MLP_DOWN = 1 } caat_layer;

typedef enum {
  CAAT_OK = 0,
  CAAT_EINVAL = 1,       /* null pointer, bad enum, value out of range          */
  CAAT_ESHAPE = 2,       /* t does not divide h / ffn, tokens < 1, S > h        */
  CAAT_EALIGN = 3,       /* a tensor pointer is not 16-byte aligned             */
  CAAT_EWORKSPACE = 4,   /* workspace NULL or smaller than caat_workspace_bytes */
  CAAT_EUNSUPPORTED = 5, /* shape outside the limits stated above               */
  CAAT_ECUDA = 6,        /* a CUDA runtime call failed (see caat_last_cuda_error) */
  CAAT_ETIMEOUT = 7,     /* a bounded device-side wait ran out                  */
  CAAT_ELIMIT = 8        /* the call needs more than the built-in scratch of
                            caat_rowpar_forward_noalloc (CAAT_NOALLOC_SCRATCH_BYTES) */
} caat_status;

typedef enum {
  CAAT_OPT_NORM = 0,            /* 0 = RMSNorm (default), 1 = LayerNorm (Eq. 9: "Norm") */
  CAAT_OPT_EPS = 1,             /* norm epsilon, default 1e-5                           */
  CAAT_OPT_PRIVATE_SCALE = 2,   /* alpha; default sqrt(t); 1 switches scaling off       */
  CAAT_OPT_SHARED_CHANNELS = 3, /* override S with an explicit integer in [0, h]        */
  CAAT_OPT_GEMM = 4,            /* 0 = automatic (default), 1 = force the CUDA-core GEMM */
  CAAT_OPT_ROWS = 5,            /* row kernels: 0 = automatic (default: warp-per-token kernels for
                                   rows of at most 1024 bf16 channels, bulk-copy staged kernels
                                   otherwise), 1 = plain-load kernels, 2 = staged kernels always */
  CAAT_OPT_DECODE = 6,          /* 0 = automatic (default: forward calls with at most 64 tokens
                                   stream the weights with swapped GEMM operands),
                                   1 = always use the large-batch forward                */
  CAAT_OPT_BACKWARD_REDUCE = 7, /* precision of the backward rank sum on the shared channels
                                   (Section 4, "fp32 accumulation"); a numerics-study switch:
                                   0 = the ranks' gradients are summed in fp32 as computed (default);
                                   1 = each rank's gradient is first rounded to the run dtype (what
                                       a 16-bit all-reduce carries), the sum runs in fp32;
                                   2 = rounded, and the running sum is rounded to the run dtype
                                       after every addition (accumulation in 16 bit).
                                   1 and 2 run on the plain-load row kernels.              */
  CAAT_OPT_TP_GROUPS = 8,       /* G >= 1 (default 1): this context holds t of t*G tensor-parallel ranks,
                                   one group of t ranks per GPU (see caat_tp_*): K_r becomes K / (t*G).
                                   Setting it also sets alpha = sqrt(t*G) (Section 4: the square root of
                                   the number of devices); CAAT_OPT_PRIVATE_SCALE may override that
                                   afterwards.  CAAT_ESHAPE unless t*G divides h and ffn.               */
  CAAT_OPT_BLOCK_OVERLAP = 9    /* caat_block_forward: 1 = the attention-out layer's row kernel (HBM-bound) runs on a second
                                   stream beside the MLP-down layer's GEMM (tensor-bound), which does not depend on it,
                                   when the workspace holds both layers' scratch (caat_block_workspace_bytes); 0 = the
                                   layers' kernels run one after the other on the caller's stream; 2 (default) = 1
                                   unless that GEMM is much the longer of the two kernels (ffn / t large, e.g. the 7B
                                   shapes, where the GPU is at its power limit and running both at once gains nothing).
                                   Worth 2-4 % of a training step at the 130M / 1.1B shapes                             */
} caat_option;

/* Creates a context for hidden size h, MLP width ffn, t ranks, synchronisation
 * factor p in [0,1] (Section 3: the first h*p channels are shared; S =
 * floor(h*p) in IEEE double, Eq. A3).  Host-only; allocates no device memory. */
caat_status caat_create(int h, int ffn, int t, double p, caat_dtype dtype, caat_ctx **out);
caat_status caat_set_option(caat_ctx *ctx, caat_option opt, double value);
void caat_destroy(caat_ctx *ctx);

/* S, the number of shared channels: channels [0,S) are summed over ranks and
 * channels [S,h) stay private to each rank (Eq. A3).  -1 if ctx is NULL. */
int caat_shared_channels(const caat_ctx *ctx);
/* alpha currently in effect. */
double caat_private_scale(const caat_ctx *ctx);

/* Bytes of device scratch for the block calls (caat_block_forward / _backward and the compact variants):
 * enough for the two layers' scratch side by side, which lets the block forward overlap the first layer's row
 * kernel with the second layer's GEMM.  A workspace of only the larger of the two layers' caat_workspace_bytes
 * is accepted as well; the block forward then runs its kernels one after the other. */
size_t caat_block_workspace_bytes(const caat_ctx *ctx, int tokens, int backward);

/* Bytes of device scratch for `tokens` tokens of `layer`: backward = 0, what the forward
 * call needs; backward = 1, enough for the forward AND the backward call (a training step
 * runs both on one buffer; neither keeps anything in it between calls).  The block calls
 * have their own figure, caat_block_workspace_bytes.
 * 0 on bad arguments. */
size_t caat_workspace_bytes(const caat_ctx *ctx, caat_layer layer, int tokens, int backward);

const char *caat_strerror(caat_status s);
/* Text of the last CUDA runtime error seen by this thread's calls ("" if none). */
const char *caat_last_cuda_error(void);

/*
 * Forward of one row-parallel sub-layer (Eq. A3 / A5, Section 4, Eq. 9):
 *   Zt[m,i,l] = sum_k Y[m,i,k] * W[m,l,k]                       per-rank GEMM
 *   Z [m,i,l] = sum_m' Zt[m',i,l]        if l <  S              partial channel-reduce
 *             = alpha * Zt[m,i,l]        if l >= S              private-channel scaling
 *   Hn[m,i,l] = Z[m,i,l] + R[m,i,l]                             residual add
 *   X [m,i,:] = Norm(Hn[m,i,:]) * gamma (+ beta)                per-rank norm over all h
 * rstd (and mean for LayerNorm) are saved for the backward.
 *
 *   Y     [t, T, K_r] dtype  in     W    [t, h, K_r] dtype in (out x in per rank)
 *   R     [t, T, h]   dtype  in     gamma [h] dtype in;  beta [h] dtype in or NULL
 *   Hn    [t, T, h]   dtype  out    X    [t, T, h] dtype out
 *   rstd  [t, T]      fp32   out    mean [t, T] fp32 out (LayerNorm) or NULL (RMSNorm)
 */
caat_status caat_rowpar_forward(const caat_ctx *ctx, caat_layer layer, int tokens,
                                const void *Y, const void *W, const void *R,
                                const void *gamma, const void *beta,
                                void *Hn, void *X, float *rstd, float *mean,
                                void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * caat_rowpar_forward for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant of the forward above, same arithmetic, same
 * kernels, same results.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits when the layer is invoked -
 * inside a serving loop whose memory pool is frozen after start-up, under a framework that
 * forbids allocation on its compute stream, or in a process whose device memory is handed
 * out by another component - and that therefore has no workspace buffer to pass.  Instead
 * of a caller-owned workspace the call uses a fixed scratch array of
 * CAAT_NOALLOC_SCRATCH_BYTES that is part of the library's device image; every GPU that
 * loads the library holds those bytes until the process exits.
 *
 * Arguments and outputs are those of caat_rowpar_forward without workspace/workspace_bytes;
 * the caller still owns and passes every input and output tensor.
 *   Limit      the call is rejected with CAAT_ELIMIT, before any launch, when
 *              caat_workspace_bytes(ctx, layer, tokens, 0) exceeds CAAT_NOALLOC_SCRATCH_BYTES
 *              (e.g. 130M shapes, t=4, h=768, p=0.5: up to 8738 tokens per call).
 *   Set-up     the first call on each device looks up the scratch array's device address
 *              (once per device, with that device current).  With CUDA's lazy module loading
 *              that lookup is also the moment the driver loads this part of the library onto
 *              the device and reserves the array there, so the FIRST call per device can
 *              take device memory and can fail with CAAT_ECUDA when none is left
 *              (caat_last_cuda_error() has the text).  Make that first call at start-up:
 *              before the memory pool is frozen and before starting any CUDA stream capture
 *              on the device.  The address is cached per device ordinal for the life of the
 *              process; after a cudaDeviceReset the library must not be used again.
 *   Allocation after that first call per device, a call performs no cudaMalloc / cudaFree and
 *              calls no allocating library routine.
 *   Sharing    all calls on a device use the same array, which keeps whatever the last call
 *              left in it.  Nothing in it needs to start at zero (every element that is read
 *              is written earlier in the same call).  Two calls that overlap on the GPU
 *              (different streams, or different host threads without ordering) race on it:
 *              order such calls on one stream or with events.
 */
#define CAAT_NOALLOC_SCRATCH_BYTES (32u * 1024u * 1024u)
caat_status caat_rowpar_forward_noalloc(const caat_ctx *ctx, caat_layer layer, int tokens,
                                        const void *Y, const void *W, const void *R,
                                        const void *gamma, const void *beta,
                                        void *Hn, void *X, float *rstd, float *mean,
                                        void *cuda_stream);

/*
 * Backward of the same sub-layer: the exact gradient of the forward map, with the
 * rank reduction placed AFTER the norm's backward (operation "h" of Fig. 2b,
 * Section 4 and Appendix B), accumulated in fp32 (Section 4), and the norm
 * parameters' gradients summed over ranks (Section 4):
 *   g  [m,i,:] = NormBwd(dX[m,i,:]; Hn, rstd, mean, gamma) + dHn[m,i,:]
 *   dR [m]     = g[m]                                     (per rank, NOT reduced)
 *   dZt[m,i,l] = sum_m' g[m',i,l] if l < S, alpha * g[m,i,l] if l >= S
 *   dY [m,i,k] = sum_l dZt[m,i,l] * W[m,l,k]
 *   dW [m,l,k] = sum_i dZt[m,i,l] * Y[m,i,k]
 *   dgamma[l]  = sum_m sum_i dX[m,i,l] * xhat[m,i,l];   dbeta[l] = sum_m sum_i dX[m,i,l]
 *
 *   dX [t,T,h] dtype in       dHn [t,T,h] dtype in or NULL (no gradient on the stream)
 *   Y, W, gamma as in the forward; Hn, rstd, mean as the forward wrote them
 *   dY [t,T,K_r] dtype out    dW [t,h,K_r] FP32 out       dR [t,T,h] dtype out
 *   dgamma [h] fp32 out       dbeta [h] fp32 out (LayerNorm) or NULL
 */
caat_status caat_rowpar_backward(const caat_ctx *ctx, caat_layer layer, int tokens,
                                 const void *dX, const void *dHn,
                                 const void *Y, const void *W, const void *Hn,
                                 const float *rstd, const float *mean, const void *gamma,
                                 void *dY, float *dW, void *dR, float *dgamma, float *dbeta,
                                 void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Block = the attention output projection followed by the MLP down-projection, the
 * two row-parallel layers (and the two reduces, Appendix C) of one transformer
 * block, chained through the residual stream: R of the second layer is Hn1.
 * Tensors as in caat_rowpar_forward with K_r = h/t for Y_attn, W_o and ffn/t for
 * Y_mlp, W_down.  beta1/beta2/mean1/mean2 are NULL for RMSNorm.
 *
 * The second layer's GEMM does not depend on the first layer's row kernel.  With a workspace of
 * caat_block_workspace_bytes (both layers' scratch side by side) and CAAT_OPT_BLOCK_OVERLAP on (or chosen automatically), that row
 * kernel runs on a stream of the library's own, forked from and joined back into `cuda_stream` with events
 * inside this call (legal inside a stream capture; the library creates that stream on the first such call per
 * device, so make one call before capturing): everything the call enqueued is ordered before whatever the caller
 * enqueues on `cuda_stream` next.  Results do not depend on the schedule.
 */
caat_status caat_block_forward(const caat_ctx *ctx, int tokens,
                               const void *Y_attn, const void *W_o,
                               const void *Y_mlp, const void *W_down, const void *R0,
                               const void *gamma1, const void *beta1,
                               const void *gamma2, const void *beta2,
                               void *Hn1, void *X1, float *rstd1, float *mean1,
                               void *Hn2, void *X2, float *rstd2, float *mean2,
                               void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Backward of the block: the MLP-down layer first (upstream dX2 through its norm,
 * dHn2 on the outgoing residual stream), then the attention-out layer whose
 * residual-stream gradient is the dR of the second layer (written to dHn1, an
 * output of this call, [t,T,h] dtype).  dHn2 may be NULL.
 */
caat_status caat_block_backward(const caat_ctx *ctx, int tokens,
                                const void *dX1, const void *dX2, const void *dHn2,
                                const void *Y_attn, const void *W_o,
                                const void *Y_mlp, const void *W_down,
                                const void *Hn1, const float *rstd1, const float *mean1,
                                const void *Hn2, const float *rstd2, const float *mean2,
                                const void *gamma1, const void *gamma2,
                                void *dY_attn, float *dW_o, void *dY_mlp, float *dW_down,
                                void *dR0, void *dHn1,
                                float *dgamma1, float *dbeta1, float *dgamma2, float *dbeta2,
                                void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Compact residual layout ("logical devices" on one GPU, Section 3.2).
 *
 * The partial channel-reduce makes the first S channels of the layer output identical on
 * every rank (Eq. A3, l < S), so when the residual entering the first layer is tied on those
 * channels the shared part of the residual stream is ONE tensor for the whole network.  These
 * entry points store it once:
 *     shared part   [T, S]          dtype   (Rs, Hns, dHns, dRs)
 *     private part  [t, T, h - S]   dtype   (Rp, Hnp, dHnp, dRp), column l of rank m at l - S
 * Same arithmetic as caat_rowpar_forward / _backward applied to R[m] = [Rs | Rp[m]]; X, rstd,
 * mean stay per rank ([t, T, h], [t, T]): the statistics of rank m cover its private
 * channels too, so X differs between ranks on the shared channels as well.
 *
 * Backward: Hns is read by every rank's norm, so its gradient collects all ranks' norm
 * backward plus the gradient arriving on the single shared stream,
 *     gs[i,l]   = dHns[i,l] + sum_m NormBwd(dX[m])[i,l]      (l <  S; fp32 sum, m ascending)
 *     gp[m,i,l] = dHnp[m,i,l] + NormBwd(dX[m])[i,l]          (l >= S)
 *     dRs = gs,  dRp = gp,  dZt[m] = [gs | alpha * gp[m]],  dY, dW, dgamma, dbeta as above.
 * gs is the backward partial channel-reduce (operation "h" of Fig. 2b) and the shared
 * residual gradient at once.  dHns and dHnp are both given or both NULL.
 *
 * Requires S % 8 == 0 (CAAT_EUNSUPPORTED otherwise).  A part that is empty (S = 0 or S = h)
 * may be passed as NULL.  Workspace sizes are those of the per-rank entry points.  Forward
 * calls with at most 64 tokens stream the weights with swapped GEMM operands here too
 * (CAAT_OPT_DECODE); this is the single-device serving arrangement of Section 3.2.
 */
caat_status caat_rowpar_forward_compact(const caat_ctx *ctx, caat_layer layer, int tokens,
                                        const void *Y, const void *W,
                                        const void *Rs, const void *Rp,
                                        const void *gamma, const void *beta,
                                        void *Hns, void *Hnp, void *X, float *rstd, float *mean,
                                        void *workspace, size_t workspace_bytes, void *cuda_stream);
caat_status caat_rowpar_backward_compact(const caat_ctx *ctx, caat_layer layer, int tokens,
                                         const void *dX, const void *dHns, const void *dHnp,
                                         const void *Y, const void *W,
                                         const void *Hns, const void *Hnp,
                                         const float *rstd, const float *mean, const void *gamma,
                                         void *dY, float *dW, void *dRs, void *dRp,
                                         float *dgamma, float *dbeta,
                                         void *workspace, size_t workspace_bytes, void *cuda_stream);
/* Block (attention-out then MLP-down) on the compact stream; dHn1s / dHn1p are outputs
 * (the residual gradient between the two layers), as dHn1 in caat_block_backward. */
caat_status caat_block_forward_compact(const caat_ctx *ctx, int tokens,
                                       const void *Y_attn, const void *W_o,
                                       const void *Y_mlp, const void *W_down,
                                       const void *R0s, const void *R0p,
                                       const void *gamma1, const void *beta1,
                                       const void *gamma2, const void *beta2,
                                       void *Hn1s, void *Hn1p, void *X1, float *rstd1, float *mean1,
                                       void *Hn2s, void *Hn2p, void *X2, float *rstd2, float *mean2,
                                       void *workspace, size_t workspace_bytes, void *cuda_stream);
caat_status caat_block_backward_compact(const caat_ctx *ctx, int tokens,
                                        const void *dX1, const void *dX2,
                                        const void *dHn2s, const void *dHn2p,
                                        const void *Y_attn, const void *W_o,
                                        const void *Y_mlp, const void *W_down,
                                        const void *Hn1s, const void *Hn1p,
                                        const float *rstd1, const float *mean1,
                                        const void *Hn2s, const void *Hn2p,
                                        const float *rstd2, const float *mean2,
                                        const void *gamma1, const void *gamma2,
                                        void *dY_attn, float *dW_o, void *dY_mlp, float *dW_down,
                                        void *dR0s, void *dR0p, void *dHn1s, void *dHn1p,
                                        float *dgamma1, float *dbeta1, float *dgamma2, float *dbeta2,
                                        void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Column-parallel half in front of a row-parallel layer (Section 3: Y_m = sigma(X_m A_m); the
 * inner sum of Eq. A3; the QKV projection in front of attention, Eq. A5).  With partially
 * synchronised activations every rank has its OWN input X_m (the per-rank norm output X of the
 * previous layer), so the layer is t independent products, no reduce:
 *   pre[m,i,n] = sum_j X[m,i,j] * A[m,n,j]                         n < n_out
 *   CAAT_ACT_NONE    Y = pre                        (QKV projection: n_out = 3 h / t)
 *   CAAT_ACT_SILU    Y[m,i,n] = silu(pre[m,i,n])    (an elementwise sigma)
 *   CAAT_ACT_SWIGLU  Y[m,i,n] = silu(pre[m,i,n]) * pre[m,i,F+n],  n < F = n_out / 2
 *                    (gated MLP of the Llama models: rows [0,F) of A_m are the gate, rows
 *                    [F,2F) the up projection; Y is the row-parallel layer's input, F = ffn/t)
 *
 *   X   [t, T, h]      dtype in      A  [t, n_out, h] dtype in (out x in per rank)
 *   pre [t, T, n_out]  dtype out (kept for the backward)
 *   Y   [t, T, n_out or n_out/2] dtype out; NULL for CAAT_ACT_NONE (pre is the result)
 * Backward, given dY (the gradient on Y; on pre for CAAT_ACT_NONE):
 *   dpre = dY through the activation,  dX[m] = dpre[m] A[m],  dA[m] = dpre[m]^T X[m]
 *   dX [t, T, h] dtype out (the upstream gradient dX of the previous row-parallel layer's norm)
 *   dA [t, n_out, h] FP32 out
 * n_out must be a multiple of 8 (16 for CAAT_ACT_SWIGLU).  The forward needs no workspace.
 */
typedef enum { CAAT_ACT_NONE = 0, CAAT_ACT_SILU = 1, CAAT_ACT_SWIGLU = 2 } caat_activation;
size_t caat_colpar_workspace_bytes(const caat_ctx *ctx, caat_activation act, int n_out, int tokens);
caat_status caat_colpar_forward(const caat_ctx *ctx, caat_activation act, int n_out, int tokens,
                                const void *X, const void *A, void *pre, void *Y, void *cuda_stream);
caat_status caat_colpar_backward(const caat_ctx *ctx, caat_activation act, int n_out, int tokens,
                                 const void *dY, const void *X, const void *A, const void *pre,
                                 void *dX, float *dA,
                                 void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Real tensor parallelism over several GPUs (Section 3: the all-reduce of the shared channels is the
 * layer's one exchange step; Appendix D: reduce-scatter + all-gather of tokens*S elements).  A layer call
 * is split into the half before and the half after that exchange; the caller owns the collective (NCCL
 * through its framework, or its own kernel over peer memory) and runs it, on the same stream, on the
 * packed slab the first half leaves in the workspace:
 *
 *   forward :  caat_tp_forward_local   slab[i,l] = sum over this GPU's ranks m of Zt[m,i,l], l < S
 *                                      (the private columns of Zt stay in the workspace as well)
 *              all-reduce(slab, sum)   over the GPUs of the tensor-parallel group
 *              caat_tp_forward_finish  private scaling, residual add, per-rank norm (Eq. 9)
 *   backward:  caat_tp_backward_local  norm backward + residual gradient: dR, this GPU's dgamma / dbeta,
 *                                      slab[i,l] = sum over this GPU's ranks of g[m,i,l], l < S
 *              all-reduce(slab, sum)   -- Section 4: accumulate this sum in fp32; also all-reduce
 *                                         dgamma / dbeta [h] fp32 (Eq. 10-11: summed over devices)
 *              caat_tp_backward_finish dY and dW from the reduced slab and this GPU's dR
 *
 * The context describes this GPU's t ranks of the t*G in the group (CAAT_OPT_TP_GROUPS = G); tensors
 * are the same as in caat_rowpar_forward / _backward with this GPU's ranks only.  The slab is
 * [tokens, S] elements of the run dtype, row-major and dense, at byte `offset` of the workspace
 * (caat_tp_slab; the forward and the backward slab may sit at different offsets).  Both halves of a
 * direction must get the same workspace, untouched in between except for the slab.  Tensor-core path
 * only (bf16, K_r and S multiples of 8): CAAT_EUNSUPPORTED otherwise.  Workspace size:
 * caat_workspace_bytes.  With G = 1 the two halves and no collective give caat_rowpar_forward /
 * _backward's results for more than 64 tokens (few-token calls take another route there).
 */
caat_status caat_tp_slab(const caat_ctx *ctx, caat_layer layer, int tokens, int backward,
                         size_t *offset_bytes, int *rows, int *cols);
caat_status caat_tp_forward_local(const caat_ctx *ctx, caat_layer layer, int tokens,
                                  const void *Y, const void *W,
                                  void *workspace, size_t workspace_bytes, void *cuda_stream);
caat_status caat_tp_forward_finish(const caat_ctx *ctx, caat_layer layer, int tokens,
                                   const void *R, const void *gamma, const void *beta,
                                   void *Hn, void *X, float *rstd, float *mean,
                                   void *workspace, size_t workspace_bytes, void *cuda_stream);
caat_status caat_tp_backward_local(const caat_ctx *ctx, caat_layer layer, int tokens,
                                   const void *dX, const void *dHn, const void *W, const void *Hn,
                                   const float *rstd, const float *mean, const void *gamma,
                                   void *dR, float *dgamma, float *dbeta,
                                   void *workspace, size_t workspace_bytes, void *cuda_stream);
caat_status caat_tp_backward_finish(const caat_ctx *ctx, caat_layer layer, int tokens,
                                    const void *Y, const void *W, const void *dR,
                                    void *dY, float *dW,
                                    void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * The exchange of the shared-channel slab over PEER MEMORY, in the library's own kernels (Section 3:
 * partial channel-reduce; Appendix D: reduce-scatter + all-gather of tokens*S elements; Section 4:
 * communicate in 16 bit, accumulate in 32 bit).  It replaces the caller's collective between the two
 * halves of a layer call (see above) when the GPUs of the group can address each other's memory
 * (NVLink / NVSwitch peers: plain loads and stores, no multicast load anywhere):
 *
 *   scatter   every GPU stores rows [q*slice, (q+1)*slice) of its slab - its ranks' partial sum -
 *             into slot `rank` of GPU q's receive buffer (16-bit payload), then raises flag `rank`
 *             on GPU q.  caat_tp_forward_local_push does the same from inside the forward GEMM: the
 *             tiles of the shared columns leave the epilogue straight for their owner's slot while
 *             the private columns' tiles are still being multiplied, and the slab is never written.
 *             caat_tp_backward_local_push is the backward's counterpart: the row kernel that forms the
 *             reduced shared gradient stores each token's row into its owner's slot instead of the slab.
 *   reduce    GPU q waits for all `world` flags, sums the `world` slots of its token slice in fp32 in
 *             the fixed order 0..world-1, rounds once to the run dtype and stores the result rows
 *             into EVERY GPU's slab (the all-gather), then raises flag `world + q` on every GPU.
 *   wait      every GPU waits for all `world` gather flags: its slab is complete; the second half of
 *             the layer call (caat_tp_forward_finish / caat_tp_backward_finish) follows on the stream.
 *
 * caat_tp_exchange runs the three phases in a row on one GPU's stream; in a job every GPU of the group
 * calls it at the same point of its stream.  The phases are also exported one by one, which is how a
 * single GPU can stand in for the whole group in a test (all scatters, then all reduces, then all waits).
 *
 *   peers->world, rank   size of the group (<= CAAT_MAX_PEERS) and this GPU's index in it
 *   peers->recv[q]       GPU q's receive buffer, caat_tp_exchange_bytes' recv_bytes, as THIS GPU addresses it
 *   peers->slab[q]       GPU q's slab (workspace + caat_tp_slab's offset), as this GPU addresses it
 *   peers->flags[q]      GPU q's flag words, CAAT_TP_FLAG_BYTES, zeroed once by their owner before first use
 *   epoch                a number every GPU of the group passes alike, larger (mod 2^32) in every new exchange
 *                        on the same buffers; flags are compared with it and never reset
 * slice = tokens per owner = caat_tp_exchange_bytes' slice_rows (the same on every GPU).  Every wait on a
 * flag is bounded (about a second): when it runs out the kernel raises the device status word
 * (caat_last_device_status returns CAAT_ETIMEOUT), skips its work and returns; nothing traps or spins on.
 * bf16 tensor-core path only, S a multiple of 8; caat_tp_forward_local_push further needs slice_rows to be
 * a multiple of 256 (CAAT_EUNSUPPORTED otherwise: use caat_tp_forward_local + the scatter phase).
 * Buffers named in `peers` are owned by the callers; the library keeps no pointer after the call returns.
 */
#define CAAT_MAX_PEERS 8
#define CAAT_TP_FLAG_BYTES 256
typedef struct caat_peers {
  int world, rank;
  void *recv[CAAT_MAX_PEERS];
  void *slab[CAAT_MAX_PEERS];
  unsigned int *flags[CAAT_MAX_PEERS];
} caat_peers;
caat_status caat_tp_exchange_bytes(const caat_ctx *ctx, caat_layer layer, int tokens, int world,
                                   size_t *recv_bytes, int *slice_rows);
caat_status caat_tp_exchange_scatter(const caat_ctx *ctx, caat_layer layer, int tokens, int backward,
                                     const caat_peers *peers, unsigned int epoch,
                                     void *workspace, size_t workspace_bytes, void *cuda_stream);
caat_status caat_tp_exchange_reduce(const caat_ctx *ctx, caat_layer layer, int tokens,
                                    const caat_peers *peers, unsigned int epoch, void *cuda_stream);
caat_status caat_tp_exchange_wait(const caat_ctx *ctx, const caat_peers *peers, unsigned int epoch,
                                  void *cuda_stream);
caat_status caat_tp_exchange(const caat_ctx *ctx, caat_layer layer, int tokens, int backward,
                             const caat_peers *peers, unsigned int epoch,
                             void *workspace, size_t workspace_bytes, void *cuda_stream);
caat_status caat_tp_forward_local_push(const caat_ctx *ctx, caat_layer layer, int tokens,
                                       const void *Y, const void *W,
                                       const caat_peers *peers, unsigned int epoch,
                                       void *workspace, size_t workspace_bytes, void *cuda_stream);
/* caat_tp_backward_local (same tensors) with the scatter phase folded into the row kernel; follow it with
 * caat_tp_exchange_reduce and caat_tp_exchange_wait, then caat_tp_backward_finish.  Any slice_rows. */
caat_status caat_tp_backward_local_push(const caat_ctx *ctx, caat_layer layer, int tokens,
                                        const void *dX, const void *dHn, const void *W, const void *Hn,
                                        const float *rstd, const float *mean, const void *gamma,
                                        void *dR, float *dgamma, float *dbeta,
                                        const caat_peers *peers, unsigned int epoch,
                                        void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Analytic bytes ONE partial channel-reduce would move on a real t-device system
 * (Appendix C: each device sends and receives tokens*h*p activations per reduce;
 * Appendix D: all-reduce = reduce-scatter + all-gather, traffic cut by 100(1-p) %).
 * elem_bytes is 2 for 16-bit communication.  Host-only.  Outputs may be NULL.
 *   payload_per_rank     = tokens * S * elem_bytes
 *   payload_per_rank_p1  = tokens * h * elem_bytes          (full all-reduce)
 *   ring_wire_per_rank   = 2 (n-1) * payload / n            (rounded down; n = t, or the number of
 *                                                             GPUs G when CAAT_OPT_TP_GROUPS > 1)
 */
caat_status caat_allreduce_bytes(const caat_ctx *ctx, int tokens, int elem_bytes,
                                 unsigned long long *payload_per_rank,
                                 unsigned long long *payload_per_rank_p1,
                                 unsigned long long *ring_wire_per_rank);

/* Synchronises `cuda_stream` and reports CAAT_ETIMEOUT if a kernel launched
 * through this library gave up on a bounded wait since the last call of this
 * function, CAAT_ECUDA if the stream is in error, else CAAT_OK.
 * The wait limits can be shortened, and a wait made to run out, from the environment
 * (read once per process; for tests of this path, no effect on a call that returns
 * CAAT_OK): CAAT_TC_SPINCAP / CAAT_TC_DEBUG=1024 (tensor-core GEMM), CAAT_ROWS_SPINCAP /
 * CAAT_ROWS_STALL=1 (bulk-copy row kernels), CAAT_TP_POLLCAP (exchange kernels). */
caat_status caat_last_device_status(const caat_ctx *ctx, void *cuda_stream);

/* Number of kernels launched through this library by the calling process since it
 * was loaded (for benchmarks' launch accounting). */
unsigned long long caat_kernel_launches(void);

/*
 * Per-kernel timing aid for benchmarks (the paper has no counterpart).  Between
 * caat_profile_begin and caat_profile_end every kernel launched through the library is
 * bracketed by CUDA events on its launching stream (up to max_launches launches; later
 * ones are counted but not timed).  caat_profile_end waits for the recorded events and
 * returns, per kernel kind, the summed device time in milliseconds and the number of
 * timed launches.  Process-wide, not thread-safe; event objects are kept for reuse.
 */
typedef enum {
  CAAT_K_ROWS_FORWARD = 0,   /* reduce hand-off + scale + residual + norm           */
  CAAT_K_ROWS_BACKWARD = 1,  /* norm backward + residual gradient + backward reduce */
  CAAT_K_NORMGRAD_REDUCE = 2,/* second stage of dgamma / dbeta                      */
  CAAT_K_GEMM_CUDA_CORE = 3, /* CUDA-core GEMM (fp32 and unaligned shapes)          */
  CAAT_K_TC_FORWARD = 4,     /* tcgen05 GEMM, forward                               */
  CAAT_K_TC_DGRAD = 5,       /* tcgen05 GEMM, data gradient                         */
  CAAT_K_TC_WGRAD = 6,       /* tcgen05 GEMM, weight gradient                       */
  CAAT_K_SPLITK_REDUCE = 7,  /* split-K reduction of the weight gradient            */
  CAAT_K_ACTIVATION = 8,     /* activation of the column-parallel half / its derivative */
  CAAT_K_TP_EXCHANGE = 9,    /* slab exchange over peer memory: scatter, reduce + gather, waits */
  CAAT_K_COUNT = 10
} caat_kernel_kind;
caat_status caat_profile_begin(int max_launches);
caat_status caat_profile_end(int n_kinds, double *ms_by_kind, unsigned long long *launches_by_kind);
const char *caat_kernel_kind_name(int kind);

#ifdef __cplusplus
}
#endif
#endif /* CAAT_H_ */
