// Internal declarations shared by the translation units of libcaat (CUDA side only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "caat.h"

struct caat_ctx {
  int h, ffn, t;
  double p;
  caat_dtype dtype;
  int S;           // shared channels, floor(h*p) or the explicit override (Eq. A3)
  double alpha;    // private-channel scale (Section 4)
  int norm;        // 0 RMSNorm, 1 LayerNorm
  double eps;
  int force_simt;  // CAAT_OPT_GEMM
  int direct_rows; // CAAT_OPT_ROWS
  int no_decode;   // CAAT_OPT_DECODE
  int bwd_reduce;  // CAAT_OPT_BACKWARD_REDUCE
  int groups;      // CAAT_OPT_TP_GROUPS: this context holds t of t * groups tensor-parallel ranks
  int block_overlap;  // CAAT_OPT_BLOCK_OVERLAP: the block forward runs the first layer's row kernel beside the second GEMM
};

namespace caat {

constexpr int kLayoutVec = 8;        // column granularity of the scratch layout (elements)
constexpr int kMaxPartialRows = 1184;  // upper bound on rows of norm-gradient partials (8 x 148)

inline int round_down(int x, int m) { return x / m * m; }
inline int round_up(int x, int m) { return (x + m - 1) / m * m; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Scratch layout.  The shared part of the layer output (or of its gradient) is
// stored ONCE for all ranks, the private part per rank:
//   zs [T, S_hi]             columns [0, S) valid, S_hi = S rounded up to 8
//   zp [t, T, h - S_lo]      column l of the layer lives at l - S_lo, S_lo = S rounded
//                            down to 8; columns below S - S_lo are not used
// so that every row starts on a 16-byte boundary for any S.
struct Scratch {
  int S_lo, S_hi, P;       // P = h - S_lo, row length of zp
  size_t zs_off, zp_off;   // forward: Zt shared / private.  backward: dZt shared / private
  size_t dgpart_off, dbpart_off;  // backward: [rows, h] fp32 partial norm-parameter gradients
  size_t splitk_off, splitk_bytes;  // backward: split-K partials of the weight gradient
  size_t wt_off;           // backward: the private rows of W times alpha, [t, h, K_r] (tensor-core path, alpha != 1)
  size_t zt_off;           // forward, few tokens: fp32 per-rank partials [t, T, h]
  size_t total;
};

Scratch scratch_layout(const caat_ctx* ctx, int K_r, int tokens, int backward);

inline size_t elem_size(caat_dtype d) { return d == CAAT_BF16 ? 2 : 4; }

// ---- generic strided batched GEMM on CUDA cores (fp32 accumulate) -------------
//   C[b][i][j] = sum_{seg} sum_{q < Q} sum_{k < Kd} A(b,q,i,k) * B(b,q,k,j)
// with element strides for every index; A and B have the run's dtype, C has the
// run's dtype or fp32.
struct GemmSeg {
  const void* A;
  const void* B;
  long long sAb, sAq, sAi, sAk;
  long long sBb, sBq, sBk, sBj;
  int Q, Kd;
};
struct GemmProblem {
  int nseg;
  GemmSeg seg[2];
  void* C;
  long long sCb, sCi;  // column stride of C is 1
  int M, N, batch;
  int c_f32;           // 1: C is fp32 regardless of dtype
};
cudaError_t launch_gemm_simt(const GemmProblem& g, caat_dtype dtype, cudaStream_t st);

// ---- tensor-core GEMMs (bf16, tcgen05 + TMA) -----------------------------------
struct RowparShapes {
  int t, T, h, K_r, S, S_lo, S_hi, P;
};
bool tc_gemm_usable(const caat_ctx* ctx, int K_r);
// Zt -> (zs, zp):   zs[i,l] = sum_m sum_k Y[m,i,k] W[m,l,k] (l < S);  zp[m,i,l-S_lo] = sum_k ... (l >= S)
// push != nullptr: the shared columns' tiles are stored into the peer GPUs' receive slots instead of zs
// (exchange of the slab over peer memory): recv[q] is GPU q's receive buffer [world][slice][S] as this GPU
// addresses it, the owner of token i is i / slice, slice a multiple of 256
struct PushTarget { int world, rank, slice; void* const* recv; };
cudaError_t launch_tc_forward(const RowparShapes& s, const void* Y, const void* W, void* zs, void* zp,
                              cudaStream_t st, const PushTarget* push = nullptr);
// The private part of dZt as the backward GEMMs read it: element (m, i, l) for l >= S sits at
// ptr[(m * T + i) * ld + col0 + (l - S)], and the gradient is alpha times the stored value.
//   scratch copy written by the row kernel:   {zp, P, S - S_lo, 1}
//   the residual gradient itself (per rank):  {dR, h, S, alpha}      (no scaled copy is written at all)
//   compact stream:                           {dRp, P, 0, alpha}
struct PrivOperand { const void* ptr; int ld; int col0; float alpha; };
// dY[m] = [gs | alpha gp[m]] W[m];  w_scaled: [t, h, K_r] scratch for the alpha-scaled private rows of W
// w_scaled_ready: the scaled rows are already in w_scaled (written by the row kernels' reduction launch)
cudaError_t launch_tc_dgrad(const RowparShapes& s, const void* gs, const PrivOperand& pv, const void* W, void* dY,
                            void* w_scaled, bool w_scaled_ready, cudaStream_t st);
// dW[m] = [gs | alpha gp[m]]^T Y[m]   (fp32 out)
cudaError_t launch_tc_wgrad(const RowparShapes& s, const void* gs, const PrivOperand& pv, const void* Y, float* dW,
                            void* splitk, size_t splitk_bytes, cudaStream_t st);
size_t tc_wgrad_splitk_bytes(const RowparShapes& s);
// decode (few tokens): per-rank fp32 partials for all channels, zt[t, T, h]
constexpr int kDecodeMaxTokens = 64;
// zt[split * t + m][i][l] = partial of sum_k W[m][l][k] Y[m][i][k]; one or two layers in one launch
struct DecodeProblem { int K_r; const void* Y; const void* W; float* zt; int splits; };
int tc_decode_splits(int K_r, int K_r_min, int T);
constexpr int kDecodeMaxSplits = 4;
cudaError_t launch_tc_forward_decode(int t, int T, int h, const DecodeProblem* pr, int n, cudaStream_t st);

// ---- row kernels ------------------------------------------------------------
struct RowFwdArgs {
  const void *zs, *zp, *R, *gamma, *beta;
  void *Hn, *X;
  float *rstd, *mean;
  int t, T, h, S, S_lo, S_hi, P;
  float alpha, eps;
  int norm;
  // compact residual layout (S a multiple of 8, so S_lo = S_hi = S): the shared channels of the
  // stream exist once, Rs / Hns [T, S]; R / Hn then hold the private parts [t, T, P]
  int compact;
  const void* Rs;
  void* Hns;
};
// direct: 0 = automatic (warp-per-token kernels for short rows, else the bulk-copy staged kernels
// whenever a ring of at least two stages fits in shared memory), 1 = plain-load kernels,
// 2 = staged kernels even for short rows.
cudaError_t launch_rows_forward(const RowFwdArgs& a, caat_dtype dtype, int direct, cudaStream_t st);
cudaError_t launch_rows_forward_staged(const RowFwdArgs& a, caat_dtype dtype, cudaStream_t st);
// forward row work from fp32 partial planes (decode); with two layers the second layer's residual is
// the first layer's new residual stream (as stored), both layers in one launch
struct PartialLayer {
  const float* zt; int splits; const void* gamma; const void* beta; void* Hn; void* X; float* rstd; float* mean;
  void* Hns;   // compact layout: the shared part of this layer's new stream, [T, S]; Hn then holds the private parts
};
struct RowPartArgs {
  PartialLayer L[2];
  int nlayers;
  const void* R;
  int t, T, h, S;
  float alpha, eps;
  int norm;
  int compact;      // R / Hn are [t, T, h - S] private parts, Rs / Hns [T, S] the shared part stored once
  const void* Rs;
};
cudaError_t launch_rows_forward_partials(const RowPartArgs& a, caat_dtype dtype, cudaStream_t st);
// warp-per-token kernels for short rows (h <= 1024 in bf16); rows_warp_cpt == 0: not applicable
int rows_warp_cpt(int h, int t, caat_dtype dtype);
cudaError_t launch_rows_forward_warp(const RowFwdArgs& a, caat_dtype dtype, cudaStream_t st);
bool rows_staged_usable(int h, int t, int S_lo, int S_hi, caat_dtype dtype, bool backward);

struct RowBwdArgs {
  const void *dX, *dHn, *Hn, *gamma;
  const float *rstd, *mean;
  void *dR, *gs, *zp;      // zp may be NULL: the scaled private copy is then not written (the GEMMs read dR)
  float *dgpart, *dbpart;  // [rows, h]
  float *dgamma, *dbeta;   // [h]
  int t, T, h, S, S_lo, S_hi, P;
  float alpha;
  int norm;
  // compact residual layout: Hns / dHns [T, S] exist once; Hn, dHn, dR hold the private parts
  // [t, T, P]; the shared residual gradient is gs itself (dRs = dZt on the shared channels)
  int compact;
  const void *Hns, *dHns;
  int reduce_mode;   // CAAT_OPT_BACKWARD_REDUCE (plain-load kernels only)
  // optional side job of the norm-gradient reduction launch: w_dst[m][l][:] = alpha * w_src[m][l][:] for the
  // private rows l >= S of the layer's weights [t, h, w_Kr] (bf16), which the data gradient reads next
  const void* w_src;
  void* w_dst;
  int w_Kr;
  // exchange of the gradient slab over peer memory: gs_slice > 0 sends row i of the reduced shared gradient to slot
  // gs_rank of GPU i / gs_slice (gs_recv[q] = that GPU's receive buffer [world][gs_slice][S]) instead of to gs
  int gs_slice, gs_rank;
  void* gs_recv[CAAT_MAX_PEERS];
};
#ifdef __CUDACC__
// where row i of the reduced shared gradient goes (S_hi == S whenever the slab is exchanged)
__device__ __forceinline__ char* gs_row(const RowBwdArgs& a, long long i, int ES) {
  if (a.gs_slice > 0) {
    const int q = (int)(i / a.gs_slice);
    return static_cast<char*>(a.gs_recv[q]) + (((long long)a.gs_rank * a.gs_slice + (i - (long long)q * a.gs_slice)) * a.S_hi) * ES;
  }
  return static_cast<char*>(a.gs) + i * a.S_hi * ES;
}
#endif
cudaError_t launch_rows_backward(const RowBwdArgs& a, caat_dtype dtype, int direct, cudaStream_t st);
cudaError_t launch_rows_backward_staged(const RowBwdArgs& a, caat_dtype dtype, int max_rows, int* rows_used,
                                        cudaStream_t st);
cudaError_t launch_rows_backward_warp(const RowBwdArgs& a, caat_dtype dtype, int max_rows, int* rows_used,
                                      cudaStream_t st);
int rows_backward_partial_rows(int h, int T, caat_dtype dtype);
// Wait limit of the bulk-copy row kernels and the switch of their time-out test, read once per process from the
// environment: CAAT_ROWS_SPINCAP (polls of one mbarrier wait, default 2^18; each poll may sleep up to 20 us in
// hardware) and CAAT_ROWS_STALL=1 (every stage announces 16 bytes that never arrive, so the first wait runs out:
// the kernels must raise the status word, let their copies land and return).  Neither changes a result of a call
// that returns CAAT_OK.
struct RowsHooks { uint32_t spin_cap; int stall; };
RowsHooks rows_hooks();

// ---- activation of the column-parallel half (streaming kernels) ---------------
// gated: pre has 2 * width_out columns [gate | up], Y = silu(gate) * up; else Y = silu(pre)
cudaError_t launch_act_forward(caat_dtype dtype, int gated, const void* pre, void* Y, long long rows, int width_out,
                               cudaStream_t st);
cudaError_t launch_act_backward(caat_dtype dtype, int gated, const void* dY, const void* pre, void* dpre,
                                long long rows, int width_out, cudaStream_t st);

// ---- programmatic dependent launch --------------------------------------------
// Kernels launched through launch_pdl may be scheduled while their predecessor in the stream is still
// draining: their CTAs set up shared memory, barriers and tensor memory, then call pdl_wait(), which
// returns once the predecessor has completed and its writes are visible.  Nothing that reads or writes
// global memory may precede pdl_wait().  (Without the launch attribute the instruction returns at once.)
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
#endif
bool pdl_enabled();   // CAAT_PDL=0 in the environment switches the launch attribute off (measurements)
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr{};
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = pdl_enabled() ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// first half of the backward (row kernel, norm-gradient reduction) with the gradient slab's rows sent to the
// owners' receive slots
caat_status tp_backward_local_push_impl(const caat_ctx* ctx, caat_layer layer, int tokens, const void* dX, const void* dHn,
                                        const void* W, const void* Hn, const float* rstd, const float* mean,
                                        const void* gamma, void* dR, float* dgamma, float* dbeta, void* workspace,
                                        size_t workspace_bytes, cudaStream_t st, const PushTarget& push);

// ---- launch limits ---------------------------------------------------------------
// A block call runs a layer's HBM-bound row kernel beside the other layer's tensor-bound GEMMs by giving
// each a share of the GPU: the row kernel is held to a few CTAs, the GEMM to the remaining workers.  The limits
// are a property of the launching host thread for the duration of one launch call (0 = no limit).
struct LaunchLimits {
  int gemm_workers = 0;   // CTAs of a tensor-core GEMM launch, at most
  int gemm_smem = 0;      // dynamic shared memory of a GEMM CTA, at most (bytes): fewer pipeline stages
  int rows_ctas = 0;      // CTAs of a row-kernel launch, at most
  int rows_per_sm = 0;    // resident row-kernel CTAs per SM the shared-memory ring is sized for
  int rows_smem = 0;      // shared memory the row kernel's CTAs of one SM may use together (bytes)
};
LaunchLimits& launch_limits();                  // this host thread's current limits
const LaunchLimits effective_limits();          // the above, or a measurement build's environment overrides
struct ScopedLimits {
  LaunchLimits saved;
  explicit ScopedLimits(const LaunchLimits& l) : saved(launch_limits()) { launch_limits() = l; }
  ~ScopedLimits() { launch_limits() = saved; }
};

// ---- bookkeeping ------------------------------------------------------------
// Brackets one kernel launch: counts it and, while profiling is on, records a CUDA event
// before and after it on the launching stream.
struct LaunchScope {
  LaunchScope(int kind, cudaStream_t st);
  ~LaunchScope();
  int slot;
  cudaStream_t st;
};
// One lock for the library's small host-side caches (per-device attribute flags, looked-up addresses and
// occupancy answers): calls from several host threads may run concurrently, the caches are filled under it.
std::mutex& host_cache_mutex();
caat_status cuda_fail(cudaError_t e);  // records the error text for caat_last_cuda_error(), returns CAAT_ECUDA
unsigned int* device_status_word();  // device address of the status word (per device)
int sm_count();                       // multiprocessors of the current device (grids are sized in multiples of it)

}  // namespace caat
