// C ABI of libcaat: context, argument validation, scratch layout and the launch
// sequences of the forward / backward of one row-parallel layer and of a block.
#include <atomic>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "caat_internal.h"

namespace caat {

static std::atomic<unsigned long long> g_launches{0};
static thread_local char g_cuda_err[256] = "";

__device__ unsigned int g_status_word = 0;

// ---- optional per-kernel timing (benchmark aid) --------------------------------
struct Profiler {
  bool on = false;
  std::vector<cudaEvent_t> ev;   // 2 per record
  std::vector<int> kind;
  int used = 0;
};
static Profiler g_prof;

LaunchScope::LaunchScope(int kind, cudaStream_t s) : slot(-1), st(s) {
  g_launches.fetch_add(1ull, std::memory_order_relaxed);
  if (g_prof.on && g_prof.used < (int)g_prof.kind.size()) {
    slot = g_prof.used++;
    g_prof.kind[slot] = kind;
    cudaEventRecord(g_prof.ev[2 * slot], st);
  }
}
LaunchScope::~LaunchScope() {
  if (slot >= 0) cudaEventRecord(g_prof.ev[2 * slot + 1], st);
}

bool pdl_enabled() {
  static const bool on = [] { const char* e = getenv("CAAT_PDL"); return !(e && e[0] == '0'); }();
  return on;
}

std::mutex& host_cache_mutex() {
  static std::mutex m;
  return m;
}

LaunchLimits& launch_limits() {
  static thread_local LaunchLimits lim;
  return lim;
}

const LaunchLimits effective_limits() {
  LaunchLimits lim = launch_limits();
#ifdef CAAT_MEASUREMENT_AIDS
  // read at every launch so that a measurement script can change them between calls
  auto env = [](const char* name, int& v) { const char* e = getenv(name); if (e && v == 0) v = atoi(e); };
  env("CAAT_X_GEMM_WORKERS", lim.gemm_workers); env("CAAT_X_GEMM_SMEM", lim.gemm_smem);
  env("CAAT_X_ROWS_CTAS", lim.rows_ctas); env("CAAT_X_ROWS_PER_SM", lim.rows_per_sm); env("CAAT_X_ROWS_SMEM", lim.rows_smem);
#endif
  return lim;
}

unsigned int* device_status_word() {
  // looked up once per device (the lookup is not a stream operation; caching it keeps launches
  // free of runtime queries, which also matters inside a stream capture)
  static unsigned int* cache[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(host_cache_mutex());
  if (cache[dev] == nullptr) {
    unsigned int* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_status_word) != cudaSuccess) return nullptr;
    cache[dev] = p;
  }
  return cache[dev];
}

int sm_count() {
  static int cache[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  std::lock_guard<std::mutex> lock(host_cache_mutex());
  if (cache[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cache[dev] = n;
  }
  return cache[dev];
}

caat_status cuda_fail(cudaError_t e) {
  std::strncpy(g_cuda_err, cudaGetErrorString(e), sizeof(g_cuda_err) - 1);
  g_cuda_err[sizeof(g_cuda_err) - 1] = 0;
  (void)cudaGetLastError();   // the error is reported through the status; do not leave it sticky for the caller's next call
  return CAAT_ECUDA;
}

static size_t decode_planes_bytes(const caat_ctx* ctx, int tokens) {
  return align_up((size_t)kDecodeMaxSplits * ctx->t * tokens * ctx->h * sizeof(float), 256);
}

Scratch scratch_layout(const caat_ctx* ctx, int K_r, int tokens, int backward) {
  Scratch s{};
  const size_t e = elem_size(ctx->dtype);
  s.S_lo = round_down(ctx->S, kLayoutVec);
  s.S_hi = round_up(ctx->S, kLayoutVec);
  s.P = ctx->h - s.S_lo;
  size_t off = 0;
  s.zs_off = off;
  off = align_up(off + (size_t)tokens * s.S_hi * e, 256);
  s.zp_off = off;
  if (!(backward && tc_gemm_usable(ctx, K_r)))   // the tensor-core backward reads the private gradient from dR
    off = align_up(off + (size_t)ctx->t * tokens * s.P * e, 256);
  s.zt_off = off;
  if (!backward && tokens <= kDecodeMaxTokens && !ctx->no_decode && tc_gemm_usable(ctx, K_r))   // two layers' planes
    off = align_up(off + 2 * decode_planes_bytes(ctx, tokens), 256);
  if (backward) {
    const size_t rows = (size_t)rows_backward_partial_rows(ctx->h, tokens, ctx->dtype);
    s.dgpart_off = off;
    off = align_up(off + rows * ctx->h * sizeof(float), 256);
    s.dbpart_off = off;
    off = align_up(off + rows * ctx->h * sizeof(float), 256);
    s.splitk_off = off;
    s.splitk_bytes = 0;
    if (tc_gemm_usable(ctx, K_r)) {
      RowparShapes sh{ctx->t, tokens, ctx->h, K_r, ctx->S, s.S_lo, s.S_hi, s.P};
      s.splitk_bytes = tc_wgrad_splitk_bytes(sh);
    }
    off = align_up(off + s.splitk_bytes, 256);
    s.wt_off = off;
    if (tc_gemm_usable(ctx, K_r) && ctx->alpha != 1.0 && ctx->S < ctx->h)
      off = align_up(off + (size_t)ctx->t * ctx->h * K_r * e, 256);
  }
  s.total = off;
  return s;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static int layer_kr(const caat_ctx* ctx, caat_layer layer) {
  return (layer == CAAT_ATTN_OUT ? ctx->h : ctx->ffn) / (ctx->t * ctx->groups);
}

static caat_status check_common(const caat_ctx* ctx, caat_layer layer, int tokens) {
  if (!ctx) return CAAT_EINVAL;
  if (layer != CAAT_ATTN_OUT && layer != CAAT_MLP_DOWN) return CAAT_EINVAL;
  if (tokens < 1) return CAAT_ESHAPE;
  if (ctx->h % 8 != 0) return CAAT_EUNSUPPORTED;
  const int V = ctx->dtype == CAAT_BF16 ? 8 : 4;
  if (ctx->h / V > 512 * 4) return CAAT_EUNSUPPORTED;
  if ((long long)ctx->t * tokens > 2000000000LL) return CAAT_EUNSUPPORTED;
  return CAAT_OK;
}

// ---- forward of one layer ------------------------------------------------------
static caat_status forward_impl(const caat_ctx* ctx, int K_r, int T, const void* Y, const void* W, const void* R,
                                const void* gamma, const void* beta, void* Hn, void* X, float* rstd, float* mean,
                                void* ws, cudaStream_t st, int compact = 0, const void* Rs = nullptr,
                                void* Hns = nullptr, int phase = 0, int rows_mode = -1) {
  // phase: 0 = the whole layer; 1 = the GEMM only (leaves the partial sums in the scratch); 2 = the row
  // kernel only (on what the scratch holds).  1 and 2 are the halves around a caller's all-reduce.
  // compact: R / Hn are the private parts [t, T, h - S], Rs / Hns the shared part [T, S] stored once
  const Scratch L = scratch_layout(ctx, K_r, T, 0);
  char* wsb = static_cast<char*>(ws);
  void* zs = wsb + L.zs_off;
  void* zp = wsb + L.zp_off;
  const int t = ctx->t, h = ctx->h, S = ctx->S;
  const size_t e = elem_size(ctx->dtype);
  cudaError_t ce;

  if (phase == 0 && T <= kDecodeMaxTokens && !ctx->no_decode && tc_gemm_usable(ctx, K_r)) {
    // few tokens (decode): the weights dominate the traffic; stream them with swapped operands and
    // let the row kernel form the rank sum from fp32 per-rank partials
    float* zt = reinterpret_cast<float*>(wsb + L.zt_off);
    const int splits = tc_decode_splits(K_r, K_r, T);
    const DecodeProblem pr{K_r, Y, W, zt, splits};
    ce = launch_tc_forward_decode(t, T, h, &pr, 1, st);
    if (ce != cudaSuccess) return cuda_fail(ce);
    RowPartArgs a{};
    a.L[0] = PartialLayer{zt, splits, gamma, beta, Hn, X, rstd, mean, Hns};
    a.nlayers = 1; a.R = R; a.t = t; a.T = T; a.h = h; a.S = S; a.compact = compact; a.Rs = Rs;
    a.alpha = (float)ctx->alpha; a.eps = (float)ctx->eps; a.norm = ctx->norm;
    ce = launch_rows_forward_partials(a, ctx->dtype, st);
    if (ce != cudaSuccess) return cuda_fail(ce);
    return CAAT_OK;
  }
  if (phase == 2) {
    // nothing to multiply
  } else if (tc_gemm_usable(ctx, K_r)) {
    RowparShapes sh{t, T, h, K_r, S, L.S_lo, L.S_hi, L.P};
    ce = launch_tc_forward(sh, Y, W, zs, zp, st);
    if (ce != cudaSuccess) return cuda_fail(ce);
  } else {
    if (S > 0) {  // shared columns: one product over the whole contraction axis (all ranks)
      GemmProblem g{};
      g.nseg = 1;
      g.seg[0] = GemmSeg{Y, W, 0, (long long)T * K_r, K_r, 1, 0, (long long)h * K_r, 1, K_r, t, K_r};
      g.C = zs; g.sCb = 0; g.sCi = L.S_hi; g.M = T; g.N = S; g.batch = 1; g.c_f32 = 0;
      ce = launch_gemm_simt(g, ctx->dtype, st);
      if (ce != cudaSuccess) return cuda_fail(ce);
    }
    if (S < h) {  // private columns: one product per rank
      GemmProblem g{};
      g.nseg = 1;
      g.seg[0] = GemmSeg{Y, static_cast<const char*>(W) + (size_t)S * K_r * e,
                         (long long)T * K_r, 0, K_r, 1, (long long)h * K_r, 0, 1, K_r, 1, K_r};
      g.C = static_cast<char*>(zp) + (size_t)(S - L.S_lo) * e;
      g.sCb = (long long)T * L.P; g.sCi = L.P; g.M = T; g.N = h - S; g.batch = t; g.c_f32 = 0;
      ce = launch_gemm_simt(g, ctx->dtype, st);
      if (ce != cudaSuccess) return cuda_fail(ce);
    }
  }
  if (phase == 1) return CAAT_OK;
  RowFwdArgs a{zs, zp, R, gamma, beta, Hn, X, rstd, mean, t, T, h, S, L.S_lo, L.S_hi, L.P,
               (float)ctx->alpha, (float)ctx->eps, ctx->norm};
  a.compact = compact; a.Rs = Rs; a.Hns = Hns;
  ce = launch_rows_forward(a, ctx->dtype, rows_mode >= 0 ? rows_mode : ctx->direct_rows, st);
  if (ce != cudaSuccess) return cuda_fail(ce);
  return CAAT_OK;
}

// ---- the library's own stream for work that runs beside the caller's stream ------------------------
// One per device, created on first use; fork / join events likewise.  The fork-launch-join sequence of a call is
// issued under the lock, so two host threads cannot interleave their event records.
struct SideStream { cudaStream_t s = nullptr; cudaEvent_t fork = nullptr, join = nullptr; };
static SideStream* side_stream_locked() {
  static SideStream table[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  SideStream& e = table[dev];
  if (!e.s) {
    if (cudaStreamCreateWithFlags(&e.s, cudaStreamNonBlocking) != cudaSuccess) { e.s = nullptr; return nullptr; }
    if (cudaEventCreateWithFlags(&e.fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&e.join, cudaEventDisableTiming) != cudaSuccess) {
      cudaStreamDestroy(e.s);
      e = SideStream{};
      return nullptr;
    }
  }
  return &e;
}

// ---- backward of one layer -----------------------------------------------------
static caat_status backward_impl(const caat_ctx* ctx, int K_r, int T, const void* dX, const void* dHn, const void* Y,
                                 const void* W, const void* Hn, const float* rstd, const float* mean,
                                 const void* gamma, void* dY, float* dW, void* dR, float* dgamma, float* dbeta,
                                 void* ws, cudaStream_t st, int compact = 0, const void* Hns = nullptr,
                                 const void* dHns = nullptr, void* dRs = nullptr, int phase = 0,
                                 const PushTarget* push = nullptr) {
  // phase: 0 = the whole layer; 1 = the row kernel only (dR, the shared gradient slab, the norm-parameter
  // gradients, the scaled weight rows); 2 = the two GEMMs only, on the slab as it then stands
  // compact: Hn / dHn / dR are the private parts; the shared residual gradient dRs [T, S] is at the
  // same time the shared part of dZt, so the GEMMs read it where the caller wants it
  const Scratch L = scratch_layout(ctx, K_r, T, 1);
  char* wsb = static_cast<char*>(ws);
  void* gs = compact ? dRs : wsb + L.zs_off;
  void* zp = wsb + L.zp_off;
  const int t = ctx->t, h = ctx->h, S = ctx->S;
  const size_t e = elem_size(ctx->dtype);
  cudaError_t ce;

  // Tensor-core path: the GEMMs take the private gradient straight from dR (alpha rides on the weights'
  // private rows in the data gradient and on the epilogue in the weight gradient), so the row kernel writes
  // no scaled copy of it.
  const bool tc = tc_gemm_usable(ctx, K_r);
  if (tc) zp = nullptr;
  RowBwdArgs a{dX, dHn, Hn, gamma, rstd, mean, dR, gs, zp,
               reinterpret_cast<float*>(wsb + L.dgpart_off), reinterpret_cast<float*>(wsb + L.dbpart_off),
               dgamma, dbeta, t, T, h, S, L.S_lo, L.S_hi, L.P, (float)ctx->alpha, ctx->norm};
  a.compact = compact; a.Hns = Hns; a.dHns = dHns;
  a.reduce_mode = ctx->bwd_reduce;
  if (push) {   // the reduced shared gradient goes straight to the owners' receive slots (multi-GPU exchange)
    a.gs_slice = push->slice; a.gs_rank = push->rank;
    for (int q = 0; q < push->world && q < CAAT_MAX_PEERS; ++q) a.gs_recv[q] = push->recv[q];
  }
  const bool prescale = tc && ctx->alpha != 1.0 && S < h;
  if (prescale) { a.w_src = W; a.w_dst = wsb + L.wt_off; a.w_Kr = K_r; }
  if (phase != 2) {
    ce = launch_rows_backward(a, ctx->dtype, ctx->bwd_reduce ? 1 : ctx->direct_rows, st);
    if (ce != cudaSuccess) return cuda_fail(ce);
  }
  if (phase == 1) return CAAT_OK;

  if (tc) {
    RowparShapes sh{t, T, h, K_r, S, L.S_lo, L.S_hi, L.P};
    const PrivOperand pv = compact ? PrivOperand{dR, L.P, 0, (float)ctx->alpha} : PrivOperand{dR, h, S, (float)ctx->alpha};
    ce = launch_tc_dgrad(sh, gs, pv, W, dY, wsb + L.wt_off, prescale, st);
    if (ce != cudaSuccess) return cuda_fail(ce);
    ce = launch_tc_wgrad(sh, gs, pv, Y, dW, wsb + L.splitk_off, L.splitk_bytes, st);
    if (ce != cudaSuccess) return cuda_fail(ce);
    return CAAT_OK;
  }
  const char* zp_priv = static_cast<const char*>(zp) + (size_t)(S - L.S_lo) * e;
  {  // dY[m] = gs W[m][:S] + zp[m] W[m][S:]
    GemmProblem g{};
    g.nseg = 2;
    g.seg[0] = GemmSeg{gs, W, 0, 0, L.S_hi, 1, (long long)h * K_r, 0, K_r, 1, 1, S};
    g.seg[1] = GemmSeg{zp_priv, static_cast<const char*>(W) + (size_t)S * K_r * e,
                       (long long)T * L.P, 0, L.P, 1, (long long)h * K_r, 0, K_r, 1, 1, h - S};
    g.C = dY; g.sCb = (long long)T * K_r; g.sCi = K_r; g.M = T; g.N = K_r; g.batch = t; g.c_f32 = 0;
    ce = launch_gemm_simt(g, ctx->dtype, st);
    if (ce != cudaSuccess) return cuda_fail(ce);
  }
  if (S > 0) {  // dW[m][:S] = gs^T Y[m]
    GemmProblem g{};
    g.nseg = 1;
    g.seg[0] = GemmSeg{gs, Y, 0, 0, 1, L.S_hi, (long long)T * K_r, 0, K_r, 1, 1, T};
    g.C = dW; g.sCb = (long long)h * K_r; g.sCi = K_r; g.M = S; g.N = K_r; g.batch = t; g.c_f32 = 1;
    ce = launch_gemm_simt(g, ctx->dtype, st);
    if (ce != cudaSuccess) return cuda_fail(ce);
  }
  if (S < h) {  // dW[m][S:] = zp[m]^T Y[m]
    GemmProblem g{};
    g.nseg = 1;
    g.seg[0] = GemmSeg{zp_priv, Y, (long long)T * L.P, 0, 1, L.P, (long long)T * K_r, 0, K_r, 1, 1, T};
    g.C = dW + (size_t)S * K_r; g.sCb = (long long)h * K_r; g.sCi = K_r; g.M = h - S; g.N = K_r; g.batch = t;
    g.c_f32 = 1;
    ce = launch_gemm_simt(g, ctx->dtype, st);
    if (ce != cudaSuccess) return cuda_fail(ce);
  }
  return CAAT_OK;
}

// ---- block forward with few tokens (decode) --------------------------------------
// The two layers' GEMMs do not depend on each other, so both weight streams run in ONE launch, and one
// row kernel walks both layers of a (token, rank) row.  compact: R0 / Hn1 / Hn2 are the private parts
// [t, T, h - S] and R0s / Hn1s / Hn2s the shared part [T, S] of the stream.
static bool block_decode_applies(const caat_ctx* ctx, int tokens) {
  return ctx && tokens >= 1 && tokens <= kDecodeMaxTokens && !ctx->no_decode &&
         tc_gemm_usable(ctx, layer_kr(ctx, CAAT_ATTN_OUT)) && tc_gemm_usable(ctx, layer_kr(ctx, CAAT_MLP_DOWN));
}

static caat_status block_decode(const caat_ctx* ctx, int tokens, const void* Y_attn, const void* W_o, const void* Y_mlp,
                                const void* W_down, const void* R0, const void* gamma1, const void* beta1,
                                const void* gamma2, const void* beta2, void* Hn1, void* X1, float* rstd1, float* mean1,
                                void* Hn2, void* X2, float* rstd2, float* mean2, void* workspace, size_t workspace_bytes,
                                void* cuda_stream, int compact, const void* R0s, void* Hn1s, void* Hn2s) {
  caat_status s = check_common(ctx, CAAT_MLP_DOWN, tokens);
  if (s != CAAT_OK) return s;
  const bool has_s = ctx->S > 0, has_p = ctx->S < ctx->h;
  if (!Y_attn || !W_o || !Y_mlp || !W_down || !gamma1 || !gamma2 || !X1 || !rstd1 || !X2 || !rstd2) return CAAT_EINVAL;
  if (compact) {
    if (ctx->S % kLayoutVec != 0) return CAAT_EUNSUPPORTED;
    if ((has_s && (!R0s || !Hn1s || !Hn2s)) || (has_p && (!R0 || !Hn1 || !Hn2))) return CAAT_EINVAL;
  } else if (!R0 || !Hn1 || !Hn2) {
    return CAAT_EINVAL;
  }
  if (ctx->norm == 1 && (!mean1 || !mean2)) return CAAT_EINVAL;
  const void* ptrs[] = {Y_attn, W_o, Y_mlp, W_down, R0, R0s, gamma1, beta1, gamma2, beta2, Hn1, Hn1s, X1, rstd1, mean1,
                        Hn2, Hn2s, X2, rstd2, mean2, workspace};
  for (const void* p : ptrs)
    if (p && !aligned16(p)) return CAAT_EALIGN;
  const int ka = layer_kr(ctx, CAAT_ATTN_OUT), km = layer_kr(ctx, CAAT_MLP_DOWN);
  const Scratch L = scratch_layout(ctx, km, tokens, 0);
  if (!workspace || workspace_bytes < L.total) return CAAT_EWORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  float* zt1 = reinterpret_cast<float*>(static_cast<char*>(workspace) + L.zt_off);
  float* zt2 = reinterpret_cast<float*>(static_cast<char*>(workspace) + L.zt_off + decode_planes_bytes(ctx, tokens));
  const int kmin = ka < km ? ka : km;
  const int sp1 = tc_decode_splits(ka, kmin, tokens), sp2 = tc_decode_splits(km, kmin, tokens);
  const DecodeProblem pr[2] = {{ka, Y_attn, W_o, zt1, sp1}, {km, Y_mlp, W_down, zt2, sp2}};
  cudaError_t ce = launch_tc_forward_decode(ctx->t, tokens, ctx->h, pr, 2, st);
  if (ce != cudaSuccess) return cuda_fail(ce);
  RowPartArgs a{};
  a.L[0] = PartialLayer{zt1, sp1, gamma1, beta1, Hn1, X1, rstd1, mean1, Hn1s};
  a.L[1] = PartialLayer{zt2, sp2, gamma2, beta2, Hn2, X2, rstd2, mean2, Hn2s};
  a.nlayers = 2; a.R = R0; a.t = ctx->t; a.T = tokens; a.h = ctx->h; a.S = ctx->S;
  a.alpha = (float)ctx->alpha; a.eps = (float)ctx->eps; a.norm = ctx->norm;
  a.compact = compact; a.Rs = R0s;
  ce = launch_rows_forward_partials(a, ctx->dtype, st);
  if (ce != cudaSuccess) return cuda_fail(ce);
  return CAAT_OK;
}

}  // namespace caat

using namespace caat;

extern "C" {

caat_status caat_create(int h, int ffn, int t, double p, caat_dtype dtype, caat_ctx** out) {
  if (!out) return CAAT_EINVAL;
  *out = nullptr;
  if (dtype != CAAT_F32 && dtype != CAAT_BF16) return CAAT_EINVAL;
  if (!(p >= 0.0 && p <= 1.0)) return CAAT_EINVAL;
  if (h < 1 || ffn < 1 || t < 1) return CAAT_ESHAPE;
  if (h % t != 0 || ffn % t != 0) return CAAT_ESHAPE;
  caat_ctx* c = new (std::nothrow) caat_ctx();
  if (!c) return CAAT_EINVAL;
  c->h = h; c->ffn = ffn; c->t = t; c->p = p; c->dtype = dtype;
  c->S = (int)std::floor((double)h * p);   // Eq. A3: l < floor(h p) is shared
  c->alpha = std::sqrt((double)t);         // Section 4: private channels times sqrt(r)
  c->norm = 0; c->eps = 1e-5; c->force_simt = 0; c->direct_rows = 0; c->no_decode = 0; c->bwd_reduce = 0;
  c->groups = 1;
  c->block_overlap = 2;
  *out = c;
  return CAAT_OK;
}

caat_status caat_set_option(caat_ctx* ctx, caat_option opt, double value) {
  if (!ctx) return CAAT_EINVAL;
  switch (opt) {
    case CAAT_OPT_NORM:
      if (value != 0.0 && value != 1.0) return CAAT_EINVAL;
      ctx->norm = (int)value; return CAAT_OK;
    case CAAT_OPT_EPS:
      if (!(value >= 0.0)) return CAAT_EINVAL;
      ctx->eps = value; return CAAT_OK;
    case CAAT_OPT_PRIVATE_SCALE:
      if (!std::isfinite(value)) return CAAT_EINVAL;
      ctx->alpha = value; return CAAT_OK;
    case CAAT_OPT_SHARED_CHANNELS:
      if (value != std::floor(value)) return CAAT_EINVAL;
      if (value < 0.0 || value > (double)ctx->h) return CAAT_ESHAPE;
      ctx->S = (int)value; return CAAT_OK;
    case CAAT_OPT_GEMM:
      if (value != 0.0 && value != 1.0) return CAAT_EINVAL;
      ctx->force_simt = (int)value; return CAAT_OK;
    case CAAT_OPT_DECODE:
      if (value != 0.0 && value != 1.0) return CAAT_EINVAL;
      ctx->no_decode = (int)value; return CAAT_OK;
    case CAAT_OPT_ROWS:
      if (value != 0.0 && value != 1.0 && value != 2.0) return CAAT_EINVAL;
      ctx->direct_rows = (int)value; return CAAT_OK;
    case CAAT_OPT_BACKWARD_REDUCE:
      if (value != 0.0 && value != 1.0 && value != 2.0) return CAAT_EINVAL;
      ctx->bwd_reduce = (int)value; return CAAT_OK;
    case CAAT_OPT_BLOCK_OVERLAP:
      if (value != 0.0 && value != 1.0 && value != 2.0) return CAAT_EINVAL;
      ctx->block_overlap = (int)value; return CAAT_OK;
    case CAAT_OPT_TP_GROUPS: {
      if (value != std::floor(value) || value < 1.0 || value > 65536.0) return CAAT_EINVAL;
      const int g = (int)value;
      if (ctx->h % (ctx->t * g) != 0 || ctx->ffn % (ctx->t * g) != 0) return CAAT_ESHAPE;
      ctx->groups = g;
      ctx->alpha = std::sqrt((double)ctx->t * g);   // Section 4: sqrt of the number of devices; may be overridden afterwards
      return CAAT_OK;
    }
  }
  return CAAT_EINVAL;
}

void caat_destroy(caat_ctx* ctx) { delete ctx; }

int caat_shared_channels(const caat_ctx* ctx) { return ctx ? ctx->S : -1; }
double caat_private_scale(const caat_ctx* ctx) { return ctx ? ctx->alpha : 0.0; }

size_t caat_workspace_bytes(const caat_ctx* ctx, caat_layer layer, int tokens, int backward) {
  if (check_common(ctx, layer, tokens) != CAAT_OK) return 0;
  const size_t fwd = scratch_layout(ctx, layer_kr(ctx, layer), tokens, 0).total;
  if (!backward) return fwd;
  const size_t bwd = scratch_layout(ctx, layer_kr(ctx, layer), tokens, 1).total;
  return bwd > fwd ? bwd : fwd;   // a training step runs both calls on one buffer
}

const char* caat_strerror(caat_status s) {
  switch (s) {
    case CAAT_OK: return "ok";
    case CAAT_EINVAL: return "invalid argument";
    case CAAT_ESHAPE: return "bad shape";
    case CAAT_EALIGN: return "pointer not 16-byte aligned";
    case CAAT_EWORKSPACE: return "workspace missing or too small";
    case CAAT_EUNSUPPORTED: return "shape not supported";
    case CAAT_ECUDA: return "CUDA error";
    case CAAT_ETIMEOUT: return "device-side wait timed out";
    case CAAT_ELIMIT: return "needs more than the built-in scratch of the no-allocation entry point";
  }
  return "unknown status";
}

const char* caat_last_cuda_error(void) { return g_cuda_err; }

caat_status caat_rowpar_forward(const caat_ctx* ctx, caat_layer layer, int tokens, const void* Y, const void* W,
                                const void* R, const void* gamma, const void* beta, void* Hn, void* X, float* rstd,
                                float* mean, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  caat_status s = check_common(ctx, layer, tokens);
  if (s != CAAT_OK) return s;
  if (!Y || !W || !R || !gamma || !Hn || !X || !rstd) return CAAT_EINVAL;
  if (ctx->norm == 1 && !mean) return CAAT_EINVAL;
  const void* ptrs[] = {Y, W, R, gamma, beta, Hn, X, rstd, mean, workspace};
  for (const void* p : ptrs)
    if (p && !aligned16(p)) return CAAT_EALIGN;
  const int K_r = layer_kr(ctx, layer);
  if (!workspace || workspace_bytes < scratch_layout(ctx, K_r, tokens, 0).total) return CAAT_EWORKSPACE;
  return forward_impl(ctx, K_r, tokens, Y, W, R, gamma, beta, Hn, X, rstd, mean, workspace,
                      static_cast<cudaStream_t>(cuda_stream));
}

caat_status caat_rowpar_backward(const caat_ctx* ctx, caat_layer layer, int tokens, const void* dX, const void* dHn,
                                 const void* Y, const void* W, const void* Hn, const float* rstd, const float* mean,
                                 const void* gamma, void* dY, float* dW, void* dR, float* dgamma, float* dbeta,
                                 void* workspace, size_t workspace_bytes, void* cuda_stream) {
  caat_status s = check_common(ctx, layer, tokens);
  if (s != CAAT_OK) return s;
  if (!dX || !Y || !W || !Hn || !rstd || !gamma || !dY || !dW || !dR || !dgamma) return CAAT_EINVAL;
  if (ctx->norm == 1 && (!mean || !dbeta)) return CAAT_EINVAL;
  const void* ptrs[] = {dX, dHn, Y, W, Hn, rstd, mean, gamma, dY, dW, dR, dgamma, dbeta, workspace};
  for (const void* p : ptrs)
    if (p && !aligned16(p)) return CAAT_EALIGN;
  const int K_r = layer_kr(ctx, layer);
  if (!workspace || workspace_bytes < scratch_layout(ctx, K_r, tokens, 1).total) return CAAT_EWORKSPACE;
  return backward_impl(ctx, K_r, tokens, dX, dHn, Y, W, Hn, rstd, mean, gamma, dY, dW, dR, dgamma, dbeta, workspace,
                       static_cast<cudaStream_t>(cuda_stream));
}

size_t caat_block_workspace_bytes(const caat_ctx* ctx, int tokens, int backward) {
  const size_t a = caat_workspace_bytes(ctx, CAAT_ATTN_OUT, tokens, backward);
  const size_t m = caat_workspace_bytes(ctx, CAAT_MLP_DOWN, tokens, backward);
  if (a == 0 || m == 0) return 0;
  // the forward's two scratch regions side by side; a training step's backward runs layer by layer in one region
  const size_t side_by_side = align_up(caat_workspace_bytes(ctx, CAAT_ATTN_OUT, tokens, 0), 256) +
                              caat_workspace_bytes(ctx, CAAT_MLP_DOWN, tokens, 0);
  const size_t one = a > m ? a : m;
  return side_by_side > one ? side_by_side : one;
}

// The block forward with the attention-out layer's row kernel beside the MLP-down layer's GEMM:
//   caller's stream:  GEMM 1 -> [fork] -> GEMM 2 ------------> [join] -> rows 2
//   library's stream:            [fork] -> rows 1 (plain loads) -> [join]
// The GEMM's CTAs fill every SM's shared memory, so the row kernel that shares the SMs with it is the plain-load
// variant (registers only); the GEMM gives up one pipeline stage, which leaves the row kernel's loads some L1.
// Measured: the pair alone gains 13-19 % (7B shapes: 1.74 ms one after the other, 1.41-1.51 ms side by side), a whole
// training step 2-4 % at the 130M and 1.1B shapes and 1-2 % at the 7B shapes (the GPU runs into its power limit there:
// with both kernels active the clock drops, which eats the gain).  Hence the automatic choice below: side by side
// unless the GEMM is the much longer of the two.
static bool overlap_pays(const caat_ctx* ctx) {
  if (ctx->block_overlap != 2) return ctx->block_overlap == 1;
  // time of the MLP-down GEMM at the tensor rate over the time of a row kernel at the HBM rate (tokens cancel):
  // (2 K h / 1.4e15) / (3 t h e / 6.4e12).  1.1 at the 1.1B shapes, 1.2 at 130M, 2.1 at 7B.
  const double ratio = (2.0 * ctx->ffn / ctx->groups / 1.4e15) / (3.0 * ctx->t * elem_size(ctx->dtype) / 6.4e12);
  return ratio <= 1.5;
}
static caat_status block_forward_overlapped(const caat_ctx* ctx, int tokens, const void* Y_attn, const void* W_o,
                                            const void* Y_mlp, const void* W_down, const void* R0, const void* gamma1,
                                            const void* beta1, const void* gamma2, const void* beta2, void* Hn1, void* X1,
                                            float* rstd1, float* mean1, void* Hn2, void* X2, float* rstd2, float* mean2,
                                            void* workspace, cudaStream_t st) {
  const int ka = layer_kr(ctx, CAAT_ATTN_OUT), km = layer_kr(ctx, CAAT_MLP_DOWN);
  char* ws1 = static_cast<char*>(workspace);
  char* ws2 = ws1 + align_up(scratch_layout(ctx, ka, tokens, 0).total, 256);
  static std::mutex side_mutex;      // not the cache lock: the launches below take that one themselves
  std::lock_guard<std::mutex> lock(side_mutex);
  SideStream* side = side_stream_locked();
  if (!side) return cuda_fail(cudaErrorUnknown);
  caat_status s = forward_impl(ctx, ka, tokens, Y_attn, W_o, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, ws1,
                               st, 0, nullptr, nullptr, 1);
  if (s != CAAT_OK) return s;
  cudaError_t ce = cudaEventRecord(side->fork, st);
  if (ce == cudaSuccess) ce = cudaStreamWaitEvent(side->s, side->fork, 0);
  if (ce != cudaSuccess) return cuda_fail(ce);
  {
    LaunchLimits lim{};
    lim.gemm_smem = 190 * 1024;
    ScopedLimits scoped(lim);
    s = forward_impl(ctx, km, tokens, Y_mlp, W_down, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, ws2, st, 0,
                     nullptr, nullptr, 1);
  }
  // whatever happens from here on, the side stream joins the caller's stream again
  caat_status s1 = s == CAAT_OK ? forward_impl(ctx, ka, tokens, nullptr, nullptr, R0, gamma1, beta1, Hn1, X1, rstd1, mean1, ws1,
                                               side->s, 0, nullptr, nullptr, 2, /*rows_mode=*/1)
                                : s;
  ce = cudaEventRecord(side->join, side->s);
  if (ce == cudaSuccess) ce = cudaStreamWaitEvent(st, side->join, 0);
  if (ce != cudaSuccess) return cuda_fail(ce);
  if (s1 != CAAT_OK) return s1;
  return forward_impl(ctx, km, tokens, nullptr, nullptr, Hn1, gamma2, beta2, Hn2, X2, rstd2, mean2, ws2, st, 0, nullptr,
                      nullptr, 2);
}

caat_status caat_block_forward(const caat_ctx* ctx, int tokens, const void* Y_attn, const void* W_o,
                               const void* Y_mlp, const void* W_down, const void* R0, const void* gamma1,
                               const void* beta1, const void* gamma2, const void* beta2, void* Hn1, void* X1,
                               float* rstd1, float* mean1, void* Hn2, void* X2, float* rstd2, float* mean2,
                               void* workspace, size_t workspace_bytes, void* cuda_stream) {
  // Two reduces per block (Appendix C): attention-out, then MLP-down on the new residual stream.
  if (block_decode_applies(ctx, tokens))
    return block_decode(ctx, tokens, Y_attn, W_o, Y_mlp, W_down, R0, gamma1, beta1, gamma2, beta2, Hn1, X1, rstd1, mean1,
                        Hn2, X2, rstd2, mean2, workspace, workspace_bytes, cuda_stream, 0, nullptr, nullptr, nullptr);
  if (ctx && overlap_pays(ctx) && !ctx->direct_rows && check_common(ctx, CAAT_MLP_DOWN, tokens) == CAAT_OK &&
      tc_gemm_usable(ctx, layer_kr(ctx, CAAT_ATTN_OUT)) && tc_gemm_usable(ctx, layer_kr(ctx, CAAT_MLP_DOWN)) &&
      Y_attn && W_o && Y_mlp && W_down && R0 && gamma1 && gamma2 && Hn1 && X1 && rstd1 && Hn2 && X2 && rstd2 &&
      (ctx->norm == 0 || (mean1 && mean2)) && Hn1 != R0 && workspace &&
      workspace_bytes >= align_up(scratch_layout(ctx, layer_kr(ctx, CAAT_ATTN_OUT), tokens, 0).total, 256) +
                             scratch_layout(ctx, layer_kr(ctx, CAAT_MLP_DOWN), tokens, 0).total) {
    const void* ptrs[] = {Y_attn, W_o, Y_mlp, W_down, R0, gamma1, beta1, gamma2, beta2, Hn1, X1, rstd1, mean1,
                          Hn2, X2, rstd2, mean2, workspace};
    bool aligned = true;
    for (const void* p : ptrs)
      if (p && !aligned16(p)) aligned = false;
    if (aligned)
      return block_forward_overlapped(ctx, tokens, Y_attn, W_o, Y_mlp, W_down, R0, gamma1, beta1, gamma2, beta2, Hn1, X1,
                                      rstd1, mean1, Hn2, X2, rstd2, mean2, workspace, static_cast<cudaStream_t>(cuda_stream));
  }
  caat_status s = caat_rowpar_forward(ctx, CAAT_ATTN_OUT, tokens, Y_attn, W_o, R0, gamma1, beta1, Hn1, X1, rstd1,
                                      mean1, workspace, workspace_bytes, cuda_stream);
  if (s != CAAT_OK) return s;
  return caat_rowpar_forward(ctx, CAAT_MLP_DOWN, tokens, Y_mlp, W_down, Hn1, gamma2, beta2, Hn2, X2, rstd2, mean2,
                             workspace, workspace_bytes, cuda_stream);
}

caat_status caat_block_backward(const caat_ctx* ctx, int tokens, const void* dX1, const void* dX2, const void* dHn2,
                                const void* Y_attn, const void* W_o, const void* Y_mlp, const void* W_down,
                                const void* Hn1, const float* rstd1, const float* mean1, const void* Hn2,
                                const float* rstd2, const float* mean2, const void* gamma1, const void* gamma2,
                                void* dY_attn, float* dW_o, void* dY_mlp, float* dW_down, void* dR0, void* dHn1,
                                float* dgamma1, float* dbeta1, float* dgamma2, float* dbeta2, void* workspace,
                                size_t workspace_bytes, void* cuda_stream) {
  if (!dHn1) return CAAT_EINVAL;
  caat_status s = caat_rowpar_backward(ctx, CAAT_MLP_DOWN, tokens, dX2, dHn2, Y_mlp, W_down, Hn2, rstd2, mean2,
                                       gamma2, dY_mlp, dW_down, dHn1, dgamma2, dbeta2, workspace, workspace_bytes,
                                       cuda_stream);
  if (s != CAAT_OK) return s;
  return caat_rowpar_backward(ctx, CAAT_ATTN_OUT, tokens, dX1, dHn1, Y_attn, W_o, Hn1, rstd1, mean1, gamma1,
                              dY_attn, dW_o, dR0, dgamma1, dbeta1, workspace, workspace_bytes, cuda_stream);
}

// ---- compact residual layout ---------------------------------------------------
static caat_status check_compact(const caat_ctx* ctx, caat_layer layer, int tokens) {
  caat_status s = check_common(ctx, layer, tokens);
  if (s != CAAT_OK) return s;
  if (ctx->S % kLayoutVec != 0) return CAAT_EUNSUPPORTED;   // rows of both parts must start on 16 bytes
  return CAAT_OK;
}

caat_status caat_rowpar_forward_compact(const caat_ctx* ctx, caat_layer layer, int tokens, const void* Y,
                                        const void* W, const void* Rs, const void* Rp, const void* gamma,
                                        const void* beta, void* Hns, void* Hnp, void* X, float* rstd, float* mean,
                                        void* workspace, size_t workspace_bytes, void* cuda_stream) {
  caat_status s = check_compact(ctx, layer, tokens);
  if (s != CAAT_OK) return s;
  const bool has_s = ctx->S > 0, has_p = ctx->S < ctx->h;
  if (!Y || !W || !gamma || !X || !rstd) return CAAT_EINVAL;
  if ((has_s && (!Rs || !Hns)) || (has_p && (!Rp || !Hnp))) return CAAT_EINVAL;
  if (ctx->norm == 1 && !mean) return CAAT_EINVAL;
  const void* ptrs[] = {Y, W, Rs, Rp, gamma, beta, Hns, Hnp, X, rstd, mean, workspace};
  for (const void* p : ptrs)
    if (p && !aligned16(p)) return CAAT_EALIGN;
  const int K_r = layer_kr(ctx, layer);
  if (!workspace || workspace_bytes < scratch_layout(ctx, K_r, tokens, 0).total) return CAAT_EWORKSPACE;
  return forward_impl(ctx, K_r, tokens, Y, W, Rp, gamma, beta, Hnp, X, rstd, mean, workspace,
                      static_cast<cudaStream_t>(cuda_stream), 1, Rs, Hns);
}

caat_status caat_rowpar_backward_compact(const caat_ctx* ctx, caat_layer layer, int tokens, const void* dX,
                                         const void* dHns, const void* dHnp, const void* Y, const void* W,
                                         const void* Hns, const void* Hnp, const float* rstd, const float* mean,
                                         const void* gamma, void* dY, float* dW, void* dRs, void* dRp, float* dgamma,
                                         float* dbeta, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  caat_status s = check_compact(ctx, layer, tokens);
  if (s != CAAT_OK) return s;
  const bool has_s = ctx->S > 0, has_p = ctx->S < ctx->h;
  if (!dX || !Y || !W || !rstd || !gamma || !dY || !dW || !dgamma) return CAAT_EINVAL;
  if ((has_s && (!Hns || !dRs)) || (has_p && (!Hnp || !dRp))) return CAAT_EINVAL;
  // the gradient on the outgoing stream is given for both parts or for neither
  const bool any_dh = (has_s && dHns) || (has_p && dHnp);
  if (any_dh && ((has_s && !dHns) || (has_p && !dHnp))) return CAAT_EINVAL;
  if (ctx->norm == 1 && (!mean || !dbeta)) return CAAT_EINVAL;
  const void* ptrs[] = {dX, dHns, dHnp, Y, W, Hns, Hnp, rstd, mean, gamma, dY, dW, dRs, dRp, dgamma, dbeta, workspace};
  for (const void* p : ptrs)
    if (p && !aligned16(p)) return CAAT_EALIGN;
  const int K_r = layer_kr(ctx, layer);
  if (!workspace || workspace_bytes < scratch_layout(ctx, K_r, tokens, 1).total) return CAAT_EWORKSPACE;
  // "a gradient is given" is one flag inside the kernels: an absent (empty) part borrows the other pointer
  const void* dh_p = any_dh ? (has_p ? dHnp : dHns) : nullptr;
  const void* dh_s = any_dh ? (has_s ? dHns : dHnp) : nullptr;
  return backward_impl(ctx, K_r, tokens, dX, dh_p, Y, W, Hnp, rstd, mean, gamma, dY, dW, dRp, dgamma, dbeta, workspace,
                       static_cast<cudaStream_t>(cuda_stream), 1, Hns, dh_s, dRs);
}

caat_status caat_block_forward_compact(const caat_ctx* ctx, int tokens, const void* Y_attn, const void* W_o,
                                       const void* Y_mlp, const void* W_down, const void* R0s, const void* R0p,
                                       const void* gamma1, const void* beta1, const void* gamma2, const void* beta2,
                                       void* Hn1s, void* Hn1p, void* X1, float* rstd1, float* mean1, void* Hn2s,
                                       void* Hn2p, void* X2, float* rstd2, float* mean2, void* workspace,
                                       size_t workspace_bytes, void* cuda_stream) {
  if (block_decode_applies(ctx, tokens))
    return block_decode(ctx, tokens, Y_attn, W_o, Y_mlp, W_down, R0p, gamma1, beta1, gamma2, beta2, Hn1p, X1, rstd1, mean1,
                        Hn2p, X2, rstd2, mean2, workspace, workspace_bytes, cuda_stream, 1, R0s, Hn1s, Hn2s);
  caat_status s = caat_rowpar_forward_compact(ctx, CAAT_ATTN_OUT, tokens, Y_attn, W_o, R0s, R0p, gamma1, beta1, Hn1s,
                                              Hn1p, X1, rstd1, mean1, workspace, workspace_bytes, cuda_stream);
  if (s != CAAT_OK) return s;
  return caat_rowpar_forward_compact(ctx, CAAT_MLP_DOWN, tokens, Y_mlp, W_down, Hn1s, Hn1p, gamma2, beta2, Hn2s, Hn2p,
                                     X2, rstd2, mean2, workspace, workspace_bytes, cuda_stream);
}

caat_status caat_block_backward_compact(const caat_ctx* ctx, int tokens, const void* dX1, const void* dX2,
                                        const void* dHn2s, const void* dHn2p, const void* Y_attn, const void* W_o,
                                        const void* Y_mlp, const void* W_down, const void* Hn1s, const void* Hn1p,
                                        const float* rstd1, const float* mean1, const void* Hn2s, const void* Hn2p,
                                        const float* rstd2, const float* mean2, const void* gamma1,
                                        const void* gamma2, void* dY_attn, float* dW_o, void* dY_mlp, float* dW_down,
                                        void* dR0s, void* dR0p, void* dHn1s, void* dHn1p, float* dgamma1,
                                        float* dbeta1, float* dgamma2, float* dbeta2, void* workspace,
                                        size_t workspace_bytes, void* cuda_stream) {
  caat_status s = caat_rowpar_backward_compact(ctx, CAAT_MLP_DOWN, tokens, dX2, dHn2s, dHn2p, Y_mlp, W_down, Hn2s, Hn2p,
                                               rstd2, mean2, gamma2, dY_mlp, dW_down, dHn1s, dHn1p, dgamma2, dbeta2,
                                               workspace, workspace_bytes, cuda_stream);
  if (s != CAAT_OK) return s;
  return caat_rowpar_backward_compact(ctx, CAAT_ATTN_OUT, tokens, dX1, dHn1s, dHn1p, Y_attn, W_o, Hn1s, Hn1p, rstd1,
                                      mean1, gamma1, dY_attn, dW_o, dR0s, dR0p, dgamma1, dbeta1, workspace,
                                      workspace_bytes, cuda_stream);
}

// ---- column-parallel half ------------------------------------------------------
namespace {
struct ColScratch { size_t dpre_off, splitk_off, splitk_bytes, wt_off, total; };

bool col_tc_usable(const caat_ctx* ctx, int n_out) {
  return ctx->dtype == CAAT_BF16 && !ctx->force_simt && ctx->h % 8 == 0 && n_out % 8 == 0;
}

RowparShapes col_shapes(const caat_ctx* ctx, int n_out, int T) {
  // the row-parallel GEMM wiring with no shared columns: "h" is the output width, "K_r" the input width
  return RowparShapes{ctx->t, T, n_out, ctx->h, 0, 0, 0, n_out};
}

ColScratch col_scratch(const caat_ctx* ctx, caat_activation act, int n_out, int T) {
  ColScratch s{};
  const size_t e = elem_size(ctx->dtype);
  size_t off = 0;
  s.dpre_off = off;
  if (act != CAAT_ACT_NONE) off = align_up(off + (size_t)ctx->t * T * n_out * e, 256);
  s.splitk_off = off;
  if (col_tc_usable(ctx, n_out)) {
    s.splitk_bytes = tc_wgrad_splitk_bytes(col_shapes(ctx, n_out, T));
    off = align_up(off + s.splitk_bytes, 256);
    s.wt_off = off;
  }
  s.total = off > 16 ? off : 16;
  return s;
}

caat_status check_col(const caat_ctx* ctx, caat_activation act, int n_out, int tokens) {
  if (!ctx) return CAAT_EINVAL;
  if (act != CAAT_ACT_NONE && act != CAAT_ACT_SILU && act != CAAT_ACT_SWIGLU) return CAAT_EINVAL;
  if (tokens < 1 || n_out < 1) return CAAT_ESHAPE;
  if (ctx->h % 8 != 0 || n_out % (act == CAAT_ACT_SWIGLU ? 16 : 8) != 0) return CAAT_EUNSUPPORTED;
  if ((long long)ctx->t * tokens > 2000000000LL) return CAAT_EUNSUPPORTED;
  return CAAT_OK;
}
}  // namespace

size_t caat_colpar_workspace_bytes(const caat_ctx* ctx, caat_activation act, int n_out, int tokens) {
  if (check_col(ctx, act, n_out, tokens) != CAAT_OK) return 0;
  return col_scratch(ctx, act, n_out, tokens).total;
}

caat_status caat_colpar_forward(const caat_ctx* ctx, caat_activation act, int n_out, int tokens, const void* X,
                                const void* A, void* pre, void* Y, void* cuda_stream) {
  caat_status s = check_col(ctx, act, n_out, tokens);
  if (s != CAAT_OK) return s;
  if (!X || !A || !pre || (act != CAAT_ACT_NONE && !Y)) return CAAT_EINVAL;
  const void* ptrs[] = {X, A, pre, Y};
  for (const void* p : ptrs)
    if (p && !aligned16(p)) return CAAT_EALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int t = ctx->t, T = tokens, h = ctx->h;
  cudaError_t ce;
  if (col_tc_usable(ctx, n_out)) {
    ce = launch_tc_forward(col_shapes(ctx, n_out, T), X, A, nullptr, pre, st);
  } else {
    GemmProblem g{};
    g.nseg = 1;
    g.seg[0] = GemmSeg{X, A, (long long)T * h, 0, h, 1, (long long)n_out * h, 0, 1, h, 1, h};
    g.C = pre; g.sCb = (long long)T * n_out; g.sCi = n_out; g.M = T; g.N = n_out; g.batch = t; g.c_f32 = 0;
    ce = launch_gemm_simt(g, ctx->dtype, st);
  }
  if (ce != cudaSuccess) return cuda_fail(ce);
  if (act != CAAT_ACT_NONE) {
    const int gated = act == CAAT_ACT_SWIGLU;
    ce = launch_act_forward(ctx->dtype, gated, pre, Y, (long long)t * T, gated ? n_out / 2 : n_out, st);
    if (ce != cudaSuccess) return cuda_fail(ce);
  }
  return CAAT_OK;
}

caat_status caat_colpar_backward(const caat_ctx* ctx, caat_activation act, int n_out, int tokens, const void* dY,
                                 const void* X, const void* A, const void* pre, void* dX, float* dA, void* workspace,
                                 size_t workspace_bytes, void* cuda_stream) {
  caat_status s = check_col(ctx, act, n_out, tokens);
  if (s != CAAT_OK) return s;
  if (!dY || !X || !A || !dX || !dA || (act != CAAT_ACT_NONE && !pre)) return CAAT_EINVAL;
  const void* ptrs[] = {dY, X, A, pre, dX, dA, workspace};
  for (const void* p : ptrs)
    if (p && !aligned16(p)) return CAAT_EALIGN;
  const ColScratch L = col_scratch(ctx, act, n_out, tokens);
  if (!workspace || workspace_bytes < L.total) return CAAT_EWORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* wsb = static_cast<char*>(workspace);
  const int t = ctx->t, T = tokens, h = ctx->h;
  cudaError_t ce;
  const void* dpre = dY;
  if (act != CAAT_ACT_NONE) {
    const int gated = act == CAAT_ACT_SWIGLU;
    ce = launch_act_backward(ctx->dtype, gated, dY, pre, wsb + L.dpre_off, (long long)t * T, gated ? n_out / 2 : n_out, st);
    if (ce != cudaSuccess) return cuda_fail(ce);
    dpre = wsb + L.dpre_off;
  }
  if (col_tc_usable(ctx, n_out)) {
    const RowparShapes sh = col_shapes(ctx, n_out, T);
    const PrivOperand pv{dpre, n_out, 0, 1.0f};
    ce = launch_tc_dgrad(sh, nullptr, pv, A, dX, nullptr, false, st);
    if (ce != cudaSuccess) return cuda_fail(ce);
    ce = launch_tc_wgrad(sh, nullptr, pv, X, dA, wsb + L.splitk_off, L.splitk_bytes, st);
    if (ce != cudaSuccess) return cuda_fail(ce);
    return CAAT_OK;
  }
  {  // dX[m] = dpre[m] A[m]
    GemmProblem g{};
    g.nseg = 1;
    g.seg[0] = GemmSeg{dpre, A, (long long)T * n_out, 0, n_out, 1, (long long)n_out * h, 0, h, 1, 1, n_out};
    g.C = dX; g.sCb = (long long)T * h; g.sCi = h; g.M = T; g.N = h; g.batch = t; g.c_f32 = 0;
    ce = launch_gemm_simt(g, ctx->dtype, st);
    if (ce != cudaSuccess) return cuda_fail(ce);
  }
  {  // dA[m] = dpre[m]^T X[m]
    GemmProblem g{};
    g.nseg = 1;
    g.seg[0] = GemmSeg{dpre, X, (long long)T * n_out, 0, 1, n_out, (long long)T * h, 0, h, 1, 1, T};
    g.C = dA; g.sCb = (long long)n_out * h; g.sCi = h; g.M = n_out; g.N = h; g.batch = t; g.c_f32 = 1;
    ce = launch_gemm_simt(g, ctx->dtype, st);
    if (ce != cudaSuccess) return cuda_fail(ce);
  }
  return CAAT_OK;
}

// ---- real tensor parallelism: the two halves of a layer call around the caller's all-reduce ---------
static caat_status check_tp(const caat_ctx* ctx, caat_layer layer, int tokens, const void* ws, size_t ws_bytes,
                            int backward) {
  caat_status s = check_common(ctx, layer, tokens);
  if (s != CAAT_OK) return s;
  const int K_r = layer_kr(ctx, layer);
  if (!tc_gemm_usable(ctx, K_r)) return CAAT_EUNSUPPORTED;   // the packed [T, S] slab exists on the tensor-core path
  if (!ws || !aligned16(ws) || ws_bytes < scratch_layout(ctx, K_r, tokens, backward).total) return CAAT_EWORKSPACE;
  return CAAT_OK;
}

caat_status caat_tp_slab(const caat_ctx* ctx, caat_layer layer, int tokens, int backward, size_t* offset_bytes,
                         int* rows, int* cols) {
  caat_status s = check_common(ctx, layer, tokens);
  if (s != CAAT_OK) return s;
  const int K_r = layer_kr(ctx, layer);
  if (!tc_gemm_usable(ctx, K_r)) return CAAT_EUNSUPPORTED;
  const Scratch L = scratch_layout(ctx, K_r, tokens, backward ? 1 : 0);
  if (L.S_hi != ctx->S) return CAAT_EUNSUPPORTED;
  if (offset_bytes) *offset_bytes = L.zs_off;
  if (rows) *rows = tokens;
  if (cols) *cols = ctx->S;
  return CAAT_OK;
}

caat_status caat_tp_forward_local(const caat_ctx* ctx, caat_layer layer, int tokens, const void* Y, const void* W,
                                  void* workspace, size_t workspace_bytes, void* cuda_stream) {
  caat_status s = check_tp(ctx, layer, tokens, workspace, workspace_bytes, 0);
  if (s != CAAT_OK) return s;
  if (!Y || !W) return CAAT_EINVAL;
  if (!aligned16(Y) || !aligned16(W)) return CAAT_EALIGN;
  return forward_impl(ctx, layer_kr(ctx, layer), tokens, Y, W, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr,
                      nullptr, workspace, static_cast<cudaStream_t>(cuda_stream), 0, nullptr, nullptr, 1);
}

caat_status caat_tp_forward_finish(const caat_ctx* ctx, caat_layer layer, int tokens, const void* R, const void* gamma,
                                   const void* beta, void* Hn, void* X, float* rstd, float* mean, void* workspace,
                                   size_t workspace_bytes, void* cuda_stream) {
  caat_status s = check_tp(ctx, layer, tokens, workspace, workspace_bytes, 0);
  if (s != CAAT_OK) return s;
  if (!R || !gamma || !Hn || !X || !rstd) return CAAT_EINVAL;
  if (ctx->norm == 1 && !mean) return CAAT_EINVAL;
  const void* ptrs[] = {R, gamma, beta, Hn, X, rstd, mean};
  for (const void* p : ptrs)
    if (p && !aligned16(p)) return CAAT_EALIGN;
  return forward_impl(ctx, layer_kr(ctx, layer), tokens, nullptr, nullptr, R, gamma, beta, Hn, X, rstd, mean, workspace,
                      static_cast<cudaStream_t>(cuda_stream), 0, nullptr, nullptr, 2);
}

caat_status caat_tp_backward_local(const caat_ctx* ctx, caat_layer layer, int tokens, const void* dX, const void* dHn,
                                   const void* W, const void* Hn, const float* rstd, const float* mean,
                                   const void* gamma, void* dR, float* dgamma, float* dbeta, void* workspace,
                                   size_t workspace_bytes, void* cuda_stream) {
  caat_status s = check_tp(ctx, layer, tokens, workspace, workspace_bytes, 1);
  if (s != CAAT_OK) return s;
  if (!dX || !W || !Hn || !rstd || !gamma || !dR || !dgamma) return CAAT_EINVAL;
  if (ctx->norm == 1 && (!mean || !dbeta)) return CAAT_EINVAL;
  const void* ptrs[] = {dX, dHn, W, Hn, rstd, mean, gamma, dR, dgamma, dbeta};
  for (const void* p : ptrs)
    if (p && !aligned16(p)) return CAAT_EALIGN;
  return backward_impl(ctx, layer_kr(ctx, layer), tokens, dX, dHn, nullptr, W, Hn, rstd, mean, gamma, nullptr, nullptr,
                       dR, dgamma, dbeta, workspace, static_cast<cudaStream_t>(cuda_stream), 0, nullptr, nullptr,
                       nullptr, 1);
}

}  // extern "C"

namespace caat {
caat_status tp_backward_local_push_impl(const caat_ctx* ctx, caat_layer layer, int tokens, const void* dX, const void* dHn,
                                        const void* W, const void* Hn, const float* rstd, const float* mean,
                                        const void* gamma, void* dR, float* dgamma, float* dbeta, void* workspace,
                                        size_t workspace_bytes, cudaStream_t st, const PushTarget& push) {
  caat_status s = check_tp(ctx, layer, tokens, workspace, workspace_bytes, 1);
  if (s != CAAT_OK) return s;
  if (!dX || !W || !Hn || !rstd || !gamma || !dR || !dgamma) return CAAT_EINVAL;
  if (ctx->norm == 1 && (!mean || !dbeta)) return CAAT_EINVAL;
  if (ctx->bwd_reduce != 0) return CAAT_EUNSUPPORTED;      // the numerics-study modes run on kernels without this path
  const void* ptrs[] = {dX, dHn, W, Hn, rstd, mean, gamma, dR, dgamma, dbeta};
  for (const void* p : ptrs)
    if (p && !aligned16(p)) return CAAT_EALIGN;
  return backward_impl(ctx, layer_kr(ctx, layer), tokens, dX, dHn, nullptr, W, Hn, rstd, mean, gamma, nullptr, nullptr, dR,
                       dgamma, dbeta, workspace, st, 0, nullptr, nullptr, nullptr, 1, &push);
}
}  // namespace caat

extern "C" {

caat_status caat_tp_backward_finish(const caat_ctx* ctx, caat_layer layer, int tokens, const void* Y, const void* W,
                                    const void* dR, void* dY, float* dW, void* workspace, size_t workspace_bytes,
                                    void* cuda_stream) {
  caat_status s = check_tp(ctx, layer, tokens, workspace, workspace_bytes, 1);
  if (s != CAAT_OK) return s;
  if (!Y || !W || !dR || !dY || !dW) return CAAT_EINVAL;
  const void* ptrs[] = {Y, W, dR, dY, dW};
  for (const void* p : ptrs)
    if (!aligned16(p)) return CAAT_EALIGN;
  return backward_impl(ctx, layer_kr(ctx, layer), tokens, nullptr, nullptr, Y, W, nullptr, nullptr, nullptr, nullptr, dY,
                       dW, const_cast<void*>(dR), nullptr, nullptr, workspace, static_cast<cudaStream_t>(cuda_stream),
                       0, nullptr, nullptr, nullptr, 2);
}


caat_status caat_allreduce_bytes(const caat_ctx* ctx, int tokens, int elem_bytes, unsigned long long* payload,
                                 unsigned long long* payload_p1, unsigned long long* ring_wire) {
  if (!ctx || elem_bytes < 1) return CAAT_EINVAL;
  if (tokens < 1) return CAAT_ESHAPE;
  const unsigned long long pay = (unsigned long long)tokens * (unsigned long long)ctx->S * (unsigned long long)elem_bytes;
  if (payload) *payload = pay;
  if (payload_p1) *payload_p1 = (unsigned long long)tokens * (unsigned long long)ctx->h * (unsigned long long)elem_bytes;
  // devices in the reduce: the t simulated ranks, or the G GPUs when the context is one group of a real run
  const unsigned long long ndev = (unsigned long long)(ctx->groups > 1 ? ctx->groups : ctx->t);
  if (ring_wire) *ring_wire = 2ull * (ndev - 1) * pay / ndev;
  return CAAT_OK;
}

caat_status caat_last_device_status(const caat_ctx* ctx, void* cuda_stream) {
  if (!ctx) return CAAT_EINVAL;
  cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream));
  if (e != cudaSuccess) return cuda_fail(e);
  unsigned int w = 0;
  e = cudaMemcpyFromSymbol(&w, g_status_word, sizeof(w));
  if (e != cudaSuccess) return cuda_fail(e);
  if (w != 0) {
    const unsigned int zero = 0;
    e = cudaMemcpyToSymbol(g_status_word, &zero, sizeof(zero));
    if (e != cudaSuccess) return cuda_fail(e);
    return CAAT_ETIMEOUT;
  }
  return CAAT_OK;
}

unsigned long long caat_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

caat_status caat_profile_begin(int max_launches) {
  if (max_launches < 1 || max_launches > (1 << 20)) return CAAT_EINVAL;
  if (g_prof.on) return CAAT_EINVAL;
  while ((int)g_prof.ev.size() < 2 * max_launches) {
    cudaEvent_t e;
    cudaError_t ce = cudaEventCreate(&e);
    if (ce != cudaSuccess) return cuda_fail(ce);
    g_prof.ev.push_back(e);
  }
  g_prof.kind.assign(max_launches, -1);
  g_prof.used = 0;
  g_prof.on = true;
  return CAAT_OK;
}

caat_status caat_profile_end(int n_kinds, double* ms_by_kind, unsigned long long* launches_by_kind) {
  if (!g_prof.on) return CAAT_EINVAL;
  g_prof.on = false;
  if (n_kinds < 1 || !ms_by_kind || !launches_by_kind) return CAAT_EINVAL;
  for (int k = 0; k < n_kinds; ++k) { ms_by_kind[k] = 0.0; launches_by_kind[k] = 0; }
  for (int i = 0; i < g_prof.used; ++i) {
    cudaError_t ce = cudaEventSynchronize(g_prof.ev[2 * i + 1]);
    if (ce != cudaSuccess) return cuda_fail(ce);
    float ms = 0.f;
    ce = cudaEventElapsedTime(&ms, g_prof.ev[2 * i], g_prof.ev[2 * i + 1]);
    if (ce != cudaSuccess) return cuda_fail(ce);
    const int k = g_prof.kind[i];
    if (k >= 0 && k < n_kinds) { ms_by_kind[k] += ms; launches_by_kind[k] += 1; }
  }
  return CAAT_OK;
}

const char* caat_kernel_kind_name(int kind) {
  switch (kind) {
    case CAAT_K_ROWS_FORWARD: return "rows_forward";
    case CAAT_K_ROWS_BACKWARD: return "rows_backward";
    case CAAT_K_NORMGRAD_REDUCE: return "normgrad_reduce";
    case CAAT_K_GEMM_CUDA_CORE: return "gemm_cuda_core";
    case CAAT_K_TC_FORWARD: return "tc_gemm_forward";
    case CAAT_K_TC_DGRAD: return "tc_gemm_dgrad";
    case CAAT_K_TC_WGRAD: return "tc_gemm_wgrad";
    case CAAT_K_SPLITK_REDUCE: return "splitk_reduce";
    case CAAT_K_ACTIVATION: return "activation";
    case CAAT_K_TP_EXCHANGE: return "tp_exchange";
  }
  return "";
}

}  // extern "C"
