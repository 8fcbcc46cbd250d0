// Row kernels: everything of the layer that is not a contraction.
//
// Forward  (F2..F5): partial channel-reduce hand-off, private scaling, residual add,
//                    per-rank norm.
// Backward (B1..B4): norm backward + residual gradient, per-rank dR, norm-parameter
//                    gradients summed over ranks, and the backward partial channel-reduce
//                    (fp32 sum over ranks, placed after the norm's backward).
//
// Mapping: one token is handled by TX consecutive threads of a CTA (TY tokens per CTA);
// a thread owns the same 16-byte column chunk(s) of EVERY rank of its token and walks
// the ranks m = 0..t-1 in order.  The rank sum of the shared channels and the
// norm-parameter gradients are therefore thread-local and run in a fixed order.
// Row statistics need one CTA-wide reduction per rank; the next rank's loads are issued
// before it so that HBM requests stay in flight across the barrier.
#include "caat_internal.h"

namespace caat {
namespace {

template <typename T_>
struct VT;
template <>
struct VT<float> {
  static constexpr int N = 4;
  using raw = float4;
  static __device__ __forceinline__ void unpack(const raw& r, float* f) {
    f[0] = r.x; f[1] = r.y; f[2] = r.z; f[3] = r.w;
  }
  static __device__ __forceinline__ raw pack(const float* f) { return make_float4(f[0], f[1], f[2], f[3]); }
  static __device__ __forceinline__ float round(float x) { return x; }
};
template <>
struct VT<__nv_bfloat16> {
  static constexpr int N = 8;
  using raw = uint4;
  static __device__ __forceinline__ void unpack(const raw& r, float* f) {
    const unsigned w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      f[2 * q] = __uint_as_float(w[q] << 16);
      f[2 * q + 1] = __uint_as_float(w[q] & 0xffff0000u);
    }
  }
  static __device__ __forceinline__ raw pack(const float* f) {
    unsigned w[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      __nv_bfloat162 b = __floats2bfloat162_rn(f[2 * q], f[2 * q + 1]);
      w[q] = *reinterpret_cast<unsigned*>(&b);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
  }
  static __device__ __forceinline__ float round(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }
};

template <typename raw>
__device__ __forceinline__ raw ld_vec(const void* base, long long elem_off, int esz) {
  return *reinterpret_cast<const raw*>(static_cast<const char*>(base) + elem_off * esz);
}
template <typename raw>
__device__ __forceinline__ void st_vec(void* base, long long elem_off, int esz, const raw& v) {
  *reinterpret_cast<raw*>(static_cast<char*>(base) + elem_off * esz) = v;
}
template <typename raw>
__device__ __forceinline__ raw zero_raw();
template <>
__device__ __forceinline__ float4 zero_raw<float4>() { return make_float4(0.f, 0.f, 0.f, 0.f); }
template <>
__device__ __forceinline__ uint4 zero_raw<uint4>() { return make_uint4(0u, 0u, 0u, 0u); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Sum of NV values over the TX threads of one token row.  `red` holds
// [2][TY][warps_x][NV] floats; `par` alternates so that one barrier per call suffices.
template <int NV>
__device__ __forceinline__ void row_reduce(float (&v)[NV], float* red, int& par) {
  const int warps_x = blockDim.x >> 5;
#pragma unroll
  for (int q = 0; q < NV; ++q) v[q] = warp_sum(v[q]);
  if (warps_x == 1) return;
  float* buf = red + ((size_t)(par * blockDim.y + threadIdx.y) * warps_x) * NV;
  if ((threadIdx.x & 31) == 0) {
#pragma unroll
    for (int q = 0; q < NV; ++q) buf[(threadIdx.x >> 5) * NV + q] = v[q];
  }
  __syncthreads();
#pragma unroll
  for (int q = 0; q < NV; ++q) {
    float s = 0.f;
    for (int w = 0; w < warps_x; ++w) s += buf[w * NV + q];
    v[q] = s;
  }
  par ^= 1;
}

// column class of a chunk [col, col+V): 0 all shared, 1 all private, 2 mixed
__device__ __forceinline__ int chunk_class(int col, int V, int S) {
  return (col + V <= S) ? 0 : (col >= S ? 1 : 2);
}

// ------------------------------------------------------------------ forward
template <typename T_, int CPT>
__global__ void __launch_bounds__(512) rows_forward_kernel(RowFwdArgs a) {
  using V_ = VT<T_>;
  using raw = typename V_::raw;
  constexpr int V = V_::N;
  constexpr int ES = sizeof(T_);
  extern __shared__ float red[];
  int par = 0;
  const int TX = blockDim.x;
  const long long i = (long long)blockIdx.x * blockDim.y + threadIdx.y;
  const bool valid = i < a.T;
  const bool ln = a.norm == 1;

  int col[CPT], cls[CPT];
  bool act[CPT];
  float gam[CPT][V], bet[CPT][V], zs[CPT][V];
#pragma unroll
  for (int j = 0; j < CPT; ++j) {
    col[j] = (threadIdx.x + j * TX) * V;
    act[j] = valid && col[j] < a.h;
    cls[j] = chunk_class(col[j], V, a.S);
#pragma unroll
    for (int e = 0; e < V; ++e) { gam[j][e] = 0.f; bet[j][e] = 0.f; zs[j][e] = 0.f; }
    if (act[j]) {
      V_::unpack(ld_vec<raw>(a.gamma, col[j], ES), gam[j]);
      if (ln && a.beta) V_::unpack(ld_vec<raw>(a.beta, col[j], ES), bet[j]);
      if (cls[j] != 1) V_::unpack(ld_vec<raw>(a.zs, i * a.S_hi + col[j], ES), zs[j]);
    }
  }

  raw rR[CPT], rZ[CPT];
  auto issue = [&](int m, raw(&R_)[CPT], raw(&Z_)[CPT]) {
#pragma unroll
    for (int j = 0; j < CPT; ++j) {
      R_[j] = zero_raw<raw>();
      Z_[j] = zero_raw<raw>();
      if (act[j]) {
        const long long row = (long long)m * a.T + i;
        R_[j] = ld_vec<raw>(a.R, row * a.h + col[j], ES);
        if (cls[j] != 0) Z_[j] = ld_vec<raw>(a.zp, row * a.P + (col[j] - a.S_lo), ES);
      }
    }
  };
  issue(0, rR, rZ);

  for (int m = 0; m < a.t; ++m) {
    raw nR[CPT], nZ[CPT];
    if (m + 1 < a.t) issue(m + 1, nR, nZ);
    const long long row = (long long)m * a.T + i;

    float hn[CPT][V];
    float st[1] = {0.f};
#pragma unroll
    for (int j = 0; j < CPT; ++j) {
      float r[V], zp[V];
      V_::unpack(rR[j], r);
      V_::unpack(rZ[j], zp);
#pragma unroll
      for (int e = 0; e < V; ++e) {
        const float z = (cls[j] == 0 || (cls[j] == 2 && col[j] + e < a.S)) ? zs[j][e] : a.alpha * zp[e];
        hn[j][e] = act[j] ? z + r[e] : 0.f;
      }
      if (act[j]) st_vec<raw>(a.Hn, row * a.h + col[j], ES, V_::pack(hn[j]));
#pragma unroll
      for (int e = 0; e < V; ++e) st[0] += ln ? hn[j][e] : hn[j][e] * hn[j][e];
    }
    row_reduce<1>(st, red, par);
    float mu = 0.f, rs;
    if (ln) {
      mu = st[0] / (float)a.h;
      float sq[1] = {0.f};
#pragma unroll
      for (int j = 0; j < CPT; ++j)
#pragma unroll
        for (int e = 0; e < V; ++e) {
          const float d = act[j] ? hn[j][e] - mu : 0.f;
          sq[0] += d * d;
        }
      row_reduce<1>(sq, red, par);
      rs = 1.0f / sqrtf(sq[0] / (float)a.h + a.eps);
    } else {
      rs = 1.0f / sqrtf(st[0] / (float)a.h + a.eps);
    }
#pragma unroll
    for (int j = 0; j < CPT; ++j) {
      if (!act[j]) continue;
      float x[V];
#pragma unroll
      for (int e = 0; e < V; ++e) x[e] = (hn[j][e] - mu) * rs * gam[j][e] + bet[j][e];
      st_vec<raw>(a.X, row * a.h + col[j], ES, V_::pack(x));
    }
    if (valid && threadIdx.x == 0) {
      a.rstd[row] = rs;
      if (ln && a.mean) a.mean[row] = mu;
    }
#pragma unroll
    for (int j = 0; j < CPT; ++j) { rR[j] = nR[j]; rZ[j] = nZ[j]; }
  }
}

// ------------------------------------------------------------------ backward
template <typename T_, int CPT>
__global__ void __launch_bounds__(512) rows_backward_kernel(RowBwdArgs a, int ngroups) {
  using V_ = VT<T_>;
  using raw = typename V_::raw;
  constexpr int V = V_::N;
  constexpr int ES = sizeof(T_);
  extern __shared__ float red[];
  int par = 0;
  const int TX = blockDim.x;
  const bool ln = a.norm == 1;
  const float inv_h = 1.0f / (float)a.h;

  int col[CPT], cls[CPT];
  bool colok[CPT];
  float gam[CPT][V], dgacc[CPT][V], dbacc[CPT][V];
#pragma unroll
  for (int j = 0; j < CPT; ++j) {
    col[j] = (threadIdx.x + j * TX) * V;
    colok[j] = col[j] < a.h;
    cls[j] = chunk_class(col[j], V, a.S);
#pragma unroll
    for (int e = 0; e < V; ++e) { gam[j][e] = 0.f; dgacc[j][e] = 0.f; dbacc[j][e] = 0.f; }
    if (colok[j]) V_::unpack(ld_vec<raw>(a.gamma, col[j], ES), gam[j]);
  }

  for (int grp = blockIdx.x; grp < ngroups; grp += gridDim.x) {
    const long long i = (long long)grp * blockDim.y + threadIdx.y;
    const bool valid = i < a.T;
    bool act[CPT];
#pragma unroll
    for (int j = 0; j < CPT; ++j) act[j] = valid && colok[j];

    raw rdX[CPT], rHn[CPT], rdH[CPT];
    float rs_c, mu_c;
    auto issue = [&](int m, raw(&dX_)[CPT], raw(&Hn_)[CPT], raw(&dH_)[CPT], float& rs, float& mu) {
      const long long row = (long long)m * a.T + i;
      rs = valid ? a.rstd[row] : 0.f;
      mu = (valid && ln) ? a.mean[row] : 0.f;
#pragma unroll
      for (int j = 0; j < CPT; ++j) {
        dX_[j] = zero_raw<raw>(); Hn_[j] = zero_raw<raw>(); dH_[j] = zero_raw<raw>();
        if (act[j]) {
          dX_[j] = ld_vec<raw>(a.dX, row * a.h + col[j], ES);
          Hn_[j] = ld_vec<raw>(a.Hn, row * a.h + col[j], ES);
          if (a.dHn) dH_[j] = ld_vec<raw>(a.dHn, row * a.h + col[j], ES);
        }
      }
    };
    issue(0, rdX, rHn, rdH, rs_c, mu_c);

    float gsum[CPT][V];
#pragma unroll
    for (int j = 0; j < CPT; ++j)
#pragma unroll
      for (int e = 0; e < V; ++e) gsum[j][e] = 0.f;

    for (int m = 0; m < a.t; ++m) {
      raw ndX[CPT], nHn[CPT], ndH[CPT];
      float rs_n = 0.f, mu_n = 0.f;
      if (m + 1 < a.t) issue(m + 1, ndX, nHn, ndH, rs_n, mu_n);
      const long long row = (long long)m * a.T + i;

      float xh[CPT][V], dxh[CPT][V];
      float s[2] = {0.f, 0.f};
#pragma unroll
      for (int j = 0; j < CPT; ++j) {
        float dx[V], hn[V];
        V_::unpack(rdX[j], dx);
        V_::unpack(rHn[j], hn);
#pragma unroll
        for (int e = 0; e < V; ++e) {
          xh[j][e] = act[j] ? (hn[e] - mu_c) * rs_c : 0.f;
          dxh[j][e] = dx[e] * gam[j][e];
          s[0] += dxh[j][e];
          s[1] += dxh[j][e] * xh[j][e];
          dgacc[j][e] += dx[e] * xh[j][e];
          dbacc[j][e] += dx[e];
        }
      }
      row_reduce<2>(s, red, par);
      const float c1 = ln ? s[0] * inv_h : 0.f;
      const float c2 = s[1] * inv_h;
#pragma unroll
      for (int j = 0; j < CPT; ++j) {
        if (!act[j]) continue;
        float dh[V], g[V], zp[V];
        V_::unpack(rdH[j], dh);
#pragma unroll
        for (int e = 0; e < V; ++e) {
          g[e] = rs_c * (dxh[j][e] - c1 - xh[j][e] * c2) + dh[e];
          const bool shared = cls[j] == 0 || (cls[j] == 2 && col[j] + e < a.S);
          gsum[j][e] += shared ? g[e] : 0.f;       // fp32 rank sum, m ascending
          zp[e] = shared ? 0.f : a.alpha * g[e];   // private gradient carries alpha
        }
        st_vec<raw>(a.dR, row * a.h + col[j], ES, V_::pack(g));
        if (cls[j] != 0) st_vec<raw>(a.zp, row * a.P + (col[j] - a.S_lo), ES, V_::pack(zp));
      }
#pragma unroll
      for (int j = 0; j < CPT; ++j) { rdX[j] = ndX[j]; rHn[j] = nHn[j]; rdH[j] = ndH[j]; }
      rs_c = rs_n; mu_c = mu_n;
    }
#pragma unroll
    for (int j = 0; j < CPT; ++j)
      if (act[j] && cls[j] != 1) st_vec<raw>(a.gs, i * a.S_hi + col[j], ES, V_::pack(gsum[j]));
  }

  // Partial norm-parameter gradients of this CTA: sum the TY token rows in order, then
  // one row of [h] per CTA.
  __syncthreads();
  float* acc = red;  // reuse: [TY][TX*CPT*V]
  const int per_row = TX * CPT * V;
  for (int which = 0; which < (ln ? 2 : 1); ++which) {
    float* out = which == 0 ? a.dgpart : a.dbpart;
    if (out == nullptr) continue;
#pragma unroll
    for (int j = 0; j < CPT; ++j)
#pragma unroll
      for (int e = 0; e < V; ++e)
        acc[(size_t)threadIdx.y * per_row + (j * TX + threadIdx.x) * V + e] = which == 0 ? dgacc[j][e] : dbacc[j][e];
    __syncthreads();
    if (threadIdx.y == 0) {
#pragma unroll
      for (int j = 0; j < CPT; ++j) {
        if (!colok[j]) continue;
        float sum[V];
#pragma unroll
        for (int e = 0; e < V; ++e) sum[e] = 0.f;
        for (int y = 0; y < (int)blockDim.y; ++y)
#pragma unroll
          for (int e = 0; e < V; ++e) sum[e] += acc[(size_t)y * per_row + (j * TX + threadIdx.x) * V + e];
#pragma unroll
        for (int e = 0; e < V; e += 4)
          *reinterpret_cast<float4*>(out + (size_t)blockIdx.x * a.h + col[j] + e) =
              make_float4(sum[e], sum[e + 1], sum[e + 2], sum[e + 3]);
      }
    }
    __syncthreads();
  }
}

// out[l] = sum over `rows` partial rows, fixed order: 32 row lanes then a serial combine.
__global__ void __launch_bounds__(1024) reduce_partials_kernel(const float* __restrict__ part, float* __restrict__ out,
                                                               int rows, int h) {
  __shared__ float sm[32][33];
  const int c = blockIdx.x * 32 + threadIdx.x;
  float s = 0.f;
  if (c < h)
    for (int r = threadIdx.y; r < rows; r += 32) s += part[(size_t)r * h + c];
  sm[threadIdx.y][threadIdx.x] = s;
  __syncthreads();
  if (threadIdx.y == 0 && c < h) {
    float tot = 0.f;
    for (int y = 0; y < 32; ++y) tot += sm[y][threadIdx.x];
    out[c] = tot;
  }
}

struct RowGeom {
  int TX, TY, CPT;
  size_t smem_fwd, smem_bwd;
};

RowGeom row_geometry(int h, caat_dtype dtype) {
  const int V = dtype == CAAT_BF16 ? 8 : 4;
  const int chunks = h / V;
  RowGeom g;
  int tx = round_up(chunks, 32);
  g.CPT = 1;
  while (tx > 512) {
    g.CPT *= 2;
    tx = round_up((chunks + g.CPT - 1) / g.CPT, 32);
  }
  g.TX = tx;
  g.TY = tx >= 256 ? 1 : 256 / tx;
  const size_t red = (size_t)2 * g.TY * (g.TX / 32) * 2 * sizeof(float);
  g.smem_fwd = red;
  const size_t acc = (size_t)g.TY * g.TX * g.CPT * V * sizeof(float);
  g.smem_bwd = red > acc ? red : acc;
  return g;
}

}  // namespace

int rows_backward_partial_rows(int h, int T, caat_dtype dtype) {
  const RowGeom g = row_geometry(h, dtype);
  const int ngroups = (T + g.TY - 1) / g.TY;
  return ngroups < kMaxPartialRows ? ngroups : kMaxPartialRows;
}

template <typename T_>
static cudaError_t launch_fwd_t(const RowFwdArgs& a, const RowGeom& g, cudaStream_t st) {
  const dim3 block(g.TX, g.TY);
  const dim3 grid((a.T + g.TY - 1) / g.TY);
  LaunchScope scope(CAAT_K_ROWS_FORWARD, st);
  switch (g.CPT) {
    case 1: rows_forward_kernel<T_, 1><<<grid, block, g.smem_fwd, st>>>(a); break;
    case 2: rows_forward_kernel<T_, 2><<<grid, block, g.smem_fwd, st>>>(a); break;
    case 4: rows_forward_kernel<T_, 4><<<grid, block, g.smem_fwd, st>>>(a); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

cudaError_t launch_rows_forward(const RowFwdArgs& a, caat_dtype dtype, cudaStream_t st) {
  const RowGeom g = row_geometry(a.h, dtype);
  return dtype == CAAT_BF16 ? launch_fwd_t<__nv_bfloat16>(a, g, st) : launch_fwd_t<float>(a, g, st);
}

template <typename T_>
static cudaError_t launch_bwd_t(const RowBwdArgs& a, const RowGeom& g, int rows, cudaStream_t st) {
  const dim3 block(g.TX, g.TY);
  const int ngroups = (a.T + g.TY - 1) / g.TY;
  const dim3 grid(rows);
  if (g.smem_bwd > 48 * 1024) {
    cudaError_t e = cudaSuccess;
    switch (g.CPT) {
      case 1: e = cudaFuncSetAttribute(rows_backward_kernel<T_, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g.smem_bwd); break;
      case 2: e = cudaFuncSetAttribute(rows_backward_kernel<T_, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g.smem_bwd); break;
      case 4: e = cudaFuncSetAttribute(rows_backward_kernel<T_, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g.smem_bwd); break;
    }
    if (e != cudaSuccess) return e;
  }
  LaunchScope scope(CAAT_K_ROWS_BACKWARD, st);
  switch (g.CPT) {
    case 1: rows_backward_kernel<T_, 1><<<grid, block, g.smem_bwd, st>>>(a, ngroups); break;
    case 2: rows_backward_kernel<T_, 2><<<grid, block, g.smem_bwd, st>>>(a, ngroups); break;
    case 4: rows_backward_kernel<T_, 4><<<grid, block, g.smem_bwd, st>>>(a, ngroups); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

cudaError_t launch_rows_backward(const RowBwdArgs& a, caat_dtype dtype, cudaStream_t st) {
  const RowGeom g = row_geometry(a.h, dtype);
  const int rows = rows_backward_partial_rows(a.h, a.T, dtype);
  cudaError_t e = dtype == CAAT_BF16 ? launch_bwd_t<__nv_bfloat16>(a, g, rows, st) : launch_bwd_t<float>(a, g, rows, st);
  if (e != cudaSuccess) return e;
  const dim3 rb(32, 32);
  const dim3 rg((a.h + 31) / 32);
  {
    LaunchScope scope(CAAT_K_NORMGRAD_REDUCE, st);
    reduce_partials_kernel<<<rg, rb, 0, st>>>(a.dgpart, a.dgamma, rows, a.h);
  }
  if (a.norm == 1 && a.dbeta && a.dbpart) {
    LaunchScope scope(CAAT_K_NORMGRAD_REDUCE, st);
    reduce_partials_kernel<<<rg, rb, 0, st>>>(a.dbpart, a.dbeta, rows, a.h);
  }
  return cudaGetLastError();
}

}  // namespace caat
