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
//
// These kernels move 3-5 bytes per arithmetic instruction, so the instruction count per
// 16-byte chunk decides whether they reach HBM speed: the norm kind and the number of
// chunks per thread are template parameters, pointers advance by one add per rank, and
// the shared/private class of a chunk is resolved by a branch per chunk, not per element.
#include <cooperative_groups.h>

#include "caat_rows_common.cuh"

namespace caat {
namespace {

using namespace rows;

// ------------------------------------------------------------------ forward
// CL: compact residual layout (shared part of R / Hn stored once, [T, S]; private parts [t, T, P])
template <typename T_, int CPT, bool LN, bool CL>
__global__ void __launch_bounds__(512, CPT == 1 ? 2 : 1) rows_forward_kernel(const RowFwdArgs a) {
  using V_ = VT<T_>;
  using raw = typename V_::raw;
  constexpr int V = V_::N;
  constexpr int ES = sizeof(T_);
  extern __shared__ float red[];
  int par = 0;
  const int TX = blockDim.x;
  const long long i = (long long)blockIdx.x * blockDim.y + threadIdx.y;
  const bool valid = i < a.T;
  const float inv_h = 1.0f / (float)a.h;
  const long long rank_h = (long long)a.T * a.h * ES;   // byte stride between ranks
  const long long rank_p = (long long)a.T * a.P * ES;

  int col[CPT], cls[CPT];
  bool act[CPT];
  float gam[CPT][V], bet[CPT][V], zs[CPT][V];
  const char* pR[CPT];
  const char* pZ[CPT];
  char* pHn[CPT];
  char* pX[CPT];
#pragma unroll
  for (int j = 0; j < CPT; ++j) {
    col[j] = (threadIdx.x + j * TX) * V;
    act[j] = valid && col[j] < a.h;
    cls[j] = chunk_class(col[j], V, a.S);
#pragma unroll
    for (int e = 0; e < V; ++e) { gam[j][e] = 0.f; bet[j][e] = 0.f; zs[j][e] = 0.f; }
    const long long off_h = (i * a.h + col[j]) * ES;
    const long long off_p = (i * a.P + (col[j] - a.S_lo)) * ES;
    if (CL) {
      const long long off_s = (i * a.S_hi + col[j]) * ES;
      pR[j] = cls[j] == 0 ? static_cast<const char*>(a.Rs) + off_s : static_cast<const char*>(a.R) + off_p;
      pHn[j] = cls[j] == 0 ? static_cast<char*>(a.Hns) + off_s : static_cast<char*>(a.Hn) + off_p;
    } else {
      pR[j] = static_cast<const char*>(a.R) + off_h;
      pHn[j] = static_cast<char*>(a.Hn) + off_h;
    }
    pX[j] = static_cast<char*>(a.X) + off_h;
    pZ[j] = static_cast<const char*>(a.zp) + off_p;
    if (act[j]) {
      V_::unpack(ldg<raw>(static_cast<const char*>(a.gamma) + (long long)col[j] * ES), gam[j]);
      if (LN && a.beta) V_::unpack(ldg<raw>(static_cast<const char*>(a.beta) + (long long)col[j] * ES), bet[j]);
      if (cls[j] != 1) V_::unpack(ldg<raw>(static_cast<const char*>(a.zs) + (i * a.S_hi + col[j]) * ES), zs[j]);
    }
  }

  raw rR[CPT], rZ[CPT];
#pragma unroll
  for (int j = 0; j < CPT; ++j) {
    rR[j] = act[j] ? ldg<raw>(pR[j]) : zero_raw<raw>();
    rZ[j] = (act[j] && cls[j] != 0) ? ldg<raw>(pZ[j]) : zero_raw<raw>();
  }
  float* rstd_p = a.rstd + i;
  float* mean_p = (LN && a.mean) ? a.mean + i : nullptr;

  for (int m = 0; m < a.t; ++m) {
    raw nR[CPT], nZ[CPT];
#pragma unroll
    for (int j = 0; j < CPT; ++j) {   // next rank's loads go out before this rank's barrier
      pR[j] += CL ? rank_p : rank_h;      // (compact, shared chunk: the pointer is not used again)
      pZ[j] += rank_p;
      const bool more = act[j] && (m + 1 < a.t);
      if (CL && cls[j] == 0) nR[j] = rR[j];   // the shared residual is the same for every rank
      else nR[j] = more ? ldg<raw>(pR[j]) : zero_raw<raw>();
      nZ[j] = (more && cls[j] != 0) ? ldg<raw>(pZ[j]) : zero_raw<raw>();
    }

    float hn[CPT][V];
    float st[1] = {0.f};
#pragma unroll
    for (int j = 0; j < CPT; ++j) {
      float r[V], zp[V];
      V_::unpack(rR[j], r);
      if (cls[j] == 0) {
#pragma unroll
        for (int e = 0; e < V; ++e) hn[j][e] = zs[j][e] + r[e];
      } else if (cls[j] == 1) {
        V_::unpack(rZ[j], zp);
#pragma unroll
        for (int e = 0; e < V; ++e) hn[j][e] = fmaf(a.alpha, zp[e], r[e]);
      } else {
        V_::unpack(rZ[j], zp);
#pragma unroll
        for (int e = 0; e < V; ++e) hn[j][e] = (col[j] + e < a.S ? zs[j][e] : a.alpha * zp[e]) + r[e];
      }
      if (act[j] && !(CL && cls[j] == 0 && m > 0)) stg<raw>(pHn[j], V_::pack(hn[j]));
      pHn[j] += CL ? rank_p : rank_h;
#pragma unroll
      for (int e = 0; e < V; ++e) st[0] = LN ? st[0] + hn[j][e] : fmaf(hn[j][e], hn[j][e], st[0]);
    }
    row_reduce<1>(st, red, par);
    float mu = 0.f, rs;
    if (LN) {
      mu = st[0] * inv_h;
      float sq[1] = {0.f};
#pragma unroll
      for (int j = 0; j < CPT; ++j)
#pragma unroll
        for (int e = 0; e < V; ++e) {
          const float d = act[j] ? hn[j][e] - mu : 0.f;
          sq[0] = fmaf(d, d, sq[0]);
        }
      row_reduce<1>(sq, red, par);
      rs = rsqrtf(fmaf(sq[0], inv_h, a.eps));
    } else {
      rs = rsqrtf(fmaf(st[0], inv_h, a.eps));
    }
#pragma unroll
    for (int j = 0; j < CPT; ++j) {
      float x[V];
#pragma unroll
      for (int e = 0; e < V; ++e) {
        if (LN) x[e] = fmaf(hn[j][e] - mu, rs * gam[j][e], bet[j][e]);
        else x[e] = hn[j][e] * (rs * gam[j][e]);
      }
      if (act[j]) stg<raw>(pX[j], V_::pack(x));
      pX[j] += rank_h;
    }
    if (valid && threadIdx.x == 0) {
      *rstd_p = rs;
      if (LN && mean_p) *mean_p = mu;
    }
    rstd_p += a.T;
    if (LN && mean_p) mean_p += a.T;
#pragma unroll
    for (int j = 0; j < CPT; ++j) { rR[j] = nR[j]; rZ[j] = nZ[j]; }
  }
}

// ------------------------------------------------------------------ backward
template <typename T_, int CPT, bool LN, bool CL>
__global__ void __launch_bounds__(512, CPT == 1 ? 2 : 1) rows_backward_kernel(const RowBwdArgs a, int ngroups) {
  using V_ = VT<T_>;
  using raw = typename V_::raw;
  constexpr int V = V_::N;
  constexpr int ES = sizeof(T_);
  extern __shared__ float red[];
  int par = 0;
  const int TX = blockDim.x;
  const float inv_h = 1.0f / (float)a.h;
  const long long rank_h = (long long)a.T * a.h * ES;
  const long long rank_p = (long long)a.T * a.P * ES;
  const bool has_dh = a.dHn != nullptr;

  int col[CPT], cls[CPT];
  bool colok[CPT];
  float gam[CPT][V], dgacc[CPT][V], dbacc[LN ? CPT : 1][V];
#pragma unroll
  for (int j = 0; j < CPT; ++j) {
    col[j] = (threadIdx.x + j * TX) * V;
    colok[j] = col[j] < a.h;
    cls[j] = chunk_class(col[j], V, a.S);
#pragma unroll
    for (int e = 0; e < V; ++e) { gam[j][e] = 0.f; dgacc[j][e] = 0.f; if constexpr (LN) dbacc[j][e] = 0.f; }
    if (colok[j]) V_::unpack(ldg<raw>(static_cast<const char*>(a.gamma) + (long long)col[j] * ES), gam[j]);
  }

  for (int grp = blockIdx.x; grp < ngroups; grp += gridDim.x) {
    const long long i = (long long)grp * blockDim.y + threadIdx.y;
    const bool valid = i < a.T;
    bool act[CPT];
    const char* pdX[CPT];
    const char* pHn[CPT];
    const char* pdH[CPT];
    char* pdR[CPT];
    char* pZ[CPT];
    raw rdX[CPT], rHn[CPT], rdH[CPT];
#pragma unroll
    for (int j = 0; j < CPT; ++j) {
      act[j] = valid && colok[j];
      const long long off_h = (i * a.h + col[j]) * ES;
      const long long off_p = (i * a.P + (col[j] - a.S_lo)) * ES;
      pdX[j] = static_cast<const char*>(a.dX) + off_h;
      if (CL) {
        const long long off_s = (i * a.S_hi + col[j]) * ES;
        pHn[j] = cls[j] == 0 ? static_cast<const char*>(a.Hns) + off_s : static_cast<const char*>(a.Hn) + off_p;
        pdH[j] = cls[j] == 0 ? static_cast<const char*>(a.dHns) + off_s : static_cast<const char*>(a.dHn) + off_p;
        pdR[j] = static_cast<char*>(a.dR) + off_p;
      } else {
        pHn[j] = static_cast<const char*>(a.Hn) + off_h;
        pdH[j] = static_cast<const char*>(a.dHn) + off_h;
        pdR[j] = static_cast<char*>(a.dR) + off_h;
      }
      pZ[j] = static_cast<char*>(a.zp) + off_p;
      rdX[j] = act[j] ? ldg<raw>(pdX[j]) : zero_raw<raw>();
      rHn[j] = act[j] ? ldg<raw>(pHn[j]) : zero_raw<raw>();
      rdH[j] = (act[j] && has_dh) ? ldg<raw>(pdH[j]) : zero_raw<raw>();
    }
    const float* rstd_p = a.rstd + i;
    const float* mean_p = LN ? a.mean + i : nullptr;
    float rs_c = valid ? *rstd_p : 0.f;
    float mu_c = (LN && valid) ? *mean_p : 0.f;

    float gsum[CPT][V];
#pragma unroll
    for (int j = 0; j < CPT; ++j) {
#pragma unroll
      for (int e = 0; e < V; ++e) gsum[j][e] = 0.f;
      if (CL && cls[j] == 0) {   // the gradient on the single shared stream enters the rank sum once
        V_::unpack(rdH[j], gsum[j]);
        rdH[j] = zero_raw<raw>();
      }
    }

    for (int m = 0; m < a.t; ++m) {
      raw ndX[CPT], nHn[CPT], ndH[CPT];
      const bool more_rank = m + 1 < a.t;
      rstd_p += a.T;
      if (LN) mean_p += a.T;
      const float rs_n = (valid && more_rank) ? *rstd_p : 0.f;
      const float mu_n = (LN && valid && more_rank) ? *mean_p : 0.f;
#pragma unroll
      for (int j = 0; j < CPT; ++j) {
        pdX[j] += rank_h; pHn[j] += CL ? rank_p : rank_h; pdH[j] += CL ? rank_p : rank_h;
        const bool more = act[j] && more_rank;
        ndX[j] = more ? ldg<raw>(pdX[j]) : zero_raw<raw>();
        if (CL && cls[j] == 0) {
          nHn[j] = rHn[j];                  // one shared row for every rank
          ndH[j] = zero_raw<raw>();
        } else {
          nHn[j] = more ? ldg<raw>(pHn[j]) : zero_raw<raw>();
          ndH[j] = (more && has_dh) ? ldg<raw>(pdH[j]) : zero_raw<raw>();
        }
      }

      float xh[CPT][V], dxh[CPT][V];
      float s[LN ? 2 : 1];
#pragma unroll
      for (int q = 0; q < (LN ? 2 : 1); ++q) s[q] = 0.f;
#pragma unroll
      for (int j = 0; j < CPT; ++j) {
        float dx[V], hn[V];
        V_::unpack(rdX[j], dx);
        V_::unpack(rHn[j], hn);
#pragma unroll
        for (int e = 0; e < V; ++e) {
          xh[j][e] = LN ? (act[j] ? (hn[e] - mu_c) * rs_c : 0.f) : hn[e] * rs_c;
          dxh[j][e] = dx[e] * gam[j][e];
          if (LN) { s[0] += dxh[j][e]; s[1] = fmaf(dxh[j][e], xh[j][e], s[1]); }
          else s[0] = fmaf(dxh[j][e], xh[j][e], s[0]);
          dgacc[j][e] = fmaf(dx[e], xh[j][e], dgacc[j][e]);
          if constexpr (LN) dbacc[j][e] += dx[e];
        }
      }
      row_reduce<LN ? 2 : 1>(s, red, par);
      const float c1 = LN ? s[0] * inv_h : 0.f;
      const float c2 = (LN ? s[1] : s[0]) * inv_h;
#pragma unroll
      for (int j = 0; j < CPT; ++j) {
        float dh[V], g[V];
        V_::unpack(rdH[j], dh);
#pragma unroll
        for (int e = 0; e < V; ++e) {
          float tt = fmaf(-xh[j][e], c2, dxh[j][e]);
          if (LN) tt -= c1;
          g[e] = fmaf(rs_c, tt, dh[e]);
        }
        if (act[j] && !(CL && cls[j] == 0)) stg<raw>(pdR[j], V_::pack(g));
        pdR[j] += CL ? rank_p : rank_h;
        if (cls[j] == 0) {
          if (a.reduce_mode == 0) {
#pragma unroll
            for (int e = 0; e < V; ++e) gsum[j][e] += g[e];          // fp32 rank sum, m ascending
          } else {   // numerics study: the rank's term as a 16-bit wire carries it; optionally a 16-bit running sum
#pragma unroll
            for (int e = 0; e < V; ++e) {
              const float sum = gsum[j][e] + V_::round(g[e]);
              gsum[j][e] = a.reduce_mode == 2 ? V_::round(sum) : sum;
            }
          }
        } else {
          float zp[V];
          if (cls[j] == 1) {
#pragma unroll
            for (int e = 0; e < V; ++e) zp[e] = a.alpha * g[e];    // private gradient carries alpha
          } else {
#pragma unroll
            for (int e = 0; e < V; ++e) {
              const bool shared = col[j] + e < a.S;
              const float term = shared ? (a.reduce_mode ? V_::round(g[e]) : g[e]) : 0.f;
              gsum[j][e] = a.reduce_mode == 2 ? V_::round(gsum[j][e] + term) : gsum[j][e] + term;
              zp[e] = shared ? 0.f : a.alpha * g[e];
            }
          }
          if (act[j] && a.zp) stg<raw>(pZ[j], V_::pack(zp));
        }
        pZ[j] += rank_p;
      }
#pragma unroll
      for (int j = 0; j < CPT; ++j) { rdX[j] = ndX[j]; rHn[j] = nHn[j]; rdH[j] = ndH[j]; }
      rs_c = rs_n; mu_c = mu_n;
    }
#pragma unroll
    for (int j = 0; j < CPT; ++j)
      if (act[j] && cls[j] != 1)
        stg<raw>(gs_row(a, i, ES) + (long long)col[j] * ES, V_::pack(gsum[j]));
  }

  // Partial norm-parameter gradients of this CTA: one row of [h] per CTA.  With several
  // token rows per CTA (TY > 1) they are first summed through shared memory, in order.
  for (int which = 0; which < (LN ? 2 : 1); ++which) {
    float* out = which == 0 ? a.dgpart : a.dbpart;
    if (out == nullptr) continue;
    if (blockDim.y == 1) {
#pragma unroll
      for (int j = 0; j < CPT; ++j) {
        if (!colok[j]) continue;
        const float* src = (which == 0 || !LN) ? dgacc[j] : dbacc[LN ? j : 0];
#pragma unroll
        for (int e = 0; e < V; e += 4)
          *reinterpret_cast<float4*>(out + (size_t)blockIdx.x * a.h + col[j] + e) =
              make_float4(src[e], src[e + 1], src[e + 2], src[e + 3]);
      }
      continue;
    }
    __syncthreads();
    float* acc = red;  // reuse: [TY][TX*CPT*V]
    const int per_row = TX * CPT * V;
#pragma unroll
    for (int j = 0; j < CPT; ++j)
#pragma unroll
      for (int e = 0; e < V; ++e)
        acc[(size_t)threadIdx.y * per_row + (j * TX + threadIdx.x) * V + e] =
            (which == 0 || !LN) ? dgacc[j][e] : dbacc[LN ? j : 0][e];
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
  }
}

// ------------------------------------------------------------------ forward from fp32 partial planes (decode)
// One CTA per (token, rank).  zt holds fp32 partial outputs [splits * t, T, h] for ALL channels (plane
// z = split * t + rank).  Shared channels: sum of every plane, z ascending; private channels: sum over
// the splits of this rank's planes, times alpha.  Every rank's CTA forms the shared sum for itself (a few
// kilobytes, L2 hits), so no CTA waits for another.  With two layers the second one's residual is the
// first one's new residual stream as stored (rounded to the storage type).
template <typename T_, bool LN>
__global__ void __launch_bounds__(512) rows_forward_partials_kernel(const RowPartArgs a) {
  using V_ = VT<T_>;
  using raw = typename V_::raw;
  constexpr int V = V_::N;
  constexpr int ES = sizeof(T_);
  extern __shared__ float sm[];
  pdl_wait();
  float* hrow = sm;                       // [h] the new residual stream of this row, fp32
  float* red = sm + a.h;                  // reduction scratch
  int par = 0;
  const int i = blockIdx.x, m = blockIdx.y;
  const long long row = (long long)m * a.T + i;
  const long long plane = (long long)a.T * a.h;
  const float inv_h = 1.0f / (float)a.h;
  for (int layer = 0; layer < a.nlayers; ++layer) {
    const PartialLayer& L = a.L[layer];
    const int nplanes = L.splits * a.t;
    float st[1] = {0.f};
    for (int c = threadIdx.x * V; c < a.h; c += blockDim.x * V) {
      float r[V], z[V], hn[V];
      const bool shared_chunk = c + V <= a.S;          // the partition is a multiple of 8 on this path
      // compact layout: where this chunk of the stream lives (shared part once, private part per rank)
      const long long coff = shared_chunk ? ((long long)i * a.S + c) * ES : (row * (a.h - a.S) + (c - a.S)) * ES;
      if (layer == 0) {
        if (a.compact) V_::unpack(ldg<raw>(static_cast<const char*>(shared_chunk ? a.Rs : a.R) + coff), r);
        else V_::unpack(ldg<raw>(static_cast<const char*>(a.R) + (row * a.h + c) * ES), r);
      } else {
#pragma unroll
        for (int e = 0; e < V; ++e) r[e] = V_::round(hrow[c + e]);
      }
#pragma unroll
      for (int e = 0; e < V; ++e) z[e] = 0.f;
      const float* base = L.zt + (long long)i * a.h + c;
      const int z0 = shared_chunk ? 0 : m, zstep = shared_chunk ? 1 : a.t;
      const int nz = shared_chunk ? nplanes : L.splits;
#pragma unroll 8
      for (int q = 0; q < nz; ++q) {
        const float* pz = base + (long long)(z0 + q * zstep) * plane;
#pragma unroll
        for (int e = 0; e < V; e += 4) {
          const float4 v = *reinterpret_cast<const float4*>(pz + e);
          z[e] += v.x; z[e + 1] += v.y; z[e + 2] += v.z; z[e + 3] += v.w;
        }
      }
#pragma unroll
      for (int e = 0; e < V; ++e) {
        hn[e] = (shared_chunk ? z[e] : a.alpha * z[e]) + r[e];
        st[0] = LN ? st[0] + hn[e] : fmaf(hn[e], hn[e], st[0]);
      }
      // (a thread reads and writes only its own chunks of hrow: no ordering between threads is needed, and a
      // warp-wide sync here would deadlock rows whose chunk count is not a multiple of 32)
#pragma unroll
      for (int e = 0; e < V; ++e) hrow[c + e] = hn[e];
      if (a.compact) {      // every rank's CTA forms the same shared values; rank 0's writes them
        if (!shared_chunk || m == 0) stg<raw>(static_cast<char*>(shared_chunk ? L.Hns : L.Hn) + coff, V_::pack(hn));
      } else {
        stg<raw>(static_cast<char*>(L.Hn) + (row * a.h + c) * ES, V_::pack(hn));
      }
    }
    row_reduce_sync<1>(st, red, par);
    float mu = 0.f, rs;
    if (LN) {
      mu = st[0] * inv_h;
      float sq[1] = {0.f};
      for (int c = threadIdx.x * V; c < a.h; c += blockDim.x * V)
#pragma unroll
        for (int e = 0; e < V; ++e) { const float d = hrow[c + e] - mu; sq[0] = fmaf(d, d, sq[0]); }
      row_reduce_sync<1>(sq, red, par);
      rs = rsqrtf(fmaf(sq[0], inv_h, a.eps));
    } else {
      rs = rsqrtf(fmaf(st[0], inv_h, a.eps));
    }
    for (int c = threadIdx.x * V; c < a.h; c += blockDim.x * V) {
      float g[V], b[V], x[V];
      V_::unpack(ldg<raw>(static_cast<const char*>(L.gamma) + (long long)c * ES), g);
#pragma unroll
      for (int e = 0; e < V; ++e) b[e] = 0.f;
      if (LN && L.beta) V_::unpack(ldg<raw>(static_cast<const char*>(L.beta) + (long long)c * ES), b);
#pragma unroll
      for (int e = 0; e < V; ++e) x[e] = LN ? fmaf(hrow[c + e] - mu, rs * g[e], b[e]) : hrow[c + e] * (rs * g[e]);
      stg<raw>(static_cast<char*>(L.X) + (row * a.h + c) * ES, V_::pack(x));
    }
    if (threadIdx.x == 0) {
      L.rstd[row] = rs;
      if (LN && L.mean) L.mean[row] = mu;
    }
  }
}


// ---- the same step for very few rows: a cluster of t CTAs per token ------------------------------
// With a handful of tokens the kernel above is one long dependency chain per CTA: every rank's CTA
// sums all splits * t planes of the shared channels, eight loads at a time, layer after layer.  Here
// the t CTAs of a token form a thread-block cluster and divide that work: CTA m fetches, with
// asynchronous 16-byte copies that are all in flight at once (both layers), a 1/t slice of the shared
// channels of every plane plus its own rank's private channels; it sums its slice (planes ascending,
// the order of the kernel above, so the results are bit-identical) and stores the sums into every peer's
// shared memory; one cluster barrier later each CTA holds the complete rank sum.  A thread owns one
// 16-byte chunk of the row for both layers (rows of up to 512 chunks), so the new residual stream stays
// in registers between the statistics, the normalisation and the second layer.
namespace cgx = cooperative_groups;

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;"
               ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// float4 slots of the staging area a CTA needs (the widest shared slice is ceil(S/4 / t) chunks)
inline size_t cluster_partials_smem(const RowPartArgs& a) {
  const int S4 = a.S / 4, P4 = (a.h - a.S) / 4;
  const int ns_max = (S4 + a.t - 1) / a.t;
  size_t f4 = (size_t)a.nlayers * S4 + 16;            // rank sums of the shared channels, reduction scratch
  for (int l = 0; l < a.nlayers; ++l) f4 += (size_t)a.L[l].splits * ((size_t)a.t * ns_max + P4);
  return f4 * sizeof(float4);
}

template <typename T_, bool LN, int MINB>
__global__ void __launch_bounds__(512, MINB) rows_forward_partials_cluster_kernel(const RowPartArgs a) {
  using V_ = VT<T_>;
  using raw = typename V_::raw;
  constexpr int V = V_::N;
  constexpr int ES = sizeof(T_);
  extern __shared__ float4 sm4[];
  cgx::cluster_group cluster = cgx::this_cluster();
  const int i = blockIdx.x, m = blockIdx.y;             // the cluster spans the ranks of token i: cluster rank == m
  const int tid = threadIdx.x, nthr = blockDim.x;
  const int S4 = a.S / 4, P4 = (a.h - a.S) / 4;
  const int cs0 = (int)((long long)S4 * m / a.t);       // this CTA's slice of the shared channels, in float4 units
  const int ns = (int)((long long)S4 * (m + 1) / a.t) - cs0;
  float4* zs = sm4;                                     // [nlayers][S4]: complete after the cluster barrier
  float* red = reinterpret_cast<float*>(sm4 + a.nlayers * S4);
  float4* stage = sm4 + a.nlayers * S4 + 16;
  const long long row = (long long)m * a.T + i;
  const long long plane = (long long)a.T * a.h;
  int par = 0;
  // a peer's shared memory may be written only once that CTA runs: arrive now, wait before the first remote store
  asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
  pdl_wait();

  // ---- every partial this CTA needs, both layers, in flight at once
  int sh_off[2] = {0, 0}, pr_off[2] = {0, 0};
  {
    int off = 0;
#pragma unroll
    for (int l = 0; l < 2; ++l) {
      if (l >= a.nlayers) break;
      const int splits = a.L[l].splits, nplanes = splits * a.t;
      const float* zt = a.L[l].zt + (long long)i * a.h;
      sh_off[l] = off;
      for (int idx = tid; idx < nplanes * ns; idx += nthr) {
        const int z = idx / ns, c = idx - z * ns;
        cp_async16(stage + off + idx, zt + z * plane + 4 * (cs0 + c));
      }
      off += nplanes * ns;
      pr_off[l] = off;
      for (int idx = tid; idx < splits * P4; idx += nthr) {
        const int q = idx / P4, c = idx - q * P4;
        cp_async16(stage + off + idx, zt + (long long)(m + q * a.t) * plane + a.S + 4 * c);
      }
      off += splits * P4;
    }
  }
  // ---- this thread's chunk of the row: residual and norm parameters, fetched behind the copies
  const int c = tid * V;
  const bool active = c < a.h;
  const bool shared_chunk = c + V <= a.S;               // the partition is a multiple of 8 on this path
  const long long coff = shared_chunk ? ((long long)i * a.S + c) * ES : (row * (a.h - a.S) + (c - a.S)) * ES;
  float r[V], g[2][V], b[2][V];
#pragma unroll
  for (int e = 0; e < V; ++e) { r[e] = 0.f; g[0][e] = g[1][e] = 0.f; b[0][e] = b[1][e] = 0.f; }
  if (active) {
    if (a.compact) V_::unpack(ldg<raw>(static_cast<const char*>(shared_chunk ? a.Rs : a.R) + coff), r);
    else V_::unpack(ldg<raw>(static_cast<const char*>(a.R) + (row * a.h + c) * ES), r);
#pragma unroll
    for (int l = 0; l < 2; ++l) {
      if (l >= a.nlayers) break;
      V_::unpack(ldg<raw>(static_cast<const char*>(a.L[l].gamma) + (long long)c * ES), g[l]);
      if (LN && a.L[l].beta) V_::unpack(ldg<raw>(static_cast<const char*>(a.L[l].beta) + (long long)c * ES), b[l]);
    }
  }
  cp_async_wait_all();
  __syncthreads();
  asm volatile("barrier.cluster.wait.aligned;" ::: "memory");

  // ---- sums: planes ascending.  Shared slice -> every CTA of the cluster; private -> in place (split 0's slot)
#pragma unroll
  for (int l = 0; l < 2; ++l) {
      if (l >= a.nlayers) break;
    const int splits = a.L[l].splits, nplanes = splits * a.t;
    for (int q = tid; q < ns; q += nthr) {
      const float4* src = stage + sh_off[l] + q;
      float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int z = 0; z < nplanes; ++z) {
        const float4 v = src[(size_t)z * ns];
        s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
      }
      for (int peer = 0; peer < a.t; ++peer) cluster.map_shared_rank(zs, peer)[l * S4 + cs0 + q] = s;
    }
    for (int q = tid; q < P4; q += nthr) {
      float4* src = stage + pr_off[l] + q;
      float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int k = 0; k < splits; ++k) {
        const float4 v = src[(size_t)k * P4];
        s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
      }
      *src = s;
    }
  }
  cluster.sync();     // every slice has arrived (and this CTA's own private sums are visible to all its threads)

  const float inv_h = 1.0f / (float)a.h;
  float hn[V];
#pragma unroll
  for (int e = 0; e < V; ++e) hn[e] = 0.f;
#pragma unroll
  for (int l = 0; l < 2; ++l) {
      if (l >= a.nlayers) break;
    const PartialLayer& L = a.L[l];
    float st[1] = {0.f};
    if (active) {
      float z[V];
      const float4* src = shared_chunk ? zs + l * S4 + c / 4 : stage + pr_off[l] + (c - a.S) / 4;
#pragma unroll
      for (int e = 0; e < V; e += 4) {
        const float4 v = src[e / 4];
        z[e] = v.x; z[e + 1] = v.y; z[e + 2] = v.z; z[e + 3] = v.w;
      }
#pragma unroll
      for (int e = 0; e < V; ++e) {
        const float res = l == 0 ? r[e] : V_::round(hn[e]);    // the second layer's residual is the first one's stream as stored
        hn[e] = (shared_chunk ? z[e] : a.alpha * z[e]) + res;
        st[0] = LN ? st[0] + hn[e] : fmaf(hn[e], hn[e], st[0]);
      }
      if (a.compact) {      // every rank's CTA forms the same shared values; rank 0's writes them
        if (!shared_chunk || m == 0) stg<raw>(static_cast<char*>(shared_chunk ? L.Hns : L.Hn) + coff, V_::pack(hn));
      } else {
        stg<raw>(static_cast<char*>(L.Hn) + (row * a.h + c) * ES, V_::pack(hn));
      }
    }
    row_reduce_sync<1>(st, red, par);
    float mu = 0.f, rs;
    if (LN) {
      mu = st[0] * inv_h;
      float sq[1] = {0.f};
      if (active) {
#pragma unroll
        for (int e = 0; e < V; ++e) { const float d = hn[e] - mu; sq[0] = fmaf(d, d, sq[0]); }
      }
      row_reduce_sync<1>(sq, red, par);
      rs = rsqrtf(fmaf(sq[0], inv_h, a.eps));
    } else {
      rs = rsqrtf(fmaf(st[0], inv_h, a.eps));
    }
    if (active) {
      float x[V];
#pragma unroll
      for (int e = 0; e < V; ++e) x[e] = LN ? fmaf(hn[e] - mu, rs * g[l][e], b[l][e]) : hn[e] * (rs * g[l][e]);
      stg<raw>(static_cast<char*>(L.X) + (row * a.h + c) * ES, V_::pack(x));
    }
    if (tid == 0) {
      L.rstd[row] = rs;
      if (LN && L.mean) L.mean[row] = mu;
    }
  }
}

// *launched = false (and cudaSuccess) when this device cannot place such a cluster: the caller then
// takes the general kernel.
template <typename T_, bool LN, int MINB>
cudaError_t launch_partials_cluster(const RowPartArgs& a, int threads, size_t smem, cudaStream_t st, bool* launched) {
  *launched = false;
  static bool attr_set[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  std::unique_lock<std::mutex> lock(host_cache_mutex());   // attribute flag and the occupancy answers below
  if (!attr_set[dev]) {
    const cudaError_t e = cudaFuncSetAttribute(rows_forward_partials_cluster_kernel<T_, LN, MINB>,
                                               cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    attr_set[dev] = true;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(a.T, a.t);
  cfg.blockDim = dim3(threads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2] = {};
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 1;
  attr[0].val.clusterDim.y = (unsigned)a.t;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  // can a cluster of t such CTAs be co-scheduled here at all?  (asked once per device, cluster size and footprint)
  struct Seen { int dev, t, threads; size_t smem; int clusters; };
  static Seen seen[8] = {};
  static int nseen = 0;
  int clusters = -1;
  for (int q = 0; q < nseen; ++q)
    if (seen[q].dev == dev && seen[q].t == a.t && seen[q].threads == threads && seen[q].smem == smem) clusters = seen[q].clusters;
  if (clusters < 0) {
    if (cudaOccupancyMaxActiveClusters(&clusters, rows_forward_partials_cluster_kernel<T_, LN, MINB>, &cfg) != cudaSuccess) {
      cudaGetLastError();
      clusters = 0;
    }
    // a full table forgets its oldest entry instead of asking the device again on every launch
    static int next = 0;
    const int slot = nseen < 8 ? nseen++ : (next++ & 7);
    seen[slot] = Seen{dev, a.t, threads, smem, clusters};
  }
  lock.unlock();
  if (clusters < 1) return cudaSuccess;
  cfg.numAttrs = pdl_enabled() ? 2 : 1;
  *launched = true;
  return cudaLaunchKernelEx(&cfg, rows_forward_partials_cluster_kernel<T_, LN, MINB>, a);
}

// out[l] = sum over `rows` partial rows, fixed order: 32 row lanes then a serial combine.
// Blocks past the first `nreduce` run an unrelated small job that has to happen between the row kernel and the
// data gradient anyway and would otherwise cost a launch of its own: scaling the private rows of the weights.
struct ScaleJob { const uint4* src; uint4* dst; int t, h, K_r, S; float alpha; };

__global__ void __launch_bounds__(1024) reduce_partials_kernel(const float* __restrict__ part, float* __restrict__ out,
                                                               int rows, int h, int nreduce, ScaleJob job) {
  __shared__ float sm[32][33];
  pdl_wait();
  if ((int)blockIdx.x >= nreduce) {
    const int row_chunks = job.K_r / 8;
    const long long per_rank = (long long)(job.h - job.S) * row_chunks, total = per_rank * job.t;
    const long long nthreads = (long long)(gridDim.x - nreduce) * 1024;
    for (long long q = (long long)(blockIdx.x - nreduce) * 1024 + threadIdx.y * 32 + threadIdx.x; q < total; q += nthreads) {
      const long long m = q / per_rank, r = q - m * per_rank;
      const long long idx = (m * job.h + job.S) * row_chunks + r;
      const uint4 v = job.src[idx];
      const unsigned w[4] = {v.x, v.y, v.z, v.w};
      unsigned o[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        __nv_bfloat162 bb = __floats2bfloat162_rn(job.alpha * __uint_as_float(w[i] << 16),
                                                  job.alpha * __uint_as_float(w[i] & 0xffff0000u));
        o[i] = *reinterpret_cast<unsigned*>(&bb);
      }
      job.dst[idx] = make_uint4(o[0], o[1], o[2], o[3]);
    }
    return;
  }
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

template <typename T_, bool LN, bool CL>
cudaError_t launch_fwd_t(const RowFwdArgs& a, const RowGeom& g, cudaStream_t st) {
  const dim3 block(g.TX, g.TY);
  const dim3 grid((a.T + g.TY - 1) / g.TY);
  LaunchScope scope(CAAT_K_ROWS_FORWARD, st);
  switch (g.CPT) {
    case 1: rows_forward_kernel<T_, 1, LN, CL><<<grid, block, g.smem_fwd, st>>>(a); break;
    case 2: rows_forward_kernel<T_, 2, LN, CL><<<grid, block, g.smem_fwd, st>>>(a); break;
    case 4: rows_forward_kernel<T_, 4, LN, CL><<<grid, block, g.smem_fwd, st>>>(a); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

template <typename T_, bool LN, bool CL>
cudaError_t launch_bwd_t(const RowBwdArgs& a, const RowGeom& g, int rows, cudaStream_t st) {
  const dim3 block(g.TX, g.TY);
  const int ngroups = (a.T + g.TY - 1) / g.TY;
  const dim3 grid(rows);
  LaunchScope scope(CAAT_K_ROWS_BACKWARD, st);
  switch (g.CPT) {
    case 1: rows_backward_kernel<T_, 1, LN, CL><<<grid, block, g.smem_bwd, st>>>(a, ngroups); break;
    case 2: rows_backward_kernel<T_, 2, LN, CL><<<grid, block, g.smem_bwd, st>>>(a, ngroups); break;
    case 4: rows_backward_kernel<T_, 4, LN, CL><<<grid, block, g.smem_bwd, st>>>(a, ngroups); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_rows_forward_partials(const RowPartArgs& a, caat_dtype dtype, cudaStream_t st) {
  const int V = dtype == CAAT_BF16 ? 8 : 4;
  int threads = round_up(a.h / V, 32);               // one chunk per thread when the row allows
  if (threads > 512) threads = 512;
  if (threads < 32) threads = 32;
  const dim3 grid(a.T, a.t);
  const size_t smem = (size_t)a.h * sizeof(float) + 2 * 16 * 2 * sizeof(float);
  LaunchScope scope(CAAT_K_ROWS_FORWARD, st);
  // few rows: the cluster kernel, as long as all its CTAs are resident at once (portable cluster size 8,
  // one chunk per thread, one CTA per SM at its register count; clusters need whole groups of SMs, hence 3/4)
#ifdef CAAT_MEASUREMENT_AIDS
  static const int cluster_mode = [] { const char* e = getenv("CAAT_DECODE_CLUSTER"); return e ? atoi(e) : 1; }();
#else
  constexpr int cluster_mode = 1;
#endif
  if (cluster_mode && dtype == CAAT_BF16 && a.t >= 2 && a.t <= 8 && a.h % V == 0 && a.h / V <= 512 && a.S % 4 == 0 &&
      (a.h - a.S) % 4 == 0) {
    const size_t csm = cluster_partials_smem(a);
    bool launched = false;
    cudaError_t e = cudaSuccess;
    if (csm <= 200 * 1024 && (long long)a.T * a.t <= (long long)sm_count() * 3 / 4) {
      e = a.norm == 1 ? launch_partials_cluster<__nv_bfloat16, true, 1>(a, threads, csm, st, &launched)
                      : launch_partials_cluster<__nv_bfloat16, false, 1>(a, threads, csm, st, &launched);
      if (launched || e != cudaSuccess) return e;
    }
    // more rows than that: two CTAs per SM (64 registers, RMSNorm variant), a few waves.  Pays when most
    // channels are shared, where the kernel below reads every shared plane once per rank (measured at
    // 64 tokens of the 7B shapes: 3 % faster at p = 1, 5 % slower at p = 0.5).
    if (a.norm != 1 && csm <= 100 * 1024 && (long long)a.S * 4 > (long long)a.h * 3 &&
        (long long)a.T * a.t <= (long long)sm_count() * 4) {
      e = launch_partials_cluster<__nv_bfloat16, false, 2>(a, threads, csm, st, &launched);
      if (launched || e != cudaSuccess) return e;
    }
  }
  // more rows than two CTAs of 512 threads per SM can hold at once (64 registers per thread): two chunks per thread in
  // CTAs of 256, four of which fit an SM, keep every row's CTA resident in one wave (7B shapes, 64 tokens: -3.6 %)
  if (threads > 256 && (long long)a.T * a.t > 2LL * sm_count()) threads = 256;
  auto go = [&](auto kernel) -> cudaError_t {
    if (smem > 48 * 1024) {   // long rows: more dynamic shared memory than a kernel gets without asking
      const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
    }
    return launch_pdl(kernel, grid, dim3(threads), smem, st, a);
  };
  if (dtype == CAAT_BF16)
    return a.norm == 1 ? go(rows_forward_partials_kernel<__nv_bfloat16, true>) : go(rows_forward_partials_kernel<__nv_bfloat16, false>);
  return a.norm == 1 ? go(rows_forward_partials_kernel<float, true>) : go(rows_forward_partials_kernel<float, false>);
}

RowsHooks rows_hooks() {
  static const RowsHooks hooks = [] {
    RowsHooks k{1u << 18, 0};
    if (const char* e = getenv("CAAT_ROWS_SPINCAP")) { const int v = atoi(e); if (v >= 16) k.spin_cap = (uint32_t)v; }
    if (const char* e = getenv("CAAT_ROWS_STALL")) k.stall = atoi(e) == 1 ? 1 : 0;
    return k;
  }();
  return hooks;
}

int rows_backward_partial_rows(int h, int T, caat_dtype dtype) {
  const RowGeom g = row_geometry(h, dtype);
  const int ngroups = (T + g.TY - 1) / g.TY;
  return ngroups < kMaxPartialRows ? ngroups : kMaxPartialRows;
}

static int rows_mode_override(int direct) {   // measurement builds: CAAT_ROWS_MODE = 0/1/2 overrides the context option
#ifdef CAAT_MEASUREMENT_AIDS
  static const int env = [] { const char* e = getenv("CAAT_ROWS_MODE"); return e ? atoi(e) : -1; }();
  return env >= 0 ? env : direct;
#else
  return direct;
#endif
}

cudaError_t launch_rows_forward(const RowFwdArgs& a, caat_dtype dtype, int direct, cudaStream_t st) {
  direct = rows_mode_override(direct);
  if (direct == 0 && rows_warp_cpt(a.h, a.t, dtype) > 0) return launch_rows_forward_warp(a, dtype, st);
  if (direct != 1 && rows_staged_usable(a.h, a.t, a.S_lo, a.S_hi, dtype, false)) return launch_rows_forward_staged(a, dtype, st);
  const RowGeom g = row_geometry(a.h, dtype);
  if (a.compact) {
    if (dtype == CAAT_BF16)
      return a.norm == 1 ? launch_fwd_t<__nv_bfloat16, true, true>(a, g, st) : launch_fwd_t<__nv_bfloat16, false, true>(a, g, st);
    return a.norm == 1 ? launch_fwd_t<float, true, true>(a, g, st) : launch_fwd_t<float, false, true>(a, g, st);
  }
  if (dtype == CAAT_BF16)
    return a.norm == 1 ? launch_fwd_t<__nv_bfloat16, true, false>(a, g, st) : launch_fwd_t<__nv_bfloat16, false, false>(a, g, st);
  return a.norm == 1 ? launch_fwd_t<float, true, false>(a, g, st) : launch_fwd_t<float, false, false>(a, g, st);
}

cudaError_t launch_rows_backward(const RowBwdArgs& a, caat_dtype dtype, int direct, cudaStream_t st) {
  direct = rows_mode_override(direct);
  const RowGeom g = row_geometry(a.h, dtype);
  int rows = rows_backward_partial_rows(a.h, a.T, dtype);
  cudaError_t e;
  if (direct == 0 && rows_warp_cpt(a.h, a.t, dtype) > 0)
    e = launch_rows_backward_warp(a, dtype, rows, &rows, st);
  else if (direct != 1 && rows_staged_usable(a.h, a.t, a.S_lo, a.S_hi, dtype, true))
    e = launch_rows_backward_staged(a, dtype, rows, &rows, st);
  else if (a.compact && dtype == CAAT_BF16)
    e = a.norm == 1 ? launch_bwd_t<__nv_bfloat16, true, true>(a, g, rows, st) : launch_bwd_t<__nv_bfloat16, false, true>(a, g, rows, st);
  else if (a.compact)
    e = a.norm == 1 ? launch_bwd_t<float, true, true>(a, g, rows, st) : launch_bwd_t<float, false, true>(a, g, rows, st);
  else if (dtype == CAAT_BF16)
    e = a.norm == 1 ? launch_bwd_t<__nv_bfloat16, true, false>(a, g, rows, st) : launch_bwd_t<__nv_bfloat16, false, false>(a, g, rows, st);
  else
    e = a.norm == 1 ? launch_bwd_t<float, true, false>(a, g, rows, st) : launch_bwd_t<float, false, false>(a, g, rows, st);
  if (e != cudaSuccess) return e;
  const dim3 rb(32, 32);
  const int nreduce = (a.h + 31) / 32;
  ScaleJob job{};
  int nscale = 0;
  if (a.w_dst && a.w_src && a.S < a.h) {
    job = ScaleJob{static_cast<const uint4*>(a.w_src), static_cast<uint4*>(a.w_dst), a.t, a.h, a.w_Kr, a.S, a.alpha};
    const long long total = (long long)a.t * (a.h - a.S) * (a.w_Kr / 8);
    nscale = (int)((total + 4 * 1024 - 1) / (4 * 1024));          // four 16-byte chunks per thread
    if (nscale > 148) nscale = 148;
    if (nscale < 1) nscale = 1;
  }
  {
    LaunchScope scope(CAAT_K_NORMGRAD_REDUCE, st);
    e = launch_pdl(reduce_partials_kernel, dim3(nreduce + nscale), rb, 0, st, (const float*)a.dgpart, a.dgamma, rows, a.h,
                   nreduce, job);
    if (e != cudaSuccess) return e;
  }
  if (a.norm == 1 && a.dbeta && a.dbpart) {
    LaunchScope scope(CAAT_K_NORMGRAD_REDUCE, st);
    e = launch_pdl(reduce_partials_kernel, dim3(nreduce), rb, 0, st, (const float*)a.dbpart, a.dbeta, rows, a.h, nreduce,
                   ScaleJob{});
    if (e != cudaSuccess) return e;
  }
  return cudaGetLastError();
}

}  // namespace caat
