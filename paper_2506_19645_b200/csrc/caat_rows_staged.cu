// Row kernels, bulk-copy staged variant (the default).
//
// The row work is pure streaming: what limits it is how many bytes a CTA keeps in flight.
// With plain loads that is bounded by registers (threads x loads per thread); here the
// inputs of one (token group, rank) - a few contiguous rows - are fetched by ONE thread
// with cp.async.bulk into a shared-memory ring, several ranks (and token groups) ahead,
// completion signalled on an mbarrier per stage.  Consumer threads keep the mapping of
// the direct kernels (a thread owns the same 16-byte column chunk of every rank of its
// token; rank sums are thread-local and run m = 0..t-1), read their chunk from shared
// memory and write results with 128-bit stores.  The CTA-wide barrier of the row
// reduction doubles as the "stage is free" signal, so there are no empty-barriers.
//
// CTAs are persistent (token groups strided by the grid).  Every mbarrier wait is bounded:
// on a timeout the CTA sets the library's status word, drains its copies in flight and
// returns.
#include "caat_rows_bulk.cuh"

namespace caat {
namespace {

using namespace rows;

// ------------------------------------------------------------------ forward
// stage buffers: a = R rows [TY, h], b = zp rows [TY, P], c = zs rows [TY, S_hi] (rank 0 only)
// compact layout (CL): a = private residual rows [TY, P], d = shared residual rows [TY, S] (rank 0 only)
template <typename T_, int CPT, bool LN, int MAXT, bool CL>
__global__ void __launch_bounds__(MAXT, MinBlocks<CPT, MAXT>::value)
rows_forward_staged(const RowFwdArgs a, const StageGeom sg, int ngroups, unsigned int* status) {
  using V_ = VT<T_>;
  using raw = typename V_::raw;
  constexpr int V = V_::N;
  constexpr int ES = sizeof(T_);
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t* ring = smem + sg.ring_off;
  const uint32_t bar0 = smem_u32(smem + sg.bar_off);
  float* red = reinterpret_cast<float*>(smem + sg.red_off);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + sg.bar_off + 8 * kMaxStages);
  int par = 0;
  const int TX = blockDim.x, TY = blockDim.y;
  const bool leader = threadIdx.x == 0 && threadIdx.y == 0;
  const float inv_h = 1.0f / (float)a.h;
  const int NS = sg.nstages;
  const bool has_priv = a.P > 0 && a.S < a.h;
  const bool has_shared = a.S > 0;

  // sequence k = n * t + m over this CTA's (token group n, rank m) pairs
  const int my_groups = blockIdx.x < ngroups ? (ngroups - blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  const long long total = (long long)my_groups * a.t;

  // Fetch the inputs of (token group nn, rank mm) into stage ss.  Every thread calls it (all keep the
  // counters); the copies of a stage are issued by lane 0 of DIFFERENT warps, so that no warp carries
  // more than one copy's issue latency into the next CTA barrier.  Warp 0 posts the expected bytes with
  // its arrival; a copy landing before that only drives the byte count negative for a moment, the phase
  // cannot complete before the arrival.
  int nn = 0, mm = 0, ss = 0;
  const int issuer = __shfl_sync(0xffffffffu, (int)(threadIdx.y * TX + threadIdx.x) >> 5, 0);   // warp index, warp-uniform
  auto issue = [&]() {
    if (nn >= my_groups) return;
    const int n = nn, m = mm, s = ss;
    if (++mm == a.t) { mm = 0; ++nn; }
    if (++ss == NS) ss = 0;
    if (issuer > 3) return;
    const long long g = blockIdx.x + (long long)n * gridDim.x;
    const long long i0 = g * TY;
    const int rowsN = (int)((a.T - i0) < TY ? (a.T - i0) : TY);
    const uint32_t bar = bar0 + 8u * s;
    const uint32_t dst = smem_u32(ring + (size_t)s * sg.stage_bytes);
    const uint32_t bP = has_priv ? (uint32_t)rowsN * a.P * ES : 0u;
    const uint32_t bR = CL ? bP : (uint32_t)rowsN * a.h * ES;
    const uint32_t bS = (m == 0 && has_shared) ? (uint32_t)rowsN * a.S_hi * ES : 0u;
    const long long row = (long long)m * a.T + i0;
    if (!elect_one()) return;
    if (issuer == 0) {
      mbar_expect_tx(bar, bR + bP + (CL ? 2 * bS : bS) + sg.stall_bytes);
      if (bR) bulk_g2s(dst + sg.off_a, static_cast<const char*>(a.R) + row * (CL ? a.P : a.h) * ES, bR, bar);
    } else if (issuer == 1) {
      if (bP) bulk_g2s(dst + sg.off_b, static_cast<const char*>(a.zp) + row * a.P * ES, bP, bar);
    } else if (issuer == 2) {
      if (bS) bulk_g2s(dst + sg.off_c, static_cast<const char*>(a.zs) + i0 * a.S_hi * ES, bS, bar);
    } else {
      if (CL && bS) bulk_g2s(dst + sg.off_d, static_cast<const char*>(a.Rs) + i0 * a.S_hi * ES, bS, bar);
    }
  };

  if (leader) {
    for (int s = 0; s < NS; ++s) mbar_init(bar0 + 8u * s, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if ((int)(threadIdx.y * TX + threadIdx.x) < NS)   // the zero slot of every stage (no copy ever lands there)
    *reinterpret_cast<uint4*>(ring + (size_t)(threadIdx.y * TX + threadIdx.x) * sg.stage_bytes + sg.zero_off) =
        make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
  pdl_wait();   // from here on global memory is touched
  for (int q = 0; q < NS; ++q) issue();

  // Per-thread constants of the hot loop: the chunk's class and its byte offsets inside a stage.  Chunks
  // past the row end read a zeroed slot that every stage carries, so the loop needs no bounds predicates
  // on its loads.
  constexpr int H2 = V / 2;
  const uint32_t ring32 = smem_u32(ring);
  int col[CPT], cls[CPT];
  bool colok[CPT];
  uint32_t oA[CPT], oB[CPT];
  float2 gam[CPT][H2], bet[LN ? CPT : 1][H2];
#pragma unroll
  for (int j = 0; j < CPT; ++j) {
    col[j] = (threadIdx.x + j * TX) * V;
    colok[j] = col[j] < a.h;
    cls[j] = chunk_class(col[j], V, a.S);
#pragma unroll
    for (int q = 0; q < H2; ++q) { gam[j][q] = f2(0.f); if constexpr (LN) bet[j][q] = f2(0.f); }
    oA[j] = oB[j] = sg.zero_off;
    if (colok[j]) {
      unpack2(ldg<raw>(static_cast<const char*>(a.gamma) + (long long)col[j] * ES), gam[j]);
      if constexpr (LN) {
        if (a.beta) unpack2(ldg<raw>(static_cast<const char*>(a.beta) + (long long)col[j] * ES), bet[j]);
      }
      const uint32_t priv = ((uint32_t)threadIdx.y * a.P + (uint32_t)(col[j] - a.S_lo)) * ES;
      if (cls[j] != 0) oB[j] = sg.off_b + priv;
      if (CL) { if (cls[j] != 0) oA[j] = sg.off_a + priv; }
      else oA[j] = sg.off_a + ((uint32_t)threadIdx.y * a.h + col[j]) * ES;
    }
  }
  const float2 alpha2 = f2(a.alpha);
  const long long rank_h = (long long)a.T * a.h * ES;
  const long long rank_hn = CL ? (long long)a.T * a.P * ES : rank_h;

  long long k = 0;
  uint32_t sb = ring32;   // consumer's stage (shared address), its index and phase parity
  int cs = 0;
  uint32_t cph = 0;
  bool dead = false;
  for (int n = 0; n < my_groups && !dead; ++n) {
    const long long g = blockIdx.x + (long long)n * gridDim.x;
    const long long i = g * TY + threadIdx.y;
    const bool valid = i < a.T;
    bool act[CPT];
    float2 zs[CPT][H2];     // shared part of the layer output (compact: of the new stream), formed once per token
    char* pHn[CPT];
    char* pX[CPT];
#pragma unroll
    for (int j = 0; j < CPT; ++j) {
      act[j] = valid && colok[j];
      const long long off_h = (i * a.h + col[j]) * ES;
      if (CL) pHn[j] = cls[j] == 0 ? static_cast<char*>(a.Hns) + (i * a.S_hi + col[j]) * ES
                                   : static_cast<char*>(a.Hn) + (i * a.P + (col[j] - a.S_lo)) * ES;
      else pHn[j] = static_cast<char*>(a.Hn) + off_h;
      pX[j] = static_cast<char*>(a.X) + off_h;
#pragma unroll
      for (int q = 0; q < H2; ++q) zs[j][q] = f2(0.f);
    }
    float* rstd_p = a.rstd + i;
    float* mean_p = (LN && a.mean) ? a.mean + i : nullptr;

    for (int m = 0; m < a.t; ++m, ++k) {
      if (!mbar_wait(bar0 + 8u * cs, cph, sg.spin_cap)) *abort_flag = 1;

      float2 hn[CPT][H2];
      float2 acc = f2(0.f);
#pragma unroll
      for (int j = 0; j < CPT; ++j) {
        if (m == 0 && cls[j] != 1 && colok[j]) {
          const uint32_t os = ((uint32_t)threadIdx.y * a.S_hi + col[j]) * ES;
          unpack2(lds32<raw>(sb + sg.off_c + os), zs[j]);
          if constexpr (CL) {       // the shared part of the new stream: zs + Rs
            float2 r0[H2];
            unpack2(lds32<raw>(sb + sg.off_d + os), r0);
#pragma unroll
            for (int q = 0; q < H2; ++q) zs[j][q] = add2(zs[j][q], r0[q]);
          }
        }
        if (cls[j] == 0) {
          if constexpr (CL) {
#pragma unroll
            for (int q = 0; q < H2; ++q) hn[j][q] = zs[j][q];
          } else {
            float2 r[H2];
            unpack2(lds32<raw>(sb + oA[j]), r);
#pragma unroll
            for (int q = 0; q < H2; ++q) hn[j][q] = add2(zs[j][q], r[q]);
          }
        } else {
          float2 r[H2], zp[H2];
          unpack2(lds32<raw>(sb + oA[j]), r);
          unpack2(lds32<raw>(sb + oB[j]), zp);
          if (cls[j] == 1) {
#pragma unroll
            for (int q = 0; q < H2; ++q) hn[j][q] = fma2(alpha2, zp[q], r[q]);
          } else {   // the one chunk that straddles the partition
#pragma unroll
            for (int q = 0; q < H2; ++q) {
              hn[j][q].x = (col[j] + 2 * q < a.S ? zs[j][q].x : a.alpha * zp[q].x) + r[q].x;
              hn[j][q].y = (col[j] + 2 * q + 1 < a.S ? zs[j][q].y : a.alpha * zp[q].y) + r[q].y;
            }
          }
        }
        if (act[j] && !(CL && cls[j] == 0 && m > 0)) stg<raw>(pHn[j], pack2(hn[j]));
        pHn[j] += rank_hn;
#pragma unroll
        for (int q = 0; q < H2; ++q) acc = LN ? add2(acc, hn[j][q]) : fma2(hn[j][q], hn[j][q], acc);
      }
      float st[1] = {acc.x + acc.y};
      row_reduce_sync<1>(st, red, par);      // CTA barrier: every thread is done reading this stage
      if (*abort_flag) { dead = true; break; }
      issue();
      sb += sg.stage_bytes;
      if (++cs == NS) { cs = 0; cph ^= 1u; sb = ring32; }
      float mu = 0.f, rs;
      if (LN) {
        mu = st[0] * inv_h;
        float2 sq2 = f2(0.f);
#pragma unroll
        for (int j = 0; j < CPT; ++j) {
          if (!colok[j]) continue;
#pragma unroll
          for (int q = 0; q < H2; ++q) {
            const float2 d = add2(hn[j][q], f2(-mu));
            sq2 = fma2(d, d, sq2);
          }
        }
        float sq[1] = {sq2.x + sq2.y};
        row_reduce_sync<1>(sq, red, par);
        rs = rsqrtf(fmaf(sq[0], inv_h, a.eps));
      } else {
        rs = rsqrtf(fmaf(st[0], inv_h, a.eps));
      }
      const float2 rs2 = f2(rs);
#pragma unroll
      for (int j = 0; j < CPT; ++j) {
        float2 x[H2];
#pragma unroll
        for (int q = 0; q < H2; ++q) {
          const float2 sc = mul2(rs2, gam[j][q]);
          if constexpr (LN) x[q] = fma2(add2(hn[j][q], f2(-mu)), sc, bet[j][q]);
          else x[q] = mul2(hn[j][q], sc);
        }
        if (act[j]) stg<raw>(pX[j], pack2(x));
        pX[j] += rank_h;
      }
      if (valid && threadIdx.x == 0) {
        *rstd_p = rs;
        if (LN && mean_p) *mean_p = mu;
      }
      rstd_p += a.T;
      if (LN && mean_p) mean_p += a.T;
    }
  }
  if (dead && leader) {
    atomicExch(status, 4u);
    // wait (bounded) for this CTA's copies still in flight before its shared memory goes away
    const long long issued = (k + NS) < total ? (k + NS) : total;
    for (long long q = k + 1; q < issued; ++q)
      for (uint32_t it = 0; it < (1u << 10); ++it)   // each poll sleeps up to the suspend hint: ~20 ms per stage at most
        if (mbar_try(bar0 + 8u * (uint32_t)(q % NS), (uint32_t)((q / NS) & 1))) break;
  }
}

// ------------------------------------------------------------------ backward
// stage buffers: a = dX rows, b = Hn rows, c = dHn rows (when given)
// compact layout (CL): b, c = private rows [TY, P]; d = shared stream rows, e = shared stream-gradient
// rows [TY, S] (rank 0 only); a thread keeps its shared chunks of the stream in registers across ranks
template <typename T_, int CPT, bool LN, int MAXT, bool CL>
__global__ void __launch_bounds__(MAXT, MinBlocks<CPT, MAXT>::value)
rows_backward_staged(const RowBwdArgs a, const StageGeom sg, int ngroups, unsigned int* status) {
  using V_ = VT<T_>;
  using raw = typename V_::raw;
  constexpr int V = V_::N;
  constexpr int ES = sizeof(T_);
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t* ring = smem + sg.ring_off;
  const uint32_t bar0 = smem_u32(smem + sg.bar_off);
  float* red = reinterpret_cast<float*>(smem + sg.red_off);
  float* stat = reinterpret_cast<float*>(smem + sg.stat_off);   // [2 buffers][2 (rstd, mean)][t * TY]
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + sg.bar_off + 8 * kMaxStages);
  int par = 0;
  const int TX = blockDim.x, TY = blockDim.y;
  const int tid = threadIdx.y * TX + threadIdx.x, nthr = TX * TY;
  const bool leader = tid == 0;
  const float inv_h = 1.0f / (float)a.h;
  const int NS = sg.nstages;
  const bool has_dh = a.dHn != nullptr;
  const int nstat = a.t * TY;

  const int my_groups = blockIdx.x < ngroups ? (ngroups - blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  const long long total = (long long)my_groups * a.t;

  // fetch (token group nn, rank mm) into stage ss: called by every thread, one copy per issuing warp
  // (see the forward kernel)
  int nn = 0, mm = 0, ss = 0;
  const int issuer = __shfl_sync(0xffffffffu, tid >> 5, 0);   // warp index, warp-uniform
  auto issue = [&]() {
    if (nn >= my_groups) return;
    const int n = nn, m = mm, s = ss;
    if (++mm == a.t) { mm = 0; ++nn; }
    if (++ss == NS) ss = 0;
    if (issuer > 4) return;
    const long long g = blockIdx.x + (long long)n * gridDim.x;
    const long long i0 = g * TY;
    const int rowsN = (int)((a.T - i0) < TY ? (a.T - i0) : TY);
    const uint32_t bar = bar0 + 8u * s;
    const uint32_t dst = smem_u32(ring + (size_t)s * sg.stage_bytes);
    const uint32_t b = (uint32_t)rowsN * a.h * ES;
    const long long off = ((long long)m * a.T + i0) * a.h * ES;
    if (!elect_one()) return;
    if constexpr (CL) {
      const uint32_t bP = (uint32_t)rowsN * a.P * ES;                       // 0 when there is no private part
      const uint32_t bS = m == 0 ? (uint32_t)rowsN * a.S_hi * ES : 0u;      // 0 when there is no shared part
      const long long offp = ((long long)m * a.T + i0) * a.P * ES, offs = i0 * a.S_hi * ES;
      if (issuer == 0) {
        mbar_expect_tx(bar, b + (has_dh ? 2 : 1) * (bP + bS) + sg.stall_bytes);
        bulk_g2s(dst + sg.off_a, static_cast<const char*>(a.dX) + off, b, bar);
      } else if (issuer == 1) {
        if (bP) bulk_g2s(dst + sg.off_b, static_cast<const char*>(a.Hn) + offp, bP, bar);
      } else if (issuer == 2) {
        if (bP && has_dh) bulk_g2s(dst + sg.off_c, static_cast<const char*>(a.dHn) + offp, bP, bar);
      } else if (issuer == 3) {
        if (bS) bulk_g2s(dst + sg.off_d, static_cast<const char*>(a.Hns) + offs, bS, bar);
      } else {
        if (bS && has_dh) bulk_g2s(dst + sg.off_e, static_cast<const char*>(a.dHns) + offs, bS, bar);
      }
    } else {
      if (issuer == 0) {
        mbar_expect_tx(bar, (has_dh ? 3 * b : 2 * b) + sg.stall_bytes);
        bulk_g2s(dst + sg.off_a, static_cast<const char*>(a.dX) + off, b, bar);
      } else if (issuer == 1) {
        bulk_g2s(dst + sg.off_b, static_cast<const char*>(a.Hn) + off, b, bar);
      } else if (issuer == 2) {
        if (has_dh) bulk_g2s(dst + sg.off_c, static_cast<const char*>(a.dHn) + off, b, bar);
      }
    }
  };
  // row statistics of token group n: element (m, ty) of rstd / mean
  auto load_stats = [&](int n, float* dst) {
    const long long g = blockIdx.x + (long long)n * gridDim.x;
    for (int q = tid; q < nstat; q += nthr) {
      const int m = q / TY, ty = q % TY;
      const long long i = g * TY + ty;
      const bool ok = n < my_groups && i < a.T;
      dst[q] = ok ? a.rstd[(long long)m * a.T + i] : 0.f;
      if (LN) dst[nstat + q] = ok ? a.mean[(long long)m * a.T + i] : 0.f;
    }
  };

  if (leader) {
    for (int s = 0; s < NS; ++s) mbar_init(bar0 + 8u * s, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (tid < NS)   // the zero slot of every stage (no copy ever lands there)
    *reinterpret_cast<uint4*>(ring + (size_t)tid * sg.stage_bytes + sg.zero_off) = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
  pdl_wait();   // from here on global memory is touched
  for (int q = 0; q < NS; ++q) issue();
  load_stats(0, stat);

  // Per-thread constants of the hot loop: chunk class and byte offsets inside a stage.  Chunks past the
  // row end, and every chunk of a token past T, read the zeroed slot each stage carries: they then add
  // exact zeros to the sums, and the loop needs no predicates on its loads.
  constexpr int H2 = V / 2;
  const uint32_t ring32 = smem_u32(ring);
  const uint32_t keep32 = smem_u32(smem + sg.keep_off);
  int col[CPT], cls[CPT];
  bool colok[CPT];
  float2 gam[CPT][H2], dgacc[CPT][H2], dbacc[LN ? CPT : 1][H2];
#pragma unroll
  for (int j = 0; j < CPT; ++j) {
    col[j] = (threadIdx.x + j * TX) * V;
    colok[j] = col[j] < a.h;
    cls[j] = chunk_class(col[j], V, a.S);
#pragma unroll
    for (int q = 0; q < H2; ++q) { gam[j][q] = f2(0.f); dgacc[j][q] = f2(0.f); if constexpr (LN) dbacc[j][q] = f2(0.f); }
    if (colok[j]) unpack2(ldg<raw>(static_cast<const char*>(a.gamma) + (long long)col[j] * ES), gam[j]);
  }
  const uint32_t off_hc = sg.off_c - sg.off_b;   // from a chunk of the stream to the same chunk of its gradient
  const float2 alpha2 = f2(a.alpha);
  const long long rank_h = (long long)a.T * a.h * ES;
  const long long rank_p = (long long)a.T * a.P * ES;
  __syncthreads();   // stats of group 0 visible

  long long k = 0;
  uint32_t sb = ring32;  // consumer's stage (shared address), its index and phase parity
  int cs = 0;
  uint32_t cph = 0;
  bool dead = false;
  for (int n = 0; n < my_groups && !dead; ++n) {
    const long long g = blockIdx.x + (long long)n * gridDim.x;
    const long long i = g * TY + threadIdx.y;
    const bool valid = i < a.T;
    const float* st_cur = stat + (size_t)(n & 1) * 2 * nstat;
    float* st_nxt = stat + (size_t)((n + 1) & 1) * 2 * nstat;
    // prefetch the next group's row statistics into registers; they are parked in shared
    // memory at the end of this group (a whole group of work hides the latency)
    float pre_r[2] = {0.f, 0.f}, pre_m[2] = {0.f, 0.f};
    {
      const long long g2 = blockIdx.x + (long long)(n + 1) * gridDim.x;
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int q = tid + u * nthr;
        if (q < nstat && n + 1 < my_groups) {
          const int m2 = q / TY, ty2 = q % TY;
          const long long i2 = g2 * TY + ty2;
          if (i2 < a.T) {
            pre_r[u] = a.rstd[(long long)m2 * a.T + i2];
            if (LN) pre_m[u] = a.mean[(long long)m2 * a.T + i2];
          }
        }
      }
    }
    bool act[CPT];
    // this group's stage-relative addresses of the dX chunk and of the stream chunk (its gradient sits at
    // the same place in its own buffer); the zero slot when the chunk is inactive.  Compact: private
    // chunks sit at l - S in rows of P, shared chunks come from the kept row.
    uint32_t aX[CPT], aH[CPT];
    // outputs: byte offset of the chunk in dR (per-rank layout) and in zp / compact dR, advanced per rank
    long long qR[CL ? 1 : CPT], qZ[CPT];
    float2 gsum[CPT][H2];
#pragma unroll
    for (int j = 0; j < CPT; ++j) {
      act[j] = valid && colok[j];
      const uint32_t oX = ((uint32_t)threadIdx.y * a.h + col[j]) * ES;
      const uint32_t oH = (CL && cls[j] != 0) ? ((uint32_t)threadIdx.y * a.P + (uint32_t)(col[j] - a.S_lo)) * ES : oX;
      aX[j] = act[j] ? sg.off_a + oX : sg.zero_off;
      aH[j] = act[j] ? sg.off_b + oH : sg.zero_off;
      qZ[j] = (i * a.P + (col[j] - a.S_lo)) * ES;
      if constexpr (!CL) qR[j] = (i * a.h + col[j]) * ES;
#pragma unroll
      for (int q = 0; q < H2; ++q) gsum[j][q] = f2(0.f);
    }

    for (int m = 0; m < a.t; ++m, ++k) {
      if (!mbar_wait(bar0 + 8u * cs, cph, sg.spin_cap)) *abort_flag = 1;
      const float rs_c = st_cur[m * TY + threadIdx.y];
      const float mu_c = LN ? st_cur[nstat + m * TY + threadIdx.y] : 0.f;
      const float2 rs2 = f2(rs_c);

      float2 xh[CPT][H2], dxh[CPT][H2];
      raw rdh[CPT];     // stream-gradient chunk, kept packed across the barrier (it is needed only after it)
      float2 s1 = f2(0.f), s2 = f2(0.f);
#pragma unroll
      for (int j = 0; j < CPT; ++j) {
        float2 dx[H2], hn[H2];
        unpack2(lds32<raw>(sb + aX[j]), dx);
        if (CL && cls[j] == 0) {
          // compact: the shared chunk of the stream (and of its gradient) arrives with rank 0 only; the
          // thread parks it in a shared-memory row of its own (written and read by this thread alone)
          const uint32_t os = ((uint32_t)threadIdx.y * a.S_hi + col[j]) * ES;
          if (m == 0 && act[j]) {
            const raw h0 = lds32<raw>(sb + sg.off_d + os);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(keep32 + os), "r"(reinterpret_cast<const uint4&>(h0).x),
                         "r"(reinterpret_cast<const uint4&>(h0).y), "r"(reinterpret_cast<const uint4&>(h0).z),
                         "r"(reinterpret_cast<const uint4&>(h0).w) : "memory");
            if (has_dh) unpack2(lds32<raw>(sb + sg.off_e + os), gsum[j]);   // enters the rank sum once
          }
          unpack2(lds32<raw>(act[j] ? keep32 + os : sb + sg.zero_off), hn);
          rdh[j] = zero_raw<raw>();
        } else {
          unpack2(lds32<raw>(sb + aH[j]), hn);
          rdh[j] = has_dh ? lds32<raw>(sb + aH[j] + (act[j] ? off_hc : 0u)) : zero_raw<raw>();
        }
#pragma unroll
        for (int q = 0; q < H2; ++q) {
          xh[j][q] = LN ? mul2(add2(hn[q], f2(-mu_c)), rs2) : mul2(hn[q], rs2);
          dxh[j][q] = mul2(dx[q], gam[j][q]);
          if (LN) s1 = add2(s1, dxh[j][q]);
          s2 = fma2(dxh[j][q], xh[j][q], s2);
          dgacc[j][q] = fma2(dx[q], xh[j][q], dgacc[j][q]);
          if constexpr (LN) dbacc[j][q] = add2(dbacc[j][q], dx[q]);
        }
      }
      float sacc[LN ? 2 : 1];
      if (LN) { sacc[0] = s1.x + s1.y; sacc[LN ? 1 : 0] = s2.x + s2.y; }
      else sacc[0] = s2.x + s2.y;
      row_reduce_sync<LN ? 2 : 1>(sacc, red, par);   // CTA barrier: stage fully read
      if (*abort_flag) { dead = true; break; }
      issue();
      sb += sg.stage_bytes;
      if (++cs == NS) { cs = 0; cph ^= 1u; sb = ring32; }
      const float c1 = LN ? sacc[0] * inv_h : 0.f;
      const float c2 = (LN ? sacc[LN ? 1 : 0] : sacc[0]) * inv_h;
      const float2 nc2 = f2(-c2), nc1 = f2(-c1);
#pragma unroll
      for (int j = 0; j < CPT; ++j) {
        float2 gg[H2], dh[H2];
        unpack2(rdh[j], dh);
#pragma unroll
        for (int q = 0; q < H2; ++q) {
          float2 tt = fma2(xh[j][q], nc2, dxh[j][q]);
          if (LN) tt = add2(tt, nc1);
          gg[q] = fma2(rs2, tt, dh[q]);
        }
        if constexpr (CL) {
          if (act[j] && cls[j] != 0) stg<raw>(static_cast<char*>(a.dR) + qZ[j], pack2(gg));
        } else {
          if (act[j]) stg<raw>(static_cast<char*>(a.dR) + qR[j], pack2(gg));
          qR[j] += rank_h;
        }
        if (cls[j] == 0) {
#pragma unroll
          for (int q = 0; q < H2; ++q) gsum[j][q] = add2(gsum[j][q], gg[q]);   // fp32 rank sum, m ascending
        } else {
          float2 zp[H2];
          if (cls[j] == 1) {
#pragma unroll
            for (int q = 0; q < H2; ++q) zp[q] = mul2(alpha2, gg[q]);         // private gradient carries alpha
          } else {
#pragma unroll
            for (int q = 0; q < H2; ++q) {
              const bool sx = col[j] + 2 * q < a.S, sy = col[j] + 2 * q + 1 < a.S;
              gsum[j][q].x += sx ? gg[q].x : 0.f;
              gsum[j][q].y += sy ? gg[q].y : 0.f;
              zp[q].x = sx ? 0.f : a.alpha * gg[q].x;
              zp[q].y = sy ? 0.f : a.alpha * gg[q].y;
            }
          }
          if (act[j] && a.zp) stg<raw>(static_cast<char*>(a.zp) + qZ[j], pack2(zp));
        }
        qZ[j] += rank_p;
      }
    }
    if (dead) break;
#pragma unroll
    for (int j = 0; j < CPT; ++j)
      if (act[j] && cls[j] != 1)
        stg<raw>(gs_row(a, i, ES) + (long long)col[j] * ES, pack2(gsum[j]));
    // park the next group's statistics; the last barrier of this group separates these writes
    // from the reads of group n-1's buffer, the barrier below from the reads of group n+1
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int q = tid + u * nthr;
      if (q < nstat) { st_nxt[q] = pre_r[u]; if (LN) st_nxt[nstat + q] = pre_m[u]; }
    }
    for (int q = tid + 2 * nthr; q < nstat && n + 1 < my_groups; q += nthr) {   // t * TY > 2 * threads: rare
      const int m2 = q / TY, ty2 = q % TY;
      const long long i2 = (blockIdx.x + (long long)(n + 1) * gridDim.x) * TY + ty2;
      st_nxt[q] = i2 < a.T ? a.rstd[(long long)m2 * a.T + i2] : 0.f;
      if (LN) st_nxt[nstat + q] = i2 < a.T ? a.mean[(long long)m2 * a.T + i2] : 0.f;
    }
    __syncthreads();
  }
  if (dead) {
    if (leader) {
      atomicExch(status, 5u);
      const long long issued = (k + NS) < total ? (k + NS) : total;
      for (long long q = k + 1; q < issued; ++q)
        for (uint32_t it = 0; it < (1u << 10); ++it)   // each poll sleeps up to the suspend hint: ~20 ms per stage at most
          if (mbar_try(bar0 + 8u * (uint32_t)(q % NS), (uint32_t)((q / NS) & 1))) break;
    }
    return;
  }

  // Partial norm-parameter gradients of this CTA: one row of [h] per CTA, token rows of the
  // CTA summed in order through shared memory when TY > 1.
  for (int which = 0; which < (LN ? 2 : 1); ++which) {
    float* out = which == 0 ? a.dgpart : a.dbpart;
    if (out == nullptr) continue;
    if (TY == 1) {
#pragma unroll
      for (int j = 0; j < CPT; ++j) {
        if (!colok[j]) continue;
        const float2* src = (which == 0 || !LN) ? dgacc[j] : dbacc[LN ? j : 0];
#pragma unroll
        for (int q = 0; q < H2; q += 2)
          *reinterpret_cast<float4*>(out + (size_t)blockIdx.x * a.h + col[j] + 2 * q) =
              make_float4(src[q].x, src[q].y, src[q + 1].x, src[q + 1].y);
      }
      continue;
    }
    __syncthreads();
    float* acc = reinterpret_cast<float*>(smem + sg.acc_off);   // [TY][TX*CPT*V], overlays the ring
    const int per_row = TX * CPT * V;
#pragma unroll
    for (int j = 0; j < CPT; ++j)
#pragma unroll
      for (int q = 0; q < H2; ++q) {
        const float2 v = (which == 0 || !LN) ? dgacc[j][q] : dbacc[LN ? j : 0][q];
        acc[(size_t)threadIdx.y * per_row + (j * TX + threadIdx.x) * V + 2 * q] = v.x;
        acc[(size_t)threadIdx.y * per_row + (j * TX + threadIdx.x) * V + 2 * q + 1] = v.y;
      }
    __syncthreads();
    if (threadIdx.y == 0) {
#pragma unroll
      for (int j = 0; j < CPT; ++j) {
        if (!colok[j]) continue;
        float sum[V];
#pragma unroll
        for (int e = 0; e < V; ++e) sum[e] = 0.f;
        for (int y = 0; y < TY; ++y)
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

// ------------------------------------------------------------------ host side
template <typename T_, bool LN, bool CL>
cudaError_t launch_fwd_staged_t(const RowFwdArgs& a, const RowGeom& g, const StageGeom& sg, int grid, int ngroups,
                                unsigned int* status, cudaStream_t st) {
  const dim3 block(g.TX, g.TY);
  cudaError_t e = cudaSuccess;
  LaunchScope scope(CAAT_K_ROWS_FORWARD, st);
  const int threads = g.TX * g.TY;
#define CAAT_LAUNCH(CPT_, MAXT_)                                                                   \
  do {                                                                                             \
    e = set_smem(rows_forward_staged<T_, CPT_, LN, MAXT_, CL>, sg.smem);                                        \
    if (e == cudaSuccess) e = launch_pdl(rows_forward_staged<T_, CPT_, LN, MAXT_, CL>, dim3(grid), block, sg.smem, st, a, sg, ngroups, status);   \
  } while (0)
  if (g.CPT == 1 && threads <= 256) CAAT_LAUNCH(1, 256);
  else if (g.CPT == 1) CAAT_LAUNCH(1, 512);
  else if (g.CPT == 2 && threads <= 256) CAAT_LAUNCH(2, 256);
  else if (g.CPT == 2) CAAT_LAUNCH(2, 512);
  else if (g.CPT == 4) CAAT_LAUNCH(4, 512);
  else return cudaErrorInvalidValue;
#undef CAAT_LAUNCH
  return e != cudaSuccess ? e : cudaGetLastError();
}

template <typename T_, bool LN, bool CL>
cudaError_t launch_bwd_staged_t(const RowBwdArgs& a, const RowGeom& g, const StageGeom& sg, int grid, int ngroups,
                                unsigned int* status, cudaStream_t st) {
  const dim3 block(g.TX, g.TY);
  cudaError_t e = cudaSuccess;
  LaunchScope scope(CAAT_K_ROWS_BACKWARD, st);
  const int threads = g.TX * g.TY;
#define CAAT_LAUNCH(CPT_, MAXT_)                                                                   \
  do {                                                                                             \
    e = set_smem(rows_backward_staged<T_, CPT_, LN, MAXT_, CL>, sg.smem);                                        \
    if (e == cudaSuccess) e = launch_pdl(rows_backward_staged<T_, CPT_, LN, MAXT_, CL>, dim3(grid), block, sg.smem, st, a, sg, ngroups, status);   \
  } while (0)
  if (g.CPT == 1 && threads <= 256) CAAT_LAUNCH(1, 256);
  else if (g.CPT == 1) CAAT_LAUNCH(1, 512);
  else if (g.CPT == 2 && threads <= 256) CAAT_LAUNCH(2, 256);
  else if (g.CPT == 2) CAAT_LAUNCH(2, 512);
  else if (g.CPT == 4) CAAT_LAUNCH(4, 512);
  else return cudaErrorInvalidValue;
#undef CAAT_LAUNCH
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

// the lean backward kernel takes over wherever it applies (a measurement build can keep the general kernel:
// CAAT_ROWS_LEAN=0)
static bool rows_lean_enabled() {
#ifdef CAAT_MEASUREMENT_AIDS
  static const bool on = [] { const char* e = getenv("CAAT_ROWS_LEAN"); return !(e && atoi(e) == 0); }();
  return on;
#else
  return true;
#endif
}

bool rows_staged_usable(int h, int t, int S_lo, int S_hi, caat_dtype dtype, bool backward) {
  const RowGeom g = row_geometry(h, dtype);
  const int ES = (int)elem_size(dtype);
  const StageGeom sg = stage_geometry(g, h, h - S_lo, S_hi, t, ES, backward, true, false, kSmemPerSm - 1024);
  return sg.nstages >= 2;
}

cudaError_t launch_rows_forward_staged(const RowFwdArgs& a, caat_dtype dtype, cudaStream_t st) {
  const RowGeom g = row_geometry(a.h, dtype);
  const int ES = (int)elem_size(dtype);
  const LaunchLimits lim = effective_limits();
  int per_sm = lim.rows_per_sm > 0 ? lim.rows_per_sm : ctas_per_sm(g);
  const size_t sm_budget = lim.rows_smem > 0 && (size_t)lim.rows_smem < kSmemPerSm ? (size_t)lim.rows_smem : kSmemPerSm;
  const bool cl = a.compact != 0;
  StageGeom sg = stage_geometry(g, a.h, a.P, a.S_hi, a.t, ES, false, true, cl, sm_budget / per_sm - 1024);
  while (sg.nstages < 3 && per_sm > 1) {   // rows too long: fewer CTAs per SM, each with a larger ring
    --per_sm;
    sg = stage_geometry(g, a.h, a.P, a.S_hi, a.t, ES, false, true, cl, sm_budget / per_sm - 1024);
  }
  if (sg.nstages < 2) return cudaErrorInvalidConfiguration;
  const int ngroups = (a.T + g.TY - 1) / g.TY;
  int grid = sm_count() * per_sm;
  if (lim.rows_ctas > 0 && grid > lim.rows_ctas) grid = lim.rows_ctas;
  if (grid > ngroups) grid = ngroups;
  unsigned int* status = device_status_word();
  if (!status) return cudaErrorUnknown;
  if (cl) {
    if (dtype == CAAT_BF16)
      return a.norm == 1 ? launch_fwd_staged_t<__nv_bfloat16, true, true>(a, g, sg, grid, ngroups, status, st)
                         : launch_fwd_staged_t<__nv_bfloat16, false, true>(a, g, sg, grid, ngroups, status, st);
    return a.norm == 1 ? launch_fwd_staged_t<float, true, true>(a, g, sg, grid, ngroups, status, st)
                       : launch_fwd_staged_t<float, false, true>(a, g, sg, grid, ngroups, status, st);
  }
  if (dtype == CAAT_BF16)
    return a.norm == 1 ? launch_fwd_staged_t<__nv_bfloat16, true, false>(a, g, sg, grid, ngroups, status, st)
                       : launch_fwd_staged_t<__nv_bfloat16, false, false>(a, g, sg, grid, ngroups, status, st);
  return a.norm == 1 ? launch_fwd_staged_t<float, true, false>(a, g, sg, grid, ngroups, status, st)
                     : launch_fwd_staged_t<float, false, false>(a, g, sg, grid, ngroups, status, st);
}

// The grid (= rows of norm-gradient partials) must not exceed what the scratch layout reserves.
cudaError_t launch_rows_backward_staged(const RowBwdArgs& a, caat_dtype dtype, int max_rows, int* rows_used,
                                        cudaStream_t st) {
  const RowGeom g = row_geometry(a.h, dtype);
  const int ES = (int)elem_size(dtype);
  const bool has_c = a.dHn != nullptr;
  const LaunchLimits lim = effective_limits();
  int per_sm = lim.rows_per_sm > 0 ? lim.rows_per_sm : ctas_per_sm(g);
  const size_t sm_budget = lim.rows_smem > 0 && (size_t)lim.rows_smem < kSmemPerSm ? (size_t)lim.rows_smem : kSmemPerSm;
  const bool cl = a.compact != 0;
  StageGeom sg = stage_geometry(g, a.h, a.P, a.S_hi, a.t, ES, true, has_c, cl, sm_budget / per_sm - 1024);
  while (sg.nstages < 3 && per_sm > 1) {
    --per_sm;
    sg = stage_geometry(g, a.h, a.P, a.S_hi, a.t, ES, true, has_c, cl, sm_budget / per_sm - 1024);
  }
  if (sg.nstages < 2) return cudaErrorInvalidConfiguration;
  const int ngroups = (a.T + g.TY - 1) / g.TY;
  int grid = sm_count() * per_sm;
  if (lim.rows_ctas > 0 && grid > lim.rows_ctas) grid = lim.rows_ctas;
  if (grid > ngroups) grid = ngroups;
  if (grid > max_rows) grid = max_rows;
  *rows_used = grid;
  unsigned int* status = device_status_word();
  if (!status) return cudaErrorUnknown;
  if (rows_lean_enabled() && rows_lean_usable(a.compact, a.h, a.T, a.S, a.S_lo, a.S_hi, dtype))
    return launch_rows_backward_lean(a, dtype, g, sg, grid, ngroups, status, st);
  if (cl) {
    if (dtype == CAAT_BF16)
      return a.norm == 1 ? launch_bwd_staged_t<__nv_bfloat16, true, true>(a, g, sg, grid, ngroups, status, st)
                         : launch_bwd_staged_t<__nv_bfloat16, false, true>(a, g, sg, grid, ngroups, status, st);
    return a.norm == 1 ? launch_bwd_staged_t<float, true, true>(a, g, sg, grid, ngroups, status, st)
                       : launch_bwd_staged_t<float, false, true>(a, g, sg, grid, ngroups, status, st);
  }
  if (dtype == CAAT_BF16)
    return a.norm == 1 ? launch_bwd_staged_t<__nv_bfloat16, true, false>(a, g, sg, grid, ngroups, status, st)
                       : launch_bwd_staged_t<__nv_bfloat16, false, false>(a, g, sg, grid, ngroups, status, st);
  return a.norm == 1 ? launch_bwd_staged_t<float, true, false>(a, g, sg, grid, ngroups, status, st)
                     : launch_bwd_staged_t<float, false, false>(a, g, sg, grid, ngroups, status, st);
}

}  // namespace caat
