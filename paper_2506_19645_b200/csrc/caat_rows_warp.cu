// Row kernels for SHORT rows (at most four 16-byte chunks per lane: h <= 1024 in bf16).
//
// With short rows the CTA-wide reduction and barrier per rank of the general kernels cost more
// than the arithmetic.  Here ONE WARP owns a token: its lanes cover the row's chunks (lane, lane+32,
// ...), it walks the ranks m = 0..t-1, row statistics are plain warp shuffles and the rank sum of
// the shared channels is lane-local.  Warps never wait for each other: a dedicated producer warp
// keeps a shared-memory ring of (token group, rank) stages filled with cp.async.bulk, consumers
// signal "stage read" on an mbarrier per stage, and the only CTA-wide step is the final fold of
// the warps' partial norm-parameter gradients.  All waits are bounded (status word on timeout).
#include "caat_rows_common.cuh"

namespace caat {
namespace {

using namespace rows;

constexpr int kW = 4;                    // consumer warps = tokens per group
constexpr int kThreads = (kW + 1) * 32;  // + one producer warp
constexpr int kMaxStages = 8;
constexpr uint32_t kSuspendHintNs = 20000u;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(kSuspendHintNs)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t cap) {
  for (uint32_t it = 0; it < cap; ++it) {
    if (mbar_try(bar, parity)) return true;
    if (*abort_flag) return false;
  }
  return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
template <typename raw>
__device__ __forceinline__ raw lds(const uint8_t* p) { return *reinterpret_cast<const raw*>(p); }

// A consumer warp whose wait for a stage ran out: it raises the abort flag and the status word (the producer may have
// issued everything and left already, so nobody else would), then gives the copies that may still be in flight into
// this CTA's ring a bounded time to land - stage by stage from the one it waited for - before it leaves the loop.
__device__ __forceinline__ void consumer_gave_up(unsigned int* status, unsigned int code, volatile int* abort_flag,
                                                 uint32_t full0, int s, uint32_t ph, int NS, int lane) {
  if (lane == 0) {
    *abort_flag = 1;
    atomicExch(status, code);
    for (int k = 0; k < NS; ++k) {
      for (uint32_t it = 0; it < (1u << 10); ++it)   // each poll sleeps up to the suspend hint: ~20 ms per stage at most
        if (mbar_try(full0 + 8u * s, ph)) break;
      if (++s == NS) { s = 0; ph ^= 1u; }
    }
  }
  __syncwarp();
}

struct WarpGeom {
  int nstages;
  uint32_t off_a, off_b, off_c, off_d, off_e, stage_bytes;   // d, e: compact layout only
  uint32_t zero_off;   // 16 zero bytes inside every stage (read by chunks past the row end)
  uint32_t keep_off;   // compact backward: [kW, S] shared rows of the stream, parked for all ranks of a token
  uint32_t bar_off, ring_off;
  size_t smem;
  uint32_t spin_cap;     // polls of one mbarrier wait before the role gives up (rows_hooks)
  uint32_t stall_bytes;  // time-out test: bytes every stage announces on top of its copies (0 otherwise)
};

// ------------------------------------------------------------------ forward
// stage: a = R rows [kW, h], b = zp rows [kW, P], c = zs rows [kW, S_hi] (rank 0 only)
// compact layout (CL): a = private residual rows [kW, P], d = shared residual rows [kW, S] (rank 0 only)
template <typename T_, int CPT, bool LN, bool CL>
__global__ void __launch_bounds__(kThreads, 3)
rows_forward_warp(const RowFwdArgs a, const WarpGeom sg, int ngroups, unsigned int* status) {
  using V_ = VT<T_>;
  using raw = typename V_::raw;
  constexpr int V = V_::N;
  constexpr int ES = sizeof(T_);
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t* ring = smem + sg.ring_off;
  const uint32_t full0 = smem_u32(smem + sg.bar_off), empty0 = full0 + 8u * kMaxStages;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + sg.bar_off + 16 * kMaxStages);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int NS = sg.nstages;
  const bool has_priv = a.P > 0 && a.S < a.h, has_shared = a.S > 0;
  const int my_groups = blockIdx.x < ngroups ? (ngroups - blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < NS; ++s) { mbar_init(full0 + 8u * s, 1); mbar_init(empty0 + 8u * s, kW); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if ((int)threadIdx.x < NS)   // the zero slot of every stage (no copy ever lands there)
    *reinterpret_cast<uint4*>(ring + (size_t)threadIdx.x * sg.stage_bytes + sg.zero_off) = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
  pdl_wait();   // from here on global memory is touched

  if (warp == kW) {
    // ---------------------------------------------------------- producer
    if (lane == 0) {
      int s = 0; uint32_t ph = 0;
      long long issued = 0;
      bool ok = true;
      for (int n = 0; n < my_groups && ok; ++n) {
        const long long i0 = (blockIdx.x + (long long)n * gridDim.x) * kW;
        const int rowsN = (int)((a.T - i0) < kW ? (a.T - i0) : kW);
        for (int m = 0; m < a.t; ++m) {
          if (!mbar_wait(empty0 + 8u * s, ph ^ 1u, abort_flag, sg.spin_cap)) { ok = false; break; }
          const uint32_t bar = full0 + 8u * s;
          const uint32_t dst = smem_u32(ring + (size_t)s * sg.stage_bytes);
          const uint32_t bP = has_priv ? (uint32_t)rowsN * a.P * ES : 0u;
          const uint32_t bR = CL ? bP : (uint32_t)rowsN * a.h * ES;
          const uint32_t bS = (m == 0 && has_shared) ? (uint32_t)rowsN * a.S_hi * ES : 0u;
          mbar_expect_tx(bar, bR + bP + (CL ? 2 * bS : bS) + sg.stall_bytes);
          const long long row = (long long)m * a.T + i0;
          if (bR) bulk_g2s(dst + sg.off_a, static_cast<const char*>(a.R) + row * (CL ? a.P : a.h) * ES, bR, bar);
          if (bP) bulk_g2s(dst + sg.off_b, static_cast<const char*>(a.zp) + row * a.P * ES, bP, bar);
          if (bS) bulk_g2s(dst + sg.off_c, static_cast<const char*>(a.zs) + i0 * a.S_hi * ES, bS, bar);
          if (CL && bS) bulk_g2s(dst + sg.off_d, static_cast<const char*>(a.Rs) + i0 * a.S_hi * ES, bS, bar);
          ++issued;
          if (++s == NS) { s = 0; ph ^= 1u; }
        }
      }
      if (!ok) {
        *abort_flag = 1;
        atomicExch(status, 6u);
        const int pending = issued < NS ? (int)issued : NS;
        for (int k = 0; k < pending; ++k) {        // let this CTA's copies in flight land
          if (--s < 0) { s = NS - 1; ph ^= 1u; }
          for (uint32_t it = 0; it < (1u << 12); ++it)
            if (mbar_try(full0 + 8u * s, ph)) break;
        }
      }
    }
    return;
  }

  // ------------------------------------------------------------ consumers: warp w owns token i0 + w
  // per-lane constants: chunk class and byte offsets inside a stage (the zero slot for chunks past the row end)
  constexpr int H2 = V / 2;
  const uint32_t ring32 = smem_u32(ring);
  int col[CPT], cls[CPT];
  bool colok[CPT];
  uint32_t oA[CPT], oB[CPT];
  float2 gam[CPT][H2], bet[LN ? CPT : 1][H2];
#pragma unroll
  for (int j = 0; j < CPT; ++j) {
    col[j] = (lane + 32 * j) * V;
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
      const uint32_t priv = ((uint32_t)warp * a.P + (uint32_t)(col[j] - a.S_lo)) * ES;
      if (cls[j] != 0) oB[j] = sg.off_b + priv;
      if (CL) { if (cls[j] != 0) oA[j] = sg.off_a + priv; }
      else oA[j] = sg.off_a + ((uint32_t)warp * a.h + col[j]) * ES;
    }
  }
  const float inv_h = 1.0f / (float)a.h;
  const float2 alpha2 = f2(a.alpha);
  const long long rank_h = (long long)a.T * a.h * ES;
  const long long rank_hn = CL ? (long long)a.T * a.P * ES : rank_h;   // rank stride of the stream's (private) rows
  int s = 0; uint32_t ph = 0;
  uint32_t sb = ring32;
  bool dead = false;
  for (int n = 0; n < my_groups && !dead; ++n) {
    const long long i = (blockIdx.x + (long long)n * gridDim.x) * kW + warp;
    const bool valid = i < a.T;
    float2 zs[CPT][H2];
#pragma unroll
    for (int j = 0; j < CPT; ++j)
#pragma unroll
      for (int q = 0; q < H2; ++q) zs[j][q] = f2(0.f);
    // compact: column l of the private rows sits at l - S
    char* pHn = CL ? static_cast<char*>(a.Hn) + (i * a.P - a.S_lo) * ES : static_cast<char*>(a.Hn) + i * a.h * ES;
    char* pX = static_cast<char*>(a.X) + i * a.h * ES;
    float* rstd_p = a.rstd + i;
    float* mean_p = (LN && a.mean) ? a.mean + i : nullptr;
    for (int m = 0; m < a.t; ++m) {
      if (!__all_sync(0xffffffffu, mbar_wait(full0 + 8u * s, ph, abort_flag, sg.spin_cap))) {   // warp-uniform verdict
        consumer_gave_up(status, 8u, abort_flag, full0, s, ph, NS, lane);
        dead = true;
        break;
      }
      float2 hn[CPT][H2];
      float2 acc = f2(0.f);
#pragma unroll
      for (int j = 0; j < CPT; ++j) {
        const bool act = valid && colok[j];
        if (m == 0 && cls[j] != 1 && colok[j]) {
          const uint32_t os = ((uint32_t)warp * a.S_hi + col[j]) * ES;
          unpack2(lds32<raw>(sb + sg.off_c + os), zs[j]);
          if constexpr (CL) {       // the shared part of the new stream, formed once: zs + Rs
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
        if constexpr (CL) {
          if (act && cls[j] != 0) stg<raw>(pHn + (long long)col[j] * ES, pack2(hn[j]));
          else if (act && m == 0) stg<raw>(static_cast<char*>(a.Hns) + (i * a.S_hi + col[j]) * ES, pack2(hn[j]));
        } else {
          if (act) stg<raw>(pHn + (long long)col[j] * ES, pack2(hn[j]));
        }
#pragma unroll
        for (int q = 0; q < H2; ++q) acc = LN ? add2(acc, hn[j][q]) : fma2(hn[j][q], hn[j][q], acc);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty0 + 8u * s);      // this warp is done with the stage
      sb += sg.stage_bytes;
      if (++s == NS) { s = 0; ph ^= 1u; sb = ring32; }
      const float st = warp_sum(acc.x + acc.y);
      float mu = 0.f, rs;
      if (LN) {
        mu = st * inv_h;
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
        rs = rsqrtf(fmaf(warp_sum(sq2.x + sq2.y), inv_h, a.eps));
      } else {
        rs = rsqrtf(fmaf(st, inv_h, a.eps));
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
        if (valid && colok[j]) stg<raw>(pX + (long long)col[j] * ES, pack2(x));
      }
      if (valid && lane == 0) {
        *rstd_p = rs;
        if (LN && mean_p) *mean_p = mu;
      }
      pHn += rank_hn; pX += rank_h; rstd_p += a.T;
      if (LN && mean_p) mean_p += a.T;
    }
  }
}

// ------------------------------------------------------------------ backward
// stage: a = dX rows, b = Hn rows, c = dHn rows (when given), kW tokens each
// compact layout (CL): b, c = private rows [kW, P]; d = shared stream rows, e = shared stream-gradient rows
// [kW, S] (rank 0 only); a lane keeps its shared chunks of the stream in registers across the ranks
template <typename T_, int CPT, bool LN, bool CL>
__global__ void __launch_bounds__(kThreads, 3)
rows_backward_warp(const RowBwdArgs a, const WarpGeom sg, int ngroups, unsigned int* status) {
  using V_ = VT<T_>;
  using raw = typename V_::raw;
  constexpr int V = V_::N;
  constexpr int ES = sizeof(T_);
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t* ring = smem + sg.ring_off;
  const uint32_t full0 = smem_u32(smem + sg.bar_off), empty0 = full0 + 8u * kMaxStages;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + sg.bar_off + 16 * kMaxStages);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int NS = sg.nstages;
  const bool has_dh = a.dHn != nullptr;
  const int my_groups = blockIdx.x < ngroups ? (ngroups - blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < NS; ++s) { mbar_init(full0 + 8u * s, 1); mbar_init(empty0 + 8u * s, kW); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if ((int)threadIdx.x < NS)   // the zero slot of every stage (no copy ever lands there)
    *reinterpret_cast<uint4*>(ring + (size_t)threadIdx.x * sg.stage_bytes + sg.zero_off) = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
  pdl_wait();   // from here on global memory is touched

  constexpr int H2 = V / 2;
  int col[CPT], cls[CPT];
  bool colok[CPT];
  float2 gam[CPT][H2], dgacc[CPT][H2], dbacc[LN ? CPT : 1][H2];
#pragma unroll
  for (int j = 0; j < CPT; ++j) {
    col[j] = (lane + 32 * j) * V;
    colok[j] = col[j] < a.h;
    cls[j] = chunk_class(col[j], V, a.S);
#pragma unroll
    for (int q = 0; q < H2; ++q) { gam[j][q] = f2(0.f); dgacc[j][q] = f2(0.f); if constexpr (LN) dbacc[j][q] = f2(0.f); }
  }

  if (warp == kW) {
    // ---------------------------------------------------------- producer
    if (lane == 0) {
      int s = 0; uint32_t ph = 0;
      long long issued = 0;
      bool ok = true;
      for (int n = 0; n < my_groups && ok; ++n) {
        const long long i0 = (blockIdx.x + (long long)n * gridDim.x) * kW;
        const int rowsN = (int)((a.T - i0) < kW ? (a.T - i0) : kW);
        const uint32_t b = (uint32_t)rowsN * a.h * ES;
        for (int m = 0; m < a.t; ++m) {
          if (!mbar_wait(empty0 + 8u * s, ph ^ 1u, abort_flag, sg.spin_cap)) { ok = false; break; }
          const uint32_t bar = full0 + 8u * s;
          const uint32_t dst = smem_u32(ring + (size_t)s * sg.stage_bytes);
          const long long off = ((long long)m * a.T + i0) * a.h * ES;
          if constexpr (CL) {
            const uint32_t bP = (uint32_t)rowsN * a.P * ES;                       // 0 when there is no private part
            const uint32_t bS = m == 0 ? (uint32_t)rowsN * a.S_hi * ES : 0u;      // 0 when there is no shared part
            mbar_expect_tx(bar, b + (has_dh ? 2 : 1) * (bP + bS) + sg.stall_bytes);
            const long long offp = ((long long)m * a.T + i0) * a.P * ES, offs = i0 * a.S_hi * ES;
            bulk_g2s(dst + sg.off_a, static_cast<const char*>(a.dX) + off, b, bar);
            if (bP) bulk_g2s(dst + sg.off_b, static_cast<const char*>(a.Hn) + offp, bP, bar);
            if (bP && has_dh) bulk_g2s(dst + sg.off_c, static_cast<const char*>(a.dHn) + offp, bP, bar);
            if (bS) bulk_g2s(dst + sg.off_d, static_cast<const char*>(a.Hns) + offs, bS, bar);
            if (bS && has_dh) bulk_g2s(dst + sg.off_e, static_cast<const char*>(a.dHns) + offs, bS, bar);
          } else {
            mbar_expect_tx(bar, (has_dh ? 3 * b : 2 * b) + sg.stall_bytes);
            bulk_g2s(dst + sg.off_a, static_cast<const char*>(a.dX) + off, b, bar);
            bulk_g2s(dst + sg.off_b, static_cast<const char*>(a.Hn) + off, b, bar);
            if (has_dh) bulk_g2s(dst + sg.off_c, static_cast<const char*>(a.dHn) + off, b, bar);
          }
          ++issued;
          if (++s == NS) { s = 0; ph ^= 1u; }
        }
      }
      if (!ok) {
        *abort_flag = 1;
        atomicExch(status, 7u);
        const int pending = issued < NS ? (int)issued : NS;
        for (int k = 0; k < pending; ++k) {
          if (--s < 0) { s = NS - 1; ph ^= 1u; }
          for (uint32_t it = 0; it < (1u << 12); ++it)
            if (mbar_try(full0 + 8u * s, ph)) break;
        }
      }
    }
  } else {
    // ---------------------------------------------------------- consumers
    // Inactive chunks (past the row end, or a token past T) read the zero slot every stage carries, so
    // they add exact zeros to the sums and the loads need no predicates.
#pragma unroll
    for (int j = 0; j < CPT; ++j)
      if (colok[j]) unpack2(ldg<raw>(static_cast<const char*>(a.gamma) + (long long)col[j] * ES), gam[j]);
    const uint32_t ring32 = smem_u32(ring);
    const uint32_t keep32 = smem_u32(smem + sg.keep_off);
    const uint32_t off_hc = sg.off_c - sg.off_b;   // from a chunk of the stream to the same chunk of its gradient
    const float inv_h = 1.0f / (float)a.h;
    const float2 alpha2 = f2(a.alpha);
    const long long rank_h = (long long)a.T * a.h * ES, rank_p = (long long)a.T * a.P * ES;
    int s = 0; uint32_t ph = 0;
    uint32_t sb = ring32;
    bool dead = false;
    // lane m holds rstd (mean) of rank m for the current token; the next token's are fetched a group ahead
    auto load_stat = [&](const float* base, int n) -> float {
      const long long i = (blockIdx.x + (long long)n * gridDim.x) * kW + warp;
      return (base != nullptr && n < my_groups && i < a.T && lane < a.t) ? base[(long long)lane * a.T + i] : 0.f;
    };
    float rs_next = load_stat(a.rstd, 0), mu_next = LN ? load_stat(a.mean, 0) : 0.f;
    for (int n = 0; n < my_groups && !dead; ++n) {
      const long long i = (blockIdx.x + (long long)n * gridDim.x) * kW + warp;
      const bool valid = i < a.T;
      const float rs_lane = rs_next, mu_lane = mu_next;
      rs_next = load_stat(a.rstd, n + 1);
      if (LN) mu_next = load_stat(a.mean, n + 1);
      float2 gsum[CPT][H2];
      // stage-relative addresses of this token's dX chunk and stream chunk; compact: private chunks sit at
      // l - S in rows of P, shared chunks come from a row the warp parks in shared memory for all ranks
      uint32_t aX[CPT], aH[CPT];
#pragma unroll
      for (int j = 0; j < CPT; ++j) {
        const bool act = valid && colok[j];
        const uint32_t oX = ((uint32_t)warp * a.h + col[j]) * ES;
        const uint32_t oH = (CL && cls[j] != 0) ? ((uint32_t)warp * a.P + (uint32_t)(col[j] - a.S_lo)) * ES : oX;
        aX[j] = act ? sg.off_a + oX : sg.zero_off;
        aH[j] = act ? sg.off_b + oH : sg.zero_off;
#pragma unroll
        for (int q = 0; q < H2; ++q) gsum[j][q] = f2(0.f);
      }
      char* pdR = CL ? static_cast<char*>(a.dR) + (i * a.P - a.S_lo) * ES : static_cast<char*>(a.dR) + i * a.h * ES;
      char* pZ = static_cast<char*>(a.zp) + (i * a.P - a.S_lo) * ES;
      for (int m = 0; m < a.t; ++m) {
        if (!__all_sync(0xffffffffu, mbar_wait(full0 + 8u * s, ph, abort_flag, sg.spin_cap))) {   // warp-uniform verdict
          consumer_gave_up(status, 9u, abort_flag, full0, s, ph, NS, lane);
          dead = true;
          break;
        }
        const float rs = __shfl_sync(0xffffffffu, rs_lane, m);
        const float mu = LN ? __shfl_sync(0xffffffffu, mu_lane, m) : 0.f;
        const float2 rs2 = f2(rs);
        if constexpr (CL) {
          if (m == 0) {
#pragma unroll
            for (int j = 0; j < CPT; ++j) {
              if (valid && colok[j] && cls[j] == 0) {
                const uint32_t os = ((uint32_t)warp * a.S_hi + col[j]) * ES;
                const raw h0 = lds32<raw>(sb + sg.off_d + os);
                const uint4& u = reinterpret_cast<const uint4&>(h0);
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(keep32 + os), "r"(u.x), "r"(u.y), "r"(u.z), "r"(u.w)
                             : "memory");
                if (has_dh) unpack2(lds32<raw>(sb + sg.off_e + os), gsum[j]);   // enters the rank sum once
              }
            }
          }
        }
        // pass 1: row statistics and norm-parameter gradients
        float2 s1 = f2(0.f), s2 = f2(0.f);
#pragma unroll
        for (int j = 0; j < CPT; ++j) {
          float2 dx[H2], hn[H2];
          unpack2(lds32<raw>(sb + aX[j]), dx);
          uint32_t hsrc = sb + aH[j];
          if (CL && cls[j] == 0) hsrc = (valid && colok[j]) ? keep32 + ((uint32_t)warp * a.S_hi + col[j]) * ES : sb + sg.zero_off;
          unpack2(lds32<raw>(hsrc), hn);
#pragma unroll
          for (int q = 0; q < H2; ++q) {
            const float2 xh = LN ? mul2(add2(hn[q], f2(-mu)), rs2) : mul2(hn[q], rs2);
            const float2 dxh = mul2(dx[q], gam[j][q]);
            if (LN) s1 = add2(s1, dxh);
            s2 = fma2(dxh, xh, s2);
            dgacc[j][q] = fma2(dx[q], xh, dgacc[j][q]);
            if constexpr (LN) dbacc[j][q] = add2(dbacc[j][q], dx[q]);
          }
        }
        const float c1 = LN ? warp_sum(s1.x + s1.y) * inv_h : 0.f;
        const float c2 = warp_sum(s2.x + s2.y) * inv_h;
        const float2 nc1 = f2(-c1), nc2 = f2(-c2);
        // pass 2: gradients (the stage is re-read: cheaper than keeping the row in registers)
#pragma unroll
        for (int j = 0; j < CPT; ++j) {
          if (!(valid && colok[j])) continue;
          float2 dx[H2], hn[H2], dh[H2], gg[H2];
          unpack2(lds32<raw>(sb + aX[j]), dx);
          if (CL && cls[j] == 0) {
            unpack2(lds32<raw>(keep32 + ((uint32_t)warp * a.S_hi + col[j]) * ES), hn);
#pragma unroll
            for (int q = 0; q < H2; ++q) dh[q] = f2(0.f);
          } else {
            unpack2(lds32<raw>(sb + aH[j]), hn);
            if (has_dh) {
              unpack2(lds32<raw>(sb + aH[j] + off_hc), dh);
            } else {
#pragma unroll
              for (int q = 0; q < H2; ++q) dh[q] = f2(0.f);
            }
          }
#pragma unroll
          for (int q = 0; q < H2; ++q) {
            const float2 xh = LN ? mul2(add2(hn[q], f2(-mu)), rs2) : mul2(hn[q], rs2);
            float2 tt = fma2(xh, nc2, mul2(dx[q], gam[j][q]));
            if (LN) tt = add2(tt, nc1);
            gg[q] = fma2(rs2, tt, dh[q]);
          }
          if (!(CL && cls[j] == 0)) stg<raw>(pdR + (long long)col[j] * ES, pack2(gg));
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
            if (a.zp) stg<raw>(pZ + (long long)col[j] * ES, pack2(zp));
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty0 + 8u * s);
        sb += sg.stage_bytes;
        if (++s == NS) { s = 0; ph ^= 1u; sb = ring32; }
        pdR += CL ? rank_p : rank_h; pZ += rank_p;
      }
      if (dead) break;
#pragma unroll
      for (int j = 0; j < CPT; ++j)
        if (valid && colok[j] && cls[j] != 1)
          stg<raw>(gs_row(a, i, ES) + (long long)col[j] * ES, pack2(gsum[j]));
    }
  }

  // fold the warps' partial norm-parameter gradients: one row of [h] per CTA (the ring is free by now:
  // every copy that was issued has been consumed, or the kernel gave up and the values do not matter)
  __syncthreads();
  float* acc = reinterpret_cast<float*>(ring);        // [kW][h]
  for (int which = 0; which < (LN ? 2 : 1); ++which) {
    float* out = which == 0 ? a.dgpart : a.dbpart;
    if (out == nullptr) continue;
    if (warp < kW) {
#pragma unroll
      for (int j = 0; j < CPT; ++j)
        if (colok[j])
#pragma unroll
          for (int q = 0; q < H2; ++q) {
            const float2 v = (which == 0 || !LN) ? dgacc[j][q] : dbacc[LN ? j : 0][q];
            acc[(size_t)warp * a.h + col[j] + 2 * q] = v.x;
            acc[(size_t)warp * a.h + col[j] + 2 * q + 1] = v.y;
          }
    }
    __syncthreads();
    for (int c = threadIdx.x; c < a.h; c += blockDim.x) {
      float sum = 0.f;
#pragma unroll
      for (int w = 0; w < kW; ++w) sum += acc[(size_t)w * a.h + c];
      out[(size_t)blockIdx.x * a.h + c] = sum;
    }
    __syncthreads();
  }
}

WarpGeom warp_geometry(int h, int P, int S_hi, int ES, bool backward, bool has_c, bool compact, size_t budget) {
  WarpGeom g{};
  const uint32_t rowA = (uint32_t)kW * h * ES;
  const uint32_t rowP = (uint32_t)kW * P * ES, rowS = (uint32_t)kW * S_hi * ES;
  if (backward && compact) {          // dX | Hnp | dHnp | Hns | dHns   (P + S_hi = h)
    g.off_a = 0; g.off_b = rowA; g.off_c = rowA + rowP;
    g.off_d = has_c ? rowA + 2 * rowP : rowA + rowP;
    g.off_e = g.off_d + rowS;
    g.stage_bytes = g.off_d + (has_c ? 2 : 1) * rowS;
  } else if (backward) {
    g.off_a = 0; g.off_b = rowA; g.off_c = 2 * rowA;
    g.stage_bytes = (has_c ? 3 : 2) * rowA;
  } else if (compact) {               // Rp | zp | zs | Rs
    g.off_a = 0; g.off_b = rowP; g.off_c = 2 * rowP; g.off_d = 2 * rowP + rowS;
    g.stage_bytes = 2 * rowP + 2 * rowS;
  } else {
    g.off_a = 0; g.off_b = rowA; g.off_c = rowA + rowP;
    g.stage_bytes = rowA + rowP + rowS;
  }
  g.zero_off = g.stage_bytes;
  g.stage_bytes = (g.stage_bytes + 16u + 127u) & ~127u;
  g.bar_off = 0;
  g.keep_off = (uint32_t)align_up(16 * kMaxStages + 16, 128);
  g.ring_off = (uint32_t)align_up(g.keep_off + ((backward && compact) ? rowS : 0u), 128);
  int ns = (int)((budget - g.ring_off) / g.stage_bytes);
  if (ns > kMaxStages) ns = kMaxStages;
  g.nstages = ns;
  size_t ring = (size_t)(ns > 0 ? ns : 0) * g.stage_bytes;
  const size_t acc = backward ? (size_t)kW * h * sizeof(float) : 0;
  if (ring < acc) ring = acc;
  g.smem = g.ring_off + ring;
  const RowsHooks hooks = rows_hooks();
  g.spin_cap = hooks.spin_cap;
  g.stall_bytes = hooks.stall ? 16u : 0u;
  return g;
}

constexpr size_t kSmemPerSm = 227 * 1024;
constexpr int kCtasPerSm = 3;

template <typename K>
cudaError_t set_smem(K kernel, size_t bytes) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

template <typename T_, bool LN, bool CL>
cudaError_t launch_fwd_warp_t(const RowFwdArgs& a, int cpt, const WarpGeom& g, int grid, int ngroups,
                              unsigned int* status, cudaStream_t st) {
  cudaError_t e = cudaSuccess;
  LaunchScope scope(CAAT_K_ROWS_FORWARD, st);
#define CAAT_LAUNCH(CPT_)                                                                      \
  do {                                                                                         \
    e = set_smem(rows_forward_warp<T_, CPT_, LN, CL>, g.smem);                                 \
    if (e == cudaSuccess) e = launch_pdl(rows_forward_warp<T_, CPT_, LN, CL>, dim3(grid), dim3(kThreads), g.smem, st, a, g, ngroups, status); \
  } while (0)
  switch (cpt) {
    case 1: CAAT_LAUNCH(1); break;
    case 2: CAAT_LAUNCH(2); break;
    case 3: CAAT_LAUNCH(3); break;
    case 4: CAAT_LAUNCH(4); break;
    default: return cudaErrorInvalidValue;
  }
#undef CAAT_LAUNCH
  return e != cudaSuccess ? e : cudaGetLastError();
}

template <typename T_, bool LN, bool CL>
cudaError_t launch_bwd_warp_t(const RowBwdArgs& a, int cpt, const WarpGeom& g, int grid, int ngroups,
                              unsigned int* status, cudaStream_t st) {
  cudaError_t e = cudaSuccess;
  LaunchScope scope(CAAT_K_ROWS_BACKWARD, st);
#define CAAT_LAUNCH(CPT_)                                                                       \
  do {                                                                                          \
    e = set_smem(rows_backward_warp<T_, CPT_, LN, CL>, g.smem);                                 \
    if (e == cudaSuccess) e = launch_pdl(rows_backward_warp<T_, CPT_, LN, CL>, dim3(grid), dim3(kThreads), g.smem, st, a, g, ngroups, status); \
  } while (0)
  switch (cpt) {
    case 1: CAAT_LAUNCH(1); break;
    case 2: CAAT_LAUNCH(2); break;
    case 3: CAAT_LAUNCH(3); break;
    case 4: CAAT_LAUNCH(4); break;
    default: return cudaErrorInvalidValue;
  }
#undef CAAT_LAUNCH
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

// chunks per lane of the warp-per-token kernels, 0 when the row is too long for them
int rows_warp_cpt(int h, int t, caat_dtype dtype) {
  const int V = dtype == CAAT_BF16 ? 8 : 4;
  const int chunks = h / V;
  const int cpt = (chunks + 31) / 32;
  return (cpt >= 1 && cpt <= 4 && t <= 32) ? cpt : 0;
}

cudaError_t launch_rows_forward_warp(const RowFwdArgs& a, caat_dtype dtype, cudaStream_t st) {
  const int cpt = rows_warp_cpt(a.h, a.t, dtype);
  const int ES = (int)elem_size(dtype);
  const LaunchLimits lim = effective_limits();
  const int per_sm = lim.rows_per_sm > 0 && lim.rows_per_sm < kCtasPerSm ? lim.rows_per_sm : kCtasPerSm;
  const size_t sm_budget = lim.rows_smem > 0 && (size_t)lim.rows_smem < kSmemPerSm ? (size_t)lim.rows_smem : kSmemPerSm;
  const WarpGeom g = warp_geometry(a.h, a.P, a.S_hi, ES, false, true, a.compact != 0, sm_budget / per_sm - 1024);
  if (cpt == 0 || g.nstages < 2) return cudaErrorInvalidConfiguration;
  const int ngroups = (a.T + kW - 1) / kW;
  int grid = sm_count() * per_sm;
  if (lim.rows_ctas > 0 && grid > lim.rows_ctas) grid = lim.rows_ctas;
  if (grid > ngroups) grid = ngroups;
  unsigned int* status = device_status_word();
  if (!status) return cudaErrorUnknown;
  if (a.compact) {
    if (dtype == CAAT_BF16)
      return a.norm == 1 ? launch_fwd_warp_t<__nv_bfloat16, true, true>(a, cpt, g, grid, ngroups, status, st)
                         : launch_fwd_warp_t<__nv_bfloat16, false, true>(a, cpt, g, grid, ngroups, status, st);
    return a.norm == 1 ? launch_fwd_warp_t<float, true, true>(a, cpt, g, grid, ngroups, status, st)
                       : launch_fwd_warp_t<float, false, true>(a, cpt, g, grid, ngroups, status, st);
  }
  if (dtype == CAAT_BF16)
    return a.norm == 1 ? launch_fwd_warp_t<__nv_bfloat16, true, false>(a, cpt, g, grid, ngroups, status, st)
                       : launch_fwd_warp_t<__nv_bfloat16, false, false>(a, cpt, g, grid, ngroups, status, st);
  return a.norm == 1 ? launch_fwd_warp_t<float, true, false>(a, cpt, g, grid, ngroups, status, st)
                     : launch_fwd_warp_t<float, false, false>(a, cpt, g, grid, ngroups, status, st);
}

cudaError_t launch_rows_backward_warp(const RowBwdArgs& a, caat_dtype dtype, int max_rows, int* rows_used,
                                      cudaStream_t st) {
  const int cpt = rows_warp_cpt(a.h, a.t, dtype);
  const int ES = (int)elem_size(dtype);
  const LaunchLimits lim = effective_limits();
  const int per_sm = lim.rows_per_sm > 0 && lim.rows_per_sm < kCtasPerSm ? lim.rows_per_sm : kCtasPerSm;
  const size_t sm_budget = lim.rows_smem > 0 && (size_t)lim.rows_smem < kSmemPerSm ? (size_t)lim.rows_smem : kSmemPerSm;
  const WarpGeom g = warp_geometry(a.h, a.P, a.S_hi, ES, true, a.dHn != nullptr, a.compact != 0, sm_budget / per_sm - 1024);
  if (cpt == 0 || g.nstages < 2) return cudaErrorInvalidConfiguration;
  const int ngroups = (a.T + kW - 1) / kW;
  int grid = sm_count() * per_sm;
  if (lim.rows_ctas > 0 && grid > lim.rows_ctas) grid = lim.rows_ctas;
  if (grid > ngroups) grid = ngroups;
  if (grid > max_rows) grid = max_rows;
  *rows_used = grid;
  unsigned int* status = device_status_word();
  if (!status) return cudaErrorUnknown;
  if (a.compact) {
    if (dtype == CAAT_BF16)
      return a.norm == 1 ? launch_bwd_warp_t<__nv_bfloat16, true, true>(a, cpt, g, grid, ngroups, status, st)
                         : launch_bwd_warp_t<__nv_bfloat16, false, true>(a, cpt, g, grid, ngroups, status, st);
    return a.norm == 1 ? launch_bwd_warp_t<float, true, true>(a, cpt, g, grid, ngroups, status, st)
                       : launch_bwd_warp_t<float, false, true>(a, cpt, g, grid, ngroups, status, st);
  }
  if (dtype == CAAT_BF16)
    return a.norm == 1 ? launch_bwd_warp_t<__nv_bfloat16, true, false>(a, cpt, g, grid, ngroups, status, st)
                       : launch_bwd_warp_t<__nv_bfloat16, false, false>(a, cpt, g, grid, ngroups, status, st);
  return a.norm == 1 ? launch_bwd_warp_t<float, true, false>(a, cpt, g, grid, ngroups, status, st)
                     : launch_bwd_warp_t<float, false, false>(a, cpt, g, grid, ngroups, status, st);
}

}  // namespace caat
