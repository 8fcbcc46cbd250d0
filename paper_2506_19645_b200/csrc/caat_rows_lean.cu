// Backward row kernel, lean variant of the bulk-copy staged kernel: per-rank residual layout, partition on a chunk
// boundary.
//
// Inside a long training step the GPU runs at its power cap (SM clocks near two thirds of the maximum) and every
// instruction the row kernels do not execute is energy the step gets back.  This kernel does the staged backward
// kernel's work with a quarter fewer instructions per 16-byte chunk (about 300 instead of 400 per rank for a thread's
// two chunks at h = 4096), most of them saved by needing fewer registers than the 128 a thread may have:
//   * the loop body exists once per WARP-UNIFORM pattern of chunk classes (NSH = how many of the thread's chunks are
//     shared channels, the rest private; -1 = classes differ between lanes or a chunk lies past the row end), so the
//     common patterns carry no class branches and no rank sum for private chunks;
//   * whether the stream's own gradient is given is a template parameter;
//   * only the three warps that issue bulk copies keep the producer's counters;
//   * outputs are addressed as a per-rank base pointer plus one 32-bit offset per chunk, stored by predicated
//     instructions instead of branches;
//   * the next token group's row statistics go from global to shared memory by asynchronous copies, not through
//     registers;
//   * the row reduction's barrier also carries the "a wait ran out" vote (barrier with OR reduction), and its second
//     stage reads the warps' partial sums as vectors.
// Warps of one CTA may run different instances of the body; they meet at the same CTA barrier (barrier 0) the same
// number of times, and every instance is entered by whole warps.
// Shared-memory ring, stage layout, bounded waits and the status word are those of the staged kernels.  (The same
// treatment of the forward kernel saves a fifth of its instructions and 3 % of its time when it runs alone, but
// nothing inside a training step, so the forward stays on the staged kernel.)
#include "caat_rows_bulk.cuh"

namespace caat {
namespace {

using namespace rows;

template <int N>
struct Int { static constexpr int value = N; };

// Sum of NV values over the threads of one token row (warps_x warps), always with ONE CTA barrier, which also
// ORs `failed` over the CTA (the return value).  `red`: [2][TY][NV][16] floats, `par` alternates.
template <int NV>
__device__ __forceinline__ int row_sum(float (&v)[NV], float* red, int& par, int warps_x, int wx, int lane, int failed) {
#pragma unroll
  for (int q = 0; q < NV; ++q) v[q] = warp_sum(v[q]);
  float* buf = red + ((par * blockDim.y + threadIdx.y) * NV) * 16;
  if (lane == 0) {
#pragma unroll
    for (int q = 0; q < NV; ++q) buf[q * 16 + wx] = v[q];
  }
  const int bad = __syncthreads_or(failed);
#pragma unroll
  for (int q = 0; q < NV; ++q) {
    const float* b = buf + q * 16;
    if (warps_x == 8) {
      const float4 x = *reinterpret_cast<const float4*>(b), y = *reinterpret_cast<const float4*>(b + 4);
      v[q] = ((x.x + x.y) + (x.z + x.w)) + ((y.x + y.y) + (y.z + y.w));
    } else if (warps_x == 4) {
      const float4 x = *reinterpret_cast<const float4*>(b);
      v[q] = (x.x + x.y) + (x.z + x.w);
    } else if (warps_x == 16) {
      const float4 x = *reinterpret_cast<const float4*>(b), y = *reinterpret_cast<const float4*>(b + 4);
      const float4 z = *reinterpret_cast<const float4*>(b + 8), w = *reinterpret_cast<const float4*>(b + 12);
      v[q] = (((x.x + x.y) + (x.z + x.w)) + ((y.x + y.y) + (y.z + y.w))) +
             (((z.x + z.y) + (z.z + z.w)) + ((w.x + w.y) + (w.z + w.w)));
    } else {
      float s = b[0];
      for (int w = 1; w < warps_x; ++w) s += b[w];
      v[q] = s;
    }
  }
  par ^= 1;
  return bad;
}

__device__ __forceinline__ void cp_async4(float* dst_shared, const float* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(dst_shared)), "l"(src) : "memory");
}

// 16-byte global store under a predicate held as an integer (nonzero = store): a predicated instruction, no branch
template <typename raw>
__device__ __forceinline__ void stg_if(uint32_t on, char* p, const raw& v) {
  static_assert(sizeof(raw) == 16, "one 16-byte chunk");
  const uint4 u = *reinterpret_cast<const uint4*>(&v);
  asm volatile("{\n .reg .pred p;\n setp.ne.u32 p, %5, 0;\n @p st.global.v4.b32 [%0], {%1, %2, %3, %4};\n}"
               ::"l"(p), "r"(u.x), "r"(u.y), "r"(u.z), "r"(u.w), "r"(on)
               : "memory");
}

// chunk pattern of this warp: the number of shared chunks when every lane has the same classes and all chunks lie
// inside the row, else -1
template <int CPT>
__device__ __forceinline__ int warp_pattern(const int (&cls)[CPT]) {
  int code = 0;
#pragma unroll
  for (int j = 0; j < CPT; ++j) code = (cls[j] == 3 || code < 0) ? -1 : code + (cls[j] == 0 ? 1 : 0);
  const int first = __shfl_sync(0xffffffffu, code, 0);
  return __all_sync(0xffffffffu, code == first) ? first : -1;
}

// ------------------------------------------------------------------ backward
// stage buffers: a = dX rows, b = Hn rows, c = dHn rows (when given), each [TY, h]
// DH: the gradient arriving at the stored stream (dHn) is given
template <typename T_, int CPT, bool LN, int MAXT, bool DH>
__global__ void __launch_bounds__(MAXT, MinBlocks<CPT, MAXT>::value)
rows_backward_lean(const RowBwdArgs a, const StageGeom sg, int ngroups, unsigned int* status) {
  using V_ = VT<T_>;
  using raw = typename V_::raw;
  constexpr int V = V_::N;
  constexpr int ES = sizeof(T_);
  constexpr int H2 = V / 2;
  extern __shared__ __align__(128) uint8_t smem[];
  const uint32_t ring32 = smem_u32(smem + sg.ring_off);
  const uint32_t bar0 = smem_u32(smem + sg.bar_off);
  float* red = reinterpret_cast<float*>(smem + sg.red_off);
  float* stat = reinterpret_cast<float*>(smem + sg.stat_off);   // [2 buffers][2 (rstd, mean)][t * TY]
  const int TX = blockDim.x, TY = blockDim.y;
  const int tid = threadIdx.y * TX + threadIdx.x, nthr = TX * TY;
  const int lane = tid & 31;
  const int wid = __shfl_sync(0xffffffffu, tid >> 5, 0);
  const int wx = __shfl_sync(0xffffffffu, (int)threadIdx.x >> 5, 0);
  const int warps_x = TX >> 5;
  const int NS = sg.nstages;
  const int t = a.t;
  const float inv_h = 1.0f / (float)a.h;
  constexpr bool has_dh = DH;
  const int nstat = t * TY;

  const int my_groups = blockIdx.x < ngroups ? (ngroups - blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  const long long total = (long long)my_groups * t;

  // producer: the next (token group, rank) to fetch, kept by the issuing warps (0: dX, 1: Hn, 2: dHn); the stage it
  // goes to is the one the consumers have just finished with
  int pn = 0, pm = 0;
  auto fetch = [&](uint32_t stage, uint32_t bar) {
    if (pn >= my_groups) return;
    const int n = pn, m = pm;
    if (++pm == t) { pm = 0; ++pn; }
    const long long i0 = (blockIdx.x + (long long)n * gridDim.x) * TY;
    const int rowsN = (int)((a.T - i0) < TY ? (a.T - i0) : TY);
    const uint32_t b = (uint32_t)rowsN * a.h * ES;
    const long long off = ((long long)m * a.T + i0) * a.h * ES;
    if (!elect_one()) return;
    if (wid == 0) {
      mbar_expect_tx(bar, (has_dh ? 3 * b : 2 * b) + sg.stall_bytes);
      bulk_g2s(stage + sg.off_a, static_cast<const char*>(a.dX) + off, b, bar);
    } else if (wid == 1) {
      bulk_g2s(stage + sg.off_b, static_cast<const char*>(a.Hn) + off, b, bar);
    } else {
      if (has_dh) bulk_g2s(stage + sg.off_c, static_cast<const char*>(a.dHn) + off, b, bar);
    }
  };

  if (tid == 0) {
    for (int s = 0; s < NS; ++s) mbar_init(bar0 + 8u * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (tid < NS)   // the zero slot of every stage (no copy ever lands there)
    *reinterpret_cast<uint4*>(smem + sg.ring_off + (size_t)tid * sg.stage_bytes + sg.zero_off) = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
  pdl_wait();   // from here on global memory is touched
  if (wid < 3)
    for (int q = 0; q < NS; ++q) fetch(ring32 + (uint32_t)q * sg.stage_bytes, bar0 + 8u * q);
  // row statistics of token group 0: element (m, ty) of rstd / mean
  for (int q = tid; q < nstat; q += nthr) {
    const int m = q / TY, ty = q % TY;
    const long long i = (long long)blockIdx.x * TY + ty;
    const bool ok = my_groups > 0 && i < a.T;
    stat[q] = ok ? a.rstd[(long long)m * a.T + i] : 0.f;
    if (LN) stat[nstat + q] = ok ? a.mean[(long long)m * a.T + i] : 0.f;
  }

  int col[CPT], cls[CPT];
  float2 gam[CPT][H2], dgacc[CPT][H2], dbacc[LN ? CPT : 1][H2];
#pragma unroll
  for (int j = 0; j < CPT; ++j) {
    col[j] = (threadIdx.x + j * TX) * V;
    cls[j] = col[j] >= a.h ? 3 : (col[j] < a.S ? 0 : 1);
#pragma unroll
    for (int q = 0; q < H2; ++q) { gam[j][q] = f2(0.f); dgacc[j][q] = f2(0.f); if constexpr (LN) dbacc[j][q] = f2(0.f); }
    if (cls[j] != 3) unpack2(ldg<raw>(static_cast<const char*>(a.gamma) + (long long)col[j] * ES), gam[j]);
  }
  const uint32_t off_hc = sg.off_c - sg.off_b;   // from a chunk of the stream to the same chunk of its gradient
  const float2 alpha2 = f2(a.alpha);
  const long long rank_h = (long long)a.T * a.h * ES;
  const int pattern = warp_pattern<CPT>(cls);
  __syncthreads();   // stats of group 0 visible

  long long k = 0;
  bool dead = false;
  auto body = [&](auto tag) {
    constexpr int NSH = decltype(tag)::value;
    auto shared_chunk = [&](int j) { if constexpr (NSH >= 0) return j < NSH; else return cls[j] == 0; };
    uint32_t sb = ring32;
    int cs = 0, par = 0;
    uint32_t cph = 0;
    for (int n = 0; n < my_groups; ++n) {
      const int i = (blockIdx.x + n * gridDim.x) * TY + threadIdx.y;   // < T + TY
      const bool valid = i < a.T;
      const float* st_cur = stat + (size_t)(n & 1) * 2 * nstat + threadIdx.y;
      float* st_nxt = stat + (size_t)((n + 1) & 1) * 2 * nstat;
      // the next group's row statistics go straight from global to shared memory (4-byte asynchronous copies into the
      // buffer nobody reads during this group); they are awaited before the barrier that ends the group
      if (n + 1 < my_groups) {
        const int g2 = blockIdx.x + (n + 1) * gridDim.x;
        for (int q = tid; q < nstat; q += nthr) {
          const int m2 = q / TY, ty2 = q % TY;
          const int i2 = g2 * TY + ty2;
          if (i2 < a.T) {
            cp_async4(st_nxt + q, a.rstd + (long long)m2 * a.T + i2);
            if (LN) cp_async4(st_nxt + nstat + q, a.mean + (long long)m2 * a.T + i2);
          } else {
            st_nxt[q] = 0.f;
            if (LN) st_nxt[nstat + q] = 0.f;
          }
        }
      }
      bool act[CPT];
      uint32_t aX[CPT], aH[CPT];   // stage-relative addresses of the dX and stream chunks; the zero slot when inactive
      uint32_t off[CPT];   // of the chunk inside one rank's [T, h] plane of dR
      float2 gsum[CPT][H2];
#pragma unroll
      for (int j = 0; j < CPT; ++j) {
        act[j] = valid && (NSH >= 0 || cls[j] != 3);
        const uint32_t oX = ((uint32_t)threadIdx.y * a.h + col[j]) * ES;
        aX[j] = act[j] ? sg.off_a + oX : sg.zero_off;
        aH[j] = act[j] ? sg.off_b + oX : sg.zero_off;
        off[j] = (uint32_t)(((long long)i * a.h + col[j]) * ES);
#pragma unroll
        for (int q = 0; q < H2; ++q) gsum[j][q] = f2(0.f);
      }
      [[maybe_unused]] const uint32_t hc = valid ? off_hc : 0u;
      char* dr_m = static_cast<char*>(a.dR);

      for (int m = 0; m < t; ++m) {
        const int failed = mbar_wait(bar0 + 8u * cs, cph, sg.spin_cap) ? 0 : 1;
        const float rs_c = st_cur[m * TY];
        const float mu_c = LN ? st_cur[nstat + m * TY] : 0.f;
        const float2 rs2 = f2(rs_c);

        float2 xh[CPT][H2], dxh[CPT][H2];
        [[maybe_unused]] raw rdh[CPT];   // stream-gradient chunk, kept packed across the barrier (needed only after it)
        float2 s1 = f2(0.f), s2 = f2(0.f);
#pragma unroll
        for (int j = 0; j < CPT; ++j) {
          float2 dx[H2], hn[H2];
          unpack2(lds32<raw>(sb + aX[j]), dx);
          unpack2(lds32<raw>(sb + aH[j]), hn);
          if constexpr (DH) rdh[j] = lds32<raw>(sb + aH[j] + ((NSH >= 0 || cls[j] != 3) ? hc : 0u));
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
        if (row_sum<LN ? 2 : 1>(sacc, red, par, warps_x, wx, lane, failed)) {   // barrier: stage fully read
          k = (long long)n * t + m;
          dead = true;
          return;
        }
        if (wid < 3) fetch(sb, bar0 + 8u * cs);
        sb += sg.stage_bytes;
        if (++cs == NS) { cs = 0; cph ^= 1u; sb = ring32; }
        const float c1 = LN ? sacc[0] * inv_h : 0.f;
        const float c2 = (LN ? sacc[LN ? 1 : 0] : sacc[0]) * inv_h;
        const float2 nc2 = f2(-c2), nc1 = f2(-c1);
#pragma unroll
        for (int j = 0; j < CPT; ++j) {
          float2 gg[H2], dh[H2];
          if constexpr (DH) unpack2(rdh[j], dh);
#pragma unroll
          for (int q = 0; q < H2; ++q) {
            float2 tt = fma2(xh[j][q], nc2, dxh[j][q]);
            if (LN) tt = add2(tt, nc1);
            gg[q] = DH ? fma2(rs2, tt, dh[q]) : mul2(rs2, tt);
          }
          stg_if<raw>(act[j] ? 1u : 0u, dr_m + off[j], pack2(gg));
          if (shared_chunk(j)) {
#pragma unroll
            for (int q = 0; q < H2; ++q) gsum[j][q] = add2(gsum[j][q], gg[q]);   // fp32 rank sum, m ascending
          } else if (a.zp) {   // the scaled private copy, for a GEMM that does not read dR in place
            float2 zp[H2];
#pragma unroll
            for (int q = 0; q < H2; ++q) zp[q] = mul2(alpha2, gg[q]);           // private gradient carries alpha
            if (act[j])
              stg<raw>(static_cast<char*>(a.zp) + (((long long)m * a.T + i) * a.P + (col[j] - a.S)) * ES, pack2(zp));
          }
        }
        dr_m += rank_h;
      }
#pragma unroll
      for (int j = 0; j < CPT; ++j)
        if (act[j] && shared_chunk(j)) stg<raw>(gs_row(a, (long long)i, ES) + (long long)col[j] * ES, pack2(gsum[j]));
      asm volatile("cp.async.wait_all;" ::: "memory");   // this thread's copies of the next group's statistics have landed
      __syncthreads();
    }
  };
  if (pattern == 0) body(Int<0>{});
  else if (pattern == CPT) body(Int<CPT>{});
  else if (CPT == 2 && pattern == 1) body(Int<(CPT == 2 ? 1 : 0)>{});
  else body(Int<-1>{});

  if (dead) {
    if (tid == 0) {
      atomicExch(status, 5u);
      const long long issued = (k + NS) < total ? (k + NS) : total;
      for (long long q = k + 1; q < issued; ++q)
        for (uint32_t it = 0; it < (1u << 10); ++it)   // each poll sleeps up to the suspend hint: ~20 ms per stage at most
          if (mbar_try(bar0 + 8u * (uint32_t)(q % NS), (uint32_t)((q / NS) & 1))) break;
    }
    return;
  }

  // Partial norm-parameter gradients of this CTA: one row of [h] per CTA, token rows of the CTA summed in order
  // through shared memory when TY > 1.
  for (int which = 0; which < (LN ? 2 : 1); ++which) {
    float* out = which == 0 ? a.dgpart : a.dbpart;
    if (out == nullptr) continue;
    if (TY == 1) {
#pragma unroll
      for (int j = 0; j < CPT; ++j) {
        if (cls[j] == 3) continue;
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
        if (cls[j] == 3) continue;
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
template <typename T_, bool LN>
cudaError_t launch_bwd_lean_t(const RowBwdArgs& a, const RowGeom& g, const StageGeom& sg, int grid, int ngroups,
                              unsigned int* status, cudaStream_t st) {
  const dim3 block(g.TX, g.TY);
  cudaError_t e = cudaSuccess;
  LaunchScope scope(CAAT_K_ROWS_BACKWARD, st);
  const int threads = g.TX * g.TY;
#define CAAT_LAUNCH(CPT_, MAXT_)                                                                                        \
  do {                                                                                                                  \
    if (a.dHn) {                                                                                                        \
      e = set_smem(rows_backward_lean<T_, CPT_, LN, MAXT_, true>, sg.smem);                                             \
      if (e == cudaSuccess)                                                                                             \
        e = launch_pdl(rows_backward_lean<T_, CPT_, LN, MAXT_, true>, dim3(grid), block, sg.smem, st, a, sg, ngroups,   \
                       status);                                                                                         \
    } else {                                                                                                            \
      e = set_smem(rows_backward_lean<T_, CPT_, LN, MAXT_, false>, sg.smem);                                            \
      if (e == cudaSuccess)                                                                                             \
        e = launch_pdl(rows_backward_lean<T_, CPT_, LN, MAXT_, false>, dim3(grid), block, sg.smem, st, a, sg, ngroups,  \
                       status);                                                                                         \
    }                                                                                                                   \
  } while (0)
  if (g.CPT == 1 && threads <= 256) CAAT_LAUNCH(1, 256);
  else if (g.CPT == 1) CAAT_LAUNCH(1, 512);
  else if (g.CPT == 2 && threads <= 256) CAAT_LAUNCH(2, 256);
  else if (g.CPT == 2) CAAT_LAUNCH(2, 512);
  else return cudaErrorInvalidValue;
#undef CAAT_LAUNCH
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

// per-rank layout, the partition on a chunk boundary, one rank's plane addressable with 32 bits, at most two chunks
// per thread (with four, rows longer than 8192 elements in bf16, the general kernels spill less) and at least the
// three warps that issue copies
bool rows_lean_usable(int compact, int h, int T, int S, int S_lo, int S_hi, caat_dtype dtype) {
  const RowGeom g = row_geometry(h, dtype);
  return !compact && S_lo == S && S_hi == S && (long long)T * h * (long long)elem_size(dtype) < (1LL << 32) &&
         g.CPT <= 2 && g.TX * g.TY >= 96;
}

cudaError_t launch_rows_backward_lean(const RowBwdArgs& a, caat_dtype dtype, const RowGeom& g, const StageGeom& sg, int grid,
                                      int ngroups, unsigned int* status, cudaStream_t st) {
  if (dtype == CAAT_BF16)
    return a.norm == 1 ? launch_bwd_lean_t<__nv_bfloat16, true>(a, g, sg, grid, ngroups, status, st)
                       : launch_bwd_lean_t<__nv_bfloat16, false>(a, g, sg, grid, ngroups, status, st);
  return a.norm == 1 ? launch_bwd_lean_t<float, true>(a, g, sg, grid, ngroups, status, st)
                     : launch_bwd_lean_t<float, false>(a, g, sg, grid, ngroups, status, st);
}

}  // namespace caat
