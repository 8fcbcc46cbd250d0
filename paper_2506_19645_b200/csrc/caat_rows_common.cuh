// Helpers shared by the row kernels (direct and bulk-copy staged variants).
#pragma once

#include <cstdlib>

#include "caat_internal.h"

namespace caat {
namespace rows {

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

// ---- packed fp32 pairs (sm_100 executes fma / add / mul on two fp32 lanes per instruction; each lane
// is the IEEE single-precision result of the scalar operation)
__device__ __forceinline__ float2 f2(float x) { return make_float2(x, x); }
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) { return __ffma2_rn(a, b, c); }
__device__ __forceinline__ float2 mul2(float2 a, float2 b) { return __fmul2_rn(a, b); }
__device__ __forceinline__ float2 add2(float2 a, float2 b) { return __fadd2_rn(a, b); }

// 16-byte chunk <-> V/2 pairs of fp32
__device__ __forceinline__ void unpack2(const uint4& r, float2 (&f)[4]) {
  const unsigned w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
  for (int q = 0; q < 4; ++q) f[q] = make_float2(__uint_as_float(w[q] << 16), __uint_as_float(w[q] & 0xffff0000u));
}
__device__ __forceinline__ void unpack2(const float4& r, float2 (&f)[2]) {
  f[0] = make_float2(r.x, r.y);
  f[1] = make_float2(r.z, r.w);
}
__device__ __forceinline__ uint4 pack2(const float2 (&f)[4]) {
  unsigned w[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    __nv_bfloat162 b = __floats2bfloat162_rn(f[q].x, f[q].y);
    w[q] = *reinterpret_cast<unsigned*>(&b);
  }
  return make_uint4(w[0], w[1], w[2], w[3]);
}
__device__ __forceinline__ float4 pack2(const float2 (&f)[2]) { return make_float4(f[0].x, f[0].y, f[1].x, f[1].y); }

// 16-byte shared-memory load through a 32-bit shared address (volatile: stays behind the barrier waits)
template <typename raw>
__device__ __forceinline__ raw lds32(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return *reinterpret_cast<raw*>(&v);
}

template <typename raw>
__device__ __forceinline__ raw zero_raw();
template <>
__device__ __forceinline__ float4 zero_raw<float4>() { return make_float4(0.f, 0.f, 0.f, 0.f); }
template <>
__device__ __forceinline__ uint4 zero_raw<uint4>() { return make_uint4(0u, 0u, 0u, 0u); }

template <typename raw>
__device__ __forceinline__ raw ldg(const char* p) { return *reinterpret_cast<const raw*>(p); }
template <typename raw>
__device__ __forceinline__ void stg(char* p, const raw& v) { *reinterpret_cast<raw*>(p) = v; }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Sum of NV values over the TX threads of one token row (TX <= 512, so at most 16 warps).
// `red` holds [2][TY][16][NV] floats; `par` alternates so one barrier per call suffices.
template <int NV>
__device__ __forceinline__ void row_reduce(float (&v)[NV], float* red, int& par) {
  const int warps_x = blockDim.x >> 5;
#pragma unroll
  for (int q = 0; q < NV; ++q) v[q] = warp_sum(v[q]);
  if (warps_x == 1) return;
  const int lane = threadIdx.x & 31;
  float* buf = red + ((par * blockDim.y + threadIdx.y) * 16) * NV;
  if (lane == 0) {
#pragma unroll
    for (int q = 0; q < NV; ++q) buf[(threadIdx.x >> 5) * NV + q] = v[q];
  }
  __syncthreads();
#pragma unroll
  for (int q = 0; q < NV; ++q) v[q] = warp_sum(lane < warps_x ? buf[lane * NV + q] : 0.f);
  par ^= 1;
}

// Same sum, but always with the CTA-wide barrier (callers rely on it as a rendezvous).
template <int NV>
__device__ __forceinline__ void row_reduce_sync(float (&v)[NV], float* red, int& par) {
  const int warps_x = blockDim.x >> 5;
#pragma unroll
  for (int q = 0; q < NV; ++q) v[q] = warp_sum(v[q]);
  const int lane = threadIdx.x & 31;
  float* buf = red + ((par * blockDim.y + threadIdx.y) * 16) * NV;
  if (lane == 0 && warps_x > 1) {
#pragma unroll
    for (int q = 0; q < NV; ++q) buf[(threadIdx.x >> 5) * NV + q] = v[q];
  }
  __syncthreads();
  if (warps_x > 1) {
#pragma unroll
    for (int q = 0; q < NV; ++q) v[q] = warp_sum(lane < warps_x ? buf[lane * NV + q] : 0.f);
  }
  par ^= 1;
}

// column class of a chunk [col, col+V): 0 all shared, 1 all private, 2 mixed
__device__ __forceinline__ int chunk_class(int col, int V, int S) {
  return (col + V <= S) ? 0 : (col >= S ? 1 : 2);
}


struct RowGeom {
  int TX, TY, CPT;
  size_t smem_fwd, smem_bwd;   // dynamic shared memory of the direct kernels
};

inline RowGeom row_geometry(int h, caat_dtype dtype) {
  const int V = dtype == CAAT_BF16 ? 8 : 4;
  const int chunks = h / V;
  RowGeom g;
  // Two chunks per thread whenever the row is long enough: the per-rank overhead (barrier
  // wait, row reduction, pointer updates) is paid once per thread, and 256 threads with up
  // to 128 registers leave room for two CTAs per SM without spills.
#ifdef CAAT_MEASUREMENT_AIDS
  static const int thr = [] { const char* e = getenv("CAAT_ROWS_CPT1_MAX"); return e ? atoi(e) : 128; }();
#else
  constexpr int thr = 128;
#endif
  g.CPT = chunks <= thr ? 1 : 2;   // short rows: one chunk per thread keeps every lane busy and more warps resident
  int tx = round_up((chunks + g.CPT - 1) / g.CPT, 32);
  while (tx > 512) {
    g.CPT *= 2;
    tx = round_up((chunks + g.CPT - 1) / g.CPT, 32);
  }
  g.TX = tx;
  g.TY = tx >= 256 ? 1 : 256 / tx;
  const size_t red = (size_t)2 * g.TY * 16 * 2 * sizeof(float);
  g.smem_fwd = red;
  const size_t acc = g.TY > 1 ? (size_t)g.TY * g.TX * g.CPT * V * sizeof(float) : 0;
  g.smem_bwd = red > acc ? red : acc;
  return g;
}

}  // namespace rows
}  // namespace caat
