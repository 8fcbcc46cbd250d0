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
  static const int thr = [] { const char* e = getenv("CAAT_ROWS_CPT1_MAX"); return e ? atoi(e) : 128; }();
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
