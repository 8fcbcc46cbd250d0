// Generic strided batched GEMM on CUDA cores with fp32 accumulation.
//
// It serves the fp32 configuration (TF32 tensor cores cannot meet a 1e-4 relative
// tolerance) and bf16 shapes the tensor-core kernels do not take (K_r or S not a
// multiple of 8).  Correctness and generality first: every operand is addressed
// through element strides, so the same kernel runs the forward product, the data
// gradient and the weight gradient, and the "two segment" form covers the
// [shared | private] split of the contraction axis.
#include "caat_internal.h"

namespace caat {
namespace {

constexpr int BM = 64, BN = 64, BK = 16;

template <typename T_>
__device__ __forceinline__ float ldf(const void* p, long long off);
template <>
__device__ __forceinline__ float ldf<float>(const void* p, long long off) {
  return static_cast<const float*>(p)[off];
}
template <>
__device__ __forceinline__ float ldf<__nv_bfloat16>(const void* p, long long off) {
  return __bfloat162float(static_cast<const __nv_bfloat16*>(p)[off]);
}

template <typename T_>
__global__ void __launch_bounds__(256) gemm_simt_kernel(GemmProblem g) {
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];
  const int b = blockIdx.z;
  const int i0 = blockIdx.y * BM, j0 = blockIdx.x * BN;
  const int tid = threadIdx.x;
  const int ti = (tid / 16) * 4, tj = (tid % 16) * 4;
  float acc[4][4];
#pragma unroll
  for (int x = 0; x < 4; ++x)
#pragma unroll
    for (int y = 0; y < 4; ++y) acc[x][y] = 0.f;

  for (int sidx = 0; sidx < g.nseg; ++sidx) {
    const GemmSeg& s = g.seg[sidx];
    const bool a_kfast = s.sAk == 1;   // thread mapping follows the unit stride
    const bool b_jfast = s.sBj == 1;
    for (int q = 0; q < s.Q; ++q) {
      const long long a0 = (long long)b * s.sAb + (long long)q * s.sAq;
      const long long b0 = (long long)b * s.sBb + (long long)q * s.sBq;
      for (int k0 = 0; k0 < s.Kd; k0 += BK) {
#pragma unroll
        for (int r = 0; r < (BM * BK) / 256; ++r) {
          const int idx = tid + r * 256;
          const int i = a_kfast ? idx / BK : idx % BM;
          const int k = a_kfast ? idx % BK : idx / BM;
          float v = 0.f;
          if (i0 + i < g.M && k0 + k < s.Kd) v = ldf<T_>(s.A, a0 + (long long)(i0 + i) * s.sAi + (long long)(k0 + k) * s.sAk);
          As[k][i] = v;
        }
#pragma unroll
        for (int r = 0; r < (BN * BK) / 256; ++r) {
          const int idx = tid + r * 256;
          const int j = b_jfast ? idx % BN : idx / BK;
          const int k = b_jfast ? idx / BN : idx % BK;
          float v = 0.f;
          if (j0 + j < g.N && k0 + k < s.Kd) v = ldf<T_>(s.B, b0 + (long long)(k0 + k) * s.sBk + (long long)(j0 + j) * s.sBj);
          Bs[k][j] = v;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < BK; ++k) {
          float av[4], bv[4];
#pragma unroll
          for (int x = 0; x < 4; ++x) av[x] = As[k][ti + x];
#pragma unroll
          for (int y = 0; y < 4; ++y) bv[y] = Bs[k][tj + y];
#pragma unroll
          for (int x = 0; x < 4; ++x)
#pragma unroll
            for (int y = 0; y < 4; ++y) acc[x][y] = fmaf(av[x], bv[y], acc[x][y]);
        }
        __syncthreads();
      }
    }
  }
#pragma unroll
  for (int x = 0; x < 4; ++x) {
    const int i = i0 + ti + x;
    if (i >= g.M) continue;
#pragma unroll
    for (int y = 0; y < 4; ++y) {
      const int j = j0 + tj + y;
      if (j >= g.N) continue;
      const long long off = (long long)b * g.sCb + (long long)i * g.sCi + j;
      if (g.c_f32 || sizeof(T_) == 4)
        static_cast<float*>(g.C)[off] = acc[x][y];
      else
        static_cast<__nv_bfloat16*>(g.C)[off] = __float2bfloat16_rn(acc[x][y]);
    }
  }
}

}  // namespace

cudaError_t launch_gemm_simt(const GemmProblem& g, caat_dtype dtype, cudaStream_t st) {
  if (g.M <= 0 || g.N <= 0 || g.batch <= 0) return cudaSuccess;
  const dim3 grid((g.N + BN - 1) / BN, (g.M + BM - 1) / BM, g.batch);
  if (grid.y > 65535 || grid.z > 65535) return cudaErrorInvalidConfiguration;
  LaunchScope scope(CAAT_K_GEMM_CUDA_CORE, st);
  if (dtype == CAAT_BF16)
    gemm_simt_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(g);
  else
    gemm_simt_kernel<float><<<grid, 256, 0, st>>>(g);
  return cudaGetLastError();
}

}  // namespace caat
