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

// 256 threads as a 16 x 16 grid, each owning a TM x TM patch of a (16 TM) x (16 TM) output tile.  TM = 4 for
// problems with enough tiles to fill the GPU; TM = 2 or 1 (32 x 32 / 16 x 16 tiles, 4 / 16 times as many blocks) for
// small ones, which are otherwise a handful of blocks grinding through the whole contraction on a handful of SMs
// (the 128 x 128 x 1024 product of the small fp32 configuration: 4 blocks, 53 us; 64 blocks, 3x faster).
constexpr int BK = 32;

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

// Position in the contraction: segment, rank q of the segment, k offset.  The k-tiles of all segments and
// ranks form one sequence, so the loads of the next tile are in flight while the current one is multiplied
// (small problems are a chain of global-memory latencies otherwise: 64 dependent round trips for the
// 128 x 128 x 1024 product of the small fp32 configuration).
struct KPos { int seg, q, k0; };

__device__ __forceinline__ bool kpos_valid(const GemmProblem& g, const KPos& p) { return p.seg < g.nseg; }
__device__ __forceinline__ KPos kpos_first(const GemmProblem& g) {
  KPos p{0, 0, 0};
  while (p.seg < g.nseg && (g.seg[p.seg].Q <= 0 || g.seg[p.seg].Kd <= 0)) ++p.seg;
  return p;
}
__device__ __forceinline__ KPos kpos_next(const GemmProblem& g, KPos p) {
  p.k0 += BK;
  if (p.k0 >= g.seg[p.seg].Kd) {
    p.k0 = 0;
    if (++p.q >= g.seg[p.seg].Q) {
      p.q = 0;
      do { ++p.seg; } while (p.seg < g.nseg && (g.seg[p.seg].Q <= 0 || g.seg[p.seg].Kd <= 0));
    }
  }
  return p;
}

template <typename T_, int BM, int BN, int RA, int RB>
__device__ __forceinline__ void fetch_tile(const GemmProblem& g, const KPos& p, int b, int i0, int j0, int tid, float (&ra)[RA],
                                           float (&rb)[RB]) {
  const GemmSeg& s = g.seg[p.seg];
  const bool a_kfast = s.sAk == 1;   // thread mapping follows the unit stride
  const bool b_jfast = s.sBj == 1;
  const long long a0 = (long long)b * s.sAb + (long long)p.q * s.sAq;
  const long long b0 = (long long)b * s.sBb + (long long)p.q * s.sBq;
#pragma unroll
  for (int r = 0; r < RA; ++r) {
    const int idx = tid + r * 256;
    const int i = a_kfast ? idx / BK : idx % BM;
    const int k = a_kfast ? idx % BK : idx / BM;
    ra[r] = (i0 + i < g.M && p.k0 + k < s.Kd) ? ldf<T_>(s.A, a0 + (long long)(i0 + i) * s.sAi + (long long)(p.k0 + k) * s.sAk) : 0.f;
  }
#pragma unroll
  for (int r = 0; r < RB; ++r) {
    const int idx = tid + r * 256;
    const int j = b_jfast ? idx % BN : idx / BK;
    const int k = b_jfast ? idx / BN : idx % BK;
    rb[r] = (j0 + j < g.N && p.k0 + k < s.Kd) ? ldf<T_>(s.B, b0 + (long long)(p.k0 + k) * s.sBk + (long long)(j0 + j) * s.sBj) : 0.f;
  }
}

template <typename T_, int TM>
__global__ void __launch_bounds__(256) gemm_simt_kernel(GemmProblem g) {
  constexpr int BM = 16 * TM, BN = 16 * TM;
  constexpr int RA = (BM * BK) / 256, RB = (BN * BK) / 256;   // elements of a k-tile each thread fetches
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];
  const int b = blockIdx.z;
  const int i0 = blockIdx.y * BM, j0 = blockIdx.x * BN;
  const int tid = threadIdx.x;
  const int ti = (tid / 16) * TM, tj = (tid % 16) * TM;
  float acc[TM][TM];
#pragma unroll
  for (int x = 0; x < TM; ++x)
#pragma unroll
    for (int y = 0; y < TM; ++y) acc[x][y] = 0.f;

  float ra[RA], rb[RB];
  KPos pos = kpos_first(g);
  if (kpos_valid(g, pos)) fetch_tile<T_, BM, BN, RA, RB>(g, pos, b, i0, j0, tid, ra, rb);
  while (kpos_valid(g, pos)) {
    {   // registers -> shared memory, in the layout the fetch used
      const GemmSeg& s = g.seg[pos.seg];
      const bool a_kfast = s.sAk == 1, b_jfast = s.sBj == 1;
#pragma unroll
      for (int r = 0; r < RA; ++r) {
        const int idx = tid + r * 256;
        As[a_kfast ? idx % BK : idx / BM][a_kfast ? idx / BK : idx % BM] = ra[r];
      }
#pragma unroll
      for (int r = 0; r < RB; ++r) {
        const int idx = tid + r * 256;
        Bs[b_jfast ? idx / BN : idx % BK][b_jfast ? idx % BN : idx / BK] = rb[r];
      }
    }
    __syncthreads();
    pos = kpos_next(g, pos);
    if (kpos_valid(g, pos)) fetch_tile<T_, BM, BN, RA, RB>(g, pos, b, i0, j0, tid, ra, rb);   // in flight during the products below
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      float av[TM], bv[TM];
#pragma unroll
      for (int x = 0; x < TM; ++x) av[x] = As[k][ti + x];
#pragma unroll
      for (int y = 0; y < TM; ++y) bv[y] = Bs[k][tj + y];
#pragma unroll
      for (int x = 0; x < TM; ++x)
#pragma unroll
        for (int y = 0; y < TM; ++y) acc[x][y] = fmaf(av[x], bv[y], acc[x][y]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int x = 0; x < TM; ++x) {
    const int i = i0 + ti + x;
    if (i >= g.M) continue;
#pragma unroll
    for (int y = 0; y < TM; ++y) {
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
  auto tiles_of = [&](int tl) { return (long long)((g.N + tl - 1) / tl) * ((g.M + tl - 1) / tl) * g.batch; };
  const int tile = tiles_of(64) >= 2LL * sm_count() ? 64 : (tiles_of(32) >= sm_count() / 2 ? 32 : 16);
  const dim3 grid((g.N + tile - 1) / tile, (g.M + tile - 1) / tile, g.batch);
  if (grid.y > 65535 || grid.z > 65535) return cudaErrorInvalidConfiguration;
  LaunchScope scope(CAAT_K_GEMM_CUDA_CORE, st);
  if (dtype == CAAT_BF16) {
    if (tile == 64) gemm_simt_kernel<__nv_bfloat16, 4><<<grid, 256, 0, st>>>(g);
    else if (tile == 32) gemm_simt_kernel<__nv_bfloat16, 2><<<grid, 256, 0, st>>>(g);
    else gemm_simt_kernel<__nv_bfloat16, 1><<<grid, 256, 0, st>>>(g);
  } else {
    if (tile == 64) gemm_simt_kernel<float, 4><<<grid, 256, 0, st>>>(g);
    else if (tile == 32) gemm_simt_kernel<float, 2><<<grid, 256, 0, st>>>(g);
    else gemm_simt_kernel<float, 1><<<grid, 256, 0, st>>>(g);
  }
  return cudaGetLastError();
}

}  // namespace caat
