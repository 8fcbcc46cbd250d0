// Column-parallel half in front of the row-parallel layer (Section 3: Y_m = sigma(X_m A_m); the
// inner sum of Eq. A3).  With partially synchronised activations every rank has its own input X_m,
// so the layer is a batch of t independent products; they run on the same tcgen05 GEMM as the
// row-parallel layer (its "private columns only" wiring, S = 0), the activation and its derivative
// in streaming kernels of their own.
#include <cstring>

#include "caat_rows_common.cuh"

namespace caat {
namespace {

using namespace rows;

template <bool FAST>
__device__ __forceinline__ float logistic(float x) {
  return FAST ? __fdividef(1.0f, 1.0f + __expf(-x)) : 1.0f / (1.0f + expf(-x));
}

// Y[r, c] = silu(pre[r, c])                      (GATED = false, width N)
// Y[r, c] = silu(pre[r, c]) * pre[r, F + c]      (GATED = true,  pre has 2F columns, Y has F)
// One 16-byte chunk of Y per thread and grid-stride step; rows = t * T.
template <typename T_, bool GATED>
__global__ void __launch_bounds__(256) act_forward_kernel(const void* __restrict__ pre, void* __restrict__ Y,
                                                          long long rows, int width_out) {
  using V_ = VT<T_>;
  using raw = typename V_::raw;
  constexpr int V = V_::N;
  constexpr int ES = sizeof(T_);
  constexpr bool FAST = ES == 2;
  const int chunks = width_out / V;
  const int ld_pre = GATED ? 2 * width_out : width_out;
  const long long total = rows * chunks;
  pdl_wait();
  for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < total; q += (long long)gridDim.x * blockDim.x) {
    const long long r = q / chunks;
    const int c = (int)(q - r * chunks) * V;
    const char* pg = static_cast<const char*>(pre) + (r * ld_pre + c) * ES;
    float g[V], y[V];
    V_::unpack(ldg<raw>(pg), g);
    if (GATED) {
      float u[V];
      V_::unpack(ldg<raw>(pg + (long long)width_out * ES), u);
#pragma unroll
      for (int e = 0; e < V; ++e) y[e] = g[e] * logistic<FAST>(g[e]) * u[e];
    } else {
#pragma unroll
      for (int e = 0; e < V; ++e) y[e] = g[e] * logistic<FAST>(g[e]);
    }
    stg<raw>(static_cast<char*>(Y) + (r * width_out + c) * ES, V_::pack(y));
  }
}

// dpre from dY and pre:  silu'(g) = s (1 + g (1 - s)), s = logistic(g)
//   plain:  dpre = dY silu'(pre)
//   gated:  dG = dY U silu'(G),  dU = dY silu(G)
template <typename T_, bool GATED>
__global__ void __launch_bounds__(256) act_backward_kernel(const void* __restrict__ dY, const void* __restrict__ pre,
                                                           void* __restrict__ dpre, long long rows, int width_out) {
  using V_ = VT<T_>;
  using raw = typename V_::raw;
  constexpr int V = V_::N;
  constexpr int ES = sizeof(T_);
  constexpr bool FAST = ES == 2;
  const int chunks = width_out / V;
  const int ld_pre = GATED ? 2 * width_out : width_out;
  const long long total = rows * chunks;
  pdl_wait();
  for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < total; q += (long long)gridDim.x * blockDim.x) {
    const long long r = q / chunks;
    const int c = (int)(q - r * chunks) * V;
    const long long op = (r * ld_pre + c) * ES;
    float dy[V], g[V], dg[V];
    V_::unpack(ldg<raw>(static_cast<const char*>(dY) + (r * width_out + c) * ES), dy);
    V_::unpack(ldg<raw>(static_cast<const char*>(pre) + op), g);
    if (GATED) {
      float u[V], du[V];
      V_::unpack(ldg<raw>(static_cast<const char*>(pre) + op + (long long)width_out * ES), u);
#pragma unroll
      for (int e = 0; e < V; ++e) {
        const float s = logistic<FAST>(g[e]);
        dg[e] = dy[e] * u[e] * (s * fmaf(g[e], 1.0f - s, 1.0f));
        du[e] = dy[e] * (g[e] * s);
      }
      stg<raw>(static_cast<char*>(dpre) + op + (long long)width_out * ES, V_::pack(du));
    } else {
#pragma unroll
      for (int e = 0; e < V; ++e) {
        const float s = logistic<FAST>(g[e]);
        dg[e] = dy[e] * (s * fmaf(g[e], 1.0f - s, 1.0f));
      }
    }
    stg<raw>(static_cast<char*>(dpre) + op, V_::pack(dg));
  }
}

int act_grid(long long rows, int width_out, int V) {
  const long long total = rows * (width_out / V);
  long long blocks = (total + 255) / 256;
  const long long cap = (long long)sm_count() * 8;     // eight resident CTAs of 256 threads per SM
  if (blocks > cap) blocks = cap;
  return (int)(blocks < 1 ? 1 : blocks);
}

}  // namespace

cudaError_t launch_act_forward(caat_dtype dtype, int gated, const void* pre, void* Y, long long rows, int width_out,
                               cudaStream_t st) {
  const int V = dtype == CAAT_BF16 ? 8 : 4;
  const int grid = act_grid(rows, width_out, V);
  LaunchScope scope(CAAT_K_ACTIVATION, st);
  if (dtype == CAAT_BF16) {
    if (gated) return launch_pdl(act_forward_kernel<__nv_bfloat16, true>, dim3(grid), dim3(256), 0, st, pre, Y, rows, width_out);
    else return launch_pdl(act_forward_kernel<__nv_bfloat16, false>, dim3(grid), dim3(256), 0, st, pre, Y, rows, width_out);
  } else {
    if (gated) return launch_pdl(act_forward_kernel<float, true>, dim3(grid), dim3(256), 0, st, pre, Y, rows, width_out);
    else return launch_pdl(act_forward_kernel<float, false>, dim3(grid), dim3(256), 0, st, pre, Y, rows, width_out);
  }
  return cudaGetLastError();
}

cudaError_t launch_act_backward(caat_dtype dtype, int gated, const void* dY, const void* pre, void* dpre,
                                long long rows, int width_out, cudaStream_t st) {
  const int V = dtype == CAAT_BF16 ? 8 : 4;
  const int grid = act_grid(rows, width_out, V);
  LaunchScope scope(CAAT_K_ACTIVATION, st);
  if (dtype == CAAT_BF16) {
    if (gated) return launch_pdl(act_backward_kernel<__nv_bfloat16, true>, dim3(grid), dim3(256), 0, st, dY, pre, dpre, rows, width_out);
    else return launch_pdl(act_backward_kernel<__nv_bfloat16, false>, dim3(grid), dim3(256), 0, st, dY, pre, dpre, rows, width_out);
  } else {
    if (gated) return launch_pdl(act_backward_kernel<float, true>, dim3(grid), dim3(256), 0, st, dY, pre, dpre, rows, width_out);
    else return launch_pdl(act_backward_kernel<float, false>, dim3(grid), dim3(256), 0, st, dY, pre, dpre, rows, width_out);
  }
  return cudaGetLastError();
}

}  // namespace caat
