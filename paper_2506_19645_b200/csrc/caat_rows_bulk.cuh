// Bulk-copy staging shared by the staged row kernels: mbarrier and cp.async.bulk wrappers (every wait bounded), the
// layout of a stage of the shared-memory ring, and how many CTAs per SM a launch asks for.
#pragma once

#include "caat_rows_common.cuh"

namespace caat {
namespace rows {

constexpr uint32_t kSuspendHintNs = 20000u;   // the waiting warp sleeps in hardware instead of spinning
constexpr int kMaxStages = 8;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
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
// one lane of a converged warp (the hardware's pick); branching on it keeps the control flow warp-uniform
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n .reg .pred P;\n elect.sync _|P, 0xffffffff;\n selp.u32 %0, 1, 0, P;\n}" : "=r"(pred));
  return pred != 0;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t cap) {
  for (uint32_t it = 0; it < cap; ++it)
    if (mbar_try(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}

template <typename raw>
__device__ __forceinline__ raw lds(const uint8_t* p) { return *reinterpret_cast<const raw*>(p); }

struct StageGeom {
  int nstages;
  uint32_t off_a, off_b, off_c;  // byte offsets of the three row buffers inside a stage
  uint32_t off_d, off_e;         // compact layout: the shared rows of the stream (and of its gradient)
  uint32_t stage_bytes;
  uint32_t ring_off, bar_off, red_off, stat_off, acc_off;
  uint32_t zero_off;             // 16 zero bytes inside every stage (read by chunks past the row end)
  uint32_t keep_off;             // compact backward: [TY, S] shared rows of the stream, kept for all ranks of a token group
  size_t smem;
  uint32_t spin_cap;             // polls of one mbarrier wait before the CTA gives up (rows_hooks)
  uint32_t stall_bytes;          // time-out test: bytes every stage announces on top of its copies (0 otherwise)
};

// resident CTAs per SM the launch bounds ask for: one chunk per thread in small CTAs leaves ~85
// registers per thread at three CTAs, two chunks per thread 128 registers at two CTAs
template <int CPT, int MAXT>
struct MinBlocks { static constexpr int value = MAXT <= 256 ? (CPT == 1 ? 3 : 2) : (CPT == 1 ? 2 : 1); };

inline StageGeom stage_geometry(const RowGeom& g, int h, int P, int S_hi, int t, int ES, bool backward, bool has_c,
                         bool compact, size_t budget) {
  StageGeom sg{};
  const uint32_t rowA = (uint32_t)g.TY * h * ES;
  const uint32_t rowP = (uint32_t)g.TY * P * ES, rowS = (uint32_t)g.TY * S_hi * ES;
  if (backward && compact) {          // dX | Hnp | dHnp | Hns | dHns   (P + S_hi = h)
    sg.off_a = 0; sg.off_b = rowA; sg.off_c = rowA + rowP;
    sg.off_d = has_c ? rowA + 2 * rowP : rowA + rowP;
    sg.off_e = sg.off_d + rowS;
    sg.stage_bytes = sg.off_d + (has_c ? 2 : 1) * rowS;
  } else if (backward) {
    sg.off_a = 0; sg.off_b = rowA; sg.off_c = 2 * rowA;
    sg.stage_bytes = (has_c ? 3 : 2) * rowA;
  } else if (compact) {               // Rp | zp | zs | Rs
    sg.off_a = 0; sg.off_b = rowP; sg.off_c = 2 * rowP; sg.off_d = 2 * rowP + rowS;
    sg.stage_bytes = 2 * rowP + 2 * rowS;
  } else {
    sg.off_a = 0; sg.off_b = rowA; sg.off_c = rowA + rowP;
    sg.stage_bytes = rowA + rowP + rowS;
  }
  sg.zero_off = sg.stage_bytes;
  sg.stage_bytes = (sg.stage_bytes + 16u + 127u) & ~127u;
  // fixed part: barriers + abort flag, reduction scratch, row statistics
  size_t off = 0;
  sg.bar_off = (uint32_t)off; off += 8 * kMaxStages + 16;
  off = align_up(off, 16);
  sg.red_off = (uint32_t)off; off += (size_t)2 * g.TY * 16 * 2 * sizeof(float);
  sg.stat_off = (uint32_t)off; off += backward ? (size_t)2 * 2 * t * g.TY * sizeof(float) : 0;
  off = align_up(off, 128);
  sg.keep_off = (uint32_t)off; off += (backward && compact) ? (size_t)rowS : 0;
  off = align_up(off, 128);
  sg.ring_off = (uint32_t)off;
  sg.acc_off = sg.ring_off;
  const size_t acc = (backward && g.TY > 1) ? (size_t)g.TY * g.TX * g.CPT * (16 / ES) * sizeof(float) : 0;
  int ns = (int)((budget - off) / sg.stage_bytes);
  if (ns > kMaxStages) ns = kMaxStages;
  sg.nstages = ns;
  size_t ring = (size_t)(ns > 0 ? ns : 0) * sg.stage_bytes;
  if (ring < acc) ring = acc;
  sg.smem = off + ring;
  const RowsHooks hooks = rows_hooks();
  sg.spin_cap = hooks.spin_cap;
  sg.stall_bytes = hooks.stall ? 16u : 0u;
  return sg;
}

template <typename K>
inline cudaError_t set_smem(K kernel, size_t bytes) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

constexpr size_t kSmemPerSm = 227 * 1024;

// resident CTAs per SM the register budget allows (64 registers per thread when CPT == 1)
inline int ctas_per_sm(const RowGeom& g) {
  const int threads = g.TX * g.TY;
  if (g.CPT != 1) return threads <= 256 ? 2 : 1;   // 128 registers per thread
  if (threads > 256) return 2;                      // 64 registers per thread
  int n = 65536 / (threads * 80);                   // 80 registers per thread
  return n < 1 ? 1 : (n > 6 ? 6 : n);
}


}  // namespace rows

// lean variant of the staged backward kernel (per-rank layout, partition on a chunk boundary); same ring and grid
bool rows_lean_usable(int compact, int h, int T, int S, int S_lo, int S_hi, caat_dtype dtype);
cudaError_t launch_rows_backward_lean(const RowBwdArgs& a, caat_dtype dtype, const rows::RowGeom& g, const rows::StageGeom& sg,
                                      int grid, int ngroups, unsigned int* status, cudaStream_t st);

}  // namespace caat
