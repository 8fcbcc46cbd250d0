// bf16 tensor-core GEMMs for sm_100a: TMA -> shared-memory ring -> tcgen05.mma with the
// fp32 accumulator in tensor memory -> tcgen05.ld epilogue.
//
// One persistent, warp-specialised kernel serves the three contractions of the layer:
//   forward   Zt = Y W^T        A = Y  (K-major),  B = W (K-major)
//   dgrad     dY = dZt W        A = dZt (K-major), B = W (N-major: K_r contiguous)
//   wgrad     dW = dZt^T Y      A = dZt (M-major: channels contiguous), B = Y (N-major)
// where dZt / Zt live in the split scratch layout [shared once | private per rank].
// Shared output columns of the forward accumulate over ALL ranks in one accumulator (the
// partial channel-reduce of Eq. A3 becomes a longer contraction), so rank partials of the
// shared channels never exist in memory.
//
// Roles per CTA (224 threads): warp 0 issues the TMA loads of the A operand and warp 6 those
// of the B operand (one thread issuing every box of a stage was the limiter when a stage is
// four boxes; two instruction streams walk the same schedule independently), warp 1 issues
// MMAs and owns the tensor-memory allocation, warps 2-5 drain accumulators (tcgen05.ld) and
// store.  Two
// accumulators of up to 256 columns alternate so a tile's epilogue overlaps the next
// tile's MMAs.  Every mbarrier wait is bounded; on a timeout the kernel records a status
// word, drains its own copies in flight, frees tensor memory and returns.
#include <cuda.h>

#include <cstdio>
#include <cstdlib>
#include <mutex>

#include "caat_internal.h"

namespace caat {
namespace {

constexpr int BM = 128;           // rows of an output tile (UMMA M, cta_group::1)
constexpr int BK = 64;            // contraction elements per pipeline stage (128 bytes of bf16)
constexpr int UMMA_K = 16;        // contraction elements per tcgen05.mma (kind::f16)
constexpr int kThreads = 224;     // warps: 0 = A producer, 1 = MMA issuer, 2..5 = epilogue, 6 = B producer
constexpr int kProducerB = 6;
constexpr int kAccCols = 256;     // column stride between the two accumulators
constexpr int kTmemCols = 512;
constexpr uint32_t kSpinCap = 1u << 22;
constexpr int kMaxStages = 8;
constexpr int kCBuf = 128 * 64;   // one output staging buffer: 128 rows x 64 bytes (32 bf16 / 16 fp32 columns)
// Measurement aids that make results wrong (phase ablation: skipped loads, stores, barriers) and the
// tile-shape overrides exist only in builds compiled with -DCAAT_MEASUREMENT_AIDS; the library as
// built by build.py honours none of them.  Bit 1024 (a stage wait made to run out, for the time-out
// test) stays: it changes no result of a call that returns CAAT_OK.
#ifdef CAAT_MEASUREMENT_AIDS
constexpr int kAidMask = ~0;
#else
constexpr int kAidMask = 1024;
#endif

struct Unit {            // one contraction segment of a tile
  int mapA, mapB;        // indices into the tensor-map array
  int ak0, am0;          // offsets added to A's K / M coordinate
  int bk0, bn0;          // offsets added to B's K / N coordinate
  int a_zb, a_zq;        // A's z coordinate = b * a_zb + q * a_zq
  int b_zb, b_zq;
  int Q;                 // rank loop (forward shared columns: all ranks, else 1)
  int ksteps;            // stages per q = ceil(extent / BK)
};

struct Region {          // a family of output tiles with the same operand wiring
  int nunits;
  Unit u[2];
  int M, N, batch;       // valid output extents per batch
  int mtiles, ntiles;    // the output goes through the region's own tensor map (TMA store);
                         // its z coordinate is split * batch + b
  float* out_t;          // transposed direct-store output (decode), else unused
  int splits;            // split-K factor of this region's tiles (set by finish_tiles from Params::splits when 0)
  int b_slowest;         // tile order: 1 = rank index slowest (a rank's weights / activations stay
                         // hot in L2 while its row tiles stream), 0 = row tile slowest
  float scale;           // fp32 outputs are multiplied by it in the epilogue (0 means 1)
};

struct Params {
  int nregions;
  Region r[2];
  int BN;                // tile width (UMMA N): multiple of 16 (of 64 when B is N-major)
  int nstages;
  int a_mn, b_mn;        // 1: operand is MN-major in global memory
  int out_f32;
  int out_transposed;    // 1: D is [channels x tokens]; store fp32 straight to the region's out_t[z][token][channel]
  long long out_t_ld;    // channels per token row of out_t
  int cg;                // CTAs per tile: 1, or 2 (tcgen05 cta_group::2, clusters of two)
  int splits;            // split-K factor (only with a single unit and Q == 1)
  int push_slice;        // > 0: tiles of region 0 (the shared columns) are stored into the peer GPUs' receive slots, the
                         // owner of a tile being its first row / push_slice (a multiple of the tile's rows)
  int tiles_r0;          // tiles of region 0 (including splits)
  int tiles_total;
  unsigned int* status;
  uint32_t spin_cap;     // polls of one mbarrier wait before the role gives up (kSpinCap; CAAT_TC_SPINCAP for the timeout test)
  int debug;             // measurement aid (env CAAT_TC_DEBUG, masked by kAidMask; results are then wrong): 1 = no operand loads,
                         // 2 = no epilogue work at all, 4 = no A loads, 8 = no B loads; epilogue stops after the
                         // tensor-memory load (32) / after the staging stores (16); 64 = no slab barrier,
                         // 128 = no TMA store; 512 = producer lanes take no second k-step; 1024 = the A boxes are
                         // announced to the stage barrier but never issued, so the consumers' waits run out
                         // (the timeout test: the kernel must flag it, drain and return)
};

// ---------------------------------------------------------------- PTX wrappers
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
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false when the cap ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t cap) {
  for (uint32_t it = 0; it < cap; ++it) {
    if (mbar_try(bar, parity)) return true;
    if ((it & 1023u) == 1023u && *abort_flag) return false;
  }
  return false;
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}

// One lane of a converged warp (the hardware's pick).  Branching on it instead of on the lane index keeps
// the surrounding control flow warp-uniform, so loop state and the operands of the tensor-core and
// TMA instructions can live in uniform registers: issuing four MMAs and a commit from a divergent
// single-lane branch cost 310 cycles per k-step, from a uniform loop 130.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n .reg .pred P;\n elect.sync _|P, 0xffffffff;\n selp.u32 %0, 1, 0, P;\n}" : "=r"(pred));
  return pred != 0;
}
// Bounded wait by a whole warp with a warp-uniform result.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t cap) {
  return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag, cap));
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, int x, int y, int z, uint32_t src) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];"
               ::"l"(map), "r"(x), "r"(y), "r"(z), "r"(src)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void epi_barrier() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle (layout type 2), descriptor version 1.
//   K-major operand : rows of 128 bytes (64 bf16 of K), 8-row groups 1024 bytes apart (SBO).
//   MN-major operand: 64-element (128-byte) MN chunks; within a chunk K rows are 128 bytes
//                     apart, 8-row groups 1024 bytes apart (SBO); chunks LBO bytes apart.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// Output maps of the peers' receive slots (the exchange of the shared-channel slab over peer memory).
struct PeerMaps { CUtensorMap m[CAAT_MAX_PEERS]; };

struct TileCoord {
  int region, b, mt, nt, split;
};

__device__ __forceinline__ TileCoord decode_tile(const Params& p, int tile) {
  TileCoord c;
  c.region = (tile >= p.tiles_r0) ? 1 : 0;
  int rem = tile - (c.region ? p.tiles_r0 : 0);
  const Region& r = p.r[c.region];
  c.nt = rem % r.ntiles; rem /= r.ntiles;
  c.split = rem % r.splits; rem /= r.splits;
  if (r.b_slowest) {
    c.mt = rem % r.mtiles; rem /= r.mtiles;
    c.b = rem;
  } else {
    c.b = rem % r.batch; rem /= r.batch;
    c.mt = rem;
  }
  return c;
}

// Columns of B a tile really needs: the last tile of a ragged N (N-major B only) is narrowed to
// whole 64-column chunks per CTA, so no padded columns are loaded or multiplied.
__device__ __forceinline__ int tile_cols(const Params& p, const Region& r, int nt, int cg) {
  if (!p.b_mn) return p.BN;
  const int left = r.N - nt * p.BN;
  if (left >= p.BN) return p.BN;
  const int q = 64 * cg;
  return (left + q - 1) / q * q;
}

// k-step range of a unit for a split
__device__ __forceinline__ void split_range(int splits, const Unit& u, int split, int& k_begin, int& k_end) {
  if (splits == 1) { k_begin = 0; k_end = u.ksteps; return; }
  const int per = (u.ksteps + splits - 1) / splits;
  k_begin = split * per;
  k_end = k_begin + per < u.ksteps ? k_begin + per : u.ksteps;
  if (k_begin > k_end) k_begin = k_end;
}

// ---- cluster helpers (CG == 2: a CTA pair works on one 256-row tile) -------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t mapa_rank(uint32_t saddr, uint32_t rank) {   // same offset in CTA `rank`
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load whose completion may be signalled on the peer CTA's mbarrier (the data lands in the issuing CTA only)
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {   // arrives on `bar` in BOTH CTAs of the pair
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(bar), "h"((unsigned short)3)
      : "memory");
}

// CG = 1: one CTA per 128-row tile.  CG = 2: a cluster of two CTAs per 256-row tile
// (tcgen05 cta_group::2): each CTA stages its own 128 rows of A and HALF of the B tile, the
// leader (cluster rank 0) issues the MMAs for both and the tensor cores read B from both CTAs'
// shared memory, so the operand bytes a CTA pulls from L2 per flop drop by a third.
template <int CG>
__global__ void __launch_bounds__(kThreads, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap map0, const __grid_constant__ CUtensorMap map1,
               const __grid_constant__ CUtensorMap map2, const __grid_constant__ CUtensorMap map3,
               const __grid_constant__ CUtensorMap cmap0, const __grid_constant__ CUtensorMap cmap1,
               const __grid_constant__ PeerMaps pm, const Params p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  constexpr int BMT = BM * CG;                     // rows of a tile (of the pair's tile)
  const uint32_t rank = CG == 2 ? cluster_ctarank() : 0u;
  const int worker = blockIdx.x / CG, nworkers = gridDim.x / CG;
  // carve: [stages x (A tile | this CTA's part of the B tile)], output staging, barriers
  const uint32_t bn_cta = (uint32_t)p.BN / CG;
  const uint32_t a_bytes = BM * BK * 2;
  const uint32_t b_bytes = bn_cta * BK * 2;
  const uint32_t stage_bytes = a_bytes + b_bytes;
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t tiles_sa = smem_u32(base);
  uint8_t* cstage = base + (size_t)p.nstages * stage_bytes;   // 3 output staging buffers of kCBuf bytes
  uint64_t* bars = reinterpret_cast<uint64_t*>(cstage + 3 * kCBuf);
  // bars: full[nstages], empty[nstages], tfull[2], tempty[2]
  const uint32_t full0 = smem_u32(bars);
  const uint32_t empty0 = full0 + 8u * p.nstages;
  const uint32_t tfull0 = empty0 + 8u * p.nstages;
  const uint32_t tempty0 = tfull0 + 16u;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * p.nstages + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const CUtensorMap* maps[4] = {&map0, &map1, &map2, &map3};
  const CUtensorMap* cmaps[2] = {&cmap0, &cmap1};

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.nstages; ++s) { mbar_init(full0 + 8u * s, 1); mbar_init(empty0 + 8u * s, 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull0 + 8u * a, 1); mbar_init(tempty0 + 8u * a, 4 * CG); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    if (CG == 2) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if (CG == 2) cluster_sync();      // the peer's barriers are initialised before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();   // set-up done; operands and outputs may still be in use by the previous kernel until here

  if (warp == 0 || warp == kProducerB) {
    // ------------------------------------------------------------ TMA producers
    // Two producer warps run the same schedule: warp 0 issues the A boxes (and, in the leader CTA, posts
    // the stage's expected bytes), warp kProducerB the B boxes.
    const bool isA = warp == 0;
    // Lanes of the producer warp share the issue work: lane = (k-step of a group of kKI consecutive k-steps,
    // box of the stage).  A K-major operand is one box per stage, an M-/N-major one a box per 64 rows or
    // columns.  All active lanes run the same instructions on different stages / boxes, so the group is
    // issued in the time of one k-step: a single lane needs ~575 cycles per k-step (240 for the wait on a
    // barrier that is already free, 250 for the announcement and one box, 85 of loop), more than the 384-512
    // cycles the tensor cores take for it.
    constexpr int kKI = 2;
    const bool multi = (isA ? p.a_mn : p.b_mn) != 0;
    const int nbmax = multi ? (isA ? BM / 64 : (int)(p.BN / CG) / 64) : 1;      // boxes per stage, at most
    // measured: pays for multi-box operands (dgrad / wgrad -5...-8 %) and the weight stream of the decode
    // path (-5 %); a K-major operand of the large GEMMs gains nothing (its tiles wait for L2, not for the
    // issue) and a ring shorter than six stages loses more to pairwise refills than it gains
    const int nki = ((multi || p.out_transposed) && p.nstages >= 6 && !(p.debug & kAidMask & 512)) ? kKI : 1;
    const int jk = lane / nbmax, box = lane - jk * nbmax;                         // this lane's k-step slot and box
    if (jk < nki) {
      int stage = 0; uint32_t phase = 0;
      long long issued = 0;
      bool ok = true;
      for (int tile = worker; tile < p.tiles_total && ok; tile += nworkers) {
        const TileCoord c = decode_tile(p, tile);
        const Region& r = p.r[c.region];
        const uint32_t cols_cta = (uint32_t)tile_cols(p, r, c.nt, CG) / CG;    // B columns this CTA stages
        const uint32_t b_tile_bytes = cols_cta * BK * 2;
        const int m0 = c.mt * BMT + (int)rank * BM, n0 = c.nt * p.BN + (int)(rank * cols_cta);
        const uint32_t tx = (uint32_t)CG * (((p.debug & kAidMask & 4) ? 0u : a_bytes) + ((p.debug & kAidMask & 8) ? 0u : b_tile_bytes));
        const bool skip = isA ? (p.debug & kAidMask & (4 | 1024)) != 0 : (p.debug & kAidMask & 8) != 0;
        const int nb = multi ? (isA ? BM / 64 : (int)cols_cta / 64) : 1;         // boxes of this tile's stages
        for (int ui = 0; ui < r.nunits && ok; ++ui) {
          const Unit& u = r.u[ui];
          const CUtensorMap* map = maps[isA ? u.mapA : u.mapB];
          int kb, ke;
          split_range(r.splits, u, c.split, kb, ke);
          for (int q = 0; q < u.Q && ok; ++q) {
            const int z = isA ? c.b * u.a_zb + q * u.a_zq : c.b * u.b_zb + q * u.b_zq;
            for (int k0 = kb; k0 < ke; k0 += nki) {
              const int ngrp = ke - k0 < nki ? ke - k0 : nki;      // k-steps of this group
              if (jk < ngrp) {
                const int kk = k0 + jk;
                int st = stage + jk; uint32_t ph = phase;
                if (st >= p.nstages) { st -= p.nstages; ph ^= 1u; }
                if (!mbar_wait(empty0 + 8u * st, ph ^ 1u, abort_flag, p.spin_cap)) { ok = false; break; }
                const uint32_t fb_local = full0 + 8u * st;
                // completion is signalled on the LEADER's barrier; the leader expects both CTAs' bytes
                const uint32_t fb = CG == 2 ? mapa_rank(fb_local, 0) : fb_local;
                const uint32_t sa = tiles_sa + (uint32_t)st * stage_bytes, sb = sa + a_bytes;
                if (isA && rank == 0 && box == 0) {
                  if (p.debug & kAidMask & 1) mbar_arrive(fb_local); else mbar_expect_tx(fb_local, tx);
                }
                if (!(p.debug & kAidMask & 1) && !skip && box < nb) {
                  auto load = [&](uint32_t dst, int x, int y) {
                    if (CG == 2) tma_load_3d_pair(dst, map, x, y, z, fb); else tma_load_3d(dst, map, x, y, z, fb);
                  };
                  if (isA) {
                    if (!p.a_mn) load(sa, u.ak0 + kk * BK, m0);
                    else load(sa + box * (64 * BK * 2), u.am0 + m0 + box * 64, u.ak0 + kk * BK);
                  } else {
                    if (!p.b_mn) load(sb, u.bk0 + kk * BK, u.bn0 + n0);
                    else load(sb + box * (64 * BK * 2), u.bn0 + n0 + box * 64, u.bk0 + kk * BK);
                  }
                }
              }
              issued += ngrp;
              stage += ngrp;
              if (stage >= p.nstages) { stage -= p.nstages; phase ^= 1u; }
            }
          }
        }
      }
      if (!ok && lane == 0) {
        // gave up: flag it, then wait (bounded) for the copies still in flight
        // (the pair's copies complete on the leader's barriers; the peer just gives them time)
        *abort_flag = 1;
        atomicExch(p.status, 1u);
        const int pending = issued < p.nstages ? (int)issued : p.nstages;
        int s = stage; uint32_t ph = phase;
        for (int k = 0; k < pending; ++k) {
          if (--s < 0) { s = p.nstages - 1; ph ^= 1u; }
          for (uint32_t it = 0; it < (p.spin_cap < (1u << 20) ? p.spin_cap : (1u << 20)); ++it)
            if (rank == 0 && mbar_try(full0 + 8u * s, ph)) break;
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader CTA only when CG == 2)
    if (rank == 0) {                              // the whole warp walks the schedule, one elected lane issues
      const uint32_t idesc0 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)p.a_mn << 15) | ((uint32_t)p.b_mn << 16) |
                              ((uint32_t)(BMT >> 4) << 24);
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      bool ok = true;
      // Descriptors differ from stage to stage and from MMA to MMA only in their 14-bit address field:
      // the constant part is built once and the loop adds 16-byte units to the low word.  The issuing
      // thread's instruction count per k-step is what bounds short contractions.
      const uint64_t a_const = p.a_mn ? make_desc(0, 64 * BK * 2, 1024) : make_desc(0, 16, 1024);
      const uint64_t b_const = p.b_mn ? make_desc(0, 64 * BK * 2, 1024) : make_desc(0, 16, 1024);
      const uint32_t a_hi = (uint32_t)(a_const >> 32), b_hi = (uint32_t)(b_const >> 32);
      const uint32_t a_k16 = (p.a_mn ? UMMA_K * 128 : UMMA_K * 2) >> 4, b_k16 = (p.b_mn ? UMMA_K * 128 : UMMA_K * 2) >> 4;
      const uint32_t stage16 = stage_bytes >> 4;
      const uint32_t a_lo0 = (uint32_t)a_const + (tiles_sa >> 4), b_lo0 = (uint32_t)b_const + ((tiles_sa + a_bytes) >> 4);
      uint32_t a_lo = a_lo0, b_lo = b_lo0;
      uint32_t full_bar = full0, empty_bar = empty0;
      for (int tile = worker; tile < p.tiles_total && ok; tile += nworkers) {
        const TileCoord c = decode_tile(p, tile);
        const Region& r = p.r[c.region];
        if (!mbar_wait_warp(tempty0 + 8u * acc, acc_phase ^ 1u, abort_flag, p.spin_cap)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * kAccCols);
        const uint32_t idesc = idesc0 | ((uint32_t)(tile_cols(p, r, c.nt, CG) >> 3) << 17);
        uint32_t accumulate = 0;
        for (int ui = 0; ui < r.nunits && ok; ++ui) {
          const Unit& u = r.u[ui];
          int kb, ke;
          split_range(r.splits, u, c.split, kb, ke);
          for (int q = 0; q < u.Q && ok; ++q) {
            for (int kk = kb; kk < ke; ++kk) {
              if (!mbar_wait_warp(full_bar, phase, abort_flag, p.spin_cap)) { ok = false; break; }
              tc_fence_after();
              if (elect_one()) {
#pragma unroll
                for (int k = 0; k < BK / UMMA_K; ++k) {
                  const uint64_t ad = ((uint64_t)a_hi << 32) | (a_lo + (uint32_t)k * a_k16);
                  const uint64_t bd = ((uint64_t)b_hi << 32) | (b_lo + (uint32_t)k * b_k16);
                  if (CG == 2) umma_bf16_pair(d_tmem, ad, bd, idesc, k == 0 ? accumulate : 1u);
                  else umma_bf16(d_tmem, ad, bd, idesc, k == 0 ? accumulate : 1u);
                }
                // frees the stage (in both CTAs) once these MMAs have read it
                if (CG == 2) umma_commit_pair(empty_bar); else umma_commit(empty_bar);
              }
              accumulate = 1;
              a_lo += stage16; b_lo += stage16; full_bar += 8u; empty_bar += 8u;
              if (++stage == p.nstages) {
                stage = 0; phase ^= 1u;
                a_lo = a_lo0; b_lo = b_lo0; full_bar = full0; empty_bar = empty0;
              }
            }
          }
        }
        if (ok && elect_one()) {                    // accumulator complete (in both CTAs)
          if (CG == 2) umma_commit_pair(tfull0 + 8u * acc); else umma_commit(tfull0 + 8u * acc);
        }
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
      if (!ok && lane == 0) { *abort_flag = 1; atomicExch(p.status, 2u); }
    }
  } else if (warp <= 5) {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    const int quarter = warp & 3;                 // TMEM lanes [32*quarter, 32*quarter+32)
    int acc = 0; uint32_t acc_phase = 0;
    uint32_t slab = 0;
    bool ok = true;
    for (int tile = worker; tile < p.tiles_total && ok; tile += nworkers) {
      const TileCoord c = decode_tile(p, tile);
      const Region& r = p.r[c.region];
      // a tile whose contraction range is empty leaves the accumulator undefined: its value is 0
      int total_k = 0;
      for (int ui = 0; ui < r.nunits; ++ui) {
        int kb, ke;
        split_range(r.splits, r.u[ui], c.split, kb, ke);
        total_k += (ke - kb) * r.u[ui].Q;
      }
      if (!mbar_wait(tfull0 + 8u * acc, acc_phase, abort_flag, p.spin_cap)) { ok = false; break; }
      tc_fence_after();
      // Drain 64-byte-wide column slabs (32 bf16 / 16 fp32 columns): TMEM -> registers ->
      // swizzled staging buffer -> TMA store (coalesced; rows and columns outside the region's
      // extents are clipped by the tensor map).  Three buffers, one 128-thread barrier per slab.
      const int n0 = c.nt * p.BN;
      const int m0 = c.mt * BMT + (int)rank * BM;
      const int zc = c.split * r.batch + c.b;
      // where this tile's rows go: the region's own output, or - shared columns of a multi-GPU forward - the
      // receive slot of the GPU that owns these token rows, through its own map (row 0 = the owner's first token)
      const CUtensorMap* omap = cmaps[c.region];
      int om0 = m0;
      if (p.push_slice > 0 && c.region == 0) {
        const int owner = m0 / p.push_slice;
        omap = &pm.m[owner];
        om0 = m0 - owner * p.push_slice;
      }
      const int sub = p.out_f32 ? 16 : 32;
      const int rr = quarter * 32 + lane;                 // row of the tile this thread holds
      const uint32_t sw = (uint32_t)((rr >> 1) & 3);      // 64-byte swizzle: chunk ^= (row / 2) % 4
      if (p.out_transposed) {
        // swap-AB (decode): TMEM lane = output channel, column = token.  For a fixed token the 32
        // lanes of a warp hold 32 consecutive channels: plain 128-byte coalesced stores.
        const long long chan = (long long)m0 + rr;
        for (int cc = 0; cc < p.BN && n0 + cc < r.N; cc += 32) {
          uint32_t v[32];
          tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * kAccCols + cc), v);
          tmem_ld_wait();
          if (chan < r.M) {
            float* dst = r.out_t + ((long long)zc * r.N + n0 + cc) * p.out_t_ld + chan;
            const int ntok = r.N - (n0 + cc);           // tokens left from this column on (>= 1)
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              if (e < ntok) *dst = total_k == 0 ? 0.f : __uint_as_float(v[e]);
              dst += p.out_t_ld;
            }
          }
        }
      } else
      for (int cc = 0; cc < p.BN && n0 + cc < r.N && !(p.debug & kAidMask & 2); cc += sub) {
        uint32_t v[32];
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * kAccCols + cc);
        if (p.out_f32) tmem_ld16(taddr, v); else tmem_ld32(taddr, v);
        tmem_ld_wait();
        if (total_k == 0) {
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] = 0u;
        }
        if (p.out_f32 && r.scale != 0.f && r.scale != 1.f) {
#pragma unroll
          for (int e = 0; e < 16; ++e) v[e] = __float_as_uint(__uint_as_float(v[e]) * r.scale);
        }
        const uint32_t buf = smem_u32(cstage + (size_t)(slab % 3) * kCBuf);
        const uint32_t rowaddr = buf + (uint32_t)rr * 64u;
        if (p.debug & kAidMask & 32) { ++slab; continue; }
        if (p.out_f32) {
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4)
            sts128(rowaddr + (((uint32_t)q4 ^ sw) << 4), v[4 * q4], v[4 * q4 + 1], v[4 * q4 + 2], v[4 * q4 + 3]);
        } else {
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            uint32_t w[4];
#pragma unroll
            for (int q2 = 0; q2 < 4; ++q2) {
              __nv_bfloat162 bb = __floats2bfloat162_rn(__uint_as_float(v[8 * q4 + 2 * q2]), __uint_as_float(v[8 * q4 + 2 * q2 + 1]));
              w[q2] = *reinterpret_cast<uint32_t*>(&bb);
            }
            sts128(rowaddr + (((uint32_t)q4 ^ sw) << 4), w[0], w[1], w[2], w[3]);
          }
        }
        if (p.debug & kAidMask & 16) { ++slab; continue; }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        if (!(p.debug & kAidMask & 64)) epi_barrier();
        if (warp == 2 && lane == 0 && !(p.debug & kAidMask & 128)) {
          tma_store_3d(omap, n0 + cc, om0, zc, buf);
          bulk_commit();
          bulk_wait_read1();     // the store before this one has finished reading its buffer
        }
        ++slab;
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {           // this CTA's part of the accumulator is drained: tell the MMA issuer
        if (CG == 2) mbar_arrive_cluster(mapa_rank(tempty0 + 8u * acc, 0)); else mbar_arrive(tempty0 + 8u * acc);
      }
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
    if (warp == 2 && lane == 0) bulk_wait_all();   // all output stores of this CTA are complete
    if (!ok && lane == 0) { *abort_flag = 1; atomicExch(p.status, 3u); }
  }

  tc_fence_before();
  __syncthreads();
  if (CG == 2) cluster_sync();   // the leader's MMAs read the peer's shared memory: leave together
  if (warp == 1) {
    tc_fence_after();
    if (CG == 2)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    else
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// out[i] = sum_s part[s][i], s ascending (deterministic split-K reduction)
__global__ void __launch_bounds__(256) splitk_reduce_kernel(const float4* __restrict__ part, float4* __restrict__ out,
                                                            long long n4, int splits) {
  pdl_wait();
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (long long)gridDim.x * blockDim.x) {
    float4 s = part[i];
    for (int k = 1; k < splits; ++k) {
      const float4 v = part[(long long)k * n4 + i];
      s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
    }
    out[i] = s;
  }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(f);
  });
  return fn;
}

// Tensor [d2][d1][d0] (d0 contiguous) with row pitch ld1 and plane pitch ld2 (elements);
// box = (b0, b1, 1); out-of-range elements read as zero and are not written.
bool make_map(CUtensorMap* m, const void* base, long long d0, long long d1, long long d2, long long ld1, long long ld2,
              int b0, int b1, bool f32 = false, CUtensorMapSwizzle swz = CU_TENSOR_MAP_SWIZZLE_128B) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  if (d0 < 1 || d1 < 1 || d2 < 1) return false;
  const cuuint64_t es_bytes = f32 ? 4 : 2;
  cuuint64_t dims[3] = {(cuuint64_t)d0, (cuuint64_t)d1, (cuuint64_t)d2};
  cuuint64_t strides[2] = {(cuuint64_t)ld1 * es_bytes, (cuuint64_t)ld2 * es_bytes};
  cuuint32_t box[3] = {(cuuint32_t)b0, (cuuint32_t)b1, 1};
  cuuint32_t es[3] = {1, 1, 1};
  CUresult r = fn(m, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3,
                  const_cast<void*>(base), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Output map: slabs of 64 bytes x 128 rows, 64-byte swizzle (matches the epilogue's staging layout).
bool make_cmap(CUtensorMap* m, const void* base, long long d0, long long d1, long long d2, long long ld1,
               long long ld2, bool f32) {
  return make_map(m, base, d0, d1, d2, ld1, ld2, f32 ? 16 : 32, BM, f32, CU_TENSOR_MAP_SWIZZLE_64B);
}

// ---- tile configuration ------------------------------------------------------------------
// A small cost model picks the tile width BN, the CTA-pair mode cg and (weight gradient) the
// split-K factor.  Unit of time: one 128 x 256 x 64 MMA step at full tensor rate (~0.2 us).
//  * a k-step of a 128 x BN (x cg) tile costs BN/256, stretched when the operand bytes a CTA
//    pulls from L2 per flop, proportional to (128 + BN/cg) / BN, exceed what L2 delivers
//    (measured: 128 x 256 tiles with cg = 1 run at ~0.73 of the tensor rate);
//  * the epilogue of a tile (~10 units at BN = 256) overlaps the next tile's main loop, so a
//    tile costs max(main loop, epilogue) plus a fixed hand-off (larger across a CTA pair);
//  * tiles are dealt round-robin to 148 / cg workers: few tiles cost whole waves;
//  * split-K partials are written and read back once (fp32).
struct RegionShape { int M, N, batch, ksteps; };
struct TileCfg { int bn, cg, splits; double cost; };

double estimate_cost(const RegionShape* r, int nr, int bn, int cg, int splits, double out_bytes, bool b_n_major) {
  const double workers = 148.0 / cg;
  const double step = (bn / 256.0) * fmax(1.0, 0.92 * (128.0 + (double)bn / cg) / bn);
  const double epi = 10.0 * bn / 256.0;
  const double handoff = cg == 2 ? 3.5 : 2.0;
  double total = 0, ntiles = 0;
  for (int i = 0; i < nr; ++i) {
    if (r[i].M <= 0 || r[i].N <= 0) continue;
    const double rows = (double)((r[i].M + 128 * cg - 1) / (128 * cg)) * r[i].batch * splits;
    const double ks = (double)((r[i].ksteps + splits - 1) / splits);
    const int full = r[i].N / bn, rest = r[i].N % bn;
    total += rows * full * (fmax(ks * step, epi) + handoff);
    ntiles += rows * full;
    if (rest) {   // the last, ragged tile: an N-major B operand is narrowed to whole 64-column chunks
      const double w = b_n_major ? (double)((rest + 64 * cg - 1) / (64 * cg) * (64 * cg)) / bn : 1.0;
      total += rows * (fmax(ks * step * w, epi * w) + handoff);
      ntiles += rows;
    }
  }
  if (ntiles == 0) return 0;
  double t = fmax(total / workers, ceil(ntiles / workers) * (total / ntiles));
  if (splits > 1) t += 2.0 * splits * out_bytes / 6.4e12 / 0.2e-6;
  return t;
}

TileCfg pick_tile(const RegionShape* r, int nr, bool b_n_major, int max_splits, double out_bytes) {
#ifdef CAAT_MEASUREMENT_AIDS
  static const int max_cg = [] { const char* e = getenv("CAAT_TC_CG"); return e && atoi(e) == 1 ? 1 : 2; }();
  // CAAT_TC_BN / CAAT_TC_CGF pin the tile width / the pair mode instead of the model's choice
  static const int force_bn = [] { const char* e = getenv("CAAT_TC_BN"); return e ? atoi(e) : 0; }();
  static const int force_cg = [] { const char* e = getenv("CAAT_TC_CGF"); return e ? atoi(e) : 0; }();
#else
  constexpr int max_cg = 2, force_bn = 0, force_cg = 0;
#endif
  TileCfg best{256, 1, 1, -1.0};
  int min_ksteps = 1 << 30;
  for (int i = 0; i < nr; ++i)
    if (r[i].M > 0 && r[i].N > 0 && r[i].ksteps < min_ksteps) min_ksteps = r[i].ksteps;
  for (int cg = 1; cg <= max_cg; ++cg) {
    bool ok = true;
    int nmin = 1 << 30;
    for (int i = 0; i < nr; ++i) {
      if (r[i].M <= 0 || r[i].N <= 0) continue;
      if (cg == 2 && r[i].M < 256) ok = false;          // a pair needs two row blocks
      if (r[i].N < nmin) nmin = r[i].N;
    }
    if (!ok) continue;
    if (force_cg && cg != force_cg && !(force_cg == 2 && cg == 1 && max_cg == 2)) continue;
    const int step = b_n_major ? 64 * cg : 32 * cg;    // N-major B: whole 64-column chunks per CTA
    for (int bn = 256; bn >= 64 * cg; bn -= step) {
      if (force_bn && bn != force_bn && force_bn % step == 0 && force_bn >= 64 * cg) continue;
      for (int splits = 1; splits <= max_splits; ++splits) {
        if (splits > 1 && min_ksteps / splits < 8) break;
        const double c = estimate_cost(r, nr, bn, cg, splits, out_bytes, b_n_major);
        if (best.cost < 0 || c < best.cost * 0.995) best = TileCfg{bn, cg, splits, c};
      }
    }
  }
  return best;
}

cudaError_t launch(const CUtensorMap maps[4], const CUtensorMap cmaps[2], Params& p, int kind, cudaStream_t st,
                   const PeerMaps* peer_maps = nullptr) {
  const LaunchLimits lim = effective_limits();
  const int stage_bytes = BM * BK * 2 + (p.BN / p.cg) * BK * 2;
  const int budget = lim.gemm_smem > 0 && lim.gemm_smem < 227 * 1024 ? lim.gemm_smem : 227 * 1024;
  int nst = (budget - 2048 - 3 * kCBuf) / stage_bytes;
  if (nst > kMaxStages) nst = kMaxStages;
  if (nst < 2) return cudaErrorInvalidConfiguration;
  p.nstages = nst;
  const size_t smem = (size_t)nst * stage_bytes + 3 * kCBuf + 1024 /*alignment slack*/ + (2 * nst + 4) * 8 + 16;
  static bool attr_set[64] = {};      // the attribute belongs to the device's copy of the kernel: once per device
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (std::lock_guard<std::mutex> lock(host_cache_mutex()); !attr_set[dev]) {
    cudaError_t e = cudaFuncSetAttribute(tc_gemm_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_gemm_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    attr_set[dev] = true;
  }
  p.status = device_status_word();
  if (!p.status) return cudaErrorUnknown;
  static const int dbg = [] { const char* e = getenv("CAAT_TC_DEBUG"); return e ? atoi(e) : 0; }();
  p.debug = dbg & kAidMask;
  static const uint32_t cap_env = [] { const char* e = getenv("CAAT_TC_SPINCAP"); return e ? (uint32_t)atoi(e) : 0u; }();
  p.spin_cap = cap_env >= 1024 ? cap_env : kSpinCap;
  static const bool verbose = getenv("CAAT_TC_VERBOSE") != nullptr;
  if (verbose)
    fprintf(stderr, "[caat tc] kind=%d BN=%d cg=%d splits=%d stages=%d tiles=%d (r0 M=%d N=%d b=%d)\n", kind, p.BN, p.cg,
            p.splits, nst, p.tiles_total, p.r[0].M, p.r[0].N, p.r[0].batch);
  int workers_max = sm_count() / p.cg;
  if (lim.gemm_workers > 0 && lim.gemm_workers / p.cg < workers_max) workers_max = lim.gemm_workers / p.cg;
  const int workers = p.tiles_total < workers_max ? p.tiles_total : workers_max;
  if (workers < 1) return cudaSuccess;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)(workers * p.cg));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2] = {};
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)p.cg;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 2 : 1;
  LaunchScope scope(kind, st);
  static const PeerMaps no_peers{};
  const PeerMaps& pm = peer_maps ? *peer_maps : no_peers;
  if (p.cg == 2)
    return cudaLaunchKernelEx(&cfg, tc_gemm_kernel<2>, maps[0], maps[1], maps[2], maps[3], cmaps[0], cmaps[1], pm, p);
  return cudaLaunchKernelEx(&cfg, tc_gemm_kernel<1>, maps[0], maps[1], maps[2], maps[3], cmaps[0], cmaps[1], pm, p);
}

void finish_tiles(Params& p) {
  for (int g = 0; g < p.nregions; ++g) {
    Region& r = p.r[g];
    r.mtiles = (r.M + BM * p.cg - 1) / (BM * p.cg);
    r.ntiles = (r.N + p.BN - 1) / p.BN;
    if (r.splits < 1) r.splits = p.splits < 1 ? 1 : p.splits;
  }
  p.tiles_r0 = p.r[0].mtiles * p.r[0].ntiles * p.r[0].batch * p.r[0].splits;
  p.tiles_total = p.tiles_r0 + (p.nregions > 1 ? p.r[1].mtiles * p.r[1].ntiles * p.r[1].batch * p.r[1].splits : 0);
}

}  // namespace

bool tc_gemm_usable(const caat_ctx* ctx, int K_r) {
  return ctx->dtype == CAAT_BF16 && !ctx->force_simt && K_r % 8 == 0 && ctx->S % 8 == 0 && ctx->h % 8 == 0;
}

// ---- forward: zs[T,S] = sum_m Y[m] W[m][:S]^T ; zp[m][T,h-S] = Y[m] W[m][S:]^T
cudaError_t launch_tc_forward(const RowparShapes& s, const void* Y, const void* W, void* zs, void* zp,
                              cudaStream_t st, const PushTarget* push) {
  CUtensorMap maps[4], cmaps[2];
  PeerMaps pmaps{};
  Params p{};
  const int n_sh = s.S, n_pr = s.h - s.S;
  const int ksteps = (s.K_r + BK - 1) / BK;
  {
    const RegionShape rs[2] = {{s.T, n_sh, 1, ksteps * s.t}, {s.T, n_pr, s.t, ksteps}};
    const TileCfg c = pick_tile(rs, 2, false, 1, 0.0);
    p.BN = c.bn; p.cg = c.cg;
  }
  if (!make_map(&maps[0], Y, s.K_r, s.T, s.t, s.K_r, (long long)s.T * s.K_r, BK, BM)) return cudaErrorInvalidValue;
  if (!make_map(&maps[1], W, s.K_r, s.h, s.t, s.K_r, (long long)s.h * s.K_r, BK, p.BN / p.cg)) return cudaErrorInvalidValue;
  maps[2] = maps[0];
  maps[3] = maps[1];
  p.a_mn = 0; p.b_mn = 0; p.out_f32 = 0; p.splits = 1;
  int g = 0;
  if (n_sh > 0) {
    Region& r = p.r[g++];
    r.nunits = 1;
    r.u[0] = Unit{0, 1, 0, 0, 0, 0, /*a_zb*/ 0, /*a_zq*/ 1, /*b_zb*/ 0, /*b_zq*/ 1, s.t, ksteps};
    r.M = s.T; r.N = n_sh; r.batch = 1; r.b_slowest = 0;
    if (!make_cmap(&cmaps[g - 1], zs, n_sh, s.T, 1, s.S_hi, (long long)s.T * s.S_hi, false)) return cudaErrorInvalidValue;
  }
  if (n_pr > 0) {
    Region& r = p.r[g++];
    r.nunits = 1;
    r.u[0] = Unit{0, 1, 0, 0, 0, s.S, 1, 0, 1, 0, 1, ksteps};
    r.M = s.T; r.N = n_pr; r.batch = s.t; r.b_slowest = 1;
    if (!make_cmap(&cmaps[g - 1], static_cast<__nv_bfloat16*>(zp) + (s.S - s.S_lo), n_pr, s.T, s.t, s.P,
                   (long long)s.T * s.P, false))
      return cudaErrorInvalidValue;
  }
  if (g == 1) cmaps[1] = cmaps[0];
  p.nregions = g;
  if (push && n_sh > 0) {
    // shared tiles go to the owners' receive slots: slot `rank` of GPU q is [slice, S] 16-bit elements; the map of
    // owner q covers only the tokens q really owns, so rows past the end of a ragged last slice are clipped
    if (push->world < 1 || push->world > CAAT_MAX_PEERS || push->slice % (BM * p.cg) != 0) return cudaErrorInvalidValue;
    for (int q = 0; q < push->world; ++q) {
      long long rows = (long long)s.T - (long long)q * push->slice;
      if (rows > push->slice) rows = push->slice;
      if (rows < 1) { pmaps.m[q] = cmaps[0]; continue; }     // owns no token: never addressed
      __nv_bfloat16* slot = static_cast<__nv_bfloat16*>(push->recv[q]) + (size_t)push->rank * push->slice * n_sh;
      if (!make_cmap(&pmaps.m[q], slot, n_sh, rows, 1, n_sh, (long long)push->slice * n_sh, false)) return cudaErrorInvalidValue;
    }
    p.push_slice = push->slice;
  }
  finish_tiles(p);
  return launch(maps, cmaps, p, CAAT_K_TC_FORWARD, st, push && n_sh > 0 ? &pmaps : nullptr);
}

// ---- decode forward (few tokens): zt[m][i][l] = sum_k W[m][l][k] Y[m][i][k], fp32, for ALL channels.
// The operands are swapped (weights on the 128-row side, tokens on the narrow side) so that a tile
// streams 128 x K_r weights however few tokens there are; every (rank, 128-channel block) is a tile,
// which spreads the weight stream over all SMs.  The rank sum of the shared channels is left to the
// row kernel (the partials are tiny at these token counts).
int tc_decode_splits(int K_r, int K_r_min, int T) {
  // Work items are (rank, 128-channel block, split).  Splitting the longer layer's contraction until its
  // items are about as long as the shorter layer's makes the round-robin deal even; the fp32 partial
  // planes this adds (t * splits * T * h * 4 bytes) are kept near a tenth of the layer's weight bytes.
  const int ks = (K_r + BK - 1) / BK, ks_min = (K_r_min + BK - 1) / BK;
  int sp = (ks + ks_min / 2) / (ks_min > 0 ? ks_min : 1);
  const int cap_traffic = K_r / (20 * T);
  if (sp > cap_traffic) sp = cap_traffic;
  if (sp > kDecodeMaxSplits) sp = kDecodeMaxSplits;
  if (sp > ks / 2) sp = ks / 2;
  return sp < 1 ? 1 : sp;
}

cudaError_t launch_tc_forward_decode(int t, int T, int h, const DecodeProblem* pr, int n, cudaStream_t st) {
  if (n < 1 || n > 2) return cudaErrorInvalidValue;
  CUtensorMap maps[4], cmaps[2];
  Params p{};
  p.BN = (T + 31) / 32 * 32;
  if (p.BN > 256) return cudaErrorInvalidValue;
  p.cg = 1;
  p.a_mn = 0; p.b_mn = 0; p.out_f32 = 1; p.splits = 1;
  p.out_transposed = 1; p.out_t_ld = h;
  // longer contraction first: round-robin dealing then fills the tail with the short items
  int order[2] = {0, 1};
  if (n == 2 && pr[1].K_r > pr[0].K_r) { order[0] = 1; order[1] = 0; }
  for (int g = 0; g < n; ++g) {
    const DecodeProblem& q = pr[order[g]];
    if (!make_map(&maps[2 * g], q.W, q.K_r, h, t, q.K_r, (long long)h * q.K_r, BK, BM)) return cudaErrorInvalidValue;
    if (!make_map(&maps[2 * g + 1], q.Y, q.K_r, T, t, q.K_r, (long long)T * q.K_r, BK, p.BN)) return cudaErrorInvalidValue;
    Region& r = p.r[g];
    r.nunits = 1;
    r.u[0] = Unit{2 * g, 2 * g + 1, 0, 0, 0, 0, 1, 0, 1, 0, 1, (q.K_r + BK - 1) / BK};
    r.M = h; r.N = T; r.batch = t; r.b_slowest = 1;
    r.out_t = q.zt;
    r.splits = q.splits;
  }
  if (n == 1) { maps[2] = maps[0]; maps[3] = maps[1]; }
  cmaps[0] = maps[0]; cmaps[1] = maps[0];          // unused: the epilogue stores directly
  p.nregions = n;
  finish_tiles(p);
  return launch(maps, cmaps, p, CAAT_K_TC_FORWARD, st);
}

// ---- dgrad: dY[m] = gs W[m][:S] + (alpha gp[m]) W[m][S:]
// pv describes where the private gradient lives and what still multiplies it (see PrivOperand); when
// pv.alpha != 1, w_scaled ([t, h, K_r], only rows >= S are used) must hold alpha times the private rows of W.
cudaError_t launch_tc_dgrad(const RowparShapes& s, const void* gs, const PrivOperand& pv, const void* W, void* dY,
                            void* w_scaled, bool w_scaled_ready, cudaStream_t st) {
  CUtensorMap maps[4], cmaps[2];
  Params p{};
  {
    const RegionShape rs[1] = {{s.T, s.K_r, s.t, (s.S + BK - 1) / BK + (s.h - s.S + BK - 1) / BK}};
    const TileCfg c = pick_tile(rs, 1, true, 1, 0.0);
    p.BN = c.bn; p.cg = c.cg;
  }
  const int n_sh = s.S, n_pr = s.h - s.S;
  // B = W[m] as [h rows (contraction)][K_r contiguous (N)]: N-major, boxes of 64 (N) x 64 (K)
  if (!make_map(&maps[1], W, s.K_r, s.h, s.t, s.K_r, (long long)s.h * s.K_r, 64, BK)) return cudaErrorInvalidValue;
  maps[3] = maps[1];
  if (n_pr > 0 && pv.alpha != 1.0f) {
    // sum_l (alpha g[l]) W[l][k] = sum_l g[l] (alpha W[l][k]): the private gradient is read as stored in dR,
    // the weights' private rows (the small operand) carry alpha; they were scaled by the launch before this one
    if (!w_scaled || !w_scaled_ready) return cudaErrorInvalidValue;
    if (!make_map(&maps[3], w_scaled, s.K_r, s.h, s.t, s.K_r, (long long)s.h * s.K_r, 64, BK)) return cudaErrorInvalidValue;
  }
  bool okA0 = n_sh > 0 ? make_map(&maps[0], gs, n_sh, s.T, 1, s.S_hi, (long long)s.T * s.S_hi, BK, BM) : true;
  bool okA1 = n_pr > 0 ? make_map(&maps[2], pv.ptr, pv.ld, s.T, s.t, pv.ld, (long long)s.T * pv.ld, BK, BM) : true;
  if (!okA0 || !okA1) return cudaErrorInvalidValue;
  if (n_sh == 0) maps[0] = maps[2];
  if (n_pr == 0) maps[2] = maps[0];
  p.a_mn = 0; p.b_mn = 1; p.out_f32 = 0; p.splits = 1;
  Region& r = p.r[0];
  int nu = 0;
  if (n_sh > 0) r.u[nu++] = Unit{0, 1, 0, 0, 0, 0, 0, 0, 1, 0, 1, (n_sh + BK - 1) / BK};
  if (n_pr > 0) r.u[nu++] = Unit{2, 3, pv.col0, 0, s.S, 0, 1, 0, 1, 0, 1, (n_pr + BK - 1) / BK};
  r.nunits = nu;
  r.M = s.T; r.N = s.K_r; r.batch = s.t; r.b_slowest = 1; r.scale = 1.0f;
  if (!make_cmap(&cmaps[0], dY, s.K_r, s.T, s.t, s.K_r, (long long)s.T * s.K_r, false)) return cudaErrorInvalidValue;
  cmaps[1] = cmaps[0];
  p.nregions = 1;
  finish_tiles(p);
  return launch(maps, cmaps, p, CAAT_K_TC_DGRAD, st);
}

static TileCfg wgrad_cfg(const RowparShapes& s) {
  const int ksteps = (s.T + BK - 1) / BK;
  const RegionShape rs[2] = {{s.S, s.K_r, s.t, ksteps}, {s.h - s.S, s.K_r, s.t, ksteps}};
  return pick_tile(rs, 2, true, 16, (double)s.t * s.h * s.K_r * sizeof(float));
}

size_t tc_wgrad_splitk_bytes(const RowparShapes& s) {
  const int splits = wgrad_cfg(s).splits;
  return splits > 1 ? (size_t)splits * s.t * s.h * s.K_r * sizeof(float) : 0;
}

// ---- wgrad: dW[m][:S] = gs^T Y[m] ; dW[m][S:] = alpha gp[m]^T Y[m]      (fp32 out; alpha in the epilogue)
cudaError_t launch_tc_wgrad(const RowparShapes& s, const void* gs, const PrivOperand& pv, const void* Y, float* dW,
                            void* splitk, size_t splitk_bytes, cudaStream_t st) {
  CUtensorMap maps[4], cmaps[2];
  Params p{};
  const TileCfg wc = wgrad_cfg(s);
  p.BN = wc.bn; p.cg = wc.cg;
  const int n_sh = s.S, n_pr = s.h - s.S;
  const int splits = wc.splits;
  const long long dw_elems = (long long)s.t * s.h * s.K_r;
  if (splits > 1 && splitk_bytes < (size_t)splits * dw_elems * sizeof(float)) return cudaErrorInvalidValue;
  // A = dZt as [T rows (contraction)][channels contiguous (M)]: M-major, boxes of 64 (M) x 64 (K)
  bool okA0 = n_sh > 0 ? make_map(&maps[0], gs, n_sh, s.T, 1, s.S_hi, (long long)s.T * s.S_hi, 64, BK) : true;
  bool okA1 = n_pr > 0 ? make_map(&maps[2], pv.ptr, pv.ld, s.T, s.t, pv.ld, (long long)s.T * pv.ld, 64, BK) : true;
  // B = Y[m] as [T rows (contraction)][K_r contiguous (N)]: N-major
  if (!okA0 || !okA1 || !make_map(&maps[1], Y, s.K_r, s.T, s.t, s.K_r, (long long)s.T * s.K_r, 64, BK))
    return cudaErrorInvalidValue;
  if (n_sh == 0) maps[0] = maps[2];
  if (n_pr == 0) maps[2] = maps[0];
  maps[3] = maps[1];
  p.a_mn = 1; p.b_mn = 1; p.out_f32 = 1; p.splits = splits;
  const int ksteps = (s.T + BK - 1) / BK;
  float* out = splits > 1 ? static_cast<float*>(splitk) : dW;
  int g = 0;
  if (n_sh > 0) {
    Region& r = p.r[g++];
    r.nunits = 1;
    r.u[0] = Unit{0, 1, 0, 0, 0, 0, 0, 0, 1, 0, 1, ksteps};
    r.M = n_sh; r.N = s.K_r; r.batch = s.t; r.b_slowest = 0;   // the shared gradient panel serves all ranks at once
    r.scale = 1.0f;
    if (!make_cmap(&cmaps[g - 1], out, s.K_r, n_sh, (long long)s.t * splits, s.K_r, (long long)s.h * s.K_r, true))
      return cudaErrorInvalidValue;
  }
  if (n_pr > 0) {
    Region& r = p.r[g++];
    r.nunits = 1;
    r.u[0] = Unit{2, 1, 0, pv.col0, 0, 0, 1, 0, 1, 0, 1, ksteps};
    r.M = n_pr; r.N = s.K_r; r.batch = s.t; r.b_slowest = 1;
    r.scale = pv.alpha;
    if (!make_cmap(&cmaps[g - 1], out + (long long)s.S * s.K_r, s.K_r, n_pr, (long long)s.t * splits, s.K_r,
                   (long long)s.h * s.K_r, true))
      return cudaErrorInvalidValue;
  }
  if (g == 1) cmaps[1] = cmaps[0];
  p.nregions = g;
  finish_tiles(p);
  cudaError_t e = launch(maps, cmaps, p, CAAT_K_TC_WGRAD, st);
  if (e != cudaSuccess) return e;
  if (splits > 1) {
    const long long n4 = dw_elems / 4;   // K_r is a multiple of 8
    int blocks = (int)((n4 + 255) / 256);
    if (blocks > 148 * 8) blocks = 148 * 8;
    LaunchScope scope(CAAT_K_SPLITK_REDUCE, st);
    e = launch_pdl(splitk_reduce_kernel, dim3(blocks), dim3(256), 0, st, static_cast<const float4*>(splitk),
                   reinterpret_cast<float4*>(dW), n4, splits);
  }
  return e;
}

}  // namespace caat
