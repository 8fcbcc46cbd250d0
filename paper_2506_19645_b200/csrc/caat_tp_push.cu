// The exchange of the shared-channel slab between the GPUs of a tensor-parallel group over peer
// memory (Section 3: partial channel-reduce; Appendix D: reduce-scatter + all-gather; Section 4:
// 16-bit communication, 32-bit accumulation): plain peer stores and loads, flags raised with
// system-scope release stores and polled with bounded system-scope acquire loads.  No multicast,
// no library collective.
//
//   scatter   slab rows of owner q  ->  slot `rank` of q's receive buffer;  flag[q][rank] = epoch
//   reduce    wait flag[me][0..world);  sum my slots in fp32, order 0..world-1, round once;
//             result rows -> every GPU's slab;  flag[q][world + me] = epoch
//   wait      wait flag[me][world .. 2 world)
//
// A flag is raised once ALL blocks of the kernel have stored and fenced: every block bumps a
// counter in this GPU's own flag area and the last one raises the flags.  Waits poll with a sleep
// and give up after a limit: the kernel then raises the device status word, skips its work and
// returns (the host reads CAAT_ETIMEOUT); nothing spins without bound.
#include <cstdlib>

#include "caat_internal.h"

namespace caat {
namespace {

constexpr int kFlagWords = CAAT_TP_FLAG_BYTES / 4;
constexpr int kScatterCounter = 2 * CAAT_MAX_PEERS;      // word of this GPU's flag area: blocks of the scatter done
constexpr int kReduceCounter = 2 * CAAT_MAX_PEERS + 1;   // blocks of the reduce done
constexpr uint32_t kPollCap = 1u << 21;                  // polls of ~0.5 us: about a second
static_assert(2 * CAAT_MAX_PEERS + 2 <= kFlagWords, "flag area too small");

struct Peers {
  void* recv[CAAT_MAX_PEERS];
  void* slab[CAAT_MAX_PEERS];
  unsigned int* flags[CAAT_MAX_PEERS];
};

__device__ __forceinline__ unsigned int ld_acquire_sys(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_sys(unsigned int* p, unsigned int v) {
  asm volatile("st.release.sys.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Threads 0..n-1 of the block each wait for one flag to reach `epoch`; the block-uniform result is true
// when all arrived.  On a time-out the status word is raised.
__device__ bool wait_flags(const unsigned int* flags, int n, unsigned int epoch, uint32_t cap, unsigned int* status) {
  __shared__ int bad;
  if (threadIdx.x == 0) bad = 0;
  __syncthreads();
  if ((int)threadIdx.x < n) {
    bool ok = false;
    for (uint32_t it = 0; it < cap; ++it) {
      if ((int)(ld_acquire_sys(flags + threadIdx.x) - epoch) >= 0) { ok = true; break; }
      __nanosleep(200);
    }
    if (!ok) { atomicExch(&bad, 1); atomicExch(status, 5u); }
  }
  __syncthreads();
  return bad == 0;
}

// After all of this block's peer stores: fence, count the block, and let the last block raise `epoch` on
// word `word` of every peer's flag area.
__device__ void signal_when_all_blocks_done(unsigned int* counter, const Peers& pr, int world, int word, unsigned int epoch) {
  __threadfence_system();
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned int done = atomicAdd(counter, 1u);
    if (done == gridDim.x - 1) {
      *counter = 0;                       // ready for the next launch on this stream
      __threadfence_system();
      for (int q = 0; q < world; ++q) st_release_sys(pr.flags[q] + word, epoch);
    }
  }
}

__global__ void __launch_bounds__(256) tp_scatter_kernel(const uint4* __restrict__ slab, Peers pr, int T, int S8, int slice,
                                                         int world, int rank, unsigned int epoch) {
  pdl_wait();
  const long long total = (long long)T * S8;
  for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v < total; v += (long long)gridDim.x * blockDim.x) {
    const int i = (int)(v / S8), c = (int)(v - (long long)i * S8);
    const int q = i / slice;
    uint4* dst = static_cast<uint4*>(pr.recv[q]) + ((size_t)rank * slice + (i - q * slice)) * S8 + c;
    *dst = slab[v];
  }
  signal_when_all_blocks_done(pr.flags[rank] + kScatterCounter, pr, world, rank, epoch);
}

// The forward GEMM stored the tiles itself: only the flags are left to raise (the GEMM has completed: this kernel
// follows it on the stream).
__global__ void tp_signal_kernel(Peers pr, int world, int rank, unsigned int epoch) {
  pdl_wait();
  __threadfence_system();
  if ((int)threadIdx.x < world) st_release_sys(pr.flags[threadIdx.x] + rank, epoch);
}

__device__ __forceinline__ void add8(float (&acc)[8], const uint4& r) {
  const unsigned w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    acc[2 * q] += __uint_as_float(w[q] << 16);
    acc[2 * q + 1] += __uint_as_float(w[q] & 0xffff0000u);
  }
}

__global__ void __launch_bounds__(256) tp_reduce_gather_kernel(Peers pr, int T, int S8, int slice, int world, int rank,
                                                               unsigned int epoch, uint32_t cap, unsigned int* status) {
  pdl_wait();
  const bool ok = wait_flags(pr.flags[rank], world, epoch, cap, status);
  const int r0 = rank * slice;
  int nrows = T - r0;
  if (nrows > slice) nrows = slice;
  if (ok && nrows > 0) {
    const uint4* mine = static_cast<const uint4*>(pr.recv[rank]);
    const long long total = (long long)nrows * S8;
    for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v < total; v += (long long)gridDim.x * blockDim.x) {
      float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      for (int q = 0; q < world; ++q) add8(acc, mine[(size_t)q * slice * S8 + v]);      // fp32, sources in order
      unsigned w[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        __nv_bfloat162 b = __floats2bfloat162_rn(acc[2 * q], acc[2 * q + 1]);
        w[q] = *reinterpret_cast<unsigned*>(&b);
      }
      const uint4 out = make_uint4(w[0], w[1], w[2], w[3]);
      for (int q = 0; q < world; ++q) static_cast<uint4*>(pr.slab[q])[(size_t)r0 * S8 + v] = out;   // the all-gather
    }
  }
  // a GPU that gave up raises nothing: its peers' waits run out too, and every host reads the time-out
  if (ok) signal_when_all_blocks_done(pr.flags[rank] + kReduceCounter, pr, world, world + rank, epoch);
}

__global__ void tp_wait_kernel(const unsigned int* flags, int n, unsigned int epoch, uint32_t cap, unsigned int* status) {
  pdl_wait();
  wait_flags(flags, n, epoch, cap, status);
}

uint32_t poll_cap() {
  static const uint32_t cap = [] { const char* e = getenv("CAAT_TP_POLLCAP"); return e ? (uint32_t)atoi(e) : 0u; }();
  return cap >= 16 ? cap : kPollCap;
}

int slice_rows(int tokens, int world) {
  const int s = (tokens + world - 1) / world;
  return round_up(s, s >= 256 ? 256 : 8);
}

caat_status check_peers(const caat_ctx* ctx, const caat_peers* pe, Peers* out, bool need_recv, bool need_slab) {
  if (!ctx || !pe) return CAAT_EINVAL;
  if (pe->world < 1 || pe->world > CAAT_MAX_PEERS || pe->rank < 0 || pe->rank >= pe->world) return CAAT_EINVAL;
  if (ctx->dtype != CAAT_BF16 || ctx->S % kLayoutVec != 0 || ctx->S < 1) return CAAT_EUNSUPPORTED;
  for (int q = 0; q < pe->world; ++q) {
    if (!pe->flags[q] || (need_recv && !pe->recv[q]) || (need_slab && !pe->slab[q])) return CAAT_EINVAL;
    if ((reinterpret_cast<uintptr_t>(pe->flags[q]) & 15u) || (reinterpret_cast<uintptr_t>(pe->recv[q]) & 15u) ||
        (reinterpret_cast<uintptr_t>(pe->slab[q]) & 15u))
      return CAAT_EALIGN;
    out->recv[q] = pe->recv[q]; out->slab[q] = pe->slab[q]; out->flags[q] = pe->flags[q];
  }
  return CAAT_OK;
}

int grid_for(long long vectors) {
  long long b = (vectors + 255) / 256;
  const long long cap = (long long)sm_count() * 4;
  if (b > cap) b = cap;
  return b < 1 ? 1 : (int)b;
}

}  // namespace
}  // namespace caat

using namespace caat;

extern "C" {

caat_status caat_tp_exchange_bytes(const caat_ctx* ctx, caat_layer layer, int tokens, int world, size_t* recv_bytes,
                                   int* slice) {
  (void)layer;
  if (!ctx) return CAAT_EINVAL;
  if (tokens < 1) return CAAT_ESHAPE;
  if (world < 1 || world > CAAT_MAX_PEERS) return CAAT_EINVAL;
  if (ctx->dtype != CAAT_BF16 || ctx->S % kLayoutVec != 0) return CAAT_EUNSUPPORTED;
  const int sl = slice_rows(tokens, world);
  if (slice) *slice = sl;
  if (recv_bytes) *recv_bytes = align_up((size_t)world * sl * (ctx->S > 0 ? ctx->S : 8) * 2, 256);
  return CAAT_OK;
}

caat_status caat_tp_exchange_scatter(const caat_ctx* ctx, caat_layer layer, int tokens, int backward,
                                     const caat_peers* peers, unsigned int epoch, void* workspace, size_t workspace_bytes,
                                     void* cuda_stream) {
  Peers pr{};
  caat_status s = check_peers(ctx, peers, &pr, true, false);
  if (s != CAAT_OK) return s;
  size_t off = 0;
  int rows = 0, cols = 0;
  s = caat_tp_slab(ctx, layer, tokens, backward, &off, &rows, &cols);
  if (s != CAAT_OK) return s;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 15u) || workspace_bytes < off + (size_t)rows * cols * 2)
    return CAAT_EWORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int S8 = ctx->S / 8;
  LaunchScope scope(CAAT_K_TP_EXCHANGE, st);
  const cudaError_t e = launch_pdl(tp_scatter_kernel, dim3(grid_for((long long)tokens * S8)), dim3(256), 0, st,
                                   reinterpret_cast<const uint4*>(static_cast<const char*>(workspace) + off), pr, tokens, S8,
                                   slice_rows(tokens, peers->world), peers->world, peers->rank, epoch);
  return e == cudaSuccess ? CAAT_OK : cuda_fail(e);
}

caat_status caat_tp_exchange_reduce(const caat_ctx* ctx, caat_layer layer, int tokens, const caat_peers* peers,
                                    unsigned int epoch, void* cuda_stream) {
  (void)layer;
  Peers pr{};
  caat_status s = check_peers(ctx, peers, &pr, true, true);
  if (s != CAAT_OK) return s;
  if (tokens < 1) return CAAT_ESHAPE;
  unsigned int* status = device_status_word();
  if (!status) return cuda_fail(cudaErrorUnknown);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int S8 = ctx->S / 8, slice = slice_rows(tokens, peers->world);
  LaunchScope scope(CAAT_K_TP_EXCHANGE, st);
  const cudaError_t e = launch_pdl(tp_reduce_gather_kernel, dim3(grid_for((long long)slice * S8)), dim3(256), 0, st, pr, tokens,
                                   S8, slice, peers->world, peers->rank, epoch, poll_cap(), status);
  return e == cudaSuccess ? CAAT_OK : cuda_fail(e);
}

caat_status caat_tp_exchange_wait(const caat_ctx* ctx, const caat_peers* peers, unsigned int epoch, void* cuda_stream) {
  Peers pr{};
  caat_status s = check_peers(ctx, peers, &pr, false, false);
  if (s != CAAT_OK) return s;
  unsigned int* status = device_status_word();
  if (!status) return cuda_fail(cudaErrorUnknown);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  LaunchScope scope(CAAT_K_TP_EXCHANGE, st);
  const cudaError_t e = launch_pdl(tp_wait_kernel, dim3(1), dim3(32), 0, st,
                                   static_cast<const unsigned int*>(pr.flags[peers->rank] + peers->world), peers->world, epoch,
                                   poll_cap(), status);
  return e == cudaSuccess ? CAAT_OK : cuda_fail(e);
}

caat_status caat_tp_exchange(const caat_ctx* ctx, caat_layer layer, int tokens, int backward, const caat_peers* peers,
                             unsigned int epoch, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  caat_status s = caat_tp_exchange_scatter(ctx, layer, tokens, backward, peers, epoch, workspace, workspace_bytes, cuda_stream);
  if (s != CAAT_OK) return s;
  s = caat_tp_exchange_reduce(ctx, layer, tokens, peers, epoch, cuda_stream);
  if (s != CAAT_OK) return s;
  return caat_tp_exchange_wait(ctx, peers, epoch, cuda_stream);
}

caat_status caat_tp_forward_local_push(const caat_ctx* ctx, caat_layer layer, int tokens, const void* Y, const void* W,
                                       const caat_peers* peers, unsigned int epoch, void* workspace, size_t workspace_bytes,
                                       void* cuda_stream) {
  Peers pr{};
  caat_status s = check_peers(ctx, peers, &pr, true, false);
  if (s != CAAT_OK) return s;
  if (layer != CAAT_ATTN_OUT && layer != CAAT_MLP_DOWN) return CAAT_EINVAL;
  if (tokens < 1) return CAAT_ESHAPE;
  if (!Y || !W) return CAAT_EINVAL;
  if ((reinterpret_cast<uintptr_t>(Y) & 15u) || (reinterpret_cast<uintptr_t>(W) & 15u)) return CAAT_EALIGN;
  const int K_r = (layer == CAAT_ATTN_OUT ? ctx->h : ctx->ffn) / (ctx->t * ctx->groups);
  if (!tc_gemm_usable(ctx, K_r)) return CAAT_EUNSUPPORTED;
  const int slice = slice_rows(tokens, peers->world);
  if (slice % 256 != 0) return CAAT_EUNSUPPORTED;
  const Scratch L = scratch_layout(ctx, K_r, tokens, 0);
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 15u) || workspace_bytes < L.total) return CAAT_EWORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* wsb = static_cast<char*>(workspace);
  const RowparShapes sh{ctx->t, tokens, ctx->h, K_r, ctx->S, L.S_lo, L.S_hi, L.P};
  const PushTarget pt{peers->world, peers->rank, slice, pr.recv};
  cudaError_t e = launch_tc_forward(sh, Y, W, wsb + L.zs_off, wsb + L.zp_off, st, &pt);
  if (e != cudaSuccess) return cuda_fail(e);
  LaunchScope scope(CAAT_K_TP_EXCHANGE, st);
  e = launch_pdl(tp_signal_kernel, dim3(1), dim3(32), 0, st, pr, peers->world, peers->rank, epoch);
  return e == cudaSuccess ? CAAT_OK : cuda_fail(e);
}

caat_status caat_tp_backward_local_push(const caat_ctx* ctx, caat_layer layer, int tokens, const void* dX,
                                        const void* dHn, const void* W, const void* Hn, const float* rstd,
                                        const float* mean, const void* gamma, void* dR, float* dgamma, float* dbeta,
                                        const caat_peers* peers, unsigned int epoch, void* workspace,
                                        size_t workspace_bytes, void* cuda_stream) {
  Peers pr{};
  caat_status s = check_peers(ctx, peers, &pr, true, false);
  if (s != CAAT_OK) return s;
  if (tokens < 1) return CAAT_ESHAPE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const PushTarget pt{peers->world, peers->rank, slice_rows(tokens, peers->world), pr.recv};
  s = tp_backward_local_push_impl(ctx, layer, tokens, dX, dHn, W, Hn, rstd, mean, gamma, dR, dgamma, dbeta, workspace,
                                  workspace_bytes, st, pt);
  if (s != CAAT_OK) return s;
  LaunchScope scope(CAAT_K_TP_EXCHANGE, st);
  const cudaError_t e = launch_pdl(tp_signal_kernel, dim3(1), dim3(32), 0, st, pr, peers->world, peers->rank, epoch);
  return e == cudaSuccess ? CAAT_OK : cuda_fail(e);
}

}  // extern "C"
