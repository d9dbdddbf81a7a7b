// The whole layer as ONE persistent cooperative kernel: router/z, routing + gate/up parts,
// SwiGLU + z_d, down parts, weighted sum -- the phase bodies of fast_kernels.cuh separated by
// grid-wide barriers.  A kernel boundary in the five-kernel chain costs 2.5-3 us at batch 1
// (launch, cold prologue, re-staging the code book); a grid barrier costs about 1 us and the
// code book, tokens and routing lists stay in shared memory across the phases.
//
// The grid barrier is a counter + generation pair in global memory.  Co-residency of all blocks
// is guaranteed by the cooperative launch.  Every wait is bounded: after kGridSyncSpinLimit
// polls the block records MOE_VQLR_ERR_TIMEOUT in the status word and leaves the kernel.
#pragma once
#include "fast_kernels.cuh"

namespace {

constexpr int kCoopThreads = 384;
constexpr long long kGridSyncSpinLimit = 1LL << 21;     // x ~100 ns per poll: gives up after ~0.2 s

struct CoopLayout {
  size_t cb_u, x, ring, z, route, tmp, total;
  int dn_slot_u4;
};

__host__ __device__ inline size_t coop_max(size_t a, size_t b) { return a > b ? a : b; }

__host__ __device__ inline CoopLayout coop_layout(int K, int n_books, int T, int H, int I, int r, const StagePlan& pg,
                                                  const StagePlan& pd, bool dn_vq, int warps, int E, int k, int S) {
  CoopLayout L;
  const size_t gu_book = (size_t)K * 16 * (pg.repl ? 8 : 1), dn_book = dn_vq ? (size_t)K * 16 * (pd.repl ? 8 : 1) : 0;
  L.cb_u = n_books == 2 ? gu_book : 0;
  size_t o = coop_max((size_t)n_books * gu_book, dn_book);
  L.x = o;      o += pg.x_smem ? (size_t)T * (H / 8 + 1) * 16 : 0;
  L.dn_slot_u4 = dn_vq ? 2 : 8;
  // one region serves, in turn: gate/up ring, p of one pair, down ring, the combine's slot sums
  size_t region = (size_t)warps * pg.depth * 2 * 32 * 16;
  region = coop_max(region, (size_t)warps * pd.depth * L.dn_slot_u4 * 32 * 16);
  region = coop_max(region, (size_t)I * 4);
  region = coop_max(region, (size_t)(kMaxK + 8) * kCombineCols * 8);
  L.ring = o;   o += region;
  L.z = o;      o += (size_t)2 * T * 2 * ((r + 7) / 8) * 16;
  L.route = o;  o += route_smem_bytes(T, E, k, S);
  L.tmp = o;    o += (pg.repl || pd.repl) ? (size_t)2 * K * 16 : 0;
  L.total = o;
  return L;
}

__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// bar[0] = arrivals of the current barrier, bar[1] = generation.  Returns false after a timeout.
__device__ __forceinline__ bool grid_sync(unsigned int* bar, int* status) {
  __shared__ int s_ok;
  __syncthreads();
  if (threadIdx.x == 0) {
    bool ok = true;
    const unsigned int gen0 = ld_acquire_u32(bar + 1);
    __threadfence();
    const unsigned int old = atomicAdd(bar, 1u);
    if (old == gridDim.x - 1) {
      atomicExch(bar, 0u);
      __threadfence();
      atomicAdd(bar + 1, 1u);
    } else {
      long long spins = 0;
      while (ld_acquire_u32(bar + 1) == gen0) {
        if (++spins > kGridSyncSpinLimit) { ok = false; atomicExch(status, MOE_VQLR_ERR_TIMEOUT); break; }
        __nanosleep(64);
      }
    }
    __threadfence();
    s_ok = ok ? 1 : 0;
  }
  __syncthreads();
  return s_ok != 0;
}

template <typename IdxT, bool DN_DENSE>
__global__ void __launch_bounds__(kCoopThreads, 1)
k_layer_coop(const Params P, const bf16* __restrict__ x, bf16* __restrict__ out, int T, const StagePlan pg,
             const StagePlan pd, int n_books, int want_dbg, int dn_restage, int zsplit) {
  extern __shared__ uint4 s_u4[];
  char* s_base = reinterpret_cast<char*>(s_u4);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const int wid = blockIdx.x * nwarps + warp, W = gridDim.x * nwarps;
  const CoopLayout L = coop_layout(P.K, n_books, T, P.H, P.I, P.r, pg, pd, !DN_DENSE, nwarps, P.E, P.k, P.S);
  GuSmem m;
  {
    const int rb = (P.r + 7) / 8;
    m.cb_g = s_u4;
    m.cb_u = reinterpret_cast<uint4*>(s_base + L.cb_u);
    m.x = reinterpret_cast<uint4*>(s_base + L.x);
    m.ring = reinterpret_cast<uint4*>(s_base + L.ring) + (size_t)warp * pg.depth * 2 * 32 + lane;
    m.zh = reinterpret_cast<uint4*>(s_base + L.z);
    m.zl = m.zh + (size_t)T * 2 * rb;
    m.tmp = reinterpret_cast<uint4*>(s_base + L.tmp);
    m.R = carve_route(s_base + L.route, T, P.E, P.k, P.S);
  }
  unsigned int* bar = P.grid_bar;
  const int n_pos = T * (P.k + P.S);

  // ---- phase A: router logits and shared projections; code books and tokens stream in meanwhile
  TRACE_STAMP(3, 0);
  gu_stage_async<false>(P, x, T, pg, n_books, m);
  for (int unit = wid; unit < router_z_units(P, T); unit += W) router_z_unit(P, x, T, unit, lane);
  TRACE_STAMP(3, 1);
  if (!grid_sync(bar, P.status)) return;
  TRACE_STAMP(3, 2);

  // ---- phase B: routing (every block), gate/up partial tiles
  gu_route_and_finish_stage<false>(P, T, pg, n_books, m, blockIdx.x == 0, want_dbg != 0);
  TRACE_STAMP(3, 3);
  gu_tiles<IdxT, false>(P, x, T, pg, m, wid, W);
  TRACE_STAMP(3, 4);
  if (!grid_sync(bar, P.status)) return;
  TRACE_STAMP(3, 5);

  // ---- phase C: sum of parts, SwiGLU, z_d; a down code book of its own streams in meanwhile
  if (!DN_DENSE && dn_restage) {
    uint4* dst = pd.repl ? m.tmp : m.cb_g;
    for (int i = tid; i < P.K; i += blockDim.x) cp_async16(dst + i, P.down.codebook + i);
  }
  cp_async_commit();
  {
    float* s_p = reinterpret_cast<float*>(s_base + L.ring);
    const int with_zd = (!DN_DENSE && P.r > 0) ? 1 : 0;
    for (int unit = blockIdx.x; unit < n_pos * zsplit; unit += gridDim.x) {
      act_zdown_unit(P, n_pos, pg.n_parts, with_zd, zsplit, unit, s_p);
      __syncthreads();
    }
  }
  cp_async_wait_pending(0);
  TRACE_STAMP(3, 6);
  if (!grid_sync(bar, P.status)) return;
  TRACE_STAMP(3, 7);
  if (!DN_DENSE && dn_restage && pd.repl) {
    for (int i = tid; i < P.K * 8; i += blockDim.x) m.cb_g[i] = m.tmp[i >> 3];
    __syncthreads();
  }

  // ---- phase D: down partial tiles (work groups are still in shared memory)
  {
    uint4* ring = reinterpret_cast<uint4*>(s_base + L.ring) + (size_t)warp * pd.depth * L.dn_slot_u4 * 32 + lane;
    dn_tiles<IdxT, DN_DENSE>(P, T, pd, m.cb_g, ring, L.dn_slot_u4, m.R.grp_e, m.R.grp_off, m.R.grp_cnt, *m.R.n_grp, wid, W);
  }
  TRACE_STAMP(3, 8);
  if (!grid_sync(bar, P.status)) return;
  TRACE_STAMP(3, 9);

  // ---- phase E: weighted sum
  {
    float2 (*s_y)[kCombineCols] = reinterpret_cast<float2 (*)[kCombineCols]>(s_base + L.ring);
    for (int unit = blockIdx.x; unit < combine_units(P, T); unit += gridDim.x) {
      combine_unit(P, out, T, pd.n_parts, unit, s_y);
      __syncthreads();
    }
  }
  TRACE_STAMP(3, 10);
}

}  // namespace
