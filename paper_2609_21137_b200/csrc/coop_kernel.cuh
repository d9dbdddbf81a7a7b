// The whole layer as ONE persistent cooperative kernel: router/z, routing + gate/up parts,
// SwiGLU + z_d, down parts, weighted sum -- the phase bodies of fast_kernels.cuh separated by
// grid-wide barriers.  A kernel boundary in the five-kernel chain costs 2.5-3 us at batch 1
// (launch, cold prologue, re-staging the code book); a grid barrier costs about 1 us and the
// code book, tokens and routing lists stay in shared memory across the phases.
//
// The grid barrier is a counter + generation pair in global memory.  Co-residency of all blocks
// is guaranteed by the cooperative launch.  Every wait is bounded: after Params::spin_limit
// polls (kGridSyncSpinLimit unless a test shortens it) the block records MOE_VQLR_ERR_TIMEOUT in
// the status word and leaves the kernel.
#pragma once
#include "fast_kernels.cuh"

namespace {

constexpr int kCoopThreads = 384;
constexpr int kGridSyncSpinLimit = 1 << 19;     // x ~0.4 us per poll (an L2 round trip): gives up after ~0.2 s

struct CoopLayout {
  size_t cb_u, x, ring, scratch, z, route, tmp, total;
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
  L.dn_slot_u4 = dn_vq ? 2 * pd.tpu : 8;
  // the ring serves the gate/up walk, then the down walk (whose first units are requested while
  // the activation phase still runs, hence a scratch region of its own for that phase and the combine)
  size_t region = (size_t)warps * pg.depth * 2 * 32 * 16;
  region = coop_max(region, (size_t)warps * pd.depth * L.dn_slot_u4 * 32 * 16);
  L.ring = o;   o += region;
  L.scratch = o; o += coop_max((size_t)I * 4, (size_t)(kMaxK + 8) * kCombineCols * 8);
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

// bar[0] counts arrivals and is never reset: every launch adds kCoopBarriers * gridDim.x to it.
// bar[1] is the number of completed launches (mod 2^32); a block reads it once at its start and
// derives the counter value that completes each barrier, so that a barrier is one fire-and-forget
// reduction plus polling loads -- no read-modify-write on the critical path and no reset.
// Block 0 advances bar[1] after the last barrier.  Returns false after a timeout; the counters
// are then out of step and the handle must not be used for further persistent launches.
constexpr unsigned int kCoopBarriers = 4;

__device__ __forceinline__ bool grid_sync(const Params& P, unsigned int* bar, unsigned int target) {
  __shared__ int s_ok;
  __syncthreads();
  if (threadIdx.x == 0) {
    bool ok = true;
    __threadfence();
    asm volatile("red.relaxed.gpu.global.add.u32 [%0], 1;" ::"l"(bar) : "memory");
    int spins = 0;
    target += (unsigned int)P.bar_fault;       // test switch: an arrival that never comes
    while ((int)(ld_acquire_u32(bar) - target) < 0) {
      if (++spins > P.spin_limit) { ok = false; set_status(P, MOE_VQLR_ERR_TIMEOUT); break; }
    }
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
  // every thread derives the barrier targets from the launch count (read before this block's first arrival)
  const unsigned int bar_epoch = __ldcg(bar + 1);
  const unsigned int bar_base = bar_epoch * kCoopBarriers * gridDim.x;
  const int n_pos = T * (P.k + P.S);

  // ---- phase A: router logits and shared projections; code books and tokens stream in meanwhile
  TRACE_STAMP(3, 0);
  {
    // rows are dealt round-robin over the blocks first, so that every SM streams a few of them
    const int n_units = router_z_units(P, T), unit0 = warp * gridDim.x + blockIdx.x;
    gu_stage_tokens_async(x, T, pg, m);
    RouterRow u;
    uint4 wv[8];
    const bool staged = pg.x_smem && unit0 < n_units;
    if (staged) {                                    // weight row and tokens travel together
      u = router_z_row(P, T, unit0);
      router_z_load8(u, 0, P.H / 8, lane, wv);
    }
    gu_stage_books_async<false>(P, pg, n_books, m);  // lands while the block waits at the barrier
    cp_async_wait_pending(1);
    __syncthreads();                                 // tokens are in shared memory
    if (staged) router_z_finish(P, u, m.x, pg.nb + 1, lane, wv);
    for (int unit = staged ? unit0 + W : unit0; unit < n_units; unit += W) router_z_unit(P, x, T, unit, lane);
  }
  TRACE_STAMP(3, 1);
  if (!grid_sync(P, bar, bar_base + 1u * gridDim.x)) return;
  TRACE_STAMP(3, 2);

  // ---- phase B: routing (every block), gate/up partial tiles
  {
    gu_route(P, T, pg, m, blockIdx.x == 0, want_dbg != 0);
    Walk w;
    gu_tiles_begin<IdxT, false>(P, pg, m, wid, W, w);
    gu_finish_stage<false>(P, pg, n_books, m, pg.depth - 1);      // the code books landed long ago
    TRACE_STAMP(3, 3);
    gu_tiles_run<IdxT, false>(P, x, T, pg, m, w);
  }
  TRACE_STAMP(3, 4);
  if (!grid_sync(P, bar, bar_base + 2u * gridDim.x)) return;
  TRACE_STAMP(3, 5);

  // ---- phase C: sum of parts, SwiGLU, z_d; meanwhile a down code book of its own streams in
  // and so do the first index / weight bytes of this warp's down units
  if (!DN_DENSE && dn_restage) {
    uint4* dst = pd.repl ? m.tmp : m.cb_g;
    for (int i = tid; i < P.K; i += blockDim.x) cp_async16(dst + i, P.down.codebook + i);
  }
  cp_async_commit();
  DnSmem dm;
  dm.cb = m.cb_g;
  dm.ring = reinterpret_cast<uint4*>(s_base + L.ring) + (size_t)warp * pd.depth * L.dn_slot_u4 * 32 + lane;
  dm.slot_u4 = L.dn_slot_u4;
  dm.grp_e = m.R.grp_e; dm.grp_off = m.R.grp_off; dm.grp_cnt = m.R.grp_cnt; dm.n_grp = *m.R.n_grp;
  Walk dw;
  dn_tiles_begin<IdxT, DN_DENSE>(P, pd, dm, wid, W, dw);
  {
    float* s_p = reinterpret_cast<float*>(s_base + L.scratch);
    const int with_zd = (!DN_DENSE && P.r > 0) ? 1 : 0;
    for (int unit = blockIdx.x; unit < n_pos * zsplit; unit += gridDim.x) {
      act_zdown_unit(P, n_pos, pg.n_parts, with_zd, zsplit, unit, s_p);
      __syncthreads();
    }
  }
  cp_async_wait_pending(pd.depth - 1);      // the code book (the walk's groups may still travel)
  TRACE_STAMP(3, 6);
  if (!grid_sync(P, bar, bar_base + 3u * gridDim.x)) return;
  TRACE_STAMP(3, 7);
  if (!DN_DENSE && dn_restage && pd.repl) {
    for (int i = tid; i < P.K * 8; i += blockDim.x) m.cb_g[i] = m.tmp[i >> 3];
    __syncthreads();
  }

  // ---- phase D: down partial tiles (work groups are still in shared memory)
  dn_tiles_run<IdxT, DN_DENSE>(P, T, pd, dm, dw);
  TRACE_STAMP(3, 8);
  if (!grid_sync(P, bar, bar_base + 4u * gridDim.x)) return;
  TRACE_STAMP(3, 9);
  if (blockIdx.x == 0 && tid == 0) bar[1] = bar_epoch + 1u;   // this launch is past its last barrier

  // ---- phase E: weighted sum
  {
    float2 (*s_y)[kCombineCols] = reinterpret_cast<float2 (*)[kCombineCols]>(s_base + L.scratch);
    for (int unit = blockIdx.x; unit < combine_units(P, T); unit += gridDim.x) {
      combine_unit(P, out, T, pd.n_parts, unit, s_y);
      __syncthreads();
    }
  }
  TRACE_STAMP(3, 10);
}

}  // namespace
