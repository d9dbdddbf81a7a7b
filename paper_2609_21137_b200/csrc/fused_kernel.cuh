// One kernel for everything between the router and the weighted sum.
//
// The intermediate dimension I is cut into slices of `tps` row tiles (8 tps rows).  One work item
// = (work group, slice) and runs on ONE block from start to end:
//     gate / up rows of the slice from the compressed form  (Eq. 1; partial tiles meet in shared memory)
//  -> p = silu(g) * u for those rows                         (stays in shared memory)
//  -> partial z_d = basis_down[:, slice] * p                 (full mode; tiny, to global)
//  -> partial y = W_down[:, slice] * p for ALL H output rows (compressed or dense bf16)
// Both products are linear in the slice of p, so items never wait for each other: no kernel
// boundary and no grid-wide barrier between the projections, p never leaves the SM, and the index
// bytes of the down product are requested before the gate/up product starts.  The weighted-sum
// kernel adds the slices' partial y and, in full mode, the low-rank term of the down projection
// (it needs the complete z_d, which is the one sum over slices this kernel cannot form).
//
// The down product contracts over only `tps` blocks per row, so its index map is re-laid at
// create() as [expert][slice][row tile][lane][jd]: the jd = ceil(tps / 4) indices that lane (g, c)
// of a warp needs for a row tile (row g, blocks c, c + 4, ...) are adjacent (one shared-memory
// read), a tile is one contiguous run, and the tiles of an item follow each other.  Entries beyond
// the slice are 0 and meet zero activations.  A dense bf16 down matrix is read in place (8 tps
// columns = 16 tps bytes per row).
#pragma once
#include "fast_kernels.cuh"

namespace {

constexpr int kFusedMaxThreads = 512;      // a block runs 16 warps where its shared memory allows, else 12 (FusedPlan::warps)
constexpr int kFusedMaxJd = 4;       // k steps of the down product: at most 16 blocks per slice

struct FusedPlan {
  int warps;      // warps per block: 16, or 12 where the rings of 16 do not fit (more warps hide more of the read latency)
  int tps;        // row tiles of I per slice (the last slice of an expert may have fewer)
  int n_sl;       // slices per expert
  int t_last;     // row tiles of the last slice
  int jd;         // k steps of the down product = ceil(tps / 4)
  int depth_g, depth_d;
  int rp_log2;    // log2 of the power of two >= 8 tps
  FastDiv d_nsl, d_tps, d_tlast;
};

struct FusedLayout {
  size_t cb_u, x, ring_g, ring_d, z, route, parts, pf, ph, pl, tmp, total;
  int dn_slot_bytes;
};

// gu_halves: 2 = partial tiles of gate and up, 1 = of up alone (experts without a gate projection).
__host__ __device__ inline FusedLayout fused_layout(int K, int n_books, int T, int H, int r, const StagePlan& pg,
                                                    const FusedPlan& fp, bool dn_dense, int idx_bytes, int E, int k, int S,
                                                    int gu_halves = 2) {
  FusedLayout L;
  const size_t cb_bytes = (size_t)K * 16 * (pg.repl ? 8 : 1);
  L.cb_u = n_books == 2 ? cb_bytes : 0;
  size_t o = (size_t)n_books * cb_bytes;
  L.x = o;       o += pg.x_smem ? (size_t)T * (H / 8 + 1) * 16 : 0;
  L.ring_g = o;  o += (size_t)fp.warps * fp.depth_g * 2 * 32 * 16;
  L.dn_slot_bytes = dn_dense ? fp.jd * 32 * 16 : (32 * fp.jd * idx_bytes + 15) / 16 * 16;
  L.ring_d = o;  o += (size_t)fp.warps * fp.depth_d * L.dn_slot_bytes;
  L.z = o;       o += (size_t)2 * T * 2 * ((r + 7) / 8) * 16;
  L.route = o;   o += route_smem_bytes(T, E, k, S);
  L.parts = o;   o += (size_t)fp.tps * pg.n_parts * gu_halves * 64 * 4;      // [part][tile][gate|up][token 8][row 8]
  L.pf = o;      o += (size_t)8 * 8 * fp.tps * 4;                    // p as fp32 [token 8][row]
  L.ph = o;      o += (size_t)8 * 4 * fp.jd * 16;                    // p as bf16 hi blocks [token 8][4 jd]
  L.pl = o;      o += (size_t)8 * 4 * fp.jd * 16;                    // ... and the bf16 remainder
  L.tmp = o;     o += pg.repl ? (size_t)n_books * K * 16 : 0;
  L.total = o;
  return L;
}

// Re-lays the down index map: dst[e][si][tile][lane = 4 g + c][j] = src[e][8 tile + g][si tps + 4 j + c]
// (0 beyond the slice).
template <typename IdxT>
__global__ void k_relay_down_idx(const IdxT* __restrict__ src, IdxT* __restrict__ dst, int n_exp, int H, int nbI,
                                 int tps, int n_sl, int jd, int idx12) {
  const size_t total = (size_t)n_exp * n_sl * (H / 8) * 32 * jd;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int j = (int)(i % jd);
    size_t q = i / jd;
    const int lane = (int)(q % 32);
    q /= 32;
    const int tile = (int)(q % (H / 8));
    q /= (H / 8);
    const int si = (int)(q % n_sl);
    const int e = (int)(q / n_sl);
    const int g = lane >> 2, c = lane & 3, b = 4 * j + c, blk = si * tps + b;
    const size_t at = ((size_t)e * H + tile * 8 + g) * nbI + blk;
    dst[i] = (b < tps && blk < nbI) ? (idx12 ? (IdxT)read_idx12(src, at) : src[at]) : (IdxT)0;
  }
}

// JD = k steps of the down product (a compile-time constant: the down loop is bound by
// instruction issue, and with JD known its predicates and index unpacking fold away).
// SP: also experts without a gate projection and 12-bit packed indices (run-time checks in the unit
// loop that the plain instantiation folds away).
// LEAN: the single-token call whose items fit one wave and that wants no debug lists -- what a
// decode step at batch 1 runs.  Only the run-time-compiled copy of the kernel (jit_host.cuh) is built
// that way, and it also knows the layer's shape: MOE_VQLR_JIT replaces every integer of the
// parameter block and of the two plans by a constant.  At batch 1 every block runs
// most of this kernel's code exactly once, so what the kernel costs is largely the number of
// instructions fetched and the jumps over code that is not taken: with the constants folded the
// same source is two thirds of the size and the layer 15 % faster (measured).
template <typename IdxT, bool DN_DENSE, int JD, bool D4, bool SP, bool LEAN>
__device__ __forceinline__ void expert_fused_body(const Params& P_in, const bf16* __restrict__ x, int T_in, const StagePlan& pg_in,
                                                  const FusedPlan& fp_in, int n_books_in, int want_dbg_in,
                                                  const IdxT* __restrict__ idx_dp) {
  const int T = LEAN ? 1 : T_in, want_dbg = LEAN ? 0 : want_dbg_in;
  StagePlan pg = pg_in;
#ifdef MOE_VQLR_JIT
  constexpr bool kShape = true;
  constexpr int n_books = J_NBOOKS;
  Params P = P_in;
  MOE_VQLR_JIT_PARAMS(P);
  pg.nb = J_NB; pg.n_slices = J_NSLICES; pg.n_lr = J_NLR; pg.n_parts = J_NPARTS; pg.repl = J_REPL; pg.x_smem = J_XSMEM;
  FusedPlan fp = fp_in;
  fp.warps = J_WARPS; fp.tps = J_TPS; fp.n_sl = J_NSL; fp.t_last = J_TLAST; fp.jd = JD; fp.depth_g = J_DEPTH_G; fp.depth_d = J_DEPTH_D; fp.rp_log2 = J_RP_LOG2;
  (void)n_books_in;
#else
  constexpr bool kShape = false;
  const int n_books = n_books_in;
  const Params& P = P_in;
  const FusedPlan& fp = fp_in;
#endif
  extern __shared__ uint4 s_u4[];
  char* s_base = reinterpret_cast<char*>(s_u4);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, c = lane & 3;
  const int nw = fp.warps, nthr = nw * 32;       // = blockDim.x
  const int nb = pg.nb, xs = nb + 1, rb = (P.r + 7) / 8, Dg = fp.depth_g, Dd = fp.depth_d;
  const int gu_halves = (SP && P.act == 2) ? 1 : 2;      // up-only experts keep no gate tiles
  const FusedLayout L = fused_layout(P.K, n_books, T, P.H, P.r, pg, fp, DN_DENSE, (int)sizeof(IdxT), P.E, P.k, P.S, gu_halves);
  GuSmem m;
  m.cb_g = s_u4;
  m.cb_u = reinterpret_cast<uint4*>(s_base + L.cb_u);
  m.x = reinterpret_cast<uint4*>(s_base + L.x);
  m.ring = reinterpret_cast<uint4*>(s_base + L.ring_g) + (size_t)warp * Dg * 2 * 32 + lane;   // [slot][proj][lane]
  m.zh = reinterpret_cast<uint4*>(s_base + L.z);
  m.zl = m.zh + (size_t)T * 2 * rb;
  m.tmp = reinterpret_cast<uint4*>(s_base + L.tmp);
  m.R = carve_route(s_base + L.route, T, P.E, P.k, P.S);
  const RouteSmem& R = m.R;
  float* s_parts = reinterpret_cast<float*>(s_base + L.parts);
  float* s_pf = reinterpret_cast<float*>(s_base + L.pf);
  uint4* s_ph = reinterpret_cast<uint4*>(s_base + L.ph);
  uint4* s_pl = reinterpret_cast<uint4*>(s_base + L.pl);
  char* ring_d = s_base + L.ring_d + (size_t)warp * Dd * L.dn_slot_bytes;
  const uint4* s_cb_d = (n_books == 2 && P.down.codebook == P.up.codebook) ? m.cb_u : m.cb_g;
  const IdxT* idx_g = static_cast<const IdxT*>(P.gate.idx);
  const IdxT* idx_u = static_cast<const IdxT*>(P.up.idx);

  // One work item as this warp sees it.  Its gate/up units are an even share of the slice units
  // (part-major: consecutive units share their activation fragments) followed by an even share of
  // the cheap low-rank units.
  struct Item {
    int e, off, cnt, gi, si, tiles, row0, ns, n_my;
    int sp, st, lp, lt;       // (part, tile) of the first slice unit and of the first low-rank unit of this warp
  };
  struct UnitCur {            // walks the warp's units in order: slice units, then low-rank units
    int i, part, tile;
  };
  // The part of an item that does not depend on the routing (everything but the expert and its
  // pairs) ...
  auto item_static = [&](int v) {
    Item it;
    it.gi = kShape ? v / fp.n_sl : fdiv(v, fp.d_nsl);
    it.si = v - it.gi * fp.n_sl;
    it.e = 0; it.off = 0; it.cnt = 0;
    const bool last_sl = it.si == fp.n_sl - 1;
    it.tiles = last_sl ? fp.t_last : fp.tps;
    const FastDiv d_tiles = last_sl ? fp.d_tlast : fp.d_tps;
    it.row0 = it.si * fp.tps * 8;
    const int Us = pg.n_slices * it.tiles, Ul = pg.n_lr * it.tiles;
    const int s0 = Us * warp / nw, l0 = Ul * warp / nw;
    it.ns = Us * (warp + 1) / nw - s0;
    it.n_my = it.ns + Ul * (warp + 1) / nw - l0;
    it.sp = kShape ? s0 / it.tiles : fdiv(s0, d_tiles); it.st = s0 - it.sp * it.tiles;
    const int lq = kShape ? l0 / it.tiles : fdiv(l0, d_tiles);
    it.lp = pg.n_slices + lq; it.lt = l0 - lq * it.tiles;
    return it;
  };
  Item it = item_static(blockIdx.x);       // before the wait below: it costs a thousand clocks of cold scalar code
  // ... and the rest, once the work groups are known.
  auto item_bind = [&](Item& it) {
    it.e = R.grp_e[it.gi]; it.off = R.grp_off[it.gi]; it.cnt = R.grp_cnt[it.gi];
  };
  auto load_item = [&](int v) {
    Item it = item_static(v);
    item_bind(it);
    return it;
  };
  auto cur_begin = [&](const Item& it) {
    UnitCur u;
    u.i = 0;
    if (it.ns > 0) { u.part = it.sp; u.tile = it.st; } else { u.part = it.lp; u.tile = it.lt; }
    return u;
  };
  auto cur_next = [&](const Item& it, UnitCur& u) {
    ++u.i;
    if (u.i == it.ns) { u.part = it.lp; u.tile = it.lt; }
    else if (++u.tile == it.tiles) { u.tile = 0; ++u.part; }
  };
  const bool up_only = SP && P.act == 2;     // experts without a gate: its bytes are not requested, its products not formed
  const int idx12 = SP ? P.idx12 : 0;
  int g_rq = 0, g_use = 0;             // gate/up ring: next slot to request into, next to consume
  bool requests_on = true;             // off: the request code runs (and warms the instruction cache) without asking for bytes
  auto gu_request = [&](const Item& it, UnitCur& rq) {                    // requests come in the order of use
    const int part = rq.part, tile = rq.tile;
    cur_next(it, rq);
    uint4* slot = m.ring + (size_t)g_rq * 2 * 32;
    if (++g_rq == Dg) g_rq = 0;
    const size_t row = (size_t)it.e * P.I + it.row0 + tile * 8 + g;
    if (part < pg.n_slices) {
      const int b = part * 32 + 8 * c;
      if (b < nb && requests_on) {
        if (!up_only) cp_async_idx8<IdxT>(slot, idx_at(idx_g, row * nb + b, idx12), idx12);
        cp_async_idx8<IdxT>(slot + 32, idx_at(idx_u, row * nb + b, idx12), idx12);
      }
    } else {
      const int rho = (part - pg.n_slices) * 32 + 8 * c;
      if (rho < P.r && requests_on) {
        if (!up_only) cp_async16(slot, P.gate.factor + row * P.r + rho);
        cp_async16(slot + 32, P.up.factor + row * P.r + rho);
      }
    }
  };

  TRACE_STAMP(3, 0);
  gu_stage_async<false>(P, x, T, pg, n_books, m);
  const int n_pos = T * (P.k + P.S);
  const int n_dn = (P.H / 8 - warp + nw - 1) / nw;    // down row tiles of this warp: warp, warp + nw, ...
  // down tile warp + 12 i of the item -> slot `slot` of this warp's down ring
  auto dn_request = [&](const Item& it, int i, int slot_i) {
    const int jt = warp + i * nw;
    char* slot = ring_d + (size_t)slot_i * L.dn_slot_bytes;
    if (DN_DENSE) {
      const uint4* wd = reinterpret_cast<const uint4*>(P.down.dense + ((size_t)it.e * P.H + jt * 8 + g) * P.I + it.row0);
#pragma unroll
      for (int j = 0; j < JD; ++j)
        if (4 * j + c < it.tiles) cp_async16(reinterpret_cast<uint4*>(slot) + j * 32 + lane, wd + 4 * j + c);
    } else {
      const int bytes = 32 * JD * (int)sizeof(IdxT);
      const char* src = reinterpret_cast<const char*>(idx_dp + (((size_t)it.e * fp.n_sl + it.si) * (P.H / 8) + jt) * 32 * JD);
      if (lane * 16 < bytes) cp_async16(slot + lane * 16, src + lane * 16);
    }
  };
  // One block publishes the routing (slots, affinities, lists) for the weighted sum and the caller:
  // a block without an item if there is one, else block 0.  For a single token the other blocks
  // only need the selected experts in id order, which is much shorter to find.
  const int min_items = (P.k + P.S) * fp.n_sl;          // every token adds at least this many
  const int writer = (T == 1 && min_items < (int)gridDim.x) ? (int)gridDim.x - 1 : 0;
  const bool is_writer = (int)blockIdx.x == writer;
  int n_grp = 0, n_items = 0;
  UnitCur rq = cur_begin(it);            // request cursor of the current item (of the next one once its first units are requested)
  // The code that binds the item and requests its first units runs twice: a first time while the
  // router still runs, with the requests switched off, and then for real.  Straight-line code that
  // a block executes once per call runs at a few instructions per hundred clocks while it is not
  // in the instruction caches, and this piece sits between the routing and the first bytes.
  constexpr int kFirstPass = LEAN ? 1 : 0;       // the lean copy is short enough to do without the dry run (measured)
#pragma unroll 1
  for (int pass = kFirstPass; pass < 2; ++pass) {
    if (pass == 1) {
      pdl_wait();      // logits and z of this call are complete
      TRACE_STAMP(3, 1);
      gu_route(P, T, pg, m, is_writer, want_dbg != 0, T == 1 && !is_writer && P.E <= 1024);
      TRACE_STAMP(3, 2);
      n_grp = *R.n_grp;
      n_items = n_grp * fp.n_sl;
      if ((int)blockIdx.x >= n_items) { cp_async_wait_pending(0); return; }
    }
    requests_on = pass == 1;
    g_rq = 0;
    item_bind(it);
    rq = cur_begin(it);
    for (int i = 0; i < Dg - 1; ++i) {
      if (i < it.n_my) gu_request(it, rq);
      if (pass == 1) cp_async_commit();
    }
  }
  TRACE_STAMP(3, 14);
  gu_finish_stage<false>(P, pg, n_books, m, Dg - 1);     // code books, tokens, z, routing lists
  TRACE_STAMP(3, 15);
  pdl_launch();

  for (int v = blockIdx.x; v < n_items; v += LEAN ? n_items : gridDim.x) {
    const bool has_next = !LEAN && v + (int)gridDim.x < n_items;
    const Item nx = has_next ? load_item(v + gridDim.x) : it;
    const int off = it.off, cnt = it.cnt, si = it.si, tiles_here = it.tiles, row0 = it.row0, n_my = it.n_my;
    TRACE_STAMP(3, 3);
    // Compressed down projection: ALL index bytes of this warp's down tiles are requested now (one
    // cp.async group), so that they have landed long before the down product, which does two
    // lookups per tile and could not hide a DRAM round trip.
    if (!DN_DENSE) {
      const int bytes = 32 * JD * (int)sizeof(IdxT);
      const char* src = reinterpret_cast<const char*>(idx_dp + (((size_t)it.e * fp.n_sl + si) * (P.H / 8) + warp) * 32 * JD) + lane * 16;
      char* dst = ring_d + lane * 16;
      if (lane * 16 < bytes)
        for (int i = 0; i < n_dn; ++i) { cp_async16(dst, src); src += (size_t)nw * bytes; dst += L.dn_slot_bytes; }
      cp_async_commit();
    }
    // ---- gate / up partial tiles into shared memory ------------------------------------------
    {
      uint4 fx[8];
      int frag_part = -1;
      UnitCur use = cur_begin(it);
      for (int i = 0; i < n_my; ++i) {
        if (i + Dg - 1 < n_my) gu_request(it, rq);
        cp_async_commit();
        cp_async_wait_pending(Dg - 1);
        if (i < 2) TRACE_STAMP(3, 10 + 2 * i);
        const int part = use.part, tile = use.tile;
        cur_next(it, use);
        const uint4* slot = m.ring + (size_t)g_use * 2 * 32;
        if (++g_use == Dg) g_use = 0;
        const int tok = g < cnt ? R.pair_token[off + g] : -1;
        float acc_g[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
        float acc_u[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
        if (part < pg.n_slices) {
          const int b0 = part * 32 + 8 * c;
          if (frag_part != part) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
              fx[j] = (tok >= 0 && b0 + j < nb) ? (pg.x_smem ? m.x[tok * xs + b0 + j] : __ldg(reinterpret_cast<const uint4*>(x) + (size_t)tok * nb + b0 + j))
                                                : make_uint4(0, 0, 0, 0);
            frag_part = part;
          }
          // mma.sync needs the whole warp: lanes whose block group lies beyond the row run it
          // with index 0 and zero activation fragments
          uint4 raw_g = {0, 0, 0, 0}, raw_u = {0, 0, 0, 0};
          if (b0 < nb) { if (!up_only) raw_g = ring_idx8<IdxT>(slot); raw_u = ring_idx8<IdxT>(slot + 32); }
          uint32_t ig[8], iu[8];
          slot_idx8<IdxT>(raw_g, idx12, ig);
          slot_idx8<IdxT>(raw_u, idx12, iu);
          if (D4) {                   // four-value code words: two 8-byte reads per block
#pragma unroll
            for (int j = 0; j < 8; ++j) mma_block(acc_u[j & 1], fx[j], lookup_d4(m.cb_u, iu[j], lane));
            if (!up_only)
#pragma unroll
              for (int j = 0; j < 8; ++j) mma_block(acc_g[j & 1], fx[j], lookup_d4(m.cb_g, ig[j], lane));
          } else if (pg.repl) {
#pragma unroll
            for (int j = 0; j < 8; ++j) mma_block(acc_u[j & 1], fx[j], m.cb_u[(iu[j] << 3) | (lane & 7)]);
            if (!up_only)
#pragma unroll
              for (int j = 0; j < 8; ++j) mma_block(acc_g[j & 1], fx[j], m.cb_g[(ig[j] << 3) | (lane & 7)]);
          } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) mma_block(acc_u[j & 1], fx[j], m.cb_u[iu[j]]);
            if (!up_only)
#pragma unroll
              for (int j = 0; j < 8; ++j) mma_block(acc_g[j & 1], fx[j], m.cb_g[ig[j]]);
          }
        } else {
          // low-rank unit: B = 8 ranks of this lane's factor row, A = the matching z values (hi, lo)
          const int rho0 = (part - pg.n_slices) * 32 + 8 * c;
          uint4 fg = {0, 0, 0, 0}, fu = {0, 0, 0, 0};
          uint4 zgh = {0, 0, 0, 0}, zgl = {0, 0, 0, 0}, zuh = {0, 0, 0, 0}, zul = {0, 0, 0, 0};
          if (rho0 < P.r) {
            if (!up_only) fg = slot[0];
            fu = slot[32];
            if (tok >= 0) {
              const int ig2 = (tok * 2 + P.gate.zslot) * rb + (rho0 >> 3), iu2 = (tok * 2 + P.up.zslot) * rb + (rho0 >> 3);
              zgh = m.zh[ig2]; zgl = m.zl[ig2]; zuh = m.zh[iu2]; zul = m.zl[iu2];
            }
          }
          mma_block_hilo(acc_g[0], zgh, zgl, fg);     // rows 8..15 of the tile carry the lo product
          mma_block_hilo(acc_u[0], zuh, zul, fu);
          acc_g[0][0] += acc_g[0][2]; acc_g[0][1] += acc_g[0][3];
          acc_u[0][0] += acc_u[0][2]; acc_u[0][1] += acc_u[0][3];
        }
        // partial tile of this unit: token g, rows 2c and 2c+1 of the tile
        float* dst = s_parts + ((size_t)(part * fp.tps + tile) * gu_halves) * 64 + g * 8 + 2 * c;
        if (!up_only) *reinterpret_cast<float2*>(dst) = make_float2(acc_g[0][0] + acc_g[1][0], acc_g[0][1] + acc_g[1][1]);
        *reinterpret_cast<float2*>(dst + (up_only ? 0 : 64)) = make_float2(acc_u[0][0] + acc_u[1][0], acc_u[0][1] + acc_u[1][1]);
        if (i < 2) TRACE_STAMP(3, 11 + 2 * i);
      }
    }
    // what is left of the down requests; then the ring start of the other product
    int newest = 0;                      // cp.async groups that may stay in flight across the activation step
    if (DN_DENSE) {
      for (int i = 0; i < Dd - 1; ++i) { if (i < n_dn) dn_request(it, i, i); cp_async_commit(); }
      newest = Dd - 1;
    } else {
      if (has_next) {                    // the gate/up ring is free: the next item's first units start travelling
        rq = cur_begin(nx);
        for (int i = 0; i < Dg - 1; ++i) { if (i < nx.n_my) gu_request(nx, rq); cp_async_commit(); }
        newest = Dg - 1;
      }
    }
    TRACE_STAMP(3, 4);
    __syncthreads();
    TRACE_STAMP(3, 5);

    // ---- p = phi(gate) * up for the slice's rows; parts added in ascending order -------------
    const int R_here = tiles_here * 8, R_max = fp.tps * 8, RP = 1 << fp.rp_log2;
    for (int idx = tid; idx < cnt * RP; idx += nthr) {
      const int tk = idx >> fp.rp_log2, row = idx & (RP - 1);
      if (row < R_here) {
        const int tile = row >> 3, rr = row & 7;
        float gs = 0.f, us = 0.f;
        for (int part = 0; part < pg.n_parts; ++part) {
          const float* src = s_parts + ((size_t)(part * fp.tps + tile) * gu_halves) * 64 + tk * 8 + rr;
          if (!up_only) gs += src[0];
          us += src[up_only ? 0 : 64];
        }
        const float pv = gated_act(gs, us, P.act);
        s_pf[tk * R_max + row] = pv;
        const bf16 hi = __float2bfloat16_rn(pv);
        reinterpret_cast<bf16*>(s_ph)[(tk * 4 * JD + tile) * 8 + rr] = hi;
        reinterpret_cast<bf16*>(s_pl)[(tk * 4 * JD + tile) * 8 + rr] = __float2bfloat16_rn(pv - __bfloat162float(hi));
      }
    }
    __syncthreads();
    TRACE_STAMP(3, 6);

    // ---- partial z_d of the slice (compressed down projection with a low-rank term) -----------
    if (!DN_DENSE && P.r > 0) {
      for (int idx = tid; idx < cnt * P.r; idx += nthr) {
        const int tk = idx / P.r, rho = idx - tk * P.r;
        const uint4* b4 = reinterpret_cast<const uint4*>(P.down.basis + (size_t)rho * P.I + row0);
        const float* pv = s_pf + tk * R_max;
        float acc = 0.f;
        for (int q = 0; q < tiles_here; ++q) {
          float wf[8];
          unpack8(__ldg(b4 + q), wf);
#pragma unroll
          for (int j = 0; j < 8; ++j) acc = fmaf(wf[j], pv[q * 8 + j], acc);
        }
        P.zd_part[((size_t)(off + tk) * fp.n_sl + si) * P.r + rho] = acc;
      }
    }
    TRACE_STAMP(3, 7);

    // ---- partial y over all H rows: contraction over the slice ---------------------------------
    {
      uint4 fh[JD], fl[JD];
#pragma unroll
      for (int j = 0; j < JD; ++j) {
        const bool live = g < cnt && 4 * j + c < tiles_here;
        fh[j] = live ? s_ph[g * 4 * JD + 4 * j + c] : make_uint4(0, 0, 0, 0);
        fl[j] = live ? s_pl[g * 4 * JD + 4 * j + c] : make_uint4(0, 0, 0, 0);
      }
      const int pos = g < cnt ? off + g : -1;
      if (!DN_DENSE) {
        cp_async_wait_pending(newest);   // every index byte of the item's down tiles is in shared memory ...
        __syncwarp();                    // ... also the ones other lanes copied
      }
      if (DN_DENSE) {
        int d_use = 0, d_slot = Dd - 1;  // ring: slot to consume, slot to request into
        for (int i = 0; i < n_dn; ++i) {
          if (i + Dd - 1 < n_dn) dn_request(it, i + Dd - 1, d_slot);     // each lane re-uses only its own bytes: no warp sync
          if (++d_slot == Dd) d_slot = 0;
          cp_async_commit();
          cp_async_wait_pending(Dd - 1);
          const uint4* slot = reinterpret_cast<const uint4*>(ring_d + (size_t)d_use * L.dn_slot_bytes) + lane;
          if (++d_use == Dd) d_use = 0;
          const int jt = warp + i * nw;
          float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};      // two chains; each: hi product | lo product
#pragma unroll
          for (int j = 0; j < JD; ++j) {
            const uint4 w = 4 * j + c < tiles_here ? slot[j * 32] : make_uint4(0, 0, 0, 0);      // every lane runs every mma
            mma_block_hilo(acc[j & 1], fh[j], fl[j], w);
          }
          if (pos >= 0)
            *reinterpret_cast<float2*>(P.ypart + ((size_t)si * n_pos + pos) * P.H + jt * 8 + 2 * c) =
                make_float2((acc[0][0] + acc[0][2]) + (acc[1][0] + acc[1][2]), (acc[0][1] + acc[0][3]) + (acc[1][1] + acc[1][3]));
        }
      } else {
        // four row tiles per trip: their index reads, code-book reads and mma chains overlap
        constexpr int kU = 4;
        float* ydst = pos >= 0 ? P.ypart + ((size_t)si * n_pos + pos) * P.H + 2 * c : nullptr;
        for (int i0 = 0; i0 < n_dn; i0 += kU) {
          uint32_t id[kU][JD];
#pragma unroll
          for (int u = 0; u < kU; ++u) {
            // this lane's JD indices of the tile are adjacent: one read when they make up 2, 4 or 8 bytes
            constexpr int kNb = JD * (int)sizeof(IdxT);
            const char* sl = ring_d + (size_t)(i0 + u) * L.dn_slot_bytes + lane * kNb;
            uint32_t w0 = 0u, w1 = 0u;
            if (i0 + u < n_dn) {
              if (kNb == 4) w0 = *reinterpret_cast<const uint32_t*>(sl);
              else if (kNb == 8) { const uint2 v = *reinterpret_cast<const uint2*>(sl); w0 = v.x; w1 = v.y; }
              else if (kNb == 2) w0 = *reinterpret_cast<const uint16_t*>(sl);
              else if (kNb == 1) w0 = *reinterpret_cast<const uint8_t*>(sl);
              else if (kNb == 6) { w0 = reinterpret_cast<const uint16_t*>(sl)[0] | ((uint32_t)reinterpret_cast<const uint16_t*>(sl)[1] << 16); w1 = reinterpret_cast<const uint16_t*>(sl)[2]; }
              else { w0 = reinterpret_cast<const uint8_t*>(sl)[0] | ((uint32_t)reinterpret_cast<const uint8_t*>(sl)[1] << 8) | ((uint32_t)reinterpret_cast<const uint8_t*>(sl)[2] << 16); }
            }
#pragma unroll
            for (int j = 0; j < JD; ++j) {
              uint32_t v;
              if (sizeof(IdxT) == 2) v = ((j < 2 ? w0 : w1) >> (16 * (j & 1))) & 0xffffu;
              else v = (w0 >> (8 * j)) & 0xffu;
              id[u][j] = 4 * j + c < tiles_here ? v : 0u;
            }
          }
          float acc[kU][4];              // per tile: hi product (rows 0..7 of the m16 tile) | lo product (rows 8..15)
#pragma unroll
          for (int u = 0; u < kU; ++u)
#pragma unroll
            for (int q = 0; q < 4; ++q) acc[u][q] = 0.f;
#pragma unroll
          for (int j = 0; j < JD; ++j) {
#pragma unroll
            for (int u = 0; u < kU; ++u) {       // every lane runs every mma
              const uint4 w = D4 ? lookup_d4(s_cb_d, id[u][j], lane) : pg.repl ? s_cb_d[(id[u][j] << 3) | (lane & 7)] : s_cb_d[id[u][j]];
              mma_block_hilo(acc[u], fh[j], fl[j], w);
            }
          }
#pragma unroll
          for (int u = 0; u < kU; ++u)
            if (ydst && i0 + u < n_dn)
              *reinterpret_cast<float2*>(ydst + (warp + (i0 + u) * nw) * 8) =
                  make_float2(acc[u][0] + acc[u][2], acc[u][1] + acc[u][3]);
        }
      }
      if (DN_DENSE && has_next) {        // all dense groups are done with: the next item's first gate/up units
        rq = cur_begin(nx);
        for (int i = 0; i < Dg - 1; ++i) { if (i < nx.n_my) gu_request(nx, rq); cp_async_commit(); }
      }
    }
    TRACE_STAMP(3, 8);
    __syncthreads();                     // the next item reuses the partial tiles, p and the down ring
    TRACE_STAMP(3, 9);
    it = nx;
  }
  cp_async_wait_pending(0);
}

template <typename IdxT, bool DN_DENSE, int JD, bool D4 = false, bool SP = false>
__global__ void __launch_bounds__(kFusedMaxThreads, 1)
k_expert_fused(const Params P, const bf16* __restrict__ x, int T, const StagePlan pg, const FusedPlan fp, int n_books,
               int want_dbg, const IdxT* __restrict__ idx_dp) {
  expert_fused_body<IdxT, DN_DENSE, JD, D4, SP, false>(P, x, T, pg, fp, n_books, want_dbg, idx_dp);
}

// ---------------------------------------------------------------------------------------------
// Weighted sum after k_expert_fused: y[pos][h] = sum over slices of the partial y, plus (full
// mode) factor_down[e][h] . z_d[pos] with z_d = sum over slices of the partial z_d; then
// out[t][h] = sum over slots (in slot order) of affinity * y.  One block = one token and 8 pairs
// of columns; thread (column pair, quarter q, slot lane) adds the slices si = q mod 4 and the rank
// groups rg = q mod 4, quarters meet by shuffles, slots in shared memory.
// ---------------------------------------------------------------------------------------------
constexpr int kCfCols = 8;
constexpr int kCfThreads = 256;
// For a single token the kernel's 128 blocks are asked to be ALONE on their SM: the launch requests
// more than half an SM's shared memory.  Blocks of this kernel become resident one SM at a time as
// the expert kernel's blocks leave; with two per SM the first SMs to empty took two blocks each and
// those pairs shared one SM's path to memory for their cold rows of the down factor (measured: layer
// 24.4 us with two blocks per SM, 23.8 us with one).
constexpr size_t kCfAloneBytes = 120 * 1024;

template <bool LEAN>
__device__ __forceinline__ void combine_fused_body(const Params& P_in, bf16* __restrict__ out, int T_in, int n_sl_in, int lr_in) {
#ifdef MOE_VQLR_JIT
  constexpr int T = 1, n_sl = J_NSL, lr = J_LR;
  Params P = P_in;
  MOE_VQLR_JIT_PARAMS(P);
  (void)T_in; (void)n_sl_in; (void)lr_in;
#else
  const int T = LEAN ? 1 : T_in, n_sl = n_sl_in, lr = lr_in;
  const Params& P = P_in;
#endif
  extern __shared__ float s_cf[];
  const int n_slots = P.k + P.S, H2 = P.H / 2, n_pos = T * n_slots, r = P.r;
  float* s_zd = s_cf;                                                        // [n_slots][r]
  float2* s_y = reinterpret_cast<float2*>(s_cf + (lr ? (size_t)n_slots * r : 0));     // [n_slots][8]
  const int tid = threadIdx.x, col = tid & 7, q = (tid >> 3) & 3, sl = tid >> 5;
  const int units_per_tok = H2 / kCfCols;
  const int t = blockIdx.x / units_per_tok, h2 = (blockIdx.x - t * units_per_tok) * kCfCols + col;
  TRACE_STAMP(2, 8);
  // Every load of a thread is requested before the first one is used: the kernel is a handful of
  // dependent round trips long, not a loop of them.
  constexpr int kYv = 8, kAv = 4;      // slices / rank groups per thread held in registers (more: second pass)
  // Before the wait: a block of this kernel becomes resident when an SM runs out of expert-kernel
  // blocks, a microsecond or more before the LAST of them is done, and until now it sat out that
  // time.  The rows of the down factor that it needs depend only on the routing, which the expert
  // kernel published at its start: they are requested now, for the first trip over the slots, with
  // the expert ids as they stand in memory.  Memory written by the preceding kernel is only
  // guaranteed to be visible after the wait, so the ids are read again then and a thread whose id
  // has changed asks again; the speculation costs nothing when it fails and a DRAM round trip less
  // when it holds.
  // A single token's pairs are positions 0 .. k+S-1, so the loop below can walk POSITIONS instead of
  // slots: a position's partial results sit at addresses that do not depend on the routing lists (one
  // dependent round trip less), its expert, slot and affinity are read beside them, and the product
  // lands in its slot's place, so the final sum is still taken in slot order.
  const bool pm = T == 1;
  int e_spec = -1;
  uint4 a0v[kAv], a1v[kAv];
  if (lr && sl < n_slots) {
    e_spec = pm ? __ldcg(P.grp_e + sl) : sl < P.k ? __ldcg(P.topk_id + t * P.k + sl) : P.E + (sl - P.k);
    if ((unsigned int)e_spec >= (unsigned int)(P.E + P.S)) e_spec = 0;        // whatever the memory held: stay in range
    const uint4* a0 = reinterpret_cast<const uint4*>(P.down.factor + ((size_t)e_spec * P.H + 2 * h2) * r);
    const uint4* a1 = reinterpret_cast<const uint4*>(P.down.factor + ((size_t)e_spec * P.H + 2 * h2 + 1) * r);
#pragma unroll
    for (int i = 0; i < kAv; ++i) {
      const int rg = q + 4 * i;
      a0v[i] = a1v[i] = make_uint4(0, 0, 0, 0);
      if (rg < r / 8) {                  // volatile: these requests must leave before the wait below, not after it
        asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(a0v[i].x), "=r"(a0v[i].y), "=r"(a0v[i].z), "=r"(a0v[i].w) : "l"(a0 + rg));
        asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(a1v[i].x), "=r"(a1v[i].y), "=r"(a1v[i].z), "=r"(a1v[i].w) : "l"(a1 + rg));
      }
    }
  }
  pdl_wait();
  TRACE_STAMP(2, 9);
  pdl_launch();
  for (int s0 = 0; s0 < n_slots; s0 += kCfThreads / 32) {      // uniform trip count for the shuffles and barriers
    const int s = s0 + sl;
    const bool live = s < n_slots;
    int pos = 0, e = 0, slot = s;
    float w = 0.f;
    if (live) {
      if (pm) {
        pos = s;
        e = __ldcg(P.grp_e + s);
        slot = __ldcg(P.pair_slot + s);
      } else {
        pos = __ldcg(P.inv_pos + t * n_slots + s);
        e = s < P.k ? __ldcg(P.topk_id + t * P.k + s) : P.E + (s - P.k);
      }
    }
    const bool spec_ok = s0 == 0 && e == e_spec;        // the rows requested before the wait are the right ones
    // the first two z_d entries of this thread (slot sj, rank rho): their positions travel with `pos`
    const int n_here = min(kCfThreads / 32, n_slots - s0);
    const int n_zd = lr ? n_here * r : 0;
    int zsj[2], zrho[2], zpj[2];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int idx = tid + u * kCfThreads;
      zsj[u] = idx < n_zd ? idx / r : 0;
      zrho[u] = idx - zsj[u] * r;
      zpj[u] = idx >= n_zd ? 0 : pm ? s0 + zsj[u] : __ldcg(P.inv_pos + t * n_slots + s0 + zsj[u]);
    }
    float2 yv[kYv];
    const float* ysrc = P.ypart + (size_t)pos * P.H + 2 * h2;
    const uint4* a0 = reinterpret_cast<const uint4*>(P.down.factor + ((size_t)e * P.H + 2 * h2) * r);
    const uint4* a1 = reinterpret_cast<const uint4*>(P.down.factor + ((size_t)e * P.H + 2 * h2 + 1) * r);
    if (live) w = __ldcg(P.pair_w + pos);
#pragma unroll
    for (int i = 0; i < kYv; ++i) {
      const int si = q + 4 * i;
      yv[i] = (live && si < n_sl) ? __ldcg(reinterpret_cast<const float2*>(ysrc + (size_t)si * n_pos * P.H)) : make_float2(0.f, 0.f);
    }
#pragma unroll
    for (int i = 0; i < kAv; ++i) {
      const int rg = q + 4 * i;
      const bool on = live && lr && rg < r / 8;
      if (!spec_ok) {
        a0v[i] = on ? __ldg(a0 + rg) : make_uint4(0, 0, 0, 0);
        a1v[i] = on ? __ldg(a1 + rg) : make_uint4(0, 0, 0, 0);
      }
    }
    if (lr) {                            // z_d of this trip's slots: sum of the slices' parts, ascending
      float zv[2][16];
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const float* src = P.zd_part + (size_t)zpj[u] * n_sl * r + zrho[u];
#pragma unroll
        for (int i = 0; i < 16; ++i) zv[u][i] = (tid + u * kCfThreads < n_zd && i < n_sl) ? __ldcg(src + (size_t)i * r) : 0.f;
      }
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        if (tid + u * kCfThreads < n_zd) {
          float acc = 0.f;
#pragma unroll
          for (int i = 0; i < 16; ++i) acc += zv[u][i];
          const float* src = P.zd_part + (size_t)zpj[u] * n_sl * r + zrho[u];
          for (int si = 16; si < n_sl; ++si) acc += __ldcg(src + (size_t)si * r);
          s_zd[(s0 + zsj[u]) * r + zrho[u]] = acc;
        }
      }
      for (int idx = tid + 2 * kCfThreads; idx < n_zd; idx += kCfThreads) {
        const int sj = idx / r, rho = idx - sj * r;
        const int pj = pm ? s0 + sj : __ldcg(P.inv_pos + t * n_slots + s0 + sj);
        const float* src = P.zd_part + (size_t)pj * n_sl * r + rho;
        float acc = 0.f;
        for (int si = 0; si < n_sl; ++si) acc += __ldcg(src + (size_t)si * r);
        s_zd[(s0 + sj) * r + rho] = acc;
      }
      __syncthreads();
    }
    float y0 = 0.f, y1 = 0.f;
#pragma unroll
    for (int i = 0; i < kYv; ++i) { y0 += yv[i].x; y1 += yv[i].y; }
    if (live) {
      for (int si = q + 4 * kYv; si < n_sl; si += 4) {
        const float2 v = __ldcg(reinterpret_cast<const float2*>(ysrc + (size_t)si * n_pos * P.H));
        y0 += v.x; y1 += v.y;
      }
      if (lr) {
#pragma unroll
        for (int i = 0; i < kAv; ++i) {
          const int rg = q + 4 * i;
          if (rg < r / 8) {
            float f0[8], f1[8];
            unpack8(a0v[i], f0);
            unpack8(a1v[i], f1);
            const float* z = s_zd + s * r + rg * 8;
#pragma unroll
            for (int j = 0; j < 8; ++j) { y0 = fmaf(f0[j], z[j], y0); y1 = fmaf(f1[j], z[j], y1); }
          }
        }
        for (int rg = q + 4 * kAv; rg < r / 8; rg += 4) {
          float f0[8], f1[8];
          unpack8(__ldg(a0 + rg), f0);
          unpack8(__ldg(a1 + rg), f1);
          const float* z = s_zd + s * r + rg * 8;
#pragma unroll
          for (int j = 0; j < 8; ++j) { y0 = fmaf(f0[j], z[j], y0); y1 = fmaf(f1[j], z[j], y1); }
        }
      }
    }
    y0 += __shfl_xor_sync(0xffffffffu, y0, 8);  y1 += __shfl_xor_sync(0xffffffffu, y1, 8);
    y0 += __shfl_xor_sync(0xffffffffu, y0, 16); y1 += __shfl_xor_sync(0xffffffffu, y1, 16);
    if (live && q == 0) s_y[slot * kCfCols + col] = make_float2(w * y0, w * y1);
  }
  __syncthreads();
  if (tid < kCfCols) {
    float a0 = 0.f, a1 = 0.f;
    for (int s = 0; s < n_slots; ++s) { a0 += s_y[s * kCfCols + tid].x; a1 += s_y[s * kCfCols + tid].y; }
    *reinterpret_cast<__nv_bfloat162*>(out + (size_t)t * P.H + 2 * h2) = __floats2bfloat162_rn(a0, a1);
  }
  TRACE_STAMP(2, 10);
}

#ifndef MOE_VQLR_JIT
__global__ void __launch_bounds__(kCfThreads)
k_combine_fused(const Params P, bf16* __restrict__ out, int T, int n_sl, int lr) {
  combine_fused_body<false>(P, out, T, n_sl, lr);
}
#endif

}  // namespace
