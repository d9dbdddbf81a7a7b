// Gate/up through the projection code book (Section 4.2: the code words are projected onto the
// token once, T[b][k] = <x_b, codebook[k]>, and a weight row's VQ term becomes a sum of selected
// table entries) for batches of several tokens and K <= 256 (uint8 indices, d = 8).
//
// One entry costs a 4-byte shared-memory read per (token, row, block) where the reconstructing
// tensor-core kernel pays a 16-byte read and two mma's per (work group, row, block): with two or
// three tokens per work group and the per-unit bookkeeping of that kernel the table wins from a
// few tokens on.  The table of one token and both books does not fit one SM, so a block keeps the
// table of one PIECE of H (64 blocks of 8 values, both books: 128 KB at K = 256) of one token and
// walks its share of that token's (expert, row) pairs; the pieces of a row are partial tiles like
// the slices of the tensor-core kernel and meet in the activation kernel.
//
//   k_router_z(mma)_pdl -> k_gateup_lr (routing, published; low-rank term on the tensor cores)
//                       -> k_gateup_pcb (tables are built before its wait) -> k_act_zdown -> ...
//
// Layout of the table: lane l owns the blocks 2l and 2l + 1 of the piece and bank l of shared
// memory: entry (book, j = block & 1, k) of lane l sits at word ((book * 2 + j) * K + k) * 32 + l,
// so the 32 reads of a warp never share a bank.
#pragma once
#include "fast_kernels.cuh"

namespace {

constexpr int kPcbThreads = 512;
constexpr int kPcbPiece = 64;        // blocks of 8 values per table piece
constexpr int kPcbRows = 16;         // rows per batch: 16 gate + 16 up sums are reduced across the warp together

__host__ __device__ inline size_t pcb_smem_bytes(int K) {
  return (size_t)4 * K * 32 * sizeof(float) + (size_t)2 * K * 8 * sizeof(float);
}

// Low-rank term of gate and up for every (work group, 8-row tile): part 0 of gpart / upart.
// Every block redoes the routing from the logits (as the tensor-core gate/up kernel does) and block
// 0 publishes it.  A unit loads the factor rows of all rank groups, six groups at a time.
__global__ void __launch_bounds__(kFastThreads, 1)
k_gateup_lr(const Params P, const bf16* __restrict__ x, int T, const StagePlan pl, int want_dbg) {
  extern __shared__ uint4 s_u4[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5, g = lane >> 2, c = lane & 3;
  const GuLayout L = gu_layout(P.K, 0, T, P.H, P.r, pl, nwarps, P.E, P.k, P.S);
  const GuSmem m = gu_carve(reinterpret_cast<char*>(s_u4), L, P, T, warp, lane, pl.depth);
  pdl_wait();      // logits and z of this call are complete
  gu_route(P, T, pl, m, blockIdx.x == 0, want_dbg != 0);
  __syncthreads();
  pdl_launch();
  if (pl.n_lr == 0) return;
  const RouteSmem& R = m.R;
  const int n_pos = T * (P.k + P.S), rb = (P.r + 7) / 8;
  const int V = *R.n_grp * pl.tiles, W = gridDim.x * nwarps;
  for (int v = blockIdx.x * nwarps + warp; v < V; v += W) {
    const int grp = v / pl.tiles, jt = v - grp * pl.tiles;
    const int off = R.grp_off[grp], n_tok = R.grp_cnt[grp];
    const int tok = g < n_tok ? R.pair_token[off + g] : -1;
    const size_t row = (size_t)R.grp_e[grp] * P.I + jt * 8 + g;
    const uint4* fgp = reinterpret_cast<const uint4*>(P.gate.factor + row * P.r);
    const uint4* fup = reinterpret_cast<const uint4*>(P.up.factor + row * P.r);
    float acc_g[4] = {0.f, 0.f, 0.f, 0.f}, acc_u[4] = {0.f, 0.f, 0.f, 0.f};
    for (int lg0 = 0; lg0 < pl.n_lr; lg0 += 6) {
      uint4 fg[6], fu[6];
#pragma unroll
      for (int u = 0; u < 6; ++u) {
        const int rho = (lg0 + u) * 32 + 8 * c;
        const bool in = lg0 + u < pl.n_lr && rho < P.r;
        fg[u] = in ? __ldg(fgp + (rho >> 3)) : make_uint4(0, 0, 0, 0);
        fu[u] = in ? __ldg(fup + (rho >> 3)) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int u = 0; u < 6; ++u) {
        const int rho = (lg0 + u) * 32 + 8 * c;
        uint4 zgh = {0, 0, 0, 0}, zgl = {0, 0, 0, 0}, zuh = {0, 0, 0, 0}, zul = {0, 0, 0, 0};
        if (lg0 + u < pl.n_lr && rho < P.r && tok >= 0) {
          const int ig = (tok * 2 + P.gate.zslot) * rb + (rho >> 3), iu = (tok * 2 + P.up.zslot) * rb + (rho >> 3);
          zgh = m.zh[ig]; zgl = m.zl[ig]; zuh = m.zh[iu]; zul = m.zl[iu];
        }
        mma_block_hilo(acc_g, zgh, zgl, fg[u]);      // hi product in the first half of the accumulators, lo in the second
        mma_block_hilo(acc_u, zuh, zul, fu[u]);
      }
    }
    if (g < n_tok) {
      const size_t at = (size_t)(off + g) * P.I + jt * 8 + 2 * c;
      *reinterpret_cast<float2*>(P.gpart + at) = make_float2(acc_g[0] + acc_g[2], acc_g[1] + acc_g[3]);
      *reinterpret_cast<float2*>(P.upart + at) = make_float2(acc_u[0] + acc_u[2], acc_u[1] + acc_u[3]);
    }
  }
  (void)n_pos; (void)x;
}

// Sum over the 32 lanes of 32 values each: afterwards v[0] of lane l is the warp's total of value l.
__device__ __forceinline__ void warp_transpose_sum32(float (&v)[32], int lane) {
#pragma unroll
  for (int msk = 16; msk >= 1; msk >>= 1) {
    const bool upper = (lane & msk) != 0;
#pragma unroll
    for (int j = 0; j < msk; ++j) {
      const float send = upper ? v[j] : v[j + msk];
      const float keep = upper ? v[j + msk] : v[j];
      v[j] = keep + __shfl_xor_sync(0xffffffffu, send, msk);
    }
  }
}

// grid = T * Q * bpc blocks: block -> (token, piece q of H, share `sub` of the token's rows).
// part0: index of the first table part in gpart / upart (1 after the low-rank part, else 0).
__global__ void __launch_bounds__(kPcbThreads, 1)
k_gateup_pcb(const Params P, const bf16* __restrict__ x, int T, int Q, int bpc, int part0) {
  extern __shared__ float s_tab[];                      // [2 books][2][K][32]
  const int K = P.K;
  float* s_cbf = s_tab + (size_t)4 * K * 32;            // [2 books][K][8] code words as fp32
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const int combo = blockIdx.x / bpc, sub = blockIdx.x - combo * bpc;
  const int t = combo / Q, q = combo - t * Q;
  const int nb = P.H / 8;

  // ---- the part that needs the token only: both books as fp32, then this piece's table ----------
  for (int i = tid; i < 2 * K; i += blockDim.x) {
    const int book = i / K, k = i - book * K;
    const uint4 cw = __ldg((book ? P.up.codebook : P.gate.codebook) + k);
    float f[8];
    unpack8(cw, f);
    float4* dst = reinterpret_cast<float4*>(s_cbf + (size_t)i * 8);
    dst[0] = make_float4(f[0], f[1], f[2], f[3]);
    dst[1] = make_float4(f[4], f[5], f[6], f[7]);
  }
  float xb[2][8];
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    const int b = q * kPcbPiece + 2 * lane + j;
    uint4 xv = make_uint4(0, 0, 0, 0);
    if (b < nb) xv = __ldg(reinterpret_cast<const uint4*>(x + (size_t)t * P.H) + b);
    unpack8(xv, xb[j]);
  }
  __syncthreads();
  for (int i = warp; i < 2 * K; i += nwarps) {          // entry (book, k) of this lane's two blocks
    const float4 c0 = *reinterpret_cast<const float4*>(s_cbf + (size_t)i * 8);
    const float4 c1 = *reinterpret_cast<const float4*>(s_cbf + (size_t)i * 8 + 4);
    const float cf[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
    const int book = i / K, k = i - book * K;
#pragma unroll
    for (int j = 0; j < 2; ++j) s_tab[((size_t)(book * 2 + j) * K + k) * 32 + lane] = dot8(cf, xb[j], 0.f);
  }
  __syncthreads();

  pdl_wait();      // the routing lists (k_gateup_lr) are complete
  pdl_launch();

  // ---- the token's (slot, 16-row batch) pairs, this block's share of them -------------------------
  const int n_slots = P.k + P.S, n_pos = T * n_slots;
  const int per_slot = P.I / kPcbRows, n_batches = n_slots * per_slot;
  const int b_begin = (int)((long long)n_batches * sub / bpc), b_end = (int)((long long)n_batches * (sub + 1) / bpc);
  const uint8_t* idx_g = static_cast<const uint8_t*>(P.gate.idx);
  const uint8_t* idx_u = static_cast<const uint8_t*>(P.up.idx);
  const int bcol = q * kPcbPiece + 2 * lane;            // first of this lane's two blocks
  const bool live = bcol < nb;                          // H / 8 is even: both blocks or none
  const float* tab_g = s_tab + lane;
  const float* tab_u = s_tab + (size_t)2 * K * 32 + lane;

  auto fetch = [&](int batch, uint32_t (&pr)[kPcbRows]) {   // index pairs of the batch's rows: gate | up << 16
    const int s = batch / per_slot, i0 = (batch - s * per_slot) * kPcbRows;
    const int e = s < P.k ? __ldcg(P.topk_id + t * P.k + s) : P.E + (s - P.k);
    const size_t base = ((size_t)e * P.I + i0) * nb + bcol;
#pragma unroll
    for (int rr = 0; rr < kPcbRows; ++rr) {
      uint32_t pg = 0, pu = 0;
      if (live) {
        pg = __ldg(reinterpret_cast<const unsigned short*>(idx_g + base + (size_t)rr * nb));
        pu = __ldg(reinterpret_cast<const unsigned short*>(idx_u + base + (size_t)rr * nb));
      }
      pr[rr] = pg | (pu << 16);
    }
  };

  uint32_t cur[kPcbRows], nxt[kPcbRows];
  int batch = b_begin + warp;
  if (batch < b_end) fetch(batch, cur);
  for (; batch < b_end; batch += nwarps) {
    const bool more = batch + nwarps < b_end;
    if (more) fetch(batch + nwarps, nxt);
    float v[32];
#pragma unroll
    for (int rr = 0; rr < kPcbRows; ++rr) {
      const uint32_t pr = cur[rr];
      v[rr] = tab_g[(pr & 0xffu) * 32] + tab_g[(size_t)K * 32 + ((pr >> 8) & 0xffu) * 32];
      v[kPcbRows + rr] = tab_u[((pr >> 16) & 0xffu) * 32] + tab_u[(size_t)K * 32 + (pr >> 24) * 32];
    }
    warp_transpose_sum32(v, lane);
    const int s = batch / per_slot, i0 = (batch - s * per_slot) * kPcbRows;
    const int pos = __ldcg(P.inv_pos + t * n_slots + s);
    float* dst = (lane < kPcbRows ? P.gpart : P.upart) + ((size_t)(part0 + q) * n_pos + pos) * P.I + i0 + (lane & (kPcbRows - 1));
    *dst = v[0];
#pragma unroll
    for (int rr = 0; rr < kPcbRows; ++rr) cur[rr] = nxt[rr];
  }
}

}  // namespace
