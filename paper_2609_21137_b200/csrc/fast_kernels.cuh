// Tensor-core kernels of the decode layer.
//
// Design.  Every projection here is "eight output rows of one expert times up to eight token
// vectors", with the contraction cut into slices of 32 blocks (256 values).  One warp owns one
// slice: it keeps the slice of the activations as mma A fragments in registers for as long as
// the work group does not change, and for each row tile it
//     reads 16 bytes of indices (8 code-word ids of row g) that it prefetched into its own
//     shared-memory ring with cp.async several tiles earlier,
//     fetches the 8 code words from the shared-memory code book (one 16-byte read each),
//     and feeds each code word straight into two mma.sync.m16n8k16 as the B fragment.
// The k order inside an mma is free as long as A and B agree, so the fragment layout is chosen
// such that a thread's B registers of two consecutive mma's are exactly one 16-byte code word
// and its A registers are exactly the matching 16-byte activation block: no unpacking, no
// shuffles, no FMAs on the CUDA cores.  Token rows 8..15 of the m16 tile are zero; an expert
// with more than eight tokens is split into work groups of at most eight.
// The low-rank term (Eq. 1) joins the same accumulator as more k: B = a row of the private
// factor, A = z split into bf16 hi + lo so that nothing is lost against fp32.
// The warps of a team (one per slice) add their partial tiles through shared memory in a fixed
// order; nothing uses floating-point atomics, so results repeat bit for bit.
//
// Kernel chain of a call, linked by programmatic dependent launch (each kernel starts its
// routing-independent prologue while its predecessor drains):
//   k_router_z_pdl -> k_gateup_mma (routing redone in every block from the logits)
//                  -> [k_zdown_pdl] -> k_down_mma -> k_combine
#pragma once
#include "common.cuh"

namespace {

constexpr int kFastThreads = 512;
constexpr int kDenseThreads = 384;   // dense gate/up: weight tiles in flight need more registers per thread
constexpr int kDownThreads = 384;    // down: hi + lo activation fragments need 64 registers per thread
constexpr int kGroupTokens = 8;      // tokens of one work group = live rows of the m16 tile
constexpr int kMaxDepth = 4;

// Phase stamps cost instructions in the tile loops, so they are compiled in only for tracing builds
// (nvcc -DMOE_VQLR_TRACE); the phase-clock query then returns real data.
#ifdef MOE_VQLR_TRACE
#define TRACE_STAMP(kern, k) stamp(P.clk, P.clk_blocks, kern, k)
#else
#define TRACE_STAMP(kern, k) ((void)0)
#endif

__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void team_sync(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// D += A * B with A rows 8..15 zero.  a0 = A[g][2c..2c+1], a2 = A[g][2c+8..2c+9],
// b0 = B[2c..2c+1][g], b1 = B[2c+8..2c+9][g]; d0 = D[g][2c], d1 = D[g][2c+1] (g = lane/4, c = lane%4).
__device__ __forceinline__ void mma_tok8(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
  const uint32_t zero = 0u;
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(zero), "r"(a2), "r"(zero), "r"(b0), "r"(b1));
}

// One 16-byte weight block w (8 bf16 along k) against the matching activation block a.
__device__ __forceinline__ void mma_block(float (&d)[4], const uint4& a, const uint4& w) {
  mma_tok8(d, a.x, a.y, w.x, w.y);
  mma_tok8(d, a.z, a.w, w.z, w.w);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// Split eight fp32 values into bf16 hi and lo blocks: v = hi + lo up to 2^-17 relative.
__device__ __forceinline__ void split_hi_lo(const float4& p0, const float4& p1, uint4& hi, uint4& lo) {
  const float v[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
  uint32_t h[4], l[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    h[q] = pack_bf16(v[2 * q], v[2 * q + 1]);
    const float r0 = v[2 * q] - bf_lo(h[q]), r1 = v[2 * q + 1] - bf_hi(h[q]);
    l[q] = pack_bf16(r0, r1);
  }
  hi = make_uint4(h[0], h[1], h[2], h[3]);
  lo = make_uint4(l[0], l[1], l[2], l[3]);
}

template <typename IdxT>
__device__ __forceinline__ void unpack_idx8(const uint4& raw, uint32_t (&id)[8]);
template <>
__device__ __forceinline__ void unpack_idx8<uint16_t>(const uint4& v, uint32_t (&id)[8]) {
  id[0] = v.x & 0xffffu; id[1] = v.x >> 16; id[2] = v.y & 0xffffu; id[3] = v.y >> 16;
  id[4] = v.z & 0xffffu; id[5] = v.z >> 16; id[6] = v.w & 0xffffu; id[7] = v.w >> 16;
}
template <>
__device__ __forceinline__ void unpack_idx8<uint8_t>(const uint4& v, uint32_t (&id)[8]) {
  id[0] = v.x & 0xffu; id[1] = (v.x >> 8) & 0xffu; id[2] = (v.x >> 16) & 0xffu; id[3] = v.x >> 24;
  id[4] = v.y & 0xffu; id[5] = (v.y >> 8) & 0xffu; id[6] = (v.y >> 16) & 0xffu; id[7] = v.y >> 24;
}

// Eight indices of one row starting at block b0 (a multiple of 8): 16 bytes of uint16 or 8 of uint8.
template <typename IdxT>
__device__ __forceinline__ uint4 load_idx_raw(const IdxT* p) {
  if (sizeof(IdxT) == 2) return __ldg(reinterpret_cast<const uint4*>(p));
  const uint2 v = __ldg(reinterpret_cast<const uint2*>(p));
  return make_uint4(v.x, v.y, 0u, 0u);
}

// ---------------------------------------------------------------------------------------------
// Asynchronous copies: every warp streams the bytes it will need (indices, factor rows, dense
// weight rows) into a private shared-memory ring several tiles ahead, so that HBM latency is
// hidden without holding the data in registers.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void cp_async16(void* smem, const void* gptr) {
  const uint32_t sa = (uint32_t)__cvta_generic_to_shared(smem);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(sa), "l"(gptr) : "memory");
}
__device__ __forceinline__ void cp_async8(void* smem, const void* gptr) {
  const uint32_t sa = (uint32_t)__cvta_generic_to_shared(smem);
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(sa), "l"(gptr) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// waits until at most `pending` of this thread's copy groups are still in flight
__device__ __forceinline__ void cp_async_wait_pending(int pending) {
  switch (pending) {
    case 0: asm volatile("cp.async.wait_group 0;" ::: "memory"); break;
    case 1: asm volatile("cp.async.wait_group 1;" ::: "memory"); break;
    case 2: asm volatile("cp.async.wait_group 2;" ::: "memory"); break;
    default: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
  }
}
template <typename IdxT>
__device__ __forceinline__ void cp_async_idx8(uint4* smem, const IdxT* gptr) {
  if (sizeof(IdxT) == 2) cp_async16(smem, gptr); else cp_async8(smem, gptr);
}
template <typename IdxT>
__device__ __forceinline__ uint4 ring_idx8(const uint4* smem) {
  if (sizeof(IdxT) == 2) return *smem;
  const uint2 v = *reinterpret_cast<const uint2*>(smem);
  return make_uint4(v.x, v.y, 0u, 0u);
}

// How one projection stage is cut up (computed on the host, see plan_stage()).
struct StagePlan {
  int nb;          // blocks per weight row = in_dim / 8
  int n_slices;    // ceil(nb / 32)
  int team_warps;  // warps that share one row tile
  int n_teams;     // teams per block
  int tiles;       // row tiles per expert = out_dim / 8
  int n_lr;        // groups of 32 ranks = ceil(r / 32), 0 without a low-rank term
  int depth;       // tiles each warp keeps in flight in its shared-memory ring (2..4)
  int batch;       // row tiles a team finishes between two of its barriers (1..4)
};

// ---------------------------------------------------------------------------------------------
// Routing inside a block.  One warp per token finds the k best experts by k rounds of warp
// arg-max in the order (logit descending, id ascending) and turns the selected logits into
// affinities; then all threads sort the (token, slot) pairs by (expert, token) with a counting
// scan and cut them into work groups: all pairs of one expert, at most eight per group.
// ---------------------------------------------------------------------------------------------
struct RouteSmem {
  float* logit;     // [T][E]
  int* sel_id;      // [T][k]
  float* w;         // [T][k]
  int* sort_e;      // [T*k]  pairs sorted by (expert, token)
  int* sort_j;      // [T*k]  position of the pair inside its expert's run
  int* sort_c;      // [T*k]  length of that run
  int* pair_token;  // [T*(k+S)]
  int* grp_e;       // [T*(k+S)] work groups: expert, first pair position, pairs (<= 8)
  int* grp_off;
  int* grp_cnt;
  int* warp_cnt;    // [32]
  int* n_grp;       // [1]
};

__host__ __device__ inline size_t route_smem_bytes(int T, int E, int k, int S) {
  const size_t n = (size_t)T * k, m = (size_t)T * (k + S);
  size_t b = (size_t)T * E * 4 + n * 8 + n * 12 + m * 16 + 32 * 4 + 16;
  return (b + 15) / 16 * 16;
}

__device__ inline RouteSmem carve_route(char* base, int T, int E, int k, int S) {
  const size_t n = (size_t)T * k, m = (size_t)T * (k + S);
  RouteSmem r;
  r.logit = reinterpret_cast<float*>(base); base += (size_t)T * E * 4;
  r.sel_id = reinterpret_cast<int*>(base); base += n * 4;
  r.w = reinterpret_cast<float*>(base); base += n * 4;
  r.sort_e = reinterpret_cast<int*>(base); base += n * 4;
  r.sort_j = reinterpret_cast<int*>(base); base += n * 4;
  r.sort_c = reinterpret_cast<int*>(base); base += n * 4;
  r.pair_token = reinterpret_cast<int*>(base); base += m * 4;
  r.grp_e = reinterpret_cast<int*>(base); base += m * 4;
  r.grp_off = reinterpret_cast<int*>(base); base += m * 4;
  r.grp_cnt = reinterpret_cast<int*>(base); base += m * 4;
  r.warp_cnt = reinterpret_cast<int*>(base); base += 32 * 4;
  r.n_grp = reinterpret_cast<int*>(base);
  return r;
}

// Order-preserving map float -> uint32 (and back): a > b as floats <=> key(a) > key(b) as
// unsigned; +0 and -0 share a key so that they tie like the floats do.
__device__ __forceinline__ unsigned int logit_key(float v) {
  const unsigned int u = __float_as_uint(v == 0.f ? 0.f : v);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_logit(unsigned int key) {
  return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

// write_global: this block also publishes the routing for the later kernels of the chain;
// want_dbg: it additionally fills counts / offsets (only read back by the debug copies).
__device__ void route_in_block(const Params& P, int T, const RouteSmem& R, bool write_global, bool want_dbg) {
  const int E = P.E, k = P.k, S = P.S;
  const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarp = nthr >> 5;
  const int n_pairs = T * k;
  TRACE_STAMP(1, 0);
  for (int i = tid; i < T * E; i += nthr) R.logit[i] = __ldcg(P.logits + i);
  __syncthreads();
  TRACE_STAMP(1, 1);
  // ---- top-k and affinities, one warp per token -------------------------------------------
  // Logits become order-preserving unsigned keys, so that one redux.sync finds the warp maximum
  // and a second one the lowest expert id among the lanes that hold it.
  for (int t = warp; t < T; t += nwarp) {
    const float* row = R.logit + t * E;
    unsigned int taken = 0;          // bit j: expert lane + 32 j already selected (E <= 1024)
    unsigned int sel_key = 0;
    int sel_e = 0;
    if (E <= 256) {                  // keys live in registers
      unsigned int key[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) key[j] = lane + 32 * j < E ? logit_key(row[lane + 32 * j]) : 0u;
      for (int s = 0; s < k; ++s) {
        unsigned int bk = 0;         // key 0 is below every finite logit's key
        int bi = 0x7fffffff;
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (!((taken >> j) & 1u) && key[j] > bk) { bk = key[j]; bi = lane + 32 * j; }   // ascending e: '>' keeps the lower id
        const unsigned int mk = __reduce_max_sync(0xffffffffu, bk);
        int win = __reduce_min_sync(0xffffffffu, bk == mk ? bi : 0x7fffffff);
        if (win >= E) win = s;       // only NaN / -inf left: stay in bounds
        if (lane == (win & 31)) taken |= 1u << (win >> 5);
        if (lane == s) { sel_key = mk; sel_e = win; }
      }
    } else {
      for (int s = 0; s < k; ++s) {
        unsigned int bk = 0;
        int bi = 0x7fffffff;
        for (int e = lane, j = 0; e < E; e += 32, ++j) {
          const unsigned int key = logit_key(row[e]);
          if (!((taken >> j) & 1u) && key > bk) { bk = key; bi = e; }
        }
        const unsigned int mk = __reduce_max_sync(0xffffffffu, bk);
        int win = __reduce_min_sync(0xffffffffu, bk == mk ? bi : 0x7fffffff);
        if (win >= E) win = s;
        if (lane == (win & 31)) taken |= 1u << (win >> 5);
        if (lane == s) { sel_key = mk; sel_e = win; }
      }
    }
    const float sel_l = key_logit(sel_key);
    const float lmax = __shfl_sync(0xffffffffu, sel_l, 0);
    const float ev = lane < k ? expf(sel_l - lmax) : 0.f;
    float denom = ev;
    if (!P.renorm)
      for (int e = lane, j = 0; e < E; e += 32, ++j)
        if (!((taken >> j) & 1u) && row[e] != -INFINITY) denom += expf(row[e] - lmax);
    denom = warp_sum(denom);
    const float aff = ev / denom;
    if (lane < k) {
      R.sel_id[t * k + lane] = sel_e;
      R.w[t * k + lane] = aff;
    }
    if (T == 1) {
      // a single token: its k experts are k groups of one pair, ordered by expert id; the same
      // warp finishes the routing without another block-wide pass
      int pos = 0;
      for (int s2 = 0; s2 < k; ++s2) pos += __shfl_sync(0xffffffffu, sel_e, s2) < sel_e;
      if (lane < k) {
        R.pair_token[pos] = 0;
        R.grp_e[pos] = sel_e; R.grp_off[pos] = pos; R.grp_cnt[pos] = 1;
        if (write_global) {
          P.pair_token[pos] = 0; P.pair_slot[pos] = lane; P.pair_w[pos] = aff; P.inv_pos[lane] = pos;
          P.grp_e[pos] = sel_e; P.grp_off[pos] = pos; P.grp_cnt[pos] = 1;
          P.topk_id[lane] = sel_e; P.topk_w[lane] = aff;
          if (want_dbg) { /* counts / offsets are filled below */ }
        }
      }
      for (int s2 = lane; s2 < S; s2 += 32) {
        R.pair_token[k + s2] = 0;
        R.grp_e[k + s2] = E + s2; R.grp_off[k + s2] = k + s2; R.grp_cnt[k + s2] = 1;
        if (write_global) {
          P.pair_token[k + s2] = 0; P.pair_slot[k + s2] = k + s2; P.pair_w[k + s2] = 1.f; P.inv_pos[k + s2] = k + s2;
          P.grp_e[k + s2] = E + s2; P.grp_off[k + s2] = k + s2; P.grp_cnt[k + s2] = 1;
        }
      }
      if (lane == 0) { *R.n_grp = k + S; if (write_global) *P.grp_n = k + S; }
    }
  }
  __syncthreads();
  if (T == 1) {
    if (write_global && want_dbg) {
      for (int e = tid; e < E; e += nthr) P.counts[e] = 0;
      __syncthreads();
      if (tid < k) P.counts[R.sel_id[tid]] = 1;
      __syncthreads();
      if (tid == 0) {
        int run = 0;
        for (int e = 0; e < E; ++e) { P.offsets[e] = run; run += P.counts[e]; }
        P.offsets[E] = run;
      }
    }
    return;
  }
  TRACE_STAMP(1, 2);
  // ---- sort the pairs by (expert, token): four lanes share a pair and scan a quarter each ---
  for (int q0 = 0; q0 < n_pairs; q0 += nthr >> 2) {       // uniform trip count for the shuffles
    const int q = q0 + (tid >> 2);
    const bool live = q < n_pairs;
    const int e = live ? R.sel_id[q] : 0;
    int lt = 0, eq_before = 0, eq_total = 0;
    if (live)
      for (int q2 = tid & 3; q2 < n_pairs; q2 += 4) {
        const int e2 = R.sel_id[q2];
        lt += e2 < e;
        eq_total += e2 == e;
        eq_before += (e2 == e) && (q2 < q);                // same expert: pair order = token order
      }
    lt += __shfl_xor_sync(0xffffffffu, lt, 1);        lt += __shfl_xor_sync(0xffffffffu, lt, 2);
    eq_before += __shfl_xor_sync(0xffffffffu, eq_before, 1);  eq_before += __shfl_xor_sync(0xffffffffu, eq_before, 2);
    eq_total += __shfl_xor_sync(0xffffffffu, eq_total, 1);    eq_total += __shfl_xor_sync(0xffffffffu, eq_total, 2);
    if (live && (tid & 3) == 0) {
      const int pos = lt + eq_before, t = q / k, s = q - t * k;
      R.sort_e[pos] = e; R.sort_j[pos] = eq_before; R.sort_c[pos] = eq_total;
      R.pair_token[pos] = t;
      if (write_global) { P.pair_token[pos] = t; P.pair_slot[pos] = s; P.pair_w[pos] = R.w[q]; P.inv_pos[t * (k + S) + s] = pos; }
    }
  }
  for (int q = tid; q < S * T; q += nthr) {                 // shared experts: every token, weight 1
    R.pair_token[n_pairs + q] = q % T;
    if (write_global) {
      P.pair_token[n_pairs + q] = q % T; P.pair_slot[n_pairs + q] = k + q / T; P.pair_w[n_pairs + q] = 1.f;
      P.inv_pos[(q % T) * (k + S) + k + q / T] = n_pairs + q;
    }
  }
  __syncthreads();
  TRACE_STAMP(1, 3);
  // ---- work groups: a new group starts at every eighth pair of an expert's run -------------
  int base = 0;
  for (int p0 = 0; p0 < n_pairs; p0 += nthr) {
    const int pos = p0 + tid;
    const bool first = pos < n_pairs && (R.sort_j[pos] % kGroupTokens) == 0;
    const unsigned int bal = __ballot_sync(0xffffffffu, first);
    if (lane == 0) R.warp_cnt[warp] = __popc(bal);
    __syncthreads();
    int before = base;
    for (int w = 0; w < warp; ++w) before += R.warp_cnt[w];
    if (first) {
      const int gi = before + __popc(bal & ((1u << lane) - 1u));
      R.grp_e[gi] = R.sort_e[pos];
      R.grp_off[gi] = pos;
      R.grp_cnt[gi] = min(kGroupTokens, R.sort_c[pos] - R.sort_j[pos]);
    }
    for (int w = 0; w < nwarp; ++w) base += R.warp_cnt[w];
    __syncthreads();
  }
  const int sh_groups = (T + kGroupTokens - 1) / kGroupTokens;
  for (int q = tid; q < S * sh_groups; q += nthr) {
    const int s = q / sh_groups, pg = q - s * sh_groups;
    R.grp_e[base + q] = E + s;
    R.grp_off[base + q] = n_pairs + s * T + pg * kGroupTokens;
    R.grp_cnt[base + q] = min(kGroupTokens, T - pg * kGroupTokens);
  }
  if (tid == 0) *R.n_grp = base + S * sh_groups;
  __syncthreads();
  TRACE_STAMP(1, 4);
  if (write_global) {
    const int n_grp = *R.n_grp;
    for (int i = tid; i < n_pairs; i += nthr) { P.topk_id[i] = R.sel_id[i]; P.topk_w[i] = R.w[i]; }
    for (int i = tid; i < n_grp; i += nthr) { P.grp_e[i] = R.grp_e[i]; P.grp_off[i] = R.grp_off[i]; P.grp_cnt[i] = R.grp_cnt[i]; }
    if (tid == 0) *P.grp_n = n_grp;
    if (want_dbg) {           // counts / offsets of the E routed experts (off the hot path)
      for (int e = tid; e < E; e += nthr) P.counts[e] = 0;
      __syncthreads();
      for (int pos = tid; pos < n_pairs; pos += nthr)
        if (R.sort_j[pos] == 0) P.counts[R.sort_e[pos]] = R.sort_c[pos];
      __syncthreads();
      if (tid == 0) {
        int run = 0;
        for (int e = 0; e < E; ++e) { P.offsets[e] = run; run += P.counts[e]; }
        P.offsets[E] = run;
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// k_router_z_pdl: head of the chain.  One warp per (row of [router_w ; basis_gate ; basis_up],
// group of four tokens).  Per (row, token) the summation order is the one of k_router_z
// (lane-strided 16-byte chunks, sequential FMAs inside a chunk, xor butterfly), so identical
// router rows give bitwise identical logits.
// ---------------------------------------------------------------------------------------------
constexpr int kRouterWarps = 2;

__global__ void __launch_bounds__(32 * kRouterWarps) k_router_z_pdl(const Params P, const bf16* __restrict__ x, int T) {
  pdl_wait();      // the previous call's kernels may still read logits / z
  pdl_launch();
  const int lane = threadIdx.x & 31;
  const int unit = blockIdx.x * kRouterWarps + (threadIdx.x >> 5);
  const int n_rows = P.E + P.n_zrows;
  const int n_groups = (T + kTokGroup - 1) / kTokGroup;
  if (unit >= n_rows * n_groups) return;
  const int row = unit / n_groups, t0 = (unit - row * n_groups) * kTokGroup;
  const bf16* wrow;
  float* dst;
  int dst_stride;
  float bias = 0.f;
  if (row < P.E) {
    wrow = P.router_w + (size_t)row * P.H;
    dst = P.logits + row;
    dst_stride = P.E;
    if (P.router_bias) bias = P.router_bias[row];
  } else {
    const int q = row - P.E;
    const int slot = q / P.r, rho = q - slot * P.r;
    const bf16* basis = (slot == P.gate.zslot && P.gate.basis) ? P.gate.basis : P.up.basis;
    wrow = basis + (size_t)rho * P.H;
    dst = P.z + slot * P.r + rho;
    dst_stride = 2 * P.r;
  }
  const int nchunk = P.H / 8;
  const uint4* w4 = reinterpret_cast<const uint4*>(wrow);
  const int nt = min(kTokGroup, T - t0);
  float acc[kTokGroup] = {0.f, 0.f, 0.f, 0.f};
  for (int c0 = 0; c0 < nchunk; c0 += 32 * 4) {          // four chunks per lane in flight
    uint4 wv[4], xv[4][kTokGroup];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int c = c0 + q * 32 + lane;
      wv[q] = c < nchunk ? __ldg(w4 + c) : make_uint4(0, 0, 0, 0);
#pragma unroll
      for (int tt = 0; tt < kTokGroup; ++tt)
        xv[q][tt] = (c < nchunk && tt < nt) ? __ldg(reinterpret_cast<const uint4*>(x + (size_t)(t0 + tt) * P.H) + c)
                                            : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      if (c0 + q * 32 + lane < nchunk) {
        float wf[8];
        unpack8(wv[q], wf);
#pragma unroll
        for (int tt = 0; tt < kTokGroup; ++tt) {
          float xf[8];
          unpack8(xv[q][tt], xf);
          acc[tt] = dot8(wf, xf, acc[tt]);
        }
      }
    }
  }
#pragma unroll
  for (int tt = 0; tt < kTokGroup; ++tt) {
    const float sum = warp_sum(acc[tt]);
    if (lane == 0 && tt < nt) dst[(size_t)(t0 + tt) * dst_stride] = sum + bias;
  }
}

// Splits `total` tiles evenly over `parts` teams: first tile of team `idx`.
__device__ __forceinline__ int split_begin(int total, int parts, int idx) {
  return (int)(((long long)total * idx) / parts);
}

// ---------------------------------------------------------------------------------------------
// k_gateup_mma
// ---------------------------------------------------------------------------------------------
struct GuLayout {         // byte offsets into dynamic shared memory
  size_t cb_u, x, ring, fring, z, part, meta, route, total;
};

__host__ __device__ inline GuLayout gu_layout(int K, int n_books, int T, int H, int r, const StagePlan& pl,
                                              int warps, int E, int k, int S) {
  GuLayout L;
  size_t o = 0;
  L.cb_u = n_books == 2 ? (size_t)K * 16 : 0;
  o = (size_t)n_books * K * 16;
  L.x = o;      o += (size_t)T * (H / 8 + 1) * 16;
  L.ring = o;   o += (size_t)warps * pl.depth * 2 * 32 * 16;
  L.fring = o;  o += (size_t)pl.n_teams * (pl.n_lr > 0 ? pl.n_lr : 0) * pl.depth * 2 * 32 * 16;
  L.z = o;      o += (size_t)2 * T * 2 * ((r + 7) / 8) * 16;            // hi and lo blocks of z
  L.part = o;   o += (size_t)2 * pl.n_teams * pl.batch * 2 * pl.team_warps * 32 * 8;
  L.meta = o;   o += (size_t)2 * pl.n_teams * pl.batch * 16;
  L.route = o;  o += route_smem_bytes(T, E, k, S);
  L.total = o;
  return L;
}

template <typename IdxT, bool DENSE>
__global__ void __launch_bounds__(DENSE ? kDenseThreads : kFastThreads, 1)
k_gateup_mma(const Params P, const bf16* __restrict__ x, int T, const StagePlan pl, int n_books, int want_dbg) {
  extern __shared__ uint4 s_u4[];
  char* s_base = reinterpret_cast<char*>(s_u4);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, c = lane & 3;
  const int nb = pl.nb, xs = nb + 1, D = pl.depth, rb = (P.r + 7) / 8;
  const GuLayout L = gu_layout(P.K, n_books, T, P.H, P.r, pl, blockDim.x >> 5, P.E, P.k, P.S);
  uint4* s_cb_g = s_u4;
  uint4* s_cb_u = reinterpret_cast<uint4*>(s_base + L.cb_u);
  uint4* s_x = reinterpret_cast<uint4*>(s_base + L.x);
  uint4* s_ring = reinterpret_cast<uint4*>(s_base + L.ring);
  uint4* s_fring = reinterpret_cast<uint4*>(s_base + L.fring);
  uint4* s_zh = reinterpret_cast<uint4*>(s_base + L.z);          // [T][2][rb]
  uint4* s_zl = s_zh + (size_t)T * 2 * rb;
  float2* s_part = reinterpret_cast<float2*>(s_base + L.part);
  int4* s_meta = reinterpret_cast<int4*>(s_base + L.meta);     // [buf][team][tile of the batch] (pair offset, tile, tokens)
  const RouteSmem R = carve_route(s_base + L.route, T, P.E, P.k, P.S);

  TRACE_STAMP(0, 0);
  // ---- routing-independent prologue: code books and tokens start streaming into shared memory
  if (!DENSE) {
    for (int i = tid; i < P.K; i += blockDim.x) cp_async16(s_cb_g + i, P.gate.codebook + i);
    if (n_books == 2)
      for (int i = tid; i < P.K; i += blockDim.x) cp_async16(s_cb_u + i, P.up.codebook + i);
  }
  {
    const uint4* x4 = reinterpret_cast<const uint4*>(x);
    for (int i = tid; i < T * nb; i += blockDim.x) {
      const int t = i / nb, b = i - t * nb;
      cp_async16(s_x + t * xs + b, x4 + i);
    }
  }
  cp_async_commit();
  TRACE_STAMP(0, 1);
  pdl_wait();      // logits and z of this call are complete
  TRACE_STAMP(0, 2);
  if (pl.n_lr > 0)
    for (int i = tid; i < T * 2 * rb; i += blockDim.x) {      // z as bf16 hi / lo blocks
      const float* zp = P.z + (size_t)i * 8;                   // z is [T][2][r], r a multiple of 8
      split_hi_lo(__ldcg(reinterpret_cast<const float4*>(zp)), __ldcg(reinterpret_cast<const float4*>(zp + 4)), s_zh[i], s_zl[i]);
    }
  route_in_block(P, T, R, blockIdx.x == 0, want_dbg != 0);
  TRACE_STAMP(1, 5);
  pdl_launch();
  cp_async_wait_pending(0);       // this thread's share of code book and tokens has landed ...
  __syncthreads();                // ... and so has everybody else's
  TRACE_STAMP(0, 3);

  const int team = warp / pl.team_warps, wi = warp - team * pl.team_warps;
  const int team_threads = pl.team_warps * 32;
  const int n_grp = *R.n_grp;
  const int U = n_grp * pl.tiles;
  const int G = gridDim.x * pl.n_teams, tau = blockIdx.x * pl.n_teams + team;
  const int u_begin = team < pl.n_teams ? split_begin(U, G, tau) : 0;
  const int n_my = team < pl.n_teams ? split_begin(U, G, tau + 1) - u_begin : 0;
  const bool spw_one = pl.n_slices <= pl.team_warps;         // one slice per warp: fragments stay put
  const bool ringed = !DENSE && spw_one;
  // low-rank group handled by this warp (groups are dealt from the last warp of the team down)
  const int lr_group = pl.team_warps - 1 - wi;
  const bool has_lr = lr_group < pl.n_lr;                    // n_lr is 0 for a dense projection
  const int b_first = wi * 32 + 8 * c, rho_first = lr_group * 32 + 8 * c;
  const bool idx_live = b_first < nb, fac_live = has_lr && rho_first < P.r;

  // per-lane bases: row g of a tile, this warp's first block group / rank group
  const IdxT* idx_g = static_cast<const IdxT*>(P.gate.idx) + (size_t)g * nb + b_first;
  const IdxT* idx_u = static_cast<const IdxT*>(P.up.idx) + (size_t)g * nb + b_first;
  const bf16* fac_gp = P.gate.factor + (size_t)g * P.r + rho_first;
  const bf16* fac_up = P.up.factor + (size_t)g * P.r + rho_first;
  uint4* ring = s_ring + (size_t)warp * D * 2 * 32 + lane;                            // [slot][proj][lane]
  uint4* fring = s_fring + (size_t)(team * pl.n_lr + (has_lr ? lr_group : 0)) * D * 2 * 32 + lane;

  // (group, tile) of the next tile to prefetch and of the tile being computed advance in step
  int pf_grp = n_my > 0 ? u_begin / pl.tiles : 0, pf_jt = n_my > 0 ? u_begin - pf_grp * pl.tiles : 0;
  int cur_grp = pf_grp, cur_jt = pf_jt;
  int pf_slot = 0, cur_slot = 0;
  auto issue = [&]() {
    const size_t row0 = (size_t)R.grp_e[pf_grp] * P.I + pf_jt * 8;     // first row of the tile
    if (ringed && idx_live) {
      cp_async_idx8<IdxT>(ring + (pf_slot * 2 + 0) * 32, idx_g + row0 * nb);
      cp_async_idx8<IdxT>(ring + (pf_slot * 2 + 1) * 32, idx_u + row0 * nb);
    }
    if (fac_live) {
      cp_async16(fring + (pf_slot * 2 + 0) * 32, fac_gp + row0 * P.r);
      cp_async16(fring + (pf_slot * 2 + 1) * 32, fac_up + row0 * P.r);
    }
    if (++pf_jt == pl.tiles) { pf_jt = 0; ++pf_grp; }
    if (++pf_slot == D) pf_slot = 0;
  };

  TRACE_STAMP(1, 6);
  uint4 fx[8];                       // activation fragments of the current slice
  int frag_grp = -1, frag_slice = -1;
  int buf = 0, r_in = 0;
  const int tid_team = tid - team * team_threads;

  for (int i = 0; i < D - 1; ++i) { if (i < n_my) issue(); cp_async_commit(); }
  TRACE_STAMP(1, 7);
  for (int i = 0; i < n_my; ++i) {
    if (i + D - 1 < n_my) issue();
    cp_async_commit();
    TRACE_STAMP(0, 4 + 3 * i);
    cp_async_wait_pending(D - 1);
    TRACE_STAMP(0, 5 + 3 * i);
    const int grp = cur_grp, jt = cur_jt, slot = cur_slot;
    if (++cur_jt == pl.tiles) { cur_jt = 0; ++cur_grp; }
    if (++cur_slot == D) cur_slot = 0;
    const int e = R.grp_e[grp], off = R.grp_off[grp], n_tok = R.grp_cnt[grp];
    const size_t row = (size_t)e * P.I + jt * 8 + g;       // this lane's weight row
    uint4 raw_g = {0, 0, 0, 0}, raw_u = {0, 0, 0, 0};
    uint4 fac_g = {0, 0, 0, 0}, fac_u = {0, 0, 0, 0};
    if (ringed && idx_live) {
      raw_g = ring_idx8<IdxT>(ring + (slot * 2 + 0) * 32);
      raw_u = ring_idx8<IdxT>(ring + (slot * 2 + 1) * 32);
    }
    if (fac_live) {
      fac_g = fring[(slot * 2 + 0) * 32];
      fac_u = fring[(slot * 2 + 1) * 32];
    }
    const int tok = g < n_tok ? R.pair_token[off + g] : -1;
    float acc_g[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    float acc_u[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    for (int sl = wi; sl < pl.n_slices; sl += pl.team_warps) {
      const int b0 = sl * 32 + (DENSE ? c : 8 * c);
      if (frag_grp != grp || frag_slice != sl) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int b = b0 + (DENSE ? 4 * j : j);
          fx[j] = (tok >= 0 && b < nb) ? s_x[tok * xs + b] : make_uint4(0, 0, 0, 0);
        }
        frag_grp = grp; frag_slice = sl;
      }
      if (DENSE) {
        const uint4* wg = reinterpret_cast<const uint4*>(P.gate.dense + row * P.H);
        const uint4* wu = reinterpret_cast<const uint4*>(P.up.dense + row * P.H);
        uint4 vg[8], vu[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int b = b0 + 4 * j;
          vg[j] = b < nb ? __ldg(wg + b) : make_uint4(0, 0, 0, 0);
          vu[j] = b < nb ? __ldg(wu + b) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) { mma_block(acc_g[j & 1], fx[j], vg[j]); mma_block(acc_u[j & 1], fx[j], vu[j]); }
      } else {
        if (!ringed) {
          if (b0 < nb) {
            raw_g = load_idx_raw<IdxT>(static_cast<const IdxT*>(P.gate.idx) + row * nb + b0);
            raw_u = load_idx_raw<IdxT>(static_cast<const IdxT*>(P.up.idx) + row * nb + b0);
          } else {
            raw_g = raw_u = make_uint4(0, 0, 0, 0);
          }
        }
        // mma.sync needs the whole warp: lanes whose group lies beyond the row run it with
        // index 0 and zero activation fragments
        uint32_t ig[8], iu[8];
        unpack_idx8<IdxT>(raw_g, ig);
        unpack_idx8<IdxT>(raw_u, iu);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          mma_block(acc_g[j & 1], fx[j], s_cb_g[ig[j]]);
          mma_block(acc_u[j & 1], fx[j], s_cb_u[iu[j]]);
        }
      }
    }
    // joint accumulation of the low-rank term: more k for the same tile
    for (int lg = lr_group; lg < pl.n_lr; lg += pl.team_warps) {
      const int rho0 = lg * 32 + 8 * c;
      uint4 fg = fac_g, fu = fac_u;
      if (lg != lr_group) {
        fg = fu = make_uint4(0, 0, 0, 0);
        if (rho0 < P.r) {
          fg = __ldg(reinterpret_cast<const uint4*>(P.gate.factor + row * P.r + rho0));
          fu = __ldg(reinterpret_cast<const uint4*>(P.up.factor + row * P.r + rho0));
        }
      }
      uint4 zgh = {0, 0, 0, 0}, zgl = {0, 0, 0, 0}, zuh = {0, 0, 0, 0}, zul = {0, 0, 0, 0};
      if (tok >= 0 && rho0 < P.r) {
        const int ig2 = (tok * 2 + P.gate.zslot) * rb + (rho0 >> 3), iu2 = (tok * 2 + P.up.zslot) * rb + (rho0 >> 3);
        zgh = s_zh[ig2]; zgl = s_zl[ig2]; zuh = s_zh[iu2]; zul = s_zl[iu2];
      }
      mma_block(acc_g[0], zgh, fg); mma_block(acc_g[1], zgl, fg);
      mma_block(acc_u[0], zuh, fu); mma_block(acc_u[1], zul, fu);
    }
    // ---- add the team's partial tiles and apply SwiGLU -----------------------------------
    TRACE_STAMP(0, 6 + 3 * i);
    const int bslot = (buf * pl.n_teams + team) * pl.batch + r_in;
    float2* part = s_part + (size_t)bslot * 2 * pl.team_warps * 32;
    part[(0 * pl.team_warps + wi) * 32 + lane] = make_float2(acc_g[0][0] + acc_g[1][0], acc_g[0][1] + acc_g[1][1]);
    part[(1 * pl.team_warps + wi) * 32 + lane] = make_float2(acc_u[0][0] + acc_u[1][0], acc_u[0][1] + acc_u[1][1]);
    if (wi == 0 && lane == 0) s_meta[bslot] = make_int4(off, jt, n_tok, 0);
    if (++r_in == pl.batch || i == n_my - 1) {
      // one barrier per batch of tiles; then the batch's outputs (64 per tile: 8 tokens x 8 rows)
      // are summed over the team's warps in a fixed order and passed through SwiGLU
      if (pl.team_warps > 1) team_sync(1 + team, team_threads); else __syncwarp();
      const int bbase = (buf * pl.n_teams + team) * pl.batch;
      for (int q = tid_team; q < r_in * 64; q += team_threads) {
        const int rt = q >> 6, m = (q >> 3) & 7, n = q & 7;   // tile of the batch, token, row
        const int4 mt = s_meta[bbase + rt];
        if (m < mt.z) {
          const float2* pt = s_part + (size_t)(bbase + rt) * 2 * pl.team_warps * 32;
          const int src = 4 * m + (n >> 1);
          float gs = 0.f, us = 0.f;
#pragma unroll 4
          for (int w = 0; w < pl.team_warps; ++w) {
            const float2 pg = pt[(0 * pl.team_warps + w) * 32 + src];
            const float2 pu = pt[(1 * pl.team_warps + w) * 32 + src];
            gs += (n & 1) ? pg.y : pg.x;
            us += (n & 1) ? pu.y : pu.x;
          }
          const float pv = gs / (1.f + expf(-gs)) * us;       // silu(g) * u
          const size_t at = (size_t)(mt.x + m) * P.I + mt.y * 8 + n;
          const bf16 hi = __float2bfloat16_rn(pv);
          P.p[at] = pv;
          P.p_hi[at] = hi;                                       // the down kernel's mma fragments
          P.p_lo[at] = __float2bfloat16_rn(pv - __bfloat162float(hi));
        }
      }
      buf ^= 1;
      r_in = 0;
    }
  }
  cp_async_wait_pending(0);
  TRACE_STAMP(0, 15);
}

// ---------------------------------------------------------------------------------------------
// k_down_mma: y[token][slot][h] for every (work group, 8-row tile of H); activations are the
// fp32 intermediates p split into bf16 hi + lo fragments.
// ---------------------------------------------------------------------------------------------
struct DnLayout {
  size_t ring, fring, part, yrow, grp, total;
  int slot_u4;      // uint4 per lane per ring slot: 1 (indices) or 8 (a dense 256-value slice of a row)
};

__host__ __device__ inline DnLayout dn_layout(int K, bool vq, const StagePlan& pl, int warps, int max_groups) {
  DnLayout L;
  size_t o = vq ? (size_t)K * 16 : 0;
  L.slot_u4 = vq ? 1 : 8;
  L.ring = o;   o += (size_t)warps * pl.depth * L.slot_u4 * 32 * 16;
  L.fring = o;  o += (size_t)pl.n_teams * (pl.n_lr > 0 ? pl.n_lr : 0) * pl.depth * 32 * 16;
  L.part = o;   o += (size_t)2 * pl.n_teams * pl.batch * pl.team_warps * 32 * 8;
  L.yrow = o;   o += (size_t)2 * pl.n_teams * pl.batch * 16;
  L.grp = o;    o += ((size_t)max_groups * 12 + 15) / 16 * 16;
  L.total = o;
  return L;
}

template <typename IdxT, bool DENSE>
__global__ void __launch_bounds__(kDownThreads, 1)
k_down_mma(const Params P, int T, const StagePlan pl) {
  extern __shared__ uint4 s_u4[];
  char* s_base = reinterpret_cast<char*>(s_u4);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, c = lane & 3;
  const int nb = pl.nb, D = pl.depth;
  const int max_groups = T * (P.k + P.S);
  const DnLayout L = dn_layout(P.K, !DENSE, pl, blockDim.x >> 5, max_groups);
  uint4* s_cb = s_u4;
  uint4* s_ring = reinterpret_cast<uint4*>(s_base + L.ring);
  uint4* s_fring = reinterpret_cast<uint4*>(s_base + L.fring);
  float2* s_part = reinterpret_cast<float2*>(s_base + L.part);
  int4* s_meta = reinterpret_cast<int4*>(s_base + L.yrow);   // [buf][team][tile of the batch] (pair offset, tile, tokens)
  int* s_grp_e = reinterpret_cast<int*>(s_base + L.grp);
  int* s_grp_off = s_grp_e + max_groups;
  int* s_grp_cnt = s_grp_off + max_groups;
  TRACE_STAMP(2, 0);
  if (!DENSE)
    for (int i = tid; i < P.K; i += blockDim.x) cp_async16(s_cb + i, P.down.codebook + i);
  cp_async_commit();
  pdl_wait();      // p (and z_d) and the routing lists are complete
  TRACE_STAMP(2, 1);
  pdl_launch();
  const int n_grp = __ldcg(P.grp_n);
  for (int i = tid; i < n_grp; i += blockDim.x) {
    s_grp_e[i] = __ldcg(P.grp_e + i); s_grp_off[i] = __ldcg(P.grp_off + i); s_grp_cnt[i] = __ldcg(P.grp_cnt + i);
  }
  cp_async_wait_pending(0);
  __syncthreads();
  TRACE_STAMP(2, 2);

  const int team = warp / pl.team_warps, wi = warp - team * pl.team_warps;
  const int team_threads = pl.team_warps * 32;
  const int tid_team = tid - team * team_threads;
  const int U = n_grp * pl.tiles;
  const int G = gridDim.x * pl.n_teams, tau = blockIdx.x * pl.n_teams + team;
  const int u_begin = team < pl.n_teams ? split_begin(U, G, tau) : 0;
  const int n_my = team < pl.n_teams ? split_begin(U, G, tau + 1) - u_begin : 0;
  const bool spw_one = pl.n_slices <= pl.team_warps;
  const bool ringed = spw_one;
  const int lr_group = pl.team_warps - 1 - wi;
  const bool has_lr = lr_group < pl.n_lr;
  const int b_first = wi * 32 + (DENSE ? c : 8 * c), rho_first = lr_group * 32 + 8 * c;
  const bool idx_live = DENSE ? (wi * 32 < nb) : (b_first < nb), fac_live = has_lr && rho_first < P.r;

  const IdxT* idx_d = static_cast<const IdxT*>(P.down.idx) + (size_t)g * nb + b_first;
  const uint4* dense_d = reinterpret_cast<const uint4*>(P.down.dense + (size_t)g * P.I) + b_first;
  const bf16* fac_dp = P.down.factor + (size_t)g * P.r + rho_first;
  uint4* ring = s_ring + (size_t)warp * D * L.slot_u4 * 32 + lane;                 // [slot][chunk][lane]
  uint4* fring = s_fring + (size_t)(team * pl.n_lr + (has_lr ? lr_group : 0)) * D * 32 + lane;

  int pf_grp = n_my > 0 ? u_begin / pl.tiles : 0, pf_jt = n_my > 0 ? u_begin - pf_grp * pl.tiles : 0;
  int cur_grp = pf_grp, cur_jt = pf_jt;
  int pf_slot = 0, cur_slot = 0;
  auto issue = [&]() {
    const size_t row0 = (size_t)s_grp_e[pf_grp] * P.H + pf_jt * 8;
    if (ringed && idx_live) {
      if (DENSE) {
        const uint4* wd = dense_d + row0 * (P.I / 8);
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (b_first + 4 * j < nb) cp_async16(ring + (pf_slot * 8 + j) * 32, wd + 4 * j);
      } else {
        cp_async_idx8<IdxT>(ring + pf_slot * 32, idx_d + row0 * nb);
      }
    }
    if (fac_live) cp_async16(fring + pf_slot * 32, fac_dp + row0 * P.r);
    if (++pf_jt == pl.tiles) { pf_jt = 0; ++pf_grp; }
    if (++pf_slot == D) pf_slot = 0;
  };

  uint4 fh[8], fl[8];
  uint4 zh = {0, 0, 0, 0}, zl = {0, 0, 0, 0};
  int frag_grp = -1, frag_slice = -1, z_grp = -1, z_lg = -1;
  int buf = 0, r_in = 0;

  for (int i = 0; i < D - 1; ++i) { if (i < n_my) issue(); cp_async_commit(); }
  TRACE_STAMP(2, 3);
  for (int i = 0; i < n_my; ++i) {
    if (i + D - 1 < n_my) issue();
    cp_async_commit();
    cp_async_wait_pending(D - 1);
    if (i < 5) TRACE_STAMP(2, 4 + 2 * i);
    const int grp = cur_grp, jt = cur_jt, slot = cur_slot;
    if (++cur_jt == pl.tiles) { cur_jt = 0; ++cur_grp; }
    if (++cur_slot == D) cur_slot = 0;
    const int e = s_grp_e[grp], off = s_grp_off[grp], n_tok = s_grp_cnt[grp];
    const size_t row = (size_t)e * P.H + jt * 8 + g;
    uint4 raw = {0, 0, 0, 0}, fac = {0, 0, 0, 0};
    if (!DENSE && ringed && idx_live) raw = ring_idx8<IdxT>(ring + slot * 32);
    if (fac_live) fac = fring[slot * 32];
    const int pos = g < n_tok ? off + g : -1;
    float acc[4][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};   // four independent chains
    for (int sl = wi; sl < pl.n_slices; sl += pl.team_warps) {
      const int b0 = sl * 32 + (DENSE ? c : 8 * c);
      if (frag_grp != grp || frag_slice != sl) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int b = b0 + (DENSE ? 4 * j : j);
          if (pos >= 0 && b < nb) {
            fh[j] = __ldcg(reinterpret_cast<const uint4*>(P.p_hi + (size_t)pos * P.I) + b);
            fl[j] = __ldcg(reinterpret_cast<const uint4*>(P.p_lo + (size_t)pos * P.I) + b);
          } else {
            fh[j] = fl[j] = make_uint4(0, 0, 0, 0);
          }
        }
        frag_grp = grp; frag_slice = sl;
      }
      if (DENSE) {
        const uint4* wd = reinterpret_cast<const uint4*>(P.down.dense + row * P.I);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int b = b0 + 4 * j;
          uint4 v = make_uint4(0, 0, 0, 0);
          if (b < nb) v = ringed ? ring[(slot * 8 + j) * 32] : __ldg(wd + b);
          mma_block(acc[j & 1], fh[j], v);
          mma_block(acc[2 + (j & 1)], fl[j], v);
        }
      } else {
        if (!ringed) raw = b0 < nb ? load_idx_raw<IdxT>(static_cast<const IdxT*>(P.down.idx) + row * nb + b0) : make_uint4(0, 0, 0, 0);
        uint32_t id[8];                      // out-of-range groups: index 0, zero fragments
        unpack_idx8<IdxT>(raw, id);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const uint4 w = s_cb[id[j]];
          mma_block(acc[j & 1], fh[j], w);
          mma_block(acc[2 + (j & 1)], fl[j], w);
        }
      }
    }
    for (int lg = lr_group; lg < pl.n_lr; lg += pl.team_warps) {
      const int rho0 = lg * 32 + 8 * c;
      uint4 f = fac;
      if (lg != lr_group)
        f = rho0 < P.r ? __ldg(reinterpret_cast<const uint4*>(P.down.factor + row * P.r + rho0)) : make_uint4(0, 0, 0, 0);
      if (z_grp != grp || z_lg != lg) {
        if (pos >= 0 && rho0 < P.r) {
          const float4* zp = reinterpret_cast<const float4*>(P.zd + (size_t)pos * P.r + rho0);
          split_hi_lo(__ldcg(zp), __ldcg(zp + 1), zh, zl);
        } else {
          zh = zl = make_uint4(0, 0, 0, 0);
        }
        z_grp = grp; z_lg = lg;
      }
      mma_block(acc[0], zh, f);
      mma_block(acc[2], zl, f);
    }
    if (i < 5) TRACE_STAMP(2, 5 + 2 * i);
    const int bslot = (buf * pl.n_teams + team) * pl.batch + r_in;
    float2* part = s_part + (size_t)bslot * pl.team_warps * 32;
    part[wi * 32 + lane] = make_float2((acc[0][0] + acc[1][0]) + (acc[2][0] + acc[3][0]), (acc[0][1] + acc[1][1]) + (acc[2][1] + acc[3][1]));
    if (wi == 0 && lane == 0) s_meta[bslot] = make_int4(off, jt, n_tok, 0);
    if (++r_in == pl.batch || i == n_my - 1) {
      if (pl.team_warps > 1) team_sync(1 + team, team_threads); else __syncwarp();
      const int bbase = (buf * pl.n_teams + team) * pl.batch;
      for (int q = tid_team; q < r_in * 64; q += team_threads) {
        const int rt = q >> 6, m = (q >> 3) & 7, n = q & 7;
        const int4 mt = s_meta[bbase + rt];
        if (m < mt.z) {
          const float2* pt = s_part + (size_t)(bbase + rt) * pl.team_warps * 32;
          const int src = 4 * m + (n >> 1);
          float sum = 0.f;
#pragma unroll 4
          for (int w = 0; w < pl.team_warps; ++w) {
            const float2 v = pt[w * 32 + src];
            sum += (n & 1) ? v.y : v.x;
          }
          P.y[(size_t)(mt.x + m) * P.H + mt.y * 8 + n] = sum;
        }
      }
      buf ^= 1;
      r_in = 0;
    }
  }
  cp_async_wait_pending(0);
  TRACE_STAMP(2, 15);
}

// z_d[pos][rho] = <basis_down[rho], p[pos]> (link of the chain between gate/up and down).
__global__ void __launch_bounds__(256) k_zdown_pdl(const Params P, int n_pos) {
  pdl_wait();
  pdl_launch();
  const int lane = threadIdx.x & 31;
  const int w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (w >= n_pos * P.r) return;
  const int pos = w / P.r, rho = w - pos * P.r;
  const uint4* brow = reinterpret_cast<const uint4*>(P.down.basis + (size_t)rho * P.I);
  const float4* prow = reinterpret_cast<const float4*>(P.p + (size_t)pos * P.I);
  float acc = 0.f;
  for (int cidx = lane; cidx < P.I / 8; cidx += 32) {
    float wf[8];
    unpack8(__ldg(brow + cidx), wf);
    const float4 p0 = __ldcg(prow + 2 * cidx), p1 = __ldcg(prow + 2 * cidx + 1);
    const float pf[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
    acc = dot8(wf, pf, acc);
  }
  acc = warp_sum(acc);
  if (lane == 0) P.zd[(size_t)pos * P.r + rho] = acc;
}

// out[t][h] = sum over slots (in slot order) of affinity * y[t][slot][h]; shared experts weigh 1.
__global__ void __launch_bounds__(256) k_combine(const Params P, bf16* __restrict__ out, int T) {
  pdl_wait();
  pdl_launch();
  const int n_slots = P.k + P.S, H2 = P.H / 2;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < T * H2; i += gridDim.x * blockDim.x) {
    const int t = i / H2, h2 = i - t * H2;
    float a0 = 0.f, a1 = 0.f;
    for (int s = 0; s < n_slots; ++s) {
      const int pos = __ldcg(P.inv_pos + t * n_slots + s);
      const float w = __ldcg(P.pair_w + pos);
      const float2 v = __ldcg(reinterpret_cast<const float2*>(P.y + (size_t)pos * P.H + 2 * h2));
      a0 = fmaf(w, v.x, a0);
      a1 = fmaf(w, v.y, a1);
    }
    *reinterpret_cast<__nv_bfloat162*>(out + (size_t)t * P.H + 2 * h2) = __floats2bfloat162_rn(a0, a1);
  }
}

}  // namespace
