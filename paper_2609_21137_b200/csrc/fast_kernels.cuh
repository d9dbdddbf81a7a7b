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
// The low-rank term (Eq. 1) is the same product with more k: B = a row of the private factor,
// A = z split into bf16 hi + lo so that nothing is lost against fp32; each group of 32 ranks is
// one more "part" next to the slices.
// Warps never wait for each other: a warp writes the partial tile of its part to global memory
// and the next kernel of the chain adds the parts in a fixed order (the SwiGLU link for gate/up,
// the combine for down).  Nothing uses floating-point atomics, so results repeat bit for bit.
//
// Kernel chain of a call, linked by programmatic dependent launch (each kernel starts its
// routing-independent prologue while its predecessor drains):
//   k_router_z_pdl -> k_gateup_mma (routing redone in every block from the logits)
//                  -> k_act_zdown (sum of parts, SwiGLU, z_d) -> k_down_mma -> k_combine
#pragma once
#include "common.cuh"

namespace {

constexpr int kFastThreads = 512;
constexpr int kDenseThreads = 384;   // dense gate/up: weight tiles in flight need more registers per thread
constexpr int kDownThreads = 384;    // down: hi + lo activation fragments need 64 registers per thread
constexpr int kGroupTokens = 8;      // tokens of one work group = live rows of the m16 tile
constexpr int kMaxDepth = 2;

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

// The same block against an activation block given as bf16 hi + lo halves: hi fills token rows
// 0..7 of the m16 tile, lo rows 8..15, so ONE pair of mma's forms both products (the tensor pipe
// issues 0.4 m16n8k16 per clock per SM, which is as scarce here as the shared-memory lookups).
// d[0], d[1]: hi product of token g, rows 2c and 2c+1; d[2], d[3]: the lo product.
__device__ __forceinline__ void mma_block_hilo(float (&d)[4], const uint4& hi, const uint4& lo, const uint4& w) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(hi.x), "r"(lo.x), "r"(hi.y), "r"(lo.y), "r"(w.x), "r"(w.y));
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(hi.z), "r"(lo.z), "r"(hi.w), "r"(lo.w), "r"(w.z), "r"(w.w));
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
    case 3: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
    case 4: asm volatile("cp.async.wait_group 4;" ::: "memory"); break;
    case 5: asm volatile("cp.async.wait_group 5;" ::: "memory"); break;
    case 6: asm volatile("cp.async.wait_group 6;" ::: "memory"); break;
    default: asm volatile("cp.async.wait_group 7;" ::: "memory"); break;
  }
}
__device__ __forceinline__ void cp_async4(void* smem, const void* gptr) {
  const uint32_t sa = (uint32_t)__cvta_generic_to_shared(smem);
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(sa), "l"(gptr) : "memory");
}
// Eight indices of a row into a 16-byte ring slot: 16 bytes of uint16, 8 of uint8, or (idx12) the
// 12 bytes of eight packed twelve-bit indices, which start on a 4-byte boundary only.
template <typename IdxT>
__device__ __forceinline__ void cp_async_idx8(uint4* smem, const IdxT* gptr, int idx12 = 0) {
  if (sizeof(IdxT) == 2) {
    if (idx12) {
      const char* g = reinterpret_cast<const char*>(gptr);
      char* d = reinterpret_cast<char*>(smem);
      cp_async4(d, g); cp_async4(d + 4, g + 4); cp_async4(d + 8, g + 8);
    } else {
      cp_async16(smem, gptr);
    }
  } else {
    cp_async8(smem, gptr);
  }
}
// The eight indices of a ring slot.
template <typename IdxT>
__device__ __forceinline__ void slot_idx8(const uint4& raw, int idx12, uint32_t (&id)[8]) {
  if (sizeof(IdxT) == 2 && idx12) unpack_idx12x8(raw.x, raw.y, raw.z, id);
  else unpack_idx8<IdxT>(raw, id);
}
template <typename IdxT>
__device__ __forceinline__ uint4 ring_idx8(const uint4* smem) {
  if (sizeof(IdxT) == 2) return *smem;
  const uint2 v = *reinterpret_cast<const uint2*>(smem);
  return make_uint4(v.x, v.y, 0u, 0u);
}

// Four-value code words (d = 4): a row's uint8 indices are read two at a time as one 16-bit
// pair (low byte = first word), i.e. with the uint16 plumbing, and the eight weights of a block are
// two 8-byte words.  The book is stored sixteen times, word i of copy c at 8-byte slot 16 i + c:
// lane l reads copy l % 16, so the sixteen lanes of a half warp never share a bank pair.
__device__ __forceinline__ uint4 lookup_d4(const uint4* s_cb, uint32_t pair, int lane) {
  const uint2* cb2 = reinterpret_cast<const uint2*>(s_cb);
  const uint2 lo = cb2[((pair & 0xffu) << 4) | (lane & 15)], hi = cb2[((pair >> 8) << 4) | (lane & 15)];
  return make_uint4(lo.x, lo.y, hi.x, hi.y);
}

// Division by a run-time constant as multiply-high and shift (the magic numbers come from the
// host): exact for 0 <= n < 2^31.  A hardware-emulated 32-bit division costs about a hundred
// clocks of dependent instructions, and the work-list arithmetic below sits on the critical path
// of a warp that has nothing else to overlap it with.
struct FastDiv {
  unsigned int mul, shr;      // mul == 0: divisor 1
};
__host__ __device__ inline FastDiv make_fastdiv(unsigned int d) {
  FastDiv f = {0u, 0u};
  if (d <= 1u) return f;
  unsigned int L = 0;
  while ((1ull << L) < d) ++L;
  const unsigned int p = 31u + L;
  f.mul = (unsigned int)(((1ull << p) + d - 1ull) / d);
  f.shr = p - 32u;
  return f;
}
__device__ __forceinline__ int fdiv(int n, const FastDiv& f) {
  return f.mul ? (int)(__umulhi((unsigned int)n, f.mul) >> f.shr) : n;
}

// How one projection stage is cut up (computed on the host, see plan_stage() / finish_plan()).
struct StagePlan {
  int nb;          // blocks per weight row = in_dim / 8
  int n_slices;    // ceil(nb / 32)
  int n_lr;        // groups of 32 ranks = ceil(r / 32), 0 without a low-rank term
  int n_parts;     // n_slices + n_lr: partial tiles that add up to one output tile
  int tiles;       // row tiles per expert = out_dim / 8
  int depth;       // tiles each warp keeps in flight in its shared-memory ring (2..4)
  int chunk;       // consecutive row tiles of one part in the work order (see Cursor)
  int x_smem;      // gate/up: tokens are staged in shared memory (else fragments come from global)
  int repl;        // code book stored eight times, entry i of copy c at slot 8 i + c: lane l reads
                   // copy l % 8, so the eight lanes of a quarter warp never share a bank group
  int W;           // warps of the launch that walks this plan (grid * warps per block)
  int only_grp;    // -1: the launch walks every work group; >= 0 (ablation): only this one
  int tpu;         // compressed down stage: 8-row tiles of H per unit (one set of p fragments, one request group and
                   // one step of the work cursor for 8 * tpu rows); `tiles` then counts units.  1 elsewhere
  int tail;        // tiles % chunk: length of a shorter last chunk (0: none)
  FastDiv d_per_grp, d_per_chunk, d_chunk, d_tail, d_W;   // n_parts*tiles, n_parts*chunk, chunk, tail, W
};

#ifdef MOE_VQLR_JIT
// Run-time-compiled copies (jit_host.cuh): the integers of a work plan as constants, X = GU or DN.
#define MOE_VQLR_JIT_PLAN(pl, X)                                                                          \
  do {                                                                                                    \
    (pl).nb = J_##X##_NB; (pl).n_slices = J_##X##_NSLICES; (pl).n_lr = J_##X##_NLR;                       \
    (pl).n_parts = J_##X##_NPARTS; (pl).tiles = J_##X##_TILES; (pl).depth = J_##X##_DEPTH;                \
    (pl).chunk = J_##X##_CHUNK; (pl).x_smem = J_##X##_XSMEM; (pl).repl = J_##X##_REPL; (pl).W = J_##X##_W; \
    (pl).only_grp = -1; (pl).tpu = J_##X##_TPU; (pl).tail = J_##X##_TAIL;                                 \
    (pl).d_per_grp = make_fastdiv((unsigned int)(J_##X##_NPARTS * J_##X##_TILES));                        \
    (pl).d_per_chunk = make_fastdiv((unsigned int)(J_##X##_NPARTS * J_##X##_CHUNK));                      \
    (pl).d_chunk = make_fastdiv((unsigned int)J_##X##_CHUNK);                                             \
    (pl).d_tail = make_fastdiv((unsigned int)(J_##X##_TAIL > 0 ? J_##X##_TAIL : 1));                      \
    (pl).d_W = make_fastdiv((unsigned int)J_##X##_W);                                                     \
  } while (0)
#endif

// Position in the flattened work list of a stage.  Units are ordered (group, chunk of `chunk`
// row tiles, part, tile inside the chunk): a warp's contiguous range then mixes cheap low-rank
// parts with lookup-heavy slice parts instead of drawing only one kind, while consecutive tiles
// of one part still share its activation fragments.  chunk = tiles gives (group, part, tile).
struct Cursor {
  int grp, part, jt, chunk_end;       // jt = absolute tile, chunk_end = first tile after its chunk
  __device__ __forceinline__ void set(int v, const StagePlan& pl) {
    const int per_grp = pl.n_parts * pl.tiles;
    grp = fdiv(v, pl.d_per_grp);
    int rem = v - grp * per_grp;
    const int per_chunk = pl.n_parts * pl.chunk;
    const int ch = fdiv(rem, pl.d_per_chunk);       // the last chunk may be shorter
    rem -= ch * per_chunk;
    const int c0 = ch * pl.chunk;
    const int clen = min(pl.chunk, pl.tiles - c0);
    part = clen == pl.chunk ? fdiv(rem, pl.d_chunk) : fdiv(rem, pl.d_tail);
    jt = c0 + (rem - part * clen);
    chunk_end = c0 + clen;
  }
  __device__ __forceinline__ void next(const StagePlan& pl) {
    if (++jt == chunk_end) {
      const int c0 = chunk_end - min(pl.chunk, chunk_end - fdiv(chunk_end - 1, pl.d_chunk) * pl.chunk);
      if (++part == pl.n_parts) {
        part = 0;
        if (chunk_end == pl.tiles) { ++grp; jt = 0; chunk_end = min(pl.chunk, pl.tiles); }
        else { jt = chunk_end; chunk_end = min(chunk_end + pl.chunk, pl.tiles); }
      } else {
        jt = c0;
      }
    }
  }
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
    bool bad = false;                // fewer than k experts with a finite logit
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
        if (win >= E) { win = s; bad = true; }     // only NaN / -inf left: stay in bounds, report it
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
        if (win >= E) { win = s; bad = true; }
        if (lane == (win & 31)) taken |= 1u << (win >> 5);
        if (lane == s) { sel_key = mk; sel_e = win; }
      }
    }
    const float sel_l = key_logit(sel_key);
    // a selected logit that is not finite (NaN sorts above every number here, -inf is only taken
    // when nothing else is left): the ids stay in bounds, the call is reported as invalid
    if (lane < k && !(fabsf(sel_l) <= 3.402823466e38f)) bad = true;
    if (__any_sync(0xffffffffu, bad) && write_global && lane == 0) set_status(P, MOE_VQLR_ERR_INVALID_ARG);
    const float lmax = __shfl_sync(0xffffffffu, sel_l, 0);
    const float ev = lane < k ? expf(sel_l - lmax) : 0.f;
    float denom = ev;
    if (!P.renorm)
      for (int e = lane, j = 0; e < E; e += 32, ++j)
        if (!((taken >> j) & 1u) && row[e] != -CUDART_INF_F) denom += expf(row[e] - lmax);
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
  // ---- pairs sorted by (expert, token) and cut into work groups, by counting -----------------
  // Per expert a bit map of the tokens that selected it (a token selects an expert at most once, so
  // OR-ing the bits does not depend on the order of the threads).  Population counts of the map give a
  // pair's place inside its expert's run and the run's length; an exclusive scan over the experts by
  // one warp gives the run's first pair position and first work group (a new group starts at every
  // eighth pair of a run).  T >= 2 here, so the 2 E words fit where the logits were.
  unsigned int* s_map = reinterpret_cast<unsigned int*>(R.logit);       // [E] tokens of the expert
  unsigned int* s_off = s_map + E;                                       // [E] first pair position | first group << 16
  for (int e = tid; e < E; e += nthr) s_map[e] = 0u;
  __syncthreads();
  for (int q = tid; q < n_pairs; q += nthr) atomicOr(&s_map[R.sel_id[q]], 1u << (q / k));
  __syncthreads();
  if (warp == 0) {
    const int per = (E + 31) >> 5, e0 = lane * per;          // a contiguous run of experts per lane
    unsigned int mine = 0u;                                   // pairs | groups << 16 (both at most 16 * 32)
    for (int i = 0; i < per; ++i)
      if (e0 + i < E) {
        const unsigned int c = (unsigned int)__popc(s_map[e0 + i]);
        mine += c | (((c + kGroupTokens - 1) / kGroupTokens) << 16);
      }
    unsigned int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned int n = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += n;
    }
    unsigned int run = incl - mine;
    for (int i = 0; i < per; ++i)
      if (e0 + i < E) {
        s_off[e0 + i] = run;
        const unsigned int c = (unsigned int)__popc(s_map[e0 + i]);
        run += c | (((c + kGroupTokens - 1) / kGroupTokens) << 16);
      }
    if (lane == 31) R.warp_cnt[0] = (int)(incl >> 16);      // work groups of the routed experts
  }
  __syncthreads();
  const int base = R.warp_cnt[0];
  for (int q = tid; q < n_pairs; q += nthr) {
    const int t = q / k, s = q - t * k, e = R.sel_id[q];
    const unsigned int bm = s_map[e], o = s_off[e];
    const int j = __popc(bm & ((1u << t) - 1u)), c = __popc(bm);      // same expert: pair order = token order
    const int pos = (int)(o & 0xffffu) + j;
    R.sort_e[pos] = e; R.sort_j[pos] = j; R.sort_c[pos] = c;
    R.pair_token[pos] = t;
    if (write_global) { P.pair_token[pos] = t; P.pair_slot[pos] = s; P.pair_w[pos] = R.w[q]; P.inv_pos[t * (k + S) + s] = pos; }
    if (j % kGroupTokens == 0) {
      const int gi = (int)(o >> 16) + j / kGroupTokens;
      R.grp_e[gi] = e;
      R.grp_off[gi] = pos;
      R.grp_cnt[gi] = min(kGroupTokens, c - j);
    }
  }
  for (int q = tid; q < S * T; q += nthr) {                 // shared experts: every token, weight 1
    R.pair_token[n_pairs + q] = q % T;
    if (write_global) {
      P.pair_token[n_pairs + q] = q % T; P.pair_slot[n_pairs + q] = k + q / T; P.pair_w[n_pairs + q] = 1.f;
      P.inv_pos[(q % T) * (k + S) + k + q / T] = n_pairs + q;
    }
  }
  TRACE_STAMP(1, 3);
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

// Routing of a single token as far as a block of the fused kernel needs it: WHICH experts are
// selected, in ascending id order (= the work groups).  Expert e is selected iff fewer than k
// experts precede it in the order (logit descending, id ascending) -- one thread per expert counts
// them, no dependent rounds; slots, affinities and the global lists are left to the one block that
// runs route_in_block.  E <= 1024.
__device__ void route_light_t1(const Params& P, const RouteSmem& R) {
  const int E = P.E, k = P.k, S = P.S;
  const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31;
  unsigned int* s_key = reinterpret_cast<unsigned int*>(R.logit);
  for (int i = tid; i < E; i += nthr) s_key[i] = logit_key(__ldcg(P.logits + i));
  __syncthreads();
  const int n_chunks = (E + 31) >> 5;                       // ballots of 32 experts each
  for (int e0 = (tid >> 5) << 5; e0 < E; e0 += nthr) {      // warp-uniform trip count
    const int e = e0 + lane;
    bool sel = false;
    if (e < E) {
      const unsigned int key = s_key[e];
      int c0 = 0, c1 = 0, c2 = 0, c3 = 0;
      if ((E & 3) == 0) {
#pragma unroll 8
        for (int e2 = 0; e2 < E; e2 += 4) {
          const uint4 v = *reinterpret_cast<const uint4*>(s_key + e2);
          c0 += (v.x > key) | ((v.x == key) & (e2 < e));
          c1 += (v.y > key) | ((v.y == key) & (e2 + 1 < e));
          c2 += (v.z > key) | ((v.z == key) & (e2 + 2 < e));
          c3 += (v.w > key) | ((v.w == key) & (e2 + 3 < e));
        }
      } else {
        for (int e2 = 0; e2 < E; ++e2) c0 += (s_key[e2] > key) | ((s_key[e2] == key) & (e2 < e));
      }
      sel = (c0 + c1) + (c2 + c3) < k;
    }
    const unsigned int bal = __ballot_sync(0xffffffffu, sel);
    if (lane == 0) R.warp_cnt[e0 >> 5] = (int)bal;
  }
  __syncthreads();
  for (int e = tid; e < E; e += nthr) {
    const unsigned int bal = (unsigned int)R.warp_cnt[e >> 5];
    if ((bal >> (e & 31)) & 1u) {
      int pos = __popc(bal & ((1u << (e & 31)) - 1u));
      for (int w = 0; w < (e >> 5); ++w) pos += __popc((unsigned int)R.warp_cnt[w]);
      R.pair_token[pos] = 0;
      R.grp_e[pos] = e; R.grp_off[pos] = pos; R.grp_cnt[pos] = 1;
    }
  }
  for (int s2 = tid; s2 < S; s2 += nthr) {
    R.pair_token[k + s2] = 0;
    R.grp_e[k + s2] = E + s2; R.grp_off[k + s2] = k + s2; R.grp_cnt[k + s2] = 1;
  }
  if (tid == 0) *R.n_grp = k + S;
  (void)n_chunks;
  __syncthreads();
}

// ---------------------------------------------------------------------------------------------
// k_router_z_pdl: head of the chain.  One warp per (row of [router_w ; basis_gate ; basis_up],
// group of four tokens).  Per (row, token) the summation order is the one of k_router_z
// (lane-strided 16-byte chunks, sequential FMAs inside a chunk, xor butterfly), so identical
// router rows give bitwise identical logits.
// ---------------------------------------------------------------------------------------------
constexpr int kRouterWarps = 2;

// One unit = one (row, group of four tokens); executed by one warp.
__host__ __device__ __forceinline__ int router_z_units(const Params& P, int T) {
  return (P.E + P.n_zrows) * ((T + kTokGroup - 1) / kTokGroup);
}

// Units of a k_router_z_pdl launch: with z_repeat > 1 (Section 5.4's variant that recomputes the
// shared projections for every expert) the basis rows are walked z_repeat times.
__host__ __device__ __forceinline__ int router_z_units_launched(const Params& P, int T) {
  return (P.E + P.n_zrows * P.z_repeat) * ((T + kTokGroup - 1) / kTokGroup);
}

__device__ __forceinline__ void router_z_unit(const Params& P, const bf16* __restrict__ x, int T, int unit, int lane) {
  const int n_groups = (T + kTokGroup - 1) / kTokGroup;
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

// The same unit in two steps for a persistent kernel: the weight row (first 8 chunks per lane)
// is requested into registers BEFORE the block waits for the tokens to land in shared memory,
// so that both round trips overlap; summation order as in router_z_unit.
struct RouterRow {
  const uint4* w4;
  float* dst;
  int dst_stride, t0, nt;
  float bias;
};

__device__ __forceinline__ RouterRow router_z_row(const Params& P, int T, int unit) {
  const int n_groups = (T + kTokGroup - 1) / kTokGroup;
  const int row = unit / n_groups;
  RouterRow u;
  u.t0 = (unit - row * n_groups) * kTokGroup;
  u.nt = min(kTokGroup, T - u.t0);
  u.bias = 0.f;
  if (row < P.E) {
    u.w4 = reinterpret_cast<const uint4*>(P.router_w + (size_t)row * P.H);
    u.dst = P.logits + row;
    u.dst_stride = P.E;
    if (P.router_bias) u.bias = P.router_bias[row];
  } else {
    const int q = row - P.E;
    const int slot = q / P.r, rho = q - slot * P.r;
    const bf16* basis = (slot == P.gate.zslot && P.gate.basis) ? P.gate.basis : P.up.basis;
    u.w4 = reinterpret_cast<const uint4*>(basis + (size_t)rho * P.H);
    u.dst = P.z + slot * P.r + rho;
    u.dst_stride = 2 * P.r;
  }
  return u;
}

__device__ __forceinline__ void router_z_load8(const RouterRow& u, int c0, int nchunk, int lane, uint4 (&wv)[8]) {
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    const int c = c0 + q * 32 + lane;
    wv[q] = c < nchunk ? __ldg(u.w4 + c) : make_uint4(0, 0, 0, 0);
  }
}

// s_x: tokens in shared memory, row stride xs blocks.  wv: chunks 0..255 of the row, already requested.
__device__ __forceinline__ void router_z_finish(const Params& P, const RouterRow& u, const uint4* s_x, int xs, int lane, uint4 (&wv)[8]) {
  const int nchunk = P.H / 8;
  float acc[kTokGroup] = {0.f, 0.f, 0.f, 0.f};
  for (int c0 = 0; c0 < nchunk; c0 += 32 * 8) {
    if (c0 > 0) router_z_load8(u, c0, nchunk, lane, wv);
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int c = c0 + q * 32 + lane;
      if (c < nchunk) {
        float wf[8];
        unpack8(wv[q], wf);
#pragma unroll
        for (int tt = 0; tt < kTokGroup; ++tt) {
          if (tt < u.nt) {
            float xf[8];
            unpack8(s_x[(u.t0 + tt) * xs + c], xf);
            acc[tt] = dot8(wf, xf, acc[tt]);
          }
        }
      }
    }
  }
#pragma unroll
  for (int tt = 0; tt < kTokGroup; ++tt) {
    const float sum = warp_sum(acc[tt]);
    if (lane == 0 && tt < u.nt) u.dst[(size_t)(u.t0 + tt) * u.dst_stride] = sum + u.bias;
  }
}

// A single token: the row and the token are requested 2048 values at a time (8 + 8 loads per lane
// in flight) instead of 512; same summation order.  wv holds chunks 0..255 of the row, requested by
// the caller before it waited for the previous kernel (weights do not depend on it).
__device__ __forceinline__ void router_z_finish_t1(const Params& P, const RouterRow& u, const bf16* __restrict__ x, int lane, uint4 (&wv)[8]) {
  const int nchunk = P.H / 8;
  const uint4* x4 = reinterpret_cast<const uint4*>(x);
  float acc = 0.f;
  for (int c0 = 0; c0 < nchunk; c0 += 256) {
    uint4 xv[8];
    if (c0 > 0) router_z_load8(u, c0, nchunk, lane, wv);
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int c = c0 + q * 32 + lane;
      xv[q] = c < nchunk ? __ldg(x4 + c) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      if (c0 + q * 32 + lane < nchunk) {
        float wf[8], xf[8];
        unpack8(wv[q], wf);
        unpack8(xv[q], xf);
        acc = dot8(wf, xf, acc);
      }
    }
  }
  const float sum = warp_sum(acc);
  if (lane == 0) u.dst[0] = sum + u.bias;
}

// Up to four tokens and a row of at most 2048 values: the whole weight row (wv, requested before
// the wait) is the DRAM round trip, the tokens' chunks follow from L1 / L2; same summation order.
__device__ __forceinline__ void router_z_finish_row8(const Params& P, const RouterRow& u, const bf16* __restrict__ x, int lane, uint4 (&wv)[8]) {
  const int nchunk = P.H / 8;
  float acc[kTokGroup] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    const int c = q * 32 + lane;
    uint4 xv[kTokGroup];
#pragma unroll
    for (int tt = 0; tt < kTokGroup; ++tt)
      xv[tt] = (c < nchunk && tt < u.nt) ? __ldg(reinterpret_cast<const uint4*>(x + (size_t)(u.t0 + tt) * P.H) + c) : make_uint4(0, 0, 0, 0);
    if (c < nchunk) {
      float wf[8];
      unpack8(wv[q], wf);
#pragma unroll
      for (int tt = 0; tt < kTokGroup; ++tt) {
        float xf[8];
        unpack8(xv[tt], xf);
        acc[tt] = dot8(wf, xf, acc[tt]);
      }
    }
  }
#pragma unroll
  for (int tt = 0; tt < kTokGroup; ++tt) {
    const float sum = warp_sum(acc[tt]);
    if (lane == 0 && tt < u.nt) u.dst[(size_t)(u.t0 + tt) * u.dst_stride] = sum + u.bias;
  }
}

__device__ __forceinline__ void router_z_unit_row8(const Params& P, const bf16* __restrict__ x, int T, int unit, int lane) {
  const RouterRow u = router_z_row(P, T, unit);
  uint4 wv[8];
  router_z_load8(u, 0, P.H / 8, lane, wv);
  router_z_finish_row8(P, u, x, lane, wv);
}

// The weight row of a unit is requested BEFORE the wait for the previous kernel of the stream: the
// weights never depend on it (only the tokens and the logits / z buffers do), so the DRAM round
// trip of the row overlaps the previous kernel's tail.
// LEAN (the copy compiled per shape, see jit_host.cuh): a single token, the layer's sizes constants.
template <bool LEAN>
__device__ __forceinline__ void router_z_pdl_body(const Params& P_in, const bf16* __restrict__ x, int T_in) {
  const int T = LEAN ? 1 : T_in;
#ifdef MOE_VQLR_JIT
  Params P = P_in;
  MOE_VQLR_JIT_PARAMS(P);
#else
  const Params& P = P_in;
#endif
  int unit = blockIdx.x * kRouterWarps + (threadIdx.x >> 5);
  const int base_units = router_z_units(P, T), lane = threadIdx.x & 31;
  const bool has = unit < router_z_units_launched(P, T);
  if (has && unit >= base_units) {          // ablation: a repeated basis row (same operands, same result, same address)
    const int n_groups = (T + kTokGroup - 1) / kTokGroup;
    unit = P.E * n_groups + (unit - base_units) % (P.n_zrows * n_groups);
  }
  const bool early = has && (T == 1 || P.H <= 2048);
  RouterRow u;
  uint4 wv[8];
  TRACE_STAMP(0, 8);
  if (early) {
    u = router_z_row(P, T, unit);
    router_z_load8(u, 0, P.H / 8, lane, wv);
  }
  pdl_wait();      // the previous call's kernels may still read logits / z; the tokens are its output
  pdl_launch();
  TRACE_STAMP(0, 9);
  if (!has) return;
  if (T == 1) router_z_finish_t1(P, u, x, lane, wv);
  else if (P.H <= 2048) router_z_finish_row8(P, u, x, lane, wv);
  else router_z_unit(P, x, T, unit, lane);
  TRACE_STAMP(0, 10);
}

#ifndef MOE_VQLR_JIT
__global__ void __launch_bounds__(32 * kRouterWarps) k_router_z_pdl(const Params P, const bf16* __restrict__ x, int T) {
  router_z_pdl_body<false>(P, x, T);
}
#endif

// k_router_zmma_pdl: head of the chain for 9..16 tokens.  The shared projections z = basis * x
// (Section 4.2) run on the tensor cores: one block per eight basis rows, each of its eight warps
// takes an eighth of H with the tokens as the sixteen rows of the m16n8k16 tile (tokens 0..7 in
// rows 0..7, 8..15 in rows 8..15), and the warps' partial tiles meet in shared memory and are added
// in warp order.  The remaining blocks compute the router logits with the exact FMA chains of
// k_router_z_pdl, one (row, group of four tokens) per warp.  H must be a multiple of 256, r of 8.
constexpr int kZmmaWarps = 8;

__host__ __device__ __forceinline__ int zmma_blocks(const Params& P) { return P.n_zrows / 8 * P.z_repeat; }

__device__ __forceinline__ void router_zmma_pdl_body(const Params& P_in, const bf16* __restrict__ x, int T) {
#ifdef MOE_VQLR_JIT
  Params P = P_in;
  MOE_VQLR_JIT_PARAMS(P);
#else
  const Params& P = P_in;
#endif
  __shared__ float s_red[kZmmaWarps][128];
  // As in k_router_z_pdl, the weights of a unit (they never depend on the previous kernel) are
  // requested before the dependency wait: a router row of up to 2048 values, or the first half of a
  // z block's basis rows.
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n_units = P.E * ((T + kTokGroup - 1) / kTokGroup), n_logit_blocks = (n_units + kZmmaWarps - 1) / kZmmaWarps;
  if ((int)blockIdx.x < n_logit_blocks) {      // the logits blocks come first: their FMA chains take longest
    const int unit = (int)blockIdx.x * kZmmaWarps + warp;
    const bool has = unit < n_units, early = has && P.H <= 2048;
    RouterRow u;
    uint4 wv[8];
    if (early) {
      u = router_z_row(P, T, unit);
      router_z_load8(u, 0, P.H / 8, lane, wv);
    }
    pdl_wait();      // the previous call's kernels may still read logits / z; the tokens are its output
    pdl_launch();
    if (!has) return;
    if (early) router_z_finish_row8(P, u, x, lane, wv);
    else router_z_unit(P, x, T, unit, lane);
    return;
  }
  const int g = lane >> 2, c = lane & 3;
  const int q0 = (((int)blockIdx.x - n_logit_blocks) % (P.n_zrows / 8)) * 8;   // a repeated tile (ablation) recomputes the same rows
  const int slot = q0 / P.r, rho0 = q0 - slot * P.r;
  const bf16* basis = (slot == P.gate.zslot && P.gate.basis) ? P.gate.basis : P.up.basis;
  const int nblk = P.H / 8, per = nblk / kZmmaWarps;
  const uint4* w4 = reinterpret_cast<const uint4*>(basis + (size_t)(rho0 + g) * P.H) + warp * per + c;
  const uint4* xa4 = reinterpret_cast<const uint4*>(x + (size_t)g * P.H) + warp * per + c;
  const uint4* xb4 = reinterpret_cast<const uint4*>(x + (size_t)(g + 8) * P.H) + warp * per + c;
  const bool live_a = g < T, live_b = g + 8 < T;
  uint4 wv0[4];
#pragma unroll
  for (int u = 0; u < 4; ++u) wv0[u] = 4 * u < per ? __ldg(w4 + 4 * u) : make_uint4(0, 0, 0, 0);
  pdl_wait();
  pdl_launch();
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  for (int s = 0; s < per; s += 16) {                              // four steps of 32 values with their loads in flight
    uint4 wv[4], av[4], bv[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const bool in = s + 4 * u < per;
      wv[u] = s == 0 ? wv0[u] : in ? __ldg(w4 + s + 4 * u) : make_uint4(0, 0, 0, 0);
      av[u] = (in && live_a) ? __ldg(xa4 + s + 4 * u) : make_uint4(0, 0, 0, 0);
      bv[u] = (in && live_b) ? __ldg(xb4 + s + 4 * u) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) mma_block_hilo(acc, av[u], bv[u], wv[u]);
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) s_red[warp][lane * 4 + i] = acc[i];
  __syncthreads();
  if (threadIdx.x < 128) {
    float sum = 0.f;
#pragma unroll
    for (int w = 0; w < kZmmaWarps; ++w) sum += s_red[w][threadIdx.x];
    const int l2 = threadIdx.x >> 2, i = threadIdx.x & 3;
    const int tok = (l2 >> 2) + ((i & 2) ? 8 : 0), row = 2 * (l2 & 3) + (i & 1);
    if (tok < T) P.z[((size_t)tok * 2 + slot) * P.r + rho0 + row] = sum;
  }
}

#ifndef MOE_VQLR_JIT
__global__ void __launch_bounds__(32 * kZmmaWarps) k_router_zmma_pdl(const Params P, const bf16* __restrict__ x, int T) {
  router_zmma_pdl_body(P, x, T);
}
#endif

// Splits `total` units evenly over `parts` warps: first unit of warp `idx` = floor(total * idx / parts),
// in 32-bit arithmetic (parts < 65536).
__device__ __forceinline__ int split_begin(int total, int parts, int idx) {
  const unsigned int q = (unsigned int)total / (unsigned int)parts, rem = (unsigned int)total - q * (unsigned int)parts;
  return (int)(q * (unsigned int)idx + (rem * (unsigned int)idx) / (unsigned int)parts);
}

// The same with the plan's warp count and its magic number (total, idx < 2^15 or so: rem * idx < 2^31).
__device__ __forceinline__ int split_begin(int total, const StagePlan& pl, int idx) {
  const int q = fdiv(total, pl.d_W), rem = total - q * pl.W;
  return q * idx + fdiv(rem * idx, pl.d_W);
}

// ---------------------------------------------------------------------------------------------
// k_gateup_mma: partial gate / up tiles.  A warp owns one part (a 256-value slice of H, or 32
// ranks of the low-rank term) of one work group and walks a contiguous range of row tiles.
// ---------------------------------------------------------------------------------------------
struct GuLayout {         // byte offsets into dynamic shared memory
  size_t cb_u, x, ring, z, route, cb_tmp, total;
};

__host__ __device__ inline GuLayout gu_layout(int K, int n_books, int T, int H, int r, const StagePlan& pl,
                                              int warps, int E, int k, int S) {
  GuLayout L;
  size_t o = 0;
  const size_t cb_bytes = (size_t)K * 16 * (pl.repl ? 8 : 1);
  L.cb_u = n_books == 2 ? cb_bytes : 0;
  o = (size_t)n_books * cb_bytes;
  L.x = o;      o += pl.x_smem ? (size_t)T * (H / 8 + 1) * 16 : 0;
  L.ring = o;   o += (size_t)warps * pl.depth * 2 * 32 * 16;
  L.z = o;      o += (size_t)2 * T * 2 * ((r + 7) / 8) * 16;            // hi and lo blocks of z
  L.route = o;  o += route_smem_bytes(T, E, k, S);
  L.cb_tmp = o; o += pl.repl ? (size_t)n_books * K * 16 : 0;      // compact copy the replicas are made from
  L.total = o;
  return L;
}

// Shared-memory views of the gate/up stage.
struct GuSmem {
  uint4 *cb_g, *cb_u, *x, *ring, *zh, *zl, *tmp;
  RouteSmem R;
};

__device__ __forceinline__ GuSmem gu_carve(char* s_base, const GuLayout& L, const Params& P, int T, int warp, int lane, int depth) {
  GuSmem m;
  const int rb = (P.r + 7) / 8;
  m.cb_g = reinterpret_cast<uint4*>(s_base);
  m.cb_u = reinterpret_cast<uint4*>(s_base + L.cb_u);
  m.x = reinterpret_cast<uint4*>(s_base + L.x);
  m.ring = reinterpret_cast<uint4*>(s_base + L.ring) + (size_t)warp * depth * 2 * 32 + lane;   // [slot][proj][lane]
  m.zh = reinterpret_cast<uint4*>(s_base + L.z);          // [T][2][rb]
  m.zl = m.zh + (size_t)T * 2 * rb;
  m.tmp = reinterpret_cast<uint4*>(s_base + L.cb_tmp);
  m.R = carve_route(s_base + L.route, T, P.E, P.k, P.S);
  return m;
}

// Routing-independent prologue: code books and tokens start streaming into shared memory
// (one cp.async group per thread, not yet waited for).
// Requests the tokens (one cp.async group) ...
__device__ __forceinline__ void gu_stage_tokens_async(const bf16* __restrict__ x, int T, const StagePlan& pl, const GuSmem& m) {
  const int tid = threadIdx.x, nb = pl.nb, xs = nb + 1;
  const uint4* x4 = reinterpret_cast<const uint4*>(x);
  if (pl.x_smem)
    for (int i = tid; i < T * nb; i += blockDim.x) {
      const int t = i / nb, b = i - t * nb;
      cp_async16(m.x + t * xs + b, x4 + i);
    }
  cp_async_commit();
}

// ... and the code books (a second group).  A replicated book is fetched once and copied eight
// times inside shared memory later.
template <bool DENSE>
__device__ __forceinline__ void gu_stage_books_async(const Params& P, const StagePlan& pl, int n_books, const GuSmem& m) {
  const int tid = threadIdx.x;
  if (!DENSE) {
    uint4* dst_g = pl.repl ? m.tmp : m.cb_g;
    uint4* dst_u = pl.repl ? m.tmp + P.K : m.cb_u;
    // Every block fetches the same few KB from L2: each starts at its own offset, so that at any
    // moment the blocks ask for different lines (all asking for the same lines in the same order
    // serialises on single L2 slices: 5 us instead of 1-2 for 64 KB x 148 blocks).
    const int kw = P.d == 8 ? P.K : P.K / 2;      // 16-byte pieces of one book
    const int rot = (int)(((unsigned int)blockIdx.x * (unsigned int)kw) / gridDim.x);
    for (int i = tid; i < kw; i += blockDim.x) {
      int j = i + rot;
      if (j >= kw) j -= kw;
      cp_async16(dst_g + j, P.gate.codebook + j);
    }
    if (n_books == 2)
      for (int i = tid; i < kw; i += blockDim.x) {
        int j = i + rot;
        if (j >= kw) j -= kw;
        cp_async16(dst_u + j, P.up.codebook + j);
      }
  }
  cp_async_commit();
}


template <bool DENSE>
__device__ __forceinline__ void gu_stage_async(const Params& P, const bf16* __restrict__ x, int T, const StagePlan& pl,
                                               int n_books, const GuSmem& m) {
  gu_stage_tokens_async(x, T, pl, m);
  gu_stage_books_async<DENSE>(P, pl, n_books, m);
}

// After logits and z are complete: z as bf16 hi / lo blocks, routing, and the staged bytes landed.
__device__ __forceinline__ void gu_route(const Params& P, int T, const StagePlan& pl, const GuSmem& m,
                                         bool write_global, bool want_dbg, bool light = false) {
  const int tid = threadIdx.x, rb = (P.r + 7) / 8;
  float4 zv[2][2];                 // this thread's z values travel while the routing runs (up to two blocks of 8 each)
  const int nz = pl.n_lr > 0 ? T * 2 * rb : 0;
#pragma unroll
  for (int q = 0; q < 2; ++q) {
    const int i = tid + q * blockDim.x;
    if (i < nz) {
      const float* zp = P.z + (size_t)i * 8;
      zv[q][0] = __ldcg(reinterpret_cast<const float4*>(zp));
      zv[q][1] = __ldcg(reinterpret_cast<const float4*>(zp + 4));
    }
  }
  if (light) route_light_t1(P, m.R); else route_in_block(P, T, m.R, write_global, want_dbg);
#pragma unroll
  for (int q = 0; q < 2; ++q) {
    const int i = tid + q * blockDim.x;
    if (i < nz) split_hi_lo(zv[q][0], zv[q][1], m.zh[i], m.zl[i]);
  }
  for (int i = tid + 2 * blockDim.x; i < nz; i += blockDim.x) {      // z is [T][2][r], r a multiple of 8
    const float* zp = P.z + (size_t)i * 8;
    split_hi_lo(__ldcg(reinterpret_cast<const float4*>(zp)), __ldcg(reinterpret_cast<const float4*>(zp + 4)), m.zh[i], m.zl[i]);
  }
  TRACE_STAMP(1, 5);
}

// The staged bytes have landed (the `newer` most recent cp.async groups may still be in flight).
template <bool DENSE>
__device__ __forceinline__ void gu_finish_stage(const Params& P, const StagePlan& pl, int n_books, const GuSmem& m, int newer) {
  const int tid = threadIdx.x;
  cp_async_wait_pending(newer);   // this thread's share of code book and tokens has landed ...
  __syncthreads();                // ... and so has everybody else's (and z, and the routing lists)
  TRACE_STAMP(1, 6);
  if (!DENSE && pl.repl) {
    if (P.d == 8) {
      for (int i = tid; i < P.K * 8; i += blockDim.x) {
        m.cb_g[i] = m.tmp[i >> 3];
        if (n_books == 2) m.cb_u[i] = m.tmp[P.K + (i >> 3)];
      }
    } else {                        // sixteen copies of the 8-byte words
      uint2* g2 = reinterpret_cast<uint2*>(m.cb_g);
      uint2* u2 = reinterpret_cast<uint2*>(m.cb_u);
      const uint2* tg = reinterpret_cast<const uint2*>(m.tmp);
      const uint2* tu = reinterpret_cast<const uint2*>(m.tmp + P.K);
      for (int i = tid; i < P.K * 16; i += blockDim.x) {
        g2[i] = tg[i >> 4];
        if (n_books == 2) u2[i] = tu[i >> 4];
      }
    }
    __syncthreads();
  }
}

// A warp's walk over its contiguous range of the work list: the prefetch cursor runs depth - 1
// units ahead of the compute cursor through the warp's ring.
struct Walk {
  Cursor pf, cur;
  int pf_slot, cur_slot, n_my;
};

// Streams the bytes of the prefetch cursor's unit into the ring and advances that cursor.
// SP ("special formats"): the kernel also handles experts without a gate projection and 12-bit
// packed indices, at the price of run-time checks in its unit loop; the plain instantiation folds
// them away.
template <typename IdxT, bool DENSE, bool SP = false>
__device__ __forceinline__ void gu_issue(const Params& P, const StagePlan& pl, const GuSmem& m, Walk& w) {
  const int lane = threadIdx.x & 31, g = lane >> 2, c = lane & 3, nb = pl.nb;
  uint4* ring = m.ring;
  if (!DENSE) {
    const IdxT* idx_g = static_cast<const IdxT*>(P.gate.idx);
    const IdxT* idx_u = static_cast<const IdxT*>(P.up.idx);
    const size_t row = (size_t)m.R.grp_e[w.pf.grp] * P.I + w.pf.jt * 8 + g;
    const bool up_only = SP && P.act == 2;       // experts without a gate: its bytes are not requested
    const int idx12 = SP ? P.idx12 : 0;
    if (w.pf.part < pl.n_slices) {
      const int b = w.pf.part * 32 + 8 * c;
      if (b < nb) {
        if (!up_only) cp_async_idx8<IdxT>(ring + (w.pf_slot * 2 + 0) * 32, idx_at(idx_g, row * nb + b, idx12), idx12);
        cp_async_idx8<IdxT>(ring + (w.pf_slot * 2 + 1) * 32, idx_at(idx_u, row * nb + b, idx12), idx12);
      }
    } else {
      const int rho = (w.pf.part - pl.n_slices) * 32 + 8 * c;
      if (rho < P.r) {
        if (!up_only) cp_async16(ring + (w.pf_slot * 2 + 0) * 32, P.gate.factor + row * P.r + rho);
        cp_async16(ring + (w.pf_slot * 2 + 1) * 32, P.up.factor + row * P.r + rho);
      }
    }
  }
  w.pf.next(pl);
  if (++w.pf_slot == pl.depth) w.pf_slot = 0;
}

// Start of the walk of warp `wid` out of `W` warps (needs the work groups): depth - 1 units are
// requested, each as one cp.async group.
template <typename IdxT, bool DENSE, bool SP = false>
__device__ __forceinline__ void gu_tiles_begin(const Params& P, const StagePlan& pl, const GuSmem& m, int wid, int W, Walk& w) {
  const int per_grp = pl.n_parts * pl.tiles;
  int V = *m.R.n_grp * per_grp, v0 = 0;
  if (pl.only_grp >= 0) { V = pl.only_grp < *m.R.n_grp ? per_grp : 0; v0 = pl.only_grp * per_grp; }
  const int v_begin = split_begin(V, pl, wid);         // W == pl.W by construction of the launch
  w.n_my = split_begin(V, pl, wid + 1) - v_begin;
  w.pf.set(w.n_my > 0 ? v0 + v_begin : 0, pl);
  w.cur = w.pf;
  w.pf_slot = 0; w.cur_slot = 0;
  for (int i = 0; i < pl.depth - 1; ++i) { if (i < w.n_my) gu_issue<IdxT, DENSE, SP>(P, pl, m, w); cp_async_commit(); }
  TRACE_STAMP(1, 7);
}

// The tile loop proper (needs code books, tokens and z in shared memory).  LRF > 0: there are at least
// as many low-rank groups (32 ranks each) as slices; slice s then carries the groups s, s + n_slices,
// ... besides its own blocks and no group is a part of its own (fewer, fatter units and fewer
// partial tiles; with fewer groups than slices the units that carry one would lag the others).
// LRF = 2: some slices carry two or more groups; the second one's bytes are requested early as well.
template <typename IdxT, bool DENSE, bool D4 = false, int LRF = 0, bool SP = false>
__device__ __forceinline__ void gu_tiles_run(const Params& P, const bf16* __restrict__ x, int T, const StagePlan& pl,
                                             const GuSmem& m, Walk& w) {
  const int lane = threadIdx.x & 31, g = lane >> 2, c = lane & 3;
  const int nb = pl.nb, xs = nb + 1, D = pl.depth, rb = (P.r + 7) / 8;
  const uint4* x4 = reinterpret_cast<const uint4*>(x);
  uint4* s_cb_g = m.cb_g;
  uint4* s_cb_u = m.cb_u;
  uint4* s_x = m.x;
  uint4* ring = m.ring;
  uint4* s_zh = m.zh;
  uint4* s_zl = m.zl;
  const RouteSmem& R = m.R;
  const int n_pos = T * (P.k + P.S), n_my = w.n_my;
  Cursor& cur = w.cur;
  int& cur_slot = w.cur_slot;
  auto issue = [&]() { gu_issue<IdxT, DENSE, SP>(P, pl, m, w); };

  uint4 fx[8];                       // activation fragments of the current (group, part)
  int frag_grp = -1, frag_part = -1;
  const bool up_only = SP && P.act == 2;   // experts without a gate projection: only the up products are formed
  const int idx12 = SP ? P.idx12 : 0;

  for (int i = 0; i < n_my; ++i) {
    if (i + D - 1 < n_my) issue();
    cp_async_commit();
    TRACE_STAMP(0, 4 + 3 * i);
    cp_async_wait_pending(D - 1);
    TRACE_STAMP(0, 5 + 3 * i);
    const int grp = cur.grp, part = cur.part, jt = cur.jt, slot = cur_slot;
    cur.next(pl);
    if (++cur_slot == D) cur_slot = 0;
    const int off = R.grp_off[grp], n_tok = R.grp_cnt[grp];
    const int tok = g < n_tok ? R.pair_token[off + g] : -1;
    const bool is_lr = LRF == 0 && part >= pl.n_slices;
    float acc_g[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    float acc_u[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    // LRF: the factor bytes of the slice's first low-rank group are requested now and used after
    // the slice's own mma's
    const bool has_lr = LRF > 0 && part < pl.n_lr;
    size_t lr_row = 0;
    uint4 lf_g = {0, 0, 0, 0}, lf_u = {0, 0, 0, 0}, lf2_g = {0, 0, 0, 0}, lf2_u = {0, 0, 0, 0};   // first and second group
    if (LRF > 0 && has_lr) {
      lr_row = (size_t)R.grp_e[grp] * P.I + jt * 8 + g;
      const int rho = part * 32 + 8 * c, rho2 = rho + pl.n_slices * 32;
      if (rho < P.r) {
        if (!up_only) lf_g = __ldg(reinterpret_cast<const uint4*>(P.gate.factor + lr_row * P.r + rho));
        lf_u = __ldg(reinterpret_cast<const uint4*>(P.up.factor + lr_row * P.r + rho));
      }
      if (LRF == 2 && part + pl.n_slices < pl.n_lr && rho2 < P.r) {
        if (!up_only) lf2_g = __ldg(reinterpret_cast<const uint4*>(P.gate.factor + lr_row * P.r + rho2));
        lf2_u = __ldg(reinterpret_cast<const uint4*>(P.up.factor + lr_row * P.r + rho2));
      }
    }
    if (!is_lr) {
      const int b0 = part * 32 + (DENSE ? c : 8 * c);
      if (frag_grp != grp || frag_part != part) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int b = b0 + (DENSE ? 4 * j : j);
          fx[j] = (tok >= 0 && b < nb) ? (pl.x_smem ? s_x[tok * xs + b] : __ldg(x4 + (size_t)tok * nb + b)) : make_uint4(0, 0, 0, 0);
        }
        frag_grp = grp; frag_part = part;
      }
      if (DENSE) {
        const size_t row = (size_t)R.grp_e[grp] * P.I + jt * 8 + g;
        const uint4* wg = reinterpret_cast<const uint4*>(P.gate.dense + row * P.H);
        const uint4* wu = reinterpret_cast<const uint4*>(P.up.dense + row * P.H);
        uint4 vg[8], vu[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int b = b0 + 4 * j;
          vg[j] = (b < nb && !up_only) ? __ldg(wg + b) : make_uint4(0, 0, 0, 0);
          vu[j] = b < nb ? __ldg(wu + b) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) mma_block(acc_u[j & 1], fx[j], vu[j]);
        if (!up_only)
#pragma unroll
          for (int j = 0; j < 8; ++j) mma_block(acc_g[j & 1], fx[j], vg[j]);
      } else {
        // mma.sync needs the whole warp: lanes whose block group lies beyond the row run it
        // with index 0 and zero activation fragments
        uint4 raw_g = {0, 0, 0, 0}, raw_u = {0, 0, 0, 0};
        if (b0 < nb) {
          if (!up_only) raw_g = ring_idx8<IdxT>(ring + (slot * 2 + 0) * 32);
          raw_u = ring_idx8<IdxT>(ring + (slot * 2 + 1) * 32);
        }
        uint32_t ig[8], iu[8];
        slot_idx8<IdxT>(raw_g, idx12, ig);
        slot_idx8<IdxT>(raw_u, idx12, iu);
        if (up_only) {                 // one projection: half the code-word reads and mma's
          if (D4) {
#pragma unroll
            for (int j = 0; j < 8; ++j) mma_block(acc_u[j & 1], fx[j], lookup_d4(s_cb_u, iu[j], lane));
          } else if (pl.repl) {
#pragma unroll
            for (int j = 0; j < 8; ++j) mma_block(acc_u[j & 1], fx[j], s_cb_u[(iu[j] << 3) | (lane & 7)]);
          } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) mma_block(acc_u[j & 1], fx[j], s_cb_u[iu[j]]);
          }
        } else if (D4) {
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            mma_block(acc_g[j & 1], fx[j], lookup_d4(s_cb_g, ig[j], lane));
            mma_block(acc_u[j & 1], fx[j], lookup_d4(s_cb_u, iu[j], lane));
          }
        } else if (pl.repl) {
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            mma_block(acc_g[j & 1], fx[j], s_cb_g[(ig[j] << 3) | (lane & 7)]);
            mma_block(acc_u[j & 1], fx[j], s_cb_u[(iu[j] << 3) | (lane & 7)]);
          }
        } else {
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            mma_block(acc_g[j & 1], fx[j], s_cb_g[ig[j]]);
            mma_block(acc_u[j & 1], fx[j], s_cb_u[iu[j]]);
          }
        }
      }
    } else {
      // low-rank part: B = 8 ranks of this lane's factor row, A = the matching z values (hi, lo)
      const int rho0 = (part - pl.n_slices) * 32 + 8 * c;
      uint4 fg = {0, 0, 0, 0}, fu = {0, 0, 0, 0};
      uint4 zgh = {0, 0, 0, 0}, zgl = {0, 0, 0, 0}, zuh = {0, 0, 0, 0}, zul = {0, 0, 0, 0};
      if (rho0 < P.r) {
        if (!up_only) fg = ring[(slot * 2 + 0) * 32];
        fu = ring[(slot * 2 + 1) * 32];
        if (tok >= 0) {
          const int ig2 = (tok * 2 + P.gate.zslot) * rb + (rho0 >> 3), iu2 = (tok * 2 + P.up.zslot) * rb + (rho0 >> 3);
          zgh = s_zh[ig2]; zgl = s_zl[ig2]; zuh = s_zh[iu2]; zul = s_zl[iu2];
        }
      }
      mma_block_hilo(acc_g[0], zgh, zgl, fg);      // rows 8..15 of the tile carry the lo product
      mma_block_hilo(acc_u[0], zuh, zul, fu);
      acc_g[0][0] += acc_g[0][2]; acc_g[0][1] += acc_g[0][3];
      acc_u[0][0] += acc_u[0][2]; acc_u[0][1] += acc_u[0][3];
    }
    if (LRF > 0 && has_lr) {
      for (int lg = part; lg < pl.n_lr; lg += pl.n_slices) {
        const int rho = lg * 32 + 8 * c;
        if (LRF == 2 && lg == part + pl.n_slices) {     // the second group was requested with the first
          lf_g = lf2_g; lf_u = lf2_u;
        } else if (lg != part) {            // further groups of this slice (ranks beyond 64 * n_slices)
          lf_g = lf_u = make_uint4(0, 0, 0, 0);
          if (rho < P.r) {
            if (!up_only) lf_g = __ldg(reinterpret_cast<const uint4*>(P.gate.factor + lr_row * P.r + rho));
            lf_u = __ldg(reinterpret_cast<const uint4*>(P.up.factor + lr_row * P.r + rho));
          }
        }
        uint4 zgh = {0, 0, 0, 0}, zgl = {0, 0, 0, 0}, zuh = {0, 0, 0, 0}, zul = {0, 0, 0, 0};
        if (rho < P.r && tok >= 0) {
          const int ig2 = (tok * 2 + P.gate.zslot) * rb + (rho >> 3), iu2 = (tok * 2 + P.up.zslot) * rb + (rho >> 3);
          zgh = s_zh[ig2]; zgl = s_zl[ig2]; zuh = s_zh[iu2]; zul = s_zl[iu2];
        }
        mma_block_hilo(acc_g[0], zgh, zgl, lf_g);    // hi product in the accumulators' first halves, lo in the second
        mma_block_hilo(acc_u[0], zuh, zul, lf_u);
      }
      acc_g[0][0] += acc_g[0][2]; acc_g[0][1] += acc_g[0][3];
      acc_u[0][0] += acc_u[0][2]; acc_u[0][1] += acc_u[0][3];
    }
    TRACE_STAMP(0, 6 + 3 * i);
    // partial tile of this part: token g of the group, rows 2c and 2c+1 of the tile
    if (g < n_tok) {
      const size_t at = ((size_t)part * n_pos + off + g) * P.I + jt * 8 + 2 * c;
      *reinterpret_cast<float2*>(P.gpart + at) = make_float2(acc_g[0][0] + acc_g[1][0], acc_g[0][1] + acc_g[1][1]);
      *reinterpret_cast<float2*>(P.upart + at) = make_float2(acc_u[0][0] + acc_u[1][0], acc_u[0][1] + acc_u[1][1]);
    }
  }
  cp_async_wait_pending(0);
  TRACE_STAMP(0, 15);
}

template <typename IdxT, bool DENSE, bool D4, int LRF, bool SP>
__device__ __forceinline__ void gateup_mma_body(const Params& P_in, const bf16* __restrict__ x, int T, const StagePlan& pl_in,
                                                int n_books_in, int want_dbg) {
#ifdef MOE_VQLR_JIT_CHAIN      // the chain compiled for one layer shape: see jit_host.cuh
  Params P = P_in;
  MOE_VQLR_JIT_PARAMS(P);
  StagePlan pl = pl_in;
  MOE_VQLR_JIT_PLAN(pl, GU);
  constexpr int n_books = J_NBOOKS;
  (void)n_books_in;
#else
  const Params& P = P_in;
  const StagePlan& pl = pl_in;
  const int n_books = n_books_in;
#endif
  extern __shared__ uint4 s_u4[];
  const int nwarps = blockDim.x >> 5, warp = threadIdx.x >> 5;
  const GuLayout L = gu_layout(P.K, n_books, T, P.H, P.r, pl, nwarps, P.E, P.k, P.S);
  const GuSmem m = gu_carve(reinterpret_cast<char*>(s_u4), L, P, T, warp, threadIdx.x & 31, pl.depth);
  TRACE_STAMP(0, 0);
  gu_stage_async<DENSE>(P, x, T, pl, n_books, m);
  TRACE_STAMP(0, 1);
  pdl_wait();      // logits and z of this call are complete
  TRACE_STAMP(0, 2);
  gu_route(P, T, pl, m, blockIdx.x == 0, want_dbg != 0);
  Walk w;
  gu_tiles_begin<IdxT, DENSE, SP>(P, pl, m, blockIdx.x * nwarps + warp, gridDim.x * nwarps, w);   // index bytes travel ...
  gu_finish_stage<DENSE>(P, pl, n_books, m, pl.depth - 1);                                     // ... while the stage settles
  pdl_launch();
  TRACE_STAMP(0, 3);
  gu_tiles_run<IdxT, DENSE, D4, LRF, SP>(P, x, T, pl, m, w);
}

template <typename IdxT, bool DENSE, bool D4 = false, int LRF = 0, bool SP = false>
__global__ void __launch_bounds__(DENSE ? kDenseThreads : kFastThreads, 1)
k_gateup_mma(const Params P, const bf16* __restrict__ x, int T, const StagePlan pl, int n_books, int want_dbg) {
  gateup_mma_body<IdxT, DENSE, D4, LRF, SP>(P, x, T, pl, n_books, want_dbg);
}

// ---------------------------------------------------------------------------------------------
// k_act_zdown: one block per pair.  p = silu(sum of gate parts) * (sum of up parts), kept as
// bf16 hi + lo for the down kernel's fragments, then z_d = basis_down * p when the down
// projection is compressed.  Parts are added in ascending order.
// ---------------------------------------------------------------------------------------------
constexpr int kActThreads = 512;

// grid = n_pos * zsplit blocks: block (pos, zs) rebuilds p[pos] (cheap, from L2) and computes the
// z_d rows rho = zs, zs + zsplit, ...; only zs == 0 writes p_hi / p_lo.
// One unit = one (pair, z_d row class): the whole block works on it.  s_p: [I] floats.
__device__ __forceinline__ void act_zdown_unit(const Params& P, int n_pos, int n_parts, int with_zd, int zsplit,
                                               int unit, float* s_p) {
  const int pos = unit / zsplit, zs = unit - pos * zsplit, tid = threadIdx.x;
  const size_t part_stride = (size_t)n_pos * P.I;
  for (int i2 = tid; i2 < P.I / 2; i2 += blockDim.x) {
    float g0 = 0.f, g1 = 0.f, u0 = 0.f, u1 = 0.f;
    const size_t base = (size_t)pos * P.I + 2 * i2;
    for (int part0 = 0; part0 < n_parts; part0 += 6) {        // six parts' loads in flight, summed in order
      float2 gv[6], uv[6];
#pragma unroll
      for (int q = 0; q < 6; ++q) {
        const bool live = part0 + q < n_parts;
        gv[q] = live ? __ldcg(reinterpret_cast<const float2*>(P.gpart + base + (part0 + q) * part_stride)) : make_float2(0.f, 0.f);
        uv[q] = live ? __ldcg(reinterpret_cast<const float2*>(P.upart + base + (part0 + q) * part_stride)) : make_float2(0.f, 0.f);
      }
#pragma unroll
      for (int q = 0; q < 6; ++q) { g0 += gv[q].x; g1 += gv[q].y; u0 += uv[q].x; u1 += uv[q].y; }
    }
    const float p0 = gated_act(g0, u0, P.act), p1 = gated_act(g1, u1, P.act);   // phi(g) * u
    s_p[2 * i2] = p0;
    s_p[2 * i2 + 1] = p1;
    if (zs == 0) {
      const __nv_bfloat162 hi = __floats2bfloat162_rn(p0, p1);
      *reinterpret_cast<__nv_bfloat162*>(P.p_hi + base) = hi;
      *reinterpret_cast<__nv_bfloat162*>(P.p_lo + base) =
          __floats2bfloat162_rn(p0 - __low2float(hi), p1 - __high2float(hi));
    }
  }
  __syncthreads();
  if (!with_zd) return;
  const int lane = tid & 31, warp = tid >> 5, nwarp = blockDim.x >> 5;
  const int nchunk = P.I / 8;
  // two rows of the basis per warp at a time, their loads in flight together
  for (int rho = zs + warp * zsplit; rho < P.r; rho += 2 * nwarp * zsplit) {
    const int rho2 = rho + nwarp * zsplit;
    const bool two = rho2 < P.r;
    const uint4* brow0 = reinterpret_cast<const uint4*>(P.down.basis + (size_t)rho * P.I);
    const uint4* brow1 = reinterpret_cast<const uint4*>(P.down.basis + (size_t)(two ? rho2 : rho) * P.I);
    float acc0 = 0.f, acc1 = 0.f;
    for (int c0 = 0; c0 < nchunk; c0 += 96) {                // three chunks per lane and row in flight
      uint4 w0[3], w1[3];
#pragma unroll
      for (int q = 0; q < 3; ++q) {
        const int cidx = c0 + q * 32 + lane;
        w0[q] = cidx < nchunk ? __ldg(brow0 + cidx) : make_uint4(0, 0, 0, 0);
        w1[q] = cidx < nchunk ? __ldg(brow1 + cidx) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int q = 0; q < 3; ++q) {
        const int cidx = c0 + q * 32 + lane;
        if (cidx < nchunk) {
          const float4 p0 = *reinterpret_cast<const float4*>(s_p + 8 * cidx), p1 = *reinterpret_cast<const float4*>(s_p + 8 * cidx + 4);
          const float pf[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
          float wf[8];
          unpack8(w0[q], wf);
          acc0 = dot8(wf, pf, acc0);
          unpack8(w1[q], wf);
          acc1 = dot8(wf, pf, acc1);
        }
      }
    }
    acc0 = warp_sum(acc0);
    acc1 = warp_sum(acc1);
    if (lane == 0) {
      P.zd[(size_t)pos * P.r + rho] = acc0;
      if (two) P.zd[(size_t)pos * P.r + rho2] = acc1;
    }
  }
}

__device__ __forceinline__ void act_zdown_body(const Params& P_in, int n_pos, int n_parts, int with_zd, int zsplit) {
#ifdef MOE_VQLR_JIT
  Params P = P_in;
  MOE_VQLR_JIT_PARAMS(P);
#else
  const Params& P = P_in;
#endif
  extern __shared__ float s_p[];                 // [I]
  pdl_launch();                                  // the down kernel may stage its code book meanwhile
  pdl_wait();
  act_zdown_unit(P, n_pos, n_parts, with_zd, zsplit, blockIdx.x, s_p);
}

#ifndef MOE_VQLR_JIT
__global__ void __launch_bounds__(kActThreads) k_act_zdown(const Params P, int n_pos, int n_parts, int with_zd, int zsplit) {
  act_zdown_body(P, n_pos, n_parts, with_zd, zsplit);
}
#endif

// The same link as two fully parallel kernels, for layers with few pairs or a long intermediate:
// k_act (one thread per pair of p values) and k_zdown_pdl (one warp per z_d value).
#ifndef MOE_VQLR_JIT      // not part of the single-token path that is compiled per shape
__global__ void __launch_bounds__(256) k_act(const Params P, int n_pos, int n_parts) {
  pdl_launch();
  pdl_wait();
  const int I2 = P.I / 2;
  const size_t part_stride = (size_t)n_pos * P.I;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n_pos * I2; i += gridDim.x * blockDim.x) {
    const size_t base = 2 * (size_t)i;                      // = pos * I + 2 * i2
    float g0 = 0.f, g1 = 0.f, u0 = 0.f, u1 = 0.f;
    for (int part0 = 0; part0 < n_parts; part0 += 6) {
      float2 gv[6], uv[6];
#pragma unroll
      for (int q = 0; q < 6; ++q) {
        const bool live = part0 + q < n_parts;
        gv[q] = live ? __ldcg(reinterpret_cast<const float2*>(P.gpart + base + (part0 + q) * part_stride)) : make_float2(0.f, 0.f);
        uv[q] = live ? __ldcg(reinterpret_cast<const float2*>(P.upart + base + (part0 + q) * part_stride)) : make_float2(0.f, 0.f);
      }
#pragma unroll
      for (int q = 0; q < 6; ++q) { g0 += gv[q].x; g1 += gv[q].y; u0 += uv[q].x; u1 += uv[q].y; }
    }
    const float p0 = gated_act(g0, u0, P.act), p1 = gated_act(g1, u1, P.act);
    *reinterpret_cast<float2*>(P.p + base) = make_float2(p0, p1);
    const __nv_bfloat162 hi = __floats2bfloat162_rn(p0, p1);
    *reinterpret_cast<__nv_bfloat162*>(P.p_hi + base) = hi;
    *reinterpret_cast<__nv_bfloat162*>(P.p_lo + base) =
        __floats2bfloat162_rn(p0 - __low2float(hi), p1 - __high2float(hi));
  }
}
#endif

// wpd warps share one z_d value (a long intermediate would otherwise be one warp's serial stream
// of dependent loads); their partial sums meet in shared memory and are added in warp order.
#ifndef MOE_VQLR_JIT      // not part of the single-token path that is compiled per shape
__global__ void __launch_bounds__(256) k_zdown_pdl(const Params P, int n_pos, int wpd) {
  __shared__ float s_part[8];
  pdl_launch();
  pdl_wait();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int dots_per_block = 8 / wpd;
  const int d = blockIdx.x * dots_per_block + warp / wpd, seg = warp % wpd;
  const bool live_dot = d < n_pos * P.r;
  float acc = 0.f;
  if (live_dot) {
    const int pos = d / P.r, rho = d - pos * P.r;
    const uint4* brow = reinterpret_cast<const uint4*>(P.down.basis + (size_t)rho * P.I);
    const float4* prow = reinterpret_cast<const float4*>(P.p + (size_t)pos * P.I);
    const int nchunk = P.I / 8;
    const int per = (nchunk + wpd - 1) / wpd, c_begin = seg * per, c_end = min(nchunk, c_begin + per);
    for (int c0 = c_begin; c0 < c_end; c0 += 128) {
      uint4 wv[4];
      float4 pa[4], pb[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int cidx = c0 + q * 32 + lane;
        const bool live = cidx < c_end;
        wv[q] = live ? __ldg(brow + cidx) : make_uint4(0, 0, 0, 0);
        pa[q] = live ? __ldcg(prow + 2 * cidx) : make_float4(0.f, 0.f, 0.f, 0.f);
        pb[q] = live ? __ldcg(prow + 2 * cidx + 1) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        float wf[8];
        unpack8(wv[q], wf);
        const float pf[8] = {pa[q].x, pa[q].y, pa[q].z, pa[q].w, pb[q].x, pb[q].y, pb[q].z, pb[q].w};
        acc = dot8(wf, pf, acc);
      }
    }
    acc = warp_sum(acc);
  }
  if (lane == 0) s_part[warp] = acc;
  __syncthreads();
  if (live_dot && seg == 0 && lane == 0) {
    float sum = 0.f;
    for (int q = 0; q < wpd; ++q) sum += s_part[warp + q];
    P.zd[d] = sum;
  }
}
#endif

// The same with four consecutive ranks per unit (many pairs: the pair's p values, two thirds of the
// bytes of a dot product, are loaded once for four basis rows).
#ifndef MOE_VQLR_JIT      // not part of the single-token path that is compiled per shape
__global__ void __launch_bounds__(256) k_zdown4_pdl(const Params P, int n_pos, int wpd) {
  // one unit = (pair, four consecutive ranks): the pair's p values are loaded once for the four rows
  __shared__ float s_part[8][4];
  pdl_launch();
  pdl_wait();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int units_per_block = 8 / wpd, rq = P.r / 4;
  const int d = blockIdx.x * units_per_block + warp / wpd, seg = warp % wpd;
  const bool live_unit = d < n_pos * rq;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  int pos = 0, rho = 0;
  if (live_unit) {
    pos = d / rq; rho = (d - pos * rq) * 4;
    const uint4* brow = reinterpret_cast<const uint4*>(P.down.basis + (size_t)rho * P.I);
    const float4* prow = reinterpret_cast<const float4*>(P.p + (size_t)pos * P.I);
    const int nchunk = P.I / 8;
    const int per = (nchunk + wpd - 1) / wpd, c_begin = seg * per, c_end = min(nchunk, c_begin + per);
    for (int c0 = c_begin; c0 < c_end; c0 += 64) {
      uint4 wv[2][4];
      float4 pa[2], pb[2];
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const int cidx = c0 + q * 32 + lane;
        const bool live = cidx < c_end;
#pragma unroll
        for (int j = 0; j < 4; ++j) wv[q][j] = live ? __ldg(brow + (size_t)j * nchunk + cidx) : make_uint4(0, 0, 0, 0);
        pa[q] = live ? __ldcg(prow + 2 * cidx) : make_float4(0.f, 0.f, 0.f, 0.f);
        pb[q] = live ? __ldcg(prow + 2 * cidx + 1) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const float pf[8] = {pa[q].x, pa[q].y, pa[q].z, pa[q].w, pb[q].x, pb[q].y, pb[q].z, pb[q].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          float wf[8];
          unpack8(wv[q][j], wf);
          acc[j] = dot8(wf, pf, acc[j]);
        }
      }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[j] = warp_sum(acc[j]);
  }
  if (lane == 0) {
#pragma unroll
    for (int j = 0; j < 4; ++j) s_part[warp][j] = acc[j];
  }
  __syncthreads();
  if (live_unit && seg == 0 && lane < 4) {
    float sum = 0.f;
    for (int q = 0; q < wpd; ++q) sum += s_part[warp + q][lane];
    P.zd[(size_t)pos * P.r + rho + lane] = sum;
  }
}
#endif

// ---------------------------------------------------------------------------------------------
// k_down_mma: partial y tiles for every (work group, slice of I, 8-row tile of H); activations
// are the bf16 hi + lo halves of p.  The warp of slice s also adds the low-rank groups s,
// s + n_slices, ... (32 ranks each; A = z_d as hi + lo), so the parts are the slices alone.
// ---------------------------------------------------------------------------------------------
struct DnLayout {
  size_t ring, grp, cb_tmp, total;
  int slot_u4;      // uint4 per lane per ring slot: 2 (indices, factor) or 8 (a dense 256-value slice)
};

__host__ __device__ inline DnLayout dn_layout(int K, bool vq, const StagePlan& pl, int warps, int max_groups) {
  DnLayout L;
  size_t o = vq ? (size_t)K * 16 * (pl.repl ? 8 : 1) : 0;
  L.slot_u4 = vq ? 2 * pl.tpu : 8;
  L.ring = o;   o += (size_t)warps * pl.depth * L.slot_u4 * 32 * 16;
  L.grp = o;    o += ((size_t)max_groups * 12 + 15) / 16 * 16;
  L.cb_tmp = o; o += (vq && pl.repl) ? (size_t)K * 16 : 0;
  L.total = o;
  return L;
}

// Shared-memory views of the down stage.  ring: this lane's slot base; grp_*: work groups.
struct DnSmem {
  const uint4* cb;
  uint4* ring;
  int slot_u4;
  const int *grp_e, *grp_off, *grp_cnt;
  int n_grp;
};

// Streams the bytes of the prefetch cursor's unit into the ring and advances that cursor.
template <typename IdxT, bool DENSE, int TPU = 2, bool SP = false>
__device__ __forceinline__ void dn_issue(const Params& P, const StagePlan& pl, const DnSmem& m, Walk& w) {
  const int lane = threadIdx.x & 31, g = lane >> 2, c = lane & 3, nb = pl.nb;
  uint4* ring = m.ring;
  const Cursor& pf = w.pf;
  const size_t row = (size_t)m.grp_e[pf.grp] * P.H + pf.jt * (DENSE ? 8 : 8 * TPU) + g;
  if (DENSE) {
    const uint4* wd = reinterpret_cast<const uint4*>(P.down.dense + row * P.I) + pf.part * 32 + c;
#pragma unroll
    for (int j = 0; j < 8; ++j)
      if (pf.part * 32 + c + 4 * j < nb) cp_async16(ring + (w.pf_slot * 8 + j) * 32, wd + 4 * j);
  } else {
    const IdxT* idx_d = static_cast<const IdxT*>(P.down.idx);
    const int b = pf.part * 32 + 8 * c, rho = pf.part * 32 + 8 * c;
#pragma unroll
    for (int sub = 0; sub < TPU; ++sub) {
      const size_t rs = row + 8 * sub;
      uint4* slot = ring + (size_t)(w.pf_slot * TPU + sub) * 2 * 32;
      if (b < nb) cp_async_idx8<IdxT>(slot, idx_at(idx_d, rs * nb + b, SP ? P.idx12 : 0), SP ? P.idx12 : 0);
      if (pf.part < pl.n_lr && rho < P.r) cp_async16(slot + 32, P.down.factor + rs * P.r + rho);
    }
  }
  w.pf.next(pl);
  if (++w.pf_slot == pl.depth) w.pf_slot = 0;
}

// Start of the walk of warp `wid` out of `W` warps (needs only the work groups, not p).
template <typename IdxT, bool DENSE, int TPU = 2, bool SP = false>
__device__ __forceinline__ void dn_tiles_begin(const Params& P, const StagePlan& pl, const DnSmem& m, int wid, int W, Walk& w) {
  const int per_grp = pl.n_parts * pl.tiles;
  int V = m.n_grp * per_grp, v0 = 0;
  if (pl.only_grp >= 0) { V = pl.only_grp < m.n_grp ? per_grp : 0; v0 = pl.only_grp * per_grp; }
  const int v_begin = split_begin(V, pl, wid);         // W == pl.W by construction of the launch
  w.n_my = split_begin(V, pl, wid + 1) - v_begin;
  w.pf.set(w.n_my > 0 ? v0 + v_begin : 0, pl);
  w.cur = w.pf;
  w.pf_slot = 0; w.cur_slot = 0;
  for (int i = 0; i < pl.depth - 1; ++i) { if (i < w.n_my) dn_issue<IdxT, DENSE, TPU, SP>(P, pl, m, w); cp_async_commit(); }
  TRACE_STAMP(2, 3);
}

// The tile loop proper (needs p, z_d and the code book).
template <typename IdxT, bool DENSE, bool D4 = false, int TPU = 2, bool SP = false>
__device__ __forceinline__ void dn_tiles_run(const Params& P, int T, const StagePlan& pl, const DnSmem& m, Walk& w) {
  const int lane = threadIdx.x & 31, g = lane >> 2, c = lane & 3;
  const int nb = pl.nb, D = pl.depth;
  const int n_pos = T * (P.k + P.S), n_my = w.n_my;
  struct { int slot_u4; } L = {m.slot_u4};
  const uint4* s_cb = m.cb;
  uint4* ring = m.ring;
  const int *s_grp_e = m.grp_e, *s_grp_off = m.grp_off, *s_grp_cnt = m.grp_cnt;
  Cursor& cur = w.cur;
  int& cur_slot = w.cur_slot;
  auto issue = [&]() { dn_issue<IdxT, DENSE, TPU, SP>(P, pl, m, w); };

  uint4 fh[8], fl[8];
  uint4 zh = {0, 0, 0, 0}, zl = {0, 0, 0, 0};     // z_d fragments of the low-rank group this part carries
  int frag_grp = -1, frag_part = -1;

  for (int i = 0; i < n_my; ++i) {
    if (i + D - 1 < n_my) issue();
    cp_async_commit();
    cp_async_wait_pending(D - 1);
    if (i < 5) TRACE_STAMP(2, 4 + 2 * i);
    const int grp = cur.grp, part = cur.part, jt = cur.jt, slot = cur_slot;
    cur.next(pl);
    if (++cur_slot == D) cur_slot = 0;
    const int off = s_grp_off[grp], n_tok = s_grp_cnt[grp];
    const int pos = g < n_tok ? off + g : -1;
    const int b0 = part * 32 + (DENSE ? c : 8 * c);
    const int rho0 = part * 32 + 8 * c;
    if (frag_grp != grp || frag_part != part) {
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
      zh = zl = make_uint4(0, 0, 0, 0);
      if (!DENSE && part < pl.n_lr && pos >= 0 && rho0 < P.r) {
        const float4* zp = reinterpret_cast<const float4*>(P.zd + (size_t)pos * P.r + rho0);
        split_hi_lo(__ldcg(zp), __ldcg(zp + 1), zh, zl);
      }
      frag_grp = grp; frag_part = part;
    }
#pragma unroll
    for (int sub = 0; sub < (DENSE ? 1 : TPU); ++sub) {
    const int row0 = DENSE ? jt * 8 : (jt * TPU + sub) * 8;      // first row of this 8-row tile
    float acc[4][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};   // four independent chains
    if (DENSE) {
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint4 v = b0 + 4 * j < nb ? ring[(slot * 8 + j) * 32] : make_uint4(0, 0, 0, 0);
        mma_block_hilo(acc[j & 1], fh[j], fl[j], v);
      }
    } else {
      // mma.sync needs the whole warp: out-of-range block groups use index 0 and zero fragments
      const uint4* uslot = ring + (size_t)(slot * TPU + sub) * 2 * 32;
      uint4 raw = {0, 0, 0, 0};
      if (b0 < nb) raw = ring_idx8<IdxT>(uslot);
      uint32_t id[8];
      slot_idx8<IdxT>(raw, SP ? P.idx12 : 0, id);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint4 w = D4 ? lookup_d4(s_cb, id[j], lane) : s_cb[pl.repl ? ((id[j] << 3) | (lane & 7)) : id[j]];
        mma_block_hilo(acc[j & 1], fh[j], fl[j], w);      // hi product in rows 0..7 of the tile, lo in rows 8..15
      }
      if (part < pl.n_lr) {                   // warp-uniform: the low-rank group carried by this part
        const uint4 f = rho0 < P.r ? uslot[32] : make_uint4(0, 0, 0, 0);
        mma_block_hilo(acc[2], zh, zl, f);
        const size_t row = (size_t)s_grp_e[grp] * P.H + row0 + g;
        for (int lg = part + pl.n_slices; lg < pl.n_lr; lg += pl.n_slices) {   // more rank groups than slices
          const int rho = lg * 32 + 8 * c;
          uint4 f2 = {0, 0, 0, 0}, zh2 = {0, 0, 0, 0}, zl2 = {0, 0, 0, 0};
          if (rho < P.r) {
            f2 = __ldg(reinterpret_cast<const uint4*>(P.down.factor + row * P.r + rho));
            if (pos >= 0) {
              const float4* zp = reinterpret_cast<const float4*>(P.zd + (size_t)pos * P.r + rho);
              split_hi_lo(__ldcg(zp), __ldcg(zp + 1), zh2, zl2);
            }
          }
          mma_block_hilo(acc[3], zh2, zl2, f2);
        }
      }
    }
    if (pos >= 0) {
      const size_t at = ((size_t)part * n_pos + pos) * P.H + row0 + 2 * c;
      *reinterpret_cast<float2*>(P.ypart + at) =
          make_float2(((acc[0][0] + acc[0][2]) + (acc[1][0] + acc[1][2])) + ((acc[2][0] + acc[2][2]) + (acc[3][0] + acc[3][2])),
                      ((acc[0][1] + acc[0][3]) + (acc[1][1] + acc[1][3])) + ((acc[2][1] + acc[2][3]) + (acc[3][1] + acc[3][3])));
    }
    }
    if (i < 5) TRACE_STAMP(2, 5 + 2 * i);
  }
  cp_async_wait_pending(0);
  TRACE_STAMP(2, 15);
}

template <typename IdxT, bool DENSE, bool D4, int TPU, bool SP>
__device__ __forceinline__ void down_mma_body(const Params& P_in, int T, const StagePlan& pl_in) {
#ifdef MOE_VQLR_JIT_CHAIN
  Params P = P_in;
  MOE_VQLR_JIT_PARAMS(P);
  StagePlan pl = pl_in;
  MOE_VQLR_JIT_PLAN(pl, DN);
#else
  const Params& P = P_in;
  const StagePlan& pl = pl_in;
#endif
  extern __shared__ uint4 s_u4[];
  char* s_base = reinterpret_cast<char*>(s_u4);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int D = pl.depth, nwarps = blockDim.x >> 5;
  const int n_pos = T * (P.k + P.S);
  const DnLayout L = dn_layout(P.K, !DENSE, pl, nwarps, n_pos);
  uint4* s_cb = s_u4;
  uint4* ring = reinterpret_cast<uint4*>(s_base + L.ring) + (size_t)warp * D * L.slot_u4 * 32 + lane;   // [slot][chunk][lane]
  int* s_grp_e = reinterpret_cast<int*>(s_base + L.grp);
  int* s_grp_off = s_grp_e + n_pos;
  int* s_grp_cnt = s_grp_off + n_pos;
  TRACE_STAMP(2, 0);
  uint4* s_tmp = reinterpret_cast<uint4*>(s_base + L.cb_tmp);
  if (!DENSE) {
    uint4* dst = pl.repl ? s_tmp : s_cb;
    const int kw = D4 ? P.K / 2 : P.K;
    for (int i = tid; i < kw; i += blockDim.x) cp_async16(dst + i, P.down.codebook + i);
  }
  cp_async_commit();
  pdl_wait();      // p (and z_d) and the routing lists are complete
  TRACE_STAMP(2, 1);
  pdl_launch();
  const int n_grp = __ldcg(P.grp_n);
  for (int i = tid; i < n_pos; i += blockDim.x) {      // all n_pos slots (>= n_grp): no dependent second trip
    s_grp_e[i] = __ldcg(P.grp_e + i); s_grp_off[i] = __ldcg(P.grp_off + i); s_grp_cnt[i] = __ldcg(P.grp_cnt + i);
  }
  __syncthreads();                 // work groups are in shared memory
  DnSmem m;
  m.cb = s_cb; m.ring = ring; m.slot_u4 = L.slot_u4;
  m.grp_e = s_grp_e; m.grp_off = s_grp_off; m.grp_cnt = s_grp_cnt; m.n_grp = n_grp;
  Walk w;
  dn_tiles_begin<IdxT, DENSE, TPU, SP>(P, pl, m, blockIdx.x * nwarps + warp, gridDim.x * nwarps, w);   // index bytes travel ...
  cp_async_wait_pending(D - 1);                                                                // ... the code book has landed
  __syncthreads();
  if (!DENSE && pl.repl) {
    if (D4) {
      uint2* c2 = reinterpret_cast<uint2*>(s_cb);
      const uint2* t2 = reinterpret_cast<const uint2*>(s_tmp);
      for (int i = tid; i < P.K * 16; i += blockDim.x) c2[i] = t2[i >> 4];
    } else {
      for (int i = tid; i < P.K * 8; i += blockDim.x) s_cb[i] = s_tmp[i >> 3];
    }
    __syncthreads();
  }
  TRACE_STAMP(2, 2);
  dn_tiles_run<IdxT, DENSE, D4, TPU, SP>(P, T, pl, m, w);
}

template <typename IdxT, bool DENSE, bool D4 = false, int TPU = 2, bool SP = false>
__global__ void __launch_bounds__(kDownThreads, 1)
k_down_mma(const Params P, int T, const StagePlan pl) {
  down_mma_body<IdxT, DENSE, D4, TPU, SP>(P, T, pl);
}

// out[t][h] = sum over slots (in slot order) of affinity * y[t][slot][h], where y is the sum of
// the down kernel's parts (ascending); shared experts weigh 1.  One block = one token and 64
// pairs of columns; thread (column pair, slot lane) adds the parts of its slots with all loads
// in flight, then the slot sums meet in shared memory and are added in slot order.
constexpr int kCombineCols = 64;    // float2 columns per unit
constexpr int kCombineSlots = 8;    // slot lanes per column in the stand-alone kernel

__device__ __forceinline__ int combine_units(const Params& P, int T) {
  return T * ((P.H / 2 + kCombineCols - 1) / kCombineCols);
}

// One unit = one token and 64 pairs of columns; the whole block works on it (blockDim a multiple
// of 64).  s_y: [k + S][64] float2.
__device__ __forceinline__ void combine_unit(const Params& P, bf16* __restrict__ out, int T, int n_parts, int unit,
                                             float2 (*s_y)[kCombineCols]) {
  const int n_slots = P.k + P.S, H2 = P.H / 2, n_pos = T * n_slots;
  const int blocks_per_tok = (H2 + kCombineCols - 1) / kCombineCols;
  const int col = threadIdx.x % kCombineCols, sl = threadIdx.x / kCombineCols, n_sl = blockDim.x / kCombineCols;
  const int t = unit / blocks_per_tok, h2 = (unit - t * blocks_per_tok) * kCombineCols + col;
  const size_t part_stride = (size_t)n_pos * P.H;
  // fewer slots than slot lanes (few experts per token): lps lanes share one slot's parts, lane q of
  // them adds the parts q, q + lps, ...; the partial sums are added in (slot, q) order below
  const int lps = n_slots < n_sl ? n_sl / n_slots : 1;
  const int n_rows = n_slots * lps;
  if (lps == 1) {
    for (int s = sl; s < n_slots; s += n_sl) {
      const int pos = __ldcg(P.inv_pos + t * n_slots + s);
      const float w = __ldcg(P.pair_w + pos);
      float y0 = 0.f, y1 = 0.f;
      if (h2 < H2) {
        const float* src = P.ypart + (size_t)pos * P.H + 2 * h2;
        for (int part0 = 0; part0 < n_parts; part0 += 4) {
          float2 v[4];
#pragma unroll
          for (int q = 0; q < 4; ++q)
            v[q] = part0 + q < n_parts ? __ldcg(reinterpret_cast<const float2*>(src + (part0 + q) * part_stride)) : make_float2(0.f, 0.f);
#pragma unroll
          for (int q = 0; q < 4; ++q) { y0 += v[q].x; y1 += v[q].y; }
        }
      }
      s_y[s][col] = make_float2(w * y0, w * y1);
    }
  } else if (sl < n_rows) {
    const int s = sl / lps, q0 = sl - s * lps;
    const int pos = __ldcg(P.inv_pos + t * n_slots + s);
    const float w = __ldcg(P.pair_w + pos);
    float y0 = 0.f, y1 = 0.f;
    if (h2 < H2) {
      const float* src = P.ypart + (size_t)pos * P.H + 2 * h2 + q0 * part_stride;
      const size_t stride = part_stride * lps;
      const int n_mine = (n_parts - q0 + lps - 1) / lps;
      for (int i0 = 0; i0 < n_mine; i0 += 4) {
        float2 v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q)
          v[q] = i0 + q < n_mine ? __ldcg(reinterpret_cast<const float2*>(src + (i0 + q) * stride)) : make_float2(0.f, 0.f);
#pragma unroll
        for (int q = 0; q < 4; ++q) { y0 += v[q].x; y1 += v[q].y; }
      }
    }
    s_y[sl][col] = make_float2(w * y0, w * y1);
  }
  __syncthreads();
  if (sl == 0 && h2 < H2) {
    float a0 = 0.f, a1 = 0.f;
    for (int s = 0; s < n_rows; ++s) { a0 += s_y[s][col].x; a1 += s_y[s][col].y; }
    *reinterpret_cast<__nv_bfloat162*>(out + (size_t)t * P.H + 2 * h2) = __floats2bfloat162_rn(a0, a1);
  }
}

__device__ __forceinline__ void combine_body(const Params& P_in, bf16* __restrict__ out, int T, int n_parts) {
#ifdef MOE_VQLR_JIT
  Params P = P_in;
  MOE_VQLR_JIT_PARAMS(P);
#else
  const Params& P = P_in;
#endif
  __shared__ float2 s_y[kMaxK + 8][kCombineCols];       // affinity-weighted y per slot (k + S <= 40)
  pdl_wait();
  pdl_launch();
  combine_unit(P, out, T, n_parts, blockIdx.x, s_y);
}

#ifndef MOE_VQLR_JIT
__global__ void __launch_bounds__(kCombineCols * kCombineSlots)
k_combine(const Params P, bf16* __restrict__ out, int T, int n_parts) {
  combine_body(P, out, T, n_parts);
}
#endif

}  // namespace
