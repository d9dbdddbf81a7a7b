// One routed MoE decode layer on VQ + shared-basis low-rank expert weights (sm_100a).
// Host side of the C ABI declared in include/moe_vqlr.h plus the kernels it launches.
//
// Two kernel chains (all on the caller's stream):
//   fast (tensor cores, fast_kernels.cuh), for shapes whose rows split into whole groups of
//   eight blocks:  k_router_z_pdl -> k_gateup_mma -> k_act_zdown -> k_down_mma -> k_combine
//   generic (generic_kernels.cuh), for everything else:
//                  k_router_z -> k_route -> k_gateup -> [k_zdown] -> k_down
// Stages: router logits and the shared rank-r projections z = basis * x (Section 4.1: the work
// that does not depend on the routing decision); top-k, affinities, grouping; gate/up rows of
// every activated expert straight from indices + code book with the low-rank term joined in
// the same accumulator, then SwiGLU (Eq. 1); z_d = basis_down * p per pair when the down
// projection is compressed too; down rows; affinity-weighted sum.
#include "common.cuh"
#include "generic_kernels.cuh"
#include "fast_kernels.cuh"
#include "coop_kernel.cuh"
#include "fused_kernel.cuh"
#include "pcb_kernel.cuh"
#include "jit_host.cuh"

#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <string>
#include <utility>

namespace {

thread_local std::string g_create_error;

}  // namespace

struct moe_vqlr_handle {
  moe_vqlr_config cfg;
  Params P;
  int device;
  int sm_count;
  int idx_bytes;
  int two_books;
  size_t smem_gateup_per_token, smem_gateup_fixed, smem_down;
  bool fast;                 // tensor-core chain eligible for this configuration
  bool coop;                 // ... and run as one persistent cooperative kernel
  int dn_restage;            // the down projection has a code book (or layout) of its own
  size_t smem_coop;
  int want_dbg;              // the running call asked for counts / offsets
  bool gu_dense, dn_dense;
  int n_books;               // distinct gate/up code books staged by k_gateup_mma
  StagePlan plan_gu, plan_dn;
  StagePlan plan_gu_coop, plan_dn_coop;   // the same cuts with ring depths chosen for the cooperative kernel
  size_t smem_fast_dn;
  bool fused;                // router -> one kernel per (work group, slice of I) -> weighted sum
  bool fused_forced;         // ... also for calls whose items exceed one wave (tests)
  int fused_max_T;           // ... for calls of up to this many tokens (shared memory)
  FusedPlan fplan;
  signed char fused_dg[kMaxT + 1], fused_dd[kMaxT + 1];   // ring depths that fit for T tokens (0: the chain runs)
  signed char fused_w[kMaxT + 1];                         // ... and with this many warps per block (16 where they fit, else 12)
  signed char fused_xs[kMaxT + 1];                        // ... with the tokens staged in shared memory (else read from L2)
  StagePlan plan_gu_fused;
  bool per_expert_launch;   // ablation: gate/up and down run as one launch per work group
  bool special;             // up-only experts or 12-bit indices: the tensor-core kernels' SP instantiations run
  bool d4;                  // four-value code words on the tensor-core paths (uint8 indices read as pairs)
  int idx_tc;               // bytes per index element as the tensor-core kernels read it (2 with d4)
  bool lrf;                 // chain gate/up: the low-rank groups ride on the slices (at least one per slice)
  bool lrf2;                // ... and some slices carry two or more
  bool pcb;                 // gate/up through the projection code book is available (K <= 256, uint8, d = 8)
  int pcb_min_T;            // ... and used from this many tokens on
  int pcb_Q;                // table pieces per token = ceil(H / 8 / 64)
  size_t smem_lr;           // dynamic shared memory of k_gateup_lr
  const void* jit_fused;     // k_expert_fused compiled at create() for this layer's shape (single-token calls), or NULL
  const void* jit_router;    // ... and the kernels before and after it
  const void* jit_combine;
  // the chain of kernels (calls of several tokens) compiled for this layer's shape, or NULL each
  const void *jit_c_gateup, *jit_c_down, *jit_c_combine;      // (its router and activation kernels measured slower that way)
  std::string jit_note;      // why there is none
  void* idx_dp;              // down index map re-laid per slice (inside the workspace)
  void* workspace;
  size_t workspace_bytes;
  int* status_host;          // the status word: pinned host memory that the kernels write through a mapped pointer
  bf16* x_stage;     // [maxT][H] device staging for the host-buffer entry point
  bf16* out_stage;   // [maxT][H]
  cudaStream_t cap_stream;                 // only ever used to capture the graphs below
  cudaGraphExec_t host_graph[kMaxT + 1];   // kernel chain x_stage -> out_stage for T tokens
  cudaGraphExec_t io_graph[kMaxT + 1];     // the same with both host copies inside, for the host buffers below
  const void* io_x[kMaxT + 1];
  void* io_out[kMaxT + 1];
  bool io_stage_in[kMaxT + 1];             // ... whose tokens come in through k_stage_in (one more kernel per call)
  bool io_graph_failed;                    // host buffers that cannot be captured (pageable): copies stay outside
  int host_graph_launches;                 // kernels in one such graph
  int64_t launches;
  int profiling;             // record an event after every stage of a call
  cudaEvent_t ev[kStages + 1];
  bool ev_valid;
  bool stage_ran[kStages];
  std::string error;
};

namespace {

int fail(moe_vqlr_handle* h, int code, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (h) h->error = buf; else g_create_error = buf;
  return code;
}

// cudaFuncAttributeMaxDynamicSharedMemorySize belongs to the kernel (per device), not to a handle:
// it is only ever raised, so that a handle with a smaller need cannot lower it under a live one.
std::mutex g_attr_mu;
std::map<std::pair<int, const void*>, size_t> g_attr_max;
cudaError_t raise_dyn_smem(const void* fn, size_t bytes) {
  int dev = 0;
  cudaError_t ce = cudaGetDevice(&dev);
  if (ce != cudaSuccess) return ce;
  std::lock_guard<std::mutex> lock(g_attr_mu);
  size_t& cur = g_attr_max[std::make_pair(dev, fn)];
  if (bytes <= cur) return cudaSuccess;
  ce = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (ce == cudaSuccess) cur = bytes;
  return ce;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Tokens from the caller's pinned host buffer into the staging buffer, 16 bytes per thread: as a
// kernel of the programmatic-launch chain it costs less than a copy node of the graph, and the
// router's weight rows (requested before its dependency wait) travel meanwhile.
__global__ void __launch_bounds__(256) k_stage_in(const uint4* __restrict__ src_host, uint4* __restrict__ dst, int n16) {
  pdl_wait();        // the previous call's kernels may still read the staging buffer
  pdl_launch();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n16) dst[i] = src_host[i];
}


template <typename... KArgs, typename... Args>
cudaError_t launch_coop(void (*kern)(KArgs...), int grid, int block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeCooperative;
  at[0].val.cooperative = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

// Cuts one projection stage into slices and teams for `warps` warps per block.
StagePlan plan_stage(int out_dim, int in_dim, int r, bool dense) {
  StagePlan pl;
  pl.nb = in_dim / kD;
  pl.n_slices = (pl.nb + 31) / 32;
  pl.n_lr = (!dense && r > 0) ? (r + 31) / 32 : 0;
  pl.n_parts = pl.n_slices + pl.n_lr;
  pl.tiles = out_dim / 8;
  pl.depth = 2;
  pl.chunk = pl.tiles;
  pl.x_smem = 1;
  pl.repl = 0;
  pl.tpu = 1;
  return pl;
}

// After the last change to a plan: the derived constants of the work-list arithmetic.
void finish_plan(StagePlan& pl, int W) {
  pl.W = W;
  pl.only_grp = -1;
  pl.tail = pl.tiles % pl.chunk;
  pl.d_per_grp = make_fastdiv((unsigned int)(pl.n_parts * pl.tiles));
  pl.d_per_chunk = make_fastdiv((unsigned int)(pl.n_parts * pl.chunk));
  pl.d_chunk = make_fastdiv((unsigned int)pl.chunk);
  pl.d_tail = make_fastdiv((unsigned int)(pl.tail > 0 ? pl.tail : 1));
  pl.d_W = make_fastdiv((unsigned int)W);
}

// Launch as a link of a programmatic-dependent-launch chain.  On the legacy default stream
// (NULL) and the per-thread default stream the attribute is left out and the kernels run in
// plain stream order (their griddepcontrol instructions are then no-ops).
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kern)(KArgs...), int grid, int block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  const bool chain = st != nullptr && st != cudaStreamLegacy && st != cudaStreamPerThread;
  cfg.attrs = at;
  cfg.numAttrs = chain ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

int check_proj(const moe_vqlr_proj& p, const char* name, int rank) {
  if (p.kind == MOE_VQLR_PROJ_VQLR) {
    if (!p.codebook || !p.idx) return fail(nullptr, MOE_VQLR_ERR_INVALID_ARG, "%s: codebook/idx is null", name);
    if (rank > 0 && (!p.basis || !p.factor))
      return fail(nullptr, MOE_VQLR_ERR_INVALID_ARG, "%s: rank > 0 but basis/factor is null", name);
    if (!aligned16(p.codebook) || !aligned16(p.idx) || !aligned16(p.basis) || !aligned16(p.factor))
      return fail(nullptr, MOE_VQLR_ERR_INVALID_ARG, "%s: pointers must be 16-byte aligned", name);
  } else if (p.kind == MOE_VQLR_PROJ_DENSE_BF16) {
    if (!p.dense) return fail(nullptr, MOE_VQLR_ERR_INVALID_ARG, "%s: dense is null", name);
    if (!aligned16(p.dense)) return fail(nullptr, MOE_VQLR_ERR_INVALID_ARG, "%s: dense must be 16-byte aligned", name);
  } else {
    return fail(nullptr, MOE_VQLR_ERR_INVALID_ARG, "%s: unknown kind %d", name, p.kind);
  }
  return MOE_VQLR_OK;
}

ProjDev make_proj(const moe_vqlr_proj& p, int out_dim, int in_dim) {
  ProjDev d;
  d.kind = p.kind;
  d.out_dim = out_dim;
  d.in_dim = in_dim;
  d.zslot = -1;
  d.codebook = static_cast<const uint4*>(p.codebook);
  d.idx = p.idx;
  d.basis = static_cast<const bf16*>(p.basis);
  d.factor = static_cast<const bf16*>(p.factor);
  d.dense = static_cast<const bf16*>(p.dense);
  return d;
}

template <typename T>
T* carve(char*& cur, size_t n) {
  T* p = reinterpret_cast<T*>(cur);
  cur += (n * sizeof(T) + 255) / 256 * 256;
  return p;
}

// Launch through an untyped kernel pointer (the selectors below), as a link of the chain.
cudaError_t launch_pdl_ptr(const void* kern, int grid, int block, size_t smem, cudaStream_t st, void** args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  const bool chain = st != nullptr && st != cudaStreamLegacy && st != cudaStreamPerThread;
  cfg.attrs = at;
  cfg.numAttrs = chain ? 1 : 0;
  return cudaLaunchKernelExC(&cfg, kern, args);
}

// Which instantiation of a tensor-core kernel a handle runs.  SP = the instantiations that also
// handle experts without a gate projection and 12-bit packed indices.
template <bool SP>
const void* gateup_kernel_sp(bool gu_dense, bool d4, int idx_bytes, bool lrf, bool lrf2) {
  if (gu_dense) return (const void*)k_gateup_mma<uint16_t, true, false, 0, SP>;
  if (d4) return lrf2 ? (const void*)k_gateup_mma<uint16_t, false, true, 2, SP> : lrf ? (const void*)k_gateup_mma<uint16_t, false, true, 1, SP>
                                                                                       : (const void*)k_gateup_mma<uint16_t, false, true, 0, SP>;
  if (idx_bytes == 1) return lrf2 ? (const void*)k_gateup_mma<uint8_t, false, false, 2, SP> : lrf ? (const void*)k_gateup_mma<uint8_t, false, false, 1, SP>
                                                                                                   : (const void*)k_gateup_mma<uint8_t, false, false, 0, SP>;
  return lrf2 ? (const void*)k_gateup_mma<uint16_t, false, false, 2, SP> : lrf ? (const void*)k_gateup_mma<uint16_t, false, false, 1, SP>
                                                                               : (const void*)k_gateup_mma<uint16_t, false, false, 0, SP>;
}
template <bool SP>
const void* down_kernel_sp(bool dn_dense, bool d4, int idx_bytes, int tpu) {
  if (dn_dense) return (const void*)k_down_mma<uint16_t, true, false, 2, SP>;
  if (d4) return tpu == 4 ? (const void*)k_down_mma<uint16_t, false, true, 4, SP> : (const void*)k_down_mma<uint16_t, false, true, 2, SP>;
  if (idx_bytes == 1) return tpu == 4 ? (const void*)k_down_mma<uint8_t, false, false, 4, SP> : (const void*)k_down_mma<uint8_t, false, false, 2, SP>;
  return tpu == 4 ? (const void*)k_down_mma<uint16_t, false, false, 4, SP> : (const void*)k_down_mma<uint16_t, false, false, 2, SP>;
}
template <typename IdxT, bool DENSE, bool D4V, bool SP>
const void* fused_kernel_jd(int jd) {
  return jd == 1 ? (const void*)k_expert_fused<IdxT, DENSE, 1, D4V, SP> : jd == 2 ? (const void*)k_expert_fused<IdxT, DENSE, 2, D4V, SP>
       : jd == 3 ? (const void*)k_expert_fused<IdxT, DENSE, 3, D4V, SP> : (const void*)k_expert_fused<IdxT, DENSE, 4, D4V, SP>;
}
template <bool SP>
const void* fused_kernel_sp(bool dn_dense, bool d4, int idx_bytes, int jd) {
  if (d4) return dn_dense ? fused_kernel_jd<uint16_t, true, true, SP>(jd) : fused_kernel_jd<uint16_t, false, true, SP>(jd);
  if (idx_bytes == 1) return dn_dense ? fused_kernel_jd<uint8_t, true, false, SP>(jd) : fused_kernel_jd<uint8_t, false, false, SP>(jd);
  return dn_dense ? fused_kernel_jd<uint16_t, true, false, SP>(jd) : fused_kernel_jd<uint16_t, false, false, SP>(jd);
}
const void* gateup_kernel(const moe_vqlr_handle* h) {
  return h->special ? gateup_kernel_sp<true>(h->gu_dense, h->d4, h->idx_bytes, h->lrf, h->lrf2)
                    : gateup_kernel_sp<false>(h->gu_dense, h->d4, h->idx_bytes, h->lrf, h->lrf2);
}
const void* down_kernel(const moe_vqlr_handle* h, int tpu) {
  return h->special ? down_kernel_sp<true>(h->dn_dense, h->d4, h->idx_bytes, tpu) : down_kernel_sp<false>(h->dn_dense, h->d4, h->idx_bytes, tpu);
}
// Partial tiles the fused kernel keeps per unit: gate and up, or up alone for experts without a gate.
int fused_gu_halves(const moe_vqlr_handle* h) { return (h->special && h->P.act == 2) ? 1 : 2; }
const void* fused_kernel(const moe_vqlr_handle* h, int jd) {
  return h->special ? fused_kernel_sp<true>(h->dn_dense, h->d4, h->idx_bytes, jd) : fused_kernel_sp<false>(h->dn_dense, h->d4, h->idx_bytes, jd);
}

// Head of both chains: for a single token the copy compiled for this layer's shape where there is
// one, else the precompiled kernel.
cudaError_t launch_router(const moe_vqlr_handle* h, const bf16* xb, int T, bool z_by_mma, cudaStream_t st) {
  const Params& P = h->P;
  Params Pa = P;
  const bf16* xa = xb;
  int Ta = T;
  void* args[] = {&Pa, &xa, &Ta};
  if (z_by_mma) {
    return launch_pdl_ptr((const void*)k_router_zmma_pdl, zmma_blocks(P) + (P.E * ((T + kTokGroup - 1) / kTokGroup) + kZmmaWarps - 1) / kZmmaWarps,
                          32 * kZmmaWarps, 0, st, args);
  }
  const void* fn = (T == 1 && h->jit_router) ? h->jit_router : (const void*)k_router_z_pdl;
  return launch_pdl_ptr(fn, (router_z_units_launched(P, T) + kRouterWarps - 1) / kRouterWarps, 32 * kRouterWarps, 0, st, args);
}

// Enqueues the kernel of one stage (nothing for a stage this configuration does not have).
cudaError_t launch_stage(moe_vqlr_handle* h, int stage, const bf16* xb, int T, bf16* ob, cudaStream_t st, bool allow_coop) {
  const Params& P = h->P;
  // more than eight tokens: the basis projections run on the tensor cores, in the router kernel's launch
  const bool z_by_mma = h->fast && T > 8 && P.n_zrows > 0 && P.H % 256 == 0 && P.r % 8 == 0;
  cudaError_t le = cudaSuccess;
  bool ran = false;
  const int n_pos = T * (P.k + P.S);
  if (h->coop && allow_coop && !h->per_expert_launch) {
    if (stage == 0) {
      int zsplit = 1;
      if (!h->dn_dense && P.r > 0) while (n_pos * zsplit * 2 <= 3 * h->sm_count && zsplit * 2 <= 8 && zsplit * 2 <= P.r) zsplit *= 2;
      const size_t smem = coop_layout(P.K, h->n_books, T, P.H, P.I, P.r, h->plan_gu_coop, h->plan_dn_coop, !h->dn_dense, kCoopThreads / 32, P.E, P.k, P.S).total;
      // the index type is the gate/up projections' (a dense down projection has no indices)
      if (h->dn_dense && h->idx_bytes == 1) le = launch_coop(k_layer_coop<uint8_t, true>, h->sm_count, kCoopThreads, smem, st, P, xb, ob, T, h->plan_gu_coop, h->plan_dn_coop, h->n_books, h->want_dbg, h->dn_restage, zsplit);
      else if (h->dn_dense) le = launch_coop(k_layer_coop<uint16_t, true>, h->sm_count, kCoopThreads, smem, st, P, xb, ob, T, h->plan_gu_coop, h->plan_dn_coop, h->n_books, h->want_dbg, h->dn_restage, zsplit);
      else if (h->idx_bytes == 1) le = launch_coop(k_layer_coop<uint8_t, false>, h->sm_count, kCoopThreads, smem, st, P, xb, ob, T, h->plan_gu_coop, h->plan_dn_coop, h->n_books, h->want_dbg, h->dn_restage, zsplit);
      else le = launch_coop(k_layer_coop<uint16_t, false>, h->sm_count, kCoopThreads, smem, st, P, xb, ob, T, h->plan_gu_coop, h->plan_dn_coop, h->n_books, h->want_dbg, h->dn_restage, zsplit);
      ran = true;
    }
  } else if (h->fused && !h->per_expert_launch && T <= h->fused_max_T && (h->fused_forced || T * (P.k + P.S) * h->fplan.n_sl <= h->sm_count)) {
    // one wave of (work group, slice) items at most: with more, the chain's finer parts balance better
    switch (stage) {
      case 0:
        le = launch_router(h, xb, T, z_by_mma, st);
        ran = true;
        break;
      case 2: {
        FusedPlan fpl = h->fplan;
        fpl.depth_g = h->fused_dg[T];
        fpl.depth_d = h->fused_dd[T];
        fpl.warps = h->fused_w[T];
        StagePlan pgl = h->plan_gu_fused;
        pgl.x_smem = h->fused_xs[T];
        const size_t smem2 = fused_layout(P.K, h->n_books, T, P.H, P.r, pgl, fpl, h->dn_dense, h->idx_tc, P.E, P.k, P.S, fused_gu_halves(h)).total;
        {
          Params Pa = P;
          const bf16* xa = xb;
          int Ta = T, nb_a = h->n_books, dbg_a = h->want_dbg;
          const void* idp = h->dn_dense ? nullptr : h->idx_dp;
          void* args[] = {&Pa, &xa, &Ta, &pgl, &fpl, &nb_a, &dbg_a, &idp};
          const void* fn = (h->jit_fused && T == 1 && !h->want_dbg) ? h->jit_fused : fused_kernel(h, fpl.jd);
          le = launch_pdl_ptr(fn, h->sm_count, 32 * fpl.warps, smem2, st, args);
        }
        ran = true;
        break;
      }
      case 5: {
        const int lr = (!h->dn_dense && P.r > 0) ? 1 : 0;
        size_t smem = ((lr ? (size_t)(P.k + P.S) * P.r : 0) + (size_t)(P.k + P.S) * kCfCols * 2) * sizeof(float);
        if (smem < kCfAloneBytes && T == 1) smem = kCfAloneBytes;      // one block per SM (see kCfAloneBytes)
        if (h->jit_combine && T == 1) {
          Params Pa = P;
          bf16* oa = ob;
          int Ta = T, nsl_a = h->fplan.n_sl, lr_a = lr;
          void* args[] = {&Pa, &oa, &Ta, &nsl_a, &lr_a};
          le = launch_pdl_ptr(h->jit_combine, T * (P.H / 2 / kCfCols), kCfThreads, smem, st, args);
        } else
          le = launch_pdl(k_combine_fused, T * (P.H / 2 / kCfCols), kCfThreads, smem, st, P, ob, T, h->fplan.n_sl, lr);
        ran = true;
        break;
      }
      default: break;
    }
  } else if (h->fast) {
    switch (stage) {
      case 0:
        le = launch_router(h, xb, T, z_by_mma, st);
        ran = true;
        break;
      case 2: {
        const size_t smem = gu_layout(P.K, h->n_books, T, P.H, P.r, h->plan_gu, (h->gu_dense ? kDenseThreads : kFastThreads) / 32, P.E, P.k, P.S).total;
        if (h->pcb && T >= h->pcb_min_T && !h->per_expert_launch) {
          // projection code book: routing + low-rank term, then the table kernel
          StagePlan pl = h->plan_gu;
          pl.x_smem = 0; pl.repl = 0;
          le = launch_pdl(k_gateup_lr, h->sm_count, kFastThreads, h->smem_lr, st, P, xb, T, pl, h->want_dbg);
          if (le == cudaSuccess) {
            int bpc = h->sm_count / (T * h->pcb_Q);
            if (bpc < 1) bpc = 1;
            le = launch_pdl(k_gateup_pcb, T * h->pcb_Q * bpc, kPcbThreads, pcb_smem_bytes(P.K), st, P, xb, T, h->pcb_Q, bpc,
                            h->plan_gu.n_lr > 0 ? 1 : 0);
            h->launches += 1;
          }
          ran = true;
          break;
        }
        // one launch over all work groups, or (ablation) one launch per possible work group:
        // a launch whose group does not exist finds no units after the routing and ends
        const int n_launch = h->per_expert_launch ? n_pos : 1;
        for (int gi = 0; gi < n_launch && le == cudaSuccess; ++gi) {
          StagePlan pl = h->plan_gu;
          if (h->per_expert_launch) pl.only_grp = gi;
          Params Pa = P;
          const bf16* xa = xb;
          int Ta = T, nb_a = h->n_books, dbg_a = h->want_dbg;
          void* args[] = {&Pa, &xa, &Ta, &pl, &nb_a, &dbg_a};
          const void* fn = (h->jit_c_gateup && !h->per_expert_launch) ? h->jit_c_gateup : gateup_kernel(h);
          le = launch_pdl_ptr(fn, h->sm_count, h->gu_dense ? kDenseThreads : kFastThreads, smem, st, args);
        }
        h->launches += n_launch - 1;
        ran = true;
        break;
      }
      case 3: {
        const int with_zd = (!h->dn_dense && P.r > 0) ? 1 : 0;
        const int gu_parts = (h->pcb && T >= h->pcb_min_T && !h->per_expert_launch) ? h->pcb_Q + (h->plan_gu.n_lr > 0 ? 1 : 0)
                                                                                     : h->plan_gu.n_parts;
        if (P.I <= 4096) {                                // one fused block per pair (times zsplit)
          int zsplit = 1;
          if (with_zd) while (n_pos * zsplit * 2 <= 3 * h->sm_count && zsplit * 2 <= 8 && zsplit * 2 <= P.r) zsplit *= 2;
          Params Pa = P;
          int np_a = n_pos, parts_a = gu_parts, zd_a = with_zd, zs_a = zsplit;
          void* args[] = {&Pa, &np_a, &parts_a, &zd_a, &zs_a};
          le = launch_pdl_ptr((const void*)k_act_zdown, n_pos * zsplit, kActThreads, (size_t)P.I * sizeof(float), st, args);
        } else {                                          // few pairs or a long intermediate: two wide kernels
          int grid = (n_pos * (P.I / 2) + 255) / 256;
          if (grid > 4 * h->sm_count) grid = 4 * h->sm_count;
          le = launch_pdl(k_act, grid, 256, 0, st, P, n_pos, gu_parts);
          if (le == cudaSuccess && with_zd) {
            int wpd = 1;                                  // warps per z_d value: 2048 values of I each, at most 8
            while (wpd < 8 && P.I > 2048 * wpd) wpd *= 2;
            if (n_pos * (P.r / 4) * wpd >= 32 * h->sm_count)       // enough warps left with four ranks per unit
              le = launch_pdl(k_zdown4_pdl, (n_pos * (P.r / 4) * wpd + 7) / 8, 256, 0, st, P, n_pos, wpd);
            else
              le = launch_pdl(k_zdown_pdl, (n_pos * P.r * wpd + 7) / 8, 256, 0, st, P, n_pos, wpd);
            h->launches += 1;
          }
        }
        ran = true;
        break;
      }
      case 4: {
        const int n_launch = h->per_expert_launch ? n_pos : 1;
        for (int gi = 0; gi < n_launch && le == cudaSuccess; ++gi) {
          StagePlan pl = h->plan_dn;
          if (h->per_expert_launch) pl.only_grp = gi;
          Params Pa = P;
          int Ta = T;
          void* args[] = {&Pa, &Ta, &pl};
          const void* fn = (h->jit_c_down && !h->per_expert_launch) ? h->jit_c_down : down_kernel(h, pl.tpu);
          le = launch_pdl_ptr(fn, h->sm_count, kDownThreads, h->smem_fast_dn, st, args);
        }
        h->launches += n_launch - 1;
        ran = true;
        break;
      }
      case 5: {
        const int grid = T * ((P.H / 2 + kCombineCols - 1) / kCombineCols);
        Params Pa = P;
        bf16* oa = ob;
        int Ta = T, parts_a = h->plan_dn.n_parts;
        void* args[] = {&Pa, &oa, &Ta, &parts_a};
        le = launch_pdl_ptr(h->jit_c_combine ? h->jit_c_combine : (const void*)k_combine, grid, kCombineCols * kCombineSlots, 0, st, args);
        ran = true;
        break;
      }
      default: break;
    }
  } else {
    switch (stage) {
      case 0:
        k_router_z<<<(P.E + P.n_zrows + 7) / 8, 256, 0, st>>>(P, xb, T);
        ran = true;
        break;
      case 1:
        k_route<<<1, 32 * T, (size_t)T * P.E * 4 + (2 * (size_t)P.E + 1) * 4, st>>>(P, T);
        ran = true;
        break;
      case 2: {
        const size_t smem = h->smem_gateup_fixed + h->smem_gateup_per_token * T;
        if (h->idx_bytes == 1) k_gateup<uint8_t><<<h->sm_count, 512, smem, st>>>(P, xb, T, h->two_books);
        else k_gateup<uint16_t><<<h->sm_count, 512, smem, st>>>(P, xb, T, h->two_books);
        ran = true;
        break;
      }
      case 3:
        if (P.down.kind == MOE_VQLR_PROJ_VQLR && P.r > 0) {
          k_zdown<<<(n_pos * P.r + 7) / 8, 256, 0, st>>>(P, n_pos);
          ran = true;
        }
        break;
      case 4: {
        const int grid = min(h->sm_count, (P.H + 15) / 16);
        if (h->idx_bytes == 1) k_down<uint8_t><<<grid, 512, h->smem_down, st>>>(P, ob, T);
        else k_down<uint16_t><<<grid, 512, h->smem_down, st>>>(P, ob, T);
        ran = true;
        break;
      }
      default: break;
    }
    if (ran) le = cudaGetLastError();
  }
  if (ran) { h->launches += 1; h->stage_ran[stage] = true; }
  return le;
}

// Reads and clears the status word (the stream must have been synchronized).  After a device-side
// timeout the persistent kernel's barrier counters are out of step: they are cleared and the handle
// goes back to the chain of kernels (graphs captured with the persistent kernel are dropped).
int take_status(moe_vqlr_handle* h) {
  const int code = *static_cast<volatile int*>(h->status_host);
  if (code == MOE_VQLR_OK) return MOE_VQLR_OK;
  *h->status_host = 0;
  if (h->coop) {
    cudaMemset(h->P.grid_bar, 0, 2 * sizeof(unsigned int));
    h->coop = false;
    h->P.bar_fault = 0;
    for (auto& g : h->host_graph) if (g) { cudaGraphExecDestroy(g); g = nullptr; }
    for (auto& g : h->io_graph) if (g) { cudaGraphExecDestroy(g); g = nullptr; }
  }
  return fail(h, code, "a kernel of an earlier call on this handle reported: %s",
              code == MOE_VQLR_ERR_TIMEOUT ? "a bounded device-side wait gave up (results of that call are invalid)"
              : code == MOE_VQLR_ERR_INVALID_ARG ? "non-finite router logits" : "error");
}

}  // namespace

extern "C" {

int moe_vqlr_create(const moe_vqlr_config* cfg_in, moe_vqlr_handle** out) {
  if (out) *out = nullptr;
  if (!cfg_in || !out) return fail(nullptr, MOE_VQLR_ERR_INVALID_ARG, "cfg/out is null");
  // Up-only experts have no gate projection: internally it aliases the up projection, so that every
  // pointer stays valid; the tensor-core kernels skip its bytes and its arithmetic.
  moe_vqlr_config cfg_local = *cfg_in;
  if (cfg_local.flags & MOE_VQLR_FLAG_ACT_RELU2_UP_ONLY) cfg_local.gate = cfg_local.up;
  const moe_vqlr_config* cfg = &cfg_local;
  const int H = cfg->hidden, I = cfg->inter, E = cfg->n_experts, k = cfg->top_k, S = cfg->n_shared;
  const int K = cfg->codebook_size, r = cfg->rank, maxT = cfg->max_tokens;
  if (H <= 0 || I <= 0 || E <= 0 || k <= 0 || S < 0 || r < 0 || maxT <= 0)
    return fail(nullptr, MOE_VQLR_ERR_INVALID_ARG, "non-positive size");
  if (k > E) return fail(nullptr, MOE_VQLR_ERR_INVALID_ARG, "top_k %d > n_experts %d", k, E);
  if (!cfg->router_w || !aligned16(cfg->router_w))
    return fail(nullptr, MOE_VQLR_ERR_INVALID_ARG, "router_w null or not 16-byte aligned");
  if (cfg->vq_dim != kD && cfg->vq_dim != 4) return fail(nullptr, MOE_VQLR_ERR_UNSUPPORTED, "vq_dim must be 8 or 4");
  if (H % kD || I % kD) return fail(nullptr, MOE_VQLR_ERR_UNSUPPORTED, "hidden and inter must be multiples of 8");
  if (k > kMaxK) return fail(nullptr, MOE_VQLR_ERR_UNSUPPORTED, "top_k > %d", kMaxK);
  if (maxT > kMaxT) return fail(nullptr, MOE_VQLR_ERR_UNSUPPORTED, "max_tokens > %d", kMaxT);
  const bool any_vq = cfg->gate.kind == MOE_VQLR_PROJ_VQLR || cfg->up.kind == MOE_VQLR_PROJ_VQLR ||
                      cfg->down.kind == MOE_VQLR_PROJ_VQLR;
  if (any_vq && (K <= 0 || K > 65536)) return fail(nullptr, MOE_VQLR_ERR_UNSUPPORTED, "codebook_size out of 1..65536");
  if ((cfg->flags & MOE_VQLR_FLAG_IDX12) && any_vq && (K <= 256 || K > 4096 || cfg->vq_dim != kD || H % 16 || I % 16))
    return fail(nullptr, MOE_VQLR_ERR_UNSUPPORTED, "12-bit indices need 256 < codebook_size <= 4096, vq_dim 8, hidden and inter multiples of 16");
  int rc;
  if ((rc = check_proj(cfg->gate, "gate", r)) || (rc = check_proj(cfg->up, "up", r)) ||
      (rc = check_proj(cfg->down, "down", r)))
    return rc;

  moe_vqlr_handle* h = new (std::nothrow) moe_vqlr_handle();
  if (!h) return fail(nullptr, MOE_VQLR_ERR_OOM, "host allocation failed");
  h->cfg = *cfg;
  h->launches = 0;
  h->want_dbg = 0;
  h->workspace = nullptr;
  h->status_host = nullptr;
  h->profiling = 0;
  h->cap_stream = nullptr;
  for (auto& g : h->host_graph) g = nullptr;
  h->ev_valid = false;
  for (auto& e : h->ev) e = nullptr;
  h->idx_bytes = K <= 256 ? 1 : 2;
  cudaError_t ce = cudaGetDevice(&h->device);
  cudaDeviceProp prop;
  if (ce == cudaSuccess) ce = cudaGetDeviceProperties(&prop, h->device);
  if (ce != cudaSuccess) {
    rc = fail(nullptr, MOE_VQLR_ERR_CUDA, "cudaGetDeviceProperties: %s", cudaGetErrorString(ce));
    delete h;
    return rc;
  }
  h->sm_count = prop.multiProcessorCount;

  Params& P = h->P;
  memset(&P, 0, sizeof P);
  P.H = H; P.I = I; P.E = E; P.k = k; P.S = S; P.K = any_vq ? K : 0; P.r = r;
  P.renorm = cfg->renorm_topk ? 1 : 0;
  P.act = (cfg->flags & MOE_VQLR_FLAG_ACT_RELU2_UP_ONLY) ? 2 : (cfg->flags & MOE_VQLR_FLAG_ACT_GELU_TANH) ? 1 : 0;
  P.d = cfg->vq_dim;
  P.idx12 = (any_vq && (cfg->flags & MOE_VQLR_FLAG_IDX12)) ? 1 : 0;
  P.z_repeat = (cfg->flags & MOE_VQLR_FLAG_ABLATE_Z_PER_EXPERT) ? cfg->top_k + cfg->n_shared : 1;
  h->per_expert_launch = (cfg->flags & MOE_VQLR_FLAG_ABLATE_PER_EXPERT_LAUNCH) != 0;
  P.router_w = static_cast<const bf16*>(cfg->router_w);
  P.router_bias = cfg->router_bias;
  P.gate = make_proj(cfg->gate, I, H);
  P.up = make_proj(cfg->up, I, H);
  P.down = make_proj(cfg->down, H, I);
  // z slots: gate -> 0, up -> 0 when it shares gate's basis, else 1
  int n_slots = 0;
  if (r > 0 && P.gate.kind == MOE_VQLR_PROJ_VQLR) P.gate.zslot = n_slots++;
  if (r > 0 && P.up.kind == MOE_VQLR_PROJ_VQLR) {
    if (P.gate.zslot >= 0 && P.up.basis == P.gate.basis) P.up.zslot = P.gate.zslot;
    else P.up.zslot = n_slots++;
  }
  // k_router_z maps stacked row q to slot q / r; with gate dense and up VQLR the single slot is up's
  P.n_zrows = n_slots * r;
  h->two_books = (P.gate.kind == MOE_VQLR_PROJ_VQLR && P.up.kind == MOE_VQLR_PROJ_VQLR &&
                  P.gate.codebook != P.up.codebook) ? 1 : 0;

  // shared memory budgets
  const bool gu_vq = P.gate.kind == MOE_VQLR_PROJ_VQLR || P.up.kind == MOE_VQLR_PROJ_VQLR;
  h->smem_gateup_fixed = gu_vq ? (size_t)(h->two_books ? 2 : 1) * K * 16 : 0;
  h->smem_gateup_per_token = (size_t)((H / kD + 7) / 8 * 8) * 16;
  h->smem_down = (P.down.kind == MOE_VQLR_PROJ_VQLR ? (size_t)K * 16 : 0) + 16 * kMaxT * sizeof(float);
  const size_t smem_gu_max = h->smem_gateup_fixed + h->smem_gateup_per_token * maxT;
  if (smem_gu_max > (size_t)prop.sharedMemPerBlockOptin || h->smem_down > (size_t)prop.sharedMemPerBlockOptin) {
    rc = fail(nullptr, MOE_VQLR_ERR_UNSUPPORTED, "shared memory need (%zu / %zu bytes) exceeds the device limit %zu",
              smem_gu_max, h->smem_down, (size_t)prop.sharedMemPerBlockOptin);
    delete h;
    return rc;
  }
  if (h->idx_bytes == 1) {
    raise_dyn_smem((const void*)k_gateup<uint8_t>, (size_t)smem_gu_max);
    raise_dyn_smem((const void*)k_down<uint8_t>, (size_t)h->smem_down);
  } else {
    raise_dyn_smem((const void*)k_gateup<uint16_t>, (size_t)smem_gu_max);
    raise_dyn_smem((const void*)k_down<uint16_t>, (size_t)h->smem_down);
  }
  raise_dyn_smem((const void*)k_route, (size_t)maxT * E * 4 + (2 * (size_t)E + 1) * 4);

  // ---- tensor-core chain: eligibility, plans, shared-memory budgets -------------------------
  {
    const bool gu_vq = P.gate.kind == MOE_VQLR_PROJ_VQLR && P.up.kind == MOE_VQLR_PROJ_VQLR;
    const bool gu_dn = P.gate.kind == MOE_VQLR_PROJ_DENSE_BF16 && P.up.kind == MOE_VQLR_PROJ_DENSE_BF16;
    h->gu_dense = gu_dn;
    h->dn_dense = P.down.kind == MOE_VQLR_PROJ_DENSE_BF16;
    bool ok = gu_vq || gu_dn;
    const bool d4 = any_vq && cfg->vq_dim == 4;       // four-value code words: uint8 indices only, an even K
    if (d4 && (K > 256 || (K & 1))) ok = false;
    if (gu_vq && (H % 64 != 0 || (r % 8) != 0)) ok = false;       // whole groups of eight blocks / ranks
    if (!h->dn_dense && (I % 64 != 0 || (r % 8) != 0 || H % 16 != 0)) ok = false;
    if (gu_vq && r > 0 && (P.gate.zslot < 0 || P.up.zslot < 0)) ok = false;
    if (k + S > kMaxK + 8) ok = false;                            // k_combine keeps one partial per slot in shared memory
    h->n_books = gu_vq ? (h->two_books ? 2 : 1) : 0;
    h->plan_gu = plan_stage(I, H, r, gu_dn);
    h->plan_dn = plan_stage(H, I, r, h->dn_dense);
    if (h->plan_gu.n_lr > 0) h->plan_gu.chunk = h->plan_gu.tiles < 16 ? h->plan_gu.tiles : 16;   // mix slice and low-rank parts
    h->plan_dn.n_parts = h->plan_dn.n_slices;          // the down kernel folds the low-rank groups into the slices
    if (!h->dn_dense && H % 16 == 0) {                  // a compressed down unit covers two or four row tiles (four where
      h->plan_dn.tpu = (H % 32 == 0 && h->plan_dn.n_slices * (H / 32) >= 256) ? 4 : 2;   // a group still has many units)
      h->plan_dn.tiles = H / (8 * h->plan_dn.tpu);
    }
    h->plan_dn.chunk = h->plan_dn.tiles;
    {
      const bool want_coop = (cfg->flags & MOE_VQLR_FLAG_PERSISTENT) != 0;      // the persistent kernel walks the groups as parts of their own
      h->lrf = gu_vq && !want_coop && h->plan_gu.n_lr >= h->plan_gu.n_slices;
      h->lrf2 = h->lrf && h->plan_gu.n_lr > h->plan_gu.n_slices;
    }
    if (h->lrf) h->plan_gu.n_parts = h->plan_gu.n_slices;   // ... and so does gate/up where every slice gets a group
    // shared-memory plan: replicate a small code book eight times (conflict-free lookups), stage the
    // tokens when they fit, then take the deepest rings that still fit
    const size_t limit = (size_t)prop.sharedMemPerBlockOptin;
    const int gu_warps = (gu_dn ? kDenseThreads : kFastThreads) / 32;
    h->plan_gu.repl = (gu_vq && (size_t)K * 128 * h->n_books <= 72 * 1024) ? 1 : 0;
    h->plan_dn.repl = (!h->dn_dense && (size_t)K * 128 <= 72 * 1024) ? 1 : 0;
    if (d4 && ((gu_vq && !h->plan_gu.repl) || (!h->dn_dense && !h->plan_dn.repl))) ok = false;
    h->plan_gu.x_smem = 1;
    h->plan_gu.depth = 2;
    if (gu_layout(K, h->n_books, maxT, H, r, h->plan_gu, gu_warps, E, k, S).total > limit) h->plan_gu.x_smem = 0;
    for (int d = kMaxDepth; d >= 2; --d) {
      h->plan_gu.depth = d;
      if (gu_layout(K, h->n_books, maxT, H, r, h->plan_gu, gu_warps, E, k, S).total <= limit) break;
    }
    for (int d = kMaxDepth; d >= 2; --d) {
      h->plan_dn.depth = d;
      if (dn_layout(K, !h->dn_dense, h->plan_dn, kDownThreads / 32, maxT * (k + S)).total <= limit) break;
    }
    finish_plan(h->plan_gu, h->sm_count * gu_warps);
    finish_plan(h->plan_dn, h->sm_count * (kDownThreads / 32));
    const size_t smem_gu = gu_layout(K, h->n_books, maxT, H, r, h->plan_gu, gu_warps, E, k, S).total;
    h->smem_fast_dn = dn_layout(K, !h->dn_dense, h->plan_dn, kDownThreads / 32, maxT * (k + S)).total;
    if (smem_gu > limit || h->smem_fast_dn > limit || (size_t)I * sizeof(float) > limit) ok = false;
    if (cfg->flags & MOE_VQLR_FLAG_GENERIC_KERNELS) ok = false;
    h->fast = ok;
    h->d4 = ok && d4;
    h->idx_tc = h->d4 ? 2 : h->idx_bytes;
    if (ok) {
      cudaError_t e1 = cudaSuccess, e2 = cudaSuccess;
      h->special = (P.act == 2 || P.idx12) && !gu_dn;
      e1 = raise_dyn_smem(gateup_kernel(h), smem_gu);
      e2 = raise_dyn_smem(down_kernel(h, h->plan_dn.tpu), h->smem_fast_dn);
      cudaError_t e3 = raise_dyn_smem((const void*)k_act_zdown, (size_t)((size_t)I * sizeof(float)));
      if (e1 != cudaSuccess || e2 != cudaSuccess || e3 != cudaSuccess) { cudaGetLastError(); h->fast = false; }
    }
  }

  // ---- gate/up through the projection code book (several tokens, small code book) ---------------
  h->pcb = false;
  h->pcb_min_T = 0;
  h->pcb_Q = 0;
  h->smem_lr = 0;
  {
    const bool want_pcb = (cfg->flags & MOE_VQLR_FLAG_PROJECTION_CODE_BOOK) != 0;   // off by default (measured slower than the tensor-core kernels at every batch size)
    const bool gu_vq2 = P.gate.kind == MOE_VQLR_PROJ_VQLR && P.up.kind == MOE_VQLR_PROJ_VQLR;
    const size_t limit = (size_t)prop.sharedMemPerBlockOptin;
    if (h->fast && gu_vq2 && !h->d4 && cfg->vq_dim == kD && h->idx_bytes == 1 && H % 16 == 0 && I % kPcbRows == 0 &&
        pcb_smem_bytes(K) <= limit && want_pcb) {
      StagePlan pl = h->plan_gu;
      pl.x_smem = 0; pl.repl = 0;
      h->smem_lr = gu_layout(K, 0, maxT, H, r, pl, kFastThreads / 32, E, k, S).total;
      if (h->smem_lr <= limit &&
          raise_dyn_smem((const void*)k_gateup_lr, (size_t)h->smem_lr) == cudaSuccess &&
          raise_dyn_smem((const void*)k_gateup_pcb, (size_t)pcb_smem_bytes(K)) == cudaSuccess) {
        h->pcb = true;
        h->pcb_Q = (H / 8 + kPcbPiece - 1) / kPcbPiece;
        h->pcb_min_T = 1;
      } else {
        cudaGetLastError();
      }
    }
  }

  // ---- the same chain as one persistent cooperative kernel --------------------------------------
  h->coop = false;
  h->dn_restage = 0;
  h->smem_coop = 0;
  {
    int coop_attr = 0;
    cudaDeviceGetAttribute(&coop_attr, cudaDevAttrCooperativeLaunch, h->device);
    const bool want_coop = (cfg->flags & MOE_VQLR_FLAG_PERSISTENT) != 0;
    if (h->fast && !h->d4 && !h->lrf && !h->gu_dense && !P.idx12 && coop_attr && want_coop) {
      const size_t limit = (size_t)prop.sharedMemPerBlockOptin;
      const int warps = kCoopThreads / 32;
      h->plan_gu_coop = h->plan_gu;
      h->plan_dn_coop = h->plan_dn;
      if (!h->dn_dense) {                               // the persistent kernel's down walk is built for two tiles per unit
        h->plan_dn_coop.tpu = 2;
        h->plan_dn_coop.tiles = H / 16;
        h->plan_dn_coop.chunk = h->plan_dn_coop.tiles;
      }
      bool fits = false;
      for (int xs = 1; xs >= 0 && !fits; --xs)
        for (int d = kMaxDepth; d >= 2 && !fits; --d) {
          h->plan_gu_coop.x_smem = xs;
          h->plan_gu_coop.depth = d;
          h->plan_dn_coop.depth = h->dn_dense ? (d > 3 ? 3 : d) : d;
          h->smem_coop = coop_layout(K, h->n_books, maxT, H, I, r, h->plan_gu_coop, h->plan_dn_coop, !h->dn_dense, warps, E, k, S).total;
          fits = h->smem_coop <= limit;
        }
      finish_plan(h->plan_gu_coop, h->sm_count * warps);
      finish_plan(h->plan_dn_coop, h->sm_count * warps);
      if (fits) {
        h->dn_restage = (!h->dn_dense && (P.down.codebook != P.gate.codebook || h->plan_dn_coop.repl != h->plan_gu_coop.repl)) ? 1 : 0;
        const void* fn = h->dn_dense ? (h->idx_bytes == 1 ? (const void*)k_layer_coop<uint8_t, true> : (const void*)k_layer_coop<uint16_t, true>)
                         : h->idx_bytes == 1 ? (const void*)k_layer_coop<uint8_t, false> : (const void*)k_layer_coop<uint16_t, false>;
        int per_sm = 0;
        cudaError_t e1 = raise_dyn_smem((const void*)fn, (size_t)h->smem_coop);
        if (e1 == cudaSuccess) e1 = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, kCoopThreads, h->smem_coop);
        if (e1 == cudaSuccess && per_sm >= 1) h->coop = true; else cudaGetLastError();
      }
    }
  }

  // ---- one kernel per (work group, slice of I) between router and weighted sum ------------------
  h->fused = false;
  h->fused_forced = false;
  h->fused_max_T = 0;
  h->idx_dp = nullptr;
  size_t idx_dp_bytes = 0;
  {
    const bool no_fused = (cfg->flags & MOE_VQLR_FLAG_NO_FUSED) != 0, force_fused = (cfg->flags & MOE_VQLR_FLAG_FORCE_FUSED) != 0;
    const bool book_ok = h->dn_dense || P.down.codebook == P.gate.codebook || (h->n_books == 2 && P.down.codebook == P.up.codebook);
    if (h->fast && !h->gu_dense && book_ok && H % 16 == 0 && !no_fused) {
      const size_t limit = (size_t)prop.sharedMemPerBlockOptin;
      const int tiles = I / 8;
      int target = h->sm_count / (k + S);            // slices per expert that fill the GPU at one token
      if (target < 1) target = 1;
      FusedPlan fp;
      memset(&fp, 0, sizeof fp);
      StagePlan pg = h->plan_gu;
      pg.x_smem = 1;
      if (h->lrf) {                                  // the fused kernel walks the low-rank groups as parts of their own
        pg.n_parts = pg.n_slices + pg.n_lr;
        finish_plan(pg, pg.W);
      }
      bool found = false;
      for (int tps = (tiles + target - 1) / target; tps >= 1 && !found; --tps) {
        if (tps > 4 * kFusedMaxJd) tps = 4 * kFusedMaxJd;
        fp.tps = tps;
        fp.n_sl = (tiles + tps - 1) / tps;
        fp.t_last = tiles - (fp.n_sl - 1) * tps;
        fp.jd = (tps + 3) / 4;
        fp.rp_log2 = 3;
        while ((1 << fp.rp_log2) < 8 * tps) ++fp.rp_log2;
        // compressed down projection: every index byte of a warp's down tiles is resident (one slot per
        // tile); dense: a ring as deep as fits, its bytes in flight are what hides the DRAM latency
        fp.warps = 12;      // the slice plan is chosen for the smaller block; 16 warps are taken per token count below
        const int dn_tiles_per_warp = (H / 8 + fp.warps - 1) / fp.warps;
        for (int dd = h->dn_dense ? 8 : dn_tiles_per_warp; dd >= (h->dn_dense ? 2 : dn_tiles_per_warp) && !found; --dd)
          for (int dg = 3; dg >= 2 && !found; --dg) {
            fp.depth_g = dg;
            fp.depth_d = dd;
            found = fused_layout(K, h->n_books, 1, H, r, pg, fp, h->dn_dense, h->idx_tc, E, k, S, fused_gu_halves(h)).total <= limit;
          }
      }
      // many thin slices would turn the partial y into the dominant traffic: leave those shapes to the chain
      const bool forced = force_fused;
      h->fused_forced = forced;      // tests: also where the items would not fill the GPU
      if (found && fp.n_sl <= 32 && (forced || (k + S) * fp.n_sl * 2 >= h->sm_count)) {
        fp.d_nsl = make_fastdiv((unsigned int)fp.n_sl);
        fp.d_tps = make_fastdiv((unsigned int)fp.tps);
        fp.d_tlast = make_fastdiv((unsigned int)fp.t_last);
        int maxT_fit = 0;
        size_t smem_max = 0;
        memset(h->fused_dg, 0, sizeof h->fused_dg);
        memset(h->fused_dd, 0, sizeof h->fused_dd);
        memset(h->fused_xs, 0, sizeof h->fused_xs);
        memset(h->fused_w, 0, sizeof h->fused_w);
        for (int t = 1; t <= maxT; ++t) {          // staged tokens, the widest block and the deepest rings that fit beside them
          bool fit = false;
          for (int W = 16; W >= 12 && !fit; W -= 4) {
            fp.warps = W;
            const int dn_tiles_per_warp = (H / 8 + W - 1) / W;
            for (int xsm = 1; xsm >= 0 && !fit; --xsm)
              for (int dd = h->dn_dense ? 8 : dn_tiles_per_warp; dd >= (h->dn_dense ? 3 : dn_tiles_per_warp) && !fit; --dd)
                for (int dg = 3; dg >= 2 && !fit; --dg) {
                  StagePlan pgt = pg;
                  pgt.x_smem = xsm;
                  fp.depth_g = dg;
                  fp.depth_d = dd;
                  const size_t need = fused_layout(K, h->n_books, t, H, r, pgt, fp, h->dn_dense, h->idx_tc, E, k, S, fused_gu_halves(h)).total;
                  if (need <= limit) {
                    fit = true;
                    h->fused_dg[t] = (signed char)dg;
                    h->fused_dd[t] = (signed char)dd;
                    h->fused_xs[t] = (signed char)xsm;
                    h->fused_w[t] = (signed char)W;
                    if (need > smem_max) smem_max = need;
                  }
                }
          }
          if (!fit) break;                         // more tokens need more room
          maxT_fit = t;
        }
        const void* fn = fused_kernel(h, fp.jd);
        cudaError_t e1 = raise_dyn_smem((const void*)fn, (size_t)smem_max);
        size_t cf_smem = ((size_t)(k + S) * (r > 0 ? r : 0) + (size_t)(k + S) * kCfCols * 2) * sizeof(float);
        if (cf_smem < kCfAloneBytes) cf_smem = kCfAloneBytes;
        if (e1 == cudaSuccess && cf_smem > 48 * 1024)
          e1 = cf_smem <= limit ? raise_dyn_smem((const void*)k_combine_fused, (size_t)cf_smem) : cudaErrorInvalidValue;
        if (e1 == cudaSuccess && maxT_fit >= 1) {
          h->fused = true;
          h->fused_max_T = maxT_fit;
          h->fplan = fp;
          h->plan_gu_fused = pg;
          if (!h->dn_dense) idx_dp_bytes = (size_t)(E + S) * fp.n_sl * (H / 8) * 32 * fp.jd * h->idx_tc;
        } else {
          cudaGetLastError();
        }
      }
    }
  }

  // The single-token path and the chain of kernels compiled for this layer's shape (see jit_host.cuh).
  const bool want_clk = (cfg->flags & MOE_VQLR_FLAG_PHASE_CLOCKS) != 0;
  h->jit_fused = h->jit_router = h->jit_combine = nullptr;
  h->jit_c_gateup = h->jit_c_down = h->jit_c_combine = nullptr;
  std::vector<std::string> base_defs;        // the integers of the parameter block
  {
    auto def = [&](const char* name, long long v) { base_defs.push_back(std::string("-D") + name + "=" + std::to_string(v)); };
    def("J_H", H); def("J_I", I); def("J_E", E); def("J_TOPK", k); def("J_S", S); def("J_K", K); def("J_R", r);
    def("J_RENORM", P.renorm); def("J_ACT", P.act); def("J_D", P.d); def("J_IDX12", P.idx12); def("J_ZREPEAT", P.z_repeat);
    def("J_NZROWS", P.n_zrows); def("J_ZSLOT_G", P.gate.zslot); def("J_ZSLOT_U", P.up.zslot);
    def("J_NBOOKS", h->n_books);
    def("J_LR", (!h->dn_dense && r > 0) ? 1 : 0);
    base_defs.push_back(std::string("-DJ_SP=") + (h->special ? "true" : "false"));
    def("J_SZ_PARAMS", (long long)sizeof(Params)); def("J_SZ_PLAN", (long long)sizeof(StagePlan)); def("J_SZ_FPLAN", (long long)sizeof(FusedPlan));
  }
  bool want_single = false;
  if (cfg->flags & MOE_VQLR_FLAG_NO_SPECIALIZE) h->jit_note = "switched off by MOE_VQLR_FLAG_NO_SPECIALIZE";
  else if (!h->fused || h->fused_dg[1] == 0) h->jit_note = "single-token calls of this configuration do not run the fused kernel";
  else if ((k + S) * h->fplan.n_sl > h->sm_count) h->jit_note = "a single token's work items exceed one wave";
#ifndef MOE_VQLR_TRACE
  else if (want_clk) h->jit_note = "phase clocks are recorded by the generic kernels";
#endif
  else want_single = true;
  if (want_single) {
    const FusedPlan& fp = h->fplan;
    const StagePlan& pg = h->plan_gu_fused;
    std::vector<std::string> defs = base_defs;
    auto def = [&](const char* name, long long v) { defs.push_back(std::string("-D") + name + "=" + std::to_string(v)); };
    def("J_NB", pg.nb); def("J_NSLICES", pg.n_slices); def("J_NLR", pg.n_lr); def("J_NPARTS", pg.n_parts);
    def("J_REPL", pg.repl); def("J_XSMEM", h->fused_xs[1]);
    def("J_TPS", fp.tps); def("J_NSL", fp.n_sl); def("J_TLAST", fp.t_last); def("J_JD", fp.jd); def("J_RP_LOG2", fp.rp_log2);
    def("J_DEPTH_G", h->fused_dg[1]); def("J_DEPTH_D", h->fused_dd[1]); def("J_WARPS", h->fused_w[1]);
    defs.push_back(std::string("-DJ_IDXT=") + ((h->d4 || h->idx_bytes == 2) ? "uint16_t" : "uint8_t"));
    defs.push_back(std::string("-DJ_DENSE=") + (h->dn_dense ? "true" : "false"));
    defs.push_back(std::string("-DJ_D4=") + (h->d4 ? "true" : "false"));
    cudaLibrary_t lib = jit_library(kJitSource, defs, &h->jit_note);
    if (lib) {
      cudaKernel_t kern = nullptr;
      FusedPlan fp1 = fp;
      fp1.depth_g = h->fused_dg[1];
      fp1.depth_d = h->fused_dd[1];
      fp1.warps = h->fused_w[1];
      StagePlan pg1 = pg;
      pg1.x_smem = h->fused_xs[1];
      const size_t smem1 = fused_layout(K, h->n_books, 1, H, r, pg1, fp1, h->dn_dense, h->idx_tc, E, k, S, fused_gu_halves(h)).total;
      cudaKernel_t kern_r = nullptr, kern_c = nullptr;
      size_t cf_smem = ((size_t)(k + S) * (r > 0 ? r : 0) + (size_t)(k + S) * kCfCols * 2) * sizeof(float);
      if (cf_smem < kCfAloneBytes) cf_smem = kCfAloneBytes;
      cudaError_t je = cudaLibraryGetKernel(&kern, lib, "k_expert_fused_jit");
      if (je == cudaSuccess) je = cudaLibraryGetKernel(&kern_r, lib, "k_router_z_jit");
      if (je == cudaSuccess) je = cudaLibraryGetKernel(&kern_c, lib, "k_combine_fused_jit");
      if (je == cudaSuccess) je = raise_dyn_smem((const void*)kern, smem1);
      if (je == cudaSuccess) je = raise_dyn_smem((const void*)kern_c, cf_smem);
      if (je == cudaSuccess) {
        h->jit_fused = (const void*)kern;
        h->jit_router = (const void*)kern_r;
        h->jit_combine = (const void*)kern_c;
        h->jit_note.clear();
      } else {
        h->jit_note = std::string("loading the compiled kernels: ") + cudaGetErrorString(je);
        cudaGetLastError();
      }
    }
  }
  // The chain, for the calls that run it: several tokens, or every call where the fused kernel is not used.
  const bool chain_runs = h->fast && (maxT > 1 || !h->jit_fused);
#ifdef MOE_VQLR_TRACE      // a tracing build compiles the phase stamps into the per-shape copies as well
  const bool clk_ok = true;
#else
  const bool clk_ok = !want_clk;
#endif
  if (chain_runs && !(cfg->flags & MOE_VQLR_FLAG_NO_SPECIALIZE) && !h->per_expert_launch && !h->pcb && clk_ok) {
    std::vector<std::string> defs = base_defs;
    auto def = [&](const std::string& name, long long v) { defs.push_back("-D" + name + "=" + std::to_string(v)); };
    auto def_plan = [&](const std::string& x, const StagePlan& pl) {
      def("J_" + x + "_NB", pl.nb); def("J_" + x + "_NSLICES", pl.n_slices); def("J_" + x + "_NLR", pl.n_lr);
      def("J_" + x + "_NPARTS", pl.n_parts); def("J_" + x + "_TILES", pl.tiles); def("J_" + x + "_DEPTH", pl.depth);
      def("J_" + x + "_CHUNK", pl.chunk); def("J_" + x + "_XSMEM", pl.x_smem); def("J_" + x + "_REPL", pl.repl);
      def("J_" + x + "_W", pl.W); def("J_" + x + "_TPU", pl.tpu); def("J_" + x + "_TAIL", pl.tail);
    };
    def_plan("GU", h->plan_gu);
    def_plan("DN", h->plan_dn);
    const bool gu_d4 = !h->gu_dense && h->d4, dn_d4 = !h->dn_dense && h->d4;
    defs.push_back(std::string("-DJ_GU_IDXT=") + ((h->gu_dense || h->d4 || h->idx_bytes == 2) ? "uint16_t" : "uint8_t"));
    defs.push_back(std::string("-DJ_DN_IDXT=") + ((h->dn_dense || h->d4 || h->idx_bytes == 2) ? "uint16_t" : "uint8_t"));
    defs.push_back(std::string("-DJ_GU_DENSE=") + (h->gu_dense ? "true" : "false"));
    defs.push_back(std::string("-DJ_DN_DENSE=") + (h->dn_dense ? "true" : "false"));
    defs.push_back(std::string("-DJ_GU_D4=") + (gu_d4 ? "true" : "false"));
    defs.push_back(std::string("-DJ_DN_D4=") + (dn_d4 ? "true" : "false"));
    def("J_LRF", h->gu_dense ? 0 : h->lrf2 ? 2 : h->lrf ? 1 : 0);
    def("J_DN_TPUT", (!h->dn_dense && h->plan_dn.tpu == 4) ? 4 : 2);
    std::string why;
    cudaLibrary_t lib = jit_library(kJitChainSource, defs, &why);
    if (lib) {
      cudaKernel_t kg = nullptr, kd = nullptr, kc = nullptr;
      cudaError_t je = cudaLibraryGetKernel(&kg, lib, "k_gateup_mma_jit");
      if (je == cudaSuccess) je = cudaLibraryGetKernel(&kd, lib, "k_down_mma_jit");
      if (je == cudaSuccess) je = cudaLibraryGetKernel(&kc, lib, "k_combine_jit");
      const int gu_warps2 = (h->gu_dense ? kDenseThreads : kFastThreads) / 32;
      if (je == cudaSuccess) je = raise_dyn_smem((const void*)kg, gu_layout(K, h->n_books, maxT, H, r, h->plan_gu, gu_warps2, E, k, S).total);
      if (je == cudaSuccess) je = raise_dyn_smem((const void*)kd, h->smem_fast_dn);
      if (je == cudaSuccess) {
        h->jit_c_gateup = (const void*)kg; h->jit_c_down = (const void*)kd; h->jit_c_combine = (const void*)kc;
        if (!want_single) h->jit_note.clear();
      } else {
        cudaGetLastError();
        if (h->jit_note.empty()) h->jit_note = std::string("loading the compiled chain: ") + cudaGetErrorString(je);
      }
    } else if (h->jit_note.empty() || !want_single) {
      h->jit_note = "chain: " + why;
    }
  }

  // workspace
  const size_t n_pos = (size_t)maxT * (k + S);
  unsigned int* idx_max = nullptr;      // scratch of the index validation
  auto plan = [&](char* base) {
    char* cur = base;
    P.logits = carve<float>(cur, (size_t)maxT * E);
    P.z = carve<float>(cur, (size_t)maxT * 2 * (r > 0 ? r : 1));
    P.topk_id = carve<int>(cur, (size_t)maxT * k);
    P.topk_w = carve<float>(cur, (size_t)maxT * k);
    P.counts = carve<int>(cur, E);
    P.offsets = carve<int>(cur, E + 1);
    P.pair_token = carve<int>(cur, n_pos);
    P.pair_slot = carve<int>(cur, n_pos);
    P.pair_w = carve<float>(cur, n_pos);
    P.act_n = carve<int>(cur, 1);
    P.act_e = carve<int>(cur, E + S);
    P.act_off = carve<int>(cur, E + S);
    P.act_cnt = carve<int>(cur, E + S);
    P.grp_n = carve<int>(cur, 1);
    P.grp_e = carve<int>(cur, n_pos);
    P.grp_off = carve<int>(cur, n_pos);
    P.grp_cnt = carve<int>(cur, n_pos);
    P.p = carve<float>(cur, n_pos * I);
    P.p_hi = carve<bf16>(cur, n_pos * I);
    P.p_lo = carve<bf16>(cur, n_pos * I);
    P.zd = carve<float>(cur, n_pos * (r > 0 ? r : 1));
    size_t gu_parts_max = h->plan_gu.n_parts;
    if (h->pcb && (size_t)h->pcb_Q + 1 > gu_parts_max) gu_parts_max = (size_t)h->pcb_Q + 1;
    P.gpart = carve<float>(cur, h->fast ? gu_parts_max * n_pos * I : 1);
    P.upart = carve<float>(cur, h->fast ? gu_parts_max * n_pos * I : 1);
    {
      int y_parts = h->fast ? h->plan_dn.n_parts : 0;
      if (h->fused && h->fplan.n_sl > y_parts) y_parts = h->fplan.n_sl;
      P.ypart = carve<float>(cur, y_parts > 0 ? (size_t)y_parts * n_pos * H : 1);
    }
    P.zd_part = carve<float>(cur, (h->fused && !h->dn_dense && r > 0) ? n_pos * h->fplan.n_sl * r : 1);
    h->idx_dp = carve<char>(cur, idx_dp_bytes > 0 ? idx_dp_bytes : 1);
    P.inv_pos = carve<int>(cur, n_pos);
    idx_max = carve<unsigned int>(cur, 1);
    P.grid_bar = carve<unsigned int>(cur, 2);
    if (want_clk) { P.clk = carve<long long>(cur, (size_t)4 * h->sm_count * 16 * 16); P.clk_blocks = h->sm_count; }
    h->x_stage = carve<bf16>(cur, (size_t)maxT * H);
    h->out_stage = carve<bf16>(cur, (size_t)maxT * H);
    return (size_t)(cur - base);
  };
  h->workspace_bytes = plan(nullptr);
  ce = cudaMalloc(&h->workspace, h->workspace_bytes);
  if (ce != cudaSuccess) {
    rc = fail(nullptr, MOE_VQLR_ERR_OOM, "cudaMalloc(%zu): %s", h->workspace_bytes, cudaGetErrorString(ce));
    cudaGetLastError();
    delete h;
    return rc;
  }
  plan(static_cast<char*>(h->workspace));
  cudaMemset(h->workspace, 0, h->workspace_bytes);
  // the status word: host memory the device can write, so that reading it costs the host nothing
  ce = cudaHostAlloc(reinterpret_cast<void**>(&h->status_host), sizeof(int), cudaHostAllocMapped);
  if (ce == cudaSuccess) {
    *h->status_host = 0;
    ce = cudaHostGetDevicePointer(reinterpret_cast<void**>(&P.status), h->status_host, 0);
  }
  if (ce != cudaSuccess) {
    rc = fail(nullptr, MOE_VQLR_ERR_OOM, "status word (mapped host memory): %s", cudaGetErrorString(ce));
    cudaGetLastError();
    if (h->status_host) cudaFreeHost(h->status_host);
    cudaFree(h->workspace);
    delete h;
    return rc;
  }
  P.spin_limit = kGridSyncSpinLimit;
  P.bar_fault = 0;
  if ((cfg->flags & MOE_VQLR_FLAG_TEST_BARRIER_TIMEOUT) && h->coop) { P.spin_limit = 2000; P.bar_fault = 1; }
  if (h->fused && !h->dn_dense) {      // one-off: the down index map per slice
    const FusedPlan& fp = h->fplan;
    if (h->idx_tc == 1)
      k_relay_down_idx<uint8_t><<<h->sm_count * 8, 256>>>(static_cast<const uint8_t*>(P.down.idx), static_cast<uint8_t*>(h->idx_dp), E + S, H, I / kD, fp.tps, fp.n_sl, fp.jd, 0);
    else
      k_relay_down_idx<uint16_t><<<h->sm_count * 8, 256>>>(static_cast<const uint16_t*>(P.down.idx), static_cast<uint16_t*>(h->idx_dp), E + S, H, I / kD, fp.tps, fp.n_sl, fp.jd, P.idx12);
    ce = cudaDeviceSynchronize();
    if (ce != cudaSuccess) {
      rc = fail(nullptr, MOE_VQLR_ERR_CUDA, "re-laying the down index map: %s", cudaGetErrorString(ce));
      cudaFreeHost(h->status_host);
      cudaFree(h->workspace);
      delete h;
      return rc;
    }
  }

  if (cfg->flags & MOE_VQLR_FLAG_VALIDATE_INDICES) {
    unsigned int* d_max = idx_max;
    const moe_vqlr_proj* projs[3] = {&cfg->gate, &cfg->up, &cfg->down};
    for (int i = 0; i < 3; ++i) {
      if (projs[i]->kind != MOE_VQLR_PROJ_VQLR) continue;
      const size_t n = (size_t)(E + S) * H * I / cfg->vq_dim;
      if (h->idx_bytes == 1) k_max_index<uint8_t><<<h->sm_count * 4, 256>>>(static_cast<const uint8_t*>(projs[i]->idx), n, d_max, 0);
      else k_max_index<uint16_t><<<h->sm_count * 4, 256>>>(static_cast<const uint16_t*>(projs[i]->idx), n, d_max, P.idx12);
    }
    unsigned int mx = 0;
    ce = cudaMemcpy(&mx, d_max, sizeof mx, cudaMemcpyDeviceToHost);
    if (ce != cudaSuccess || mx >= (unsigned int)K) {
      rc = ce != cudaSuccess ? fail(nullptr, MOE_VQLR_ERR_CUDA, "index validation: %s", cudaGetErrorString(ce))
                             : fail(nullptr, MOE_VQLR_ERR_BAD_INDEX, "index %u >= codebook_size %d", mx, K);
      cudaFreeHost(h->status_host);
      cudaFree(h->workspace);
      delete h;
      return rc;
    }
  }
  ce = cudaDeviceSynchronize();
  if (ce != cudaSuccess) {
    rc = fail(nullptr, MOE_VQLR_ERR_CUDA, "create: %s", cudaGetErrorString(ce));
    cudaFreeHost(h->status_host);
    cudaFree(h->workspace);
    delete h;
    return rc;
  }
  *out = h;
  return MOE_VQLR_OK;
}

int moe_vqlr_decode_layer(moe_vqlr_handle* h, const void* x, int32_t T, void* out,
                          const moe_vqlr_debug* dbg, void* cuda_stream) {
  if (!h) return MOE_VQLR_ERR_INVALID_ARG;
  if (!x || !out) return fail(h, MOE_VQLR_ERR_INVALID_ARG, "x/out is null");
  if (T < 1 || T > h->cfg.max_tokens) return fail(h, MOE_VQLR_ERR_INVALID_ARG, "T=%d outside 1..%d", T, h->cfg.max_tokens);
  if (!aligned16(x) || !aligned16(out)) return fail(h, MOE_VQLR_ERR_INVALID_ARG, "x/out must be 16-byte aligned");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const Params& P = h->P;
  const bf16* xb = static_cast<const bf16*>(x);
  bf16* ob = static_cast<bf16*>(out);

  const bool prof = h->profiling != 0;
  h->want_dbg = (dbg && (dbg->counts || dbg->offsets)) ? 1 : 0;
  for (int i = 0; i < kStages; ++i) h->stage_ran[i] = false;
  for (int stage = 0; stage < kStages; ++stage) {
    if (prof) cudaEventRecord(h->ev[stage], st);
    const cudaError_t le = launch_stage(h, stage, xb, T, ob, st, true);
    if (le != cudaSuccess) return fail(h, MOE_VQLR_ERR_CUDA, "launch of stage %s: %s", kStageNames[stage], cudaGetErrorString(le));
  }
  if (prof) cudaEventRecord(h->ev[kStages], st);
  h->ev_valid = prof;
  cudaError_t ce = cudaGetLastError();
  if (ce != cudaSuccess) return fail(h, MOE_VQLR_ERR_CUDA, "launch: %s", cudaGetErrorString(ce));

  if (dbg) {
    const size_t Tk = (size_t)T * P.k;
    struct { void* dst; const void* src; size_t n; } cp[] = {
        {dbg->logits, P.logits, (size_t)T * P.E * 4}, {dbg->topk_id, P.topk_id, Tk * 4},
        {dbg->topk_w, P.topk_w, Tk * 4},              {dbg->counts, P.counts, (size_t)P.E * 4},
        {dbg->offsets, P.offsets, (size_t)(P.E + 1) * 4},
        {dbg->pair_token, P.pair_token, Tk * 4},      {dbg->pair_slot, P.pair_slot, Tk * 4}};
    for (auto& c : cp)
      if (c.dst) {
        ce = cudaMemcpyAsync(c.dst, c.src, c.n, cudaMemcpyDeviceToDevice, st);
        if (ce != cudaSuccess) return fail(h, MOE_VQLR_ERR_CUDA, "debug copy: %s", cudaGetErrorString(ce));
      }
  }
  return MOE_VQLR_OK;
}

int moe_vqlr_decode_layer_host(moe_vqlr_handle* h, const void* x_host, int32_t T, void* out_host,
                               void* cuda_stream) {
  if (!h) return MOE_VQLR_ERR_INVALID_ARG;
  if (!x_host || !out_host) return fail(h, MOE_VQLR_ERR_INVALID_ARG, "x_host/out_host is null");
  if (T < 1 || T > h->cfg.max_tokens) return fail(h, MOE_VQLR_ERR_INVALID_ARG, "T=%d outside 1..%d", T, h->cfg.max_tokens);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t bytes = (size_t)T * h->P.H * sizeof(bf16);
  // The kernel chain between the two staging buffers never changes for a given T, so it is
  // captured once into a graph and replayed: one launch instead of three to six.
  if (!h->host_graph[T] && !h->profiling) {
    cudaError_t ge = cudaSuccess;
    if (!h->cap_stream) ge = cudaStreamCreateWithFlags(&h->cap_stream, cudaStreamNonBlocking);
    cudaGraph_t graph = nullptr;
    if (ge == cudaSuccess) ge = cudaStreamBeginCapture(h->cap_stream, cudaStreamCaptureModeThreadLocal);
    if (ge == cudaSuccess) {
      const int64_t before = h->launches;
      const int rc = moe_vqlr_decode_layer(h, h->x_stage, T, h->out_stage, nullptr, h->cap_stream);
      h->host_graph_launches = (int)(h->launches - before);
      h->launches = before;
      ge = cudaStreamEndCapture(h->cap_stream, &graph);
      if (rc != MOE_VQLR_OK && ge == cudaSuccess) ge = cudaErrorUnknown;
    }
    if (ge == cudaSuccess) ge = cudaGraphInstantiate(&h->host_graph[T], graph, 0);
    if (graph) cudaGraphDestroy(graph);
    if (ge != cudaSuccess) {
      cudaGetLastError();
      h->host_graph[T] = nullptr;
      return fail(h, MOE_VQLR_ERR_CUDA, "graph capture of the layer: %s", cudaGetErrorString(ge));
    }
  }
  // Callers that reuse their (pinned) host buffers get the two copies inside the graph as well:
  // one launch and one synchronisation per call.
  if (!h->profiling && !h->io_graph_failed) {
    if (h->io_graph[T] && (h->io_x[T] != x_host || h->io_out[T] != out_host)) {
      cudaGraphExecDestroy(h->io_graph[T]);
      h->io_graph[T] = nullptr;
    }
    if (!h->io_graph[T]) {
      cudaPointerAttributes ax, ao;
      const bool pinned = cudaPointerGetAttributes(&ax, x_host) == cudaSuccess && ax.type == cudaMemoryTypeHost &&
                          cudaPointerGetAttributes(&ao, out_host) == cudaSuccess && ao.type == cudaMemoryTypeHost;
      cudaGetLastError();
      cudaGraph_t graph = nullptr;
      cudaError_t ge = pinned ? cudaStreamBeginCapture(h->cap_stream, cudaStreamCaptureModeThreadLocal) : cudaErrorNotSupported;
      if (ge == cudaSuccess) {
        const int64_t before = h->launches;
        // The result goes straight into the caller's pinned buffer where the device can address it (the
        // last kernel's 2 H bytes per token are posted writes over the bus, visible after the stream
        // synchronisation below): one graph node and one hand-off less than a copy out of the staging
        // buffer.  The tokens come in through k_stage_in (every block of the first two kernels reads them, so
        // they are staged on the device once).
        void* out_dev = (ao.devicePointer && aligned16(ao.devicePointer)) ? ao.devicePointer : nullptr;
        const void* x_dev = (ax.devicePointer && aligned16(ax.devicePointer)) ? ax.devicePointer : nullptr;
        cudaError_t c1;
        if (x_dev) c1 = launch_pdl(k_stage_in, (int)((bytes / 16 + 255) / 256), 256, 0, h->cap_stream, static_cast<const uint4*>(x_dev),
                                   reinterpret_cast<uint4*>(h->x_stage), (int)(bytes / 16));
        else c1 = cudaMemcpyAsync(h->x_stage, x_host, bytes, cudaMemcpyHostToDevice, h->cap_stream);
        const int rc = c1 == cudaSuccess ? moe_vqlr_decode_layer(h, h->x_stage, T, out_dev ? out_dev : h->out_stage, nullptr, h->cap_stream)
                                         : MOE_VQLR_ERR_CUDA;
        cudaError_t c2 = out_dev ? cudaSuccess : cudaMemcpyAsync(out_host, h->out_stage, bytes, cudaMemcpyDeviceToHost, h->cap_stream);
        h->launches = before;
        ge = cudaStreamEndCapture(h->cap_stream, &graph);
        if ((rc != MOE_VQLR_OK || c1 != cudaSuccess || c2 != cudaSuccess) && ge == cudaSuccess) ge = cudaErrorUnknown;
      }
      if (ge == cudaSuccess) ge = cudaGraphInstantiate(&h->io_graph[T], graph, 0);
      if (graph) cudaGraphDestroy(graph);
      if (ge != cudaSuccess) {
        cudaGetLastError();
        h->io_graph[T] = nullptr;
        h->io_graph_failed = true;
      } else {
        h->io_x[T] = x_host;
        h->io_out[T] = out_host;
        h->io_stage_in[T] = ax.devicePointer && aligned16(ax.devicePointer);
      }
    }
    if (h->io_graph[T]) {
      cudaError_t ce2 = cudaGraphLaunch(h->io_graph[T], st);
      if (ce2 == cudaSuccess) ce2 = cudaStreamSynchronize(st);
      if (ce2 != cudaSuccess) return fail(h, MOE_VQLR_ERR_CUDA, "graph launch with copies: %s", cudaGetErrorString(ce2));
      h->launches += h->host_graph_launches + (h->io_stage_in[T] ? 1 : 0);
      return take_status(h);
    }
  }
  cudaError_t ce = cudaMemcpyAsync(h->x_stage, x_host, bytes, cudaMemcpyHostToDevice, st);
  if (ce != cudaSuccess) return fail(h, MOE_VQLR_ERR_CUDA, "copy in: %s", cudaGetErrorString(ce));
  if (h->host_graph[T] && !h->profiling) {
    ce = cudaGraphLaunch(h->host_graph[T], st);
    if (ce != cudaSuccess) return fail(h, MOE_VQLR_ERR_CUDA, "graph launch: %s", cudaGetErrorString(ce));
    h->launches += h->host_graph_launches;
  } else {
    const int rc = moe_vqlr_decode_layer(h, h->x_stage, T, h->out_stage, nullptr, cuda_stream);
    if (rc != MOE_VQLR_OK) return rc;
  }
  ce = cudaMemcpyAsync(out_host, h->out_stage, bytes, cudaMemcpyDeviceToHost, st);
  if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
  if (ce != cudaSuccess) return fail(h, MOE_VQLR_ERR_CUDA, "copy out: %s", cudaGetErrorString(ce));
  return take_status(h);
}

int moe_vqlr_set_jit_toolkit(const char* nvrtc_library, const char* cuda_include_dir) {
  std::lock_guard<std::mutex> lock(g_jit_mu);
  g_jit_nvrtc_path = nvrtc_library ? nvrtc_library : "";
  g_jit_include_dir = cuda_include_dir ? cuda_include_dir : "";
  g_nvrtc = NvrtcApi();          // the next create() looks again
  return MOE_VQLR_OK;
}

int moe_vqlr_specialized(const moe_vqlr_handle* h) {
  if (!h) return 0;
  const void* all[] = {h->jit_router, h->jit_fused, h->jit_combine, h->jit_c_gateup, h->jit_c_down, h->jit_c_combine};
  int n = 0;
  for (const void* k : all) n += k ? 1 : 0;
  return n;
}

const char* moe_vqlr_specialization_note(const moe_vqlr_handle* h) { return h ? h->jit_note.c_str() : ""; }

int moe_vqlr_last_status(moe_vqlr_handle* h) {
  if (!h) return MOE_VQLR_ERR_INVALID_ARG;
  return take_status(h);
}

int moe_vqlr_destroy(moe_vqlr_handle* h) {
  if (!h) return MOE_VQLR_OK;
  for (auto& e : h->ev)
    if (e) cudaEventDestroy(e);
  for (auto& g : h->host_graph)
    if (g) cudaGraphExecDestroy(g);
  for (auto& g : h->io_graph)
    if (g) cudaGraphExecDestroy(g);
  if (h->cap_stream) cudaStreamDestroy(h->cap_stream);
  if (h->status_host) cudaFreeHost(h->status_host);
  cudaError_t ce = cudaFree(h->workspace);
  delete h;
  return ce == cudaSuccess ? MOE_VQLR_OK : MOE_VQLR_ERR_CUDA;
}

const char* moe_vqlr_last_error(const moe_vqlr_handle* h) {
  return h ? h->error.c_str() : g_create_error.c_str();
}

int moe_vqlr_run_stage(moe_vqlr_handle* h, int32_t stage, const void* x, int32_t T, void* out, void* cuda_stream) {
  if (!h) return MOE_VQLR_ERR_INVALID_ARG;
  if (stage < 0 || stage >= kStages || !x || !out || T < 1 || T > h->cfg.max_tokens)
    return fail(h, MOE_VQLR_ERR_INVALID_ARG, "run_stage: bad stage, pointer or T");
  const cudaError_t le = launch_stage(h, stage, static_cast<const bf16*>(x), T, static_cast<bf16*>(out),
                                      static_cast<cudaStream_t>(cuda_stream), false);
  if (le != cudaSuccess) return fail(h, MOE_VQLR_ERR_CUDA, "launch of stage %s: %s", kStageNames[stage], cudaGetErrorString(le));
  return MOE_VQLR_OK;
}

int moe_vqlr_set_profiling(moe_vqlr_handle* h, int32_t on) {
  if (!h) return MOE_VQLR_ERR_INVALID_ARG;
  if (on && !h->ev[0]) {
    for (auto& e : h->ev) {
      cudaError_t ce = cudaEventCreate(&e);
      if (ce != cudaSuccess) return fail(h, MOE_VQLR_ERR_CUDA, "cudaEventCreate: %s", cudaGetErrorString(ce));
    }
  }
  h->profiling = on ? 1 : 0;
  h->ev_valid = false;
  return MOE_VQLR_OK;
}

int moe_vqlr_stage_count(void) { return kStages; }

const char* moe_vqlr_stage_name(int32_t i) { return (i >= 0 && i < kStages) ? kStageNames[i] : ""; }

int moe_vqlr_last_stage_times(moe_vqlr_handle* h, float* ms_out, int32_t cap) {
  if (!h || !ms_out || cap < kStages) return h ? fail(h, MOE_VQLR_ERR_INVALID_ARG, "ms_out null or cap < %d", kStages) : MOE_VQLR_ERR_INVALID_ARG;
  if (!h->ev_valid) return fail(h, MOE_VQLR_ERR_INVALID_ARG, "no profiled call to report");
  cudaError_t ce = cudaEventSynchronize(h->ev[kStages]);
  if (ce != cudaSuccess) return fail(h, MOE_VQLR_ERR_CUDA, "event sync: %s", cudaGetErrorString(ce));
  for (int i = 0; i < kStages; ++i) {
    ms_out[i] = 0.f;
    if (h->stage_ran[i]) {
      ce = cudaEventElapsedTime(&ms_out[i], h->ev[i], h->ev[i + 1]);
      if (ce != cudaSuccess) return fail(h, MOE_VQLR_ERR_CUDA, "elapsed: %s", cudaGetErrorString(ce));
    }
  }
  return MOE_VQLR_OK;
}

int64_t moe_vqlr_phase_clocks(moe_vqlr_handle* h, int64_t* out, int64_t cap) {
  if (!h || !h->P.clk) return 0;
  const int64_t n = (int64_t)4 * h->P.clk_blocks * 16 * 16;
  if (!out) return n;
  if (cap < n) return -1;
  if (cudaMemcpy(out, h->P.clk, (size_t)n * 8, cudaMemcpyDeviceToHost) != cudaSuccess) return -1;
  return n;
}

int64_t moe_vqlr_launch_count(const moe_vqlr_handle* h) { return h ? h->launches : 0; }

int64_t moe_vqlr_workspace_bytes(const moe_vqlr_handle* h) { return h ? (int64_t)h->workspace_bytes : 0; }

}  // extern "C"
