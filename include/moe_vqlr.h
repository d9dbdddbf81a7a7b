/*
 * moe_vqlr — one routed Mixture-of-Experts decode layer (1..16 tokens) whose expert matrices
 * are stored as a vector-quantised part plus a shared-basis low-rank part, for NVIDIA B200
 * (sm_100a).  Plain C ABI: integers, sizes and raw pointers only.
 *
 * What one call computes (paper: Section 2.1 for the MoE block, Eq. 1 and Section 3.1 for the
 * representation, Section 4 for the order of the work):
 *
 *   logit[t][e] = <router_w[e], x[t]> (+ router_bias[e])
 *   the k experts with the largest logits per token (ties: lower expert id), affinities a =
 *       softmax over the k selected logits (or over all E when renorm_topk == 0)
 *   grouping of the (token, slot) pairs by expert, so each activated expert's payload is read
 *       once per layer whatever the batch size (Section 5.6)
 *   per projection P in {gate, up, down}, per activated expert e (Eq. 1, stored transposed):
 *       W_P,e[o][b*d+j] = codebook_P[ idx_P[e][o][b] ][j] + sum_rho factor_P[e][o][rho]*basis_P[rho][b*d+j]
 *     evaluated without ever forming W: the VQ part by code-word lookups, the low-rank part as
 *     factor_P[e] * z with z = basis_P * input computed once per token and shared by all
 *     experts (Section 3.2, "z = D^T h"); or W_P,e = dense_P[e] for a projection kept in bf16
 *     (Section 3.1 keeps the down projection uncompressed)
 *   p = phi(W_gate,e x) * (W_up,e x);    y = W_down,e p      (phi = SiLU: SwiGLU expert; or GELU;
 *                                                            or, without a gate, p = relu(W_up,e x)^2)
 *   out[t] = sum_s a[t][s] * y[t][s]  +  sum over the always-on shared experts of y (weight 1)
 *
 * Symbols: H hidden size, I expert intermediate size, E routed experts, k experts per token,
 * S shared experts (ids E..E+S-1), d block length, K code-book size, r rank, T tokens.
 * bf16 means the 16-bit brain-float format; all matrices are row-major, densely packed.
 *
 * Threading: a handle may be used by one host thread at a time.  All work of a call is
 * enqueued on the given CUDA stream and is asynchronous unless stated otherwise.
 */
#ifndef MOE_VQLR_H_
#define MOE_VQLR_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct moe_vqlr_handle moe_vqlr_handle; /* opaque, owned by the library */

typedef enum {
  MOE_VQLR_OK = 0,
  MOE_VQLR_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, T out of range, ...       */
  MOE_VQLR_ERR_UNSUPPORTED = 2, /* a shape or option this build has no kernel for            */
  MOE_VQLR_ERR_CUDA = 3,        /* a CUDA runtime call or a launch failed                     */
  MOE_VQLR_ERR_OOM = 4,         /* workspace allocation failed                                */
  MOE_VQLR_ERR_TIMEOUT = 5,     /* a bounded device-side wait gave up                         */
  MOE_VQLR_ERR_BAD_INDEX = 6    /* an index map holds a value >= K (found by validation)      */
} moe_vqlr_status;

typedef enum {
  MOE_VQLR_PROJ_VQLR = 0,      /* code book + indices (+ low-rank term when rank > 0)  (Eq. 1)  */
  MOE_VQLR_PROJ_DENSE_BF16 = 1 /* uncompressed bf16 matrix (Section 3.1, down projection)     */
} moe_vqlr_proj_kind;

/* One projection.  out x in is I x H for gate and up, H x I for down.  All pointers are DEVICE
 * pointers borrowed for the lifetime of the handle; the caller keeps them alive and unchanged.
 * Alignment: every pointer 16-byte aligned.  Pointers of different projections may alias (one
 * code book or one basis shared by gate and up is detected and staged / projected once). */
typedef struct {
  int32_t kind;         /* moe_vqlr_proj_kind                                                  */
  int32_t reserved;
  const void* codebook; /* [K][d] bf16                                     (VQLR)             */
  const void* idx;      /* [E+S][out][in/d], uint8 when K <= 256 else uint16 (or packed to twelve
                           bits, MOE_VQLR_FLAG_IDX12) (VQLR); blocks run along the contraction
                           dimension `in`                                                     */
  const void* basis;    /* [rank][in] bf16 = D^T, shared by all experts   (VQLR, rank > 0)    */
  const void* factor;   /* [E+S][out][rank] bf16 = C_e^T, expert-private  (VQLR, rank > 0)    */
  const void* dense;    /* [E+S][out][in] bf16                            (DENSE_BF16)        */
} moe_vqlr_proj;

enum {
  MOE_VQLR_FLAG_VALIDATE_INDICES = 1u, /* create() scans every index map once and fails with
                                         BAD_INDEX if a value >= K is found (costs one pass
                                         over the index maps; never done on the decode path) */
  MOE_VQLR_FLAG_PERSISTENT = 2u,      /* decode calls run the whole layer as ONE persistent
                                         cooperative kernel whose phases are separated by
                                         grid-wide barriers (every wait bounded: a barrier
                                         that gives up reports MOE_VQLR_ERR_TIMEOUT through
                                         the status word, see moe_vqlr_last_status) instead
                                         of the chain of five
                                         kernels.  Same results; measured slower than the
                                         chain on B200, so off by default.  Ignored where the
                                         configuration cannot use it. */
  MOE_VQLR_FLAG_ACT_GELU_TANH = 4u,   /* the expert activation phi of Section 2.1 (it depends
                                         on the model): p = phi(gate) * up with
                                         phi(g) = 0.5 g (1 + tanh(sqrt(2/pi) (g + 0.044715 g^3)))
                                         (the GELU form of GeGLU experts, e.g. the Gemma shape)
                                         instead of the default phi = SiLU (SwiGLU experts) */
  MOE_VQLR_FLAG_ACT_RELU2_UP_ONLY = 4096u, /* experts WITHOUT a gate projection (Section 5.7: the
                                         Nemotron-shaped layer): p = max(W_up x, 0)^2, y = W_down p.
                                         The `gate` member of the configuration is ignored.  A hidden
                                         or intermediate size that is not a multiple of the block
                                         length is padded by the caller: zero activations in the
                                         padding make its weights irrelevant */
  MOE_VQLR_FLAG_IDX12 = 8192u,          /* the index maps hold TWELVE-bit indices, two to three bytes,
                                         little end first (index 2q: byte 3q and the low half of byte
                                         3q+1; index 2q+1: the high half of byte 3q+1 and byte 3q+2):
                                         the index width between one and two bytes for 256 < K <= 4096
                                         (Appendix "Exact engine-work counts": b_J(K) changes at the
                                         encoding boundaries of K), a quarter fewer index bytes than
                                         uint16.  Needs vq_dim 8 and H, I multiples of 16; maps stay
                                         [E+S][out][in/8] indices, i.e. (in/8)*3/2 bytes per row */
  /* The next two switches turn OFF one mechanism each, to measure what it buys (the attribution
   * of Section 5.4, part A of its table).  Results are unchanged.  They act on the tensor-core
   * paths; the generic kernels and the persistent kernel ignore them. */
  MOE_VQLR_FLAG_ABLATE_Z_PER_EXPERT = 8u, /* the shared projections z = basis * x are computed
                                         once per selected (and shared) expert instead of once
                                         per token: k + S times the dot products, same values */
  MOE_VQLR_FLAG_ABLATE_PER_EXPERT_LAUNCH = 16u, /* gate/up and down run as one kernel launch per
                                         work group (expert) instead of one launch over all
                                         activated experts; implies the chain of kernels */
  /* Path selection, for tests and A/B measurements.  Which kernels a call runs never changes its
   * results beyond the summation order; without these flags create() picks the fastest path the
   * configuration allows. */
  MOE_VQLR_FLAG_NO_FUSED = 64u,          /* never run a call as router -> one fused expert kernel ->
                                         weighted sum (the default for calls whose work items fill
                                         at most one wave of blocks): always the chain of kernels */
  MOE_VQLR_FLAG_FORCE_FUSED = 128u,      /* ... or run every call that fits its shared memory that way */
  MOE_VQLR_FLAG_NO_SPECIALIZE = 16384u,  /* do not compile the single-token kernels for this layer's
                                         shape at create() (see moe_vqlr_specialized): the library's
                                         precompiled kernels run */
  MOE_VQLR_FLAG_GENERIC_KERNELS = 256u,  /* only the generic CUDA-core kernels (one warp per output
                                         row), which otherwise serve the shapes the tensor-core
                                         kernels do not cover */
  MOE_VQLR_FLAG_PROJECTION_CODE_BOOK = 512u, /* calls that run the chain of kernels (all of them with
                                         MOE_VQLR_FLAG_NO_FUSED) evaluate the VQ term of
                                         gate / up through per-token projection code books
                                         T[b][k] = <x_b, codebook[k]> (Section 4.2; needs K <= 256 and
                                         vq_dim 8; measured slower than the reconstructing tensor-core
                                         kernel on B200, hence opt-in) */
  MOE_VQLR_FLAG_PHASE_CLOCKS = 1024u,    /* the tensor-core kernels store clock readings at their phase
                                         boundaries for moe_vqlr_phase_clocks (moe_vqlr_bench.h); only
                                         in a library built with -DMOE_VQLR_TRACE */
  MOE_VQLR_FLAG_TEST_BARRIER_TIMEOUT = 32u /* test switch, only with MOE_VQLR_FLAG_PERSISTENT: the
                                         persistent kernel's grid barrier waits for one arrival
                                         more than will ever come and gives up after 2000 polls
                                         (about a millisecond), so that the report of a bounded
                                         wait that ran out (MOE_VQLR_ERR_TIMEOUT through the status
                                         word) can be exercised without hanging the GPU.  The
                                         call's output is invalid by construction. */
};

typedef struct {
  int32_t hidden;        /* H, multiple of 8                                                   */
  int32_t inter;         /* I, multiple of 8                                                   */
  int32_t n_experts;     /* E >= 1                                                             */
  int32_t top_k;         /* 1 <= k <= E, k <= 32                                               */
  int32_t n_shared;      /* S >= 0                                                             */
  int32_t vq_dim;        /* d: 8, or 4 (Section 5.5's shorter vectors: code words of 4 bf16,
                            two indices per 8 weights; tensor-core chain for K <= 256, K even) */
  int32_t codebook_size; /* K, 1..65536                                                        */
  int32_t rank;          /* r >= 0                                                             */
  int32_t max_tokens;    /* largest T a call may pass, 1..16                                   */
  int32_t renorm_topk;   /* 1: affinities sum to 1 over the selected k;  0: softmax over all E */
  uint32_t flags;        /* MOE_VQLR_FLAG_*                                                    */
  int32_t reserved;
  const void* router_w;     /* [E][H] bf16, device                                             */
  const float* router_bias; /* [E] fp32, device, or NULL                                       */
  moe_vqlr_proj gate, up, down;
} moe_vqlr_config;

/* Optional copies of the routing state, for checking.  Each member is a DEVICE pointer or
 * NULL; non-null members are filled (on the call's stream) after the layer's kernels.
 * Shared experts do not appear: these arrays cover the E routed experts only. */
typedef struct {
  float* logits;       /* [T][E]                                                              */
  int32_t* topk_id;    /* [T][k]  slot s = s-th ranked expert (logit descending, id ascending) */
  float* topk_w;       /* [T][k]  affinities                                                   */
  int32_t* counts;     /* [E]     pairs per expert                                             */
  int32_t* offsets;    /* [E+1]   exclusive prefix sum of counts                               */
  int32_t* pair_token; /* [T*k]   pairs sorted by expert, ascending token within an expert     */
  int32_t* pair_slot;  /* [T*k]                                                                */
} moe_vqlr_debug;

#ifndef __CUDACC_RTC__ /* host entry points (the library's run-time-compiled kernels include this
                          file for the types and constants above) */

/* Validates the configuration, allocates the handle and its device workspace on the CURRENT
 * CUDA device and returns the handle in *out (NULL on failure).  Synchronous.
 * Errors: INVALID_ARG, UNSUPPORTED (vq_dim not 8 or 4, H or I not a multiple of 8, K > 65536, k > 32,
 * max_tokens > 16), OOM, CUDA, BAD_INDEX (only with MOE_VQLR_FLAG_VALIDATE_INDICES).
 * The weights stay where they are (borrowed); the one exception is a copy of the DOWN index map
 * in a slice-major order (same values, at most 1/3 larger), made once here inside the workspace
 * when the configuration can run its single-token calls as router -> one fused expert kernel ->
 * weighted sum (Section 4's fused gate/up -> activation -> down pipeline).  Which kernels a call
 * runs (that path, the chain of five kernels, or the generic chain for shapes the tensor-core
 * kernels do not cover) never changes its results beyond the summation order; the path-selection
 * flags above override the choice.  create() reads no environment variable. */
int moe_vqlr_create(const moe_vqlr_config* cfg, moe_vqlr_handle** out);

/* Runs the layer for T tokens.  x: [T][H] bf16, device.  out: [T][H] bf16, device, written with
 * round-to-nearest-even; must not overlap x.  dbg may be NULL.  cuda_stream is a cudaStream_t
 * (NULL = the legacy default stream).  Returns after enqueueing; a launch failure gives
 * ERR_CUDA.  Calls on one handle must not overlap on the device (they share the workspace). */
int moe_vqlr_decode_layer(moe_vqlr_handle* h, const void* x, int32_t T, void* out,
                          const moe_vqlr_debug* dbg, void* cuda_stream);

/* Same layer with HOST buffers: copies x (T*H bf16, host) to the device, runs the layer, copies
 * out (T*H bf16) back and waits for the stream.  Pinned host memory makes the copies
 * asynchronous up to the final wait; pageable memory works but is slower.  Weights stay on
 * the device.  Synchronous on return.  The first call for each T captures the kernel chain into
 * a CUDA graph owned by the handle (later calls replay it), so that first call is slower and
 * must not itself run inside a stream capture.  With pinned host buffers the transfers are part
 * of the graph too (one launch and one wait per call) for as long as the caller passes the same
 * two pointers; other pointers re-capture it.  Pinned buffers that the device can address (16-byte
 * aligned; cudaHostAlloc / cudaHostRegister memory under unified addressing) are read and written
 * by the kernels themselves: a staging kernel fetches the tokens and the last kernel of the layer
 * stores out_host directly, so out_host is complete only when the call has returned. */
int moe_vqlr_decode_layer_host(moe_vqlr_handle* h, const void* x_host, int32_t T, void* out_host,
                               void* cuda_stream);

/* Shape specialisation.  Where a configuration's single-token calls run as router -> fused expert
 * kernel -> weighted sum, create() compiles that path once more for exactly this layer (NVRTC; the
 * library's own kernel source, found beside the library file, with the layer's sizes, expert count,
 * top-k, rank, code-book size and work plan as compile-time constants: the GPU-side counterpart of
 * the ahead-of-time, per-model mapping of Section 4).  Same arithmetic in the same order, so results
 * are bitwise those of the precompiled kernels; a batch-1 call is shorter because its blocks fetch
 * about half the instructions.  Costs a few seconds at the first create() of a shape (kept per
 * process and device afterwards).  Needs libnvrtc and the CUDA headers (under /usr/local/cuda, or where
 * moe_vqlr_set_jit_toolkit points); where they are missing, or with MOE_VQLR_FLAG_NO_SPECIALIZE, the
 * precompiled kernels run.
 * moe_vqlr_specialized: number of kernels of the handle that were compiled that way (0 if none);
 * moe_vqlr_specialization_note: why not (empty string if they were), valid until destroy. */
int moe_vqlr_specialized(const moe_vqlr_handle* h);
/* Process-wide: where to find NVRTC (path of libnvrtc.so.12) and the CUDA headers (the directory
 * that holds cuda_bf16.h) when they are not under /usr/local/cuda, e.g. the nvidia-cuda-nvrtc and
 * nvidia-cuda-runtime packages of a Python environment.  NULL restores the default search.  Takes
 * effect at the next create() of a shape that has not been compiled yet.  Returns MOE_VQLR_OK. */
int moe_vqlr_set_jit_toolkit(const char* nvrtc_library, const char* cuda_include_dir);
const char* moe_vqlr_specialization_note(const moe_vqlr_handle* h);

/* The status word of the handle: conditions that only the kernels can detect while a call runs.
 * Returns MOE_VQLR_OK, or the code a kernel of an earlier call recorded, and clears the word:
 *   MOE_VQLR_ERR_TIMEOUT      a bounded device-side wait gave up (the grid barrier of the persistent
 *                             kernel, MOE_VQLR_FLAG_PERSISTENT); that call's output is invalid.  The
 *                             handle then leaves the persistent kernel for good and runs the chain
 *                             of kernels, so later calls are correct.
 *   MOE_VQLR_ERR_INVALID_ARG  a token selected an expert whose router logit is NaN or infinite
 *                             (non-finite x or router weights); ids stay in range, out is garbage.
 * The word lives in host memory that the kernels write directly, so reading it copies nothing, but
 * it is only meaningful once the caller has synchronized the stream of the calls in question.
 * moe_vqlr_decode_layer_host, which synchronizes anyway, checks it itself and returns the code.
 * moe_vqlr_last_error() then holds a description. */
int moe_vqlr_last_status(moe_vqlr_handle* h);

/* Frees the workspace and the handle.  The caller must first make sure no call on this handle
 * is still running on the device.  NULL is accepted. */
int moe_vqlr_destroy(moe_vqlr_handle* h);

/* Text of the last error on this handle ("" if none); with NULL, of the last failed create()
 * on this thread.  The string is owned by the library. */
const char* moe_vqlr_last_error(const moe_vqlr_handle* h);

/* Routing step only, for callers that must not allocate device memory (no counterpart in the
 * paper: it exists for processes where a memory pool or the host application owns every
 * allocation, so moe_vqlr_create(), which allocates a workspace, is off limits).  Computes
 *   logit[t][e] = <router_w[e], x[t]> (+ router_bias[e]),  the k best experts per token (ties:
 *   lower id) and their affinities -- the same definition as in moe_vqlr_decode_layer, with a
 *   summation order of its own (logits agree to fp32 rounding, so ids can differ where two
 *   logits are closer than that) --
 * and writes topk_id[T][k] (int32) and topk_w[T][k] (fp32).  Logits must be finite: with fewer
 * than k finite logits for a token the remaining slots repeat low expert ids (in range, unflagged).  All pointers are DEVICE pointers;
 * x [T][H] bf16 and router_w [E][H] bf16 must be 16-byte aligned, H a multiple of 8;
 * router_bias [E] fp32 may be NULL.  Asynchronous on cuda_stream.
 *
 * The only scratch, the [T][E] fp32 logits, lives in a fixed 64 KiB array inside the library's
 * device image (held by every GPU that loads the library until the process exits).  Hence:
 *   - limits: T <= 16, E <= 1024, k <= 32; anything larger returns MOE_VQLR_ERR_UNSUPPORTED and
 *     launches nothing;
 *   - no cudaMalloc / cudaFree / allocating library call is made, ever;
 *   - all calls on one device share the array: calls that overlap on the GPU race, so keep them
 *     on one stream or order them yourself.  Each call rewrites every entry it reads; nothing
 *     carried over from an earlier call is used;
 *   - the first call on each device resolves the array's device address (with that device
 *     current); issue that first call outside any stream capture.
 * Returns MOE_VQLR_OK, ERR_INVALID_ARG, ERR_UNSUPPORTED or ERR_CUDA. */
int moe_vqlr_route_noalloc(const void* x, const void* router_w, const float* router_bias,
                           int32_t T, int32_t E, int32_t H, int32_t k, int32_t renorm_topk,
                           int32_t* topk_id, float* topk_w, void* cuda_stream);

#endif /* !__CUDACC_RTC__ */

#ifdef __cplusplus
}
#endif
#endif /* MOE_VQLR_H_ */
