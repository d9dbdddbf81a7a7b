/*
 * moe_vqlr_bench — measurement aids of the moe_vqlr library (see moe_vqlr.h for the layer itself).
 * None of these has a counterpart in the paper, whose profiles come from the Neuron tools
 * (Section 5.1); they exist so that a benchmark can time single kernels, count launches and read
 * the bound that the shared-memory lookups set.  Same C ABI rules: integers, sizes, raw pointers.
 */
#ifndef MOE_VQLR_BENCH_H_
#define MOE_VQLR_BENCH_H_

#include "moe_vqlr.h"

#ifdef __cplusplus
extern "C" {
#endif

/* With profiling on, every decode call records a CUDA event on the call's
 * stream before and after each stage.  Stages, in order: router_z, route, gateup, zdown, down,
 * combine (moe_vqlr_stage_count() of them, named by moe_vqlr_stage_name()).  The events sit between
 * the kernels, so a profiled call can run slightly slower than an unprofiled one. */
int moe_vqlr_set_profiling(moe_vqlr_handle* h, int32_t on);

/* Waits for the last profiled call on this handle and writes the device time of each stage in
 * milliseconds to ms_out[0..stage_count) (0 for a stage the configuration does not run).
 * cap = capacity of ms_out, at least moe_vqlr_stage_count().  INVALID_ARG when the last call
 * was not profiled. */
int moe_vqlr_last_stage_times(moe_vqlr_handle* h, float* ms_out, int32_t cap);

int moe_vqlr_stage_count(void);
const char* moe_vqlr_stage_name(int32_t i);

/* Enqueues the kernel of ONE stage of the layer
 * on cuda_stream, with the same arguments as moe_vqlr_decode_layer, reading whatever the
 * previous stages of an earlier full call on this handle (same x, same T) left in the
 * workspace.  Lets a benchmark time a single kernel back to back, e.g. inside a captured graph.
 * A stage the configuration does not have enqueues nothing and returns MOE_VQLR_OK.  Stages
 * always run as the separate kernels of the chain, also on a handle created with
 * MOE_VQLR_FLAG_PERSISTENT. */
int moe_vqlr_run_stage(moe_vqlr_handle* h, int32_t stage, const void* x, int32_t T, void* out,
                       void* cuda_stream);

/* Tracing aid.  When the handle was created with MOE_VQLR_FLAG_PHASE_CLOCKS and the library was
 * built with -DMOE_VQLR_TRACE,
 * the tensor-core kernels store SM clock readings at their phase boundaries: [kernel 4][block][warp 16][stamp 16] int64.  With out == NULL
 * returns the number of values; otherwise synchronously copies them to the HOST buffer out
 * (cap = its capacity in values) and returns the count, -1 on error, 0 when tracing is off. */
int64_t moe_vqlr_phase_clocks(moe_vqlr_handle* h, int64_t* out, int64_t cap);

/* Number of kernel launches this handle has enqueued since create(). */
int64_t moe_vqlr_launch_count(const moe_vqlr_handle* h);

/* Device workspace the handle owns, in bytes. */
int64_t moe_vqlr_workspace_bytes(const moe_vqlr_handle* h);

/* Runs a short probe kernel on the current device
 * and returns how many random 16-byte shared-memory reads per clock one SM sustains from a
 * code book of codebook_size entries (replicated != 0: the eightfold bank-replicated layout used
 * for small code books).  This is the rate that bounds the compressed projections.  Synchronous;
 * allocates and frees a few KB.  Returns OK, INVALID_ARG, UNSUPPORTED (book too large for shared
 * memory), OOM or CUDA. */
int moe_vqlr_probe_lookup_rate(int32_t codebook_size, int32_t replicated, double* lookups_per_clk_per_sm);

#ifdef __cplusplus
}
#endif
#endif /* MOE_VQLR_BENCH_H_ */
