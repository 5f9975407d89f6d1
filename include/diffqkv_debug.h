/*
 * diffqkv_debug.h -- test, tuning and benchmark hooks of libdiffqkv.  None of these is part of the paper's operation
 * (the paper has no counterpart for any of them); they exist so that tests can move the places where work is cut,
 * force one of two equivalent code paths, make a bounded device wait run out without anything faulting, and so that
 * benchmarks can time one kernel of a call and count launches.  All of it is process-wide host state held in atomics:
 * a setting applies to calls made after it, from any thread; it is not tied to a stream or a device.
 */
#ifndef DIFFQKV_DEBUG_H_
#define DIFFQKV_DEBUG_H_

#include "diffqkv.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Tuning hook (process-wide host state): cap the number of persistent blocks the TMA decode kernel
 * launches; 0 restores the default of one block per SM.  Workspace sizes must be queried after the
 * cap is set.  Mainly for tests, which use it to move the places where sequences are cut.
 */
void diffqkv_set_max_blocks(int32_t max_blocks);

/*
 * Test hook (process-wide host state): a non-zero value makes diffqkv_decode_topk always select over all scores of a
 * row; 0 (the default) lets it first try the selection that reads only the 16-token blocks whose largest score can
 * reach the top.  Both give the same result.
 */
void diffqkv_topk_general_only(int32_t on);

/*
 * Test hook (process-wide host state): the projections (diffqkv_augq, diffqkv_augq_rope, diffqkv_project) take a
 * weight-streaming kernel when there are at most 64 rows (decode: one token per sequence) and the tensor-core GEMM
 * otherwise; a non-zero value makes them always take the tensor-core GEMM.  Both round x and a to bf16 once and
 * accumulate in fp32; they differ in summation order only.
 */
void diffqkv_force_tensor_gemm(int32_t on);

/* Which attention kernel the most recent diffqkv_prefill call launched: 0 none yet, 1 generic, 2 tensor-core (for tests). */
int32_t diffqkv_last_prefill_kernel(void);

/* Which split kernel the most recent decode call launched: 0 none yet, 1 generic, 2 TMA (for tests). */
int32_t diffqkv_last_decode_kernel(void);

/*
 * Profiling hook for benchmarks (process-wide host state, not thread-safe).  While both arguments
 * are non-NULL cudaEvent_t handles, every decode call records `before_split` just before and
 * `after_split` just after its split kernel on the call's stream, so the split kernel can be timed
 * apart from the combine kernel.  Pass NULL, NULL to switch it off.
 */
void diffqkv_profile_split_events(void *before_split, void *after_split);

/* Kernels launched by this library since it was loaded (host counter, for benchmarks). */
int64_t diffqkv_launch_count(void);

/*
 * Test hook (process-wide host state): the generic decode path (fp32 caches, bf16 shapes without a tensor map) has
 * two kernels, one block per (split, unit of query heads, sequence) that reads every K and V row once for all heads of
 * the unit, and one block per (split, query head, sequence) for head counts and dimensions the first does not take.
 * A non-zero value makes it always take the second.  Both compute the same thing.
 */
void diffqkv_debug_decode_per_head_only(int32_t on);

/*
 * Test hook (process-wide host state) for the on-chip merge of the TMA decode kernel.  With few, short rows the
 * blocks that share a (sequence, head group) row are launched as a thread-block cluster and the first of them merges
 * the others' partial results out of their shared memory; no partials go through global memory and no combine kernel
 * is launched.  Automatically this is done when the largest power of two of blocks per row (at most 8) fills four
 * fifths of the SMs and the cache holds at most 160 MB for these rows; results differ from the two-kernel path only
 * in fp32 summation order.
 *   mode < 0  automatic (default)    mode = 0  never    mode > 0  whenever at least two blocks per row fit on the GPU
 */
void diffqkv_debug_decode_cluster(int32_t mode);

/*
 * Failure-path hook for tests.  Every wait of the library's kernels on a copy in flight is bounded: when it runs
 * out the block reports DIFFQKV_ERR_TIMEOUT in *dev_status, stops computing, lets copies already in flight land,
 * and returns; results of that call are undefined, the context stays usable.  This hook makes that path reachable
 * without breaking anything: for TMA decode launches made while it is set, the wait limit is `wait_limit_ns`
 * (default 2 000 000 000), and the producer of the block that owns flat tile `skip_tile` issues neither that tile's
 * copies nor their completion count, so nothing is in flight for it and its consumers' wait runs out.
 *   wait_limit_ns <= 0 restores the default limit; skip_tile < 0 skips nothing.
 */
void diffqkv_debug_decode_timeout(int64_t wait_limit_ns, int64_t skip_tile);

#ifdef __cplusplus
}
#endif
#endif /* DIFFQKV_DEBUG_H_ */
