/*
 * stairs_debug.h - UNSTABLE inspection hooks of the stairs library, for its own tests and
 * tuning scripts.  Not part of the supported interface (include/stairs.h): signatures and
 * buffer numbering may change without notice.  The paper has no counterpart to these calls.
 */
#ifndef STAIRS_DEBUG_H_
#define STAIRS_DEBUG_H_

#include "stairs.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Per-call device timing.  With profiling on, stairs_validate brackets the call and each
 * weight-streaming GEMM launch with events; stairs_profile_read waits and returns the
 * summed GEMM time, the number of GEMM launches and the whole call's time (ms) of the
 * most recent stairs_validate. */
int stairs_profile(stairs_ctx *ctx, int enable);
int stairs_profile_read(stairs_ctx *ctx, float *gemm_ms, int32_t *gemm_launches, float *call_ms);

/* Inspection hook for tests: device address and size of one activation buffer inside the
 * workspace after a pass (which: 0 residual x fp32 [rows, d], 1 normed h, 2 qkv fp32,
 * 3 attention output o, 4 MLP activation ff, 5 argmax keys u64, 6 per-phase timestamps of the
 * persistent kernel, u64 ns [2 CTAs][phases][8 stamps: start, work done, arrived, prologue done, first tile ready, first MMA, last MMA, first activation load], written while
 * profiling is on; 7 the persistent kernel's split-tile partial-sum slots and 8 its parked attention
 * states, both u32 words that all read 0xffffffff ("empty") between calls). */
int stairs_debug_buffer(stairs_ctx *ctx, int which, void **ptr_dev, size_t *bytes);

/* Tuning knobs of the persistent kernel, for sweeps.  what 0: 64-element k-blocks per pipeline
 * stage (0 = chosen per row box, 1 or 2); what 1: K/V chunk buffers of the attention phases
 * (0 = chosen from the context length, 1..4); what 2: non-zero stages K/V with 16-byte copies
 * from the compute warps even where tiled bulk copies apply; what 3: 1 keeps the attention
 * contractions on mma.sync even where the tcgen05 path applies, 2 uses the tcgen05 path for every
 * call it can serve (0: chosen per call).  Takes effect with the next call. */
int stairs_debug_tune(stairs_ctx *ctx, int what, long long value);

#ifdef __cplusplus
}
#endif
#endif /* STAIRS_DEBUG_H_ */
