/*
 * llmcad_profile.h -- measurement and diagnostic interface of the token-tree verification
 * library. Nothing here is part of the verification path (include/llmcad.h): these calls exist
 * for benchmarks, profiles and the tests of the failure paths. They are exported by the same
 * shared library.
 */
#ifndef LLMCAD_PROFILE_H
#define LLMCAD_PROFILE_H

#include "llmcad.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Per-launch timing of kernels in isolation. While enabled, every skinny-GEMM launch (kind 0) and
 * every tree-attention launch (kind 1) of this context is bracketed by CUDA events on the
 * launching stream (which keeps consecutive kernels from overlapping under programmatic dependent
 * launch: the figures are those of a kernel running alone). llmcad_get_kernel_timing waits for the
 * recorded launches of `kind`, returns their summed duration and count since the last query, and
 * forgets them. */
int llmcad_set_kernel_timing(llmcad_ctx *ctx, int32_t enable);
int llmcad_get_kernel_timing(llmcad_ctx *ctx, int32_t kind, double *total_ms /*HOST*/, int64_t *n_launches /*HOST*/);

/* Timeline of the kernels inside an undisturbed pass. While `trace` (DEVICE, [capacity][256][16]
 * uint64, or NULL to stop) is set, the next `capacity` tensor-core GEMMs and attention launches of
 * this context each fill one [256][16] slice: per CTA, nanosecond timestamps (%globaltimer). A GEMM
 * (streaming kernel + finishing kernel) shares one slice: streaming CTA entry (0), set-up done (1),
 * first weight copy issued (2), grid dependency resolved (3), first accumulator ready (4), last
 * weight copy issued (6), last MMA issued (7), accumulators in the workspace (8), streaming CTA
 * exit (13); finishing CTA entry (9), its grid dependency resolved (10), exit (12). Attention:
 * entry (0), grid dependency resolved (1), first key tile in shared memory (2), key loop done (3),
 * partial rows merged and handed to their owners (4), cluster barrier passed (5), output stored (6),
 * exit (12). Launch order of a pass: QKV GEMM, then per layer attention, O, gate/up,
 * down, next QKV (lm_head after the last layer). The stamps cost a predicated store each and do not
 * change how consecutive kernels overlap. */
int llmcad_set_gemm_trace(llmcad_ctx *ctx, uint64_t *trace, int32_t capacity);

/* Number of kernels this library has launched through this context so far. */
int64_t llmcad_launch_count(const llmcad_ctx *ctx);

/* Every device-side wait of this context's kernels (the shared-memory barriers between the roles of
 * a CTA; no kernel waits for another CTA) gives up after `ns` nanoseconds; the kernel
 * then sets LLMCAD_ERR_TIMEOUT in the status word, lets all its roles fall out of their loops,
 * frees its tensor memory and returns. Default 2 s; 0 restores the default. */
int llmcad_set_wait_limit_ns(llmcad_ctx *ctx, uint64_t ns);

/* Self-test of that path (bf16 tensor-core contexts only, vocab >= 160): runs a small GEMM on the
 * context's own work buffers whose activation copies are withheld (a launch flag), so that its ring
 * stages never fill and every role's wait runs out. Nothing faults or traps: the kernel returns after the wait
 * limit (set a short one first: the call refuses limits above 100 ms with LLMCAD_ERR_INVALID_ARG).
 * Synchronises `stream` and returns the device status word, LLMCAD_ERR_TIMEOUT when the path
 * works, or a negative host-detected error. The context is usable afterwards. */
int llmcad_selftest_wait_timeout(llmcad_ctx *ctx, void *stream);

/* Micro-benchmarks of the machine, context-free, on the current device (no tensor of the library is involved).
 *
 * llmcad_probe_bulk_copy: one CTA per SM, one issuing thread each, reads `bytes` (DEVICE buffer `src`, 16-byte
 * aligned; every byte once, so a buffer much larger than L2 comes from HBM) into shared memory with cp.async.bulk
 * copies of `copy_bytes` (a multiple of 16), `in_flight` (1..16) of them outstanding per CTA, copy_bytes * in_flight
 * <= 200 KB: the weight stream of the skinny GEMMs without a consumer. Returns the rate of the slowest CTA's
 * schedule, GB/s over all SMs, and the mean time from issuing a copy to its completion.
 * llmcad_probe_mma_sync: `warps` (1..32) warps per SM issue mma.sync.m16n8k16 bf16 into `accumulators` (1, 2, 4, 8)
 * independent accumulators each: multiply-adds per clock and SM, and SM cycles per MMA of one warp (with one
 * accumulator and one warp: the latency of a dependent MMA).
 * Both synchronise `stream`; LLMCAD_ERR_TIMEOUT if a copy does not arrive within the default wait limit. */
int llmcad_probe_bulk_copy(const void *src /*DEVICE*/, size_t bytes, int32_t copy_bytes, int32_t in_flight, void *stream,
                           double *gbs /*HOST*/, double *latency_us /*HOST*/);
int llmcad_probe_mma_sync(int32_t warps, int32_t accumulators, void *stream, double *fma_per_clk_sm /*HOST*/,
                          double *cycles_per_mma /*HOST*/);

#ifdef __cplusplus
}
#endif
#endif /* LLMCAD_PROFILE_H */
