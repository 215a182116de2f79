/*
 * lite3r_debug.h -- benchmarking, inspection and self-test aids of the lite3r library.  Not part of the compute
 * path: nothing here is needed to run the forward of lite3r.h.
 */
#ifndef LITE3R_DEBUG_H
#define LITE3R_DEBUG_H

#include "lite3r.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Self-test of the device-side wait bound.  Every wait inside the kernels (on an mbarrier, or a polling loop of a
 * single-thread role) gives up after one second, records a non-zero code in device_status and lets the kernel end, so a
 * lost signal can never hang the GPU.  This call runs that mechanism on purpose and harmlessly: a one-thread kernel
 * waits, with the given limit (nanoseconds, at most 1e9), on a barrier that nothing arrives on.  After synchronising,
 * *device_status (DEVICE int) must be non-zero (999) and the context must still be usable. */
LITE3R_API lite3r_status lite3r_selftest_wait_expiry(int* device_status, unsigned long long limit_ns, void* stream);

/* Stage timing for benchmarks.  After lite3r_profile_enable(1) (call it with the device current; it creates CUDA
 * events, no device memory), every lite3r_sla_forward brackets its four stages -- V operand preparation, key-block
 * summaries, marginal aggregation, attention -- with event records on the call's stream.  lite3r_profile_stage_ms
 * waits for the last forward's events (the only blocking call of the library) and writes the four durations in
 * milliseconds to ms (HOST, 4 floats; a stage that did not run reports 0).  Not thread-safe; meant for one
 * benchmarking thread. */
LITE3R_API lite3r_status lite3r_profile_enable(int enable);
LITE3R_API lite3r_status lite3r_profile_stage_ms(float* ms);

/* Number of kernel launches the library has enqueued since it was loaded (all threads). */
LITE3R_API long long lite3r_launch_count(void);

/* Test hook: which of its kernels lite3r_sla_plan (and a forward that builds its own plan) uses.  0 = chosen by the
 * size of the problem (the default); 1 = eight rows per CTA with 64-bit keys in shared memory; 2 / 3 = eight / sixteen
 * rows per CTA with single-precision scores in shared memory and exact keys recomputed for the entries at a
 * selection threshold (what long rows get); 4 = four rows per CTA with staged column sums (what rows too long for
 * the others get).  Every variant gives the same plan; a forced variant that does not fit the shape makes the plan call
 * return LITE3R_ERR_UNSUPPORTED.  Process-wide. */
LITE3R_API lite3r_status lite3r_plan_variant(int variant);

/* Test hook: the attention kernel writes its output through TMA stores where a tiled tensor map can describe the
 * output (always, for strides the forward accepts) and with plain vector stores otherwise.  on != 0 forces the plain
 * stores, so that both ways can be compared; on == 0 restores the default.  Process-wide. */
LITE3R_API lite3r_status lite3r_attention_plain_stores(int on);

/* Byte offsets, inside the workspace of lite3r_sla_forward, of its six parts, for tests that inspect intermediates
 * after a forward: offsets[0] per-key-block summaries, bf16 [tiles][4160] = ((H_j W)^T as [e][d] | z_j[d]), the
 * KV summary and normaliser of Algorithm 1 per block with the projection folded in; [1] per-query-block aggregates
 * G_i^T W-folded, bf16 [tiles][64 e][64 d]; [2] zeta_i, fp32 [tiles][64]; [3] dequantised V, fp16 [tiles*Bs][64];
 * [4] class bytes and [5] critical lists when the plan is built inside (plan_inside != 0), else the end of part 3.
 * tiles = B*H*Nb.  Host-only. */
LITE3R_API lite3r_status lite3r_workspace_layout(const lite3r_shape* shape, double crit, double neg, int plan_inside,
                                      size_t* offsets);

#ifdef __cplusplus
}
#endif
#endif /* LITE3R_DEBUG_H */
