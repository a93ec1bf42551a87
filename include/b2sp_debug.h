/*
 * b2sp -- measurement, test and tuning aids.  Not part of the method of the paper (no passage of it
 * corresponds to anything here) and not needed to use the three ops of b2sp.h; exported by the same
 * library.
 */
#ifndef B2SP_DEBUG_H
#define B2SP_DEBUG_H

#include "b2sp.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * The FP32 FMA rate the current device sustains right now (8 independent register-only FMA chains
 * per thread, 2048 threads on every SM, best of 10 launches timed with CUDA events), in GFLOP/s, for
 * the denominator of a roofline fraction.
 * `iters` = chain length in units of 64 FMAs per thread (4096 takes about a millisecond);
 * `scratch` = DEVICE pointer to at least one float (never written in practice); `gflops_host` =
 * HOST pointer for the result.  Synchronises `stream`.  B2SP_ERR_INVALID_ARG / B2SP_ERR_CUDA.
 */
b2sp_status b2sp_probe_fp32_peak(int iters, float *scratch, double *gflops_host, void *stream);

/*
 * The rate at which the SMs of the current device pull 32 KB operand chunks out of L2 into shared memory with bulk
 * asynchronous copies (`cp.async.bulk`, three in flight per SM, one CTA per SM, all SMs at once; best of 5 launches
 * timed with CUDA events), in GB/s per SM and for the whole GPU.  The dense-tile kernels stream their B / D operand
 * tiles this way; the numbers say how much of that path they use.
 * `scratch` = DEVICE buffer of `scratch_bytes` >= 1 MiB + 16 bytes, 16-byte aligned; its first 16 bytes are
 * overwritten, up to 16 MiB of the rest are read (any contents).  `gbs_per_sm_host`, `gbs_total_host` = HOST pointers
 * for the results.  Synchronises `stream`.  B2SP_ERR_INVALID_ARG, B2SP_ERR_CUDA; B2SP_ERR_TIMEOUT if a copy did not
 * land within the kernel's bounded wait.
 */
b2sp_status b2sp_probe_l2_pull(void *scratch, size_t scratch_bytes, double *gbs_per_sm_host, double *gbs_total_host, void *stream);

/*
 * Which kernel family the most recent call of the given op (B2SP_OP_*) on this host thread resolved
 * B2SP_ALGO_AUTO (or its explicit request) to: one of B2SP_ALGO_ROW, _ROW_NAT, _TILE; -1 if the
 * op has not been called.  Number of kernels that call enqueued: b2sp_last_launches(op).
 */
int b2sp_last_algo(int op);
int b2sp_last_launches(int op);

/*
 * Overrides, process-wide, the number of K splits the dense-tile planner picks (how many CTAs share
 * one tile of the output along the columns of S); 0 gives the choice back to the planner.  A value
 * larger than the number of 128-column blocks of S is ignored.  It changes b2sp_workspace_bytes for
 * the dense-tile family and the order of the floating-point sums, so set it before sizing the
 * workspace.  For tests of the K-split epilogues and for tuning only.
 */
void b2sp_debug_force_k_splits(int k_splits);

/*
 * Overrides, process-wide, how the dense-tile planner deals the work of an op to CTAs.  The planner knows two
 * partitions: "tiles x K splits" (every CTA owns one 128-row tile of the output and one of equal ranges of the
 * columns of S) and "balanced" (the 4-block accumulation granules of all output tiles, in tile order, dealt evenly
 * to one CTA per SM, so that a CTA may end one tile and begin the next; offered where the kernel mode supports it
 * and the number of 128-column blocks of S is a multiple of four).  partition = 0: the planner chooses (balanced
 * where its longest CTA is at least 6% shorter); 1: tiles x K splits only; 2: balanced wherever it is offered.
 * Like b2sp_debug_force_k_splits it changes b2sp_workspace_bytes and the order of the sums: set it before sizing
 * the workspace.  For tests and tuning only.
 */
void b2sp_debug_force_partition(int partition);

/*
 * Test hook for the bounded waits of the dense-tile kernels.  Every wait inside those kernels gives up after a
 * time limit (0.3 s), sets the workspace's device status word and lets its CTA leave through the normal
 * teardown; b2sp_device_status and the host-buffer entry points then report B2SP_ERR_TIMEOUT.  To let a test see
 * that path without stalling a GPU for long, this call (a) makes the TMA producer of every CTA of the dense-tile
 * kernels launched afterwards leave out its `chunk`-th operand chunk, whose barrier therefore never completes,
 * and (b) sets the time limit of the current device to `limit_ns` nanoseconds (a few milliseconds).  No wait is
 * unbounded at any time.  chunk < 0 switches the hook off and restores the 0.3 s limit; call that before any
 * other work.  Process-wide, synchronises the device (a copy to constant memory), not for production use.
 */
b2sp_status b2sp_debug_inject_wait_timeout(int chunk, unsigned long long limit_ns);

#ifdef __cplusplus
}
#endif
#endif /* B2SP_DEBUG_H */
