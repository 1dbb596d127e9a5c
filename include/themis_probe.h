/*
 * libthemis, measurement probes.  These entry points are NOT part of the solver
 * (include/themis.h): they exist so that the benchmark can measure the integer-ALU
 * rate its roofline is quoted against, and so that the kernels' bounded barrier
 * wait can be tested without a fault.  The paper (Themis, arXiv 2407.14843) has no
 * counterpart for either.  Same conventions as themis.h: THEMIS_OK or a negative
 * THEMIS_E_* code, "d_" pointers are caller-owned device memory, work is enqueued
 * on the given stream without synchronising, nothing is allocated.
 */
#ifndef THEMIS_PROBE_H_
#define THEMIS_PROBE_H_

#include "themis.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Integer-ALU throughput probe (not part of the method, and the paper has no
 * counterpart): every thread keeps 16 independent chains in registers and runs
 * `iters` iterations of 4 rounds, each round one add-then-min update per chain (the
 * operation pair of the recurrence), every update reading two values produced one
 * round earlier.  Instruction form by mode:
 *   0: separate 32-bit add and unsigned min;
 *   1: fused 32-bit add-min (one instruction per update);
 *   2: two adds and one three-input min per two updates;
 *   3: fused add-min on packed 2 x 16-bit (two cell updates per instruction);
 *   4: single-precision add and min;
 *   5: the packed recurrence kernel's own inner step, operands loaded from shared
 *      memory as there but without stages, barriers or global traffic: every
 *      thread walks `iters` columns of 256 chunk steps of 8 x 8 cells (threads
 *      must be 256; 128 fused instructions per 4 steps as in mode 3).
 * Launches `blocks` x `threads` (32..1024) and writes one word per thread to d_sink
 * (blocks*threads uint32).  Updates performed = blocks * threads * iters * 64
 * (x 2 cells in mode 3; blocks * 256 * iters * 256 * 64 cells in mode 5).
 */
int themis_alu_probe(int mode, int blocks, int threads, int iters, uint32_t *d_sink,
                     void *cuda_stream);

/*
 * Bounded-wait probe (not part of the method; the paper has no counterpart).  The
 * recurrence kernels stage every row G_s with an asynchronous bulk copy and wait for
 * it on a shared-memory barrier; that wait gives up after a fixed number of attempts
 * and the instance reports THEMIS_STATUS_TIMEOUT instead of hanging.  This entry point
 * runs the same wait routine in a one-warp kernel on two barriers: one whose 16-byte
 * copy from d_src16 (16-byte aligned) is issued (waited for with the kernels' own
 * limit), and one that expects 16 bytes which nothing delivers (waited for with
 * `max_polls` attempts, 1 .. 2^20).  Results:
 *   d_status[0] = THEMIS_STATUS_OK and d_dst16[0..3] = d_src16[0..3]  (the copy landed);
 *   d_status[1] = THEMIS_STATUS_TIMEOUT                               (the wait ran out);
 * the kernel returns normally in both cases and the context stays usable.
 * Returns THEMIS_E_INVALID_ARG for a NULL or misaligned pointer or max_polls out of range.
 */
int themis_wait_probe(int32_t max_polls, const uint32_t *d_src16, uint32_t *d_dst16, int32_t *d_status,
                      void *cuda_stream);

/*
 * Report of the bounds-checked build (not part of the method; the paper has no
 * counterpart).  Built with -DTHEMIS_CHECK_BOUNDS (python -m paper_2407_14843_b200.build
 * --check-bounds writes libthemis_check.so), the solver kernels pass every index into
 * shared or global memory that they compute through a range check; the first index found
 * outside its range is recorded in the workspace (and clamped, so that nothing faults and
 * the kernels run to their end), and every solve starts with a clear record.  This call
 * waits for the stream and copies the record of the last solve on `d_workspace` to the
 * host:
 *   h_report[0]  site number of the first violation, 0 if there was none
 *   h_report[1]  the offending index        h_report[2]  the limit it had to stay below
 *   h_report[3]  1 if the library was built with the checks, else 0 (then the rest is 0)
 * The normal build checks nothing and pays nothing.  Results of a checked solve equal
 * those of the normal build as long as no violation is reported.
 */
int themis_bounds_check_report(const themis_problem_t *problem, int vertical, const void *d_workspace,
                               size_t workspace_bytes, int32_t *h_report, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* THEMIS_PROBE_H_ */
