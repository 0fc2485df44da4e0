/*
 * freebalance_aids.h - measurement and diagnostic aids of the FreeBalance library.
 *
 * Nothing here is part of the per-layer path of the paper's method (the paper has no
 * counterpart for any of these calls); benchmarks and tests use them to count launches, to
 * time one kernel inside a multi-kernel call, and to exercise the bounded device-side wait.
 * Same conventions as freebalance.h.
 */
#ifndef FREEBALANCE_AIDS_H_
#define FREEBALANCE_AIDS_H_

#include "freebalance.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Kernels this library has launched through `ctx` so far. */
uint64_t fb_launch_count(const fb_ctx* ctx);

/* How many of the launches counted by fb_launch_count were the persistent router kernel. */
uint64_t fb_persistent_launch_count(const fb_ctx* ctx);

/* The next router-kernel launch made through ctx records the two CUDA events (cudaEvent_t
 * handles owned by the caller, either may be NULL) on its stream, one directly before and
 * one directly after the launch, and then forgets them.  Lets a caller time that kernel
 * alone inside a call that launches several kernels. */
fb_status fb_time_next_router_launch(fb_ctx* ctx, void* event_before, void* event_after);

/* Diagnostic: later router launches of this context use at most `stages` stages of the
 * operand pipeline (0 lifts the limit; 1 is not a pipeline: FB_ERR_INVALID_ARG).  Results do
 * not depend on the depth, only the speed does.  Exists so that tests can run short rings and
 * rings with an odd number of stages, in which a stage alternates between the two MMA issuers
 * (they then keep each other informed of their progress; with an even number a stage always
 * serves the same issuer). */
fb_status fb_set_stage_limit(fb_ctx* ctx, int32_t stages);

/* Floor of the one-tile router kernel's main loop.  Launches that kernel for x exactly as
 * fb_predict_load would (same grid, block pairs, pipeline stages and tensor maps; never the
 * persistent kernel, never the k-range split), but with what = 1 the operands are only loaded
 * (no MMA is issued) and with what = 2 they are loaded and multiplied; in both cases nothing
 * follows the main loop: no gating, no selection, no histogram, no output, no status.  Timed
 * by the caller it shows what launch, set-up and the operand stream alone cost for this
 * tiling (1) and what the tensor pipe adds (2).  Errors as fb_predict_load; what outside
 * {1, 2}: FB_ERR_INVALID_ARG. */
fb_status fb_router_floor(fb_ctx* ctx, const fb_router* router, const void* x, int32_t T, int32_t what,
                          fb_stream stream);

/* Stand-in for an attention kernel, for overlap experiments on one GPU (the method hides
 * prediction, planning and weight transfer behind the target layer's attention; "Overlap
 * Analysis").  A compute-bound kernel of `blocks` blocks, one per SM (1024 threads and 120 KB
 * of shared memory each), each running iters x 32 dependent FMAs per thread: it occupies
 * exactly `blocks` SMs for a time proportional to iters and leaves the other SMs - and room
 * beside it for small memory-bound blocks - to other streams.  out: dev f32 [blocks * 1024]
 * (receives meaningless values).  blocks 1..1024, iters 0..2^24. */
fb_status fb_standin_attention(float* out, int32_t blocks, int32_t iters, fb_stream stream);

/* SM clock probe.  A one-thread kernel on `stream` writes n pairs (global nanosecond timer,
 * SM cycle counter) into samples (dev u64 [2 n]), about period_ns apart, and ends by itself
 * (n <= 65536, period_ns <= 100000: at most a few seconds).  Between two samples the SMs ran
 * at (cycle difference) / (time difference) GHz: launched on a side stream beside other work
 * it shows the clock that work really got, at microsecond resolution; with n = 1 on the
 * work's own stream it is a device time stamp.  Reads counters only; changes no setting.
 * Errors: FB_ERR_INVALID_ARG for a NULL or non-device buffer or a size out of range. */
fb_status fb_clock_probe(uint64_t* samples, int32_t n, uint32_t period_ns, fb_stream stream);

/* Phase time stamps of the one-tile router kernel.  Only a library built with -DFB_TIMING
 * carries the stamp code (paper_2608_14205_b200/phase_timing.py builds one beside the normal
 * library and prints the table); the normal build returns FB_ERR_UNSUPPORTED_SHAPE here and
 * its kernels contain none of it.  stamps: dev u64 [blocks][64], or NULL to stop stamping:
 * every block of every following router launch through ctx writes the global nanosecond
 * timer in slots 0..31 and the SM cycle counter in slots 32..63 at its phase boundaries
 * (the slot list is at the top of csrc/fb_router.cuh).  The buffer must hold 64 words per
 * block of the largest launch. */
fb_status fb_set_stamp_buffer(fb_ctx* ctx, uint64_t* stamps);

/* Self-test of the bounded wait that every kernel of the library uses for its barriers: a
 * one-block kernel waits for at most limit_ns (1 .. 100 000 000) on a barrier at which
 * nobody ever arrives, gives up, records FB_ERR_TIMEOUT in ctx's device status word and
 * returns normally; nothing traps and the context stays usable.  fb_device_status then
 * reports FB_ERR_TIMEOUT once and clears it.  waited_ns (dev u64 [1], optional) receives
 * the time the wait actually took.  Asynchronous on `stream`.  Errors: FB_ERR_INVALID_ARG
 * for a NULL context or a limit outside the range. */
fb_status fb_selftest_wait_timeout(fb_ctx* ctx, uint64_t limit_ns, uint64_t* waited_ns, fb_stream stream);

#ifdef __cplusplus
}
#endif
#endif  /* FREEBALANCE_AIDS_H_ */
