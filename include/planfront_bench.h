/*
 * planfront_bench.h -- measurement hooks for benchmarks of libplanfront.so.  Not part of the scoring ABI
 * (planfront.h): the paper has no counterpart for anything declared here and no scoring call depends on it.
 *
 * Two groups:
 *   - pf_timing_enable / pf_timing_classes / pf_timing_read / pf_launch_count are exported by libplanfront.so itself, because they
 *     instrument launches the library makes on streams of its own, which a caller's events cannot bracket;
 *   - pf_probe_alu / pf_probe_write are exported by a separate library, libplanfront_probe.so: micro-kernels that
 *     measure the denominators of the rooflines (instruction issue rates, the pure streaming-write rate).
 */
#ifndef PLANFRONT_BENCH_H
#define PLANFRONT_BENCH_H

#include "planfront.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Optional device timing of the library's own kernels, by class, for roofline accounting (the paper has
 * no counterpart).  While enabled, every call brackets the launches of each class with a CUDA event pair
 * on the stream they are launched on; pf_timing_read waits for the recorded events, adds the elapsed times (ms) and
 * kernel counts per class into ms[PF_T_CLASSES] / kernels[PF_T_CLASSES], and forgets them.
 * PF_T_SCORE: the scoring kernel; PF_T_TOPK: top-k list kernels (merge passes, dense top-k);
 * PF_T_SELECT: the survivor-selection kernels; PF_T_SIMPREP: the simulator's pre-pass (binning, records);
 * PF_T_SIMULATE: the simulator kernel; PF_T_COMPACT: the kernels of pf_compact; PF_T_AGGREGATE: the per-plan
 * serving aggregate; PF_T_FILL: inside pf_search, the kernel that streams the constant blocks of the dense outputs
 * on a stream of its own, from right behind the scoring kernel to the end of the call.  Classes that run on
 * different streams overlap, so their times may add up to more than the call's. */
enum {
    PF_T_SCORE = 0, PF_T_TOPK = 1, PF_T_SELECT = 2, PF_T_SIMULATE = 3, PF_T_AGGREGATE = 4, PF_T_FILL = 5,
    PF_T_SIMPREP = 6, PF_T_COMPACT = 7, PF_T_CLASSES = 8
};
int pf_timing_enable(pf_plan_t *plan, int on);
int pf_timing_read(pf_plan_t *plan, float *ms, uint32_t *kernels);
/* Restrict the timing to the classes whose bit (1 << PF_T_...) is set in `mask` (default: all) and to every
 * `every`-th launch group of a class (default 1: all; 0 counts as 1).  An event between two kernels of a chain costs
 * the chain its overlapped launches, and a timed event in front of the kernel a call waits for last costs the call
 * microseconds, so a benchmark that needs one kernel's duration inside its timed region selects that class alone,
 * samples it, and reads the other classes in a pass of their own.  PF_EINVAL: plan NULL. */
int pf_timing_classes(pf_plan_t *plan, uint32_t mask, uint32_t every);

/* Number of kernels this library has launched in this process (for launch accounting in benchmarks). */
uint64_t pf_launch_count(void);

/* The checked build (the library compiled with -DPF_BOUNDS_CHECK: every index into a shared-memory image, queue,
 * table, timeline, order table, key list or output array is range-checked on the device; a violation is recorded
 * and the access redirected to element 0 -- nothing traps).  pf_check_read waits for the device, copies the plan's
 * record to out[6] and clears it: out[0] = one bit per kind of array that saw a bad index (0 = clean), out[1] = the
 * last such kind, out[2..3] = the offending index, out[4..5] = the array's length.  The ordinary build returns
 * PF_EUNSUPPORTED and zeros. */
int pf_check_read(pf_plan_t *plan, uint32_t *out);
/* The checks' own check (checked build only, else PF_EUNSUPPORTED): one device thread asks for element 7 of a
 * 4-element array through the checking macro; the store is redirected inside the array and the next pf_check_read
 * must show bit 17, index 7, length 4. */
int pf_check_selftest(pf_plan_t *plan);

/* How the plan's latest scoring call inside pf_search was divided between the scoring kernel and the kernel that
 * streams constant blocks: the number of blocks of candidates the call's range was cut into, candidates per block,
 * how many blocks the scoring kernel took itself (the evaluated ones), and how many the fill kernel counted as
 * streamed (the rest, when the call has completed).  Reads a few words back from the device (synchronizes the
 * device).
 * Errors: PF_EINVAL (NULL pointer, or the plan has no such record), PF_ECUDA. */
int pf_bench_fill_span(pf_plan_t *plan, uint64_t *n_blocks, uint64_t *block_candidates, uint64_t *scored_blocks,
                       uint64_t *filled_blocks);

/* Roofline probes (libplanfront_probe.so).
 * The caller times them with events on `stream`; neither call synchronises or allocates.
 *
 * pf_probe_alu: one launch at full occupancy (8 blocks of 256 threads per SM) in which every thread runs
 * 8 independent dependency chains of one instruction kind for `iters` loop trips of 4 steps each:
 * PF_PROBE_FFMA fp32 fused multiply-add, PF_PROBE_IMAD 32-bit integer multiply-add, PF_PROBE_LOGIC an
 * alternation of 3-input logic ops and 32-bit adds.  *h_thread_instructions (host) receives the number of
 * thread-level instructions of that kind the launch executes; dividing by the launch's duration gives the
 * issue-rate peak for that kind.  d_sink: 4 device bytes, practically never written.  1 <= iters <= 2^24.
 *
 * pf_probe_write: fills `bytes` (a multiple of 16, below 2^35, 16-byte aligned device buffer) with 16-byte
 * streaming stores, one per thread over a grid as large as the buffer -- the store the scoring kernel uses for
 * its dense outputs, in the fastest pure-write pattern; bytes / duration is the write ceiling.
 * Errors: PF_EINVAL for a null pointer, a bad kind, iters or size; PF_ECUDA if the launch fails (the probe library
 * keeps no error text). */
enum { PF_PROBE_FFMA = 0, PF_PROBE_IMAD = 1, PF_PROBE_LOGIC = 2 };
int pf_probe_alu(int kind, uint32_t iters, uint32_t *d_sink, uint64_t *h_thread_instructions, void *stream);
int pf_probe_write(void *d_buf, size_t bytes, void *stream);

#ifdef __cplusplus
}
#endif
#endif
