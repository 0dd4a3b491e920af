/*
 * nuna_debug.h -- test hooks exported by libnuna.so besides the public C ABI (include/nuna.h).
 *
 * They expose host-side pieces (planning, probe analysis, the probe's pointer chain) and two
 * host-made failure cases (a barrier that is one arrival short, ready flags that nobody publishes) to
 * the tests.  Not part of the supported interface; signatures may change.
 */
#ifndef NUNA_DEBUG_H
#define NUNA_DEBUG_H

#include "../../include/nuna.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Per-SM work lists planned for a one-shot of `ntiles` tiles under `topo` (NULL = no probe), by the
 * general planner (generic != 0) or its closed form, dealt to `domains` SM domains (0 = what the
 * topology holds).  off: [num_sms + 1], tiles: [ntiles].                                             */
int nuna_debug_plan_oneshot(const nuna_topology_t* topo, int num_sms, int nranks, size_t ntiles, size_t tile_bytes,
                            int generic, int domains, unsigned* off, unsigned* tiles);

/* Every block of a `grid`-block launch arrives at a flag barrier that expects `expected` arrivals and
 * waits at most timeout_ms; writes how many blocks passed.  expected > grid makes the waits run out.    */
int nuna_debug_barrier_selftest(unsigned grid, unsigned expected, unsigned timeout_ms, unsigned* passed);

/* The flag-synchronised two-shot allreduce with an explicit timeout.  debug_bits = 1: consumers wait for a
 * flag value nobody publishes, so every wait runs out after timeout_ms, the kernel returns and the status
 * word latches NUNA_ERR_TIMEOUT.                                                                        */
int nuna_debug_twoshot(const void* const* src, void* const* dst, int nranks, size_t count, int dtype,
                       unsigned timeout_ms, unsigned debug_bits);

/* One launch of the one-shot allreduce (8 ranks, bf16, count a multiple of 8) under a placement -- 0 round-
 * robin, 1 co-located groups, 2 per-SM work lists -- with the latency of every work item's first load sampled
 * per warp: hist[b] += samples with latency in [b * NUNA_DEBUG_LAT_STEP, +NUNA_DEBUG_LAT_STEP) SM cycles, the last
 * bin taking everything above.  The analogue of the paper's per-access latency distributions under its two
 * placements (Section 6.2).  Destinations receive the ordinary result.  Synchronises the device.          */
#define NUNA_DEBUG_LAT_BINS 64
#define NUNA_DEBUG_LAT_STEP 32
int nuna_debug_access_latency(const void* const* src, void* const* dst, size_t count, int placement, unsigned* hist);

/* One launch of the register-sharing one-shot allreduce (8 ranks, bf16, all destinations per thread, launched
 * as nuna_allreduce_oneshot launches it for `flags`: NUNA_LAUNCH_PDL, NUNA_HINT_RESIDENT; tile size and prefetch
 * as the options say) on `stream`, in which thread 0 of block b < NUNA_DEBUG_TRACE_BLOCKS also writes to device
 * memory trace[(slot * NUNA_DEBUG_TRACE_BLOCKS + b) * 4 + k], k = 0: global-timer ns at block start, 1: when its
 * wait for the predecessor kernel returned, 2: when the block had issued its last store, 3: the SM it ran on.
 * Capturable (no allocation, no synchronisation): a caller records a graph of such launches with slot = node
 * index and reads where the time between dependent launches goes.  *grid_blocks (optional) receives the grid.  */
#define NUNA_DEBUG_TRACE_BLOCKS 1024
int nuna_debug_oneshot_regs_traced(const void* const* src, void* const* dst, size_t count, unsigned flags, unsigned slot,
                                   unsigned long long* trace, unsigned* grid_blocks, void* stream);

/* nuna_launch_floor's empty kernel; with trigger_first != 0 it releases its dependent launch before it waits
 * for its own predecessor instead of after.                                                              */
int nuna_debug_launch_floor(unsigned blocks, unsigned flags, int trigger_first, void* stream);

/* The probe's host-side clustering / verdict on a caller-supplied (num_sms x nlines) latency matrix.   */
int nuna_debug_analyse_topology(const float* lat, const float* lat_rep, int num_sms, int nlines, nuna_topology_t* out);

/* The probe's single-cycle permutation over nnodes nodes (next[]) and the node a host walk of `steps`
 * steps from `start` ends on.                                                                            */
int nuna_debug_chain(unsigned* next, int nnodes, unsigned long long seed, unsigned start, int steps, unsigned* end);

#ifdef __cplusplus
}
#endif
#endif /* NUNA_DEBUG_H */
