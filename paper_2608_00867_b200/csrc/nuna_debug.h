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

/* A flag-synchronised two-shot allreduce whose consumers wait for a flag value nobody publishes: every
 * wait runs out after timeout_ms, the kernel returns and the status word latches NUNA_ERR_TIMEOUT.     */
int nuna_debug_twoshot_unset_flags(const void* const* src, void* const* dst, int nranks, size_t count, int dtype,
                                   unsigned timeout_ms);

/* The probe's host-side clustering / verdict on a caller-supplied (num_sms x nlines) latency matrix.   */
int nuna_debug_analyse_topology(const float* lat, const float* lat_rep, int num_sms, int nlines, nuna_topology_t* out);

/* The probe's single-cycle permutation over nnodes nodes (next[]) and the node a host walk of `steps`
 * steps from `start` ends on.                                                                            */
int nuna_debug_chain(unsigned* next, int nnodes, unsigned long long seed, unsigned start, int steps, unsigned* end);

#ifdef __cplusplus
}
#endif
#endif /* NUNA_DEBUG_H */
