/*
 * nuna.h -- C ABI of the B200 (sm_100a) emulated-rank collective library.
 *
 * N ranks are emulated as N separate device buffers on ONE GPU.  Every
 * collective reads N "rank" source buffers and writes N "rank" destination
 * buffers; there is no inter-GPU traffic.  The operations are those the paper
 * uses for tensor-parallel inference (Section 2.1: allreduce aggregates the
 * ranks' partial activations, allgather assembles every rank's chunk in every
 * rank's buffer, reduce-scatter is named with them in Section 2.2), executed
 * with the latency-optimised direct / all-pairs algorithm (Section 5.1), and
 * the thread-block placement idea of Section 4.2 (Algorithm 1) mapped onto SMs.
 *
 * Numerics: dst = rne_T((((f(src[0]) + f(src[1])) + ...) + f(src[N-1]))) where f
 * widens the storage type T exactly to binary32, every partial sum is an IEEE
 * binary32 (round to nearest even, subnormals kept), ranks are folded in the
 * fixed order 0..N-1 starting from rank 0's value, and there is ONE final
 * round-to-nearest-even to T (none for T = binary32).  T is bf16 (the type the
 * benchmarks use), IEEE binary16 or binary32.  A NaN result is canonical
 * (0x7FFF / 0x7FFFFFFF).  Every destination receives the same bits.  Allgather
 * and alltoall are bit copies.
 *
 * Conventions, all entry points:
 *  - `src` / `dst` are HOST arrays of `nranks` DEVICE pointers (except in
 *    nuna_allreduce_host).  The arrays are read during the call and may be
 *    freed on return.  The caller owns every rank buffer.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream);
 *    collective calls are asynchronous on it and perform no host
 *    synchronisation, no allocation and no host<->device copy once the
 *    per-device context exists (see nuna_init), so they can be stream-captured.
 *  - The return value is a nuna_status_t.  Argument errors launch nothing.
 *    Conditions detected on the device (a barrier that timed out) are latched
 *    in a status word read by nuna_device_status.
 *  - 1 <= nranks <= NUNA_MAX_RANKS.  count == 0 returns NUNA_OK without a
 *    launch.  Every pointer must be 16-byte aligned (NUNA_ERR_ALIGNMENT).
 *    No destination range may overlap a source range or another destination
 *    range (NUNA_ERR_ALIAS): in the emulation another rank's thread blocks
 *    may still be reading a source, so in-place operation is not defined.
 *  - Sizes quoted in KB/MB anywhere in this project are binary.
 */
#ifndef NUNA_H
#define NUNA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    NUNA_OK = 0,
    NUNA_ERR_INVALID_ARG = 1,
    NUNA_ERR_UNSUPPORTED_DTYPE = 2,
    NUNA_ERR_ALIGNMENT = 3,
    NUNA_ERR_ALIAS = 4,
    NUNA_ERR_CUDA = 5,
    NUNA_ERR_TIMEOUT = 6,
    NUNA_ERR_CAPTURING = 7,
    NUNA_ERR_TOO_MANY_RANKS = 8,
    NUNA_ERR_TOO_LARGE = 9
} nuna_status_t;

typedef enum { NUNA_BF16 = 0, NUNA_F16 = 1, NUNA_F32 = 2 } nuna_dtype_t;   /* element (storage) type; 2, 2, 4 bytes */

#define NUNA_MAX_RANKS 16

/* `flags`, bits 0-1: thread-block placement (Section 4.2 / Section 5.3 baseline). */
#define NUNA_PLACE_ROUNDROBIN 0u   /* locality-unaware: work item i -> thread block i mod grid          */
#define NUNA_PLACE_AWARE      1u   /* a tile's N work items (one logical group, Section 4.2.1) are co-located:
                                      in one thread block, sharing the tile through L1, by default; through
                                      registers, shared memory, per-SM work lists or a cluster with
                                      NUNA_PLACE_REGS / _STAGED / _SM_LISTS / _CLUSTER; only the one-shot
                                      allreduce distinguishes placements                                   */
#define NUNA_PLACE_AUTO       2u   /* the placement-aware kernel measured fastest for the size and launch: the
                                      co-located group that shares its tile through registers (NUNA_PLACE_REGS)
                                      at every size with NUNA_LAUNCH_PDL or NUNA_HINT_RESIDENT, otherwise from
                                      1 MiB of sources in total at 8 ranks or more, 2 MiB below; else exactly
                                      the ROUNDROBIN kernel                                                */
#define NUNA_PLACE_MASK       3u
/* `flags`, bit 4 (nuna_allreduce_twoshot only): the reducing block stores its tile straight into all N
 * destinations, with no intermediate shard and no barrier.                                             */
#define NUNA_TWOSHOT_PUT      16u
/* `flags`, bit 5: hint that the sources were just written and are L2-resident (the decode case: a GEMM
 * epilogue produced them).  The register-sharing and shared-memory-staged one-shot kernels then co-locate
 * all destinations of a tile (one fetch per tile) at every size, store with the ordinary cache policy
 * instead of evict-first, and no kernel prefetches ahead of a dependent launch's wait.                  */
#define NUNA_HINT_RESIDENT    32u
/* `flags`, bit 6: launch with programmatic stream serialization.  The kernel may be scheduled while its
 * predecessor in the stream drains; it waits for that grid's completion and memory visibility before
 * its first global access, so results are those of an ordinary stream-ordered launch.  The round-robin
 * one-shot ignores it above 16 MiB of sources, where it was measured not to pay.  Unless
 * NUNA_HINT_RESIDENT is set, a block of the register-sharing one-shot (below 8 MiB per rank), of either
 * two-shot form (up to 128 MiB of sources; 8 MiB beyond 8 ranks) and of the bulk-copy allgather and
 * alltoall also asks L2, before that wait, to fetch its first tile of the sources (a prefetch returns
 * nothing to the kernel; L2 is the point of coherence, so what the predecessor still writes is what the
 * loads after the wait see).                                                                            */
#define NUNA_LAUNCH_PDL       64u
/* `flags`, bit 7, with NUNA_PLACE_AWARE on nuna_allreduce_oneshot: dispatch the co-located groups through
 * per-SM work lists.  The lists are planned by Algorithm 1 from the topology the last
 * nuna_probe_topology call on this device found (none: one domain, SMs in index order); persistent blocks
 * read %smid, claim the groups planned for their SM and then take over what is left elsewhere.  The
 * first call for a given (nranks, count) builds and uploads the plan (allocates: NUNA_ERR_CAPTURING on a
 * capturing stream); later calls only launch.  Calls sharing a plan must be stream-ordered.             */
#define NUNA_PLACE_SM_LISTS   128u
/* `flags`, bit 8, with NUNA_PLACE_AWARE on nuna_allreduce_oneshot, 2 <= nranks <= 8: run each tile's N work
 * items as one thread-block cluster of N blocks (placed by the hardware on one GPC).  Block r fetches
 * source r's tile once into shared memory; after a cluster barrier every block reads all N tiles from its
 * neighbours' shared memory and folds them for its own destination.  Ignored for other rank counts.
 * Experimental: measured 3.5-6x slower than the baseline at every size; NUNA_PLACE_AUTO never picks it. */
#define NUNA_PLACE_CLUSTER    256u
/* `flags`, bit 9, with NUNA_PLACE_AWARE on nuna_allreduce_oneshot: the co-located group staged through
 * shared memory.  One thread of the block fetches the tile's N source slices with bulk asynchronous
 * copies (global -> shared, completion on an mbarrier, this GPU's memory only); every emulated rank's row
 * then folds the N slices out of shared memory and stores its own destination.                          */
#define NUNA_PLACE_STAGED     512u
/* `flags`, bit 10, nuna_allreduce only: for messages beyond the one-shot range use the flag-synchronised
 * two-shot (reduce-scatter, per-tile ready flags, allgather) instead of the put form.                   */
#define NUNA_TWOSHOT_SYNC     1024u
/* `flags`, bits 11-12, nuna_chain_create only: run the chain as ONE kernel on a single thread-block
 * cluster with a cluster barrier as node boundary (NUNA_CHAIN_PERSISTENT; one-shot nodes, at most 8
 * buffer sets, at most 4 MiB per rank, else NUNA_ERR_INVALID_ARG), or always as a CUDA graph of one kernel
 * per node (NUNA_CHAIN_GRAPH).  With neither bit the library picks by measurement, which on B200 means the
 * graph at every size: the single kernel's node (two dependent memory round trips on one cluster's SMs)
 * costs 1.45 us at 16 KiB per rank against 1.08 us for a graph node launched behind its predecessor.    */
#define NUNA_CHAIN_PERSISTENT 2048u
#define NUNA_CHAIN_GRAPH      4096u
/* `flags`, bit 13, flag-synchronised two-shot only: publish and poll the ready flags with system-scope
 * release / acquire (st.release.sys / ld.acquire.sys) instead of device scope.  On one GPU the result and
 * the algorithm are the same; this is the form the synchronisation takes when the rank buffers, the shard
 * and the flags live in peer GPUs' memory (plain loads and stores through peer-mapped pointers).  Not tested
 * across GPUs.                                                                                          */
#define NUNA_TWOSHOT_SYS_SCOPE 8192u
/* `flags`, bit 14, with NUNA_PLACE_AWARE on nuna_allreduce_oneshot: the co-located group sharing the tile
 * through registers.  The work items of C destinations (NUNA_OPT_COLOC: 2, 4 or 8) of one tile run in the
 * same threads: a thread loads its vector of all N sources once and then does, for each of the C emulated
 * ranks in turn, that rank's own rank-ordered fold and its store.                                        */
#define NUNA_PLACE_REGS       16384u

/* ---- topology probe --------------------------------------------------------------------------------
 * Result of nuna_probe_topology: caller-owned, plain data, fixed maximum sizes.  Latencies are in SM
 * clock cycles per dependent load.  Entries for SMs that did not report are zero.                      */
#define NUNA_MAX_SMS          256
#define NUNA_MAX_PROBE_BUFS   32
#define NUNA_PROBE_REGIONS    8
#define NUNA_MAX_PROBE_LINES  2048
#define NUNA_TOPO_UNIFORM     0
#define NUNA_TOPO_NONUNIFORM  1
#define NUNA_HIST_BINS        48
#define NUNA_HIST_FIRST       200
#define NUNA_HIST_STEP        4
#define NUNA_SCAN_LINES       512   /* consecutive 128-byte lines of buffer 0 whose home domain is mapped      */
#define NUNA_SCAN_RUN_BINS    16    /* run-length histogram: bin b = runs of 2^b .. 2^(b+1)-1 lines               */
#define NUNA_SCAN_LEVELS      3     /* granularities of the home-share table: 4 KiB, 64 KiB, 2 MiB             */
#define NUNA_SCAN_BLOCKS      8     /* consecutive blocks of each granularity, from the start of buffer 0       */

typedef struct nuna_topology {
    int num_sms;                     /* cudaDeviceProp.multiProcessorCount                                 */
    int sms_reported;                /* SMs that ran a probe block (one block per SM is requested)         */
    int num_bufs, num_regions;       /* buffers probed; each is cut into num_regions equal regions         */
    int num_lines;                   /* 128-byte lines sampled in total                                    */
    int num_domains;                 /* 1 = uniform; 2 = the SMs split into a near and a far side           */
    int verdict;                     /* NUNA_TOPO_UNIFORM / NUNA_TOPO_NONUNIFORM                           */
    int chain_nodes, chain_steps;    /* miss walk: nodes of the single-cycle permutation, steps per SM     */
    int chain_walk_ok;               /* 1 if every SM's device walk ended on the node the host walk predicts */
    int self_pointer_mismatches;     /* hit walk sanity: loads that did not return the line's own address   */
    float nonuniformity;             /* (max - min) / min of the per-SM mean hit latencies                  */
    float noise;                     /* median |repetition 0 - repetition 1| over all (SM, line) pairs      */
    float near_lat, far_lat;         /* mean hit latency to lines at home in the SM's own / other domain    */
    float domain_gap;                /* far_lat - near_lat                                                   */
    int sm_reported[NUNA_MAX_SMS];
    int sm_domain[NUNA_MAX_SMS];     /* 0 or 1; SM 0's side is domain 0; all 0 when uniform                  */
    float sm_lat_hit[NUNA_MAX_SMS];  /* mean L2-hit latency of this SM over all sampled lines               */
    float sm_lat_miss[NUNA_MAX_SMS]; /* mean latency of this SM's cold (DRAM) walk                           */
    float lat_hit[NUNA_MAX_SMS][NUNA_MAX_PROBE_BUFS];               /* mean hit latency, SM x buffer          */
    float region_home0[NUNA_MAX_PROBE_BUFS][NUNA_PROBE_REGIONS];    /* share of the region's sampled lines
                                                                       that domain 0 reaches faster; -1 none */
    unsigned char line_buf[NUNA_MAX_PROBE_LINES];                   /* per sampled line: buffer, region,      */
    unsigned char line_region[NUNA_MAX_PROBE_LINES];                /* and the domain that reaches it faster  */
    unsigned char line_home[NUNA_MAX_PROBE_LINES];
    /* Histograms of the per-(SM, line) hit latencies: bin b counts latencies in
     * [NUNA_HIST_FIRST + b*NUNA_HIST_STEP, +NUNA_HIST_STEP) cycles; the last bin also takes everything above.
     * hist_near: line at home in the SM's own domain; hist_far: in the other one (all pairs go to hist_near
     * when the verdict is uniform).  The analogue of the paper's per-access latency distributions
     * (Section 6.2).                                                                                     */
    unsigned hist_near[NUNA_HIST_BINS];
    unsigned hist_far[NUNA_HIST_BINS];
    /* At which granularity does the home domain of an address change (Section 3.2: latency depends on the
     * target address)?  scan_home[i] is the home domain of the i-th of scan_lines CONSECUTIVE 128-byte
     * lines of buffer 0 (from its first 128-byte boundary); scan_run_hist counts the runs of equal home
     * among them by length (power-of-two bins), scan_longest_run is the longest.  scan_level_share[g][b] is the share of 16
     * sampled lines at home in domain 0 inside the b-th consecutive block of 4 KiB (g = 0), 64 KiB (1) or
     * 2 MiB (2) of buffer 0, -1 where buffer 0 is too short; scan_level_spread[g] = max - min over the
     * blocks of that granularity (-1 with fewer than two blocks).  A spread near zero with shares near one
     * half means the address hash is finer than that granularity: no block of that size is "near" a domain.
     * All zero / -1 when the verdict is uniform.                                                          */
    int scan_lines;
    int scan_longest_run;
    unsigned char scan_home[NUNA_SCAN_LINES];
    unsigned scan_run_hist[NUNA_SCAN_RUN_BINS];
    float scan_level_share[NUNA_SCAN_LEVELS][NUNA_SCAN_BLOCKS];
    float scan_level_spread[NUNA_SCAN_LEVELS];
    /* Streaming read rate of each SM on its own, GB/s: one block of 256 threads on that SM (every other SM
     * idle) reads a 1 MiB L2-resident window four times with 16-byte L2-only loads.  Zero for SMs that did
     * not report.                                                                                          */
    float sm_read_gbs[NUNA_MAX_SMS];
} nuna_topology_t;

/* Measures, for every SM (indexed by %smid) and every buffer, the latency of dependent L2-only loads
 * to sampled lines of the caller's buffers (the analogue of the paper's per-compute-unit, per-address
 * remote-access sweep, Section 3.2), plus each SM's cold DRAM latency, clusters the SMs into domains
 * maps the home domain of a window of consecutive lines and of blocks of 4 KiB / 64 KiB / 2 MiB of buffer 0,
 * measures each SM's solo streaming read rate,
 * and stores the result in *out and in the device context (where NUNA_PLACE_SM_LISTS plans read it).
 * bufs: HOST array of nbufs (<= NUNA_MAX_PROBE_BUFS) device pointers, bytes[b] >= 128 each, 16-byte
 * aligned.  One 8-byte word per sampled line (about 3000 lines at most) is overwritten during the measurement and restored
 * before return; the buffers must not be in use by other work meanwhile.  Synchronises `stream`,
 * allocates temporary device memory (about 2.3 x the L2 size): NUNA_ERR_CAPTURING on a capturing
 * stream.  Work lists planned earlier for NUNA_PLACE_SM_LISTS are retired and rebuilt under the new
 * topology on the next call of each shape; chains created earlier keep using the lists they captured.
 * Latency values are hardware facts and carry no parity claim.                                        */
int nuna_probe_topology(const void* const* bufs, const size_t* bytes, int nbufs,
                        nuna_topology_t* out, void* stream);

/* ---- placement planner (host only; no CUDA call) ----------------------------------------------------
 * The paper's Algorithm 1 (Section 4.2): logical allocation of thread blocks and the chunks they touch
 * into groups, groups dealt round-robin to nar_max domains, then per block the first compute unit of
 * its domain with budget left and a memory stack near it.  Chunks -- the paper's
 * (chunk_id, buffer_type, gpu_id) tuples -- are numbered 0..num_chunks-1 by the caller.
 * Conventions where the text leaves a choice: first group -> domain 0; a block joins the group owning
 * most of its chunks, ties to the group created first; owned chunks stay where they are; groups sorted
 * by decreasing chunk bytes, stable; no CU with budget -> the CU of the domain with most budget left;
 * stack preference = the CU's nearest stack, then the others in increasing index; a chunk keeps the
 * first stack it was given.  Budgets are counted per (gpu, CU) and per (gpu, stack), in bytes.          */
typedef struct nuna_plan_input {
    int num_tbs;                 /* |W|                                                                    */
    const int* tb_gpu;           /* [num_tbs] gpu of each thread block                                      */
    const int* tb_chunk_begin;   /* [num_tbs + 1] CSR offsets into tb_chunks                                */
    const int* tb_chunks;        /* chunk ids touched by each block (C_tb)                                  */
    int num_chunks;
    const long long* chunk_bytes;/* [num_chunks]                                                            */
    int num_cus;
    const int* cu_domain;        /* [num_cus] domain of each compute unit, 0..nar_max-1                     */
    const int* cu_rank;          /* [num_cus] preference inside the domain, lower = nearer (ties: CU index) */
    int num_stacks;
    const int* cu_stack;         /* [num_cus] nearest memory stack                                          */
    long long r_max_cu;          /* budget per compute unit, bytes                                          */
    long long r_max_stack;       /* budget per memory stack, bytes                                          */
    int nar_max;                 /* number of domains                                                       */
} nuna_plan_input_t;

/* Outputs, caller-allocated: m_compute[num_tbs] (CU per block); optional (may be NULL):
 * m_memory[num_chunks] (stack per chunk, -1 if untouched), tb_domain[num_tbs], tb_group[num_tbs]
 * (index of the block's group in placement order).  Returns NUNA_ERR_INVALID_ARG on malformed input.   */
int nuna_plan_placement(const nuna_plan_input_t* in, int* m_compute, int* m_memory, int* tb_domain, int* tb_group);

/* Create the calling thread's current device's context (flag-barrier words, status word, work cursors,
 * two-shot shard scratch of `scratch_bytes`).  Called implicitly by the first collective on a device;
 * call it explicitly before stream capture, because it allocates.  Growing the scratch later also
 * allocates.  Returns NUNA_ERR_CUDA if no device is usable.                                            */
int nuna_init(size_t scratch_bytes);

/* Tuning knobs of the current device's context (also read once from the environment variables of the
 * same names, NUNA_BLOCKS etc., when the context is created).  value 0 restores the default.
 *  NUNA_OPT_BLOCKS          cap on the grid size of every kernel (the paper's "number of thread blocks",
 *                           Section 6.5: few blocks vs many)
 *  NUNA_OPT_UNROLL          vectors per thread per work item (1, 2, 4; limited so that N * unroll <= 16)
 *  NUNA_OPT_COLOC           destinations of a tile that share a block (co-located group, work lists) or a thread
 *                           (NUNA_PLACE_REGS; also 16 beyond 8 ranks) in the placement-aware one-shot (2, 4, 8; 0 = by rank count and hint)
 *  NUNA_OPT_AUTO_MIN_BYTES  NUNA_PLACE_AUTO never picks a placement-aware kernel below this many bytes per rank
 *                           (on top of its measured crossover)
 *  NUNA_OPT_TIMEOUT_MS      limit of every in-kernel wait (ready flags, barrier, bulk-copy completion)
 *  NUNA_OPT_DOMAINS         number of SM domains the NUNA_PLACE_SM_LISTS planner deals groups to (the paper's
 *                           sweep over routing domains, Section 6.5): 1 = one domain, 2 = the probed split,
 *                           more = every probed domain cut into equal latency quantiles; 0 = what the probe found
 *  NUNA_OPT_STAGE_VECS      16-byte vectors per source per tile of the NUNA_PLACE_STAGED kernel (0 = by size)
 *  NUNA_OPT_TWOSHOT_VECS    16-byte vectors per tile (= per ready flag) of the flag-synchronised two-shot (0 = by size)
 *  NUNA_OPT_AG_BULK_VECS    0 (default): nuna_allgather uses 16-byte loads and stores on small tiles up to 128 MiB of
 *                           output and, like nuna_alltoall at every size, the bulk-copy engine beyond (one bulk load
 *                           into shared memory, one bulk store per destination; tile size by message size);
 *                           >= 8: the bulk-copy form with tiles of that many 16-byte vectors; 1: the register form
 *                           with full tiles (16-byte loads and stores by every thread)
 *  NUNA_OPT_REGS_VECS       16-byte vectors per source per tile of the NUNA_PLACE_REGS kernel (8 ... 256; 0 = by size)
 *  NUNA_OPT_PREFETCH        1: kernels launched with NUNA_LAUNCH_PDL do not ask L2 for their first tile ahead of the
 *                           wait for their predecessor (0 = they do, unless NUNA_HINT_RESIDENT is given); a
 *                           measurement aid, the prefetch changes no result
 * Returns NUNA_ERR_INVALID_ARG for an unknown option or a negative value.  Creates the context.          */
enum { NUNA_OPT_BLOCKS = 0, NUNA_OPT_UNROLL = 1, NUNA_OPT_COLOC = 2, NUNA_OPT_AUTO_MIN_BYTES = 3, NUNA_OPT_TIMEOUT_MS = 4,
       NUNA_OPT_DOMAINS = 5, NUNA_OPT_STAGE_VECS = 6, NUNA_OPT_TWOSHOT_VECS = 7,
       NUNA_OPT_AG_BULK_VECS = 8, NUNA_OPT_REGS_VECS = 9, NUNA_OPT_PREFETCH = 10 };
int nuna_set_option(int option, long long value);

/* One-shot allreduce (Section 5.1, direct algorithm): every emulated rank d reads all N sources and
 * writes dst[d].  src[r], dst[d]: `count` elements each.  Work item = (tile, destination rank).       */
int nuna_allreduce_oneshot(const void* const* src, void* const* dst, int nranks,
                           size_t count, int dtype, unsigned flags, void* stream);

/* Two-shot allreduce: reduce-scatter over N contiguous chunks (the chunk a tile lies in names the emulated
 * rank that reduces it), per-tile ready flags in place of a host synchronisation, then a put-style
 * allgather of the reduced tiles into every destination -- all in one kernel.  Every thread block takes one
 * work item, numbered by a ticket drawn from a device counter: it reduces one tile into the shard scratch
 * and publishes the tile's flag with a release store, and it gathers an earlier tile into all destinations
 * after acquire-polling that tile's flag (bounded wait: on expiry NUNA_ERR_TIMEOUT is latched and the block
 * returns).  A wait is only ever for an item with a smaller ticket, held by a block that already runs, so
 * the kernel needs no co-residency guarantee and no cooperative launch.  Consumed shard lines are dropped
 * from L2 (discard) instead of being written back.  Same bits as the one-shot.  Any `count`; chunk =
 * ceil(count/N) rounded up to a whole 16-byte vector, trailing chunks may be short or empty.  Uses the
 * context's shard scratch (count*elemsize bytes plus one flag word per 256 bytes, grown on demand; an
 * outgrown scratch stays allocated until nuna_shutdown because captured graphs may still name it) unless
 * NUNA_TWOSHOT_PUT is set.  Calls that share the context must be stream-ordered with respect to each other. */
int nuna_allreduce_twoshot(const void* const* src, void* const* dst, int nranks,
                           size_t count, int dtype, unsigned flags, void* stream);

/* Allreduce with the algorithm chosen by message size -- the counterpart of the paper's per-collective
 * choice between routing schemes by a size threshold (Section 4.1.2): one-shot while the message is small
 * enough for its single step to win (measured: up to 1 MiB per rank at 2 ranks, 512 KiB at 4, 128 KiB at
 * 8, 64 KiB at 16; under NUNA_PLACE_AUTO, whose one-shot kernel shares each tile's loads between the
 * destinations, 8 MiB of sources in total with NUNA_LAUNCH_PDL, without it 2 MiB (512 KiB beyond 8 ranks);
 * and again from 8 MiB per rank at 8 ranks or fewer, cold), beyond that the put form of the two-shot.
 * With NUNA_TWOSHOT_SYNC the large-message choice is the flag-synchronised two-shot instead, from eight
 * times those sizes (below, the one-shot is faster than it).  Same bits whichever is chosen.            */
int nuna_allreduce(const void* const* src, void* const* dst, int nranks,
                   size_t count, int dtype, unsigned flags, void* stream);

/* Reduce-scatter: src[k] holds nranks*shard_count elements, dst[r] holds shard_count elements;
 * dst[r][j] = fold over k of src[k][r*shard_count + j].                                               */
int nuna_reduce_scatter(const void* const* src, void* const* dst, int nranks,
                        size_t shard_count, int dtype, unsigned flags, void* stream);

/* Allgather in the paper's form (Figure "Allocation_Diagram": local load, remote store): src[r] holds
 * shard_count elements, every dst[d] holds nranks*shard_count; dst[d][r*shard_count + j] = src[r][j],
 * copied bit for bit.                                                                                   */
int nuna_allgather(const void* const* src, void* const* dst, int nranks,
                   size_t shard_count, int dtype, unsigned flags, void* stream);

/* Alltoall (Section 2.1: expert token routing, the paper's third collective): src[r] holds nranks blocks
 * of block_count elements, block d being what rank r sends to rank d; dst[d] holds nranks blocks, block
 * r being what it received from rank r: dst[d][r*block_count + i] = src[r][d*block_count + i], copied
 * bit for bit.  Placement bits of `flags` are accepted and ignored (every block is touched once).      */
int nuna_alltoall(const void* const* src, void* const* dst, int nranks,
                  size_t block_count, int dtype, unsigned flags, void* stream);

/* Two-shot allreduce for callers that must not allocate device memory.  (The paper has no counterpart:
 * this is a deployment convenience of the library.)  Some hosts of this code cannot call cudaMalloc
 * on the request path: an inference server that has handed the whole GPU to its own memory pool, where
 * a raw allocation can fail or fragment the pool, or a latency-critical loop that cannot afford the
 * device-wide synchronisation and the failure modes an allocation brings.  This entry point computes
 * exactly what nuna_allreduce_twoshot computes (flag-synchronised form, same bits) but takes its shard
 * intermediate, ready flags and control words from fixed arrays compiled into the library, so it never calls
 * cudaMalloc, cudaFree or any allocating routine, and it does not create the per-device context.
 *  - Limit: 4 MiB per rank, i.e. count <= NUNA_STATIC_MAX_COUNT elements of a 16-bit type (half that
 *    many of binary32); larger messages return NUNA_ERR_TOO_LARGE and print the limit.  The array
 *    costs 4 MiB of device memory on every GPU that loads the library, for the life of the process.
 *  - The first call on a device looks up the arrays' device addresses and zeroes the flags and control
 *    words (two small synchronous cudaMemset calls); make that first call before starting any stream capture.
 *  - All calls on a device share the one array, which keeps the previous call's shard; the kernel
 *    overwrites every element it later reads, so stale contents never reach a result.  Two calls that
 *    overlap on the GPU (different streams, no ordering) race on it: keep calls stream-ordered.
 *  - A wait that times out (1 s) latches NUNA_ERR_TIMEOUT in the arrays' own status word; results are
 *    then undefined.  nuna_device_status reports that word too (the worse of it and the context's) and
 *    rewinds the control words after a timeout.  src / dst / nranks / dtype / stream and the argument
 *    errors are those of nuna_allreduce_twoshot; there is no flags word.                               */
#define NUNA_STATIC_MAX_COUNT (2 * 1024 * 1024)
int nuna_allreduce_twoshot_static(const void* const* src, void* const* dst, int nranks,
                                  size_t count, int dtype, void* stream);

/* End-to-end variant with HOST buffers: src[r] / dst[d] are HOST pointers to `count` elements (pinned
 * or pageable).  Copies the sources to library-owned device staging buffers, runs the one-shot
 * (two_shot == 0) or two-shot allreduce, copies every destination back and synchronises.  Allocates
 * staging on first use or growth.  With two_shot != 0 and NUNA_TWOSHOT_PUT, and every buffer page-locked
 * (cudaHostAlloc / cudaHostRegister) and 16-byte aligned, the kernel works on the host buffers in place
 * instead: every byte crosses the host link once, in both directions at the same time, with no copies.   */
int nuna_allreduce_host(const void* const* src, void* const* dst, int nranks,
                        size_t count, int dtype, unsigned flags, int two_shot);

/* Decode-step chain: `nnodes` back-to-back allreduces (two per transformer layer) captured once into a
 * CUDA graph and replayed with a single launch.  src_sets / dst_sets are HOST arrays of nsets*nranks
 * device pointers, set s occupying entries [s*nranks, (s+1)*nranks); node k works on set k mod nsets
 * and starts reading only after node k-1 has finished writing.  flags as for the allreduce calls
 * (NUNA_LAUNCH_PDL overlaps each node's launch with its predecessor's drain); two_shot selects
 * nuna_allreduce_twoshot.  One-shot nodes can also run as a single kernel instead of a graph (see
 * NUNA_CHAIN_PERSISTENT / NUNA_CHAIN_GRAPH): one thread-block cluster loops over the nodes with a cluster
 * barrier between them, which removes the per-node launch.  Creation allocates and synchronises
 * nothing on the caller's streams; the chain reads the buffers named at creation on every launch.
 * *chain_out is an opaque handle.                                                                       */
int nuna_chain_create(const void* const* src_sets, void* const* dst_sets, int nsets, int nnodes, int nranks,
                      size_t count, int dtype, unsigned flags, int two_shot, void** chain_out);
int nuna_chain_launch(void* chain, void* stream);      /* one replay of all nodes, asynchronous on `stream` */
int nuna_chain_destroy(void* chain);

/* Reads and clears the device status of the current device (NUNA_OK or NUNA_ERR_TIMEOUT) after
 * synchronising the device: the worse of the context's status word and the allocation-free entry
 * point's.  After a timeout the control words are rewound (the epoch keeps counting).                  */
int nuna_device_status(int* out);

/* Launches an empty kernel of `blocks` thread blocks with the collectives' block shape on `stream`: the
 * single-kernel-launch floor that small-message latencies are reported against.  flags: 0 or
 * NUNA_LAUNCH_PDL.                                                                                      */
int nuna_launch_floor(unsigned blocks, unsigned flags, void* stream);

/* Number of kernels this library has launched on any device since load (the callers' launch count).   */
unsigned long long nuna_launch_count(void);

const char* nuna_status_string(int status);

/* Frees the current device's context (scratch, staging, graphs are NOT freed: destroy chains first).  */
int nuna_shutdown(void);

#ifdef __cplusplus
}
#endif
#endif /* NUNA_H */
