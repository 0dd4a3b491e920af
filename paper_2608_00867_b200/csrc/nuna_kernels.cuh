// Device code of the emulated-rank collectives (sm_100a).
//
// Two families of kernels.  Register kernels: all data movement is 16-byte
// vectorised and coalesced, one thread moves one uint4 (8 bf16) per source per
// step, a warp covers 512 contiguous bytes of every buffer it touches; a thread
// first issues the loads of all N sources (N independent 16-byte requests in
// flight per thread give the memory-level parallelism), then folds them in rank
// order in binary32 and rounds once.  Bulk-copy kernels: one thread of a block
// issues one-dimensional cp.async.bulk copies (plain form: this GPU's memory,
// no multicast) that bring a tile's slices into shared memory and complete on an
// mbarrier; the bytes in flight hold no registers, and pure copies (allgather,
// alltoall) leave shared memory again by bulk stores.  Every wait in this file
// (ready flag, barrier, copy completion) is bounded and ends in a latched status,
// never in a trap or an endless spin.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "nuna_types.h"

namespace nuna {


// Blocks per SM the compiler is asked to keep resident for a kernel that holds `vectors` 16-byte
// loads in flight per thread.  Stating it makes ptxas spend registers on keeping ALL of a thread's
// loads outstanding at once (4 registers per vector plus about 20) instead of batching them to
// stay at 32 registers, which would expose two to four memory round trips per item.
constexpr int min_blocks(int vectors)
{
    const int regs = 4 * vectors + 20;
    const int b = 65536 / (kThreads * regs);
    return b < 1 ? 1 : (b > 8 ? 8 : b);
}


// ---- programmatic dependent launch ---------------------------------------------------------------
//
// Every collective kernel opens with pdl_wait() and calls pdl_trigger() when its block has issued
// its main work.  When a kernel is launched with programmatic stream serialization
// (NUNA_LAUNCH_PDL) its blocks may be scheduled while the predecessor in the stream drains:
// griddepcontrol.wait holds them, before their first global access, until the predecessor grid has
// completed and its memory operations are visible; griddepcontrol.launch_dependents, issued once a
// block is past its main loop, lets the successor's blocks take the freed SM slots so that their
// launch latency overlaps this kernel's tail.  (Triggering at kernel entry, or as soon as a block has
// issued its loads, was measured slower -- 8 x 512 KiB one-shot: 3.07 against 2.81 us -- the successor's
// waiting blocks then compete with this kernel's own blocks for slots.)
// Launched normally, both instructions do nothing.
__device__ __forceinline__ void pdl_wait()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

__device__ __forceinline__ void pdl_trigger()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// Asks L2 to fetch `bytes` (a multiple of 16; 16-byte aligned address) of this GPU's memory.  Nothing is
// returned to the thread and nothing is waited for, so it may be issued BEFORE pdl_wait(): L2 is the
// point of coherence, a line the predecessor writes after the fetch is updated in place, and the loads
// after the wait read the current data.  What it buys: the successor's blocks arrive while the
// predecessor's last blocks drain and its writes are flushed; that window covers most of a DRAM round
// trip, so cold sources are L2 hits by the time the wait returns.
__device__ __forceinline__ void prefetch_l2_bulk(const void* g, unsigned bytes)
{
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" :: "l"(g), "r"(bytes) : "memory");
}

// Nanoseconds of the device-wide timer (bounds every in-kernel wait; timestamps of the measurement aids).
__device__ __forceinline__ unsigned long long globaltimer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// ---- memory access helpers ----------------------------------------------------------------

// Sources are read-only for the duration of a kernel and are re-read by other
// emulated ranks from other SMs: keep them out of L1, let L2 hold them.
__device__ __forceinline__ uint4 ld_src(const uint4* p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// Data produced earlier in the same kernel by other blocks (two-shot shard): coherent L2 load.
__device__ __forceinline__ uint4 ld_cg(const uint4* p)
{
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}

// Destination of a streaming kernel: written once and not read again by this kernel, so it is stored
// with the evict-first policy and does not push the sources out of L2 (measured: two-shot put
// 164.1 -> 160.9 us at 64 MiB per rank, 12.06 -> 11.68 us at 4 MiB; one-shot 234.7 -> 225.8 us).
__device__ __forceinline__ void st_stream(uint4* p, uint4 v)
{
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// Ordinary store: data another block of this kernel reads back (the two-shot shard) and the destinations
// of the placement-aware kernels, which are used when the buffers are meant to stay in L2.
__device__ __forceinline__ void st_dst(uint4* p, uint4 v)
{
    asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

__device__ __forceinline__ uint16_t ld_src16(const uint16_t* p)
{
    uint16_t v;
    asm volatile("ld.global.nc.u16 %0, [%1];" : "=h"(v) : "l"(p));
    return v;
}

// ---- the fold ------------------------------------------------------------------------------

// Element types (the values of nuna_dtype_t): 0 = bf16, 1 = f16 (IEEE binary16), 2 = f32.
// Storage is 2 or 4 bytes; a 16-byte vector holds kElems elements; every type is widened exactly
// to binary32, folded in binary32 in rank order, and rounded once to the storage type.
constexpr int kBf16 = 0, kF16 = 1, kF32 = 2;

template <int DT> struct Elem { static constexpr int kElems = 8; static constexpr int kBytes = 2; };
template <> struct Elem<kF32> { static constexpr int kElems = 4; static constexpr int kBytes = 4; };

// bf16 -> binary32 is a 16-bit shift; a 32-bit word holds element 2k in its low half and 2k+1 in
// its high half.  Rank 0's value is widened (shift / mask for bf16, cvt for f16); ranks 1..N-1 are
// folded in with the sm_100 mixed-precision add, d = f32(a) + c rounded once to binary32 (nearest
// even, subnormals kept), so no instruction is spent on widening them.  At large sizes the one-shot is
// limited by instruction issue and L1 throughput (N times the work of a plain sum), which is why the
// instruction count matters.
template <int DT>
__device__ __forceinline__ float add_narrow(float acc, uint16_t h)
{
    float d;
    if (DT == kBf16) asm("add.rn.f32.bf16 %0, %1, %2;" : "=f"(d) : "h"(h), "f"(acc));
    else             asm("add.rn.f32.f16 %0, %1, %2;" : "=f"(d) : "h"(h), "f"(acc));
    return d;
}

template <int DT>
__device__ __forceinline__ void widen_word(float& lo, float& hi, uint32_t w)
{
    if (DT == kBf16) {
        lo = __uint_as_float(w << 16);
        hi = __uint_as_float(w & 0xFFFF0000u);
    } else {
        uint16_t l, h;
        asm("mov.b32 {%0, %1}, %2;" : "=h"(l), "=h"(h) : "r"(w));
        asm("cvt.f32.f16 %0, %1;" : "=f"(lo) : "h"(l));
        asm("cvt.f32.f16 %0, %1;" : "=f"(hi) : "h"(h));
    }
}

template <int DT>
__device__ __forceinline__ void fold_word(float& lo, float& hi, uint32_t w)
{
    uint16_t l, h;
    asm("mov.b32 {%0, %1}, %2;" : "=h"(l), "=h"(h) : "r"(w));
    lo = add_narrow<DT>(lo, l);
    hi = add_narrow<DT>(hi, h);
}

// Two binary32 -> one word of two 16-bit elements, round to nearest even, NaN -> 0x7FFF.
template <int DT>
__device__ __forceinline__ uint32_t pack2(float lo, float hi)
{
    uint32_t d;
    if (DT == kBf16) asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    else             asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

// Fold N already-loaded vectors in rank order: acc starts from rank 0's value, N-1 additions.
template <int N, int DT>
__device__ __forceinline__ uint4 fold_vectors(const uint4 (&v)[N])
{
    if (DT == kF32) {
        float a0 = __uint_as_float(v[0].x), a1 = __uint_as_float(v[0].y);
        float a2 = __uint_as_float(v[0].z), a3 = __uint_as_float(v[0].w);
#pragma unroll
        for (int r = 1; r < N; ++r) {
            a0 = __fadd_rn(a0, __uint_as_float(v[r].x));
            a1 = __fadd_rn(a1, __uint_as_float(v[r].y));
            a2 = __fadd_rn(a2, __uint_as_float(v[r].z));
            a3 = __fadd_rn(a3, __uint_as_float(v[r].w));
        }
        return make_uint4(__float_as_uint(a0), __float_as_uint(a1), __float_as_uint(a2), __float_as_uint(a3));
    }
    float a[8];
    widen_word<DT>(a[0], a[1], v[0].x);
    widen_word<DT>(a[2], a[3], v[0].y);
    widen_word<DT>(a[4], a[5], v[0].z);
    widen_word<DT>(a[6], a[7], v[0].w);
#pragma unroll
    for (int r = 1; r < N; ++r) {
        fold_word<DT>(a[0], a[1], v[r].x);
        fold_word<DT>(a[2], a[3], v[r].y);
        fold_word<DT>(a[4], a[5], v[r].z);
        fold_word<DT>(a[6], a[7], v[r].w);
    }
    return make_uint4(pack2<DT>(a[0], a[1]), pack2<DT>(a[2], a[3]), pack2<DT>(a[4], a[5]), pack2<DT>(a[6], a[7]));
}

// One element (ragged tails and unaligned shards): returns the storage word of the folded value.
template <int N, int DT>
__device__ __forceinline__ uint32_t fold_scalar(const RankPtrs& p, size_t elem)
{
    if (DT == kF32) {
        float acc = __uint_as_float(__ldg(reinterpret_cast<const uint32_t*>(p.src[0]) + elem));
#pragma unroll
        for (int r = 1; r < N; ++r)
            acc = __fadd_rn(acc, __uint_as_float(__ldg(reinterpret_cast<const uint32_t*>(p.src[r]) + elem)));
        return __float_as_uint(acc);
    }
    float acc, unused;
    widen_word<DT>(acc, unused, (uint32_t)ld_src16(reinterpret_cast<const uint16_t*>(p.src[0]) + elem));
#pragma unroll
    for (int r = 1; r < N; ++r)
        acc = add_narrow<DT>(acc, ld_src16(reinterpret_cast<const uint16_t*>(p.src[r]) + elem));
    return pack2<DT>(acc, 0.0f) & 0xFFFFu;
}

template <int DT>
__device__ __forceinline__ void store_elem(void* base, size_t elem, uint32_t word)
{
    if (DT == kF32) reinterpret_cast<uint32_t*>(base)[elem] = word;
    else            reinterpret_cast<uint16_t*>(base)[elem] = (uint16_t)word;
}

// Element written earlier in this kernel by another block: L2-coherent load.
template <int DT>
__device__ __forceinline__ uint32_t load_elem_cg(const void* base, size_t elem)
{
    uint32_t w;
    if (DT == kF32) {
        asm volatile("ld.global.cg.u32 %0, [%1];" : "=r"(w) : "l"(reinterpret_cast<const uint32_t*>(base) + elem) : "memory");
    } else {
        uint16_t v;
        asm volatile("ld.global.cg.u16 %0, [%1];" : "=h"(v) : "l"(reinterpret_cast<const uint16_t*>(base) + elem) : "memory");
        w = v;
    }
    return w;
}

// ---- access-latency sampling (measurement builds of the one-shot kernels only) ----------------------------
//
// The timed variants below are the production loops with two clock reads around a work item's loads: t0
// before the first load is issued, t1 once the first loaded vector can be used (a shared-memory store
// consumes it, and instructions issue in order).  Lane 0 of every warp adds one sample per item to a
// histogram of kLatBins bins of kLatStep cycles (the last bin also takes everything above): the
// distribution of access latencies under a placement (Section 6.2).
constexpr int kLatBins = 64, kLatStep = 32;

__device__ __forceinline__ long long clock_now()
{
    long long t;
    asm volatile("mov.u64 %0, %%clock64;" : "=l"(t) :: "memory");
    return t;
}

__device__ __forceinline__ void latency_sample(unsigned* hist, long long t0, unsigned first_word)
{
    __shared__ unsigned sink[kThreads];
    asm volatile("st.shared.u32 [%0], %1;" :: "r"((unsigned)__cvta_generic_to_shared(&sink[threadIdx.x])), "r"(first_word) : "memory");
    const long long t1 = clock_now();
    if ((threadIdx.x & 31u) == 0u) {
        const long long bin = (t1 - t0) / kLatStep;
        atomicAdd(hist + (bin < 0 ? 0 : bin >= kLatBins ? kLatBins - 1 : (int)bin), 1u);
    }
}

// ---- one-shot allreduce: work item = (tile, destination rank) ---------------------------------
//
// Item i = tile * N + d, destination fastest, so the N emulated ranks that read
// the same source tile are adjacent in the item order.  A tile is
// kThreads * U vectors.  Round-robin placement: item i is taken by block
// i mod gridDim.x (the locality-unaware baseline of Section 5.3).
template <int N, int U, int DT, bool kTimed = false>
__device__ __forceinline__ void oneshot_item(const RankPtrs& p, size_t nvec, size_t tile, int d, unsigned* hist = nullptr)
{
    const size_t base = tile * (size_t)(kThreads * U) + threadIdx.x;
    uint4 v[U][N];
    long long t0 = 0;
    if (kTimed) t0 = clock_now();
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t i = base + (size_t)u * kThreads;
        if (i < nvec) {
#pragma unroll
            for (int r = 0; r < N; ++r) v[u][r] = ld_src(p.src[r] + i);
        }
    }
    if (kTimed && base < nvec) latency_sample(hist, t0, v[0][0].x);
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t i = base + (size_t)u * kThreads;
        if (i < nvec) st_stream(p.dst[d] + i, fold_vectors<N, DT>(v[u]));
    }
}

template <int N, int U, int DT>
__global__ void __launch_bounds__(kThreads, min_blocks(N * U))
k_oneshot_rr(const RankPtrs p, const size_t count, const size_t ntiles)
{
    pdl_wait();
    const size_t nvec = count / Elem<DT>::kElems;
    const size_t nitems = ntiles * N;
    for (size_t item = blockIdx.x; item < nitems; item += gridDim.x)
        oneshot_item<N, U, DT>(p, nvec, item / N, (int)(item % N));
    pdl_trigger();
    // ragged tail (count % 8 elements): block d handles destination d
    const size_t tail0 = nvec * Elem<DT>::kElems;
    if (tail0 < count) {
        for (int d = blockIdx.x; d < N; d += gridDim.x) {
            const size_t e = tail0 + threadIdx.x;
            if (e < count) store_elem<DT>(p.dst[d], e, fold_scalar<N, DT>(p, e));
        }
    }
}

// The round-robin kernel's main loop with latency sampling (whole vectors only; a measurement aid).
template <int N, int DT>
__global__ void __launch_bounds__(kThreads, min_blocks(N))
k_latency_rr(const RankPtrs p, const size_t count, const size_t ntiles, unsigned* hist)
{
    const size_t nvec = count / Elem<DT>::kElems;
    const size_t nitems = ntiles * N;
    for (size_t item = blockIdx.x; item < nitems; item += gridDim.x)
        oneshot_item<N, 1, DT, true>(p, nvec, item / N, (int)(item % N), hist);
}

// ---- one-shot allreduce, co-located groups (placement-aware) ------------------------------------------
//
// Logical allocation (Section 4.2.1) puts the thread blocks that touch the same chunks into
// one group, and physical placement keeps a group on one compute unit.  For the one-shot the N
// work items (tile, d), d = 0..N-1, share all N source tiles, so a group is "one tile, every
// destination".  Here a group runs inside ONE thread block: row d of the block (kThreads / rows
// threads, rows = N rounded up to a power of two) is emulated rank d's work item for that tile.
// Every row still issues its own loads of all N sources and does its own fold, but the rows'
// requests for the same lines meet in that SM's L1, so each source line crosses the L2 -> SM
// fabric once per group instead of once per destination.
__device__ __forceinline__ uint4 ld_src_l1(const uint4* p)
{
    uint4 v;
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// Co-location factor C (a power of two, at most N rounded up to one): a block holds the work items
// of C destinations of one tile, so a tile's group is spread over ceil(N / C) blocks.  This is the
// resource budget of Section 4.2.2 in SM terms: the more items of a group share an SM, the fewer
// distinct bytes that SM has in flight (kThreads / C vectors per source), so cold data wants a small
// C (more outstanding requests per SM) and L2-resident data a large one (fewer L2 -> SM transfers).
template <int N, int C, int DT, bool kTimed = false>
__device__ __forceinline__ void oneshot_group(const RankPtrs& p, size_t nvec, size_t tile, int dst0, unsigned* hist = nullptr)
{
    constexpr int kLanes = kThreads / C;                 // vectors per tile
    const int d = dst0 + threadIdx.x / kLanes;
    const size_t i = tile * kLanes + (threadIdx.x % kLanes);
    if (d < N && i < nvec) {
        uint4 v[N];
        long long t0 = 0;
        if (kTimed) t0 = clock_now();
#pragma unroll
        for (int r = 0; r < N; ++r) v[r] = ld_src_l1(p.src[r] + i);
        if (kTimed) latency_sample(hist, t0, v[0].x);
        st_dst(p.dst[d] + i, fold_vectors<N, DT>(v));
    }
}

// The co-located group kernel's main loop with latency sampling (whole vectors only; a measurement aid).
template <int N, int C, int DT>
__global__ void __launch_bounds__(kThreads, min_blocks(N))
k_latency_group(const RankPtrs p, const size_t count, const size_t ntiles, unsigned* hist)
{
    constexpr int kSplit = (N + C - 1) / C;
    const size_t nvec = count / Elem<DT>::kElems;
    const size_t nitems = ntiles * kSplit;
    for (size_t it = blockIdx.x; it < nitems; it += gridDim.x)
        oneshot_group<N, C, DT, true>(p, nvec, it / kSplit, (int)(it % kSplit) * C, hist);
}

template <int N, int C, int DT>
__global__ void __launch_bounds__(kThreads, min_blocks(N))
k_oneshot_group(const RankPtrs p, const size_t count, const size_t ntiles)
{
    pdl_wait();
    constexpr int kSplit = (N + C - 1) / C;              // blocks per tile group
    const size_t nvec = count / Elem<DT>::kElems;
    const size_t nitems = ntiles * kSplit;
    for (size_t it = blockIdx.x; it < nitems; it += gridDim.x)
        oneshot_group<N, C, DT>(p, nvec, it / kSplit, (int)(it % kSplit) * C);
    pdl_trigger();
    const size_t tail0 = nvec * Elem<DT>::kElems;
    if (tail0 < count) {
        for (int d = blockIdx.x; d < N; d += gridDim.x) {
            const size_t e = tail0 + threadIdx.x;
            if (e < count) store_elem<DT>(p.dst[d], e, fold_scalar<N, DT>(p, e));
        }
    }
}

// ---- one-shot allreduce, co-located group sharing the tile through registers -----------------------------
//
// The tightest co-location of a logical group: the work items (tile, d) of C destinations run in the SAME
// threads.  A thread loads its vector of all N sources once and then performs, for each of the C emulated
// ranks in turn, that rank's own fold in rank order and the store to that rank's destination.  The C folds
// are separate instruction sequences (every addition is an opaque instruction, so the compiler cannot merge
// the ranks' work into one); what the ranks share is the fetched data, as they share it through L1 in
// k_oneshot_group and through shared memory in k_oneshot_stage -- here without a second trip through any
// memory.  Loads and L2 -> SM traffic drop by C, the arithmetic stays N-fold.
template <int DT>
__device__ __forceinline__ float add_narrow_own(float acc, uint16_t h)
{
    float d;
    if (DT == kBf16) asm volatile("add.rn.f32.bf16 %0, %1, %2;" : "=f"(d) : "h"(h), "f"(acc));
    else             asm volatile("add.rn.f32.f16 %0, %1, %2;" : "=f"(d) : "h"(h), "f"(acc));
    return d;
}

__device__ __forceinline__ float add_f32_own(float a, float b)
{
    float d;
    asm volatile("add.rn.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
    return d;
}

template <int DT>
__device__ __forceinline__ void fold_word_own(float& lo, float& hi, uint32_t w)
{
    uint16_t l, h;
    asm("mov.b32 {%0, %1}, %2;" : "=h"(l), "=h"(h) : "r"(w));
    lo = add_narrow_own<DT>(lo, l);
    hi = add_narrow_own<DT>(hi, h);
}

// fold_vectors with additions the compiler must keep per call: same order, same instructions, same bits.
template <int N, int DT>
__device__ __forceinline__ uint4 fold_vectors_own(const uint4 (&v)[N])
{
    if (DT == kF32) {
        float a0 = __uint_as_float(v[0].x), a1 = __uint_as_float(v[0].y);
        float a2 = __uint_as_float(v[0].z), a3 = __uint_as_float(v[0].w);
#pragma unroll
        for (int r = 1; r < N; ++r) {
            a0 = add_f32_own(a0, __uint_as_float(v[r].x));
            a1 = add_f32_own(a1, __uint_as_float(v[r].y));
            a2 = add_f32_own(a2, __uint_as_float(v[r].z));
            a3 = add_f32_own(a3, __uint_as_float(v[r].w));
        }
        return make_uint4(__float_as_uint(a0), __float_as_uint(a1), __float_as_uint(a2), __float_as_uint(a3));
    }
    float a[8];
    widen_word<DT>(a[0], a[1], v[0].x);
    widen_word<DT>(a[2], a[3], v[0].y);
    widen_word<DT>(a[4], a[5], v[0].z);
    widen_word<DT>(a[6], a[7], v[0].w);
#pragma unroll
    for (int r = 1; r < N; ++r) {
        fold_word_own<DT>(a[0], a[1], v[r].x);
        fold_word_own<DT>(a[2], a[3], v[r].y);
        fold_word_own<DT>(a[4], a[5], v[r].z);
        fold_word_own<DT>(a[6], a[7], v[r].w);
    }
    return make_uint4(pack2<DT>(a[0], a[1]), pack2<DT>(a[2], a[3]), pack2<DT>(a[4], a[5]), pack2<DT>(a[6], a[7]));
}

// Work item = (tile of `tv` <= kThreads vectors, group of C destinations); one item per block while the
// grid allows.  The host sizes the tile by the message: a small message is cut into many small tiles
// (every SM gets a few blocks of a few warps each; measured faster than few full blocks at every size
// below 4 MiB per rank), a large one uses full tiles.
// mode bit 0: streaming stores (destinations are not re-read soon); bit 1: every block asks L2 for its
// first tile's source slices before it waits for the predecessor kernel (dependent launches with cold
// sources only: without a predecessor there is nothing to overlap with).
// kTimed (a measurement aid): thread 0 of every block also records, in nanoseconds of the global timer, when the
// block started, when its wait for the predecessor returned and when it had issued its last store, plus the SM
// it ran on: trace[(slot * trace_blocks + blockIdx.x) * 4 + {0, 1, 2, 3}] for blockIdx.x < trace_blocks.
template <int N, int C, int DT, bool kTimed>
__device__ __forceinline__ void oneshot_regs_body(const RankPtrs& p, const size_t count, const size_t ntiles, const unsigned tv,
                                                  const int mode, unsigned long long* trace, const unsigned slot,
                                                  const unsigned trace_blocks)
{
    constexpr int kSplit = (N + C - 1) / C;
    const size_t nvec = count / Elem<DT>::kElems;
    const size_t nitems = ntiles * kSplit;
    unsigned long long t_in = 0, t_wait = 0;
    if (kTimed && threadIdx.x == 0) t_in = globaltimer_ns();
    if ((mode & 2) && blockIdx.x < nitems && threadIdx.x < N) {
        const size_t i0 = ((size_t)blockIdx.x / kSplit) * tv;        // thread r fetches source r's slice
        const uint4* a = p.src[0];
#pragma unroll
        for (int r = 1; r < N; ++r) if ((int)threadIdx.x == r) a = p.src[r];
        if (i0 < nvec) prefetch_l2_bulk(a + i0, (unsigned)(nvec - i0 < (size_t)tv ? nvec - i0 : (size_t)tv) * 16u);
    }
    pdl_wait();
    if (kTimed && threadIdx.x == 0) t_wait = globaltimer_ns();
    const int stream_stores = mode & 1;
    for (size_t item = blockIdx.x; item < nitems; item += gridDim.x) {
        const size_t i = (item / kSplit) * tv + threadIdx.x;
        const int d0 = (int)(item % kSplit) * C;
        if (threadIdx.x < tv && i < nvec) {
            uint4 v[N];
#pragma unroll
            for (int r = 0; r < N; ++r) v[r] = ld_src(p.src[r] + i);
#pragma unroll
            for (int c = 0; c < C; ++c) {
                const int d = d0 + c;
                if (d < N) {
                    const uint4 o = fold_vectors_own<N, DT>(v);
                    if (stream_stores) st_stream(p.dst[d] + i, o); else st_dst(p.dst[d] + i, o);
                }
            }
        }
    }
    pdl_trigger();
    if (kTimed) {
        __syncthreads();                                              // every warp of the block has issued its stores
        if (threadIdx.x == 0 && blockIdx.x < trace_blocks) {
            unsigned sm;
            asm volatile("mov.u32 %0, %%smid;" : "=r"(sm));
            unsigned long long* o = trace + ((size_t)slot * trace_blocks + blockIdx.x) * 4;
            o[0] = t_in; o[1] = t_wait; o[2] = globaltimer_ns(); o[3] = sm;
        }
    }
    const size_t tail0 = nvec * Elem<DT>::kElems;
    if (tail0 < count) {
        for (int d = blockIdx.x; d < N; d += gridDim.x) {
            const size_t e = tail0 + threadIdx.x;
            if (e < count) store_elem<DT>(p.dst[d], e, fold_scalar<N, DT>(p, e));
        }
    }
}

template <int N, int C, int DT>
__global__ void __launch_bounds__(kThreads, min_blocks(N))
k_oneshot_regs(const RankPtrs p, const size_t count, const size_t ntiles, const unsigned tv, const int mode)
{
    oneshot_regs_body<N, C, DT, false>(p, count, ntiles, tv, mode, nullptr, 0u, 0u);
}

template <int N, int C, int DT>
__global__ void __launch_bounds__(kThreads, min_blocks(N))
k_oneshot_regs_timed(const RankPtrs p, const size_t count, const size_t ntiles, const unsigned tv, const int mode,
                     unsigned long long* trace, const unsigned slot, const unsigned trace_blocks)
{
    oneshot_regs_body<N, C, DT, true>(p, count, ntiles, tv, mode, trace, slot, trace_blocks);
}

// ---- one-shot allreduce, co-located group staged through shared memory ---------------------------------
//
// The same logical group as above (one tile, every destination, on one compute unit), but the N
// source slices of the tile are fetched ONCE per block by the bulk-copy engine: one elected thread
// issues N one-dimensional cp.async.bulk copies global -> shared (plain form, this GPU's memory, no
// multicast) that complete on an mbarrier; all N * tile bytes of a block are in flight at once without
// holding a register.  Row d of the block (emulated rank d) then folds the N slices out of shared
// memory in rank order and stores its destination.  Each emulated rank still reads all N sources and
// does its own fold; what changes is where the N-fold re-read is served from (shared memory instead
// of L1 / L2), so the L2 -> SM fabric carries every source byte once per tile.
// One tile per block: the hardware block scheduler balances, and several resident blocks per SM
// overlap one block's copy latency with another's fold.
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned arrivals)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(bar)), "r"(arrivals) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");   // visible to the bulk-copy engine
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(smem_u32(bar)), "r"(bytes) : "memory");
}

// Bulk copy of `bytes` (a multiple of 16; both addresses 16-byte aligned) from global to this block's shared memory.
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, unsigned bytes, uint64_t* bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, unsigned parity)
{
    unsigned done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return done != 0;
}

// Bounded wait for phase `parity` of an mbarrier: after timeout_ns the thread latches NUNA_ERR_TIMEOUT in
// *status and gives up (the caller skips its work and returns; nothing traps).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, unsigned parity, unsigned* status, unsigned long long timeout_ns)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = globaltimer_ns();
    unsigned polls = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++polls & 255u) == 0u && globaltimer_ns() - t0 > timeout_ns) {
            atomicMax(status, 6u);                     // NUNA_ERR_TIMEOUT
            return false;
        }
    }
    return true;
}

__device__ __forceinline__ uint4 ld_shared_v4(const uint4* p)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(smem_u32(p)));
    return v;
}

__host__ __device__ constexpr int pow2_at_least(int n) { return n <= 1 ? 1 : n <= 2 ? 2 : n <= 4 ? 4 : n <= 8 ? 8 : 16; }

// tv = vectors per source per tile (a multiple of kThreads / rows); shared memory = N * tv * 16 bytes.
// (Filling the tile with ordinary 16-byte loads parked in shared memory instead of bulk copies was
// measured too: never faster, and the registers that hold the loads in flight cost resident blocks.)
template <int N, int DT>
__global__ void __launch_bounds__(kThreads)
k_oneshot_stage(const RankPtrs p, const size_t count, const unsigned tv, const int stream_stores,
                unsigned* status, const unsigned long long timeout_ns)
{
    constexpr int kRows = pow2_at_least(N);
    constexpr int kLanes = kThreads / kRows;
    extern __shared__ __align__(128) unsigned char stage_raw[];
    uint4* stage = reinterpret_cast<uint4*>(stage_raw);            // [N][tv]
    __shared__ __align__(8) uint64_t bar;
    const size_t nvec = count / Elem<DT>::kElems;
    const size_t base = (size_t)blockIdx.x * tv;
    const unsigned nv = base < nvec ? (unsigned)((nvec - base < tv) ? nvec - base : tv) : 0u;
    if (threadIdx.x == 0) mbar_init(&bar, 1u);
    __syncthreads();
    pdl_wait();                                                     // before the first global access
    if (nv != 0u) {
        if (threadIdx.x == 0) {
            mbar_expect_tx(&bar, (unsigned)N * nv * 16u);
#pragma unroll
            for (int r = 0; r < N; ++r) bulk_load(stage + (size_t)r * tv, p.src[r] + base, nv * 16u, &bar);
        }
        if (mbar_wait(&bar, 0u, status, timeout_ns)) {
            const int d = threadIdx.x / kLanes;
            if (d < N) {
                uint4* out = p.dst[d] + base;
                for (unsigned j = threadIdx.x % kLanes; j < nv; j += kLanes) {
                    uint4 v[N];
#pragma unroll
                    for (int r = 0; r < N; ++r) v[r] = ld_shared_v4(stage + (size_t)r * tv + j);
                    const uint4 o = fold_vectors<N, DT>(v);
                    if (stream_stores) st_stream(out + j, o); else st_dst(out + j, o);
                }
            }
        }
    }
    pdl_trigger();
    const size_t tail0 = nvec * Elem<DT>::kElems;
    if (tail0 < count) {
        for (int d = blockIdx.x; d < N; d += gridDim.x) {
            const size_t e = tail0 + threadIdx.x;
            if (e < count) store_elem<DT>(p.dst[d], e, fold_scalar<N, DT>(p, e));
        }
    }
}

// ---- one-shot allreduce, a logical group per thread-block cluster --------------------------------------
//
// The hardware's own locality domain is the GPC: the blocks of a thread-block cluster are placed on
// one GPC and can read each other's shared memory.  Here the N work items (tile, d) of one tile --
// one logical group of Section 4.2.1 -- form one cluster of N blocks.  Block r first loads source
// r's tile, one 16-byte vector per thread, into its shared memory: the cluster as a whole fetches
// every source byte exactly once, with all of its loads in flight at the same time.  After a
// cluster barrier, block d (emulated rank d) reads the N source tiles out of the N blocks' shared
// memories (ld.shared::cluster), folds them in rank order and stores its own destination.  Each
// emulated rank still does its own N reads and its own fold; the reads are served by the
// neighbours' shared memory instead of L2.  Few registers are live, so all groups of a mid-sized
// message are resident at once (no second wave).
__device__ __forceinline__ unsigned cluster_ctarank()
{
    unsigned r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}

__device__ __forceinline__ void cluster_sync()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__device__ __forceinline__ uint4 ld_dsmem(const uint4* local_ptr, unsigned cta)
{
    unsigned local = (unsigned)__cvta_generic_to_shared(local_ptr), remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(cta));
    uint4 v;
    asm volatile("ld.shared::cluster.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(remote) : "memory");
    return v;
}

template <int N, int DT>
__global__ void __launch_bounds__(kThreads)
k_oneshot_cluster(const RankPtrs p, const size_t count, const size_t ntiles)
{
    pdl_wait();
    __shared__ __align__(16) uint4 tile[kThreads];
    const unsigned r = cluster_ctarank();                  // this block's source to fetch and destination to write
    const size_t nvec = count / Elem<DT>::kElems;
    const size_t nclusters = gridDim.x / N, cluster_id = blockIdx.x / N;
    for (size_t t = cluster_id; t < ntiles; t += nclusters) {
        const size_t i = t * kThreads + threadIdx.x;
        if (i < nvec) tile[threadIdx.x] = ld_src(p.src[r] + i);
        cluster_sync();                                    // every block's tile is in its shared memory
        if (i < nvec) {
            uint4 v[N];
#pragma unroll
            for (int s = 0; s < N; ++s) v[s] = ld_dsmem(&tile[threadIdx.x], (unsigned)s);
            st_dst(p.dst[r] + i, fold_vectors<N, DT>(v));
        }
        cluster_sync();                                    // nobody still reads a tile that is about to be replaced
    }
    pdl_trigger();
    const size_t tail0 = nvec * Elem<DT>::kElems;
    if (tail0 < count && cluster_id == 0) {
        const size_t e = tail0 + threadIdx.x;
        if (e < count) store_elem<DT>(p.dst[r], e, fold_scalar<N, DT>(p, e));
    }
}

// ---- one-shot allreduce through per-SM work lists (the planner's M_compute at SM granularity) ------------
//
// CUDA has no thread-block -> SM affinity mask (the paper's dispatcher mechanism, Section 4.2.3), so
// affinity is taken from the other end: a block reads %smid and claims, one group at a time, the
// groups the planner put on that SM's list (an atomic cursor per SM, so two blocks that land on the
// same SM share its list).  Each SM with a list records that a block arrived there.  A block that
// runs out of work leaves once every list has such a block; if some list has none (the hardware
// scheduler gave that SM no block) it adopts that list instead -- the paper's fall-back of ignoring
// the affinity (Section 4.2.3).  Completion therefore never depends on where blocks land, and no
// block ever waits for another.  The last block to finish rewinds all counters, which makes the
// launch replayable from a CUDA graph without host work.
struct SmLists {
    const unsigned* off;        // [num_sms + 1] offsets into tiles
    const unsigned* tiles;      // tile index of every planned group, grouped by SM
    unsigned* cursor;           // [num_sms] next unclaimed entry of each SM's list
    unsigned* present;          // [num_sms] non-zero once a block has arrived on that SM
    unsigned* ctl;              // ctl[0]: non-empty lists whose SM has a block; ctl[1]: blocks that have left
    unsigned nonempty;          // number of non-empty lists
    int num_sms;
};

__device__ __forceinline__ unsigned read_smid_reg()
{
    unsigned s;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(s));
    return s;
}

__device__ __forceinline__ unsigned ld_volatile_u32(const unsigned* p)
{
    unsigned v;
    asm volatile("ld.volatile.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

constexpr unsigned kMaxBatch = 32;

// Lane 0 claims up to `batch` entries of list v with one atomic add (the cursor may run past the end;
// the last block rewinds it); the warp's lanes then fetch the claimed tile indices in one parallel
// load.  `announce`: lane 1 records, in the same round trip, that SM v's list has a block serving it.
// `exhausted` is set when the claim reached the end of the list.
__device__ __forceinline__ unsigned claim_from(const SmLists& sl, unsigned v, unsigned len, unsigned batch, bool announce,
                                               unsigned* sh_tiles, bool& exhausted)
{
    const unsigned lane = threadIdx.x & 31u;
    unsigned j0 = 0u;
    if (lane == 0 && len != 0u) j0 = atomicAdd(sl.cursor + v, batch);
    if (lane == 1 && announce && len != 0u && atomicExch(sl.present + v, 1u) == 0u) atomicAdd(sl.ctl, 1u);
    j0 = __shfl_sync(0xFFFFFFFFu, j0, 0);
    const unsigned n = (len != 0u && j0 < len) ? min(batch, len - j0) : 0u;
    exhausted = (len == 0u) || (j0 + batch >= len);
    if (lane < n) sh_tiles[lane] = sl.tiles[sl.off[v] + j0 + lane];
    return n;
}

// A list nobody is serving: its SM has no block (the hardware scheduler is free to do that).  Scans the
// SMs 32 at a time and returns one such SM, or ~0u.
__device__ __forceinline__ unsigned find_orphan(const SmLists& sl, unsigned own)
{
    const unsigned lane = threadIdx.x & 31u;
    for (unsigned base = 0; base < (unsigned)sl.num_sms; base += 32u) {
        const bool valid = base + lane < (unsigned)sl.num_sms;
        const unsigned w = (own + 1u + base + lane) % (unsigned)sl.num_sms;
        const unsigned wl = valid ? sl.off[w + 1] - sl.off[w] : 0u;
        const bool orphan = wl != 0u && ld_volatile_u32(sl.present + w) == 0u && ld_volatile_u32(sl.cursor + w) < wl;
        const unsigned mask = __ballot_sync(0xFFFFFFFFu, orphan);
        if (mask != 0u) return __shfl_sync(0xFFFFFFFFu, w, __ffs(mask) - 1);
    }
    return 0xFFFFFFFFu;
}

template <int N, int C, int DT, bool kTimed = false>
__global__ void __launch_bounds__(kThreads, min_blocks(N))
k_oneshot_sm(const RankPtrs p, const size_t count, const SmLists sl, const unsigned blocks_per_sm, unsigned* hist)
{
    pdl_wait();
    constexpr int kSplit = (N + C - 1) / C;
    __shared__ unsigned sh_n;
    __shared__ unsigned sh_tiles[kMaxBatch];
    const size_t nvec = count / Elem<DT>::kElems;
    const unsigned own = read_smid_reg() % (unsigned)sl.num_sms;
    const unsigned own_len = sl.off[own + 1] - sl.off[own];
    // an SM's list is shared by the blocks resident there: one claim per block takes its whole share
    const unsigned batch = min(kMaxBatch, max(1u, (own_len + blocks_per_sm - 1u) / blocks_per_sm));

    unsigned serving = own, serving_len = own_len;
    bool first = true, exhausted = false;
    while (true) {
        if (threadIdx.x < 32) {
            unsigned n = 0u;
            if (!exhausted) n = claim_from(sl, serving, serving_len, batch, first && serving == own, sh_tiles, exhausted);
            first = false;
            if (n == 0u) {
                // This list is done.  If every non-empty list has a block on its SM, those blocks will
                // finish them and this block may leave; otherwise adopt a list nobody is serving.
                unsigned served = 0u;
                if (own_len == 0u) __nanosleep(500);              // helpers: let the owners announce themselves first
                if (threadIdx.x == 0) served = ld_volatile_u32(sl.ctl);
                served = __shfl_sync(0xFFFFFFFFu, served, 0);
                if (served < sl.nonempty) {
                    const unsigned orphan = find_orphan(sl, own);
                    if (orphan != 0xFFFFFFFFu) {
                        serving = orphan;
                        serving_len = sl.off[orphan + 1] - sl.off[orphan];
                        n = claim_from(sl, serving, serving_len, batch, false, sh_tiles, exhausted);
                        if (n == 0u) { n = 0xFFFFFFFFu; exhausted = true; }      // lost the race for it: look again
                    }
                }
            }
            if (threadIdx.x == 0) sh_n = n;
        }
        __syncthreads();
        const unsigned n = sh_n;
        if (n == 0u) break;
        if (n != 0xFFFFFFFFu) {
            for (unsigned i = 0; i < n; ++i) {
                const size_t tile = sh_tiles[i];
#pragma unroll
                for (int sub = 0; sub < kSplit; ++sub) oneshot_group<N, C, DT, kTimed>(p, nvec, tile, sub * C, hist);
            }
        }
        __syncthreads();
    }
    pdl_trigger();
    const size_t tail0 = nvec * Elem<DT>::kElems;
    if (tail0 < count) {
        for (int d = blockIdx.x; d < N; d += gridDim.x) {
            const size_t e = tail0 + threadIdx.x;
            if (e < count) store_elem<DT>(p.dst[d], e, fold_scalar<N, DT>(p, e));
        }
    }
    // the last block out rewinds cursors, presence flags and counters for the next launch
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(sl.ctl + 1, 1u) == gridDim.x - 1u) {
            for (int s = 0; s < sl.num_sms; ++s) { sl.cursor[s] = 0u; sl.present[s] = 0u; }
            sl.ctl[0] = 0u;
            sl.ctl[1] = 0u;
            __threadfence();
        }
    }
}

// ---- reduce-scatter: work item = (rank r, tile of shard r) -------------------------------------
//
// dst[r][j] = fold_k src[k][r*S + j].  `shard_vec` = S/8 (vector path requires S % 8 == 0, which
// keeps r*S 16-byte aligned); `out` overrides dst (the fused two-shot writes into its shard scratch).
template <int N, int U, int DT, bool kStream>
__device__ __forceinline__ void reduce_tile(const RankPtrs& p, uint4* out, size_t src_off_vec,
                                            size_t nvec, size_t tile)
{
    const size_t base = tile * (size_t)(kThreads * U) + threadIdx.x;
    uint4 v[U][N];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t i = base + (size_t)u * kThreads;
        if (i < nvec) {
#pragma unroll
            for (int r = 0; r < N; ++r) v[u][r] = ld_src(p.src[r] + src_off_vec + i);
        }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t i = base + (size_t)u * kThreads;
        if (i < nvec) {
            if (kStream) st_stream(out + i, fold_vectors<N, DT>(v[u]));
            else st_dst(out + i, fold_vectors<N, DT>(v[u]));
        }
    }
}

// (No L2 prefetch ahead of the dependent-launch wait here: this kernel reads N bytes for every byte it writes and is
// bound by the reads at every size, so the extra requests only cost -- 8 x 512 KiB 2.43 against 2.16 us, 8 x 4 MiB 7.27
// against 6.40.)
template <int N, int U, int DT>
__global__ void __launch_bounds__(kThreads, min_blocks(N * U))
k_reduce_scatter(const RankPtrs p, const size_t shard_vec, const size_t tiles_per_shard)
{
    pdl_wait();
    const size_t nitems = tiles_per_shard * N;
    for (size_t item = blockIdx.x; item < nitems; item += gridDim.x) {
        const int r = (int)(item / tiles_per_shard);
        const size_t tile = item % tiles_per_shard;
        reduce_tile<N, U, DT, true>(p, p.dst[r], (size_t)r * shard_vec, shard_vec, tile);
    }
    pdl_trigger();
}

// Any shard length: one element per thread (slow path, used when S % 8 != 0).
template <int N, int DT>
__global__ void __launch_bounds__(kThreads)
k_reduce_scatter_scalar(const RankPtrs p, const size_t shard)
{
    pdl_wait();
    const size_t total = shard * N;
    for (size_t e = (size_t)blockIdx.x * kThreads + threadIdx.x; e < total; e += (size_t)gridDim.x * kThreads) {
        const int r = (int)(e / shard);
        store_elem<DT>(p.dst[r], e - (size_t)r * shard, fold_scalar<N, DT>(p, e));
    }
}

// ---- allgather: work item = (rank r, tile of shard r, group of destinations); local load, remote store ----
//
// The paper's form (Figure "Allocation_Diagram"): a thread block loads a chunk of its own rank's
// buffer and stores it into the peers' buffers.  `dsplit` blocks share one tile, each storing to
// nranks / dsplit destinations: small messages need the extra blocks to fill the machine (N stores per
// load from one thread are issue-bound), large ones use dsplit = 1 and read every source byte once.
template <int U>
__device__ __forceinline__ void gather_tile(const uint4* in, const RankPtrs& p, int d0, int d1, size_t dst_off_vec,
                                            size_t nvec, size_t tile, bool coherent)
{
    const size_t base = tile * (size_t)(kThreads * U) + threadIdx.x;
    uint4 v[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t i = base + (size_t)u * kThreads;
        if (i < nvec) v[u] = coherent ? ld_cg(in + i) : ld_src(in + i);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t i = base + (size_t)u * kThreads;
        if (i < nvec) {
            for (int d = d0; d < d1; ++d) st_stream(p.dst[d] + dst_off_vec + i, v[u]);
        }
    }
}

template <int U>
__global__ void __launch_bounds__(kThreads, min_blocks(U))
k_allgather(const RankPtrs p, const int nranks, const size_t shard_vec, const size_t tiles_per_shard, const int dsplit)
{
    pdl_wait();
    const int per = (nranks + dsplit - 1) / dsplit;
    const size_t nitems = tiles_per_shard * nranks * dsplit;
    for (size_t item = blockIdx.x; item < nitems; item += gridDim.x) {
        const int g = (int)(item % dsplit);
        const size_t rt = item / dsplit;
        const int r = (int)(rt % nranks);
        const size_t tile = rt / nranks;
        const int d0 = g * per, d1 = min(nranks, d0 + per);
        gather_tile<U>(p.src[r], p, d0, d1, (size_t)r * shard_vec, shard_vec, tile, false);
    }
    pdl_trigger();
}

// Small and mid-sized gathers: one block per (rank, tile of tv <= kThreads vectors), a thread loads its vector once and
// stores it to the N destinations.  With the tile sized so that every SM gets about four blocks this is faster than
// the bulk-copy form below up to 128 MiB of output (16 x 8 KiB 1.28 against 1.68 us, 16 x 64 KiB 3.46 against 3.81,
// 8 x 64 KiB 1.60 against 1.92, 16 x 512 KiB 22.9 against 24.1; 8 x 8 MiB 96.5 against 93.9).
__global__ void __launch_bounds__(kThreads)
k_allgather_small(const RankPtrs p, const int nranks, const size_t shard_vec, const size_t tiles_per_shard, const unsigned tv,
                  const int prefetch)
{
    const int r = (int)(blockIdx.x % (unsigned)nranks);
    const size_t tile = blockIdx.x / (unsigned)nranks;
    const size_t i0 = tile * tv;
    if (prefetch && threadIdx.x == 0 && i0 < shard_vec)
        prefetch_l2_bulk(p.src[r] + i0, (unsigned)(shard_vec - i0 < (size_t)tv ? shard_vec - i0 : (size_t)tv) * 16u);
    pdl_wait();
    const size_t i = i0 + threadIdx.x;
    if (threadIdx.x < tv && i < shard_vec) {
        const uint4 v = ld_src(p.src[r] + i);
        for (int d = 0; d < nranks; ++d) st_stream(p.dst[d] + (size_t)r * shard_vec + i, v);
    }
    pdl_trigger();
}

// The same work item moved entirely by the bulk-copy engine: one bulk load of the tile into shared memory,
// then one bulk store per destination straight out of shared memory, each issued by its own thread.  No
// register ever holds the data and the SM's load / store pipes carry none of the N-fold stores.
__device__ __forceinline__ void bulk_store(void* gdst, const void* smem_src, unsigned bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 :: "l"(gdst), "r"(smem_u32(smem_src)), "r"(bytes) : "memory");
}

__device__ __forceinline__ void bulk_store_drain()       // this thread's bulk stores have finished reading shared memory
{
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}

// tv = vectors per tile; shared memory = tv * 16 bytes.
__global__ void __launch_bounds__(kThreads)
k_allgather_bulk(const RankPtrs p, const int nranks, const size_t shard_vec, const size_t tiles_per_shard, const unsigned tv,
                 unsigned* status, const unsigned long long timeout_ns, const int prefetch)
{
    extern __shared__ __align__(128) unsigned char stage_raw[];
    __shared__ __align__(8) uint64_t bar;
    const int r = (int)(blockIdx.x % (unsigned)nranks);
    const size_t tile = blockIdx.x / (unsigned)nranks;
    const size_t base = tile * tv;
    const unsigned nv = (tile < tiles_per_shard && base < shard_vec) ? (unsigned)((shard_vec - base < tv) ? shard_vec - base : tv) : 0u;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1u);
        if (prefetch && nv != 0u) prefetch_l2_bulk(p.src[r] + base, nv * 16u);     // ahead of the wait: see prefetch_l2_bulk
    }
    __syncthreads();
    pdl_wait();
    if (nv != 0u && threadIdx.x < (unsigned)nranks) {
        if (threadIdx.x == 0) {
            mbar_expect_tx(&bar, nv * 16u);
            bulk_load(stage_raw, p.src[r] + base, nv * 16u, &bar);
        }
        if (mbar_wait(&bar, 0u, status, timeout_ns)) {
            bulk_store(p.dst[threadIdx.x] + (size_t)r * shard_vec + base, stage_raw, nv * 16u);
            bulk_store_drain();
        }
    }
    pdl_trigger();
}

__global__ void __launch_bounds__(kThreads)
k_allgather_scalar(const RankPtrs p, const int nranks, const size_t shard)
{
    pdl_wait();
    const size_t total = shard * nranks;
    for (size_t e = (size_t)blockIdx.x * kThreads + threadIdx.x; e < total; e += (size_t)gridDim.x * kThreads) {
        const int r = (int)(e / shard);
        const uint16_t v = ld_src16(reinterpret_cast<const uint16_t*>(p.src[r]) + (e - (size_t)r * shard));
        for (int d = 0; d < nranks; ++d) reinterpret_cast<uint16_t*>(p.dst[d])[e] = v;
    }
}

// ---- alltoall: work item = (sender r, receiver d, tile of the block r sends to d) -------------------------
//
// dst[d][r*S + j] = src[r][d*S + j]: the paper's third collective (expert token routing), a block
// transpose.  Local load from the sender's buffer, store into the receiver's (the put form).
template <int U>
__global__ void __launch_bounds__(kThreads, min_blocks(U))
k_alltoall(const RankPtrs p, const int nranks, const size_t block_vec, const size_t tiles_per_block)
{
    pdl_wait();
    const size_t pairs = (size_t)nranks * nranks;
    const size_t nitems = tiles_per_block * pairs;
    for (size_t item = blockIdx.x; item < nitems; item += gridDim.x) {
        const size_t pair = item % pairs, tile = item / pairs;   // pairs fastest: neighbours hit different buffers
        const int r = (int)(pair / nranks), d = (int)(pair % nranks);
        const uint4* in = p.src[r] + (size_t)d * block_vec;
        uint4* out = p.dst[d] + (size_t)r * block_vec;
        const size_t base = tile * (size_t)(kThreads * U) + threadIdx.x;
        uint4 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t i = base + (size_t)u * kThreads;
            if (i < block_vec) v[u] = ld_src(in + i);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t i = base + (size_t)u * kThreads;
            if (i < block_vec) st_stream(out + i, v[u]);
        }
    }
    pdl_trigger();
}

// The same block transpose moved by the bulk-copy engine: a tile goes global -> shared -> global without
// touching a register.  tv = vectors per tile; shared memory = tv * 16 bytes; one block per (pair, tile).
__global__ void __launch_bounds__(kThreads)
k_alltoall_bulk(const RankPtrs p, const int nranks, const size_t block_vec, const size_t tiles_per_block, const unsigned tv,
                unsigned* status, const unsigned long long timeout_ns, const int prefetch)
{
    extern __shared__ __align__(128) unsigned char stage_raw[];
    __shared__ __align__(8) uint64_t bar;
    const size_t pairs = (size_t)nranks * nranks;
    const size_t pair = blockIdx.x % pairs, tile = blockIdx.x / pairs;   // pairs fastest: neighbours hit different buffers
    const int r = (int)(pair / nranks), d = (int)(pair % nranks);
    const size_t base = tile * tv;
    const unsigned nv = (tile < tiles_per_block && base < block_vec) ? (unsigned)((block_vec - base < tv) ? block_vec - base : tv) : 0u;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1u);
        if (prefetch && nv != 0u) prefetch_l2_bulk(p.src[r] + (size_t)d * block_vec + base, nv * 16u);
        pdl_wait();
        if (nv != 0u) {
            mbar_expect_tx(&bar, nv * 16u);
            bulk_load(stage_raw, p.src[r] + (size_t)d * block_vec + base, nv * 16u, &bar);
            if (mbar_wait(&bar, 0u, status, timeout_ns)) {
                bulk_store(p.dst[d] + (size_t)r * block_vec + base, stage_raw, nv * 16u);
                bulk_store_drain();
            }
        }
    }
    pdl_trigger();
}

// Any block length (used when S % 8 != 0): one element per thread.
__global__ void __launch_bounds__(kThreads)
k_alltoall_scalar(const RankPtrs p, const int nranks, const size_t block)
{
    pdl_wait();
    const size_t per_rank = block * nranks, total = per_rank * nranks;
    for (size_t e = (size_t)blockIdx.x * kThreads + threadIdx.x; e < total; e += (size_t)gridDim.x * kThreads) {
        const int d = (int)(e / per_rank);
        const size_t within = e - (size_t)d * per_rank;
        const int r = (int)(within / block);
        const size_t i = within - (size_t)r * block;
        reinterpret_cast<uint16_t*>(p.dst[d])[within] = ld_src16(reinterpret_cast<const uint16_t*>(p.src[r]) + (size_t)d * block + i);
    }
    pdl_trigger();
}

// ---- flag barrier among the co-resident blocks of one launch ----------------------------------------
//
// Stands where a real system has a cross-GPU flag synchronisation between the
// reduce-scatter and the allgather.  Two words in device memory: `arrive` counts
// arrivals of the current round and is reset by the last arriver, `epoch` is
// bumped by the last arriver and polled by everyone else.  The epoch only ever
// grows, so graph replays need no host reset.  Every wait is bounded: after
// `timeout_ns` the block latches NUNA_ERR_TIMEOUT in `status` and returns false;
// the caller then skips the rest of its work and exits.  Nothing traps or hangs.

__device__ __forceinline__ unsigned int ld_acquire(const unsigned int* p)
{
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Returns true when all `expected` blocks arrived.  Must be called by every thread of the block.
__device__ __forceinline__ bool flag_barrier(BarrierWords* bw, unsigned int expected, unsigned int epoch0,
                                             unsigned long long timeout_ns)
{
    __shared__ int ok;
    __syncthreads();                                   // this block's phase-1 stores are issued
    if (threadIdx.x == 0) {
        int good = 1;
        __threadfence();                               // ... and visible device-wide before we arrive
        unsigned int prev;
        asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(prev) : "l"(&bw->arrive) : "memory");
        if (prev == expected - 1) {
            bw->arrive = 0;                            // nobody touches it again before the epoch moves
            asm volatile("red.release.gpu.global.add.u32 [%0], 1;" :: "l"(&bw->epoch) : "memory");
        } else {
            const unsigned long long t0 = globaltimer_ns();
            unsigned int polls = 0;
            while (ld_acquire(&bw->epoch) == epoch0) {
                if ((++polls & 63u) == 0u && globaltimer_ns() - t0 > timeout_ns) {
                    atomicMax(&bw->status, 6u);        // NUNA_ERR_TIMEOUT
                    good = 0;
                    break;
                }
            }
        }
        ok = good;
    }
    __syncthreads();
    return ok != 0;
}

// ---- fused two-shot allreduce, synchronised by per-tile ready flags ---------------------------------------
//
// Reduce-scatter, flag synchronisation and put-style allgather in ONE kernel, with no grid-wide barrier
// and no host synchronisation.  The message is cut into tiles of tv vectors; the chunk a tile lies in
// names the emulated rank that owns its reduction.  Every thread block takes ONE work item, numbered by a
// ticket it draws from a device-wide counter when it starts; item i (0 <= i < tiles + lead) has two
// halves, run side by side by the two halves of the block:
//   produce tile i (while i < tiles; threads 0..127): the tile's N source slices are fetched into shared
//       memory by bulk asynchronous copies (one thread issues them; they complete on an mbarrier), folded
//       in rank order, stored to the shard scratch, and flag[i] = this launch's epoch is published with a
//       release store (the producing rank's "chunk ready" signal);
//   consume tile i - lead (once i >= lead; threads 128..255): acquire-poll that tile's flag until it
//       holds this launch's epoch (bounded wait), then load the tile from the scratch once and store it
//       into all N destinations (the put-style allgather).
// `lead` is about what the whole device holds at once, so a tile is normally consumed long after it was
// produced and its flag is found set; blocks flow from reducing into gathering without a common stop,
// and because every block handles one item the hardware block scheduler does the load balancing.
//
// Progress: an item waits only for the flag of an item with a smaller ticket.  Tickets are drawn by
// running blocks in the order they start, so that item belongs to a block that is running or has
// finished, and whose own wait (if any) is again for a smaller ticket; by induction every wait ends, for
// any grid size and without any co-residency requirement.  Every wait (flag, copy completion) is bounded
// all the same: on expiry the block latches NUNA_ERR_TIMEOUT and leaves; nothing traps or spins forever.
//
// Replays: one 64-bit word in device memory carries the launch epoch (high half) and the next ticket (low
// half), so a block learns both with its one atomic add.  The block that draws the last ticket knows that
// every ticket of this launch is taken and stores (epoch + 1, 0) for the next launch.  Flags are compared
// for equality with the epoch, so stale flags of earlier launches (or of another tiling) never match and
// nothing is reset from the host.
// sys_scope: release / acquire at system scope, which is what the flags need once the ranks are separate
// GPUs writing into each other's memory; within one GPU device scope is enough and cheaper.
__device__ __forceinline__ void st_release(unsigned int* p, unsigned int v, bool sys_scope)
{
    if (sys_scope) asm volatile("st.release.sys.global.u32 [%0], %1;" :: "l"(p), "r"(v) : "memory");
    else           asm volatile("st.release.gpu.global.u32 [%0], %1;" :: "l"(p), "r"(v) : "memory");
}

__device__ __forceinline__ unsigned int ld_acquire_scoped(const unsigned int* p, bool sys_scope)
{
    unsigned int v;
    if (sys_scope) asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    else           asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Polls *flag until it equals `want`.  Returns false (and latches the timeout) when timeout_ns runs out.
__device__ __forceinline__ bool wait_flag(const unsigned int* flag, unsigned int want, unsigned long long timeout_ns,
                                          unsigned int* status, bool sys_scope)
{
    if (ld_acquire_scoped(flag, sys_scope) == want) return true;
    const unsigned long long t0 = globaltimer_ns();
    unsigned int polls = 0;
    while (ld_acquire_scoped(flag, sys_scope) != want) {
        if ((++polls & 63u) == 0u && globaltimer_ns() - t0 > timeout_ns) {
            atomicMax(status, 6u);                     // NUNA_ERR_TIMEOUT
            return false;
        }
    }
    return true;
}

// Barrier among the 128 threads of one half of the block (ids 1 and 2; 0 is __syncthreads).
__device__ __forceinline__ void half_sync(int id) { asm volatile("bar.sync %0, 128;" :: "r"(id) : "memory"); }

// (Working ahead on the guess "my ticket will be my block index" while the ticket is on its way was tried
// and measured slower: the blocks of a wave start together, so their tickets come back in no particular
// order and most guesses are wrong.)
//
// tv: vectors per tile; shared memory = N * tv * 16 bytes.  lead_max: upper bound of `lead`.
// mode bits: 0 in normal use; bit 0: consumers wait for a flag value nobody publishes (test of the bounded
// wait); bit 2: keep consumed shard lines in L2 (for measuring what the discard saves); bit 3: flags are
// released and acquired at system scope (NUNA_TWOSHOT_SYS_SCOPE).
// kMinBlocks: resident blocks per SM the register allocation is held to.  4 (64 registers) gives the shortest
// path per block, best while the message is small enough for latency to dominate (8 KiB per rank: 3.4 us
// against 3.7 us).  6 holds it to 40 registers: more tiles in flight per SM, which is what counts once the
// message is bandwidth-bound (measured at 8 ranks: 16 MiB per rank 48.7 -> 45.6 us).
template <int N, int DT, int kMinBlocks>
__global__ void __launch_bounds__(kThreads, kMinBlocks)
k_twoshot_flags(const RankPtrs p, uint4* scratch, unsigned int* flags, const size_t count, const unsigned tv,
                const unsigned lead_max, BarrierWords* bw, const unsigned long long timeout_ns, const unsigned int debug)
{
    constexpr unsigned kHalf = kThreads / 2;
    const unsigned wait_bias = debug & 1u;
    const bool discard_shard = (debug & 4u) == 0u;
    const bool sys_scope = (debug & 8u) != 0u;
    extern __shared__ __align__(128) unsigned char stage_raw[];
    uint4* stage = reinterpret_cast<uint4*>(stage_raw);            // [N][tv]
    __shared__ __align__(8) uint64_t bar;
    __shared__ unsigned long long sh_ticket;
    __shared__ int sh_ok, sh_landed;
    const size_t nvec = count / Elem<DT>::kElems;
    const size_t tail0 = nvec * Elem<DT>::kElems;
    const size_t ntiles = nvec ? (nvec + tv - 1) / tv : 1;         // a ragged tail rides on the last tile
    const size_t lead = ntiles < lead_max ? ntiles : lead_max;
    if (threadIdx.x == 0) mbar_init(&bar, 1u);
    if ((debug & 16u) && blockIdx.x < ntiles && threadIdx.x < N) {
        // tickets come out nearly in block order: ask L2 for the tile this block will most likely produce
        const size_t i0 = (size_t)blockIdx.x * tv;
        const uint4* a = p.src[0];
#pragma unroll
        for (int r = 1; r < N; ++r) if ((int)threadIdx.x == r) a = p.src[r];
        if (i0 < nvec) prefetch_l2_bulk(a + i0, (unsigned)(nvec - i0 < (size_t)tv ? nvec - i0 : (size_t)tv) * 16u);
    }
    pdl_wait();                                                     // before the first global load or store
    if (threadIdx.x == 0) {
        const unsigned long long t = atomicAdd(&bw->ticket, 1ull);  // epoch and ticket in one round trip
        if ((unsigned)t == gridDim.x - 1u)                          // the last ticket: set up the next launch
            *reinterpret_cast<volatile unsigned long long*>(&bw->ticket) = ((t >> 32) + 1ull) << 32;
        sh_ticket = t;
    }
    __syncthreads();
    const size_t item = (unsigned)sh_ticket;
    const unsigned epoch1 = (unsigned)(sh_ticket >> 32) + 1u;
    const bool produce = item < ntiles, consume = item >= lead && item < ntiles + lead;

    if (threadIdx.x < kHalf) {
        // ---- produce half ----
        if (produce) {
            const size_t pbase = item * tv;
            const unsigned pnv = pbase < nvec ? (unsigned)((nvec - pbase < tv) ? nvec - pbase : tv) : 0u;
            bool landed = true;
            if (pnv != 0u) {
                if (threadIdx.x == 0) {
                    mbar_expect_tx(&bar, (unsigned)N * pnv * 16u);
#pragma unroll
                    for (int r = 0; r < N; ++r) bulk_load(stage + (size_t)r * tv, p.src[r] + pbase, pnv * 16u, &bar);
                }
                landed = mbar_wait(&bar, 0u, &bw->status, timeout_ns);
                if (landed) {
                    for (unsigned j = threadIdx.x; j < pnv; j += kHalf) {
                        uint4 v[N];
#pragma unroll
                        for (int r = 0; r < N; ++r) v[r] = ld_shared_v4(stage + (size_t)r * tv + j);
                        st_dst(scratch + pbase + j, fold_vectors<N, DT>(v));
                    }
                }
            }
            if (item == ntiles - 1 && tail0 < count) {
                const size_t e = tail0 + threadIdx.x;
                if (e < count) store_elem<DT>(scratch, e, fold_scalar<N, DT>(p, e));
            }
            if (threadIdx.x == 0) sh_landed = 1;
            half_sync(1);
            if (!landed) sh_landed = 0;
            half_sync(1);                              // every thread's shard stores are issued ...
            if (threadIdx.x == 0 && sh_landed) st_release(flags + item, epoch1, sys_scope);   // ... and ordered before the flag
        }
    } else {
        // ---- consume half ----
        if (consume) {
            const size_t ct = item - lead, cbase = ct * tv;
            if (threadIdx.x == kHalf)
                sh_ok = wait_flag(flags + ct, epoch1 + wait_bias, timeout_ns, &bw->status, sys_scope) ? 1 : 0;
            half_sync(2);                              // flag acquired by one thread -> every thread may read the tile
            if (sh_ok) {
                const unsigned cnv = cbase < nvec ? (unsigned)((nvec - cbase < tv) ? nvec - cbase : tv) : 0u;
                for (unsigned j = threadIdx.x - kHalf; j < cnv; j += kHalf) {
                    const uint4 c = ld_cg(scratch + cbase + j);
#pragma unroll
                    for (int d = 0; d < N; ++d) st_stream(p.dst[d] + cbase + j, c);
                }
                // The tile has exactly one consumer, so its shard lines are dead now: drop them from L2
                // instead of letting them be written back to DRAM (whole, 128-byte aligned lines only).
                if (discard_shard && (((uintptr_t)scratch | (uintptr_t)(cbase * 16u)) & 127u) == 0u) {
                    half_sync(2);                      // every thread's loads of the tile have returned
                    for (unsigned line = threadIdx.x - kHalf; line < cnv / 8u; line += kHalf)
                        asm volatile("discard.global.L2 [%0], 128;" :: "l"(scratch + cbase + (size_t)line * 8u) : "memory");
                }
                if (ct == ntiles - 1 && tail0 < count) {
                    const size_t e = tail0 + (threadIdx.x - kHalf);
                    if (e < count) {
                        const uint32_t w = load_elem_cg<DT>(scratch, e);
                        for (int d = 0; d < N; ++d) store_elem<DT>(p.dst[d], e, w);
                    }
                }
            }
        }
    }
    pdl_trigger();
}

// Two-shot without the intermediate: the block that reduces a tile stores it into all N destinations.
// (A form that moves the tile through shared memory with bulk copies in both directions was measured too:
// slower up to 4 MiB per rank -- 512 KiB: 3.2 vs 2.85 us -- and within 1.5 % beyond, so it was not kept.)
template <int N, int U, int DT>
__global__ void __launch_bounds__(kThreads, min_blocks(N * U))
k_twoshot_put(const RankPtrs p, const size_t count, const size_t ntiles, const int prefetch)
{
    const size_t nvec = count / Elem<DT>::kElems;
    if (prefetch && blockIdx.x < ntiles && threadIdx.x < N) {        // thread r: source r's slice of the first tile
        const size_t i0 = (size_t)blockIdx.x * (size_t)(kThreads * U);
        const uint4* a = p.src[0];
#pragma unroll
        for (int r = 1; r < N; ++r) if ((int)threadIdx.x == r) a = p.src[r];
        if (i0 < nvec) prefetch_l2_bulk(a + i0, (unsigned)(nvec - i0 < (size_t)(kThreads * U) ? nvec - i0 : (size_t)(kThreads * U)) * 16u);
    }
    pdl_wait();
    for (size_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const size_t base = tile * (size_t)(kThreads * U) + threadIdx.x;
        uint4 v[U][N];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t i = base + (size_t)u * kThreads;
            if (i < nvec) {
#pragma unroll
                for (int r = 0; r < N; ++r) v[u][r] = ld_src(p.src[r] + i);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t i = base + (size_t)u * kThreads;
            if (i < nvec) {
                const uint4 o = fold_vectors<N, DT>(v[u]);
#pragma unroll
                for (int d = 0; d < N; ++d) st_stream(p.dst[d] + i, o);
            }
        }
    }
    pdl_trigger();
    const size_t tail0 = nvec * Elem<DT>::kElems;
    if (tail0 < count && blockIdx.x == 0) {
        const size_t e = tail0 + threadIdx.x;
        if (e < count) {
            const uint32_t v = fold_scalar<N, DT>(p, e);
            for (int d = 0; d < N; ++d) store_elem<DT>(p.dst[d], e, v);
        }
    }
}

// ---- decode-step chain in one kernel --------------------------------------------------------------------
//
// For small nodes a kernel launch (about 1.1 us even as a graph node with dependent launch) costs many
// times the data time, so the whole chain of back-to-back one-shot allreduces runs as ONE kernel on one
// thread-block cluster.  Node k works on buffer set k mod nsets; the node boundary is a cluster barrier
// with release / acquire semantics, so node k+1 reads only after every block has finished writing node k
// (a node may read what its predecessor wrote).  Within a node the work is the register-sharing co-located
// one-shot, items dealt to the cluster's threads in order.  Loads go to L2 (ld.global.cg): a source may have
// been written by another SM in the previous node, and L1 is not coherent between SMs.
__device__ __forceinline__ unsigned cluster_nctarank()
{
    unsigned r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}

__device__ __forceinline__ uint4 ld_coherent(const uint4* p)
{
    uint4 v;
    asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}

template <int N, int C, int DT>
__global__ void __launch_bounds__(kThreads, 1)
k_chain_persistent(const __grid_constant__ ChainSets sets, const int nsets, const int nnodes, const size_t count)
{
    constexpr int kSplit = (N + C - 1) / C;                // destination groups per vector
    const unsigned nblk = cluster_nctarank(), blk = cluster_ctarank();
    const size_t nvec = count / Elem<DT>::kElems;
    const size_t nitems = nvec * kSplit;                   // item = (vector, group of C destinations), group fastest
    const size_t tail0 = nvec * Elem<DT>::kElems;
    const size_t first = (size_t)blk * kThreads + threadIdx.x, stride = (size_t)nblk * kThreads;
    int set = 0;
    for (int node = 0; node < nnodes; ++node) {
        const RankPtrs& p = sets.s[set];
        // within a node the work is the register-sharing one-shot: N loads once, C rank-ordered folds and stores
        for (size_t item = first; item < nitems; item += stride) {
            const size_t i = item / kSplit;
            const int d0 = (int)(item % kSplit) * C;
            uint4 v[N];
#pragma unroll
            for (int r = 0; r < N; ++r) v[r] = ld_cg(p.src[r] + i);
#pragma unroll
            for (int c = 0; c < C; ++c)
                if (d0 + c < N) st_dst(p.dst[d0 + c] + i, fold_vectors_own<N, DT>(v));
        }
        if (tail0 < count && blk == 0) {
            const size_t e = tail0 + (threadIdx.x % 32);
            for (int d = threadIdx.x / 32; d < N && e < count; d += kThreads / 32) {
                uint32_t w;
                if (DT == kF32) {
                    float acc = __uint_as_float(load_elem_cg<DT>(p.src[0], e));
                    for (int r = 1; r < N; ++r) acc = __fadd_rn(acc, __uint_as_float(load_elem_cg<DT>(p.src[r], e)));
                    w = __float_as_uint(acc);
                } else {
                    float acc, unused;
                    widen_word<DT>(acc, unused, load_elem_cg<DT>(p.src[0], e));
                    for (int r = 1; r < N; ++r) acc = add_narrow<DT>(acc, (uint16_t)load_elem_cg<DT>(p.src[r], e));
                    w = pack2<DT>(acc, 0.0f) & 0xFFFFu;
                }
                store_elem<DT>(p.dst[d], e, w);
            }
        }
        cluster_sync();                                // node boundary: writes of node k before reads of node k+1
        set = (set + 1 == nsets) ? 0 : set + 1;
    }
}

// Barrier self-test: every block arrives at a barrier that expects `expected` arrivals.
__global__ void k_barrier_selftest(BarrierWords* bw, unsigned int expected, unsigned long long timeout_ns,
                                   unsigned int* passed)
{
    unsigned int epoch0 = 0;
    if (threadIdx.x == 0) epoch0 = ld_acquire(&bw->epoch);
    if (flag_barrier(bw, expected, epoch0, timeout_ns) && threadIdx.x == 0) atomicAdd(passed, 1u);
}

// Launch-floor reference: same grid shape, no memory traffic.
// The launch floor: waits for its predecessor and lets its successor go, like every collective kernel.
__global__ void __launch_bounds__(kThreads) k_empty(int) { pdl_wait(); pdl_trigger(); }

// The same, releasing the successor before waiting (a measurement aid: how closely launches can follow one
// another when nothing delays the trigger).  A kernel of its own: reading a parameter ahead of the wait made the
// plain floor kernel 0.12 us slower per graph node.
__global__ void __launch_bounds__(kThreads) k_empty_trigger_first(int) { pdl_trigger(); pdl_wait(); }

}  // namespace nuna
