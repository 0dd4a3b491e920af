// Topology probe: how non-uniform is memory access latency from each SM to each rank buffer?
//
// The paper measures, on real multi-die GPUs, the latency of a remote access issued from every
// compute unit to a range of target addresses (Section 3.2) and finds that it depends on both.
// This is the single-GPU analogue for the two-die B200: one block per SM (identified by %smid)
// times dependent L2-only loads (ld.global.cg) to sampled 128-byte lines inside the caller's own
// buffers, and a cold pointer chase through private scratch for the DRAM-miss case.
//
//  * hit latency:  a sampled line holds a pointer to itself; K dependent loads of it from one SM,
//    after two warming loads, give that SM's L2-hit latency to that line.  SMs start at different
//    lines and rotate, so a line is rarely probed by two SMs at once.
//  * miss latency: a random single-cycle permutation (Sattolo) over 4 KiB-spaced nodes of a scratch
//    region; the region is evicted from L2 by writing a second region larger than L2; every SM then
//    walks its own disjoint segment of the cycle, touching each node once.
//  * host analysis: SMs are split into two domains by the sign of the first principal component of
//    the doubly-centred (SM x line) latency matrix (power iteration); each line's "home" domain is
//    the side that reaches it faster.  The verdict is NONUNIFORM only if the far-near gap exceeds
//    three times the run-to-run noise and three percent of the median latency.
//
// The sampled words are saved before and restored after the measurement, so buffer contents are
// unchanged on return.  Not capturable: it allocates, copies and synchronises.
#include "nuna_internal.h"
#include "nuna_debug.h"

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <unordered_map>
#include <vector>

namespace nuna {

constexpr int kHitLoads = 16;
constexpr int kMissSteps = 48;
constexpr size_t kNodeStride = 4096;

__device__ __forceinline__ unsigned read_smid()
{
    unsigned s;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(s));
    return s;
}

__device__ __forceinline__ unsigned long long ld_cg_u64(unsigned long long addr)
{
    unsigned long long v;
    asm volatile("ld.global.cg.u64 %0, [%1];" : "=l"(v) : "l"(addr) : "memory");
    return v;
}

// mode 0: save the word at every sampled line and replace it by a pointer to itself; mode 1: restore.
__global__ void k_probe_words(unsigned long long* const* lines, unsigned long long* saved, int nlines, int mode)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= nlines) return;
    if (mode == 0) {
        saved[i] = *lines[i];
        *lines[i] = (unsigned long long)lines[i];
    } else {
        *lines[i] = saved[i];
    }
}

// One block per SM (the dynamic shared memory request forces that); lane 0 measures.
__global__ void k_probe_hit(unsigned long long* const* lines, int nlines, float* lat /* [max_sms][nlines] */,
                            int* sm_seen, int max_sms, unsigned* bad)
{
    extern __shared__ unsigned char force_one_block_per_sm[];
    if (threadIdx.x != 0) return;
    const unsigned s = read_smid();
    if ((int)s >= max_sms) return;
    atomicAdd(&sm_seen[s], 1);
    for (int j = 0; j < nlines; ++j) {
        const int li = (int)((blockIdx.x * 7u + (unsigned)j) % (unsigned)nlines);
        unsigned long long p = (unsigned long long)lines[li];
        const unsigned long long self = p;
        p = ld_cg_u64(p);
        p = ld_cg_u64(p);
        const long long t0 = clock64();
#pragma unroll
        for (int k = 0; k < kHitLoads; ++k) p = ld_cg_u64(p);
        const long long t1 = clock64();
        if (p != self) atomicAdd(bad, 1u);
        lat[(size_t)s * nlines + li] = (float)(t1 - t0) / kHitLoads;
    }
}

// Writes the chain: node i (at base + i * stride) holds the index of its successor.
__global__ void k_chain_write(unsigned char* base, const unsigned* next, int nnodes)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < nnodes) *reinterpret_cast<unsigned long long*>(base + (size_t)i * kNodeStride) = next[i];
}

__global__ void k_flush(uint4* p, size_t nvec)
{
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += (size_t)gridDim.x * blockDim.x)
        p[i] = make_uint4(0u, 0u, 0u, 0u);
}

__global__ void k_probe_miss(const unsigned char* base, const unsigned* starts, float* lat_miss, unsigned* ends, int max_sms)
{
    extern __shared__ unsigned char force_one_block_per_sm[];
    if (threadIdx.x != 0) return;
    const unsigned s = read_smid();
    if ((int)s >= max_sms) return;
    unsigned long long idx = starts[blockIdx.x];
    const long long t0 = clock64();
    for (int k = 0; k < kMissSteps; ++k)
        idx = ld_cg_u64((unsigned long long)(base + (size_t)idx * kNodeStride));
    const long long t1 = clock64();
    lat_miss[s] = (float)(t1 - t0) / kMissSteps;
    ends[blockIdx.x] = (unsigned)idx;
}

// Solo streaming read rate of one SM: the block that lands on SM `target` reads the window `passes` times
// with 16-byte L2-only loads (after one untimed pass that brings it into L2); every other block leaves at
// once, so the measuring SM has the memory system to itself.  bytes / nanoseconds = GB/s.
__global__ void k_probe_bw(const uint4* window, unsigned nvec, unsigned target, int passes, float* gbs, int max_sms)
{
    extern __shared__ unsigned char force_one_block_per_sm[];
    __shared__ unsigned sink;
    const unsigned s = read_smid();
    if (s != target || (int)s >= max_sms) return;
    unsigned acc = 0;
    for (unsigned i = threadIdx.x; i < nvec; i += blockDim.x) acc ^= (unsigned)ld_cg_u64((unsigned long long)(window + i));
    __syncthreads();
    unsigned long long t0, t1;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t0) :: "memory");
    for (int p = 0; p < passes; ++p) {
#pragma unroll 8
        for (unsigned i = threadIdx.x; i < nvec; i += blockDim.x) {
            unsigned x, y, z, w;
            asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(x), "=r"(y), "=r"(z), "=r"(w) : "l"(window + i) : "memory");
            acc ^= x ^ y ^ z ^ w;
        }
    }
    __syncthreads();
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t1) :: "memory");
    if (acc == 0x9E3779B9u) sink = acc;                            // keeps the loads alive
    if (threadIdx.x == 0 && t1 > t0) gbs[s] = (float)((double)nvec * 16.0 * passes / (double)(t1 - t0));
}

static uint64_t splitmix(uint64_t& x)
{
    uint64_t z = (x += 0x9E3779B97F4A7C15ull);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

// Sattolo's algorithm: a uniformly random permutation that is one single cycle over all nodes.
void sattolo_cycle(std::vector<unsigned>& next, uint64_t seed)
{
    const size_t n = next.size();
    std::vector<unsigned> order(n);
    for (size_t i = 0; i < n; ++i) order[i] = (unsigned)i;
    for (size_t i = n - 1; i > 0; --i) {
        const size_t j = (size_t)(splitmix(seed) % i);          // j < i: never a fixed point
        std::swap(order[i], order[j]);
    }
    for (size_t i = 0; i < n; ++i) next[order[i]] = order[(i + 1) % n];
}

// Splits SMs in two by the first principal component of the doubly-centred latency matrix and
// fills the analysis fields of `out`.  lat[s * nlines + l], valid only for reported SMs.
void analyse_topology(const std::vector<float>& lat, const std::vector<float>& lat_rep, int nlines, nuna_topology_t* out,
                      std::vector<int>* homes = nullptr)
{
    std::vector<int> sms;
    for (int s = 0; s < out->num_sms && s < NUNA_MAX_SMS; ++s)
        if (out->sm_reported[s]) sms.push_back(s);
    const int S = (int)sms.size(), L = nlines;
    out->num_domains = 1;
    out->verdict = NUNA_TOPO_UNIFORM;
    out->domain_gap = out->near_lat = out->far_lat = 0.f;
    if (S < 2 || L < 2) return;
    std::vector<double> X((size_t)S * L), rowm(S, 0.0), colm(L, 0.0);
    double all = 0.0;
    for (int i = 0; i < S; ++i)
        for (int l = 0; l < L; ++l) {
            const double v = lat[(size_t)sms[i] * L + l];
            X[(size_t)i * L + l] = v;
            rowm[i] += v / L;
            colm[l] += v / S;
            all += v / ((double)S * L);
        }
    for (int i = 0; i < S; ++i) out->sm_lat_hit[sms[i]] = (float)rowm[i];
    const double mn = *std::min_element(rowm.begin(), rowm.end()), mx = *std::max_element(rowm.begin(), rowm.end());
    out->nonuniformity = (float)((mx - mn) / mn);
    // run-to-run noise: median absolute difference between the two repetitions
    std::vector<float> diff;
    diff.reserve((size_t)S * L);
    for (int i = 0; i < S; ++i)
        for (int l = 0; l < L; ++l)
            diff.push_back(std::fabs(lat[(size_t)sms[i] * L + l] - lat_rep[(size_t)sms[i] * L + l]));
    std::nth_element(diff.begin(), diff.begin() + diff.size() / 2, diff.end());
    out->noise = diff[diff.size() / 2];
    std::vector<float> allv(X.begin(), X.end());
    std::nth_element(allv.begin(), allv.begin() + allv.size() / 2, allv.end());
    const double median = allv[allv.size() / 2];
    for (int i = 0; i < S; ++i)
        for (int l = 0; l < L; ++l) X[(size_t)i * L + l] += all - rowm[i] - colm[l];
    // power iteration for the leading singular pair of X (S x L)
    std::vector<double> u(S), v(L);
    for (int l = 0; l < L; ++l) v[l] = ((l * 2654435761u) >> 16 & 1) ? 1.0 : -1.0;
    for (int it = 0; it < 60; ++it) {
        double nu = 0.0, nv = 0.0;
        for (int i = 0; i < S; ++i) {
            double a = 0.0;
            for (int l = 0; l < L; ++l) a += X[(size_t)i * L + l] * v[l];
            u[i] = a;
            nu += a * a;
        }
        nu = std::sqrt(nu) + 1e-30;
        for (auto& a : u) a /= nu;
        for (int l = 0; l < L; ++l) {
            double a = 0.0;
            for (int i = 0; i < S; ++i) a += X[(size_t)i * L + l] * u[i];
            v[l] = a;
            nv += a * a;
        }
        nv = std::sqrt(nv) + 1e-30;
        for (auto& a : v) a /= nv;
    }
    // orient: the lowest-numbered reporting SM is in domain 0
    const double sign = u[0] >= 0.0 ? 1.0 : -1.0;
    std::vector<int> dom(S), home(L);
    int n1 = 0;
    for (int i = 0; i < S; ++i) { dom[i] = (u[i] * sign >= 0.0) ? 0 : 1; n1 += dom[i]; }
    // a line is "at home" in the domain whose SMs see it faster: for domain-0 SMs the centred latency
    // is u_i * sigma * v_l with u_i * sign > 0, so the line is near domain 0 when v_l * sign < 0
    for (int l = 0; l < L; ++l) home[l] = (v[l] * sign < 0.0) ? 0 : 1;
    double near_sum = 0.0, far_sum = 0.0;
    size_t near_n = 0, far_n = 0;
    for (int i = 0; i < S; ++i)
        for (int l = 0; l < L; ++l) {
            const double val = lat[(size_t)sms[i] * L + l];
            if (dom[i] == home[l]) { near_sum += val; ++near_n; } else { far_sum += val; ++far_n; }
        }
    auto bin_of = [](double cycles) {
        int b = (int)std::floor((cycles - NUNA_HIST_FIRST) / NUNA_HIST_STEP);
        return b < 0 ? 0 : (b >= NUNA_HIST_BINS ? NUNA_HIST_BINS - 1 : b);
    };
    const bool two_sided = !(n1 == 0 || n1 == S || !near_n || !far_n);
    for (int i = 0; i < S; ++i)
        for (int l = 0; l < L; ++l) {
            const double val = lat[(size_t)sms[i] * L + l];
            if (!two_sided || dom[i] == home[l]) out->hist_near[bin_of(val)]++; else out->hist_far[bin_of(val)]++;
        }
    if (!two_sided) return;
    out->near_lat = (float)(near_sum / near_n);
    out->far_lat = (float)(far_sum / far_n);
    out->domain_gap = out->far_lat - out->near_lat;
    for (int l = 0; l < L && l < NUNA_MAX_PROBE_LINES; ++l) out->line_home[l] = (unsigned char)home[l];
    if (homes) *homes = home;
    if (!(out->domain_gap > 3.0 * out->noise && out->domain_gap > 0.03 * median)) {
        for (int b = 0; b < NUNA_HIST_BINS; ++b) { out->hist_near[b] += out->hist_far[b]; out->hist_far[b] = 0; }
    } else {
        out->verdict = NUNA_TOPO_NONUNIFORM;
        out->num_domains = 2;
        for (int i = 0; i < S; ++i) out->sm_domain[sms[i]] = dom[i];
    }
}

}  // namespace nuna

using namespace nuna;

#define PROBE_CK(call)                          \
    do {                                        \
        if ((call) != cudaSuccess) {            \
            status = NUNA_ERR_CUDA;             \
            goto done;                          \
        }                                       \
    } while (0)

extern "C" {

/* Test hook: the host-side analysis on a caller-supplied latency matrix (no GPU needed). */
int nuna_debug_analyse_topology(const float* lat, const float* lat_rep, int num_sms, int nlines, nuna_topology_t* out)
{
    if (!lat || !lat_rep || !out || num_sms < 1 || num_sms > NUNA_MAX_SMS || nlines < 1 || nlines > NUNA_MAX_PROBE_LINES)
        return NUNA_ERR_INVALID_ARG;
    memset(out, 0, sizeof *out);
    out->num_sms = num_sms;
    out->num_lines = nlines;
    for (int s = 0; s < num_sms; ++s) out->sm_reported[s] = 1;
    std::vector<float> a(lat, lat + (size_t)num_sms * nlines), b(lat_rep, lat_rep + (size_t)num_sms * nlines);
    analyse_topology(a, b, nlines, out);
    return NUNA_OK;
}

/* Test hook: the Sattolo chain used for the miss walk, and a host walk of it. */
int nuna_debug_chain(unsigned* next, int nnodes, unsigned long long seed, unsigned start, int steps, unsigned* end)
{
    if (!next || nnodes < 2 || !end) return NUNA_ERR_INVALID_ARG;
    std::vector<unsigned> nx((size_t)nnodes);
    sattolo_cycle(nx, seed);
    memcpy(next, nx.data(), (size_t)nnodes * sizeof(unsigned));
    unsigned i = start % (unsigned)nnodes;
    for (int k = 0; k < steps; ++k) i = nx[i];
    *end = i;
    return NUNA_OK;
}

int nuna_probe_topology(const void* const* bufs, const size_t* bytes, int nbufs, nuna_topology_t* out, void* stream_)
{
    if (!out || !bufs || !bytes || nbufs < 1 || nbufs > NUNA_MAX_PROBE_BUFS) return NUNA_ERR_INVALID_ARG;
    for (int b = 0; b < nbufs; ++b) {
        if (!bufs[b] || bytes[b] < 128) return NUNA_ERR_INVALID_ARG;
        if ((uintptr_t)bufs[b] & 15u) return NUNA_ERR_ALIGNMENT;
    }
    cudaStream_t stream = (cudaStream_t)stream_;
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &cs) == cudaSuccess && cs != cudaStreamCaptureStatusNone) return NUNA_ERR_CAPTURING;
    Context* c = nullptr;
    int status = get_context(&c);
    if (status != NUNA_OK) return status;
    memset(out, 0, sizeof *out);
    out->num_sms = c->num_sms;
    out->num_bufs = nbufs;
    out->num_regions = NUNA_PROBE_REGIONS;
    const int max_sms = std::min(c->num_sms, NUNA_MAX_SMS);

    // ---- sample lines: per buffer, per region, a few 128-byte lines at seeded offsets ------------------
    const int per_region = std::max(1, std::min(8, NUNA_MAX_PROBE_LINES / (nbufs * NUNA_PROBE_REGIONS)));
    std::vector<unsigned long long*> lines;
    uint64_t seed = 0x6E756E61ull;
    for (int b = 0; b < nbufs; ++b) {
        const uintptr_t lo = ((uintptr_t)bufs[b] + 127) & ~(uintptr_t)127;
        const uintptr_t hi = ((uintptr_t)bufs[b] + bytes[b]) & ~(uintptr_t)127;
        const size_t nl = hi > lo ? (hi - lo) / 128 : 0;
        for (int r = 0; r < NUNA_PROBE_REGIONS; ++r) {
            const size_t r0 = nl * r / NUNA_PROBE_REGIONS, r1 = nl * (r + 1) / NUNA_PROBE_REGIONS;
            for (int k = 0; k < per_region; ++k) {
                if (r1 <= r0 || (size_t)k >= r1 - r0) continue;     // region smaller than the sample count
                size_t pick = r0 + (size_t)(splitmix(seed) % (r1 - r0));
                unsigned long long* p = reinterpret_cast<unsigned long long*>(lo + pick * 128);
                if (std::find(lines.begin(), lines.end(), p) != lines.end()) continue;
                lines.push_back(p);
                out->line_buf[lines.size() - 1] = (unsigned char)b;
                out->line_region[lines.size() - 1] = (unsigned char)r;
            }
        }
    }
    const int nregular = (int)lines.size();
    if (nregular < 2) return NUNA_ERR_INVALID_ARG;
    out->num_lines = nregular;

    // ---- address-granularity scan of buffer 0: a window of consecutive lines, and 16 sampled lines in each of
    // up to eight consecutive blocks of 4 KiB, 64 KiB and 2 MiB.  A line is measured once; index_of maps an
    // address to its row in the latency matrix.
    std::unordered_map<uintptr_t, int> index_of;
    for (int l = 0; l < nregular; ++l) index_of[(uintptr_t)lines[l]] = l;
    auto line_index = [&](uintptr_t addr) {
        auto it = index_of.find(addr);
        if (it != index_of.end()) return it->second;
        lines.push_back(reinterpret_cast<unsigned long long*>(addr));
        index_of[addr] = (int)lines.size() - 1;
        return (int)lines.size() - 1;
    };
    static const size_t kLevelBytes[NUNA_SCAN_LEVELS] = {(size_t)4 << 10, (size_t)64 << 10, (size_t)2 << 20};
    std::vector<int> scan_idx;
    std::vector<int> level_idx[NUNA_SCAN_LEVELS][NUNA_SCAN_BLOCKS];
    {
        const uintptr_t lo = ((uintptr_t)bufs[0] + 127) & ~(uintptr_t)127;
        const uintptr_t hi = ((uintptr_t)bufs[0] + bytes[0]) & ~(uintptr_t)127;
        const size_t nl = hi > lo ? (hi - lo) / 128 : 0;
        const size_t window = std::min<size_t>(NUNA_SCAN_LINES, nl);
        for (size_t i = 0; i < window; ++i) scan_idx.push_back(line_index(lo + i * 128));
        for (int g = 0; g < NUNA_SCAN_LEVELS; ++g) {
            const size_t per_block = kLevelBytes[g] / 128;
            for (int b = 0; b < NUNA_SCAN_BLOCKS; ++b) {
                if ((size_t)(b + 1) * per_block > nl) break;
                for (int k = 0; k < 16; ++k)
                    level_idx[g][b].push_back(line_index(lo + ((size_t)b * per_block + (size_t)(splitmix(seed) % per_block)) * 128));
            }
        }
    }
    const int L = (int)lines.size();

    // ---- device scratch ---------------------------------------------------------------------------------
    unsigned long long** d_lines = nullptr;
    unsigned long long* d_saved = nullptr;
    float *d_lat = nullptr, *d_miss = nullptr, *d_gbs = nullptr;
    int* d_seen = nullptr;
    unsigned *d_bad = nullptr, *d_next = nullptr, *d_starts = nullptr, *d_ends = nullptr;
    unsigned char *d_chain = nullptr, *d_flush = nullptr;
    const int nnodes = (int)std::max<size_t>(4096, std::min<size_t>(32768, c->l2_bytes / kNodeStride));
    const size_t flush_bytes = c->l2_bytes + (c->l2_bytes >> 2);
    const size_t smem_one_per_sm = 120 * 1024;
    std::vector<float> lat0((size_t)max_sms * L), lat1((size_t)max_sms * L), miss(max_sms, 0.f), gbs(max_sms, 0.f);
    std::vector<int> seen(max_sms, 0);
    std::vector<unsigned> next((size_t)nnodes), starts(c->num_sms), ends(c->num_sms, 0);
    unsigned bad = 0;
    bool words_replaced = false;

    PROBE_CK(cudaMalloc(&d_lines, sizeof(void*) * L));
    PROBE_CK(cudaMalloc(&d_saved, sizeof(unsigned long long) * L));
    PROBE_CK(cudaMalloc(&d_lat, sizeof(float) * (size_t)max_sms * L));
    PROBE_CK(cudaMalloc(&d_miss, sizeof(float) * max_sms));
    PROBE_CK(cudaMalloc(&d_gbs, sizeof(float) * max_sms));
    PROBE_CK(cudaMalloc(&d_seen, sizeof(int) * max_sms));
    PROBE_CK(cudaMalloc(&d_bad, sizeof(unsigned)));
    PROBE_CK(cudaMalloc(&d_next, sizeof(unsigned) * nnodes));
    PROBE_CK(cudaMalloc(&d_starts, sizeof(unsigned) * c->num_sms));
    PROBE_CK(cudaMalloc(&d_ends, sizeof(unsigned) * c->num_sms));
    PROBE_CK(cudaMalloc(&d_chain, (size_t)nnodes * kNodeStride));
    PROBE_CK(cudaMalloc(&d_flush, flush_bytes));
    PROBE_CK(cudaFuncSetAttribute(k_probe_hit, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_one_per_sm));
    PROBE_CK(cudaFuncSetAttribute(k_probe_miss, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_one_per_sm));
    PROBE_CK(cudaFuncSetAttribute(k_probe_bw, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_one_per_sm));
    PROBE_CK(cudaMemsetAsync(d_gbs, 0, sizeof(float) * max_sms, stream));
    PROBE_CK(cudaMemcpyAsync(d_lines, lines.data(), sizeof(void*) * L, cudaMemcpyHostToDevice, stream));
    PROBE_CK(cudaMemsetAsync(d_bad, 0, sizeof(unsigned), stream));
    PROBE_CK(cudaMemsetAsync(d_miss, 0, sizeof(float) * max_sms, stream));

    // ---- hit latency, two repetitions ---------------------------------------------------------------------
    k_probe_words<<<(L + 127) / 128, 128, 0, stream>>>(d_lines, d_saved, L, 0);
    words_replaced = true;
    for (int rep = 0; rep < 2; ++rep) {
        PROBE_CK(cudaMemsetAsync(d_seen, 0, sizeof(int) * max_sms, stream));
        PROBE_CK(cudaMemsetAsync(d_lat, 0, sizeof(float) * (size_t)max_sms * L, stream));
        k_probe_hit<<<c->num_sms, 32, smem_one_per_sm, stream>>>(d_lines, L, d_lat, d_seen, max_sms, d_bad);
        PROBE_CK(cudaMemcpyAsync(rep ? lat1.data() : lat0.data(), d_lat, sizeof(float) * (size_t)max_sms * L,
                                 cudaMemcpyDeviceToHost, stream));
        if (rep == 0) PROBE_CK(cudaMemcpyAsync(seen.data(), d_seen, sizeof(int) * max_sms, cudaMemcpyDeviceToHost, stream));
    }
    k_probe_words<<<(L + 127) / 128, 128, 0, stream>>>(d_lines, d_saved, L, 1);
    words_replaced = false;
    g_launches.fetch_add(4, std::memory_order_relaxed);

    // ---- miss latency: cold walk of a single-cycle permutation -----------------------------------------------
    sattolo_cycle(next, 0x70726F6265ull);
    {
        // SM block b starts kMissSteps * b nodes along the cycle, so the segments are disjoint
        unsigned i = 0;
        for (int b = 0; b < c->num_sms; ++b) {
            starts[b] = i;
            for (int k = 0; k < kMissSteps; ++k) i = next[i];
        }
    }
    PROBE_CK(cudaMemcpyAsync(d_next, next.data(), sizeof(unsigned) * nnodes, cudaMemcpyHostToDevice, stream));
    PROBE_CK(cudaMemcpyAsync(d_starts, starts.data(), sizeof(unsigned) * c->num_sms, cudaMemcpyHostToDevice, stream));
    k_chain_write<<<(nnodes + 255) / 256, 256, 0, stream>>>(d_chain, d_next, nnodes);
    k_flush<<<c->num_sms * 4, 256, 0, stream>>>(reinterpret_cast<uint4*>(d_flush), flush_bytes / 16);
    k_probe_miss<<<c->num_sms, 32, smem_one_per_sm, stream>>>(d_chain, d_starts, d_miss, d_ends, max_sms);
    g_launches.fetch_add(3, std::memory_order_relaxed);
    // ---- solo streaming read rate, one SM after the other (the window is the start of the flush region) ---------
    for (int s = 0; s < max_sms; ++s)
        k_probe_bw<<<c->num_sms, 256, smem_one_per_sm, stream>>>(reinterpret_cast<const uint4*>(d_flush), 65536u, (unsigned)s, 4, d_gbs,
                                                                  max_sms);
    g_launches.fetch_add((unsigned long long)max_sms, std::memory_order_relaxed);
    PROBE_CK(cudaMemcpyAsync(gbs.data(), d_gbs, sizeof(float) * max_sms, cudaMemcpyDeviceToHost, stream));
    PROBE_CK(cudaMemcpyAsync(miss.data(), d_miss, sizeof(float) * max_sms, cudaMemcpyDeviceToHost, stream));
    PROBE_CK(cudaMemcpyAsync(ends.data(), d_ends, sizeof(unsigned) * c->num_sms, cudaMemcpyDeviceToHost, stream));
    PROBE_CK(cudaMemcpyAsync(&bad, d_bad, sizeof(unsigned), cudaMemcpyDeviceToHost, stream));
    PROBE_CK(cudaStreamSynchronize(stream));
    PROBE_CK(cudaGetLastError());

    // ---- host analysis --------------------------------------------------------------------------------------------
    {
        int reported = 0;
        for (int s = 0; s < max_sms; ++s) {
            out->sm_reported[s] = seen[s] > 0;
            reported += seen[s] > 0;
            out->sm_lat_miss[s] = miss[s];
            out->sm_read_gbs[s] = gbs[s];
        }
        out->sms_reported = reported;
        out->self_pointer_mismatches = (int)bad;
        // the device walk must end where the host walk of the same permutation ends
        int walk_ok = 1;
        for (int b = 0; b < c->num_sms; ++b) {
            unsigned i = starts[b];
            for (int k = 0; k < kMissSteps; ++k) i = next[i];
            if (i != ends[b]) walk_ok = 0;
        }
        out->chain_walk_ok = walk_ok;
        out->chain_nodes = nnodes;
        out->chain_steps = kMissSteps;
        std::vector<int> homes;
        analyse_topology(lat0, lat1, L, out, &homes);
        out->num_lines = nregular;
        // granularity scan: runs of equal home among the consecutive lines, home shares per block size
        for (int g = 0; g < NUNA_SCAN_LEVELS; ++g) {
            out->scan_level_spread[g] = -1.f;
            for (int b = 0; b < NUNA_SCAN_BLOCKS; ++b) out->scan_level_share[g][b] = -1.f;
        }
        if (out->verdict == NUNA_TOPO_NONUNIFORM && (int)homes.size() == L) {
            out->scan_lines = (int)scan_idx.size();
            int run = 0;
            for (size_t i = 0; i < scan_idx.size(); ++i) {
                out->scan_home[i] = (unsigned char)homes[scan_idx[i]];
                ++run;
                if (i + 1 == scan_idx.size() || homes[scan_idx[i + 1]] != homes[scan_idx[i]]) {
                    int bin = 0;
                    while ((2 << bin) <= run && bin < NUNA_SCAN_RUN_BINS - 1) ++bin;     // 2^bin <= run < 2^(bin+1)
                    out->scan_run_hist[bin]++;
                    out->scan_longest_run = std::max(out->scan_longest_run, run);
                    run = 0;
                }
            }
            for (int g = 0; g < NUNA_SCAN_LEVELS; ++g) {
                float mn = 2.f, mx = -1.f;
                int blocks = 0;
                for (int b = 0; b < NUNA_SCAN_BLOCKS; ++b) {
                    if (level_idx[g][b].empty()) continue;
                    int h0 = 0;
                    for (int li : level_idx[g][b]) h0 += homes[li] == 0;
                    const float share = (float)h0 / (float)level_idx[g][b].size();
                    out->scan_level_share[g][b] = share;
                    mn = std::min(mn, share);
                    mx = std::max(mx, share);
                    ++blocks;
                }
                if (blocks >= 2) out->scan_level_spread[g] = mx - mn;
            }
        }
        // per (SM, buffer, region) mean hit latency and per (buffer, region) share of lines at home in domain 0
        std::vector<int> cnt((size_t)NUNA_MAX_PROBE_BUFS * NUNA_PROBE_REGIONS, 0), home0(cnt.size(), 0);
        for (int l = 0; l < nregular; ++l) {
            const int idx = out->line_buf[l] * NUNA_PROBE_REGIONS + out->line_region[l];
            cnt[idx]++;
            home0[idx] += out->line_home[l] == 0;
        }
        for (int b = 0; b < nbufs; ++b)
            for (int r = 0; r < NUNA_PROBE_REGIONS; ++r) {
                const int idx = b * NUNA_PROBE_REGIONS + r;
                out->region_home0[b][r] = cnt[idx] ? (float)home0[idx] / cnt[idx] : -1.f;
            }
        for (int s = 0; s < max_sms; ++s) {
            if (!out->sm_reported[s]) continue;
            float sum[NUNA_MAX_PROBE_BUFS] = {};
            int n[NUNA_MAX_PROBE_BUFS] = {};
            for (int l = 0; l < nregular; ++l) { sum[out->line_buf[l]] += lat0[(size_t)s * L + l]; n[out->line_buf[l]]++; }
            for (int b = 0; b < nbufs; ++b) out->lat_hit[s][b] = n[b] ? sum[b] / n[b] : -1.f;
        }
        std::lock_guard<std::mutex> lock(c->mutex);
        c->topology = *out;
        c->have_topology = true;
        // work lists planned under the previous topology are stale: retire them (kept allocated until
        // shutdown, because captured graphs may still name them) and rebuild on the next call of each shape
        for (auto& kv : c->sm_plans) c->retired_plans.push_back(kv.second.base);
        c->sm_plans.clear();
    }

done:
    if (words_replaced && d_lines && d_saved) {
        k_probe_words<<<(L + 127) / 128, 128, 0, stream>>>(d_lines, d_saved, L, 1);
        cudaStreamSynchronize(stream);
    }
    cudaFree(d_lines); cudaFree(d_saved); cudaFree(d_lat); cudaFree(d_miss); cudaFree(d_gbs); cudaFree(d_seen); cudaFree(d_bad);
    cudaFree(d_next); cudaFree(d_starts); cudaFree(d_ends); cudaFree(d_chain); cudaFree(d_flush);
    return status;
}

}  // extern "C"
