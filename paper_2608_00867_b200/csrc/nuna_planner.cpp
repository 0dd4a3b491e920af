// NUNA-aware placement (the paper's Algorithm 1, Section 4.2) as a host-side planner.
//
// Input: a workload W of thread blocks, each with the chunks it touches; a topology (which domain
// each compute unit belongs to, its preference rank inside the domain, its nearest HBM stack);
// per-CU and per-stack budgets R_max in bytes; the number of domains nar_max.
// logical_allocation (Section 4.2.1) walks the blocks in order: a block none of whose chunks is
// owned yet opens a new group; otherwise it joins the group that already owns most of its chunks
// (ties: the group created first) and brings its unowned chunks along.  Groups are sorted by
// decreasing chunk bytes (stable) and dealt to the domains round-robin, first group to domain 0.
// physical_placement (Section 4.2.2) gives each block the first CU of its domain, in preference
// order, whose remaining budget covers the block's chunk bytes (if none: the CU with most budget
// left, earliest in preference order on ties), and a stack: the CU's nearest one if it has budget,
// else the remaining stacks in increasing index, else the one with most budget left.  A chunk keeps
// the first stack it was given.  Budgets are per (gpu, CU) and per (gpu, stack).
#include <algorithm>
#include <cstdint>
#include <numeric>
#include <vector>

#include "../../include/nuna.h"

namespace {

struct Group {
    std::vector<int> tbs;
    long long bytes = 0;
};

}  // namespace

extern "C" int nuna_plan_placement(const nuna_plan_input_t* in, int* m_compute, int* m_memory, int* tb_domain,
                                   int* tb_group)
{
    if (!in || !m_compute) return NUNA_ERR_INVALID_ARG;
    const int T = in->num_tbs, C = in->num_chunks, U = in->num_cus, S = in->num_stacks, D = in->nar_max;
    if (T < 0 || C < 0 || U < 1 || S < 1 || D < 1) return NUNA_ERR_INVALID_ARG;
    if (!in->tb_chunk_begin || (T > 0 && !in->tb_gpu) || !in->cu_domain || !in->cu_rank || !in->cu_stack ||
        (C > 0 && (!in->chunk_bytes || !in->tb_chunks)))
        return NUNA_ERR_INVALID_ARG;
    int num_gpus = 1;
    for (int t = 0; t < T; ++t) {
        if (in->tb_gpu[t] < 0 || in->tb_chunk_begin[t] > in->tb_chunk_begin[t + 1]) return NUNA_ERR_INVALID_ARG;
        num_gpus = std::max(num_gpus, in->tb_gpu[t] + 1);
        for (int k = in->tb_chunk_begin[t]; k < in->tb_chunk_begin[t + 1]; ++k)
            if (in->tb_chunks[k] < 0 || in->tb_chunks[k] >= C) return NUNA_ERR_INVALID_ARG;
    }
    // CUs of each domain in preference order (rank ascending, CU index on ties)
    std::vector<std::vector<int>> dom_cus(D);
    for (int u = 0; u < U; ++u) {
        if (in->cu_domain[u] < 0 || in->cu_domain[u] >= D || in->cu_stack[u] < 0 || in->cu_stack[u] >= S)
            return NUNA_ERR_INVALID_ARG;
        dom_cus[in->cu_domain[u]].push_back(u);
    }
    for (auto& v : dom_cus) {
        if (v.empty()) return NUNA_ERR_INVALID_ARG;
        std::stable_sort(v.begin(), v.end(), [&](int a, int b) { return in->cu_rank[a] < in->cu_rank[b]; });
    }

    // ---- logical_allocation ------------------------------------------------------------------------
    std::vector<int> owner(C, -1);
    std::vector<Group> groups;
    std::vector<int> tb_grp(T, -1);
    std::vector<int> share;
    for (int t = 0; t < T; ++t) {
        share.assign(groups.size(), 0);
        int best = -1, best_n = 0;
        for (int k = in->tb_chunk_begin[t]; k < in->tb_chunk_begin[t + 1]; ++k) {
            const int g = owner[in->tb_chunks[k]];
            if (g >= 0) ++share[g];
        }
        for (int g = 0; g < (int)groups.size(); ++g)
            if (share[g] > best_n) { best_n = share[g]; best = g; }       // strict '>' keeps the oldest on ties
        if (best < 0) {
            best = (int)groups.size();
            groups.emplace_back();
        }
        groups[best].tbs.push_back(t);
        tb_grp[t] = best;
        for (int k = in->tb_chunk_begin[t]; k < in->tb_chunk_begin[t + 1]; ++k) {
            const int c = in->tb_chunks[k];
            if (owner[c] < 0) {
                owner[c] = best;
                groups[best].bytes += in->chunk_bytes[c];
            }
        }
    }
    std::vector<int> order(groups.size());
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return groups[a].bytes > groups[b].bytes; });

    // ---- round-robin over domains + physical_placement ------------------------------------------------
    std::vector<long long> r_cu((size_t)num_gpus * U, in->r_max_cu), r_stack((size_t)num_gpus * S, in->r_max_stack);
    if (m_memory) std::fill(m_memory, m_memory + C, -1);
    std::vector<int> chunk_stack(C, -1);
    int nar = 0;
    for (size_t gi = 0; gi < order.size(); ++gi) {
        const Group& grp = groups[order[gi]];
        for (int t : grp.tbs) {
            const int gpu = in->tb_gpu[t];
            long long cs = 0;
            for (int k = in->tb_chunk_begin[t]; k < in->tb_chunk_begin[t + 1]; ++k) cs += in->chunk_bytes[in->tb_chunks[k]];
            const std::vector<int>& cus = dom_cus[nar];
            int cu = -1;
            for (int u : cus)
                if (r_cu[(size_t)gpu * U + u] >= cs) { cu = u; break; }
            if (cu < 0) {
                cu = cus[0];
                for (int u : cus)
                    if (r_cu[(size_t)gpu * U + u] > r_cu[(size_t)gpu * U + cu]) cu = u;
            }
            int stack = -1;
            const int nearest = in->cu_stack[cu];
            if (r_stack[(size_t)gpu * S + nearest] >= cs) stack = nearest;
            for (int s = 0; s < S && stack < 0; ++s)
                if (s != nearest && r_stack[(size_t)gpu * S + s] >= cs) stack = s;
            if (stack < 0) {
                stack = nearest;
                for (int s = 0; s < S; ++s) {
                    if (s == nearest) continue;
                    // preference order is nearest first, then increasing index: strict '>' keeps the earlier one
                    if (r_stack[(size_t)gpu * S + s] > r_stack[(size_t)gpu * S + stack]) stack = s;
                }
            }
            r_cu[(size_t)gpu * U + cu] -= cs;
            r_stack[(size_t)gpu * S + stack] -= cs;
            m_compute[t] = cu;
            if (tb_domain) tb_domain[t] = nar;
            if (tb_group) tb_group[t] = (int)gi;
            for (int k = in->tb_chunk_begin[t]; k < in->tb_chunk_begin[t + 1]; ++k) {
                const int c = in->tb_chunks[k];
                if (chunk_stack[c] < 0) chunk_stack[c] = stack;
            }
        }
        nar = (nar + 1) % D;
    }
    if (m_memory) std::copy(chunk_stack.begin(), chunk_stack.end(), m_memory);
    return NUNA_OK;
}
