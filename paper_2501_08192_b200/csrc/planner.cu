// Prefetch operator insertion as a graph pass (Algorithm 1, "Prefetch Operator Insertion").
//
// The pass visits every communication operator of an operator graph, walks its successors
// breadth-first until the next communication operator (or the end of the graph), and inserts a
// prefetch beside the communication operator for every MatMul (its weights) and SelfAttention
// (its cached K and V) node it meets while the running sum of their sizes stays below the L2
// budget C (Section 3, "L2 capacity requirements").  Host code only; no device work.
//
// Readings where the listing and the prose leave a choice: the comparison is strict
// (cacheSum < C); a node that does not fit is not inserted and ends the walk for this
// communication operator; the walk also ends when no successors remain; other node kinds add
// nothing and are walked through.  PRESERVE_PLAN_TRUNCATE (not in the paper) inserts the leading
// bytes of the first node that does not fit, rounded down to 128, before the walk ends.
#include <cstdint>
#include <deque>
#include <vector>

#include "../../include/preserve.h"
#include "kernels.h"

namespace prsv {

int plan_graph(int n_nodes, const int32_t *kind, const uint64_t *mem_bytes, const int32_t *succ_off,
               const int32_t *succ, uint64_t budget, int mode, std::vector<PlanHit> &out)
{
    out.clear();
    if (n_nodes < 0)
        return PRESERVE_EINVAL;
    for (int i = 0; i < n_nodes; ++i) {
        if (kind[i] < PRESERVE_NODE_COMM || kind[i] > PRESERVE_NODE_OTHER)
            return PRESERVE_EINVAL;
        if (succ_off[i] < 0 || succ_off[i + 1] < succ_off[i])
            return PRESERVE_EINVAL;
        for (int e = succ_off[i]; e < succ_off[i + 1]; ++e)
            if (succ[e] < 0 || succ[e] >= n_nodes)
                return PRESERVE_EINVAL;
    }
    std::vector<int> seen_by((size_t)n_nodes, -1);      // last communication op whose walk queued the node
    std::deque<int> queue;
    for (int op = 0; op < n_nodes; ++op) {
        if (kind[op] != PRESERVE_NODE_COMM)
            continue;
        uint64_t cache_sum = 0;
        bool reached_end = false;
        queue.clear();
        seen_by[op] = op;
        auto push_successors = [&](int node) {
            for (int e = succ_off[node]; e < succ_off[node + 1]; ++e)
                if (seen_by[succ[e]] != op) {
                    seen_by[succ[e]] = op;
                    queue.push_back(succ[e]);
                }
        };
        push_successors(op);
        while (!reached_end && !queue.empty()) {
            const int node = queue.front();
            queue.pop_front();
            if (kind[node] == PRESERVE_NODE_COMM) {
                reached_end = true;                       // the next communication operator ends the walk
                continue;
            }
            if (kind[node] == PRESERVE_NODE_MATMUL || kind[node] == PRESERVE_NODE_ATTENTION) {
                const uint64_t mem = mem_bytes[node];
                if (cache_sum + mem < budget) {
                    cache_sum += mem;
                    out.push_back({op, node, mem});
                } else {
                    if (mode == PRESERVE_PLAN_TRUNCATE) {
                        const uint64_t room = budget > cache_sum ? budget - cache_sum : 0;
                        uint64_t part = room & ~uint64_t(127);
                        if (part > mem)
                            part = mem;
                        if (part)
                            out.push_back({op, node, part});
                    }
                    reached_end = true;
                    continue;
                }
            }
            push_successors(node);
        }
    }
    return PRESERVE_OK;
}

}  // namespace prsv

extern "C" int preserve_plan_graph(int32_t n_nodes, const int32_t *kind, const uint64_t *mem_bytes,
                                   const int32_t *succ_off, const int32_t *succ, uint64_t budget, int32_t mode,
                                   int32_t max_out, int32_t *out_comm, int32_t *out_node, uint64_t *out_bytes,
                                   int32_t *n_out)
{
    if (!n_out || n_nodes < 0 || max_out < 0 || (n_nodes > 0 && (!kind || !mem_bytes || !succ_off)) ||
        (max_out > 0 && (!out_comm || !out_node || !out_bytes)))
        return PRESERVE_EINVAL;
    if (mode != PRESERVE_PLAN_WHOLE_NODE && mode != PRESERVE_PLAN_TRUNCATE)
        return PRESERVE_EINVAL;
    if (n_nodes > 0 && succ_off[n_nodes] > 0 && !succ)
        return PRESERVE_EINVAL;
    std::vector<prsv::PlanHit> hits;
    const int rc = prsv::plan_graph(n_nodes, kind, mem_bytes, succ_off, succ, budget, mode, hits);
    if (rc != PRESERVE_OK)
        return rc;
    *n_out = (int32_t)hits.size();
    if ((int32_t)hits.size() > max_out)
        return PRESERVE_ETOOBIG;
    for (size_t i = 0; i < hits.size(); ++i) {
        out_comm[i] = hits[i].comm;
        out_node[i] = hits[i].node;
        out_bytes[i] = hits[i].bytes;
    }
    return PRESERVE_OK;
}
