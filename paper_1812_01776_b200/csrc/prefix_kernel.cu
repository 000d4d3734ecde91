// Sharing simulation work between candidates with a common configuration prefix.
//
// The pipeline is a feed-forward tree with zero delay, so the completion stream
// of a stage depends only on the configurations of the stages on its path from
// the root (Section 4.2: the Estimator's result is a function of configuration,
// profiles and trace).  Two candidates that agree on all of those stages have
// the same stream there.  The Planner's candidate sets are full of such pairs:
// every action of Algorithm 2 changes ONE model of the current plan, and an
// exhaustive sweep is a product of per-stage choices.
//
// A NODE is a distinct (stage, configuration of the stage, node of the parent
// stage) triple.  This file builds the nodes of a candidate batch on the
// device, one stage after the other in index order (a parent has a smaller
// index than its children):
//
//   insert   every candidate puts the key (parent node, hw, max batch, replicas)
//            of its stage-s configuration into an open-addressing hash table
//            and remembers the slot;
//   number   every occupied slot gets the next node id of the stage and
//            records the node's configuration and parent;
//   lookup   every candidate reads its node id back through its slot.
//
// The nodes are then simulated once each, level by level, by the stage loops of
// the warp-per-candidate kernel (des_packed_kernel.cu), and a candidate's P99
// and miss count are put together from the nodes where its queries leave the
// pipeline (select_kernel.cu, combine step below).
#include "il_internal.h"

#include <algorithm>

namespace il {

namespace {

constexpr uint64_t kEmpty = ~0ull;

__device__ __forceinline__ uint64_t mix64(uint64_t x)
{
    x ^= x >> 33; x *= 0xff51afd7ed558ccdull;
    x ^= x >> 33; x *= 0xc4ceb9fe1a85ec53ull;
    x ^= x >> 33;
    return x;
}

// keys[cap] must be all kEmpty.  slot_of[c] receives the slot of candidate c's key.
__global__ void __launch_bounds__(256)
prefix_insert_kernel(const il_stage_config *configs, int64_t n_cand, int S, int s, int H, int Bmax,
                     const int32_t *parent_node, uint64_t *keys, uint32_t cap_mask, int32_t *slot_of, int *status)
{
    for (int64_t c = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; c < n_cand; c += (int64_t)gridDim.x * blockDim.x) {
        const il_stage_config cfg = configs[c * S + s];
        if (cfg.hw >= H || cfg.max_batch < 1 || cfg.max_batch > Bmax || cfg.replicas < 1 ||
            cfg.replicas > IL_MAX_REPLICAS) {
            atomicCAS(status, 0, IL_ERR_BAD_CONFIG);
            slot_of[c] = 0;
            continue;
        }
        const uint64_t par = parent_node ? (uint64_t)(uint32_t)parent_node[c] : 0ull;
        const uint64_t key = (par << 24) | ((uint64_t)cfg.replicas << 16) | ((uint64_t)cfg.max_batch << 8) | cfg.hw;
        uint32_t slot = (uint32_t)mix64(key) & cap_mask;
        // the table has at least twice as many slots as there are candidates, so a probe sequence ends
        for (uint32_t probes = 0; probes <= cap_mask; probes++) {
            const uint64_t seen = atomicCAS(reinterpret_cast<unsigned long long *>(keys + slot), kEmpty, key);
            if (seen == kEmpty || seen == key) break;
            slot = (slot + 1u) & cap_mask;
        }
        slot_of[c] = (int32_t)slot;
    }
}

// Numbers the occupied slots (any order) and records what each node is.
__global__ void __launch_bounds__(256)
prefix_number_kernel(const uint64_t *keys, uint32_t cap, int32_t *vals, int *count, uint32_t *node_cfg,
                     int32_t *node_parent)
{
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < cap; i += gridDim.x * blockDim.x) {
        const uint64_t key = keys[i];
        if (key == kEmpty) continue;
        const int id = atomicAdd(count, 1);
        vals[i] = id;
        node_cfg[id] = (uint32_t)key & 0xffffffu;
        node_parent[id] = (int32_t)(key >> 24);
    }
}

// node_of[c] = id of candidate c's node; clears the slots that were used on the way (the table is
// reused by the next stage).
__global__ void __launch_bounds__(256)
prefix_lookup_kernel(const int32_t *slot_of, const int32_t *vals, int64_t n_cand, int32_t *node_of)
{
    for (int64_t c = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; c < n_cand; c += (int64_t)gridDim.x * blockDim.x)
        node_of[c] = vals[slot_of[c]];
}

// ---- covering candidates ------------------------------------------------------------------------
// The nodes can be simulated by the lane kernel, which only knows whole candidates: pick a set of
// candidates of the batch that between them contain every node that queries leave after (the
// candidate with the smallest index for each such node), simulate those, and read each node's leaving
// records from the slab row of its candidate.

// rep[k] = smallest candidate index whose node of this stage is k (rep filled with a large value).
__global__ void __launch_bounds__(256)
cover_rep_kernel(const int32_t *node_of, int64_t n_cand, int32_t *rep)
{
    for (int64_t c = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; c < n_cand; c += (int64_t)gridDim.x * blockDim.x)
        atomicMin(&rep[node_of[c]], (int32_t)c);
}

__global__ void __launch_bounds__(256)
cover_mark_kernel(const int32_t *rep, int64_t n_nodes, uint8_t *flags)
{
    for (int64_t k = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; k < n_nodes; k += (int64_t)gridDim.x * blockDim.x)
        flags[rep[k]] = 1;
}

// The marked candidates, in any order: list[i] = candidate, pos[candidate] = i.
__global__ void __launch_bounds__(256)
cover_list_kernel(const uint8_t *flags, int64_t n_cand, int32_t *list, int32_t *pos, int *count)
{
    for (int64_t c = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; c < n_cand; c += (int64_t)gridDim.x * blockDim.x) {
        if (!flags[c]) continue;
        const int i = atomicAdd(count, 1);
        list[i] = (int32_t)c;
        pos[c] = i;
    }
}

// row[k] = slab row of the candidate that stands for node k.
__global__ void __launch_bounds__(256)
cover_rows_kernel(const int32_t *rep, const int32_t *pos, int64_t n_nodes, int32_t *row)
{
    for (int64_t k = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; k < n_nodes; k += (int64_t)gridDim.x * blockDim.x)
        row[k] = pos[rep[k]];
}

// P99 and miss count of every candidate from the nodes where its queries leave the pipeline.
// Node i of leaving stage e has its `top` largest latencies in top_e[i][0 .. top), sorted in
// descending order (entries beyond the node's own count are 0, below every latency), and its miss
// count in miss_e[i].  A candidate's latencies are the union over its leaving nodes, so with
// T = n - k queries allowed above the answer, P99 (the k-th smallest of n) is the (T + 1)-th largest
// of the union: the smallest value v such that at most T elements are greater than v.
__global__ void __launch_bounds__(128)
prefix_combine_kernel(const __grid_constant__ CombineParams p)
{
    for (int64_t c = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; c < p.n_cand; c += (int64_t)gridDim.x * blockDim.x) {
        const int64_t *list[IL_MAX_STAGES];
        int64_t miss = 0, hi = 0;
#pragma unroll
        for (int e = 0; e < IL_MAX_STAGES; e++) {
            if (e < p.n_exit) {
                const int64_t node = p.node_of[(int64_t)p.exit_stage[e] * p.n_cand + c];
                list[e] = p.top[e] + node * p.top_len;
                miss += p.miss[e][node];
                hi = max(hi, list[e][0]);
            }
        }
        int64_t lo = 0;     // invariant: more than T elements are > lo - 1 ... found by bisection on v
        // smallest v in [0, hi] with count(> v) <= T
        while (lo < hi) {
            const int64_t mid = lo + ((hi - lo) >> 1);
            int64_t above = 0;
#pragma unroll
            for (int e = 0; e < IL_MAX_STAGES; e++) {
                if (e < p.n_exit) {
                    // first position whose value is <= mid (the list is descending)
                    int a = 0, b = p.top_len;
                    while (a < b) {
                        const int m = (a + b) >> 1;
                        if (list[e][m] > mid) a = m + 1; else b = m;
                    }
                    above += a;
                }
            }
            if (above <= p.allowed) hi = mid; else lo = mid + 1;
        }
        p.out_p99[c] = lo;
        p.out_miss[c] = miss;
    }
}

}  // namespace

cudaError_t launch_prefix_stage(const il_stage_config *configs, int64_t n_cand, int S, int s, int H, int Bmax,
                                const int32_t *parent_node, uint64_t *keys, uint32_t cap, int32_t *vals,
                                int32_t *slot_of, int *count, uint32_t *node_cfg, int32_t *node_parent,
                                int32_t *node_of, int *status, cudaStream_t stream)
{
    cudaError_t e = cudaMemsetAsync(keys, 0xff, (size_t)cap * 8, stream);
    if (e != cudaSuccess) return e;
    const int grid_c = (int)std::min<int64_t>((n_cand + 255) / 256, 2368);
    const int grid_t = (int)std::min<int64_t>(((int64_t)cap + 255) / 256, 2368);
    prefix_insert_kernel<<<grid_c, 256, 0, stream>>>(configs, n_cand, S, s, H, Bmax, parent_node, keys, cap - 1u,
                                                     slot_of, status);
    prefix_number_kernel<<<grid_t, 256, 0, stream>>>(keys, cap, vals, count, node_cfg, node_parent);
    prefix_lookup_kernel<<<grid_c, 256, 0, stream>>>(slot_of, vals, n_cand, node_of);
    return cudaGetLastError();
}

static int cover_grid(int64_t items) { return (int)std::max<int64_t>(1, std::min<int64_t>((items + 255) / 256, 2368)); }

cudaError_t launch_cover_rep(const int32_t *node_of, int64_t n_cand, int32_t *rep, int64_t n_nodes, uint8_t *flags,
                             cudaStream_t stream)
{
    cudaError_t e = cudaMemsetAsync(rep, 0x7f, (size_t)n_nodes * 4, stream);
    if (e != cudaSuccess) return e;
    cover_rep_kernel<<<cover_grid(n_cand), 256, 0, stream>>>(node_of, n_cand, rep);
    cover_mark_kernel<<<cover_grid(n_nodes), 256, 0, stream>>>(rep, n_nodes, flags);
    return cudaGetLastError();
}

cudaError_t launch_cover_list(const uint8_t *flags, int64_t n_cand, int32_t *list, int32_t *pos, int *count,
                              cudaStream_t stream)
{
    cover_list_kernel<<<cover_grid(n_cand), 256, 0, stream>>>(flags, n_cand, list, pos, count);
    return cudaGetLastError();
}

cudaError_t launch_cover_rows(const int32_t *rep, const int32_t *pos, int64_t n_nodes, int32_t *row, cudaStream_t stream)
{
    cover_rows_kernel<<<cover_grid(n_nodes), 256, 0, stream>>>(rep, pos, n_nodes, row);
    return cudaGetLastError();
}

cudaError_t launch_prefix_combine(const CombineParams &p, cudaStream_t stream)
{
    const int grid = (int)std::min<int64_t>((p.n_cand + 127) / 128, 148 * 16);
    prefix_combine_kernel<<<grid, 128, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace il
