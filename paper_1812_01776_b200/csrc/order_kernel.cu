// Scheduling order of a chunk of candidates: costliest first.
//
// One warp simulates one candidate from start to end, and candidates differ in
// cost by more than an order of magnitude (a lightly loaded stage dispatches
// about one batch per query, an overloaded stage with a large max batch one
// batch per max-batch queries), so the kernel's run time is set by how the long
// candidates are spread over the warps.  Warps take candidates from a shared
// counter; handing out the costliest first is the classic longest-processing-
// time-first rule.  The cost is a rough estimate from the configuration and the
// mean arrival rate; it only affects the order, never a result.
#include "il_internal.h"

namespace il {

namespace {

constexpr int kOrderThreads = 1024;
constexpr int kBuckets = 1024;

__device__ float candidate_cost(const OrderParams &p, const il_stage_config *cfg)
{
    float cost = 0.f;
    for (int s = 0; s < p.S; s++) {
        const float n = (float)p.n_s[s];
        if (n == 0.f) continue;
        const int hw = cfg[s].hw < p.H ? cfg[s].hw : 0;
        const int mb = cfg[s].max_batch >= 1 && cfg[s].max_batch <= p.Bmax ? cfg[s].max_batch : 1;
        const float R = (float)(cfg[s].replicas >= 1 ? cfg[s].replicas : 1);
        const int32_t *row = p.lat + (s * p.H + hw) * p.Bmax;
        if (mb == 1) { cost += 3.f * n; continue; }            // scan: a few instructions per query
        const float rate = n / p.span_us;                       // queries per microsecond
        // smallest batch size that keeps up with the arrival rate
        int b = 1;
        while (b < mb && rate * (float)row[b - 1] > 0.8f * R * (float)b) b++;
        // about one dispatch per b queries; single dispatches mostly go through the cheaper run step
        cost += (b == 1 ? 30.f : 90.f / (float)b + 4.f) * n;
    }
    return cost;
}

__global__ void __launch_bounds__(kOrderThreads) order_kernel(const __grid_constant__ OrderParams p)
{
    __shared__ unsigned hist[kBuckets];
    __shared__ unsigned start[kBuckets];
    float total = 0.f;
    for (int s = 0; s < p.S; s++) total += 90.f * (float)p.n_s[s];
    const float scale = (float)(kBuckets - 1) / fmaxf(total, 1.f);
    for (int i = threadIdx.x; i < kBuckets; i += kOrderThreads) hist[i] = 0;
    __syncthreads();
    for (int64_t c = threadIdx.x; c < p.n_cand; c += kOrderThreads) {
        const int b = kBuckets - 1 - min(kBuckets - 1, (int)(candidate_cost(p, p.configs + c * p.S) * scale));
        atomicAdd(&hist[b], 1u);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned acc = 0;
        for (int i = 0; i < kBuckets; i++) { start[i] = acc; acc += hist[i]; }
    }
    __syncthreads();
    for (int64_t c = threadIdx.x; c < p.n_cand; c += kOrderThreads) {
        const int b = kBuckets - 1 - min(kBuckets - 1, (int)(candidate_cost(p, p.configs + c * p.S) * scale));
        p.order[atomicAdd(&start[b], 1u)] = (int32_t)c;
    }
}

}  // namespace

cudaError_t launch_order(const OrderParams &p, cudaStream_t stream)
{
    order_kernel<<<1, kOrderThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace il
