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

#include <algorithm>

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

// Candidates the lane kernel gave up on (ring overflow), as a list for the warp-per-candidate
// kernel: order[0 .. count) in any order, count to counters[3] (and added to counters[4]); the
// work counter counters[0] is cleared for the kernel that follows.
__global__ void __launch_bounds__(1024) overflow_list_kernel(const uint8_t *ovf, int64_t n_cand, int32_t *order,
                                                            unsigned long long *counters)
{
    __shared__ unsigned count;
    if (threadIdx.x == 0) count = 0;
    __syncthreads();
    for (int64_t c = threadIdx.x; c < n_cand; c += blockDim.x)
        if (ovf[c]) order[atomicAdd(&count, 1u)] = (int32_t)c;
    __syncthreads();
    if (threadIdx.x == 0) {
        counters[3] = count;
        counters[4] += count;
        counters[0] = 0;
    }
}

// largest replica count over `count` stage configurations (values above the limit count as the limit:
// the simulation kernel rejects them)
__global__ void __launch_bounds__(256) max_replicas_kernel(const il_stage_config *configs, int64_t count, int *out)
{
    int m = 0;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x)
        m = max(m, min((int)configs[i].replicas, IL_MAX_REPLICAS));
    m = __reduce_max_sync(0xffffffffu, m);
    if ((threadIdx.x & 31) == 0 && m > 0) atomicMax(out, m);
}

// configs of the listed candidates, packed one after the other
__global__ void gather_configs_kernel(const il_stage_config *configs, const int32_t *list, int64_t count, int S,
                                      il_stage_config *out)
{
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < count * S; i += (int64_t)gridDim.x * blockDim.x)
        out[i] = configs[(int64_t)list[i / S] * S + i % S];
}

// Feasible (Section 4.3): P99 <= objective.  With a list, entry i belongs to candidate list[i].
__global__ void feasible_from_p99_kernel(const int64_t *p99, const int32_t *list, int64_t count, int64_t slo_us,
                                         uint8_t *out)
{
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x)
        out[list ? list[i] : i] = p99[i] <= slo_us ? 1 : 0;
}

}  // namespace

cudaError_t launch_max_replicas(const il_stage_config *configs, int64_t count, int *out, cudaStream_t stream)
{
    const int grid = (int)std::min<int64_t>((count + 255) / 256, 1184);
    max_replicas_kernel<<<grid, 256, 0, stream>>>(configs, count, out);
    return cudaGetLastError();
}

cudaError_t launch_gather_configs(const il_stage_config *configs, const int32_t *list, int64_t count, int S,
                                  il_stage_config *out, cudaStream_t stream)
{
    const int grid = (int)std::min<int64_t>((count * S + 255) / 256, 1184);
    gather_configs_kernel<<<grid, 256, 0, stream>>>(configs, list, count, S, out);
    return cudaGetLastError();
}

cudaError_t launch_feasible_from_p99(const int64_t *p99, const int32_t *list, int64_t count, int64_t slo_us,
                                     uint8_t *out, cudaStream_t stream)
{
    const int grid = (int)std::min<int64_t>((count + 255) / 256, 1184);
    feasible_from_p99_kernel<<<grid, 256, 0, stream>>>(p99, list, count, slo_us, out);
    return cudaGetLastError();
}

cudaError_t launch_overflow_list(const uint8_t *ovf, int64_t n_cand, int32_t *order, unsigned long long *counters,
                                 cudaStream_t stream)
{
    overflow_list_kernel<<<1, 1024, 0, stream>>>(ovf, n_cand, order, counters);
    return cudaGetLastError();
}

cudaError_t launch_order(const OrderParams &p, cudaStream_t stream)
{
    order_kernel<<<1, kOrderThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace il
