// Per-candidate P99 and SLO-miss count over the latency slab.
//
// P99 is the k-th smallest of the candidate's n latencies with
// k = ceil(0.99 n) = (99 n + 99) / 100 (Section 2: 99% of the query latencies
// must lie below the objective); a query misses iff latency > slo.  The k-th
// smallest is found by most-significant-digit radix select: each pass
// histograms one 8-bit digit of the keys that still match the prefix found so
// far, then descends into the bucket that holds rank k.  Digits above the
// highest set bit of any latency (known from the simulation kernel's OR) are
// skipped.  One CTA per candidate.
//
// When the slab comes from a packed-record simulation kernel it holds
// (finish time, query) records; a first sweep replaces each by
// latency = finish - arrival[query], ORs the latencies and counts the misses.
// When the slab's regions are known (lane kernel: one region per stage that
// queries leave after, each in finish order), the last record of each region
// gives the candidate's largest finish time, and largest finish - first arrival
// bounds every latency before the sweep: if that is below 2^32 the sweep writes 32-bit latencies (into the front
// half of the row; one barrier per 256 records keeps the writes behind the
// reads) and histograms the top digit on the way, and the remaining passes read
// half the bytes.
#include "il_internal.h"

namespace il {

__global__ void __launch_bounds__(kSelectThreads)
select_kernel(const __grid_constant__ SelectParams p)
{
    __shared__ unsigned hist[256];
    __shared__ unsigned long long s_prefix;
    __shared__ unsigned s_rank;
    __shared__ unsigned s_miss;
    __shared__ unsigned long long s_or;

    for (int64_t c = blockIdx.x; c < p.n_cand; c += gridDim.x) {
        int64_t *lat = p.slab + c * p.slab_stride;
        unsigned miss = 0;
        bool counted_miss = false;
        uint64_t bits_used;
        if (p.packed && p.n_regions > 0 && !(p.ovf && p.ovf[c])) {
            uint64_t last = 0;
#pragma unroll
            for (int r = 0; r < IL_MAX_STAGES; r++)      // unrolled: constant indices into the parameter block
                if (r < p.n_regions) last = max(last, (uint64_t)lat[p.region_end[r] - 1] >> p.qbits);
            const int64_t bound64 = (int64_t)last - p.arrival[0];
            if (bound64 < (INT64_C(1) << 32)) {
                const uint32_t bound = bound64 > 0 ? (uint32_t)bound64 : 0u;
                int top32 = 0;
                while (top32 < 4 && (bound >> (8 * top32)) != 0) top32++;
                hist[threadIdx.x] = 0;
                if (threadIdx.x == 0) {
                    s_prefix = 0;
                    s_rank = (unsigned)((99ll * p.n + 99) / 100);
                    s_miss = 0;
                }
                __syncthreads();
                uint32_t *lat32 = reinterpret_cast<uint32_t *>(lat);
                const uint64_t qmask = (1ull << p.qbits) - 1ull;
                const int sh_top = top32 > 0 ? 8 * (top32 - 1) : 0;
                for (int base = 0; base < p.n; base += kSelectThreads) {
                    const int i = base + (int)threadIdx.x;
                    uint32_t l = 0;
                    if (i < p.n) {
                        const uint64_t rec = (uint64_t)lat[i];
                        if (IL_IN_RANGE(rec & qmask, p.n, p.status))
                            l = (uint32_t)((int64_t)(rec >> p.qbits) - p.arrival[rec & qmask]);
                        miss += ((int64_t)l > p.slo_us);
                    }
                    __syncthreads();        // all records of this block are read before their row space is reused
                    if (i < p.n) {
                        lat32[i] = l;
                        atomicAdd(&hist[(l >> sh_top) & 0xff], 1u);
                    }
                }
                __syncthreads();
                for (int d = top32 - 1; d >= 0; d--) {
                    const int shift = 8 * d;
                    if (d != top32 - 1) {
                        hist[threadIdx.x] = 0;
                        __syncthreads();
                        const uint32_t prefix = (uint32_t)s_prefix;
                        const uint32_t himask = ~0u << (shift + 8);     // d <= 2 here
                        for (int i = threadIdx.x; i < p.n; i += kSelectThreads) {
                            const uint32_t v = lat32[i];
                            if ((v & himask) == prefix) atomicAdd(&hist[(v >> shift) & 0xff], 1u);
                        }
                        __syncthreads();
                    }
                    if (threadIdx.x == 0) {
                        unsigned r = s_rank, acc = 0;
                        int b = 0;
                        for (; b < 255; b++) {
                            if (acc + hist[b] >= r) break;
                            acc += hist[b];
                        }
                        s_rank = r - acc;
                        s_prefix = s_prefix | ((unsigned long long)b << shift);
                    }
                    __syncthreads();
                }
                if (miss) atomicAdd(&s_miss, miss);
                __syncthreads();
                if (threadIdx.x == 0) {
                    p.out_p99[c] = (int64_t)s_prefix;
                    p.out_miss[c] = (int64_t)s_miss;
                }
                __syncthreads();
                continue;
            }
        }
        if (p.packed) {
            if (threadIdx.x == 0) s_or = 0;
            __syncthreads();
            const uint64_t qmask = (1ull << p.qbits) - 1ull;
            unsigned long long my_or = 0;
            for (int i = threadIdx.x; i < p.n; i += kSelectThreads) {
                const uint64_t rec = (uint64_t)lat[i];
                int64_t l = 0;
                if (IL_IN_RANGE(rec & qmask, p.n, p.status)) l = (int64_t)(rec >> p.qbits) - p.arrival[rec & qmask];
                lat[i] = l;
                my_or |= (unsigned long long)l;
                miss += (l > p.slo_us);
            }
            counted_miss = true;
            my_or |= __shfl_xor_sync(0xffffffffu, my_or, 16);
            my_or |= __shfl_xor_sync(0xffffffffu, my_or, 8);
            my_or |= __shfl_xor_sync(0xffffffffu, my_or, 4);
            my_or |= __shfl_xor_sync(0xffffffffu, my_or, 2);
            my_or |= __shfl_xor_sync(0xffffffffu, my_or, 1);
            if ((threadIdx.x & 31) == 0 && my_or) atomicOr(&s_or, my_or);
            __syncthreads();   // also orders the latency writes before the passes below
            bits_used = s_or;
        } else {
            bits_used = p.lat_or[c];
        }
        int top = 0;                                   // number of 8-bit digits that matter
        while (top < 8 && (bits_used >> (8 * top)) != 0) top++;

        if (threadIdx.x == 0) {
            s_prefix = 0;
            s_rank = (unsigned)((99ll * p.n + 99) / 100);   // 1-indexed rank still to find
            s_miss = 0;
        }
        __syncthreads();

        for (int d = top - 1; d >= 0; d--) {
            hist[threadIdx.x] = 0;                     // kSelectThreads == 256 bins
            __syncthreads();
            const unsigned long long prefix = s_prefix;
            const int shift = 8 * d;
            // keys whose digits above d equal the prefix are still in the running
            const unsigned long long himask = (d == 7) ? 0ull : (~0ull << (shift + 8));
            for (int i = threadIdx.x; i < p.n; i += kSelectThreads) {
                const unsigned long long v = (unsigned long long)lat[i];
                if (!counted_miss) miss += ((int64_t)v > p.slo_us);
                if ((v & himask) == prefix) atomicAdd(&hist[(v >> shift) & 0xff], 1u);
            }
            counted_miss = true;
            __syncthreads();
            if (threadIdx.x == 0) {
                unsigned r = s_rank, acc = 0;
                int b = 0;
                for (; b < 255; b++) {
                    if (acc + hist[b] >= r) break;
                    acc += hist[b];
                }
                s_rank = r - acc;
                s_prefix = prefix | ((unsigned long long)b << shift);
            }
            __syncthreads();
        }
        if (!counted_miss) {   // every latency is zero: cannot happen (tables >= 1); kept for safety
            for (int i = threadIdx.x; i < p.n; i += kSelectThreads) miss += (lat[i] > p.slo_us);
        }
        if (miss) atomicAdd(&s_miss, miss);
        __syncthreads();
        if (threadIdx.x == 0) {
            p.out_p99[c] = (int64_t)s_prefix;
            p.out_miss[c] = (int64_t)s_miss;
        }
        __syncthreads();
    }
}

// Shared-prefix evaluation: the largest latencies of one node of a stage that queries leave after.
// A candidate's P99 is the (T + 1)-th largest latency of the union of its leaving nodes, T = n - k
// being the number of queries allowed above it, so no node ever contributes more than its own T + 1
// largest: they are kept, in descending order, for the combine step (prefix_kernel.cu), together with
// the node's miss count.  One CTA per node: records -> latencies (in place), radix select of the
// (T + 1)-th largest, collection of everything above it into shared memory, bitonic sort.
__global__ void __launch_bounds__(kSelectThreads)
node_top_kernel(const __grid_constant__ NodeTopParams p)
{
    extern __shared__ __align__(16) unsigned char top_raw[];
    int64_t *s_top = reinterpret_cast<int64_t *>(top_raw);
    __shared__ unsigned hist[256];
    __shared__ unsigned long long s_prefix, s_or;
    __shared__ unsigned s_rank, s_miss, s_fill;

    int pow2 = 1;
    while (pow2 < p.top_len) pow2 <<= 1;
    const uint64_t qmask = (1ull << p.qbits) - 1ull;
    for (int64_t node = blockIdx.x; node < p.n_nodes; node += gridDim.x) {
        int64_t *lat = reinterpret_cast<int64_t *>(p.records + (p.row_of ? (int64_t)p.row_of[node] : node) * p.stride + p.offset);
        if (threadIdx.x == 0) { s_or = 0; s_miss = 0; s_fill = 0; s_prefix = 0; }
        __syncthreads();
        unsigned miss = 0;
        unsigned long long my_or = 0;
        for (int i = threadIdx.x; i < p.len; i += kSelectThreads) {
            const uint64_t rec = (uint64_t)lat[i];
            const int64_t l = (int64_t)(rec >> p.qbits) - p.arrival[rec & qmask];
            lat[i] = l;
            my_or |= (unsigned long long)l;
            miss += (l > p.slo_us);
        }
        for (int o = 16; o > 0; o >>= 1) my_or |= __shfl_xor_sync(0xffffffffu, my_or, o);
        if ((threadIdx.x & 31) == 0 && my_or) atomicOr(&s_or, my_or);
        if (miss) atomicAdd(&s_miss, miss);
        __syncthreads();
        long long threshold = -1;       // keep every latency above this value
        if (p.len > p.top_len) {
            // the top_len-th largest = the (len - top_len + 1)-th smallest
            int top = 0;
            while (top < 8 && (s_or >> (8 * top)) != 0) top++;
            if (threadIdx.x == 0) s_rank = (unsigned)(p.len - p.top_len + 1);
            __syncthreads();
            for (int d = top - 1; d >= 0; d--) {
                hist[threadIdx.x] = 0;
                __syncthreads();
                const unsigned long long prefix = s_prefix;
                const int shift = 8 * d;
                const unsigned long long himask = (d == 7) ? 0ull : (~0ull << (shift + 8));
                for (int i = threadIdx.x; i < p.len; i += kSelectThreads) {
                    const unsigned long long v = (unsigned long long)lat[i];
                    if ((v & himask) == prefix) atomicAdd(&hist[(v >> shift) & 0xff], 1u);
                }
                __syncthreads();
                if (threadIdx.x == 0) {
                    unsigned r = s_rank, acc = 0;
                    int b = 0;
                    for (; b < 255; b++) {
                        if (acc + hist[b] >= r) break;
                        acc += hist[b];
                    }
                    s_rank = r - acc;
                    s_prefix = prefix | ((unsigned long long)b << shift);
                }
                __syncthreads();
            }
            threshold = (long long)s_prefix;
        }
        // everything above the threshold, then copies of the threshold up to top_len entries, then zeros
        for (int i = threadIdx.x; i < p.len; i += kSelectThreads) {
            const int64_t l = lat[i];
            if (l > threshold) s_top[atomicAdd(&s_fill, 1u)] = l;
        }
        __syncthreads();
        const int got = (int)s_fill;
        const int keep = p.len > p.top_len ? p.top_len : got;
        for (int i = got + (int)threadIdx.x; i < pow2; i += kSelectThreads) s_top[i] = i < keep ? threshold : 0;
        __syncthreads();
        // bitonic sort, descending
        for (int k = 2; k <= pow2; k <<= 1) {
            for (int j = k >> 1; j > 0; j >>= 1) {
                for (int i = threadIdx.x; i < pow2; i += kSelectThreads) {
                    const int partner = i ^ j;
                    if (partner > i) {
                        const int64_t a = s_top[i], b = s_top[partner];
                        const bool desc = (i & k) == 0;
                        if (desc ? a < b : a > b) { s_top[i] = b; s_top[partner] = a; }
                    }
                }
                __syncthreads();
            }
        }
        int64_t *out = p.top + node * p.top_len;
        for (int i = threadIdx.x; i < p.top_len; i += kSelectThreads) out[i] = s_top[i];
        if (threadIdx.x == 0) p.miss[node] = (int64_t)s_miss;
        __syncthreads();
    }
}

size_t node_top_smem(int top_len)
{
    size_t pow2 = 1;
    while (pow2 < (size_t)top_len) pow2 <<= 1;
    return pow2 * sizeof(int64_t);
}

cudaError_t launch_node_top(const NodeTopParams &p, cudaStream_t stream)
{
    const size_t smem = node_top_smem(p.top_len);
    cudaError_t e = cudaFuncSetAttribute(node_top_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int grid = (int)(p.n_nodes < 148 * 8 ? p.n_nodes : 148 * 8);
    node_top_kernel<<<grid, kSelectThreads, smem, stream>>>(p);
    return cudaGetLastError();
}

// Per-query answer of one candidate: the slab row holds one (finish, query)
// record per query, in the order the queries left the pipeline; the latency of
// query q goes to out[q].
__global__ void __launch_bounds__(256)
scatter_latency_kernel(const uint64_t *__restrict__ slab_row, const int64_t *__restrict__ arrival,
                       int n, int qbits, int64_t *__restrict__ out)
{
    const uint64_t qmask = (1ull << qbits) - 1ull;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
        const uint64_t rec = slab_row[i];
        const uint64_t q = rec & qmask;
        out[q] = (int64_t)(rec >> qbits) - arrival[q];
    }
}

cudaError_t launch_scatter_latency(const int64_t *slab_row, const int64_t *arrival, int n, int qbits,
                                   int64_t *out, cudaStream_t stream)
{
    const int grid = (n + 255) / 256 < 1184 ? (n + 255) / 256 : 1184;
    scatter_latency_kernel<<<grid, 256, 0, stream>>>(reinterpret_cast<const uint64_t *>(slab_row), arrival, n,
                                                     qbits, out);
    return cudaGetLastError();
}

cudaError_t launch_select(const SelectParams &p, cudaStream_t stream)
{
    const int grid = (int)(p.n_cand < 65535 * 16 ? p.n_cand : 65535 * 16);
    select_kernel<<<grid, kSelectThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace il
