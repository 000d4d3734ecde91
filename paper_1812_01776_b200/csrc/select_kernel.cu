// Per-candidate P99 and SLO-miss count over the latency slab.
//
// P99 is the k-th smallest of the candidate's n latencies with
// k = ceil(0.99 n) = (99 n + 99) / 100 (Section 2: 99% of the query latencies
// must lie below the objective); a query misses iff latency > slo.  One CTA per
// candidate.  The row is never rewritten: a slab of packed (finish time, query)
// records is turned into latencies on the fly, latency = finish - arrival[query]
// (the trace stays in L2), in every pass that needs them.
//
// The k-th smallest is found by a radix select whose FIRST digit needs no bound
// on the latencies: a latency falls into one of 8,192 bins by its bit length and
// the seven bits below its leading one (values below 256 have a bin each), which
// is monotone in the value and resolves it to better than 1 %.  The pass that
// fills this histogram also counts the misses.  The bin that holds rank k spans
// 2^e consecutive values.  If it holds at most 4,096 latencies (the rule, since
// rank k sits in the thin upper tail), a second pass over the row collects them
// into shared memory, in the space of the histogram, and the select ends there;
// otherwise passes with plain 13-bit digits over the bin's offsets narrow it
// until that holds or no bit is left (all latencies equal: two passes).  A
// thread requests the records of its next turn before it uses those of the
// current one (eight independent 8-byte loads in flight), which is what the row
// passes need to run near memory speed.
#include "il_internal.h"

namespace il {

namespace {

constexpr int kSelBins = 8192;       // bins of a histogram pass
constexpr int kSelCap = 4096;        // latencies the shared-memory list holds (the same 32 KB)
// Records a thread requests per turn (it has two turns in flight) and resident CTAs per SM.  Measured on
// 50,000- to 1,000,000-record rows: 4 x 4 as here 0.68 / 40.4 / 50.2 ms on three workloads, 8 x 4 0.70 / 40.8 /
// 52.4, 4 x 6 (40 registers) 0.81 / 62.2 / 67.0, 2 x 6 0.74 / 56.1 / 62.3, 8 x 3 0.92 / 49.8 / 60.6.
constexpr int kSelUnroll = 4;
constexpr int kSelCtasPerSm = 4;
constexpr int kSelDigit = 13;        // bits of a refinement digit: 2^13 = kSelBins

// Bin of the first pass.  Monotone in l; bin B >= 128 holds the values [m << e, (m + 1) << e) with
// e = (B >> 7) - 1 and m = B - (e << 7) in [128, 256); B < 128 holds the value B alone.
__device__ __forceinline__ unsigned first_bin(uint64_t l)
{
    if (l < 128u) return (unsigned)l;
    const int e = 56 - __clzll((long long)l);
    return ((unsigned)e << 7) + (unsigned)(l >> e);
}

struct SelectShared {
    unsigned warp_sum[kSelectThreads / 32];
    unsigned bin, rank, count;       // result of find_rank
    unsigned fill, miss;
    unsigned long long prefix;
};

// The bin of h[0 .. PER * 256) that holds the rank-th smallest element (1-based), the rank inside
// that bin and the bin's count, left in sh.bin / sh.rank / sh.count.  Thread t owns bins
// [PER * t, PER * (t + 1)); it reads them in a rotated order so that the threads of a warp never meet in
// a bank.  Called by all threads; ends with a barrier.
template <int PER>
__device__ __forceinline__ void find_rank(const unsigned *h, unsigned rank, SelectShared &sh)
{
    const int t = threadIdx.x, lane = t & 31, w = t >> 5;
    unsigned mine = 0;
#pragma unroll
    for (int j = 0; j < PER; j++) mine += h[PER * t + ((j + t) & (PER - 1))];
    unsigned incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) sh.warp_sum[w] = incl;
    __syncthreads();
    unsigned before = incl - mine;
    for (int k = 0; k < w; k++) before += sh.warp_sum[k];
    if (before < rank && rank <= before + mine) {      // exactly one thread
        unsigned acc = before;
        for (int j = 0; j < PER; j++) {
            const unsigned c = h[PER * t + j];
            if (acc + c >= rank) { sh.bin = (unsigned)(PER * t + j); sh.rank = rank - acc; sh.count = c; break; }
            acc += c;
        }
    }
    __syncthreads();
}

// One pass over a row.  MODE 0: first-bin histogram of every latency, misses counted.  MODE 1:
// histogram of ((latency - lo) >> sh) over the latencies in [lo, lo + 2^e).  MODE 2: the offsets
// latency - lo of those latencies appended to the list.
template <bool PACKED, int MODE>
__device__ __forceinline__ void row_pass(const SelectParams &p, const uint64_t *__restrict__ row, unsigned *hist,
                                         SelectShared &sh, uint64_t lo, int e, int shift, unsigned &miss)
{
    const uint64_t qmask = (1ull << p.qbits) - 1ull;
    const uint64_t width_m1 = e >= 64 ? ~0ull : ((1ull << e) - 1ull);
    uint64_t *list = reinterpret_cast<uint64_t *>(hist);
    const int n = p.n;
    // software pipeline: the records of the next turn are requested before this turn's are used
    uint64_t nx[kSelUnroll];
#pragma unroll
    for (int u = 0; u < kSelUnroll; u++) {
        const int i = u * kSelectThreads + (int)threadIdx.x;
        nx[u] = i < n ? __ldg(row + i) : 0ull;
    }
    for (int base = 0; base < n; base += kSelectThreads * kSelUnroll) {
        uint64_t v[kSelUnroll];
#pragma unroll
        for (int u = 0; u < kSelUnroll; u++) {
            const int i = base + (kSelUnroll + u) * kSelectThreads + (int)threadIdx.x;
            v[u] = nx[u];
            nx[u] = i < n ? __ldg(row + i) : 0ull;
        }
        if (PACKED) {
#pragma unroll
            for (int u = 0; u < kSelUnroll; u++) {
                const int i = base + u * kSelectThreads + (int)threadIdx.x;
                const uint64_t q = v[u] & qmask;
                if (i < n && IL_IN_RANGE(q, p.n, p.status))
                    v[u] = (v[u] >> p.qbits) - (uint64_t)__ldg(p.arrival + q);
                else
                    v[u] = 0ull;
            }
        }
#pragma unroll
        for (int u = 0; u < kSelUnroll; u++) {
            const int i = base + u * kSelectThreads + (int)threadIdx.x;
            if (i >= n) continue;
            if (MODE == 0) {
                miss += ((int64_t)v[u] > p.slo_us) ? 1u : 0u;
                atomicAdd(&hist[first_bin(v[u])], 1u);
            } else {
                const uint64_t off = v[u] - lo;
                if (off <= width_m1) {
                    if (MODE == 1) {
                        atomicAdd(&hist[(unsigned)(off >> shift)], 1u);
                    } else {
                        const unsigned pos = atomicAdd(&sh.fill, 1u);
                        if (pos < (unsigned)kSelCap) list[pos] = off;
                    }
                }
            }
        }
    }
}

template <bool PACKED>
__device__ __forceinline__ void select_rows(const SelectParams &p, unsigned *hist, unsigned *hist256, SelectShared &sh)
{
    uint64_t *list = reinterpret_cast<uint64_t *>(hist);
    for (int64_t c = blockIdx.x; c < p.n_cand; c += gridDim.x) {
        const uint64_t *row = reinterpret_cast<const uint64_t *>(p.slab + c * p.slab_stride);
        for (int i = threadIdx.x; i < kSelBins; i += kSelectThreads) hist[i] = 0u;
        if (threadIdx.x == 0) sh.miss = 0u;
        __syncthreads();
        unsigned miss = 0, unused = 0;
        row_pass<PACKED, 0>(p, row, hist, sh, 0ull, 0, 0, miss);
        for (int o = 16; o > 0; o >>= 1) miss += __shfl_xor_sync(0xffffffffu, miss, o);
        if ((threadIdx.x & 31) == 0 && miss) atomicAdd(&sh.miss, miss);
        __syncthreads();
        find_rank<kSelBins / kSelectThreads>(hist, (unsigned)((99ll * p.n + 99) / 100), sh);
        unsigned rank = sh.rank, count = sh.count;
        int e = sh.bin < 128u ? 0 : (int)(sh.bin >> 7) - 1;
        uint64_t lo = sh.bin < 128u ? (uint64_t)sh.bin : (uint64_t)(sh.bin - ((unsigned)e << 7)) << e;
        // narrow [lo, lo + 2^e) until its latencies fit the list
        while (e > 0 && count > (unsigned)kSelCap) {
            const int d = e < kSelDigit ? e : kSelDigit;
            __syncthreads();                 // everybody has read sh.bin / sh.rank / sh.count
            for (int i = threadIdx.x; i < kSelBins; i += kSelectThreads) hist[i] = 0u;
            __syncthreads();
            row_pass<PACKED, 1>(p, row, hist, sh, lo, e, e - d, unused);
            __syncthreads();
            find_rank<kSelBins / kSelectThreads>(hist, rank, sh);
            lo += (uint64_t)sh.bin << (e - d);
            e -= d;
            rank = sh.rank; count = sh.count;
        }
        if (e > 0) {
            // the rest in shared memory: collect the offsets, then 8-bit digits over the list
            __syncthreads();
            if (threadIdx.x == 0) sh.fill = 0u;
            __syncthreads();
            row_pass<PACKED, 2>(p, row, hist, sh, lo, e, 0, unused);
            __syncthreads();
            const unsigned got = sh.fill < (unsigned)kSelCap ? sh.fill : (unsigned)kSelCap;
            uint64_t prefix = 0;
            for (int shift = ((e - 1) >> 3) << 3; shift >= 0; shift -= 8) {
                hist256[threadIdx.x] = 0u;
                __syncthreads();
                const uint64_t himask = shift + 8 >= 64 ? 0ull : (~0ull << (shift + 8));
                for (unsigned i = threadIdx.x; i < got; i += kSelectThreads) {
                    const uint64_t v = list[i];
                    if ((v & himask) == prefix) atomicAdd(&hist256[(unsigned)(v >> shift) & 0xffu], 1u);
                }
                __syncthreads();
                find_rank<1>(hist256, rank, sh);
                prefix |= (uint64_t)sh.bin << shift;
                rank = sh.rank;
                __syncthreads();
            }
            lo += prefix;
        }
        if (threadIdx.x == 0) {
            p.out_p99[c] = (int64_t)lo;
            p.out_miss[c] = (int64_t)sh.miss;
        }
        __syncthreads();
    }
}

}  // namespace

__global__ void __launch_bounds__(kSelectThreads, kSelCtasPerSm)
select_kernel(const __grid_constant__ SelectParams p)
{
    __shared__ __align__(16) unsigned hist[kSelBins];
    __shared__ unsigned hist256[kSelectThreads];
    __shared__ SelectShared sh;
    if (p.packed) select_rows<true>(p, hist, hist256, sh);
    else select_rows<false>(p, hist, hist256, sh);
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
