// Traffic envelope of the bound trace (Section 5): for each window length, the
// largest number of arrivals inside any window of that length.  A maximising
// window can be moved right until it starts at an arrival, so thread j counts
// the arrivals in [a_j, a_j + window) for every window length -- a binary search
// for the first arrival at or after a_j + window, started where the search for
// the previous (shorter) window ended when the lengths ascend -- and the
// per-window maxima are combined with a warp reduction and one atomic per warp.
// The trace is read-only and L2-resident; the work is n * W searches.
#include "il_internal.h"

namespace il {

namespace {
constexpr int kEnvThreads = 256;
constexpr int kMaxWindows = 64;
}

struct EnvParams {
    const int64_t *arrival;
    int32_t n;
    int32_t n_windows;
    int64_t window[kMaxWindows];
    int *out;                  // [n_windows], zero on entry
};

__global__ void __launch_bounds__(kEnvThreads) envelope_kernel(const __grid_constant__ EnvParams p)
{
    for (int j0 = blockIdx.x * kEnvThreads; j0 < p.n; j0 += gridDim.x * kEnvThreads) {
        const int j = j0 + threadIdx.x;
        const bool act = j < p.n;
        const int64_t a = act ? p.arrival[j] : 0;
        int lo_hint = j;
        int64_t prev_win = 0;
        for (int w = 0; w < p.n_windows; w++) {
            int count = 0;
            if (act) {
                // first index hi with arrival[hi] - a >= window; the arrivals before it are inside
                int lo = p.window[w] >= prev_win ? lo_hint : j, hi = p.n;
                while (lo < hi) {
                    const int mid = lo + (hi - lo) / 2;
                    if (p.arrival[mid] - a < p.window[w]) lo = mid + 1; else hi = mid;
                }
                count = lo - j;
                lo_hint = lo;
                prev_win = p.window[w];
            }
            count = __reduce_max_sync(0xffffffffu, count);
            if ((threadIdx.x & 31) == 0 && count > 0) atomicMax(&p.out[w], count);
        }
    }
}

cudaError_t launch_envelope(const int64_t *d_arrival, int n, const int64_t *h_windows, int n_windows,
                            int *d_out, int num_sms, cudaStream_t stream)
{
    EnvParams p;
    p.arrival = d_arrival; p.n = n; p.n_windows = n_windows; p.out = d_out;
    for (int w = 0; w < n_windows; w++) p.window[w] = h_windows[w];
    const int blocks = (n + kEnvThreads - 1) / kEnvThreads;
    const int grid = blocks < num_sms * 8 ? blocks : num_sms * 8;
    envelope_kernel<<<grid, kEnvThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

int envelope_max_windows() { return kMaxWindows; }

}  // namespace il
