// il_estimate_device_static: the estimate call for processes that must not
// allocate device memory after start-up.  The scratch the simulation kernel
// needs (inter-stage streams, latency slab, counters) is a static device array
// that is part of this library's image; nothing here calls cudaMalloc, cudaFree
// or any other allocating routine.
#include "il_internal.h"

#include <algorithm>
#include <mutex>

using namespace il;

namespace {

// The scratch itself.  In host code this name is only a handle for the runtime's
// symbol lookup, not a device address: the address is fetched per device below.
static __device__ __align__(256) unsigned char g_static_scratch[IL_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
constexpr int kMaxStaticSlots = 32;      // warps resident in the static variant
constexpr size_t kHeaderBytes = 256;     // counters (4 x u64) at 0, status word at 64

std::mutex g_mutex;
unsigned char *g_scratch_addr[kMaxDevices] = {};

// Device address of the array on `dev`, which must be the current device.
// Looked up once per device.
cudaError_t scratch_address(int dev, unsigned char **out)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_addr[dev]) {
        void *ptr = nullptr;
        cudaError_t ce = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (ce != cudaSuccess) return ce;
        g_scratch_addr[dev] = static_cast<unsigned char *>(ptr);
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace

// Enqueues the whole call; on a failing CUDA call records it and returns IL_ERR_CUDA.
static int enqueue_static(const BoundView &v, unsigned char *base, const il_stage_config *d_configs,
                          int64_t n_cand, int64_t slo_us, int64_t *d_out_p99, int64_t *d_out_miss,
                          int64_t slots, size_t off_time, size_t off_qid, size_t off_slab,
                          size_t off_order, int *h_status)
{
#define IL_ST(call)                                                          \
    do { cudaError_t e_ = (call); if (e_ != cudaSuccess) { set_last_cuda_error((int)e_); return IL_ERR_CUDA; } } while (0)
    cudaStream_t st = v.stream;
    // the array keeps the last call's contents: the work counter, the batch
    // counters and the status word must start at zero
    IL_ST(cudaMemsetAsync(base, 0, kHeaderBytes, st));

    DesParams p = v.base;
    p.counters = reinterpret_cast<unsigned long long *>(base);
    p.status = reinterpret_cast<int *>(base + 64);
    p.configs = d_configs;
    p.n_cand = n_cand;
    p.slot_elems = v.slot_elems;
    p.ws_time = reinterpret_cast<int64_t *>(base + off_time);
    p.ws_qid = reinterpret_cast<int32_t *>(base + off_qid);
    p.slab = reinterpret_cast<int64_t *>(base + off_slab);
    p.slab_stride = v.n_pad;
    p.order = reinterpret_cast<int32_t *>(base + off_order);
    OrderParams op;
    op.configs = d_configs; op.n_cand = n_cand; op.lat = v.base.lat;
    op.S = v.S; op.H = v.base.H; op.Bmax = v.base.Bmax;
    for (int s = 0; s < IL_MAX_STAGES; s++) op.n_s[s] = v.base.n_s[s];
    op.span_us = v.span_us;
    op.order = reinterpret_cast<int32_t *>(base + off_order);
    IL_ST(launch_order(op, st));
    IL_ST(launch_simulation(p, v.kernel, (int)(slots / kWarpsPerCta), v.smem, st));

    SelectParams sp = {};
    sp.slab = p.slab; sp.slab_stride = v.n_pad;
    sp.arrival = p.arrival; sp.qbits = p.qbits; sp.packed = v.kernel != kSimWide ? 1 : 0;
    sp.status = p.status;
    sp.n = (int32_t)v.n; sp.n_cand = n_cand; sp.slo_us = slo_us;
    sp.out_p99 = d_out_p99; sp.out_miss = d_out_miss;
    IL_ST(launch_select(sp, st));
    IL_ST(cudaMemcpyAsync(h_status, p.status, sizeof(int), cudaMemcpyDeviceToHost, st));
#undef IL_ST
    return IL_OK;
}

extern "C" int il_estimate_device_static(il_estimator *est, const il_stage_config *d_configs,
                                         int64_t n_cand, int64_t slo_us, int64_t *d_out_p99,
                                         int64_t *d_out_miss)
{
    if (!est || n_cand < 0) return IL_ERR_INVALID_ARG;
    if (n_cand == 0) return IL_OK;
    if (!d_configs || !d_out_p99 || !d_out_miss) return IL_ERR_INVALID_ARG;
    BoundView v;
    bound_view(est, &v);
    if (v.device < 0 || v.device >= kMaxDevices) return IL_ERR_INVALID_ARG;

    // does the request fit the array?  Only the kernel with separate time and
    // query streams needs the 4-byte query array.
    const int64_t slots = std::min<int64_t>(kMaxStaticSlots,
                                            (n_cand + kWarpsPerCta - 1) / kWarpsPerCta * kWarpsPerCta);
    const size_t qid_bytes = v.kernel == kSimWide ? 4 : 0;
    size_t off = kHeaderBytes;
    const size_t off_time = off; off = align_up(off + (size_t)slots * v.slot_elems * 8, 256);
    const size_t off_qid = off;  off = align_up(off + (size_t)slots * v.slot_elems * qid_bytes, 256);
    const size_t off_slab = off;
    // guard the multiplication before it can wrap
    if ((size_t)n_cand > IL_STATIC_SCRATCH_BYTES / 8 || (size_t)v.n_pad > IL_STATIC_SCRATCH_BYTES / 8)
        return IL_ERR_TOO_LARGE;
    off = align_up(off + (size_t)n_cand * v.n_pad * 8, 256);
    const size_t off_order = off; off = align_up(off + (size_t)n_cand * 4, 256);
    if (off > IL_STATIC_SCRATCH_BYTES) return IL_ERR_TOO_LARGE;

    // the caller's current device is put back before returning
    int prev = 0;
    cudaError_t ce = cudaGetDevice(&prev);
    if (ce == cudaSuccess) ce = cudaSetDevice(v.device);
    if (ce != cudaSuccess) { set_last_cuda_error((int)ce); return IL_ERR_CUDA; }
    unsigned char *base = nullptr;
    ce = scratch_address(v.device, &base);
    if (ce != cudaSuccess) { set_last_cuda_error((int)ce); cudaSetDevice(prev); return IL_ERR_CUDA; }

    int status = 0;
    int rc = enqueue_static(v, base, d_configs, n_cand, slo_us, d_out_p99, d_out_miss, slots, off_time,
                            off_qid, off_slab, off_order, &status);
    // whatever was enqueued (all of it, or the part before a failing call) is
    // waited for: nothing may still be writing the shared array or the caller's
    // outputs when the call returns
    ce = cudaStreamSynchronize(v.stream);
    if (ce != cudaSuccess && rc == IL_OK) { set_last_cuda_error((int)ce); rc = IL_ERR_CUDA; }
    cudaSetDevice(prev);
    return rc != IL_OK ? rc : status;
}
