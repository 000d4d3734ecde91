// Host side of the C ABI declared in il_estimator.h: validation, device copies
// of the bound inputs, workspace planning, chunked launches and error codes.
#include "il_internal.h"

#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

using namespace il;

static thread_local int g_last_cuda_error = 0;

#define IL_CUDA(call)                                   \
    do {                                                \
        cudaError_t e_ = (call);                        \
        if (e_ != cudaSuccess) {                        \
            g_last_cuda_error = (int)e_;                \
            return IL_ERR_CUDA;                         \
        }                                               \
    } while (0)

static constexpr int kCounters = 8;

struct il_estimator {
    int device = 0;
    int num_sms = 0;
    int ctas_per_sm = 0;
    cudaStream_t stream = nullptr;

    int32_t S = 0, H = 0, Bmax = 0;
    int64_t n = 0;
    int64_t n_pad = 0;                 // n rounded up to 32: one slab row
    int64_t visits[IL_MAX_STAGES] = {};
    int64_t events_per_candidate = 0;
    float span_us = 1.f;
    DesParams base = {};               // bound-input part of the kernel parameters
    size_t smem = 0;
    int64_t slot_elems = 0;

    int64_t *d_arrival = nullptr;
    uint64_t *d_ptrace = nullptr;      // packed root stream
    uint64_t *d_ptrace_b = nullptr;    // the same with the branch bits inside each record (lane kernel)
    int rec_bits = 0;                  // branch bits a record of d_ptrace_b carries (0: there is none)
    bool can_pack = false;             // every reachable time fits a packed record
    bool fork = false;                 // fan-out: one query can enter two children of a stage
    bool join = false;                 // some stage has two incoming edges (implies fork: copies of a query exist)
    bool lane_ok = false;              // the lane kernel applies (packed records, stream offsets fit 31 bits)
    int variant = IL_VARIANT_AUTO;
    int ctas_per_sm_wide = 0, ctas_per_sm_packed = 0, ctas_per_sm_staged = 0, ctas_per_sm_lane = 0;
    int64_t lane_elems = 0;            // lane kernel: stream records per candidate (all rings of a candidate)
    int lane_ring_log2 = 0;            // lane kernel: a stream ring holds 2^this records
    int lane_ring_cap_log2 = 0;        // test knob: force rings of at most 2^this records (0: the library's choice)
    bool lane_wrap = false;            // the rings are shorter than the longest stream
    unsigned long long iter_limit = 0; // test knob: iteration bound of the device loops (0 = their own)
    int share_mode = 0;                // shared-prefix evaluation: 0 when it pays, 1 always (tests), 2 never, 3 always and node by node
    int32_t parent[IL_MAX_STAGES] = {};
    int cpw = 1;                       // lane kernel: candidates per warp
    size_t smem_lane[2] = {0, 0};       // lane kernel with 16 / 32 batch ring positions per lane
    int ctas_lane[2] = {0, 0};
    int lane_slots = 32;               // batch ring positions used by the current call
    int64_t setup_launches = 0;        // kernels a call launched before its simulation: the replica reduction, the node probe
    int lane_ctas_knob = 0;            // test knob: resident CTAs per SM of the lane kernel (0: the library's choice)
    int *d_maxrep = nullptr;           // device word: largest replica count of a batch
    uint8_t *d_bits = nullptr;
    int32_t *d_lat = nullptr;
    unsigned long long *d_counters = nullptr;   // [kCounters]: next candidate, batches, algorithmic ops,
                                                // overflow list length of the chunk, overflows of the call
    int *d_status = nullptr;
    unsigned long long *h_counters = nullptr;   // pinned: [kCounters] counters, then the status word
    int *h_status = nullptr;

    void *user_ws = nullptr; size_t user_ws_bytes = 0;
    void *own_ws = nullptr;  size_t own_ws_bytes = 0;

    il_stage_config *d_cfg = nullptr; int64_t d_cfg_cap = 0;   // staging for il_estimate
    int64_t *d_out = nullptr; int64_t d_out_cap = 0;           // [2][cap]

    std::vector<cudaEvent_t> events;
    il_stats stats = {};
};

namespace {

// When a chunk fits the GPU in about one wave (at most 1.5 candidates per warp
// slot), resident CTAs per SM are capped below the occupancy limit: on B200, 24
// warps per SM (6 CTAs) measured faster than 28 on the 4,096-candidate workload
// (each warp is a long dependent chain and the kernel ends with its slowest
// warp; fewer co-resident warps let the long ones run faster).  Larger chunks
// are throughput-bound and use every slot.
constexpr int kOneWaveCtasPerSm = 6;

struct Plan {
    int64_t slots = 0;       // warp slots with stream buffers
    int64_t chunk = 0;       // candidates per (simulate, select) pair
    int64_t fb_slots = 0;    // lane kernel with wrapping rings: warp slots of the kernel that takes over
                             // the candidates given up on ring overflow
    size_t off_time = 0, off_qid = 0, off_slab = 0, off_order = 0, off_ovf = 0, off_fb = 0, total = 0;
};

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Resident CTAs (of two warps) per SM for the lane kernel.  Every stream record reaches its lane through
// L1, and L1 is what the 256 KB of an SM have left after the shared-memory carve-out, which the launch
// sets to what the resident CTAs use (des_lane_kernel.cu).  More CTAs mean more lanes sharing less L1:
// on B200, 3 / 4 / 5 / 6 / 8 CTAs gave 42.8 / 39.3 / 43.0 / 46.8 / 70.4 ms on workload 2 with 16,384
// candidates and 298 / 245 / 336 / 336 / 335 ms on workload 3 with 16,384.  (Left to the driver, the
// carve-out was the largest one whatever the grid, and the same cases took 70 and 336 ms.)
constexpr int kLaneCtasPerSm = 4;

bool use_packed(const il_estimator *e)
{
    return e->can_pack && e->variant != IL_VARIANT_WIDE;
}

int sim_kernel(const il_estimator *e)
{
    if (!use_packed(e) || e->join) return kSimWide;     // joins: only the kernel with separate streams merges them
    // fan-out is implemented by the lane kernel and by the kernel with separate streams
    if (e->fork) return (e->variant == IL_VARIANT_AUTO || e->variant == IL_VARIANT_LANES) && e->lane_ok ? kSimLane : kSimWide;
    if (e->variant == IL_VARIANT_LANES && e->lane_ok) return kSimLane;
    if (e->variant == IL_VARIANT_AUTO && e->lane_ok) return kSimLane;
    return e->variant == IL_VARIANT_STAGED ? kSimPackedStaged : kSimPacked;
}

int ctas_for(const il_estimator *e)
{
    const int k = sim_kernel(e);
    return k == kSimWide ? e->ctas_per_sm_wide
         : k == kSimPacked ? e->ctas_per_sm_packed
         : k == kSimLane ? e->ctas_per_sm_lane : e->ctas_per_sm_staged;
}

// A warp slot is the stream memory one resident warp works in.  The
// warp-per-candidate kernels serve one candidate at a time from it, the lane
// kernel cpw candidates.
bool is_lane(const il_estimator *e) { return sim_kernel(e) == kSimLane; }
int warps_per_cta(const il_estimator *e) { return is_lane(e) ? des_lane_warps_per_cta() : kWarpsPerCta; }
int64_t cands_per_slot(const il_estimator *e) { return is_lane(e) ? e->cpw : 1; }

size_t slot_time_bytes(const il_estimator *e)
{
    return is_lane(e) ? (size_t)e->cpw * e->lane_elems * 8 : (size_t)e->slot_elems * 8;
}
size_t slot_qid_bytes(const il_estimator *e) { return is_lane(e) ? 0 : (size_t)e->slot_elems * 4; }
size_t slot_bytes(const il_estimator *e) { return slot_time_bytes(e) + slot_qid_bytes(e); }
size_t cand_bytes(const il_estimator *e) { return (size_t)e->n_pad * 8 + 5; }   // slab row, order entry, overflow mark
bool lane_fallback(const il_estimator *e) { return is_lane(e) && e->lane_wrap; }
size_t fb_slot_bytes(const il_estimator *e) { return (size_t)e->slot_elems * 8; }

int lane_ctas(const il_estimator *e)
{
    const int fit = e->ctas_lane[e->lane_slots == 16 ? 0 : 1];
    return std::max(1, std::min(fit, e->lane_ctas_knob > 0 ? e->lane_ctas_knob : kLaneCtasPerSm));
}

int64_t full_slots(const il_estimator *e)
{
    return (int64_t)e->num_sms * (is_lane(e) ? lane_ctas(e) : e->ctas_per_sm) * warps_per_cta(e);
}

int64_t wanted_slots(const il_estimator *e, int64_t n_cand)
{
    const int64_t w = warps_per_cta(e), cps = cands_per_slot(e);
    const int64_t need = ((n_cand + cps - 1) / cps + w - 1) / w * w;
    return std::max<int64_t>(w, std::min(full_slots(e), need));
}

size_t layout(const il_estimator *e, Plan &pl)
{
    size_t off = 0;
    pl.off_time = off; off = align_up(off + (size_t)pl.slots * slot_time_bytes(e), 256);
    pl.off_qid = off;  off = align_up(off + (size_t)pl.slots * slot_qid_bytes(e), 256);
    pl.off_slab = off; off = align_up(off + (size_t)pl.chunk * e->n_pad * 8, 256);
    pl.off_order = off; off = align_up(off + (size_t)pl.chunk * 4, 256);
    pl.off_ovf = off;  off = align_up(off + (size_t)pl.chunk, 256);
    pl.off_fb = off;   off = align_up(off + (size_t)pl.fb_slots * fb_slot_bytes(e), 256);
    pl.total = off;
    return off;
}

// Warp slots for the kernel that takes over after a ring overflow: about 6 % of the space, between one
// CTA and one CTA per SM.
int64_t fallback_slots(const il_estimator *e, size_t usable)
{
    if (!lane_fallback(e)) return 0;
    const int64_t fit = (int64_t)(usable / 16 / fb_slot_bytes(e)) / kWarpsPerCta * kWarpsPerCta;
    return std::max<int64_t>(kWarpsPerCta, std::min<int64_t>(fit, (int64_t)e->num_sms * kWarpsPerCta));
}

size_t recommended_bytes(const il_estimator *e, int64_t n_cand)
{
    Plan pl;
    n_cand = std::max<int64_t>(n_cand, 1);
    pl.slots = wanted_slots(e, n_cand);
    pl.chunk = std::max<int64_t>(std::min<int64_t>(n_cand, 8 * full_slots(e) * cands_per_slot(e)),
                                 2 * pl.slots * cands_per_slot(e));
    pl.fb_slots = lane_fallback(e) ? (int64_t)e->num_sms * kWarpsPerCta : 0;
    return layout(e, pl) + 2048;
}

size_t min_bytes(const il_estimator *e)
{
    Plan pl;
    pl.slots = warps_per_cta(e);
    pl.chunk = 2 * warps_per_cta(e);
    pl.fb_slots = lane_fallback(e) ? kWarpsPerCta : 0;
    return layout(e, pl) + 2048;
}

// Splits `bytes` of workspace between warp slots and the latency slab.
bool make_plan(const il_estimator *e, size_t bytes, int64_t n_cand, Plan &pl)
{
    if (bytes < min_bytes(e)) return false;
    size_t usable = bytes - 1024;
    pl.fb_slots = fallback_slots(e, usable);
    if (pl.fb_slots > 0) usable -= (size_t)pl.fb_slots * fb_slot_bytes(e) + 256;
    const size_t sb = slot_bytes(e), cb = cand_bytes(e);
    const int64_t w = warps_per_cta(e);
    int64_t slots = std::min<int64_t>(wanted_slots(e, n_cand), (int64_t)(usable / (sb + 2 * cands_per_slot(e) * cb)));
    slots = slots / w * w;
    if (slots < w) return false;
    pl.slots = slots;
    pl.chunk = std::min<int64_t>(n_cand, (int64_t)((usable - (size_t)slots * sb) / cb));
    // several chunks: whole waves of the resident warps per chunk, so that only the last chunk has a
    // partly filled wave
    const int64_t wave = slots * cands_per_slot(e);
    if (pl.chunk < n_cand && pl.chunk > wave) pl.chunk = pl.chunk / wave * wave;
    // alignment padding may push the layout over: shrink the chunk until it fits
    while (pl.chunk > 0 && layout(e, pl) > bytes) pl.chunk -= std::max<int64_t>(1, pl.chunk / 64);
    return pl.chunk >= 1;
}

int check_topology(const il_profiles *pr, const il_join_edges *jn)
{
    const int S = pr->n_stages;
    if (pr->parent[0] != -1) return IL_ERR_BAD_TOPOLOGY;
    if (jn && jn->parent2[0] != -1) return IL_ERR_BAD_TOPOLOGY;
    for (int s = 1; s < S; s++) {
        if (pr->parent[s] < 0 || pr->parent[s] >= s) return IL_ERR_BAD_TOPOLOGY;
        if (pr->cond_bit[s] < -1 || pr->cond_bit[s] > 7) return IL_ERR_BAD_TOPOLOGY;
        if (pr->cond_bit[s] >= 0 && pr->cond_val[s] > 1) return IL_ERR_BAD_TOPOLOGY;
        if (jn && jn->parent2[s] != -1) {
            if (jn->parent2[s] <= pr->parent[s] || jn->parent2[s] >= s) return IL_ERR_BAD_TOPOLOGY;
            if (jn->cond_bit2[s] < -1 || jn->cond_bit2[s] > 7) return IL_ERR_BAD_TOPOLOGY;
            if (jn->cond_bit2[s] >= 0 && jn->cond_val2[s] > 1) return IL_ERR_BAD_TOPOLOGY;
        }
    }
    for (int par = 0; par < S; par++) {
        int nk = 0;
        for (int c = 1; c < S; c++) nk += (pr->parent[c] == par) + (jn && jn->parent2[c] == par);
        if (nk > 2) return IL_ERR_BAD_TOPOLOGY;
    }
    return IL_OK;
}

// Two children of one stage are alternatives when they are guarded by the same bit with different
// values; otherwise one query can enter both (fan-out).
bool has_fan_out(const il_profiles *pr)
{
    const int S = pr->n_stages;
    for (int par = 0; par < S; par++) {
        int kids[2], nk = 0;
        for (int c = 1; c < S; c++) if (pr->parent[c] == par && nk < 2) kids[nk++] = c;
        if (nk == 2) {
            const int a = kids[0], b = kids[1];
            const bool alternatives = pr->cond_bit[a] >= 0 && pr->cond_bit[b] == pr->cond_bit[a] &&
                                      pr->cond_val[a] != pr->cond_val[b];
            if (!alternatives) return true;
        }
    }
    return false;
}

// Lays the stages' input streams out inside one warp slot.  Stage c's stream is
// written while its parent is simulated and read while c is; stages are
// simulated in index order, so the stream is live over the steps
// [parent[c], c] and two streams may share memory when these ranges are disjoint.
int64_t plan_stream_buffers(const il_profiles *pr, const int64_t *visits, int32_t *buf_off)
{
    const int S = pr->n_stages;
    struct Live { int64_t off, size; int end; };
    std::vector<Live> live;
    std::vector<int> order;
    for (int c = 1; c < S; c++) order.push_back(c);
    std::stable_sort(order.begin(), order.end(),
                     [&](int a, int b) { return pr->parent[a] < pr->parent[b]; });
    int64_t top = 0;
    buf_off[0] = 0;
    for (int c : order) {
        const int start = pr->parent[c];
        const int64_t size = (visits[c] + 31) / 32 * 32;
        buf_off[c] = 0;
        if (size == 0) continue;
        std::vector<Live> busy;
        for (const Live &l : live) if (l.end >= start) busy.push_back(l);
        std::sort(busy.begin(), busy.end(), [](const Live &a, const Live &b) { return a.off < b.off; });
        int64_t off = 0;
        for (const Live &l : busy) {
            if (off + size <= l.off) break;
            off = std::max(off, l.off + l.size);
        }
        buf_off[c] = (int32_t)off;
        live.push_back({off, size, c});
        top = std::max(top, off + size);
    }
    return top;
}

// Layout of a candidate's inter-stage streams in the lane kernel.  While the streams of all resident
// candidates fit kLaneExactBytes, every stage keeps its whole arrival stream (nothing wraps, and the
// kernel instantiation without the ring protocol runs, which is the faster one per iteration).  Beyond
// that -- long traces through deep pipelines -- a stage's stream lives in a ring of 2^13 records and the
// scratch per resident candidate no longer grows with the trace.  lane_ring_cap_log2 > 0 (test knob)
// forces rings of at most that length.
constexpr int64_t kLaneExactBytes = INT64_C(48) << 30;
constexpr int kLaneRingLog2 = 13;

void configure_lane_rings(il_estimator *e)
{
    DesParams &bp = e->base;
    int64_t longest = 8, exact = 0;
    for (int s = 1; s < e->S; s++) {
        longest = std::max(longest, e->visits[s]);
        exact += (e->visits[s] + 3) / 4 * 4;
    }
    const int64_t resident = (int64_t)e->num_sms * kLaneCtasPerSm * des_lane_warps_per_cta() * e->cpw;
    const bool rings = !e->fork && (e->lane_ring_cap_log2 > 0 || exact * 8 * resident > kLaneExactBytes ||
                                    exact >= (INT64_C(1) << 31));
    bp.lane_off[0] = 0;
    if (!rings) {
        int64_t off = 0;
        for (int s = 1; s < e->S; s++) { bp.lane_off[s] = (int32_t)off; off += (e->visits[s] + 3) / 4 * 4; }
        e->lane_elems = std::max<int64_t>(exact, 4);
        e->lane_ring_log2 = 31;
        e->lane_wrap = false;
    } else {
        int need = 3;
        while ((INT64_C(1) << need) < longest) need++;
        e->lane_ring_log2 = std::min(need, e->lane_ring_cap_log2 > 0 ? e->lane_ring_cap_log2 : kLaneRingLog2);
        e->lane_wrap = (INT64_C(1) << e->lane_ring_log2) < longest;
        for (int s = 1; s < e->S; s++) bp.lane_off[s] = (int32_t)((int64_t)(s - 1) << e->lane_ring_log2);
        e->lane_elems = std::max<int64_t>((int64_t)(e->S - 1) << e->lane_ring_log2, 4);
    }
    bp.lane_elems = e->lane_elems;
    bp.lane_ring_log2 = e->lane_ring_log2;
    bp.lane_wrap = e->lane_wrap ? 1 : 0;
}

void free_device(il_estimator *e)
{
    cudaFree(e->d_arrival); cudaFree(e->d_ptrace); cudaFree(e->d_ptrace_b); cudaFree(e->d_bits); cudaFree(e->d_lat);
    cudaFree(e->d_counters); cudaFree(e->d_status); cudaFree(e->d_maxrep);
    cudaFree(e->own_ws); cudaFree(e->d_cfg); cudaFree(e->d_out);
    if (e->h_counters) cudaFreeHost(e->h_counters);
    for (cudaEvent_t ev : e->events) cudaEventDestroy(ev);
}

int ensure_events(il_estimator *e, size_t count)
{
    while (e->events.size() < count) {
        cudaEvent_t ev;
        IL_CUDA(cudaEventCreate(&ev));
        e->events.push_back(ev);
    }
    return IL_OK;
}

}  // namespace

void il::set_last_cuda_error(int cuda_error) { g_last_cuda_error = cuda_error; }

void il::bound_view(const il_estimator *e, BoundView *out)
{
    out->base = e->base;
    out->kernel = e->fork ? (int)kSimWide : sim_kernel(e) == kSimLane ? (int)kSimPacked : sim_kernel(e);   // its user has no lane layout
    out->S = e->S;
    out->n = e->n; out->n_pad = e->n_pad; out->slot_elems = e->slot_elems;
    out->smem = e->smem;
    out->span_us = e->span_us;
    out->device = e->device;
    out->stream = e->stream;
}

// The scratch buffer a call may use: the caller's (il_set_workspace) or the
// library's own, (re)allocated here if it is too small for n_cand candidates.
static int acquire_workspace(il_estimator *e, int64_t n_cand, char **ws_out, size_t *bytes_out)
{
    char *ws = static_cast<char *>(e->user_ws);
    size_t ws_bytes = e->user_ws_bytes;
    if (!ws) {
        const size_t want = recommended_bytes(e, n_cand);
        if (e->own_ws_bytes < want) {
            size_t free_b = 0, total_b = 0;
            IL_CUDA(cudaMemGetInfo(&free_b, &total_b));
            const size_t grant = std::min(want, (size_t)((free_b + e->own_ws_bytes) * 0.8));
            if (grant > e->own_ws_bytes) {
                IL_CUDA(cudaStreamSynchronize(e->stream));
                if (e->own_ws) { cudaFree(e->own_ws); e->own_ws = nullptr; e->own_ws_bytes = 0; }
                if (grant < min_bytes(e)) return IL_ERR_NOMEM;
                cudaError_t ce = cudaMalloc(&e->own_ws, grant);
                if (ce != cudaSuccess) { g_last_cuda_error = (int)ce; e->own_ws = nullptr; return IL_ERR_NOMEM; }
                e->own_ws_bytes = grant;
            }
        }
        ws = static_cast<char *>(e->own_ws);
        ws_bytes = e->own_ws_bytes;
    }
    *ws_out = ws;
    *bytes_out = ws_bytes;
    return IL_OK;
}

// Device staging of the host entry points: configurations and the two output arrays.
static int ensure_staging(il_estimator *e, int64_t n_cand)
{
    const int64_t total = n_cand * e->S;
    if (e->d_cfg_cap < total) {
        IL_CUDA(cudaStreamSynchronize(e->stream));
        cudaFree(e->d_cfg); e->d_cfg = nullptr; e->d_cfg_cap = 0;
        cudaError_t ce = cudaMalloc(&e->d_cfg, (size_t)total * sizeof(il_stage_config));
        if (ce != cudaSuccess) { g_last_cuda_error = (int)ce; return IL_ERR_NOMEM; }
        e->d_cfg_cap = total;
    }
    if (e->d_out_cap < n_cand) {
        IL_CUDA(cudaStreamSynchronize(e->stream));
        cudaFree(e->d_out); e->d_out = nullptr; e->d_out_cap = 0;
        cudaError_t ce = cudaMalloc(&e->d_out, (size_t)n_cand * 24);   // P99, misses, feasibility flags
        if (ce != cudaSuccess) { g_last_cuda_error = (int)ce; return IL_ERR_NOMEM; }
        e->d_out_cap = n_cand;
    }
    return IL_OK;
}

// Kernel parameters of one chunk: the bound inputs plus this chunk's scratch.
static DesParams chunk_params(const il_estimator *e, const Plan &pl, char *ws, const il_stage_config *d_configs,
                              int64_t cnt)
{
    DesParams p = e->base;
    p.configs = d_configs;
    p.n_cand = cnt;
    p.slot_elems = e->slot_elems;
    p.ws_time = reinterpret_cast<int64_t *>(ws + pl.off_time);
    p.ws_qid = reinterpret_cast<int32_t *>(ws + pl.off_qid);
    p.lane_ws = reinterpret_cast<uint64_t *>(ws + pl.off_time);
    p.slab = reinterpret_cast<int64_t *>(ws + pl.off_slab);
    p.slab_stride = e->n_pad;
    p.order = reinterpret_cast<int32_t *>(ws + pl.off_order);
    p.ovf = reinterpret_cast<uint8_t *>(ws + pl.off_ovf);
    p.iter_limit = e->iter_limit;
    p.lane_slots = e->lane_slots;
    p.lane_ctas_per_sm = lane_ctas(e);
    return p;
}

// Batch ring positions per lane for this batch: 16 when no candidate has more than 14 replicas at any
// stage (the ring must hold the slots in use and the batches waiting to be handed on; with 16 replicas on
// 16 positions a stage stalls until each batch has been handed on, and workload 4 ran 1.6x slower), else 32.  One
// small reduction over the configurations and a 4-byte read-back.
static int choose_lane_slots(il_estimator *e, const il_stage_config *d_configs, int64_t n_cand)
{
    e->lane_slots = 32;
    e->setup_launches = 0;
    if (!is_lane(e)) return IL_OK;
    e->setup_launches = 1;
    int h = 0;
    IL_CUDA(cudaMemsetAsync(e->d_maxrep, 0, sizeof(int), e->stream));
    IL_CUDA(launch_max_replicas(d_configs, n_cand * e->S, e->d_maxrep, e->stream));
    IL_CUDA(cudaMemcpyAsync(&h, e->d_maxrep, sizeof(int), cudaMemcpyDeviceToHost, e->stream));
    IL_CUDA(cudaStreamSynchronize(e->stream));
    e->lane_slots = h <= 14 ? 16 : 32;
    return IL_OK;
}

// Enqueues the simulation of one chunk whose work counter is zero: the kernel the handle uses
// and, behind the lane kernel with wrapping rings, the pass that evaluates the candidates it gave
// up on with the warp-per-candidate kernel.  `launches` counts the kernels.
static int enqueue_simulation(il_estimator *e, const DesParams &p, const Plan &pl, char *ws, int64_t ctas,
                              cudaStream_t st, int64_t *launches)
{
    const int kernel = sim_kernel(e);
    const bool fb = kernel == kSimLane && e->lane_wrap;
    if (fb) IL_CUDA(cudaMemsetAsync(p.ovf, 0, (size_t)p.n_cand, st));
    // fan-out: the lane kernel keeps per query the largest leaving record, starting from zero
    if (kernel == kSimLane && e->fork)
        IL_CUDA(cudaMemsetAsync(p.slab, 0, (size_t)p.n_cand * p.slab_stride * 8, st));
    IL_CUDA(launch_simulation(p, kernel, (int)ctas, kernel == kSimLane ? e->smem_lane[e->lane_slots == 16 ? 0 : 1] : e->smem, st));
    (*launches)++;
    if (fb) {
        IL_CUDA(launch_overflow_list(p.ovf, p.n_cand, const_cast<int32_t *>(p.order), e->d_counters, st));
        DesParams q = p;
        q.ws_time = reinterpret_cast<int64_t *>(ws + pl.off_fb);
        q.n_cand_dev = e->d_counters + 3;
        IL_CUDA(launch_simulation(q, kSimPacked, (int)(pl.fb_slots / kWarpsPerCta), e->smem, st));
        *launches += 2;
    }
    return IL_OK;
}

// End of a shared-prefix call: events[0], events[1] and the work in between are on the stream.
static int finish_shared(il_estimator *e, int64_t n_cand, int64_t launches, int64_t stage_runs)
{
    cudaStream_t st = e->stream;
    IL_CUDA(cudaEventRecord(e->events[2], st));
    IL_CUDA(cudaMemcpyAsync(e->h_counters, e->d_counters, kCounters * sizeof(unsigned long long),
                            cudaMemcpyDeviceToHost, st));
    IL_CUDA(cudaMemcpyAsync(e->h_status, e->d_status, sizeof(int), cudaMemcpyDeviceToHost, st));
    IL_CUDA(cudaStreamSynchronize(st));
    float ms = 0.f;
    IL_CUDA(cudaEventElapsedTime(&ms, e->events[0], e->events[1]));
    e->stats.sim_ms = ms;
    IL_CUDA(cudaEventElapsedTime(&ms, e->events[1], e->events[2]));
    e->stats.select_ms = ms;
    e->stats.total_ms = e->stats.sim_ms + e->stats.select_ms;
    e->stats.candidates = n_cand;
    e->stats.query_events = n_cand * e->events_per_candidate;
    e->stats.batches = (int64_t)e->h_counters[1];
    e->stats.algorithmic_ops = (int64_t)e->h_counters[2];
    e->stats.chunks = 1;
    e->stats.kernel_launches = launches;
    e->stats.error_detail = (int64_t)e->h_counters[5];
    e->stats.stage_runs = stage_runs;
    return *e->h_status;
}

// Shared-prefix evaluation, simulation by the lane kernel.  The nodes that queries leave after are
// covered by a set of whole candidates of the batch (per node the candidate with the smallest index
// that contains it); those are simulated like any batch, and a node's leaving records are the region
// of its stage in the slab row of its candidate.  Candidates of the set repeat the work of the
// prefixes they share, but they run on the kernel that is an order of magnitude faster per stage run
// than the node-by-node one, and all at once instead of level by level.  Needs whole streams (no
// rings, so that every row has the region layout) and room for all rows in one chunk; *done stays
// false when that is not so, and the caller simulates the nodes one by one.
// On entry `off` bytes of the workspace are in use; events[0] has been recorded.
struct SharedCommon {
    const il_stage_config *d_configs;
    int64_t n_cand, slo_us, allowed, top_len;
    int64_t *d_out_p99, *d_out_miss;
    const int32_t *node_of;
    const int *h_count;
    const int64_t *leaving;
};

static int shared_by_cover(il_estimator *e, const SharedCommon &c, char *ws, size_t ws_bytes, size_t off,
                           int64_t *launches, int64_t *stage_runs, bool *done)
{
    *done = false;
    if (e->share_mode == 3 || !is_lane(e) || e->lane_wrap) return IL_OK;
    const int S = e->S;
    const int64_t n_cand = c.n_cand;
    auto take = [&](size_t bytes) { const size_t at = off; off = align_up(off + bytes, 256); return at; };
    int64_t exit_nodes = 0;
    size_t o_rep[IL_MAX_STAGES] = {}, o_row[IL_MAX_STAGES] = {}, o_top[IL_MAX_STAGES] = {}, o_miss[IL_MAX_STAGES] = {};
    for (int s = 0; s < S; s++) {
        if (c.leaving[s] <= 0) continue;
        exit_nodes += c.h_count[s];
        o_rep[s] = take((size_t)c.h_count[s] * 4); o_row[s] = take((size_t)c.h_count[s] * 4);
        o_top[s] = take((size_t)c.h_count[s] * c.top_len * 8); o_miss[s] = take((size_t)c.h_count[s] * 8);
    }
    const int64_t most = std::min(n_cand, exit_nodes);
    const size_t o_flags = take((size_t)n_cand), o_pos = take((size_t)n_cand * 4), o_list = take((size_t)most * 4);
    const size_t o_cnt = take(4), o_cfg = take((size_t)most * S * sizeof(il_stage_config));
    if (off > ws_bytes) return IL_OK;
    Plan pl;
    if (!make_plan(e, ws_bytes - off, most, pl) || pl.chunk < most) return IL_OK;   // all rows must be there at once

    cudaStream_t st = e->stream;
    uint8_t *flags = reinterpret_cast<uint8_t *>(ws + o_flags);
    int32_t *pos = reinterpret_cast<int32_t *>(ws + o_pos), *list = reinterpret_cast<int32_t *>(ws + o_list);
    int *d_cnt = reinterpret_cast<int *>(ws + o_cnt);
    il_stage_config *cfg = reinterpret_cast<il_stage_config *>(ws + o_cfg);
    IL_CUDA(cudaMemsetAsync(flags, 0, (size_t)n_cand, st));
    IL_CUDA(cudaMemsetAsync(d_cnt, 0, 4, st));
    for (int s = 0; s < S; s++)
        if (c.leaving[s] > 0) {
            IL_CUDA(launch_cover_rep(c.node_of + (size_t)s * n_cand, n_cand, reinterpret_cast<int32_t *>(ws + o_rep[s]),
                                     c.h_count[s], flags, st));
            *launches += 2;
        }
    IL_CUDA(launch_cover_list(flags, n_cand, list, pos, d_cnt, st));
    for (int s = 0; s < S; s++)
        if (c.leaving[s] > 0) {
            IL_CUDA(launch_cover_rows(reinterpret_cast<int32_t *>(ws + o_rep[s]), pos, c.h_count[s],
                                      reinterpret_cast<int32_t *>(ws + o_row[s]), st));
            (*launches)++;
        }
    int m = 0;
    IL_CUDA(cudaMemcpyAsync(&m, d_cnt, 4, cudaMemcpyDeviceToHost, st));
    IL_CUDA(cudaStreamSynchronize(st));
    if (m < 1 || m > most) return IL_ERR_ITER_LIMIT;      // cannot happen: every node has a candidate
    IL_CUDA(launch_gather_configs(c.d_configs, list, m, S, cfg, st));
    *launches += 2;
    *done = true;

    char *sim_ws = ws + off;
    DesParams p = chunk_params(e, pl, sim_ws, cfg, m);
    const int64_t wpc = warps_per_cta(e);
    const int64_t groups = (m + cands_per_slot(e) - 1) / cands_per_slot(e);
    const int64_t ctas = std::min<int64_t>(pl.slots / wpc, (groups + wpc - 1) / wpc);
    int rc = enqueue_simulation(e, p, pl, sim_ws, ctas, st, launches);
    if (rc) return rc;
    IL_CUDA(cudaEventRecord(e->events[1], st));

    CombineParams cp = {};
    cp.n_cand = n_cand; cp.node_of = c.node_of; cp.top_len = (int32_t)c.top_len; cp.allowed = c.allowed;
    cp.out_p99 = c.d_out_p99; cp.out_miss = c.d_out_miss;
    int64_t region = 0;
    for (int s = 0; s < S; s++) {
        if (c.leaving[s] <= 0) continue;
        NodeTopParams tp = {};
        tp.records = reinterpret_cast<uint64_t *>(p.slab);
        tp.stride = e->n_pad; tp.len = (int32_t)c.leaving[s];
        tp.row_of = reinterpret_cast<int32_t *>(ws + o_row[s]);
        tp.offset = region;
        tp.arrival = e->d_arrival; tp.qbits = e->base.qbits; tp.slo_us = c.slo_us;
        tp.top_len = (int32_t)c.top_len;
        tp.top = reinterpret_cast<int64_t *>(ws + o_top[s]);
        tp.miss = reinterpret_cast<int64_t *>(ws + o_miss[s]);
        tp.n_nodes = c.h_count[s];
        IL_CUDA(launch_node_top(tp, st));
        (*launches)++;
        cp.exit_stage[cp.n_exit] = s; cp.top[cp.n_exit] = tp.top; cp.miss[cp.n_exit] = tp.miss; cp.n_exit++;
        region += c.leaving[s];
    }
    IL_CUDA(launch_prefix_combine(cp, st));
    (*launches)++;
    *stage_runs = (int64_t)m * S;
    return IL_OK;
}

// ---- shared-prefix evaluation -------------------------------------------------------------------
// Candidates that agree on the configurations of all stages on a path from the root have the same
// completion stream at the end of that path; the batch is turned into the set of distinct (stage,
// configuration, parent node) nodes, every node is simulated once, and each candidate's P99 and miss
// count are put together from the nodes where its queries leave (prefix_kernel.cu).  Used when the
// node count is at most a quarter of candidates x stages (exhaustive sweeps over per-stage choices);
// *used tells whether the batch was evaluated here.
constexpr int64_t kShareMinCandidates = 2048;
constexpr int kShareMaxTop = 16384;

static int estimate_shared(il_estimator *e, const il_stage_config *d_configs, int64_t n_cand, int64_t slo_us,
                           int64_t *d_out_p99, int64_t *d_out_miss, char *ws, size_t ws_bytes, bool *used)
{
    *used = false;
    const int S = e->S;
    const int64_t n = e->n;
    const int64_t allowed = n - (99 * n + 99) / 100;           // T: queries allowed above the P99
    const int64_t top_len = allowed + 1;
    if (e->share_mode == 2 || e->fork || !e->can_pack || e->variant != IL_VARIANT_AUTO || top_len > kShareMaxTop ||
        n_cand >= (INT64_C(1) << 30) || (e->share_mode == 0 && n_cand < kShareMinCandidates))
        return IL_OK;
    uint32_t cap = 1024;
    while ((int64_t)cap < 2 * n_cand) cap <<= 1;

    size_t off = 0;
    auto take = [&](size_t bytes) { const size_t at = off; off = align_up(off + bytes, 256); return at; };
    const size_t o_node_of = take((size_t)S * n_cand * 4), o_slot = take((size_t)n_cand * 4);
    const size_t o_keys = take((size_t)cap * 8), o_vals = take((size_t)cap * 4);
    const size_t o_cfg = take((size_t)S * n_cand * 4), o_par = take((size_t)S * n_cand * 4);
    const size_t o_count = take((size_t)IL_MAX_STAGES * 4), o_work = take((size_t)IL_MAX_STAGES * 8);
    if (off > ws_bytes) return IL_OK;
    int32_t *node_of = reinterpret_cast<int32_t *>(ws + o_node_of);
    uint32_t *node_cfg = reinterpret_cast<uint32_t *>(ws + o_cfg);
    int32_t *node_par = reinterpret_cast<int32_t *>(ws + o_par);
    int *d_count = reinterpret_cast<int *>(ws + o_count);
    unsigned long long *d_work = reinterpret_cast<unsigned long long *>(ws + o_work);

    int rc = ensure_events(e, 5);
    if (rc) return rc;
    cudaStream_t st = e->stream;
    IL_CUDA(cudaMemsetAsync(e->d_counters, 0, kCounters * sizeof(unsigned long long), st));
    IL_CUDA(cudaMemsetAsync(e->d_status, 0, sizeof(int), st));
    IL_CUDA(cudaMemsetAsync(d_count, 0, (size_t)IL_MAX_STAGES * 4, st));
    IL_CUDA(cudaMemsetAsync(d_work, 0, (size_t)IL_MAX_STAGES * 8, st));
    IL_CUDA(cudaEventRecord(e->events[0], st));
    for (int s = 0; s < S; s++)
        IL_CUDA(launch_prefix_stage(d_configs, n_cand, S, s, e->H, e->Bmax,
                                    s == 0 ? nullptr : node_of + (size_t)e->parent[s] * n_cand,
                                    reinterpret_cast<uint64_t *>(ws + o_keys), cap,
                                    reinterpret_cast<int32_t *>(ws + o_vals), reinterpret_cast<int32_t *>(ws + o_slot),
                                    d_count + s, node_cfg + (size_t)s * n_cand, node_par + (size_t)s * n_cand,
                                    node_of + (size_t)s * n_cand, e->d_status, st));
    int h_count[IL_MAX_STAGES];
    IL_CUDA(cudaMemcpyAsync(h_count, d_count, (size_t)IL_MAX_STAGES * 4, cudaMemcpyDeviceToHost, st));
    IL_CUDA(cudaMemcpyAsync(e->h_status, e->d_status, sizeof(int), cudaMemcpyDeviceToHost, st));
    IL_CUDA(cudaStreamSynchronize(st));
    if (*e->h_status) { *used = true; return *e->h_status; }       // an invalid candidate: the call fails here
    int64_t total_nodes = 0;
    for (int s = 0; s < S; s++) total_nodes += h_count[s];
    e->setup_launches += 3 * S;
    if (e->share_mode == 0 && total_nodes * 4 > n_cand * S) return IL_OK;

    int64_t leaving[IL_MAX_STAGES], stride_in[IL_MAX_STAGES], stride_ex[IL_MAX_STAGES];
    for (int s = 0; s < S; s++) {
        const int a = e->base.dest_a[s], b = e->base.dest_b[s];
        int64_t kids = 0;
        if (a >= 0) kids += e->visits[a];
        if (b >= 0 && b != a) kids += e->visits[b];
        leaving[s] = e->visits[s] - kids;
    }
    int64_t launches = e->setup_launches, stage_runs = total_nodes;
    {
        // the fast way first: the nodes covered by whole candidates on the lane kernel
        SharedCommon sc = {d_configs, n_cand, slo_us, allowed, top_len, d_out_p99, d_out_miss, node_of, h_count, leaving};
        bool done = false;
        rc = shared_by_cover(e, sc, ws, ws_bytes, off, &launches, &stage_runs, &done);
        if (rc) { *used = true; return rc; }
        if (done) {
            *used = true;
            return finish_shared(e, n_cand, launches, stage_runs);
        }
    }
    // streams between the nodes, leaving records, top lists and miss counts
    size_t o_in[IL_MAX_STAGES] = {}, o_ex[IL_MAX_STAGES] = {}, o_top[IL_MAX_STAGES] = {}, o_miss[IL_MAX_STAGES] = {};
    for (int s = 0; s < S; s++) {
        stride_in[s] = (e->visits[s] + 3) / 4 * 4;
        stride_ex[s] = (leaving[s] + 3) / 4 * 4;
        if (s > 0 && e->visits[s] > 0)
            o_in[s] = take((size_t)h_count[e->parent[s]] * stride_in[s] * 8);
        if (leaving[s] > 0) {
            o_ex[s] = take((size_t)h_count[s] * stride_ex[s] * 8);
            o_top[s] = take((size_t)h_count[s] * top_len * 8);
            o_miss[s] = take((size_t)h_count[s] * 8);
        }
    }
    if (off > ws_bytes) return IL_OK;
    *used = true;

    for (int s = 0; s < S; s++) {
        if (e->visits[s] == 0) continue;
        const int a = e->base.dest_a[s], b = e->base.dest_b[s];
        NodeStageParams np = {};
        np.lat_stage = e->d_lat + (size_t)s * e->H * e->Bmax;
        np.bits = e->d_bits; np.ptrace = e->d_ptrace;
        np.qbits = e->base.qbits; np.H = e->H; np.Bmax = e->Bmax;
        np.n_queries = (int32_t)e->n;
        np.n_in = (int32_t)e->visits[s];
        np.bit = e->base.bit[s];
        np.n_nodes = h_count[s];
        np.node_cfg = node_cfg + (size_t)s * n_cand;
        np.node_parent = node_par + (size_t)s * n_cand;
        np.in = s == 0 ? nullptr : reinterpret_cast<const uint64_t *>(ws + o_in[s]);
        np.stride_in = stride_in[s];
        uint64_t *ex = reinterpret_cast<uint64_t *>(ws + o_ex[s]);
        np.out_a = a >= 0 ? reinterpret_cast<uint64_t *>(ws + o_in[a]) : ex;
        np.stride_a = a >= 0 ? stride_in[a] : stride_ex[s];
        np.out_b = b >= 0 ? reinterpret_cast<uint64_t *>(ws + o_in[b]) : ex;
        np.stride_b = b >= 0 ? stride_in[b] : stride_ex[s];
        np.work = d_work + s;
        np.counters = e->d_counters;
        np.status = e->d_status;
        const int grid = (int)std::min<int64_t>((h_count[s] + kWarpsPerCta - 1) / kWarpsPerCta,
                                                (int64_t)e->num_sms * kOneWaveCtasPerSm);
        IL_CUDA(launch_node_stage(np, grid, st));
        launches++;
    }
    IL_CUDA(cudaEventRecord(e->events[1], st));
    CombineParams cp = {};
    cp.n_cand = n_cand; cp.node_of = node_of; cp.top_len = (int32_t)top_len; cp.allowed = allowed;
    cp.out_p99 = d_out_p99; cp.out_miss = d_out_miss;
    for (int s = 0; s < S; s++) {
        if (leaving[s] <= 0) continue;
        NodeTopParams tp = {};
        tp.records = reinterpret_cast<uint64_t *>(ws + o_ex[s]);
        tp.stride = stride_ex[s]; tp.len = (int32_t)leaving[s];
        tp.arrival = e->d_arrival; tp.qbits = e->base.qbits; tp.slo_us = slo_us;
        tp.top_len = (int32_t)top_len;
        tp.top = reinterpret_cast<int64_t *>(ws + o_top[s]);
        tp.miss = reinterpret_cast<int64_t *>(ws + o_miss[s]);
        tp.n_nodes = h_count[s];
        IL_CUDA(launch_node_top(tp, st));
        launches++;
        cp.exit_stage[cp.n_exit] = s;
        cp.top[cp.n_exit] = tp.top;
        cp.miss[cp.n_exit] = tp.miss;
        cp.n_exit++;
    }
    IL_CUDA(launch_prefix_combine(cp, st));
    launches++;
    return finish_shared(e, n_cand, launches, stage_runs);
}

extern "C" {

const char *il_strerror(int code)
{
    switch (code) {
    case IL_OK: return "ok";
    case IL_ERR_INVALID_ARG: return "invalid argument";
    case IL_ERR_BAD_TOPOLOGY: return "pipeline is not a tree of the accepted form";
    case IL_ERR_BAD_PROFILE: return "latency table entry below 1";
    case IL_ERR_BAD_TRACE: return "arrival trace negative, decreasing or too large";
    case IL_ERR_BAD_CONFIG: return "candidate configuration out of range";
    case IL_ERR_NOMEM: return "out of memory or workspace too small";
    case IL_ERR_CUDA: return "CUDA call failed";
    case IL_ERR_ITER_LIMIT: return "device loop exceeded its iteration bound";
    case IL_ERR_TOO_LARGE: return "request needs more than the built-in static scratch (IL_STATIC_SCRATCH_BYTES)";
    case IL_ERR_BOUNDS: return "a device index left its array (checked build)";
    default: return "unknown error";
    }
}

int il_last_cuda_error(void) { return g_last_cuda_error; }

int il_estimator_create(const il_profiles *pr, const il_trace *tr, il_estimator **out)
{
    return il_estimator_create_dag(pr, nullptr, tr, out);
}

int il_estimator_create_dag(const il_profiles *pr, const il_join_edges *jn, const il_trace *tr, il_estimator **out)
{
    if (!pr || !tr || !out) return IL_ERR_INVALID_ARG;
    if (jn && (!jn->parent2 || !jn->cond_bit2 || !jn->cond_val2)) return IL_ERR_INVALID_ARG;
    if (pr->n_stages < 1 || pr->n_stages > IL_MAX_STAGES || pr->n_hw < 1 || pr->n_hw > IL_MAX_HW ||
        pr->max_batch < 1 || pr->max_batch > IL_MAX_BATCH)
        return IL_ERR_INVALID_ARG;
    if (!pr->parent || !pr->cond_bit || !pr->cond_val || !pr->latency_us || !tr->arrival_us)
        return IL_ERR_INVALID_ARG;
    if (tr->n_queries < 1 || tr->n_queries > INT32_MAX) return IL_ERR_INVALID_ARG;
    int rc = check_topology(pr, jn);
    if (rc) return rc;
    const int S = pr->n_stages, H = pr->n_hw, B = pr->max_batch;
    const int64_t n = tr->n_queries;
    bool any_cond = false, any_join = false;
    for (int s = 1; s < S; s++) {
        any_cond |= pr->cond_bit[s] >= 0;
        if (jn && jn->parent2[s] >= 0) { any_join = true; any_cond |= jn->cond_bit2[s] >= 0; }
    }
    if (!any_join) jn = nullptr;
    if (any_cond && !tr->branch_bits) return IL_ERR_INVALID_ARG;

    int64_t worst = 0;   // bound on how far the clock can run past the last arrival
    for (int s = 0; s < S; s++) {
        int32_t mx = 0;
        for (int i = 0; i < H * B; i++) {
            const int32_t v = pr->latency_us[(size_t)s * H * B + i];
            if (v < 1) return IL_ERR_BAD_PROFILE;
            mx = std::max(mx, v);
        }
        worst += n * (int64_t)mx;   // n < 2^31, mx < 2^31, S <= 16: no overflow
    }
    if (tr->arrival_us[0] < 0) return IL_ERR_BAD_TRACE;
    for (int64_t i = 1; i < n; i++)
        if (tr->arrival_us[i] < tr->arrival_us[i - 1]) return IL_ERR_BAD_TRACE;
    if (tr->arrival_us[n - 1] > (INT64_C(1) << 62) - worst) return IL_ERR_BAD_TRACE;
    int qbits = 5;                       // bits of a packed record that hold the query index
    while ((INT64_C(1) << qbits) < n) qbits++;
    const bool can_pack = tr->arrival_us[n - 1] + worst < (INT64_C(1) << (63 - qbits));

    int dev = 0;
    cudaDeviceProp prop;
    IL_CUDA(cudaGetDevice(&dev));
    IL_CUDA(cudaGetDeviceProperties(&prop, dev));
    if (prop.major != 10) { g_last_cuda_error = (int)cudaErrorNoKernelImageForDevice; return IL_ERR_CUDA; }

    il_estimator *e = new (std::nothrow) il_estimator();
    if (!e) return IL_ERR_NOMEM;
    e->device = dev;
    e->num_sms = prop.multiProcessorCount;
    e->S = S; e->H = H; e->Bmax = B; e->n = n;
    e->n_pad = (n + 31) / 32 * 32;
    e->span_us = (float)std::max<int64_t>(1, tr->arrival_us[n - 1] - tr->arrival_us[0]);

    // routing table and visits per stage
    DesParams &bp = e->base;
    for (int s = 0; s < IL_MAX_STAGES; s++) { bp.dest_a[s] = -1; bp.dest_b[s] = -1; bp.bit[s] = -1; }
    for (int c = 1; c < S; c++) {
        const int par = pr->parent[c];
        if (pr->cond_bit[c] < 0) { bp.dest_a[par] = (int8_t)c; bp.dest_b[par] = (int8_t)c; }
        else {
            bp.bit[par] = pr->cond_bit[c];
            if (pr->cond_val[c] == 0) bp.dest_a[par] = (int8_t)c; else bp.dest_b[par] = (int8_t)c;
        }
    }
    for (int s = 0; s < S; s++) e->parent[s] = pr->parent[s];
    e->join = any_join;
    e->fork = any_join || has_fan_out(pr);
    bp.fork = e->fork ? 1 : 0;
    for (int s = 0; s < IL_MAX_STAGES; s++) {
        bp.child_a[s] = -1; bp.child_b[s] = -1; bp.cbit_a[s] = -1; bp.cbit_b[s] = -1; bp.join_b[s] = -1;
    }
    // outgoing edges of every stage, first-parent and second-parent edges alike
    auto add_edge = [&](int par, int c, int bit, int val) {
        if (bp.child_a[par] < 0) { bp.child_a[par] = (int8_t)c; bp.cbit_a[par] = (int8_t)bit; bp.cval_a[par] = (uint8_t)val; }
        else { bp.child_b[par] = (int8_t)c; bp.cbit_b[par] = (int8_t)bit; bp.cval_b[par] = (uint8_t)val; }
    };
    for (int c = 1; c < S; c++) {
        add_edge(pr->parent[c], c, pr->cond_bit[c], pr->cond_val[c]);
        if (jn && jn->parent2[c] >= 0) {
            add_edge(jn->parent2[c], c, jn->cond_bit2[c], jn->cond_val2[c]);
            bp.join_b[c] = (int8_t)jn->parent2[c];
        }
    }
    // Which stages a query visits follows from its branch bits alone (parents have smaller indices):
    // count the visits per stage, the records on each edge into a join, and the copies that leave.
    bp.total_leaving = 0;
    int64_t edge_a[IL_MAX_STAGES] = {}, edge_b[IL_MAX_STAGES] = {};
    for (int64_t q = 0; q < n; q++) {
        const unsigned bits = tr->branch_bits ? tr->branch_bits[q] : 0u;
        bool reach[IL_MAX_STAGES] = {};
        reach[0] = true;
        for (int c = 1; c < S; c++) {
            const bool a = reach[pr->parent[c]] && (pr->cond_bit[c] < 0 || ((bits >> pr->cond_bit[c]) & 1u) == pr->cond_val[c]);
            const bool b = jn && jn->parent2[c] >= 0 && reach[jn->parent2[c]] &&
                           (jn->cond_bit2[c] < 0 || ((bits >> jn->cond_bit2[c]) & 1u) == jn->cond_val2[c]);
            reach[c] = a || b;
            edge_a[c] += a; edge_b[c] += b;
        }
        for (int s = 0; s < S; s++) {
            if (!reach[s]) continue;
            e->visits[s]++;
            int taken = 0;
            for (int side = 0; side < 2; side++) {
                const int c = side == 0 ? bp.child_a[s] : bp.child_b[s];
                if (c < 0) continue;
                const int bit = side == 0 ? bp.cbit_a[s] : bp.cbit_b[s];
                const unsigned val = side == 0 ? bp.cval_a[s] : bp.cval_b[s];
                taken += (bit < 0 || ((bits >> bit) & 1u) == val);
            }
            if (taken == 0) bp.total_leaving++;
        }
    }
    e->events_per_candidate = 0;
    for (int s = 0; s < S; s++) e->events_per_candidate += e->visits[s];
    if (!e->join) {
        e->slot_elems = std::max<int64_t>(32, plan_stream_buffers(pr, e->visits, bp.buf_off));
    } else {
        // joins: every stream gets memory of its own (arrival stream per stage, the two incoming streams of
        // a join), then the scratch of the merge: its two halves and the per-query input times
        auto pad = [](int64_t v) { return (v + 31) / 32 * 32; };
        int64_t off = 0, tmp = 0;
        bp.buf_off[0] = 0;
        for (int c = 1; c < S; c++) {
            bp.buf_off[c] = (int32_t)std::min<int64_t>(off, INT32_MAX); off += pad(e->visits[c]);
            if (bp.join_b[c] < 0) continue;
            bp.join_in_a[c] = (int32_t)std::min<int64_t>(off, INT32_MAX); off += pad(edge_a[c]);
            bp.join_in_b[c] = (int32_t)std::min<int64_t>(off, INT32_MAX); off += pad(edge_b[c]);
            bp.join_na[c] = (int32_t)edge_a[c]; bp.join_nb[c] = (int32_t)edge_b[c];
            tmp = std::max(tmp, pad(edge_a[c]) + pad(edge_b[c]));
        }
        bp.join_tmp_off = (int32_t)std::min<int64_t>(off, INT32_MAX); off += tmp;
        bp.join_t_off = (int32_t)std::min<int64_t>(off, INT32_MAX); off += 2 * e->n_pad;
        if (off > INT32_MAX) { delete e; return IL_ERR_TOO_LARGE; }
        e->slot_elems = std::max<int64_t>(32, off);
    }
    // where each stage writes the records of its two outgoing edges (kernel with separate streams)
    for (int s = 0; s < S; s++) {
        for (int side = 0; side < 2; side++) {
            const int c = side == 0 ? bp.child_a[s] : bp.child_b[s];
            int32_t at = 0;
            if (c >= 0) at = bp.join_b[c] < 0 ? bp.buf_off[c] : (bp.join_b[c] == s ? bp.join_in_b[c] : bp.join_in_a[c]);
            (side == 0 ? bp.out_off_a : bp.out_off_b)[s] = at;
        }
    }
    for (int s = 0; s < S; s++) bp.n_s[s] = (int32_t)e->visits[s];
    // lane kernel: every stage but the root reads its arrival stream from a ring
    e->cpw = 32 / S;
    bp.cpw = e->cpw;
    configure_lane_rings(e);
    bp.S = S; bp.H = H; bp.Bmax = B; bp.n = (int32_t)n;
    e->smem = (size_t)S * H * B * sizeof(int32_t);

    auto fail = [&](int code) { free_device(e); delete e; return code; };
#define IL_CUDA_E(call)                                                   \
    do { cudaError_t e_ = (call); if (e_ != cudaSuccess) {                \
        g_last_cuda_error = (int)e_;                                      \
        return fail(e_ == cudaErrorMemoryAllocation ? IL_ERR_NOMEM : IL_ERR_CUDA); } } while (0)

    IL_CUDA_E(cudaMalloc(&e->d_arrival, (size_t)n * 8));
    IL_CUDA_E(cudaMalloc(&e->d_bits, (size_t)n));
    e->can_pack = can_pack;
    e->lane_ok = can_pack && !e->join && e->lane_elems < (INT64_C(1) << 31);   // (with fan-out the streams are kept whole)
    bp.qbits = qbits;
    if (can_pack) {
        // padded with "never" records to whole tiles, so that bulk copies always move full tiles
        const int64_t tile = trace_tile_records();
        const int64_t n_padded = (n + tile - 1) / tile * tile;
        std::vector<uint64_t> packed((size_t)n_padded, ~0ull);
        for (int64_t i = 0; i < n; i++)
            packed[(size_t)i] = ((uint64_t)tr->arrival_us[i] << qbits) | (uint64_t)i;
        IL_CUDA_E(cudaMalloc(&e->d_ptrace, (size_t)n_padded * 8));
        IL_CUDA_E(cudaMemcpy(e->d_ptrace, packed.data(), (size_t)n_padded * 8, cudaMemcpyHostToDevice));
        // Branch bits inside the records, where the time range leaves room for them: a stage of the lane
        // kernel then routes a query by the record it hands on instead of looking its bits up.
        int nb = 0;
        for (int s = 0; s < pr->n_stages; s++)
            if (pr->cond_bit[s] >= 0) nb = std::max(nb, (int)pr->cond_bit[s] + 1);
        if (nb > 0 && tr->branch_bits && !e->join &&
            tr->arrival_us[n - 1] + worst < (INT64_C(1) << (63 - qbits - nb))) {
            for (int64_t i = 0; i < n; i++)
                packed[(size_t)i] = ((uint64_t)tr->arrival_us[i] << (qbits + nb)) |
                                    ((uint64_t)(tr->branch_bits[i] & ((1u << nb) - 1u)) << qbits) | (uint64_t)i;
            IL_CUDA_E(cudaMalloc(&e->d_ptrace_b, (size_t)n_padded * 8));
            IL_CUDA_E(cudaMemcpy(e->d_ptrace_b, packed.data(), (size_t)n_padded * 8, cudaMemcpyHostToDevice));
            e->rec_bits = nb;
        }
    }
    IL_CUDA_E(cudaMalloc(&e->d_lat, e->smem));
    IL_CUDA_E(cudaMalloc(&e->d_counters, kCounters * sizeof(unsigned long long)));
    IL_CUDA_E(cudaMalloc(&e->d_status, sizeof(int)));
    IL_CUDA_E(cudaMalloc(&e->d_maxrep, sizeof(int)));
    IL_CUDA_E(cudaMallocHost(&e->h_counters, (kCounters + 2) * sizeof(unsigned long long)));
    e->h_status = reinterpret_cast<int *>(e->h_counters + kCounters);
    IL_CUDA_E(cudaMemcpy(e->d_arrival, tr->arrival_us, (size_t)n * 8, cudaMemcpyHostToDevice));
    if (tr->branch_bits) IL_CUDA_E(cudaMemcpy(e->d_bits, tr->branch_bits, (size_t)n, cudaMemcpyHostToDevice));
    else IL_CUDA_E(cudaMemset(e->d_bits, 0, (size_t)n));
    IL_CUDA_E(cudaMemcpy(e->d_lat, pr->latency_us, e->smem, cudaMemcpyHostToDevice));
#undef IL_CUDA_E
    bp.arrival = e->d_arrival; bp.bits = e->d_bits; bp.lat = e->d_lat; bp.ptrace = e->d_ptrace;
    bp.ptrace_b = e->d_ptrace_b; bp.rec_bits = e->rec_bits;
    bp.counters = e->d_counters; bp.status = e->d_status;

    e->ctas_per_sm_wide = des_max_ctas_per_sm(e->smem);
    e->ctas_per_sm_packed = des_packed_max_ctas_per_sm(false, e->smem);
    e->ctas_per_sm_staged = des_packed_max_ctas_per_sm(true, e->smem);
    for (int k = 0; k < 2; k++) {
        e->smem_lane[k] = des_lane_smem(S * H * B, B, k == 0 ? 16 : 32);
        e->ctas_lane[k] = des_lane_max_ctas_per_sm(e->smem_lane[k]);
    }
    e->ctas_per_sm_lane = std::min(e->ctas_lane[1], kLaneCtasPerSm);
    if (e->ctas_per_sm_wide < 1 || e->ctas_per_sm_packed < 1 || e->ctas_per_sm_staged < 1 ||
        e->ctas_per_sm_lane < 1) {
        g_last_cuda_error = (int)cudaErrorLaunchOutOfResources;
        return fail(IL_ERR_CUDA);
    }
    e->ctas_per_sm = ctas_for(e);
    *out = e;
    return IL_OK;
}

void il_estimator_destroy(il_estimator *e)
{
    if (!e) return;
    int prev = 0;
    cudaGetDevice(&prev);
    cudaSetDevice(e->device);
    free_device(e);
    cudaSetDevice(prev);
    delete e;
}

int il_set_stream(il_estimator *e, void *cuda_stream)
{
    if (!e) return IL_ERR_INVALID_ARG;
    e->stream = static_cast<cudaStream_t>(cuda_stream);
    return IL_OK;
}

int il_set_variant(il_estimator *e, int variant)
{
    if (!e || variant < IL_VARIANT_AUTO || variant > IL_VARIANT_PACKED) return IL_ERR_INVALID_ARG;
    e->variant = variant;
    e->ctas_per_sm = ctas_for(e);
    return IL_OK;
}

int il_set_test_knob(il_estimator *e, int knob, int64_t value)
{
    if (!e) return IL_ERR_INVALID_ARG;
    if (knob == IL_KNOB_LANE_RING_LOG2) {
        if (value < 6 || value > 24) return IL_ERR_INVALID_ARG;
        e->lane_ring_cap_log2 = (int)value;
        configure_lane_rings(e);
        return IL_OK;
    }
    if (knob == IL_KNOB_SHARE_PREFIXES) {
        if (value < 0 || value > 3) return IL_ERR_INVALID_ARG;
        e->share_mode = (int)value;
        return IL_OK;
    }
    if (knob == IL_KNOB_LANE_CTAS) {
        if (value < 0 || value > 16) return IL_ERR_INVALID_ARG;
        e->lane_ctas_knob = (int)value;
        return IL_OK;
    }
    if (knob == IL_KNOB_BITS_IN_RECORDS) {
        if (value != 0 && value != 1) return IL_ERR_INVALID_ARG;
        e->base.rec_bits = (value == 1 && e->d_ptrace_b) ? e->rec_bits : 0;
        return IL_OK;
    }
    if (knob == IL_KNOB_ITER_LIMIT) {
        if (value < 0) return IL_ERR_INVALID_ARG;
        e->iter_limit = (unsigned long long)value;
        return IL_OK;
    }
    return IL_ERR_INVALID_ARG;
}

const char *il_kernel_name(const il_estimator *e)
{
    if (!e) return "";
    switch (sim_kernel(e)) {
    case kSimLane: return "des_lane_kernel";
    case kSimPacked: return "des_packed_kernel";
    case kSimPackedStaged: return "des_packed_kernel<staged>";
    default: return "des_kernel";
    }
}

int il_workspace_bytes(const il_estimator *e, int64_t n_candidates, size_t *bytes)
{
    if (!e || !bytes || n_candidates < 0) return IL_ERR_INVALID_ARG;
    *bytes = recommended_bytes(e, n_candidates);
    return IL_OK;
}

int il_workspace_min_bytes(const il_estimator *e, size_t *bytes)
{
    if (!e || !bytes) return IL_ERR_INVALID_ARG;
    *bytes = min_bytes(e);
    return IL_OK;
}

int il_set_workspace(il_estimator *e, void *d_ws, size_t bytes)
{
    if (!e) return IL_ERR_INVALID_ARG;
    if (!d_ws || bytes == 0) { e->user_ws = nullptr; e->user_ws_bytes = 0; return IL_OK; }
    if (reinterpret_cast<uintptr_t>(d_ws) % 256 != 0) return IL_ERR_INVALID_ARG;
    if (bytes < min_bytes(e)) return IL_ERR_NOMEM;
    e->user_ws = d_ws;
    e->user_ws_bytes = bytes;
    return IL_OK;
}

int il_get_stats(const il_estimator *e, il_stats *out)
{
    if (!e || !out) return IL_ERR_INVALID_ARG;
    *out = e->stats;
    return IL_OK;
}

int il_stage_visits(const il_estimator *e, int64_t *out_visits)
{
    if (!e || !out_visits) return IL_ERR_INVALID_ARG;
    for (int s = 0; s < e->S; s++) out_visits[s] = e->visits[s];
    return IL_OK;
}

int il_estimate_device(il_estimator *e, const il_stage_config *d_configs, int64_t n_cand,
                       int64_t slo_us, int64_t *d_out_p99, int64_t *d_out_miss)
{
    if (!e || n_cand < 0) return IL_ERR_INVALID_ARG;
    e->stats = il_stats{};
    if (n_cand == 0) return IL_OK;
    if (!d_configs || !d_out_p99 || !d_out_miss) return IL_ERR_INVALID_ARG;
    IL_CUDA(cudaSetDevice(e->device));

    int lrc = choose_lane_slots(e, d_configs, n_cand);
    if (lrc) return lrc;
    char *ws = nullptr;
    size_t ws_bytes = 0;
    int wrc = acquire_workspace(e, n_cand, &ws, &ws_bytes);
    if (wrc) return wrc;
    bool shared = false;
    int src = estimate_shared(e, d_configs, n_cand, slo_us, d_out_p99, d_out_miss, ws, ws_bytes, &shared);
    if (shared || src) return src;
    Plan pl;
    if (!make_plan(e, ws_bytes, n_cand, pl)) return IL_ERR_NOMEM;

    const int64_t n_chunks = (n_cand + pl.chunk - 1) / pl.chunk;
    int rc = ensure_events(e, (size_t)(2 + 3 * n_chunks));
    if (rc) return rc;

    cudaStream_t st = e->stream;
    IL_CUDA(cudaMemsetAsync(e->d_counters, 0, kCounters * sizeof(unsigned long long), st));
    IL_CUDA(cudaMemsetAsync(e->d_status, 0, sizeof(int), st));
    IL_CUDA(cudaEventRecord(e->events[0], st));

    int64_t launches = e->setup_launches;
    for (int64_t ch = 0; ch < n_chunks; ch++) {
        const int64_t lo = ch * pl.chunk;
        const int64_t cnt = std::min(pl.chunk, n_cand - lo);
        DesParams p = chunk_params(e, pl, ws, d_configs + lo * e->S, cnt);
        if (ch > 0) IL_CUDA(cudaMemsetAsync(e->d_counters, 0, sizeof(unsigned long long), st));
        const bool lane = is_lane(e);
        const int64_t wpc = warps_per_cta(e);
        const int64_t groups = (cnt + cands_per_slot(e) - 1) / cands_per_slot(e);
        int64_t ctas = std::min<int64_t>(pl.slots / wpc, (groups + wpc - 1) / wpc);
        if (!lane) {   // the lane kernel's warps take candidates in index order
            OrderParams op;
            op.configs = p.configs; op.n_cand = cnt; op.lat = e->d_lat;
            op.S = e->S; op.H = e->H; op.Bmax = e->Bmax;
            for (int s = 0; s < IL_MAX_STAGES; s++) op.n_s[s] = e->base.n_s[s];
            op.span_us = e->span_us;
            op.order = const_cast<int32_t *>(p.order);
            IL_CUDA(launch_order(op, st));
            launches++;
            if (2 * cnt <= 3 * full_slots(e))
                ctas = std::min<int64_t>(ctas, (int64_t)e->num_sms * std::min(e->ctas_per_sm, kOneWaveCtasPerSm));
        }
        IL_CUDA(cudaEventRecord(e->events[2 + 3 * ch], st));
        rc = enqueue_simulation(e, p, pl, ws, ctas, st, &launches);
        if (rc) return rc;
        IL_CUDA(cudaEventRecord(e->events[3 + 3 * ch], st));
        SelectParams sp = {};
        sp.slab = p.slab; sp.slab_stride = e->n_pad;
        sp.arrival = e->d_arrival; sp.qbits = p.qbits; sp.packed = sim_kernel(e) != kSimWide ? 1 : 0;
        sp.status = e->d_status;
        sp.n = (int32_t)e->n; sp.n_cand = cnt; sp.slo_us = slo_us;
        sp.out_p99 = d_out_p99 + lo; sp.out_miss = d_out_miss + lo;
        IL_CUDA(launch_select(sp, st));
        IL_CUDA(cudaEventRecord(e->events[4 + 3 * ch], st));
        launches++;
    }
    IL_CUDA(cudaEventRecord(e->events[1], st));
    IL_CUDA(cudaMemcpyAsync(e->h_counters, e->d_counters, kCounters * sizeof(unsigned long long),
                            cudaMemcpyDeviceToHost, st));
    IL_CUDA(cudaMemcpyAsync(e->h_status, e->d_status, sizeof(int), cudaMemcpyDeviceToHost, st));
    IL_CUDA(cudaStreamSynchronize(st));

    float ms = 0.f;
    IL_CUDA(cudaEventElapsedTime(&ms, e->events[0], e->events[1]));
    e->stats.total_ms = ms;
    for (int64_t ch = 0; ch < n_chunks; ch++) {
        IL_CUDA(cudaEventElapsedTime(&ms, e->events[2 + 3 * ch], e->events[3 + 3 * ch]));
        e->stats.sim_ms += ms;
        IL_CUDA(cudaEventElapsedTime(&ms, e->events[3 + 3 * ch], e->events[4 + 3 * ch]));
        e->stats.select_ms += ms;
    }
    e->stats.candidates = n_cand;
    e->stats.query_events = n_cand * e->events_per_candidate;
    e->stats.batches = (int64_t)e->h_counters[1];
    e->stats.algorithmic_ops = (int64_t)e->h_counters[2];
    e->stats.chunks = n_chunks;
    e->stats.kernel_launches = launches;
    e->stats.fallback_candidates = (int64_t)e->h_counters[4];
    e->stats.error_detail = (int64_t)e->h_counters[5];
    e->stats.early_exits = 0;
    e->stats.stage_runs = n_cand * e->S;
    return *e->h_status;
}

int il_estimate_latencies(il_estimator *e, const il_stage_config *d_config, int64_t *d_out_latency)
{
    if (!e || !d_config || !d_out_latency) return IL_ERR_INVALID_ARG;
    IL_CUDA(cudaSetDevice(e->device));
    e->lane_slots = 32;
    char *ws = nullptr;
    size_t ws_bytes = 0;
    int rc = acquire_workspace(e, 1, &ws, &ws_bytes);
    if (rc) return rc;
    Plan pl;
    if (!make_plan(e, ws_bytes, 1, pl)) return IL_ERR_NOMEM;
    cudaStream_t st = e->stream;
    IL_CUDA(cudaMemsetAsync(e->d_counters, 0, kCounters * sizeof(unsigned long long), st));
    IL_CUDA(cudaMemsetAsync(e->d_status, 0, sizeof(int), st));
    DesParams p = chunk_params(e, pl, ws, d_config, 1);
    IL_CUDA(cudaMemsetAsync(ws + pl.off_order, 0, sizeof(int32_t), st));   // the one candidate is number 0
    const int kernel = sim_kernel(e);
    int64_t launches = 0;
    rc = enqueue_simulation(e, p, pl, ws, 1, st, &launches);
    if (rc) return rc;
    if (kernel == kSimWide)   // the wide kernel writes latencies in trace order
        IL_CUDA(cudaMemcpyAsync(d_out_latency, p.slab, (size_t)e->n * 8, cudaMemcpyDeviceToDevice, st));
    else
        IL_CUDA(launch_scatter_latency(p.slab, e->d_arrival, (int)e->n, p.qbits, d_out_latency, st));
    IL_CUDA(cudaMemcpyAsync(e->h_status, e->d_status, sizeof(int), cudaMemcpyDeviceToHost, st));
    IL_CUDA(cudaStreamSynchronize(st));
    return *e->h_status;
}

int il_traffic_envelope(il_estimator *e, const int64_t *window_us, int32_t n_windows, int64_t *out_max_count)
{
    if (!e || n_windows < 0 || n_windows > envelope_max_windows()) return IL_ERR_INVALID_ARG;
    if (n_windows == 0) return IL_OK;
    if (!window_us || !out_max_count) return IL_ERR_INVALID_ARG;
    for (int w = 0; w < n_windows; w++) if (window_us[w] < 1) return IL_ERR_INVALID_ARG;
    IL_CUDA(cudaSetDevice(e->device));
    // the counts fit the 4-word counter block that every estimate call clears before use
    static_assert(sizeof(unsigned long long) * kCounters >= sizeof(int) * 8, "counter block too small");
    int host_out[64];
    cudaStream_t st = e->stream;
    for (int w0 = 0; w0 < n_windows; w0 += 8) {
        const int cnt = std::min(8, n_windows - w0);
        IL_CUDA(cudaMemsetAsync(e->d_counters, 0, kCounters * sizeof(unsigned long long), st));
        IL_CUDA(launch_envelope(e->d_arrival, (int)e->n, window_us + w0, cnt,
                                reinterpret_cast<int *>(e->d_counters), e->num_sms, st));
        IL_CUDA(cudaMemcpyAsync(host_out + w0, e->d_counters, cnt * sizeof(int), cudaMemcpyDeviceToHost, st));
    }
    IL_CUDA(cudaStreamSynchronize(st));
    for (int w = 0; w < n_windows; w++) out_max_count[w] = host_out[w];
    return IL_OK;
}

int il_estimate(il_estimator *e, const il_stage_config *configs, int64_t n_cand, int64_t slo_us,
                int64_t *out_p99, int64_t *out_miss)
{
    if (!e || n_cand < 0) return IL_ERR_INVALID_ARG;
    if (n_cand == 0) { e->stats = il_stats{}; return IL_OK; }
    if (!configs || !out_p99 || !out_miss) return IL_ERR_INVALID_ARG;
    const int64_t total = n_cand * e->S;
    for (int64_t i = 0; i < total; i++) {
        const il_stage_config &c = configs[i];
        if (c.hw >= e->H || c.max_batch < 1 || c.max_batch > e->Bmax || c.replicas < 1 ||
            c.replicas > IL_MAX_REPLICAS)
            return IL_ERR_BAD_CONFIG;
    }
    IL_CUDA(cudaSetDevice(e->device));
    int rc0 = ensure_staging(e, n_cand);
    if (rc0) return rc0;
    IL_CUDA(cudaMemcpyAsync(e->d_cfg, configs, (size_t)total * sizeof(il_stage_config),
                            cudaMemcpyHostToDevice, e->stream));
    int rc = il_estimate_device(e, e->d_cfg, n_cand, slo_us, e->d_out, e->d_out + e->d_out_cap);
    if (rc) return rc;
    IL_CUDA(cudaMemcpyAsync(out_p99, e->d_out, (size_t)n_cand * 8, cudaMemcpyDeviceToHost, e->stream));
    IL_CUDA(cudaMemcpyAsync(out_miss, e->d_out + e->d_out_cap, (size_t)n_cand * 8,
                            cudaMemcpyDeviceToHost, e->stream));
    IL_CUDA(cudaStreamSynchronize(e->stream));
    return IL_OK;
}

int il_feasible_device(il_estimator *e, const il_stage_config *d_configs, int64_t n_cand, int64_t slo_us,
                       uint8_t *d_out_feasible)
{
    if (!e || n_cand < 0) return IL_ERR_INVALID_ARG;
    e->stats = il_stats{};
    if (n_cand == 0) return IL_OK;
    if (!d_configs || !d_out_feasible) return IL_ERR_INVALID_ARG;
    IL_CUDA(cudaSetDevice(e->device));
    cudaStream_t st = e->stream;

    if (!is_lane(e) || e->fork) {
        // no early exit on the other kernels, nor with fan-out (a query is late if ANY of its copies
        // is, so copies cannot be counted as they leave): P99 as usual, then the comparison
        int rc = ensure_staging(e, n_cand);
        if (rc) return rc;
        rc = il_estimate_device(e, d_configs, n_cand, slo_us, e->d_out, e->d_out + e->d_out_cap);
        if (rc) return rc;
        IL_CUDA(launch_feasible_from_p99(e->d_out, nullptr, n_cand, slo_us, d_out_feasible, st));
        IL_CUDA(cudaStreamSynchronize(st));
        e->stats.kernel_launches++;
        return IL_OK;
    }

    // lane kernel: no slab and no percentile pass, so the whole batch is one chunk
    int rc = choose_lane_slots(e, d_configs, n_cand);
    if (rc) return rc;
    char *ws = nullptr;
    size_t ws_bytes = 0;
    rc = acquire_workspace(e, std::min<int64_t>(n_cand, 4096), &ws, &ws_bytes);
    if (rc) return rc;
    if (e->share_mode == 1 || e->share_mode == 3 || (e->share_mode == 0 && n_cand >= kShareMinCandidates)) {
        // a batch full of common configuration prefixes is cheaper to evaluate node by node
        rc = ensure_staging(e, n_cand);
        if (rc) return rc;
        bool shared = false;
        rc = estimate_shared(e, d_configs, n_cand, slo_us, e->d_out, e->d_out + e->d_out_cap, ws, ws_bytes, &shared);
        if (rc) return rc;
        if (shared) {
            IL_CUDA(launch_feasible_from_p99(e->d_out, nullptr, n_cand, slo_us, d_out_feasible, st));
            IL_CUDA(cudaStreamSynchronize(st));
            e->stats.kernel_launches++;
            return IL_OK;
        }
    }
    const int64_t wpc = des_lane_warps_per_cta();
    const size_t sb = slot_time_bytes(e);
    const size_t tail_bytes = align_up((size_t)n_cand, 256) + align_up((size_t)n_cand * 4, 256) + 1024;
    if (ws_bytes < tail_bytes + (size_t)wpc * sb) return IL_ERR_NOMEM;
    int64_t slots = std::min<int64_t>(wanted_slots(e, n_cand), (int64_t)((ws_bytes - tail_bytes) / sb)) / wpc * wpc;
    if (slots < wpc) return IL_ERR_NOMEM;
    const size_t off_ovf = align_up((size_t)slots * sb, 256);
    const size_t off_order = off_ovf + align_up((size_t)n_cand, 256);
    rc = ensure_events(e, 4);
    if (rc) return rc;

    IL_CUDA(cudaMemsetAsync(e->d_counters, 0, kCounters * sizeof(unsigned long long), st));
    IL_CUDA(cudaMemsetAsync(e->d_status, 0, sizeof(int), st));
    DesParams p = e->base;
    p.configs = d_configs;
    p.n_cand = n_cand;
    p.lane_ws = reinterpret_cast<uint64_t *>(ws);
    p.ovf = reinterpret_cast<uint8_t *>(ws + off_ovf);
    p.iter_limit = e->iter_limit;
    p.lane_slots = e->lane_slots;
    p.lane_ctas_per_sm = lane_ctas(e);
    p.out_feasible = d_out_feasible;
    // latency > objective is tested on time fields shifted by qbits: keep the objective in that range
    // (latencies are at least 1 and every reachable time is below 2^(63 - qbits))
    p.slo_us = std::min<int64_t>(std::max<int64_t>(slo_us, 0), INT64_C(1) << (62 - p.qbits - p.rec_bits));
    p.miss_allow = (uint32_t)(e->n - (99 * e->n + 99) / 100);
    if (e->lane_wrap) IL_CUDA(cudaMemsetAsync(p.ovf, 0, (size_t)n_cand, st));
    const int64_t groups = (n_cand + e->cpw - 1) / e->cpw;
    const int64_t ctas = std::min<int64_t>(slots / wpc, (groups + wpc - 1) / wpc);
    IL_CUDA(cudaEventRecord(e->events[0], st));
    IL_CUDA(launch_des_lane(p, (int)ctas, e->smem_lane[e->lane_slots == 16 ? 0 : 1], st));
    IL_CUDA(cudaEventRecord(e->events[1], st));
    int64_t launches = 1;
    if (e->lane_wrap) {
        IL_CUDA(launch_overflow_list(p.ovf, n_cand, reinterpret_cast<int32_t *>(ws + off_order), e->d_counters, st));
        launches++;
    }
    IL_CUDA(cudaMemcpyAsync(e->h_counters, e->d_counters, kCounters * sizeof(unsigned long long),
                            cudaMemcpyDeviceToHost, st));
    IL_CUDA(cudaMemcpyAsync(e->h_status, e->d_status, sizeof(int), cudaMemcpyDeviceToHost, st));
    IL_CUDA(cudaStreamSynchronize(st));
    float ms = 0.f;
    IL_CUDA(cudaEventElapsedTime(&ms, e->events[0], e->events[1]));
    il_stats stats = {};
    stats.candidates = n_cand;
    stats.query_events = n_cand * e->events_per_candidate;
    stats.batches = (int64_t)e->h_counters[1];
    stats.algorithmic_ops = (int64_t)e->h_counters[2];
    stats.chunks = 1;
    stats.sim_ms = ms;
    stats.total_ms = ms;
    stats.fallback_candidates = (int64_t)e->h_counters[3];
    stats.error_detail = (int64_t)e->h_counters[5];
    stats.early_exits = (int64_t)e->h_counters[6];
    stats.stage_runs = n_cand * e->S;
    rc = *e->h_status;
    const int64_t n_fb = (int64_t)e->h_counters[3];
    if (rc == IL_OK && n_fb > 0) {
        // Rare: candidates the lane kernel gave up on (stream ring overflow).  They are evaluated in
        // full by the warp-per-candidate kernel; this path allocates its temporaries.
        char *tmp = nullptr;
        const size_t cfg_b = align_up((size_t)n_fb * e->S * sizeof(il_stage_config), 256);
        const size_t lst_b = align_up((size_t)n_fb * 4, 256), out_b = align_up((size_t)n_fb * 8, 256);
        cudaError_t ce = cudaMalloc(&tmp, cfg_b + lst_b + 2 * out_b);
        if (ce != cudaSuccess) { g_last_cuda_error = (int)ce; return IL_ERR_NOMEM; }
        il_stage_config *cfg2 = reinterpret_cast<il_stage_config *>(tmp);
        int32_t *list = reinterpret_cast<int32_t *>(tmp + cfg_b);
        int64_t *p99 = reinterpret_cast<int64_t *>(tmp + cfg_b + lst_b);
        int64_t *miss = reinterpret_cast<int64_t *>(tmp + cfg_b + lst_b + out_b);
        cudaError_t c1 = cudaMemcpyAsync(list, ws + off_order, (size_t)n_fb * 4, cudaMemcpyDeviceToDevice, st);
        if (c1 == cudaSuccess) c1 = launch_gather_configs(d_configs, list, n_fb, e->S, cfg2, st);
        const int variant = e->variant;
        if (c1 == cudaSuccess) {
            il_set_variant(e, IL_VARIANT_PACKED);
            rc = il_estimate_device(e, cfg2, n_fb, slo_us, p99, miss);
            il_set_variant(e, variant);
            stats.batches += e->stats.batches;
            stats.algorithmic_ops += e->stats.algorithmic_ops;
            stats.sim_ms += e->stats.sim_ms;
            stats.select_ms += e->stats.select_ms;
            stats.total_ms += e->stats.total_ms;
            launches += e->stats.kernel_launches + 2;
            if (rc == IL_OK) c1 = launch_feasible_from_p99(p99, list, n_fb, slo_us, d_out_feasible, st);
        }
        if (c1 == cudaSuccess) c1 = cudaStreamSynchronize(st);
        else cudaStreamSynchronize(st);
        cudaFree(tmp);
        if (c1 != cudaSuccess) { g_last_cuda_error = (int)c1; return IL_ERR_CUDA; }
    }
    stats.kernel_launches = launches;
    e->stats = stats;
    return rc;
}

int il_feasible(il_estimator *e, const il_stage_config *configs, int64_t n_cand, int64_t slo_us,
                uint8_t *out_feasible)
{
    if (!e || n_cand < 0) return IL_ERR_INVALID_ARG;
    if (n_cand == 0) { e->stats = il_stats{}; return IL_OK; }
    if (!configs || !out_feasible) return IL_ERR_INVALID_ARG;
    const int64_t total = n_cand * e->S;
    for (int64_t i = 0; i < total; i++) {
        const il_stage_config &c = configs[i];
        if (c.hw >= e->H || c.max_batch < 1 || c.max_batch > e->Bmax || c.replicas < 1 ||
            c.replicas > IL_MAX_REPLICAS)
            return IL_ERR_BAD_CONFIG;
    }
    IL_CUDA(cudaSetDevice(e->device));
    int rc = ensure_staging(e, n_cand);
    if (rc) return rc;
    IL_CUDA(cudaMemcpyAsync(e->d_cfg, configs, (size_t)total * sizeof(il_stage_config),
                            cudaMemcpyHostToDevice, e->stream));
    // the flags go behind the two output arrays of the staging (which the warp-per-candidate
    // kernels fill with P99 and misses first)
    uint8_t *d_flags = reinterpret_cast<uint8_t *>(e->d_out + 2 * e->d_out_cap);
    rc = il_feasible_device(e, e->d_cfg, n_cand, slo_us, d_flags);
    if (rc) return rc;
    IL_CUDA(cudaMemcpyAsync(out_feasible, d_flags, (size_t)n_cand, cudaMemcpyDeviceToHost, e->stream));
    IL_CUDA(cudaStreamSynchronize(e->stream));
    return IL_OK;
}

int il_measure_int_issue(void *cuda_stream, double *out_warp_inst_per_s, double *out_ms)
{
    if (!out_warp_inst_per_s) return IL_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int dev = 0;
    cudaDeviceProp prop;
    IL_CUDA(cudaGetDevice(&dev));
    IL_CUDA(cudaGetDeviceProperties(&prop, dev));
    unsigned *sink = nullptr;
    cudaEvent_t a = nullptr, b = nullptr;
    cudaError_t ce = cudaMalloc(&sink, sizeof(unsigned));
    if (ce == cudaSuccess) ce = cudaEventCreate(&a);
    if (ce == cudaSuccess) ce = cudaEventCreate(&b);
    const int grid = prop.multiProcessorCount * 8;   // 8 CTAs of 8 warps per SM
    const int iters = 4096;
    if (ce == cudaSuccess) ce = launch_int_issue(sink, grid, 64, st);   // warm-up
    float best = 1e30f;
    for (int rep = 0; rep < 3 && ce == cudaSuccess; rep++) {
        cudaEventRecord(a, st);
        ce = launch_int_issue(sink, grid, iters, st);
        cudaEventRecord(b, st);
        if (ce == cudaSuccess) ce = cudaEventSynchronize(b);
        float ms = 0.f;
        if (ce == cudaSuccess) ce = cudaEventElapsedTime(&ms, a, b);
        best = std::min(best, ms);
    }
    if (a) cudaEventDestroy(a);
    if (b) cudaEventDestroy(b);
    cudaFree(sink);
    if (ce != cudaSuccess) { g_last_cuda_error = (int)ce; return IL_ERR_CUDA; }
    // per inner step: 4 multiply-adds + 4 x (xor, add) = 12 instructions per thread
    const double inst = (double)grid * 8.0 * iters * 16.0 * 12.0;
    *out_warp_inst_per_s = inst / (best * 1e-3);
    if (out_ms) *out_ms = best;
    return IL_OK;
}

}  // extern "C"
