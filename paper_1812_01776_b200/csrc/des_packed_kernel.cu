// Batched discrete-event simulation of the InferLine Estimator (Section 4.2),
// one candidate configuration per warp -- packed-record version.
//
// Same stage-by-stage formulation as des_kernel.cu (see the header comment
// there): per stage the sorted arrival stream is consumed one batch at a time,
//
//     t      = max(earliest time a replica is free, arrival[head])
//     b      = min(max batch, number of arrivals from head on with time <= t)
//     finish = t + latency[stage][hw][b-1]            (Section 4.1 profile)
//
// and batches leave in (finish, dispatch order) order.  What differs is the
// data layout, chosen to cut the number of warp instructions per batch:
//
//   * a stream element is ONE 64-bit record  (time << q) | query,  q =
//     max(5, ceil(log2 n)); times along a stream never decrease, and "arrived by
//     t" is the single unsigned compare  rec <= (t << q | mask);
//   * a replica slot is ONE 64-bit key  (finish << q) | head-index-at-dispatch.
//     The head index grows with every dispatch, so the key is unique and its
//     unsigned order is exactly (finish, dispatch order): the warp-wide minimum
//     (two redux.sync) yields at once the finish time, which lane owns the slot,
//     and where in the input stream the batch it holds starts;
//   * the next 128 arrivals sit in four registers per lane, refilled 32 at a
//     time one rotation ahead of use, so no global load is on the serial chain;
//     the queue count is two or three ballots and a funnel shift.
//
// The host selects this kernel when every time the simulation can reach fits
// in 63 - q bits.
#include "il_internal.h"

namespace il {

namespace {

constexpr uint64_t kNeverKey = ~0ull;

enum RouteKind { kForward = 0, kExit = 1, kBranch = 2 };

struct WarpCtx {
    int lane;
    unsigned lt_mask;
    uint32_t qmask;
    int qbits;
};

__device__ __forceinline__ uint64_t ld_rec(const uint64_t *in, int idx, int n_in)
{
    return idx < n_in ? in[idx] : kNeverKey;
}

// One stage of one candidate.  WIDE: max batch > 32 (the queue count looks at
// up to 64 arrivals).  Returns the number of batches dispatched.
template <bool WIDE, int KIND>
__device__ __forceinline__ int run_stage(const DesParams &p, const WarpCtx &w, const int32_t *row,
                                         const int mb, const int R, const int n_in,
                                         const uint64_t *in, uint64_t *out_a, uint64_t *out_b,
                                         const int bit, const bool a_exit, const bool b_exit,
                                         int64_t *__restrict__ slab, int &exits, uint64_t &lat_or,
                                         int *status)
{
    const unsigned full = 0xffffffffu;
    const int lane = w.lane;
    const uint32_t qmask = w.qmask;
    const int qb = w.qbits;
    int tail_a = 0, tail_b = 0;

    // Hands the batch [start, start + b) of the input stream, finished at the
    // time held in the high bits of `mk`, to the next stage / the latency slab.
    auto emit = [&](const uint64_t mk, const int b) {
        const int start = (int)((uint32_t)mk & qmask);
        const uint64_t tbits = mk & ~(uint64_t)qmask;
#pragma unroll 1
        for (int j0 = 0; j0 < b; j0 += 32) {
            const int j = j0 + lane;
            const bool act = j < b;
            if (KIND == kForward) {
                if (act) {
                    const uint32_t q = (uint32_t)in[start + j] & qmask;
                    out_a[tail_a + j] = tbits | q;
                }
            } else if (KIND == kExit) {
                if (act) {
                    const uint32_t q = (uint32_t)in[start + j] & qmask;
                    const int64_t l = (int64_t)(mk >> qb) - p.arrival[q];
                    slab[exits + j] = l;
                    lat_or |= (uint64_t)l;
                }
            } else {
                uint32_t q = 0;
                bool bitv = false;
                if (act) {
                    q = (uint32_t)in[start + j] & qmask;
                    bitv = (p.bits[q] >> bit) & 1;
                }
                const unsigned ma = __ballot_sync(full, act && !bitv);
                const unsigned mb_ = __ballot_sync(full, act && bitv);
                const bool to_exit = bitv ? b_exit : a_exit;
                if (act) {
                    if (to_exit) {
                        // both sides may leave: ranks of the two groups interleave in lane order
                        const unsigned me = (a_exit ? ma : 0u) | (b_exit ? mb_ : 0u);
                        const int64_t l = (int64_t)(mk >> qb) - p.arrival[q];
                        slab[exits + __popc(me & w.lt_mask)] = l;
                        lat_or |= (uint64_t)l;
                    } else if (bitv) {
                        out_b[tail_b + __popc(mb_ & w.lt_mask)] = tbits | q;
                    } else {
                        out_a[tail_a + __popc(ma & w.lt_mask)] = tbits | q;
                    }
                }
                const int na = __popc(ma), nb = __popc(mb_);
                exits += (a_exit ? na : 0) + (b_exit ? nb : 0);
                tail_a += a_exit ? 0 : na;
                tail_b += b_exit ? 0 : nb;
            }
        }
        if (KIND == kForward) tail_a += b;
        if (KIND == kExit) exits += b;
    };

    // replica slots: lane r < R holds replica r.  Idle slots get distinct keys
    // below every real key (real finish times are >= 1, and q >= 5).
    uint64_t key = (lane < R) ? (uint64_t)lane : kNeverKey;
    int sl_b = 0;

    // lookahead window: A, B, C, D hold in[base + 32 k + lane]
    int base = 0, off = 0, head = 0;
    uint64_t A = ld_rec(in, lane, n_in), B = ld_rec(in, 32 + lane, n_in),
             C = ld_rec(in, 64 + lane, n_in), D = ld_rec(in, 96 + lane, n_in);

    int nbatch = 0;
    while (head < n_in) {
        // slot with the smallest (finish, dispatch order)
        const uint32_t khi = (uint32_t)(key >> 32), klo = (uint32_t)key;
        const uint32_t mhi = __reduce_min_sync(full, khi);
        const uint32_t mlo = __reduce_min_sync(full, khi == mhi ? klo : 0xffffffffu);
        const bool mine = (khi == mhi) && (klo == mlo);
        const uint64_t mk = ((uint64_t)mhi << 32) | mlo;
        const int pb = __reduce_add_sync(full, mine ? sl_b : 0);

        // dispatch time as a packed threshold: (t << q) | mask
        const uint64_t a_head = __shfl_sync(full, A, off);
        const uint64_t k1 = mk | qmask, k2 = a_head | qmask;
        const uint64_t thr = k1 > k2 ? k1 : k2;

        // queue length at t, capped at mb
        const unsigned mA = __ballot_sync(full, A <= thr);
        const unsigned mB = __ballot_sync(full, B <= thr);
        int cnt = __popc(__funnelshift_r(mA, mB, off));
        if (WIDE) {
            const unsigned mC = __ballot_sync(full, C <= thr);
            cnt += __popc(__funnelshift_r(mB, mC, off));
        }
        cnt = min(cnt, mb);
        if (cnt < 1) {   // cannot happen: the head element satisfies rec <= thr
            if (lane == 0) atomicCAS(status, 0, IL_ERR_ITER_LIMIT);
            break;
        }

        const uint64_t nk = thr + ((uint64_t)(uint32_t)row[cnt - 1] << qb) + (uint64_t)head - qmask;

        if (pb > 0) emit(mk, pb);
        if (mine) { key = nk; sl_b = cnt; }
        head += cnt;
        off += cnt;
        nbatch++;
        while (off >= 32) {
            A = B; B = C; C = D;
            base += 32;
            D = ld_rec(in, base + 96 + lane, n_in);
            off -= 32;
        }
    }
    // drain what is still in flight, in key order
#pragma unroll 1
    for (int k = 0; k < 32; k++) {
        const uint32_t khi = (uint32_t)(key >> 32), klo = (uint32_t)key;
        const uint32_t mhi = __reduce_min_sync(full, khi);
        const uint32_t mlo = __reduce_min_sync(full, khi == mhi ? klo : 0xffffffffu);
        const uint64_t mk = ((uint64_t)mhi << 32) | mlo;
        if (mk == kNeverKey) break;
        const bool mine = (khi == mhi) && (klo == mlo);
        const int pb = __reduce_add_sync(full, mine ? sl_b : 0);
        if (pb > 0) emit(mk, pb);
        if (mine) { key = kNeverKey; sl_b = 0; }
    }
    return nbatch;
}

// A stage whose max batch is 1.  Every batch is a single query with the same
// service time D = latency[1], so the multi-replica FIFO queue behaves like R
// interleaved single-server queues: query i starts at
//     s_i = max(a_i, s_{i-R} + D)
// and queries leave in arrival order.  Unrolled, s_i is a running maximum of
// a_{i-jR} + j D over j, which 32 lanes evaluate for 32 consecutive queries
// with log2(32/R) shuffle steps plus one carry from the previous 32.
template <int KIND>
__device__ __forceinline__ int run_stage_mb1(const DesParams &p, const WarpCtx &w, const int32_t *row,
                                             const int R, const int n_in, const uint64_t *in,
                                             uint64_t *out_a, uint64_t *out_b, const int bit,
                                             const bool a_exit, const bool b_exit,
                                             int64_t *__restrict__ slab, int &exits, uint64_t &lat_or)
{
    const unsigned full = 0xffffffffu;
    const int lane = w.lane;
    const uint32_t qmask = w.qmask;
    const int qb = w.qbits;
    const int64_t D = row[0];
    const int64_t kLongAgo = -(INT64_C(1) << 62);
    // where in the previous 32 starts the chain of this lane continues, and how many services lie between
    const int hops = lane / R + 1;
    const int carry_src = 32 + lane - hops * R;
    const int64_t carry_add = (int64_t)hops * D;
    int64_t prev = kLongAgo;            // start times of the previous 32 queries
    int tail_a = 0, tail_b = 0;

    uint64_t rec = ld_rec(in, lane, n_in);
    for (int base = 0; base < n_in; base += 32) {
        const uint64_t cur = rec;
        rec = ld_rec(in, base + 32 + lane, n_in);          // next 32, off the dependent chain
        const bool act = base + lane < n_in;
        int64_t v = act ? (int64_t)(cur >> qb) : (INT64_C(1) << 62);
        int64_t mul = D;
        for (int d = R; d < 32; d <<= 1, mul <<= 1) {
            const int64_t u = __shfl_up_sync(full, v, d);
            if (lane >= d && u + mul > v) v = u + mul;
        }
        const int64_t c = __shfl_sync(full, prev, carry_src) + carry_add;
        if (c > v) v = c;
        prev = v;
        const int64_t fin = v + D;
        const uint32_t q = (uint32_t)cur & qmask;
        const uint64_t orec = ((uint64_t)fin << qb) | q;
        if (KIND == kForward) {
            if (act) out_a[base + lane] = orec;
        } else if (KIND == kExit) {
            if (act) {
                const int64_t l = fin - p.arrival[q];
                slab[exits + base + lane] = l;
                lat_or |= (uint64_t)l;
            }
        } else {
            bool bitv = false;
            if (act) bitv = (p.bits[q] >> bit) & 1;
            const unsigned ma = __ballot_sync(full, act && !bitv);
            const unsigned mb_ = __ballot_sync(full, act && bitv);
            const bool to_exit = bitv ? b_exit : a_exit;
            if (act) {
                if (to_exit) {
                    const unsigned me = (a_exit ? ma : 0u) | (b_exit ? mb_ : 0u);
                    const int64_t l = fin - p.arrival[q];
                    slab[exits + __popc(me & w.lt_mask)] = l;
                    lat_or |= (uint64_t)l;
                } else if (bitv) {
                    out_b[tail_b + __popc(mb_ & w.lt_mask)] = orec;
                } else {
                    out_a[tail_a + __popc(ma & w.lt_mask)] = orec;
                }
            }
            const int na = __popc(ma), nb = __popc(mb_);
            exits += (a_exit ? na : 0) + (b_exit ? nb : 0);
            tail_a += a_exit ? 0 : na;
            tail_b += b_exit ? 0 : nb;
        }
    }
    if (KIND == kExit) exits += n_in;
    return n_in;
}

}  // namespace

__global__ void __launch_bounds__(kWarpsPerCta * 32)
des_packed_kernel(const __grid_constant__ DesParams p)
{
    extern __shared__ int32_t s_lat[];
    const int n_tab = p.S * p.H * p.Bmax;
    for (int i = threadIdx.x; i < n_tab; i += blockDim.x) s_lat[i] = p.lat[i];
    __syncthreads();

    const unsigned full = 0xffffffffu;
    WarpCtx w;
    w.lane = threadIdx.x & 31;
    w.lt_mask = (1u << w.lane) - 1u;
    w.qbits = p.qbits;
    w.qmask = (1u << p.qbits) - 1u;
    const int lane = w.lane;
    const int64_t slot = (int64_t)blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5);
    uint64_t *my_rec = reinterpret_cast<uint64_t *>(p.ws_time) + slot * p.slot_elems;
    unsigned long long batches = 0, alg_ops = 0;

    for (;;) {
        unsigned long long c = 0;
        if (lane == 0) c = atomicAdd(&p.counters[0], 1ull);
        c = __shfl_sync(full, c, 0);
        if (c >= (unsigned long long)p.n_cand) break;

        il_stage_config my_cfg = {0, 1, 1, 0};
        if (lane < p.S) my_cfg = p.configs[c * p.S + lane];
        const bool bad = lane < p.S && (my_cfg.hw >= p.H || my_cfg.max_batch < 1 ||
                                        my_cfg.max_batch > p.Bmax || my_cfg.replicas < 1 ||
                                        my_cfg.replicas > IL_MAX_REPLICAS);
        if (__any_sync(full, bad)) {
            if (lane == 0) { atomicCAS(p.status, 0, IL_ERR_BAD_CONFIG); p.lat_or[c] = 0; }
            for (int i = lane; i < p.n; i += 32) p.slab[c * p.slab_stride + i] = 0;
            continue;
        }

        int64_t *slab = p.slab + c * p.slab_stride;
        int exits = 0;
        uint64_t lat_or = 0;

        for (int s = 0; s < p.S; s++) {
            const int n_in = p.n_s[s];
            if (n_in == 0) continue;
            const int hw = __shfl_sync(full, (int)my_cfg.hw, s);
            const int mb = __shfl_sync(full, (int)my_cfg.max_batch, s);
            const int R = __shfl_sync(full, (int)my_cfg.replicas, s);
            const int32_t *row = s_lat + (s * p.H + hw) * p.Bmax;
            const uint64_t *in = (s == 0) ? p.ptrace : my_rec + p.buf_off[s];
            const int da = p.dest_a[s], db = p.dest_b[s], bit = p.bit[s];
            uint64_t *out_a = da < 0 ? nullptr : my_rec + p.buf_off[da];
            uint64_t *out_b = db < 0 ? nullptr : my_rec + p.buf_off[db];
            const int kind = bit >= 0 ? kBranch : (da < 0 ? kExit : kForward);
            int nb;
#define IL_STAGE(WIDE_, KIND_)                                                               \
    nb = run_stage<WIDE_, KIND_>(p, w, row, mb, R, n_in, in, out_a, out_b, bit, da < 0, db < 0, \
                                 slab, exits, lat_or, p.status)
            if (mb == 1) {
                if (kind == kForward)
                    nb = run_stage_mb1<kForward>(p, w, row, R, n_in, in, out_a, out_b, bit, da < 0, db < 0, slab, exits, lat_or);
                else if (kind == kExit)
                    nb = run_stage_mb1<kExit>(p, w, row, R, n_in, in, out_a, out_b, bit, da < 0, db < 0, slab, exits, lat_or);
                else
                    nb = run_stage_mb1<kBranch>(p, w, row, R, n_in, in, out_a, out_b, bit, da < 0, db < 0, slab, exits, lat_or);
            } else if (mb > 32) {
                if (kind == kForward) IL_STAGE(true, kForward);
                else if (kind == kExit) IL_STAGE(true, kExit);
                else IL_STAGE(true, kBranch);
            } else {
                if (kind == kForward) IL_STAGE(false, kForward);
                else if (kind == kExit) IL_STAGE(false, kExit);
                else IL_STAGE(false, kBranch);
            }
#undef IL_STAGE
            batches += (unsigned)nb;
            alg_ops += 3ull * (unsigned)n_in + (unsigned long long)nb * (unsigned)(R + mb + 4);
            __syncwarp();   // this stage's stream writes are read by the next stage's other lanes
        }

        const uint32_t lo = __reduce_or_sync(full, (uint32_t)lat_or);
        const uint32_t hi = __reduce_or_sync(full, (uint32_t)(lat_or >> 32));
        if (lane == 0) {
            p.lat_or[c] = ((uint64_t)hi << 32) | lo;
            if (exits != p.n) atomicCAS(p.status, 0, IL_ERR_ITER_LIMIT);
        }
    }
    if (lane == 0 && batches) { atomicAdd(&p.counters[1], batches); atomicAdd(&p.counters[2], alg_ops); }
}

cudaError_t launch_des_packed(const DesParams &p, int grid, size_t smem, cudaStream_t stream)
{
    des_packed_kernel<<<grid, kWarpsPerCta * 32, smem, stream>>>(p);
    return cudaGetLastError();
}

int des_packed_max_ctas_per_sm(size_t smem)
{
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, des_packed_kernel, kWarpsPerCta * 32, smem) != cudaSuccess)
        return 0;
    return n;
}

}  // namespace il
