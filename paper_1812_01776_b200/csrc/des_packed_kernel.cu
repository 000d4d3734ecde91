// Batched discrete-event simulation of the InferLine Estimator (Section 4.2),
// one candidate configuration per warp -- packed-record version.
//
// Same stage-by-stage formulation as des_kernel.cu (see the header comment
// there): per stage the arrival stream (times never decrease) is consumed one
// batch at a time,
//
//     t      = max(earliest time a replica is free, arrival[head])
//     b      = min(max batch, number of arrivals from head on with time <= t)
//     finish = t + latency[stage][hw][b-1]            (Section 4.1 profile)
//
// and batches leave in (finish, dispatch order) order.  What differs is the
// data layout and two ways of taking more than one step at a time:
//
//   * a stream element is ONE 64-bit record  (time << q) | query,  q =
//     max(5, ceil(log2 n)); "arrived by t" is the single unsigned compare
//     rec <= (t << q | mask).  Queries that leave the pipeline are written to
//     the candidate's slab as the same kind of record (finish time, query); the
//     percentile kernel turns them into latencies;
//   * a replica slot is ONE 64-bit key  (finish << q) | head-index-at-dispatch.
//     The head index grows with every dispatch, so the key is unique and its
//     unsigned order is exactly (finish, dispatch order): the warp-wide minimum
//     (two redux.sync) yields at once the finish time, which lane owns the slot,
//     and where in the input stream the batch it holds starts;
//   * the next 128 arrivals sit in four registers per lane, refilled 32 at a
//     time one rotation ahead of use, so no global load is on the serial chain;
//     the queue count is two or three ballots and a funnel shift;
//   * a stage with max batch 1 is a max-plus scan over 32 queries at a time
//     (run_stage_mb1);
//   * while arrivals find a free replica on arrival and do not share a time
//     stamp, every batch is a single query: up to 31 such dispatches are
//     verified and committed at once (the "run" step in run_stage).
//
// The host selects this kernel when every time the simulation can reach fits
// in 63 - q bits.
#include "il_internal.h"

namespace il {

namespace {

constexpr uint64_t kNeverKey = ~0ull;
constexpr int kMinRun = 3;          // shortest run of single dispatches worth committing at once

enum RouteKind { kForward = 0, kBranch = 1 };

struct WarpCtx {
    int lane;
    unsigned lt_mask;
    uint32_t qmask;
    int qbits;
    const uint8_t *bits;
    uint64_t *stage_buf;     // shared memory, 32 records: ordering buffer of the run step
    uint64_t *slot_key;      // shared memory, 32 slot keys
    uint32_t *slot_q;        // shared memory, 32 slot query ids
    int *slot_b;             // shared memory, 32 slot batch sizes
};

__device__ __forceinline__ uint64_t ld_rec(const uint64_t *in, int idx, int n_in)
{
    return idx < n_in ? in[idx] : kNeverKey;
}

// Where one stage's completions go: the next stage's stream, or the slab (a
// query that leaves), per value of the branch bit.
struct Sink {
    uint64_t *out_a, *out_b;
    int tail_a, tail_b;
    int bit;
};

// Appends the records held by lanes [0, n_act) in lane order.
template <int KIND>
__device__ __forceinline__ void append(const WarpCtx &w, Sink &sk, const uint64_t rec, const int n_act)
{
    const bool act = w.lane < n_act;
    if (KIND == kForward) {
        if (act) sk.out_a[sk.tail_a + w.lane] = rec;
        sk.tail_a += n_act;
    } else {
        bool bitv = false;
        if (act) bitv = (w.bits[(uint32_t)rec & w.qmask] >> sk.bit) & 1;
        const unsigned ma = __ballot_sync(0xffffffffu, act && !bitv);
        const unsigned mb = __ballot_sync(0xffffffffu, act && bitv);
        if (act) {
            if (bitv) sk.out_b[sk.tail_b + __popc(mb & w.lt_mask)] = rec;
            else sk.out_a[sk.tail_a + __popc(ma & w.lt_mask)] = rec;
        }
        sk.tail_a += __popc(ma);
        sk.tail_b += __popc(mb);
    }
}

// One stage of one candidate, max batch >= 2.  WIDE: max batch > 32 (the queue
// count looks at up to 64 arrivals).  Returns the number of batches dispatched.
template <bool WIDE, int KIND>
__device__ __forceinline__ int run_stage(const WarpCtx &w, const int32_t *row, const int mb,
                                         const int R, const int n_in, const uint64_t *in, Sink &sk,
                                         int *status)
{
    const unsigned full = 0xffffffffu;
    const int lane = w.lane;
    const uint32_t qmask = w.qmask;
    const int qb = w.qbits;
    const uint64_t d1k = (uint64_t)(uint32_t)row[0] << qb;   // service time of a single, in key units

    // Hands over the batch a slot held: `b` queries starting at the input index
    // in the key's low bits, finished at the time in its high bits.
    auto emit = [&](const uint64_t mk, const int b, const uint32_t q_first) {
        const uint64_t tbits = mk & ~(uint64_t)qmask;
        if (b == 1) {
            append<KIND>(w, sk, tbits | q_first, 1);
            return;
        }
        const int start = (int)((uint32_t)mk & qmask);
#pragma unroll 1
        for (int j0 = 0; j0 < b; j0 += 32) {
            const int j = j0 + lane;
            uint64_t rec = 0;
            if (j < b) rec = tbits | ((uint32_t)in[start + j] & qmask);
            append<KIND>(w, sk, rec, min(32, b - j0));
        }
    };

    // replica slots: lane r < R holds replica r.  Never-used slots get distinct
    // keys below every real key (real finish times are >= 1, and q >= 5).
    uint64_t key = (lane < R) ? (uint64_t)lane : kNeverKey;
    int sl_b = 0;            // size of the batch the slot holds (0: none)
    uint32_t sl_q = 0;       // its first query
    bool sorted = true;      // slot keys ascend with the lane index

    // lookahead window: A, B, C, D hold in[base + 32 k + lane]
    int base = 0, off = 0, head = 0;
    uint64_t A = ld_rec(in, lane, n_in), B = ld_rec(in, 32 + lane, n_in),
             C = ld_rec(in, 64 + lane, n_in), D = ld_rec(in, 96 + lane, n_in);

    int nbatch = 0;
    int cooldown = 0, penalty = 1;   // when to try the run step again after it did not pay off
    bool try_run = true;

    while (head < n_in) {
        // ------------------------------------------------------------------
        // Run step: how many of the next arrivals are dispatched alone, at
        // their arrival time?  Arrival i (i-th from head, time x_i) is, given
        // that all earlier ones of the run were, iff
        //   (1) x_{i+1} > x_i (nobody else is queued at the dispatch instant), and
        //   (2) fewer than R replicas are busy at x_i: with phi_i old slots free
        //       by x_i, the phi_i-th most recent single of the run has finished,
        //       x_{i - phi_i} + D1 <= x_i (or i < phi_i).
        // The leading m such arrivals are committed together: their keys join
        // the old slots' keys, the m smallest keys of the union are emitted in
        // order and the R largest become the slots.
        // ------------------------------------------------------------------
        if (try_run && cooldown == 0 && __ballot_sync(full, sl_b > 1) == 0) {
            const int pos = off + lane;
            const uint64_t xa = __shfl_sync(full, A, pos & 31), xb = __shfl_sync(full, B, pos & 31);
            const uint64_t X = pos < 32 ? xa : xb;                  // in[head + lane]
            const uint64_t XK = X | qmask;                          // kNever stays kNever
            const uint64_t XKn = __shfl_down_sync(full, XK, 1);
            const uint64_t XK0 = __shfl_sync(full, XK, 0);
            // old slots free by the first arrival are free for the whole run
            const unsigned idle0 = __ballot_sync(full, key <= XK0);
            const unsigned busy = __ballot_sync(full, lane < R && key > XK0);
            int phi = __popc(idle0);
            for (unsigned bm = busy; bm; bm &= bm - 1) {
                const uint64_t kr = __shfl_sync(full, key, __ffs(bm) - 1);
                phi += (kr <= XK);
            }
            const uint64_t Y = __shfl_sync(full, XK, max(lane - phi, 0));
            const bool ok = (X != kNeverKey) && (lane < 31) && (XKn > XK) &&
                            (lane < phi || Y + d1k <= XK);
            const int m = __ffs(~__ballot_sync(full, ok)) - 1;       // lane 31 is never ok
            if (m >= kMinRun) {
                const uint64_t NK = (XK - qmask) + d1k + (uint64_t)(head + lane);
                // rank of every old key among the old keys
                int orank = lane;
                if (!sorted) {
                    orank = 0;
                    for (int r = 0; r < R; r++) orank += (__shfl_sync(full, key, r) < key);
                }
                // merge: o = old keys below my new key, e = new keys below my old key
                int o = __popc(idle0), e = 0;
                const unsigned run_mask = (1u << m) - 1u;
                for (unsigned bm = busy; bm; bm &= bm - 1) {
                    const int r = __ffs(bm) - 1;
                    const uint64_t kr = __shfl_sync(full, key, r);
                    const unsigned below = __ballot_sync(full, NK < kr) & run_mask;
                    o += (kr < NK);
                    if (lane == r) e = __popc(below);
                }
                // never-used slots hold the smallest keys and emit nothing
                const int z = __popc(__ballot_sync(full, lane < R && sl_b == 0));
                const int u_new = lane + o;          // union rank of my new key (lane < m)
                const int u_old = orank + e;         // union rank of my old key (lane < R)
                // emitted: union rank < m, at output position rank - z
                if (lane < m && u_new < m)
                    w.stage_buf[u_new - z] = (NK & ~(uint64_t)qmask) | ((uint32_t)X & qmask);
                if (lane < R && sl_b == 1 && u_old < m)
                    w.stage_buf[u_old - z] = (key & ~(uint64_t)qmask) | sl_q;
                // kept: union rank >= m, in slot lane rank - m
                if (lane < m && u_new >= m) {
                    w.slot_key[u_new - m] = NK;
                    w.slot_q[u_new - m] = (uint32_t)X & qmask;
                    w.slot_b[u_new - m] = 1;
                }
                if (lane < R && u_old >= m) {
                    w.slot_key[u_old - m] = key;
                    w.slot_q[u_old - m] = sl_q;
                    w.slot_b[u_old - m] = sl_b;
                }
                __syncwarp();
                const int n_emit = m - min(z, m);
                const uint64_t rec = lane < n_emit ? w.stage_buf[lane] : 0;
                if (lane < R) { key = w.slot_key[lane]; sl_q = w.slot_q[lane]; sl_b = w.slot_b[lane]; }
                __syncwarp();
                append<KIND>(w, sk, rec, n_emit);
                sorted = true;
                penalty = 1;
                head += m; off += m; nbatch += m;
                while (off >= 32) {
                    A = B; B = C; C = D;
                    base += 32;
                    D = ld_rec(in, base + 96 + lane, n_in);
                    off -= 32;
                }
                continue;
            }
            cooldown = penalty;
            penalty = min(penalty * 2, 64);
        }
        if (cooldown > 0) cooldown--;

        // ------------------------------------------------------------------
        // Single step: one batch.
        // ------------------------------------------------------------------
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

        if (pb > 0) {
            const uint32_t pq = __reduce_add_sync(full, mine ? sl_q : 0u);
            emit(mk, pb, pq);
        }
        if (mine) { key = nk; sl_b = cnt; sl_q = (uint32_t)a_head & qmask; }
        sorted = false;
        // a single that did not wait suggests a calm stretch: worth trying a run
        try_run = (cnt == 1) && (k2 >= k1);
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
        if (pb > 0) {
            const uint32_t pq = __reduce_add_sync(full, mine ? sl_q : 0u);
            emit(mk, pb, pq);
        }
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
__device__ __forceinline__ int run_stage_mb1(const WarpCtx &w, const int32_t *row, const int R,
                                             const int n_in, const uint64_t *in, Sink &sk)
{
    const unsigned full = 0xffffffffu;
    const int lane = w.lane;
    const uint32_t qmask = w.qmask;
    const int qb = w.qbits;
    const int64_t D = row[0];
    const int64_t kLongAgo = -(INT64_C(1) << 62);
    // where in the previous 32 the chain of this lane continues, and how many services lie between
    const int hops = lane / R + 1;
    const int carry_src = 32 + lane - hops * R;
    const int64_t carry_add = (int64_t)hops * D;
    int64_t prev = kLongAgo;            // start times of the previous 32 queries

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
        const uint64_t orec = ((uint64_t)(v + D) << qb) | ((uint32_t)cur & qmask);
        append<KIND>(w, sk, orec, min(32, n_in - base));
    }
    return n_in;
}

}  // namespace

__global__ void __launch_bounds__(kWarpsPerCta * 32)
des_packed_kernel(const __grid_constant__ DesParams p)
{
    extern __shared__ int32_t s_lat[];
    __shared__ uint64_t s_stage[kWarpsPerCta][32];
    __shared__ uint64_t s_slot_key[kWarpsPerCta][32];
    __shared__ uint32_t s_slot_q[kWarpsPerCta][32];
    __shared__ int s_slot_b[kWarpsPerCta][32];
    const int n_tab = p.S * p.H * p.Bmax;
    for (int i = threadIdx.x; i < n_tab; i += blockDim.x) s_lat[i] = p.lat[i];
    __syncthreads();

    const unsigned full = 0xffffffffu;
    const int wid = threadIdx.x >> 5;
    WarpCtx w;
    w.lane = threadIdx.x & 31;
    w.lt_mask = (1u << w.lane) - 1u;
    w.qbits = p.qbits;
    w.qmask = (1u << p.qbits) - 1u;
    w.bits = p.bits;
    w.stage_buf = s_stage[wid];
    w.slot_key = s_slot_key[wid];
    w.slot_q = s_slot_q[wid];
    w.slot_b = s_slot_b[wid];
    const int lane = w.lane;
    const int64_t slot = (int64_t)blockIdx.x * kWarpsPerCta + wid;
    uint64_t *my_rec = reinterpret_cast<uint64_t *>(p.ws_time) + slot * p.slot_elems;
    unsigned long long batches = 0, alg_ops = 0;

    for (;;) {
        unsigned long long c = 0;
        if (lane == 0) c = atomicAdd(&p.counters[0], 1ull);
        c = __shfl_sync(full, c, 0);
        if (c >= (unsigned long long)p.n_cand) break;

        uint64_t *slab = reinterpret_cast<uint64_t *>(p.slab + c * p.slab_stride);
        il_stage_config my_cfg = {0, 1, 1, 0};
        if (lane < p.S) my_cfg = p.configs[c * p.S + lane];
        const bool bad = lane < p.S && (my_cfg.hw >= p.H || my_cfg.max_batch < 1 ||
                                        my_cfg.max_batch > p.Bmax || my_cfg.replicas < 1 ||
                                        my_cfg.replicas > IL_MAX_REPLICAS);
        if (__any_sync(full, bad)) {
            if (lane == 0) atomicCAS(p.status, 0, IL_ERR_BAD_CONFIG);
            for (int i = lane; i < p.n; i += 32) slab[i] = 0;
            continue;
        }

        int exits = 0;
        for (int s = 0; s < p.S; s++) {
            const int n_in = p.n_s[s];
            if (n_in == 0) continue;
            const int hw = __shfl_sync(full, (int)my_cfg.hw, s);
            const int mb = __shfl_sync(full, (int)my_cfg.max_batch, s);
            const int R = __shfl_sync(full, (int)my_cfg.replicas, s);
            const int32_t *row = s_lat + (s * p.H + hw) * p.Bmax;
            const uint64_t *in = (s == 0) ? p.ptrace : my_rec + p.buf_off[s];
            const int da = p.dest_a[s], db = p.dest_b[s];
            Sink sk;
            sk.bit = p.bit[s];
            sk.out_a = da < 0 ? slab + exits : my_rec + p.buf_off[da];
            sk.out_b = db < 0 ? slab + exits : my_rec + p.buf_off[db];
            sk.tail_a = 0; sk.tail_b = 0;
            const bool branch = sk.bit >= 0;
            int nb;
            if (mb == 1) {
                nb = branch ? run_stage_mb1<kBranch>(w, row, R, n_in, in, sk)
                            : run_stage_mb1<kForward>(w, row, R, n_in, in, sk);
            } else if (mb > 32) {
                nb = branch ? run_stage<true, kBranch>(w, row, mb, R, n_in, in, sk, p.status)
                            : run_stage<true, kForward>(w, row, mb, R, n_in, in, sk, p.status);
            } else {
                nb = branch ? run_stage<false, kBranch>(w, row, mb, R, n_in, in, sk, p.status)
                            : run_stage<false, kForward>(w, row, mb, R, n_in, in, sk, p.status);
            }
            // a guarded stage has at most one side that leaves the pipeline
            if (!branch) { if (da < 0) exits += sk.tail_a; }
            else exits += (da < 0 ? sk.tail_a : 0) + (db < 0 ? sk.tail_b : 0);
            batches += (unsigned)nb;
            alg_ops += 3ull * (unsigned)n_in + (unsigned long long)nb * (unsigned)(R + mb + 4);
            __syncwarp();   // this stage's stream writes are read by the next stage's other lanes
        }
        if (lane == 0 && exits != p.n) atomicCAS(p.status, 0, IL_ERR_ITER_LIMIT);
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
