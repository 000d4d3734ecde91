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
//     unsigned order is exactly (finish, dispatch order).  The slots are kept
//     sorted across lanes 0..R-1: the next one to be reused is lane 0, and a
//     new batch is inserted with one shuffle, one compare and one ballot;
//   * the next 128 arrivals sit in four registers per lane, refilled 32 at a
//     time one rotation ahead of use, so no global load is on the serial chain;
//     the queue count is two or three ballots and a funnel shift;
//   * a stage with max batch 1 is a max-plus scan over 32 queries at a time
//     (run_stage_mb1);
//   * while no arrival comes in before the previous one has been dispatched,
//     every batch is a single query and the replicas are reused round-robin:
//     up to 31 such dispatches are computed by a scan, verified and committed
//     at once (the "run" step in run_stage).
//
// The host selects this kernel when every time the simulation can reach fits
// in 63 - q bits.
#include "il_internal.h"

namespace il {

namespace {

constexpr uint64_t kNeverKey = ~0ull;
constexpr int kMinRun = 3;          // shortest run of single dispatches worth committing at once (measured: 3-4 best)

enum RouteKind { kForward = 0, kBranch = 1 };

struct WarpCtx {
    int lane;
    unsigned lt_mask;
    uint32_t qmask;
    int qbits;
    const uint8_t *bits;
    int n_queries;           // length of bits
    uint64_t *slot_key;      // shared memory, 32 slot keys: staging for re-ordering the slots
    uint32_t *slot_q;        // shared memory, 32 slot query ids
    int *slot_b;             // shared memory, 32 slot batch sizes
};

// ---------------------------------------------------------------------------
// Where a stage reads its arrival stream from.
//
// GlobalSrc: a stream in global memory (the warp's own inter-stage buffer, or
// the packed trace through L1/L2).
//
// TileSrc: the root stage's stream, i.e. the shared trace, staged through
// shared memory once per CTA.  The trace is cut into tiles of kTileRecs
// records; a ring of kTiles tiles is filled by bulk asynchronous copies
// (cp.async.bulk, completion signalled on an mbarrier per ring slot) and read
// by all warps of the CTA, each at its own pace.  A warp releases a tile when
// its lookahead has moved past it; the warp that releases a tile last re-arms
// the slot and issues the copy of the tile kTiles further on.  Every wait is
// bounded: on a time-out the warp records IL_ERR_ITER_LIMIT and from then on
// reads "no more arrivals", which ends its loops.
// ---------------------------------------------------------------------------
constexpr int kTileLog = 9;
constexpr int kTileRecs = 1 << kTileLog;        // 512 records = 4 KB
constexpr int kTiles = 4;                       // ring depth
constexpr unsigned kTileBytes = kTileRecs * 8;
constexpr int kWaitLimit = 1 << 24;             // polls of an mbarrier before giving up

struct TileRing {
    uint64_t tiles[kTiles][kTileRecs];          // 128-byte aligned by the declaration below
    uint64_t full[kTiles];                      // mbarriers: "the copy into this slot has landed"
    int released[kTiles];                       // warps that are done with the slot's current tile
    int uses[kTiles];                           // how often the slot has been armed
    int base_uses[kTiles];                      // `uses` at the start of the current group
    int group_base;                             // first position (in the order array) of the group
};

__device__ __forceinline__ uint32_t smem_addr(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint64_t *bar, int count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, unsigned parity)
{
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
    return ok != 0;
}

// Waits until the slot's barrier has completed the phase with this parity.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t *bar, unsigned parity)
{
    for (int i = 0; i < kWaitLimit; i++)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

// Arms the slot's barrier for kTileBytes and starts the copy of trace tile `tile` into it.
__device__ __forceinline__ void tile_issue(TileRing *ring, const uint64_t *ptrace, int tile)
{
    const int slot = tile & (kTiles - 1);
    const uint32_t bar = smem_addr(&ring->full[slot]);
    ring->uses[slot]++;
    // order the CTA's earlier generic-proxy reads of the slot before the async-proxy write
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(kTileBytes) : "memory");
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(smem_addr(ring->tiles[slot])), "l"(ptrace + (size_t)tile * kTileRecs), "r"(kTileBytes), "r"(bar)
        : "memory");
}

struct GlobalSrc {
    static constexpr bool kRereadable = true;
    const uint64_t *in;
    bool root;               // the packed trace: the query of record i is i
    // 32 consecutive records starting at the 32-aligned index `idx0`
    __device__ __forceinline__ uint64_t load32(int idx0, int lane, int n_in)
    {
        return idx0 + lane < n_in ? in[idx0 + lane] : kNeverKey;
    }
    __device__ __forceinline__ uint32_t query_at(int idx, uint32_t qmask) const
    {
        return root ? (uint32_t)idx : ((uint32_t)in[idx] & qmask);
    }
    __device__ __forceinline__ void finish(int, int) {}
};

struct TileSrc {
    static constexpr bool kRereadable = false;   // released tiles are gone
    TileRing *ring;
    const uint64_t *ptrace;
    int n_tiles;
    int cur;                 // oldest tile this warp has not released
    int waited;              // newest tile this warp has seen land
    bool dead;               // a wait timed out
    int *status;

    __device__ __forceinline__ void release(int tile, int lane)
    {
        __syncwarp();
        if (lane == 0) {
            const int slot = tile & (kTiles - 1);
            if (atomicAdd(&ring->released[slot], 1) == kWarpsPerCta - 1) {
                ring->released[slot] = 0;
                __threadfence_block();
                if (tile + kTiles < n_tiles) tile_issue(ring, ptrace, tile + kTiles);
            }
        }
    }
    // Waits (bounded) until tile t has landed.  Tiles must be waited for in
    // order before they are read or released: a slot is only re-armed after all
    // warps have released its previous tile, so waiting keeps the per-slot
    // release counts from mixing two tiles.
    __device__ __forceinline__ bool wait_tile(int t, int lane)
    {
        static_assert(kTiles == 4, "tile / kTiles is written as a shift by 2");
        const int slot = t & (kTiles - 1);
        const unsigned parity = (unsigned)(ring->base_uses[slot] + (t >> 2)) & 1u;
        if (!mbar_wait_bounded(&ring->full[slot], parity)) {
            if (lane == 0) atomicCAS(status, 0, IL_ERR_ITER_LIMIT);
            dead = true;
            return false;
        }
        waited = t;
        return true;
    }
    __device__ __forceinline__ uint64_t load32(int idx0, int lane, int n_in)
    {
        if (idx0 >= n_in || dead) return kNeverKey;
        const int t = idx0 >> kTileLog;
        while (cur < t) { release(cur, lane); cur++; }
        if (t > waited && !wait_tile(t, lane)) return kNeverKey;
        // the trace is padded with "never" records up to a whole tile
        return ring->tiles[t & (kTiles - 1)][(idx0 & (kTileRecs - 1)) + lane];
    }
    __device__ __forceinline__ uint32_t query_at(int idx, uint32_t) const { return (uint32_t)idx; }
    // releases whatever this warp still holds, so that the ring can move on for the others
    __device__ __forceinline__ void finish(int lane, int)
    {
        while (cur < n_tiles) {
            if (cur > waited && !dead) wait_tile(cur, lane);
            release(cur, lane);
            cur++;
        }
    }
};

// Where one stage's completions go: the next stage's stream, or the slab (a
// query that leaves), per value of the branch bit.
struct Sink {
    uint64_t *out_a, *out_b;
    int tail_a, tail_b;
    int bit;
    int size_a, size_b;      // records each side can take (compared with in the checked build)
    int *status;
};

// Appends the records held by lanes [0, n_act) in lane order.
template <int KIND>
__device__ __forceinline__ void append(const WarpCtx &w, Sink &sk, const uint64_t rec, const int n_act)
{
    const bool act = w.lane < n_act;
    if (KIND == kForward) {
        if (act && IL_IN_RANGE(sk.tail_a + w.lane, sk.size_a, sk.status)) sk.out_a[sk.tail_a + w.lane] = rec;
        sk.tail_a += n_act;
    } else {
        bool bitv = false;
        if (act && IL_IN_RANGE((uint32_t)rec & w.qmask, w.n_queries, sk.status))
            bitv = (w.bits[(uint32_t)rec & w.qmask] >> sk.bit) & 1;
        const unsigned ma = __ballot_sync(0xffffffffu, act && !bitv);
        const unsigned mb = __ballot_sync(0xffffffffu, act && bitv);
        if (act) {
            const int at = bitv ? sk.tail_b + __popc(mb & w.lt_mask) : sk.tail_a + __popc(ma & w.lt_mask);
            if (IL_IN_RANGE(at, bitv ? sk.size_b : sk.size_a, sk.status)) {
                if (bitv) sk.out_b[at] = rec;
                else sk.out_a[at] = rec;
            }
        }
        sk.tail_a += __popc(ma);
        sk.tail_b += __popc(mb);
    }
}

// Where a stage stands when the 32-bit loop (run_stage_narrow) hands it over to
// the 64-bit loop (run_stage).
struct StageState {
    bool resume;         // false: start the stage from scratch
    int head;            // arrivals consumed so far
    int nbatch;          // batches dispatched so far
    uint64_t key;        // this lane's slot
    int sl_b;
    uint32_t sl_q;
};

// One stage of one candidate, max batch >= 2.  WIDE: max batch > 32 (the queue
// count looks at up to 64 arrivals).  Returns the number of batches dispatched.
//
// Replica slots live in lanes 0..R-1, always sorted by key, so the next slot to
// be reused is lane 0 and the one after it lane 1.
template <bool WIDE, int KIND, class Src>
__device__ __forceinline__ int run_stage(const WarpCtx &w, const int32_t *row, const int mb,
                                      const int R, const int n_in, Src &src, Sink &sk,
                                      int *status, const StageState &st)
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
            if (j < b) rec = tbits | src.query_at(start + j, qmask);
            append<KIND>(w, sk, rec, min(32, b - j0));
        }
    };

    // Never-used slots get distinct keys below every real key (real finish
    // times are >= 1, and q >= 5); lanes >= R never hold a slot.
    uint64_t key = (lane < R) ? (uint64_t)lane : kNeverKey;
    int sl_b = 0;            // size of the batch the slot holds (0: none)
    uint32_t sl_q = 0;       // its first query
    int head = 0, nbatch = 0;
    if (st.resume) { key = st.key; sl_b = st.sl_b; sl_q = st.sl_q; head = st.head; nbatch = st.nbatch; }

    // lookahead window: A, B, C, D hold in[base + 32 k + lane]
    int base = head & ~31, off = head & 31;
    uint64_t A = src.load32(base, lane, n_in), B = src.load32(base + 32, lane, n_in),
             C = src.load32(base + 64, lane, n_in), D = src.load32(base + 96, lane, n_in);

    int cooldown = 0, penalty = 1;   // when to try the run step again after it did not pay off
    // the slot in lane 0, known to every lane
    uint64_t m1 = __shfl_sync(full, key, 0);
    int pb1 = __shfl_sync(full, sl_b, 0);
    uint32_t pq1 = __shfl_sync(full, sl_q, 0);

    while (head < n_in) {
        // ------------------------------------------------------------------
        // Run step.  While every batch is a single query (service time D1),
        // the R replicas are reused round-robin: with the old slots' finish
        // times g_0 <= ... <= g_{R-1}, the i-th next arrival starts at
        //     s_i = max(x_i, g_i)            (i < R)
        //     s_i = max(x_i, s_{i-R} + D1)   (i >= R)
        // as long as the old slots reused so far finish by s_0 + D1, and it is
        // dispatched alone iff x_{i+1} > s_i.  The s_i are a
        // max-plus scan over the lanes; the leading m arrivals that pass are
        // committed at once.  Slots are popped in the order g_0.., then the new
        // finishes, so the first m of that sequence are emitted and the last R
        // become the slots.
        // ------------------------------------------------------------------
        if (cooldown == 0) {
            const int pos = off + lane;
            const uint64_t xa = __shfl_sync(full, A, pos & 31), xb = __shfl_sync(full, B, pos & 31);
            const uint64_t X = pos < 32 ? xa : xb;                  // in[head + lane]
            const uint64_t XK = X | qmask;                          // kNever stays kNever
            const uint64_t XKn = __shfl_down_sync(full, XK, 1);
            // a start is never before the arrival, so arrivals that share a time stamp bound the run
            if (__ffs(~__ballot_sync(full, X != kNeverKey && lane < 31 && XKn > XK)) - 1 < kMinRun) goto single_step;
            const uint64_t gk = key | qmask;
            uint64_t v = (lane < R && gk > XK) ? gk : XK;
            uint64_t mul = d1k;
            for (int d = R; d < 32; d <<= 1, mul <<= 1) {
                const uint64_t u = __shfl_up_sync(full, v, d);
                if (lane >= d && u + mul > v && v != kNeverKey) v = u + mul;
            }
            const uint64_t f0 = __shfl_sync(full, v, 0) + d1k;
            const bool ok = (X != kNeverKey) && (lane < 31) && (XKn > v);
            int m = __ffs(~__ballot_sync(full, ok)) - 1;             // lane 31 is never ok
            // old slots that finish after the first new single ("late") are not
            // reused in round-robin order: the run must end before their turn
            const int c0 = __popc(__ballot_sync(full, lane < R && gk <= f0));   // a prefix of the lanes
            if (c0 < R) m = min(m, c0);
            if (m >= kMinRun) {
                const uint64_t NK = (v - qmask) + d1k + (uint64_t)(head + lane);
                const uint32_t xq = (uint32_t)X & qmask;
                // emit old slots 0 .. min(m, R) - 1 in lane order; never-used ones
                // (the lowest z lanes) hold nothing, slots with a larger batch go one by one
                const int z = __popc(__ballot_sync(full, lane < R && sl_b == 0));
                const int n_old = min(m, R);
                const uint64_t oldrec = (key & ~(uint64_t)qmask) | sl_q;
                unsigned multi = __ballot_sync(full, lane < n_old && sl_b > 1);
                int p0 = min(z, n_old);
                while (p0 < n_old) {
                    const int nxt = multi ? __ffs(multi) - 1 : n_old;
                    if (nxt > p0) append<KIND>(w, sk, __shfl_sync(full, oldrec, (lane + p0) & 31), nxt - p0);
                    if (nxt < n_old) {
                        emit(__shfl_sync(full, key, nxt), __shfl_sync(full, sl_b, nxt), __shfl_sync(full, sl_q, nxt));
                        multi &= multi - 1;
                    }
                    p0 = nxt + 1;
                }
                // ... then the new singles 0 .. m - R - 1
                if (m > R) append<KIND>(w, sk, (NK & ~(uint64_t)qmask) | xq, m - R);
                if (c0 >= R) {
                    // new slots: positions m .. m + R - 1 of the sequence (old 0..R-1, new 0..m-1)
                    const bool take_old = m + lane < R;
                    const int src_old = (m + lane) & 31, src_new = (m + lane - R) & 31;
                    const uint64_t k_o = __shfl_sync(full, key, src_old), k_n = __shfl_sync(full, NK, src_new);
                    const uint32_t q_o = __shfl_sync(full, sl_q, src_old), q_n = __shfl_sync(full, xq, src_new);
                    const int b_o = __shfl_sync(full, sl_b, src_old);
                    if (lane < R) {
                        key = take_old ? k_o : k_n;
                        sl_q = take_old ? q_o : q_n;
                        sl_b = take_old ? b_o : 1;
                    }
                } else {
                    // m <= c0 < R: kept are old m..c0-1 (all before the new ones), then the
                    // new singles merged with the late old slots c0..R-1
                    int above = 0, below = 0;   // late old keys below my new key / new keys below my late old key
                    for (int r = c0; r < R; r++) {
                        const uint64_t kr = __shfl_sync(full, key, r);
                        const unsigned lt = __ballot_sync(full, lane < m && NK < kr);
                        above += (kr < NK);
                        if (lane == r) below = __popc(lt);
                    }
                    if (lane >= m && lane < R) {
                        const int dst = lane < c0 ? lane - m : lane - m + below;
                        w.slot_key[dst] = key; w.slot_q[dst] = sl_q; w.slot_b[dst] = sl_b;
                    }
                    if (lane < m) {
                        const int dst = c0 - m + lane + above;
                        w.slot_key[dst] = NK; w.slot_q[dst] = xq; w.slot_b[dst] = 1;
                    }
                    __syncwarp();
                    if (lane < R) { key = w.slot_key[lane]; sl_q = w.slot_q[lane]; sl_b = w.slot_b[lane]; }
                    __syncwarp();
                }
                penalty = 1;
                head += m; off += m; nbatch += m;
                while (off >= 32) {
                    A = B; B = C; C = D;
                    base += 32;
                    D = src.load32(base + 96, lane, n_in);
                    off -= 32;
                }
                m1 = __shfl_sync(full, key, 0);
                pb1 = __shfl_sync(full, sl_b, 0);
                pq1 = __shfl_sync(full, sl_q, 0);
                continue;
            }
            cooldown = penalty;
            penalty = min(penalty * 2, 64);
        }
        if (cooldown > 0) cooldown--;
    single_step:
        // ------------------------------------------------------------------
        // Single step: one batch.  (m1, pb1, pq1) is the slot in lane 0.
        // ------------------------------------------------------------------
        // the slot that will be first once lane 0's is gone: lane 1, or the new batch
        const uint64_t m2 = __shfl_sync(full, key, 1);
        const int pb2 = __shfl_sync(full, sl_b, 1);
        const uint32_t pq2 = __shfl_sync(full, sl_q, 1);

        // dispatch time as a packed threshold: (t << q) | mask
        const uint64_t a_head = __shfl_sync(full, A, off);
        const uint64_t k1 = m1 | qmask, k2 = a_head | qmask;
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
        const uint32_t qh = (uint32_t)a_head & qmask;

        if (pb1 > 0) emit(m1, pb1, pq1);

        // drop lane 0's slot and insert the new one at its place in the order
        uint64_t u = __shfl_down_sync(full, key, 1);
        const int ub = __shfl_down_sync(full, sl_b, 1);
        const uint32_t uq = __shfl_down_sync(full, sl_q, 1);
        if (lane == 31) u = kNeverKey;
        const bool le = u < nk;
        const bool here = __ballot_sync(full, le) == w.lt_mask;
        key = le ? u : (here ? nk : key);
        sl_b = le ? ub : (here ? cnt : sl_b);
        sl_q = le ? uq : (here ? qh : sl_q);
        const bool second_first = m2 < nk;
        m1 = second_first ? m2 : nk;
        pb1 = second_first ? pb2 : cnt;
        pq1 = second_first ? pq2 : qh;

        head += cnt;
        off += cnt;
        nbatch++;
        while (off >= 32) {
            A = B; B = C; C = D;
            base += 32;
            D = src.load32(base + 96, lane, n_in);
            off -= 32;
        }
    }
    // drain what is still in flight: slots are in key order
#pragma unroll 1
    for (int r = 0; r < R; r++) {
        const uint64_t mk = __shfl_sync(full, key, r);
        const int pb = __shfl_sync(full, sl_b, r);
        const uint32_t pq = __shfl_sync(full, sl_q, r);
        if (pb > 0) emit(mk, pb, pq);
    }
    src.finish(lane, n_in);
    return nbatch;
}

// ---------------------------------------------------------------------------
// The same stage loop in 32-bit arithmetic.
//
// Times are kept relative to an epoch E (a 64-bit value known to every lane),
// as unsigned 32-bit offsets below kNarrowLimit; a slot is (finish offset,
// start index) in two registers, ordered by finish and, at equal finish, by
// start -- since a new batch starts after every batch in flight, "<=" on the
// finish offsets alone decides where it goes.  Everything else is the 64-bit
// loop above, instruction for instruction at half the width.  When an offset
// would leave the range the epoch is moved forward to the oldest time still
// needed (the head arrival, or the finish of the oldest batch not yet handed
// over); if that does not help (a batch or a gap in the arrivals spans more than
// the range) the stage continues in the 64-bit loop from the state reached.
// Needs every table entry of the row to be below kNarrowLatLimit.
// ---------------------------------------------------------------------------
constexpr uint32_t kNarrowLimit = 1u << 30;
constexpr uint32_t kNarrowLatLimit = 1u << 24;     // 32 services still fit below the limit
constexpr uint32_t kFar = 0x7fffffffu;             // an arrival beyond the range (still a real record)
constexpr uint32_t kNever32 = 0xffffffffu;         // no record

template <bool WIDE, int KIND, class Src>
__device__ __forceinline__ int run_stage_narrow(const WarpCtx &w, const int32_t *row, const int mb,
                                             const int R, const int n_in, Src &src, Sink &sk,
                                             int *status)
{
    const unsigned full = 0xffffffffu;
    const int lane = w.lane;
    const uint32_t qmask = w.qmask;
    const int qb = w.qbits;
    const uint32_t d1 = (uint32_t)row[0];

    uint64_t E = 0;                                 // epoch, set from the first arrival below

    auto mkrec = [&](const uint32_t fin, const uint32_t q) -> uint64_t {
        return ((E + fin) << qb) | q;
    };
    // Hands over the batch a slot held (b queries from input index `start`, finished at offset fin).
    auto emit = [&](const uint32_t fin, const int b, const uint32_t q_first, const int start) {
        if (b == 1) {
            append<KIND>(w, sk, mkrec(fin, q_first), 1);
            return;
        }
#pragma unroll 1
        for (int j0 = 0; j0 < b; j0 += 32) {
            const int j = j0 + lane;
            uint64_t rec = 0;
            if (j < b) rec = mkrec(fin, src.query_at(start + j, qmask));
            append<KIND>(w, sk, rec, min(32, b - j0));
        }
    };

    // slots, sorted over lanes 0..R-1 by (fin, sl_s); never-used slots have fin 0 and hold nothing
    uint32_t fin = (lane < R) ? 0u : kNever32;
    int sl_b = 0, sl_s = lane;
    uint32_t sl_q = 0;

    int base = 0, off = 0, head = 0, nbatch = 0;
    uint32_t At, Bt, Ct, Dt, Aq, Bq, Cq, Dq;
    auto load_win = [&](const int idx0, uint32_t &t, uint32_t &q) {
        const uint64_t rec = src.load32(idx0, lane, n_in);
        q = (uint32_t)rec & qmask;
        if (rec == kNeverKey) { t = kNever32; return; }
        const uint64_t rel = (rec >> qb) - E;       // arrivals before the epoch only occur in a backlog:
        t = (rec >> qb) < E ? 0u                    //   "already there" is all that matters
          : (rel >= kNarrowLimit ? kFar : (uint32_t)rel);
    };
    {
        const uint64_t first = src.load32(0, lane, n_in);
        E = __shfl_sync(full, first, 0) >> qb;
    }
    load_win(0, At, Aq); load_win(32, Bt, Bq); load_win(64, Ct, Cq); load_win(96, Dt, Dq);

    int cooldown = 0, penalty = 1;
    uint32_t m1 = 0; int pb1 = 0, ps1 = 0; uint32_t pq1 = 0;    // the slot in lane 0
    bool bail = false;

    // Moves the epoch forward to the oldest time still needed.  Returns false if that is no progress.
    auto re_epoch = [&]() -> bool {
        const uint32_t ah = __shfl_sync(full, off < 32 ? At : Bt, off & 31);
        const uint32_t held = __reduce_min_sync(full, (lane < R && sl_b > 0) ? fin : kNever32);
        const uint32_t delta = min(ah == kFar ? kNever32 : ah, held);
        uint32_t d = delta;
        if (ah == kFar && held == kNever32) {
            // nothing in flight and the next arrival is beyond the range: jump to it
            const uint64_t rec = src.load32(head & ~31, lane, n_in);
            const uint64_t t = __shfl_sync(full, rec, head & 31) >> qb;
            E = t; d = 0;
            if (lane < R) fin = 0;
        } else {
            if (d == 0 || d == kNever32) return false;
            E += d;
            if (lane < R) fin = fin > d ? fin - d : 0u;
        }
        load_win(base, At, Aq); load_win(base + 32, Bt, Bq); load_win(base + 64, Ct, Cq); load_win(base + 96, Dt, Dq);
        m1 = __shfl_sync(full, fin, 0);
        return true;
    };

    while (head < n_in) {
        // the head arrival must be in range to be dispatched here
        uint32_t ah = __shfl_sync(full, At, off);
        if (ah >= kNarrowLimit / 2 || m1 >= kNarrowLimit / 2) {
            if (ah == kNever32) break;      // cannot happen while head < n_in
            if (!re_epoch()) { bail = true; break; }
            ah = __shfl_sync(full, At, off);
            if (ah >= kNarrowLimit / 2 || __shfl_sync(full, fin, 0) >= kNarrowLimit / 2) { bail = true; break; }
        }
        // ---------------- run step (see run_stage) ----------------
        if (cooldown == 0) {
            const int pos = off + lane;
            const uint32_t xa = __shfl_sync(full, At, pos & 31), xb = __shfl_sync(full, Bt, pos & 31);
            const uint32_t X = pos < 32 ? xa : xb;
            const uint32_t Xn = __shfl_down_sync(full, X, 1);
            const bool valid = X < kNarrowLimit / 2;
            // a start is never before the arrival, so arrivals that share a time stamp bound the run
            if (__ffs(~__ballot_sync(full, valid && lane < 31 && Xn > X)) - 1 < kMinRun) { cooldown = 1; goto single_step; }
            uint32_t v = (lane < R && fin > X) ? fin : X;
            uint32_t mul = d1;
            for (int d = R; d < 32; d <<= 1, mul <<= 1) {
                const uint32_t u = __shfl_up_sync(full, v, d);
                if (lane >= d && valid && u + mul > v) v = u + mul;
            }
            const uint32_t f0 = __shfl_sync(full, v, 0) + d1;
            // a start beyond half the range ends the run (the epoch moves before the next step)
            const bool ok = valid && (lane < 31) && (Xn > v) && (v < kNarrowLimit / 2);
            int m = __ffs(~__ballot_sync(full, ok)) - 1;
            const int c0 = __popc(__ballot_sync(full, lane < R && fin <= f0));
            if (c0 < R) m = min(m, c0);
            if (m >= kMinRun) {
                const uint32_t NF = v + d1;
                const uint32_t qa = __shfl_sync(full, Aq, pos & 31), qb2 = __shfl_sync(full, Bq, pos & 31);
                const uint32_t xq = pos < 32 ? qa : qb2;
                const int z = __popc(__ballot_sync(full, lane < R && sl_b == 0));
                const int n_old = min(m, R);
                const uint64_t oldrec = mkrec(fin, sl_q);
                unsigned multi = __ballot_sync(full, lane < n_old && sl_b > 1);
                int p0 = min(z, n_old);
                while (p0 < n_old) {
                    const int nxt = multi ? __ffs(multi) - 1 : n_old;
                    if (nxt > p0) append<KIND>(w, sk, __shfl_sync(full, oldrec, (lane + p0) & 31), nxt - p0);
                    if (nxt < n_old) {
                        emit(__shfl_sync(full, fin, nxt), __shfl_sync(full, sl_b, nxt),
                             __shfl_sync(full, sl_q, nxt), __shfl_sync(full, sl_s, nxt));
                        multi &= multi - 1;
                    }
                    p0 = nxt + 1;
                }
                if (m > R) append<KIND>(w, sk, mkrec(NF, xq), m - R);
                if (c0 >= R) {
                    const bool take_old = m + lane < R;
                    const int src_old = (m + lane) & 31, src_new = (m + lane - R) & 31;
                    const uint32_t f_o = __shfl_sync(full, fin, src_old), f_n = __shfl_sync(full, NF, src_new);
                    const uint32_t q_o = __shfl_sync(full, sl_q, src_old), q_n = __shfl_sync(full, xq, src_new);
                    const int b_o = __shfl_sync(full, sl_b, src_old);
                    const int s_o = __shfl_sync(full, sl_s, src_old);
                    if (lane < R) {
                        fin = take_old ? f_o : f_n;
                        sl_q = take_old ? q_o : q_n;
                        sl_b = take_old ? b_o : 1;
                        sl_s = take_old ? s_o : head + src_new;
                    }
                } else {
                    int above = 0, below = 0;
                    for (int r = c0; r < R; r++) {
                        const uint32_t fr = __shfl_sync(full, fin, r);
                        const unsigned lt = __ballot_sync(full, lane < m && NF < fr);
                        above += (fr <= NF);
                        if (lane == r) below = __popc(lt);
                    }
                    // re-ordering through shared memory: key holds the finish offset, q and b as usual,
                    // the start index travels in the upper half of the key word
                    if (lane >= m && lane < R) {
                        const int dst = lane < c0 ? lane - m : lane - m + below;
                        w.slot_key[dst] = ((uint64_t)(uint32_t)sl_s << 32) | fin; w.slot_q[dst] = sl_q; w.slot_b[dst] = sl_b;
                    }
                    if (lane < m) {
                        const int dst = c0 - m + lane + above;
                        w.slot_key[dst] = ((uint64_t)(uint32_t)(head + lane) << 32) | NF; w.slot_q[dst] = xq; w.slot_b[dst] = 1;
                    }
                    __syncwarp();
                    if (lane < R) {
                        const uint64_t k = w.slot_key[lane];
                        fin = (uint32_t)k; sl_s = (int)(k >> 32); sl_q = w.slot_q[lane]; sl_b = w.slot_b[lane];
                    }
                    __syncwarp();
                }
                penalty = 1;
                head += m; off += m; nbatch += m;
                while (off >= 32) {
                    At = Bt; Bt = Ct; Ct = Dt; Aq = Bq; Bq = Cq; Cq = Dq;
                    base += 32;
                    load_win(base + 96, Dt, Dq);
                    off -= 32;
                }
                m1 = __shfl_sync(full, fin, 0);
                pb1 = __shfl_sync(full, sl_b, 0);
                pq1 = __shfl_sync(full, sl_q, 0);
                ps1 = __shfl_sync(full, sl_s, 0);
                continue;
            }
            cooldown = penalty;
            penalty = min(penalty * 2, 64);
        }
        if (cooldown > 0) cooldown--;
    single_step:
        // ---------------- single step ----------------
        const uint32_t m2 = __shfl_sync(full, fin, 1);
        const int pb2 = __shfl_sync(full, sl_b, 1), ps2 = __shfl_sync(full, sl_s, 1);
        const uint32_t pq2 = __shfl_sync(full, sl_q, 1);
        const uint32_t a_head = ah;
        const uint32_t qh = __shfl_sync(full, Aq, off);
        const uint32_t t = max(m1, a_head);
        const unsigned mA = __ballot_sync(full, At <= t);
        const unsigned mB = __ballot_sync(full, Bt <= t);
        int cnt = __popc(__funnelshift_r(mA, mB, off));
        if (WIDE) {
            const unsigned mC = __ballot_sync(full, Ct <= t);
            cnt += __popc(__funnelshift_r(mB, mC, off));
        }
        cnt = min(cnt, mb);
        if (cnt < 1) {
            if (lane == 0) atomicCAS(status, 0, IL_ERR_ITER_LIMIT);
            break;
        }
        const uint32_t nf = t + (uint32_t)row[cnt - 1];      // < 2^29 + 2^24: in range

        if (pb1 > 0) emit(m1, pb1, pq1, ps1);

        uint32_t u = __shfl_down_sync(full, fin, 1);
        const int ub = __shfl_down_sync(full, sl_b, 1), us = __shfl_down_sync(full, sl_s, 1);
        const uint32_t uq = __shfl_down_sync(full, sl_q, 1);
        if (lane == 31) u = kNever32;
        const bool le = u <= nf;                              // equal finish: the older batch first
        const bool here = __ballot_sync(full, le) == w.lt_mask;
        fin = le ? u : (here ? nf : fin);
        sl_b = le ? ub : (here ? cnt : sl_b);
        sl_q = le ? uq : (here ? qh : sl_q);
        sl_s = le ? us : (here ? head : sl_s);
        const bool second_first = m2 <= nf;
        m1 = second_first ? m2 : nf;
        pb1 = second_first ? pb2 : cnt;
        pq1 = second_first ? pq2 : qh;
        ps1 = second_first ? ps2 : head;

        head += cnt;
        off += cnt;
        nbatch++;
        while (off >= 32) {
            At = Bt; Bt = Ct; Ct = Dt; Aq = Bq; Bq = Cq; Cq = Dq;
            base += 32;
            load_win(base + 96, Dt, Dq);
            off -= 32;
        }
    }
    if (bail) {
        // continue in 64-bit arithmetic from here
        StageState st;
        st.resume = true; st.head = head; st.nbatch = nbatch;
        st.key = lane < R ? (((E + fin) << qb) | (uint32_t)sl_s) : kNeverKey;
        if (lane < R && sl_b == 0) st.key = (uint64_t)lane;     // never-used slots keep their tiny keys
        st.sl_b = sl_b; st.sl_q = sl_q;
        return run_stage<WIDE, KIND>(w, row, mb, R, n_in, src, sk, status, st);
    }
#pragma unroll 1
    for (int r = 0; r < R; r++) {
        const uint32_t f = __shfl_sync(full, fin, r);
        const int pb = __shfl_sync(full, sl_b, r), ps = __shfl_sync(full, sl_s, r);
        const uint32_t pq = __shfl_sync(full, sl_q, r);
        if (pb > 0) emit(f, pb, pq, ps);
    }
    src.finish(lane, n_in);
    return nbatch;
}

// A stage whose max batch is 1.  Every batch is a single query with the same
// service time D = latency[1], so the multi-replica FIFO queue behaves like R
// interleaved single-server queues: query i starts at
//     s_i = max(a_i, s_{i-R} + D)
// and queries leave in arrival order.  Unrolled, s_i is a running maximum of
// a_{i-jR} + j D over j, which 32 lanes evaluate for 32 consecutive queries
// with log2(32/R) shuffle steps plus one carry from the previous 32.
template <int KIND, class Src>
__device__ __forceinline__ int run_stage_mb1(const WarpCtx &w, const int32_t *row, const int R,
                                             const int n_in, Src &src, Sink &sk)
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

    uint64_t rec = src.load32(0, lane, n_in);
    for (int base = 0; base < n_in; base += 32) {
        const uint64_t cur = rec;
        rec = src.load32(base + 32, lane, n_in);           // next 32, off the dependent chain
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
    src.finish(lane, n_in);
    return n_in;
}

template <class Src>
__device__ __forceinline__ int dispatch_stage(const WarpCtx &w, const int32_t *row, const int mb,
                                              const int R, const int n_in, Src &src, Sink &sk,
                                              int *status)
{
    const bool branch = sk.bit >= 0;
    if (mb == 1)
        return branch ? run_stage_mb1<kBranch>(w, row, R, n_in, src, sk)
                      : run_stage_mb1<kForward>(w, row, R, n_in, src, sk);
    // the 32-bit loop needs small table entries and a source it may read twice
    uint32_t row_max = 0;
    for (int b = w.lane; b < mb; b += 32) row_max = max(row_max, (uint32_t)row[b]);
    row_max = __reduce_max_sync(0xffffffffu, row_max);
    if (Src::kRereadable && row_max < kNarrowLatLimit) {
        if (mb > 32)
            return branch ? run_stage_narrow<true, kBranch>(w, row, mb, R, n_in, src, sk, status)
                          : run_stage_narrow<true, kForward>(w, row, mb, R, n_in, src, sk, status);
        return branch ? run_stage_narrow<false, kBranch>(w, row, mb, R, n_in, src, sk, status)
                      : run_stage_narrow<false, kForward>(w, row, mb, R, n_in, src, sk, status);
    }
    StageState st;
    st.resume = false;
    if (mb > 32)
        return branch ? run_stage<true, kBranch>(w, row, mb, R, n_in, src, sk, status, st)
                      : run_stage<true, kForward>(w, row, mb, R, n_in, src, sk, status, st);
    return branch ? run_stage<false, kBranch>(w, row, mb, R, n_in, src, sk, status, st)
                  : run_stage<false, kForward>(w, row, mb, R, n_in, src, sk, status, st);
}

// Simulates candidate `c` of the chunk on this warp.  STAGED: the root stage
// reads the trace from the CTA's tile ring (all warps of the CTA must then enter
// together, also those without a candidate of their own: has == false).
template <bool STAGED>
__device__ __forceinline__ void simulate_candidate(const DesParams &p, const WarpCtx &w,
                                                   const int32_t *s_lat, uint64_t *my_rec,
                                                   TileRing *ring, const bool has, const int64_t c,
                                                   unsigned long long &batches,
                                                   unsigned long long &alg_ops)
{
    const unsigned full = 0xffffffffu;
    const int lane = w.lane;
    const int n_tiles = (p.n + kTileRecs - 1) >> kTileLog;
    uint64_t *slab = reinterpret_cast<uint64_t *>(p.slab + (has ? c : 0) * p.slab_stride);
    il_stage_config my_cfg = {0, 1, 1, 0};
    if (has && lane < p.S) my_cfg = p.configs[c * p.S + lane];
    const bool bad = lane < p.S && (my_cfg.hw >= p.H || my_cfg.max_batch < 1 ||
                                    my_cfg.max_batch > p.Bmax || my_cfg.replicas < 1 ||
                                    my_cfg.replicas > IL_MAX_REPLICAS);
    const bool skip = !has || __any_sync(full, bad);
    if (skip) {
        if (has) {
            if (lane == 0) atomicCAS(p.status, 0, IL_ERR_BAD_CONFIG);
            for (int i = lane; i < p.n; i += 32) slab[i] = 0;
        }
        if (STAGED) {   // keep the ring moving for the other warps of the CTA
            TileSrc src = {ring, p.ptrace, n_tiles, 0, -1, false, p.status};
            src.finish(lane, p.n);
        }
        return;
    }

    int exits = 0;
    unsigned long long cand_batches = 0;
    bool over = false;       // the candidate has dispatched more batches than the iteration bound allows
    for (int s = 0; s < p.S; s++) {
        const int n_in = p.n_s[s];
        if (n_in == 0) continue;
        const int hw = __shfl_sync(full, (int)my_cfg.hw, s);
        const int mb = __shfl_sync(full, (int)my_cfg.max_batch, s);
        const int R = __shfl_sync(full, (int)my_cfg.replicas, s);
        const int32_t *row = s_lat + (s * p.H + hw) * p.Bmax;
        const int da = p.dest_a[s], db = p.dest_b[s];
        Sink sk;
        sk.bit = p.bit[s];
        sk.out_a = da < 0 ? slab + exits : my_rec + p.buf_off[da];
        sk.out_b = db < 0 ? slab + exits : my_rec + p.buf_off[db];
        sk.tail_a = 0; sk.tail_b = 0;
        sk.size_a = da < 0 ? (int)p.slab_stride - exits : (int)(p.slot_elems - p.buf_off[da]);
        sk.size_b = db < 0 ? (int)p.slab_stride - exits : (int)(p.slot_elems - p.buf_off[db]);
        sk.status = p.status;
        int nb;
        if (STAGED && s == 0) {
            TileSrc src = {ring, p.ptrace, n_tiles, 0, -1, false, p.status};
            nb = dispatch_stage(w, row, mb, R, n_in, src, sk, p.status);
        } else {
            GlobalSrc src = {s == 0 ? p.ptrace : my_rec + p.buf_off[s], s == 0};
            nb = dispatch_stage(w, row, mb, R, n_in, src, sk, p.status);
        }
        // a guarded stage has at most one side that leaves the pipeline
        if (sk.bit < 0) { if (da < 0) exits += sk.tail_a; }
        else exits += (da < 0 ? sk.tail_a : 0) + (db < 0 ? sk.tail_b : 0);
        batches += (unsigned)nb;
        alg_ops += 3ull * (unsigned)n_in + (unsigned long long)nb * (unsigned)(R + mb + 4);
        __syncwarp();   // this stage's stream writes are read by the next stage's other lanes
        // Every stage loop ends by itself (a batch takes at least one query); the bound is checked
        // between stages, where giving the candidate up leaves nothing half-written behind.
        cand_batches += (unsigned)nb;
        if (p.iter_limit && cand_batches > p.iter_limit) {
            if (lane == 0) atomicCAS(p.status, 0, IL_ERR_ITER_LIMIT);
            over = true;
            break;
        }
    }
    // (the root stage, the only one that reads the staged trace, has been run to its end either way)
    if (lane == 0 && !over && exits != p.n) { atomicCAS(p.status, 0, IL_ERR_ITER_LIMIT); atomicOr(&p.counters[5], 8ull); }
}

}  // namespace

template <bool STAGED>
__global__ void __launch_bounds__(kWarpsPerCta * 32)
des_packed_kernel(const __grid_constant__ DesParams p)
{
    extern __shared__ int32_t s_lat[];
    __shared__ uint64_t s_slot_key[kWarpsPerCta][32];
    __shared__ uint32_t s_slot_q[kWarpsPerCta][32];
    __shared__ int s_slot_b[kWarpsPerCta][32];
    __shared__ __align__(128) unsigned char s_ring_mem[STAGED ? sizeof(TileRing) : 16];
    TileRing *ring = reinterpret_cast<TileRing *>(s_ring_mem);
    const int n_tab = p.S * p.H * p.Bmax;
    for (int i = threadIdx.x; i < n_tab; i += blockDim.x) s_lat[i] = p.lat[i];
    if (STAGED && threadIdx.x == 0) {
        for (int k = 0; k < kTiles; k++) { mbar_init(&ring->full[k], 1); ring->uses[k] = 0; ring->released[k] = 0; }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const unsigned full = 0xffffffffu;
    const int wid = threadIdx.x >> 5;
    WarpCtx w;
    w.lane = threadIdx.x & 31;
    w.lt_mask = (1u << w.lane) - 1u;
    w.qbits = p.qbits;
    w.qmask = (1u << p.qbits) - 1u;
    w.bits = p.bits;
    w.n_queries = p.n;
    w.slot_key = s_slot_key[wid];
    w.slot_q = s_slot_q[wid];
    w.slot_b = s_slot_b[wid];
    const int lane = w.lane;
    const int64_t slot = (int64_t)blockIdx.x * kWarpsPerCta + wid;
    uint64_t *my_rec = reinterpret_cast<uint64_t *>(p.ws_time) + slot * p.slot_elems;
    unsigned long long batches = 0, alg_ops = 0;

    if (!STAGED) {
        // every warp on its own: take the next candidate in the order array (whose length may have
        // been written by an earlier kernel of the stream)
        const unsigned long long n_list = p.n_cand_dev ? *p.n_cand_dev : (unsigned long long)p.n_cand;
        for (;;) {
            unsigned long long c = 0;
            if (lane == 0) c = atomicAdd(&p.counters[0], 1ull);
            c = __shfl_sync(full, c, 0);
            if (c >= n_list) break;
            simulate_candidate<false>(p, w, s_lat, my_rec, nullptr, true, (int64_t)p.order[c], batches, alg_ops);
        }
    } else {
        // the CTA takes kWarpsPerCta consecutive positions of the order array at
        // a time (neighbours in that order cost about the same) and its warps go
        // through the staged trace together
        const int n_tiles = (p.n + kTileRecs - 1) >> kTileLog;
        for (;;) {
            __syncthreads();      // everybody is done with the previous group's tiles
            if (threadIdx.x == 0) {
                const unsigned long long g = atomicAdd(&p.counters[0], (unsigned long long)kWarpsPerCta);
                ring->group_base = g < (unsigned long long)p.n_cand ? (int)g : -1;
                for (int k = 0; k < kTiles; k++) { ring->released[k] = 0; ring->base_uses[k] = ring->uses[k]; }
                if (ring->group_base >= 0)
                    for (int t = 0; t < kTiles && t < n_tiles; t++) tile_issue(ring, p.ptrace, t);
            }
            __syncthreads();
            const int g = ring->group_base;
            if (g < 0) break;
            const int64_t pos = (int64_t)g + wid;
            const bool has = pos < p.n_cand;
            simulate_candidate<true>(p, w, s_lat, my_rec, ring, has, has ? (int64_t)p.order[pos] : 0, batches, alg_ops);
        }
        // no copy may still be in flight into this CTA's shared memory when it exits
        __syncthreads();
        if (threadIdx.x == 0)
            for (int k = 0; k < kTiles; k++)
                if (ring->uses[k] > 0) mbar_wait_bounded(&ring->full[k], (unsigned)(ring->uses[k] - 1) & 1u);
        __syncthreads();
    }
    if (lane == 0 && batches) { atomicAdd(&p.counters[1], batches); atomicAdd(&p.counters[2], alg_ops); }
}

// One stage of the shared-prefix evaluation (prefix_kernel.cu): every warp takes nodes of stage
// p.s from the work counter and runs the stage's queue simulation once per node, from the
// completion stream of the node's parent (or the trace) to the node's own output streams.
__global__ void __launch_bounds__(kWarpsPerCta * 32)
des_node_stage_kernel(const __grid_constant__ NodeStageParams p)
{
    extern __shared__ int32_t s_row[];     // the stage's profile, [H][Bmax]
    __shared__ uint64_t s_slot_key[kWarpsPerCta][32];
    __shared__ uint32_t s_slot_q[kWarpsPerCta][32];
    __shared__ int s_slot_b[kWarpsPerCta][32];
    for (int i = threadIdx.x; i < p.H * p.Bmax; i += blockDim.x) s_row[i] = p.lat_stage[i];
    __syncthreads();

    const unsigned full = 0xffffffffu;
    const int wid = threadIdx.x >> 5;
    WarpCtx w;
    w.lane = threadIdx.x & 31;
    w.lt_mask = (1u << w.lane) - 1u;
    w.qbits = p.qbits;
    w.qmask = (1u << p.qbits) - 1u;
    w.bits = p.bits;
    w.n_queries = p.n_queries;
    w.slot_key = s_slot_key[wid];
    w.slot_q = s_slot_q[wid];
    w.slot_b = s_slot_b[wid];
    unsigned long long batches = 0, alg_ops = 0;
    for (;;) {
        unsigned long long k = 0;
        if (w.lane == 0) k = atomicAdd(p.work, 1ull);
        k = __shfl_sync(full, k, 0);
        if (k >= (unsigned long long)p.n_nodes) break;
        const uint32_t cfg = p.node_cfg[k];
        const int hw = (int)(cfg & 0xffu), mb = (int)((cfg >> 8) & 0xffu), R = (int)((cfg >> 16) & 0xffu);
        Sink sk;
        sk.bit = p.bit;
        sk.out_a = p.out_a + (int64_t)k * p.stride_a;
        sk.out_b = p.out_b + (int64_t)k * p.stride_b;
        sk.tail_a = 0; sk.tail_b = 0;
        sk.size_a = (int)p.stride_a; sk.size_b = (int)p.stride_b;
        sk.status = p.status;
        GlobalSrc src = {p.in ? p.in + (int64_t)p.node_parent[k] * p.stride_in : p.ptrace, p.in == nullptr};
        const int nb = dispatch_stage(w, s_row + hw * p.Bmax, mb, R, p.n_in, src, sk, p.status);
        batches += (unsigned)nb;
        alg_ops += 3ull * (unsigned)p.n_in + (unsigned long long)nb * (unsigned)(R + mb + 4);
        // every record of the stage must have gone to one of the two sides
        if (w.lane == 0 && sk.tail_a + sk.tail_b != p.n_in) {
            atomicCAS(p.status, 0, IL_ERR_ITER_LIMIT);
            atomicOr(&p.counters[5], 8ull);
        }
        __syncwarp();
    }
    if (w.lane == 0 && batches) { atomicAdd(&p.counters[1], batches); atomicAdd(&p.counters[2], alg_ops); }
}

cudaError_t launch_node_stage(const NodeStageParams &p, int grid, cudaStream_t stream)
{
    const size_t smem = (size_t)p.H * p.Bmax * sizeof(int32_t);
    des_node_stage_kernel<<<grid, kWarpsPerCta * 32, smem, stream>>>(p);
    return cudaGetLastError();
}

namespace {
// Static plus dynamic shared memory passes 48 KB for the largest table shapes the interface takes
// (16 stages x 8 hardware types x 64 batch sizes = 32 KB of tables): opt in before every use.
cudaError_t packed_opt_in(bool staged, size_t smem)
{
    return staged
        ? cudaFuncSetAttribute(des_packed_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)
        : cudaFuncSetAttribute(des_packed_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
}
}  // namespace

cudaError_t launch_des_packed(const DesParams &p, bool staged, int grid, size_t smem, cudaStream_t stream)
{
    cudaError_t e = packed_opt_in(staged, smem);
    if (e != cudaSuccess) return e;
    if (staged) des_packed_kernel<true><<<grid, kWarpsPerCta * 32, smem, stream>>>(p);
    else des_packed_kernel<false><<<grid, kWarpsPerCta * 32, smem, stream>>>(p);
    return cudaGetLastError();
}

int des_packed_max_ctas_per_sm(bool staged, size_t smem)
{
    int n = 0;
    if (packed_opt_in(staged, smem) != cudaSuccess) return 0;
    cudaError_t e = staged
        ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, des_packed_kernel<true>, kWarpsPerCta * 32, smem)
        : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, des_packed_kernel<false>, kWarpsPerCta * 32, smem);
    return e == cudaSuccess ? n : 0;
}

int trace_tile_records() { return kTileRecs; }

}  // namespace il
