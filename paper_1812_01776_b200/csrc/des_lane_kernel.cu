// Batched discrete-event simulation of the InferLine Estimator (Section 4.2),
// lane-parallel version: one LANE per (candidate, stage), the stages of a
// candidate running side by side as a pipeline inside one warp.
//
// The pipeline is a feed-forward tree with zero delay between stages, so a
// stage is a function from its arrival stream (times never decrease) to its
// completion stream, and the batch recurrence of the centralized batched queue
// (Section 3) is, per stage,
//
//     t      = max(earliest time a replica is free, arrival[head])
//     b      = min(max batch, number of arrivals from head on with time <= t)
//     finish = t + latency[stage][hw][b-1]            (Section 4.1 profile)
//
// with batches leaving in (finish, dispatch order) order.  The warp-per-candidate
// kernels (des_kernel.cu, des_packed_kernel.cu) run this chain one stage after
// the other and spend a warp instruction per step of ONE chain.  Here a warp
// holds floor(32 / S) candidates; lane (j, s) runs the scalar chain of stage s
// of candidate j, and all 32 chains advance together, one record per loop
// iteration and lane:
//
//   * examine: the lane looks at ONE record of its arrival stream.  Either the
//     record joins the open batch (arrived by the batch's dispatch time and the
//     batch is not full), or the open batch is closed (finish time from the
//     table, sorted insert into the lane's list of replica slots) and the record
//     opens the next batch, which takes over the slot with the smallest key;
//   * emit: the batch that held that slot leaves the stage, ONE record per
//     iteration, to the child stage selected by the query's branch bit or, at a
//     leaf, to the candidate's slab as a (finish, query) record.
//
// Stage s+1 reads what stage s wrote a few iterations earlier.  A lane knows
// how far its parent has got from one word in shared memory that the parent
// publishes every iteration: the number of records written so far, and a flag
// once it has written all of them.  A batch that is not full is closed when the
// next record turns out not to belong to it (or the stream has ended), so a
// stage simply trails its parent by a few records; parents never wait for
// children, so the root always advances and every wait ends.
//
// Everything a lane reads from a stream in global memory (the record it
// examines, the record it hands on) is copied into a small per-lane staging ring
// in shared memory by an asynchronous copy (cp.async) issued three iterations
// before its use; one commit group per iteration, at most two groups pending, so
// that no instruction of the loop waits for global memory.
//
// With few candidates a warp has a scheduler to itself and is paced by its own
// dependency chain, so the loop body is ordered for that: whatever the end of
// an iteration needs from shared or global memory is loaded at its top,
// unconditionally, and the close / open steps are straight-line code under
// predicates, so that independent work can issue while a dependent value is on
// its way.  Each lane keeps its own copy of its stage's profile row in shared
// memory, [batch][lane], so that table look-ups never conflict.
//
// Stream memory.  A stage's arrival stream lives in a RING of K records (K a
// power of two chosen by the host), not in a buffer of its full length, so the
// scratch a resident candidate needs does not grow with the trace.  A lane still
// needs every record from the first one of its oldest batch in flight (whose
// records it re-reads when the batch leaves) up to the one it examines, so the
// parent may run at most K records ahead of that point: each lane publishes,
// now and then, the index below which it needs nothing any more, and a parent
// that would overrun a child's ring holds its hand-on step until the child has
// moved on (simulated times do not depend on the order in which lanes take their
// steps).  Leaves write to the slab and never wait, so every wait ends -- except
// when one batch stays in flight while more than K later records pass through
// the other replicas of its stage: then parent and child wait for each other.
// The child detects that (ring full, nothing left to examine or hand on, no
// progress), marks the candidate in the overflow array and ends the candidate's
// lanes; the host evaluates marked candidates with the warp-per-candidate
// kernel, which has no such limit.  With K >= the longest stream (RING = false)
// none of this code is compiled in.
//
// Scheduling.  The floor(32 / S) groups of a warp are independent of each other:
// when all lanes of a group have finished their candidate, the group takes the
// next candidate from a global work counter (looked at every eighth iteration)
// while the other groups carry on, so a warp never idles behind its slowest
// candidate.  In the feasibility-only instantiation (Section 4.3, "Feasible")
// the leaves compare each leaving query with the objective instead of writing
// it to the slab, and a group drops its candidate as soon as more queries have
// missed the objective than the P99 rule allows.
//
// Records and keys are the packed 64-bit words of des_packed_kernel.cu:
// (time << q) | query for stream records, (finish << q) | index of the batch's
// first arrival for replica slots, whose unsigned order is (finish, dispatch
// order).  The host selects this kernel only when every reachable time fits.
#include "il_internal.h"

namespace il {

namespace {

constexpr int kLaneWarps = 2;                  // warps per CTA
constexpr uint32_t kDone = 0x80000000u;
constexpr uint64_t kInf = ~0ull;
constexpr uint32_t kAbort = 0xffffffffu;      // ring mailbox: the candidate is given up (ring overflow)
constexpr uint32_t kRingSlack = 4;            // records a parent may have under way when it checks for room
constexpr int kLag = 40;        // records a stage stays behind its parent while the parent is running
constexpr int kStage = 4;       // staging ring positions (pending groups + 2)
constexpr int kPending = 2;     // commit groups that may still be in flight at the end of an iteration

__device__ __forceinline__ void cp_async8(void *smem_dst, const void *gsrc)
{
    const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(d), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Shared memory of one warp, laid out for the launch: the batch ring has `kr` positions (a power of
// two of at least the largest replica count of the launch's candidates; 16 or 32) and the profile copy
// Bmax rows, so a launch pays only for what its candidates need.
struct WarpMem {
    // Per lane a ring of batches, [pos][lane].  Positions [epos, lpos): batches whose slot has been
    // taken over, waiting to be handed on, in key order.  Positions [lpos, tpos): the slots in use,
    // sorted by key.
    uint64_t (*key)[32];         // [kr] (finish << q) | index of the batch's first arrival
    uint8_t (*cnt)[32];          // [kr] batch size (at most IL_MAX_BATCH = 64)
    // The lane's row of the profile, [b - 1][lane]: time of a batch of b on the stage's hardware type.
    // One copy per lane, so that lanes with different rows or batch sizes never meet in a bank.
    uint32_t (*lat)[32];         // [Bmax]
    // Staging rings filled by cp.async, [position][lane]: the next records of the lane's arrival stream
    // (position = record index mod kStage), and the records it is handing on (position = iteration
    // mod kStage; the finish << q of their batch waits in a three-deep delay line of registers)
    uint64_t (*stage_x)[32];     // [kStage]
    uint64_t (*stage_e)[32];
    // Mailboxes, double-buffered by iteration parity: what iteration k publishes in buffer k & 1 is read
    // in iteration k + 1, while iteration k + 1 publishes into the other buffer; one warp barrier per
    // iteration then separates every write of a word from the reads of its previous value.
    uint32_t (*avail)[32];       // [2] records written so far into the lane's arrival stream (by its parent
                                 // lane); kDone set once that is all of them
    // Ring streams only: index below which the lane needs no record of its arrival stream any more
    // (its parent may overwrite those ring positions), or kAbort.  Grows monotonically; a reader that
    // sees an older value only waits longer.
    uint32_t *freed;             // [32]
    // Feasibility only: queries of the group's candidate that have missed the objective so far, [group]
    uint32_t *miss;              // [32]
};

__host__ __device__ inline size_t warp_mem_bytes(int kr, int Bmax)
{
    return (size_t)kr * 32 * 9 + (size_t)2 * kStage * 32 * 8 + (size_t)(2 + 1 + 1) * 32 * 4 + (size_t)Bmax * 32 * 4;
}

__device__ __forceinline__ WarpMem warp_mem_at(unsigned char *base, int kr, int Bmax)
{
    WarpMem wm;
    wm.key = reinterpret_cast<uint64_t (*)[32]>(base);          base += (size_t)kr * 256;
    wm.stage_x = reinterpret_cast<uint64_t (*)[32]>(base);      base += (size_t)kStage * 256;
    wm.stage_e = reinterpret_cast<uint64_t (*)[32]>(base);      base += (size_t)kStage * 256;
    wm.cnt = reinterpret_cast<uint8_t (*)[32]>(base);           base += (size_t)kr * 32;
    wm.lat = reinterpret_cast<uint32_t (*)[32]>(base);          base += (size_t)Bmax * 128;
    wm.avail = reinterpret_cast<uint32_t (*)[32]>(base);        base += 256;
    wm.freed = reinterpret_cast<uint32_t *>(base);              base += 128;
    wm.miss = reinterpret_cast<uint32_t *>(base);
    return wm;
}

}  // namespace

// BRANCHY: some stage routes by a branch bit (otherwise every stage has one way out).
// RING: the stream rings are shorter than the longest stream, so positions wrap and parents wait for room.
// FEAS: feasibility only (Section 4.3, "Feasible"): leaving queries are compared with the objective as
//       they leave, nothing is written to a slab, and a candidate is dropped as soon as more queries
//       have missed the objective than the P99 rule allows.
// FORK: fan-out -- a query goes down every edge whose condition holds, a copy that finds none leaves, and
//       the slab keeps per query the record of the copy that left last (only with BRANCHY, without RING
//       and FEAS).
template <bool BRANCHY, bool RING, bool FEAS, bool FORK = false>
__global__ void __launch_bounds__(kLaneWarps * 32)
des_lane_kernel(const __grid_constant__ DesParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    // (the profile tables stay in global memory: a lane copies its row from there once per candidate, and
    // shared memory not spent on them is L1 for the stream records)
    unsigned char *wm_base = smem_raw;
    // A stream record is (time << q) | low part; the low part is the query index, below the query's
    // branch bits when the records carry them (rb > 0: no stage then looks the bits up).  Keys of batches
    // use the same q, with the index of the batch's first arrival in the low part.
    const int qi = p.qbits, rb = BRANCHY ? p.rec_bits : 0;
    const int q = qi + rb;
    const uint64_t qmask = (1ull << q) - 1ull;
    const uint32_t imask = (uint32_t)((1ull << qi) - 1ull);
    const uint64_t *trace = rb > 0 ? p.ptrace_b : p.ptrace;

    const unsigned full = 0xffffffffu;
    const int wid = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t kr = p.lane_slots == 16 ? 16u : 32u, rmask = kr - 1u;      // batch ring positions of a lane
    const WarpMem wm = warp_mem_at(wm_base + (size_t)wid * warp_mem_bytes((int)kr, p.Bmax), (int)kr, p.Bmax);
    const int S = p.S, cpw = p.cpw;
    const int j = lane / S, s = lane - j * S;
    const bool lane_used = j < cpw;

    // static facts of this lane's stage
    int exit_off = 0;
    for (int u = 0; u < s; u++) {
        const int a = p.dest_a[u], b2 = p.dest_b[u];
        int kids = 0;
        if (a >= 0) kids += p.n_s[a];
        if (b2 >= 0 && b2 != a) kids += p.n_s[b2];
        exit_off += p.n_s[u] - kids;
    }
    const int da = FORK ? p.child_a[s] : p.dest_a[s], db = FORK ? p.child_b[s] : p.dest_b[s];
    // fan-out: the guard of either edge; the branch bits are needed if one of them is conditional
    const int cbit_a = p.cbit_a[s], cbit_b = p.cbit_b[s];
    const unsigned cval_a = p.cval_a[s], cval_b = p.cval_b[s];
    const int bit = FORK ? ((cbit_a >= 0 || cbit_b >= 0) ? 0 : -1) : p.bit[s];
    const uint32_t n_in = lane_used ? (uint32_t)p.n_s[s] : 0u;
    const unsigned group_mask = lane_used ? (((1u << S) - 1u) << (j * S)) : 0u;
    const int root_lane = lane_used ? j * S : 0;
    // mailbox of the child on either side; a lane without that child writes a word nobody reads
    // (its own entry of a spare row would do as well: lanes j * S + child are always in range)
    const int lane_a = (da < 0 || !lane_used) ? -1 : j * S + da;
    const int lane_b = (db < 0 || db == da || !lane_used) ? -1 : j * S + db;

    const int64_t wslot = (int64_t)blockIdx.x * kLaneWarps + wid;
    uint64_t *my_block = p.lane_ws + (wslot * cpw + (lane_used ? j : 0)) * p.lane_elems;
    const uint64_t *in = s == 0 ? trace : my_block + p.lane_off[s];
    // ring positions: index & mask (the trace and the slab are not rings)
    const uint32_t K = 1u << p.lane_ring_log2;
    const uint32_t in_mask = (RING && s != 0) ? K - 1u : 0xffffffffu;
    const uint32_t mask_a = (RING && da >= 0) ? K - 1u : 0xffffffffu;
    const uint32_t mask_b = (RING && db >= 0) ? K - 1u : 0xffffffffu;
    const unsigned long long iter_limit = p.iter_limit;
    const unsigned long long n_cand = (unsigned long long)p.n_cand;
    // sizes of what this lane reads and writes, for the checked build: its arrival stream (or the trace),
    // and per side the child's stream or the rest of the slab row
    const unsigned long long in_size = s == 0 ? (unsigned long long)p.n : (unsigned long long)(p.lane_elems - p.lane_off[s]);
    const unsigned long long size_a = da < 0 ? (unsigned long long)(p.slab_stride - exit_off)
                                             : (unsigned long long)(p.lane_elems - p.lane_off[da]);
    const unsigned long long size_b = db < 0 ? (unsigned long long)(p.slab_stride - exit_off)
                                             : (unsigned long long)(p.lane_elems - p.lane_off[db]);
    (void)in_size; (void)size_a; (void)size_b;
    const uint64_t slo_q = FEAS ? (uint64_t)p.slo_us << q : 0ull;   // the objective, aligned with a record's time field
    unsigned long long batches = 0, alg_ops = 0, exits_seen = 0, exits_due = 0;
    unsigned early = 0;          // candidates dropped before the end of the trace (feasibility only)

    // The groups of a warp (one candidate each) are independent: a group whose lanes have all finished
    // takes the next candidate from the work counter while the other groups carry on.  State of the
    // lane's candidate:
    int64_t c = 0;
    bool has = false;            // the group holds a candidate
    bool exhausted = !lane_used; // the group will get no further candidate
    bool live = false, done = true, cand_bad = false;
    uint32_t R = 1;
    int mb = 1;
    uint64_t *out_a = nullptr, *out_b = nullptr;
    unsigned long long *slab_row = nullptr;   // fan-out: the candidate's slab row, indexed by query
    uint32_t n_left = 0;                      // fan-out: copies that left the pipeline at this lane
    uint32_t epos = 0, lpos = 0, tpos = 0;   // ring positions, see WarpMem
    uint64_t kfront = kInf;      // key at lpos (kInf when no slot is in use)
    uint64_t ktail = 0;          // largest key in [lpos, tpos)
    uint32_t head = 0;           // index of the open batch's first record
    int b = 0;                   // size of the open batch (0: none)
    uint64_t tk = 0;             // open batch's dispatch time as (t << q) | qmask
    uint64_t e_base = 0;         // finish << q of the batch being handed on
    uint32_t e_idx = 0;          // its next record in the arrival stream
    uint32_t e_left = 0;         // records of it not yet fetched
    uint32_t vmask = 0;          // bit k: the record fetched k + 1 iterations ago is on its way out
    uint64_t eb1 = 0, eb2 = 0, eb3 = 0;   // finish << q of the batches of those records, a delay line in registers
    // fetch cursor of the arrival stream: records below fx have been requested; fx1..fx3 are its
    // values at the end of the previous three iterations, so records below fx3 have arrived
    uint32_t fx = 0, fx1 = 0, fx2 = 0, fx3 = 0;
    uint32_t tail_a = 0, tail_b = 0;
    unsigned nb = 0;
    uint32_t guard = 0, guard_hi = 0;        // iteration bound, counted down in 32-bit pieces
    // ring streams: how far the lane's children let it write, what it has told its own parent,
    // and a new value for that, found at one eighth iteration and published at the next
    uint32_t lim_a = 0xffffffffu, lim_b = 0xffffffffu;
    uint32_t low_pub = 0, low_new = 0, e_first = 0;
    bool low_pending = false, aborted = false;
    // feasibility only: a leaving record waits one iteration for the arrival time of its query
    uint64_t late_fin = 0, late_arr = 0;     // late_fin == 0: no record is waiting (finish times are at least 1)
    uint32_t miss_local = 0;     // misses seen by this lane since it last added them to the group's count
    uint32_t av = 0;             // mailbox word this iteration works with: the one read an iteration ago
    int par = 0;                 // mailbox buffer this iteration publishes into; it reads the other one
    uint32_t it = 0;

    for (;;) {
        // ---- every eighth iteration: drop decided candidates, hand finished groups their next candidate
        if ((it & 7u) == 0u) {
            if (RING && !done) {
                // parent side: how far the children have moved on, and whether one has given up
                if (lane_a >= 0) { const uint32_t f = wm.freed[lane_a]; aborted |= f == kAbort; lim_a = f + K; }
                if (lane_b >= 0) { const uint32_t f = wm.freed[lane_b]; aborted |= f == kAbort; lim_b = f + K; }
                if (s != 0) {
                    // Child side: tell the parent how far it may overwrite the ring.  The lane needs every
                    // record from the first one of any batch it still has to hand on, and from the open
                    // batch on.  The minimum is taken when half the ring is in use and published eight
                    // iterations later: copies under way at the time it was taken (records of batches
                    // already picked up for handing on) have landed by then, and every later copy reads a
                    // batch that was counted.
                    const uint32_t written = av & ~kDone;
                    if (low_pending) {
                        low_pending = false;
                        if (low_new > low_pub) {
                            low_pub = low_new;
                            wm.freed[lane] = low_pub;
                        } else if ((av & kDone) == 0u && written - low_pub + kRingSlack >= K &&
                                   fx + (uint32_t)kLag >= written && head + (uint32_t)b >= fx && epos == lpos &&
                                   e_left == 0 && vmask == 0u) {
                            // the ring is full, this lane has nothing left to examine or hand on, and what
                            // pins the ring is a batch still in flight: parent and child would wait for
                            // each other for ever.  Give the candidate up.
                            aborted = true;
                        }
                    }
                    if (written - low_pub >= (K >> 1)) {
                        uint32_t lo = head;
                        if (e_left > 0) lo = min(lo, e_first);
                        for (uint32_t pp = epos; pp != tpos; pp++)
                            lo = min(lo, (uint32_t)wm.key[pp & rmask][lane] & (uint32_t)qmask);
                        low_new = lo;
                        low_pending = true;
                    }
                }
                if (aborted) {
                    p.ovf[c] = 1;
                    wm.freed[lane] = kAbort;
                    done = true;
                }
            }
            if (FEAS) {
                if (miss_local) { atomicAdd(&wm.miss[j], miss_local); miss_local = 0; }
                __syncwarp();
                if (has && !done && wm.miss[j] > p.miss_allow) done = true;   // same word, same moment: the whole group
            }
            // Feasibility only: a group moves on as soon as its own lanes have finished (candidates are
            // dropped at very different points of the trace).  Otherwise the groups of a warp start their
            // candidates together: they then walk the trace side by side and share its cache lines.
            const unsigned dm = __ballot_sync(full, done);
            const bool turn = !exhausted && (FEAS ? (dm & group_mask) == group_mask : dm == full);
            if (__any_sync(full, turn)) {
                // a candidate that was dropped (decided, given up, out of iterations) may still have
                // copies under way into the lane's staging rings: let them land before the rings are reused
                cp_async_wait<0>();
                // wrap up the candidate the group has finished
                const bool cand_aborted = RING && (__ballot_sync(full, aborted && turn) & group_mask) != 0u;
                if (turn && has) {
                    if (live && !cand_aborted) {
                        batches += nb;
                        alg_ops += 3ull * n_in + (unsigned long long)nb * (unsigned)(R + mb + 4);
                    }
                    const bool decided = FEAS && wm.miss[j] > p.miss_allow;
                    // every query of a candidate that ran to its end must have left through exactly one
                    // leaf (checked over all candidates of the warp when the kernel ends)
                    if (live && !cand_aborted && !decided)
                        exits_seen += FORK ? n_left : (da < 0 ? tail_a : 0u) + ((db < 0 && bit >= 0) ? tail_b : 0u);
                    if (s == 0 && !cand_bad && !cand_aborted && !decided)
                        exits_due += FORK ? (unsigned long long)p.total_leaving : (unsigned long long)(unsigned)p.n;
                    if (FEAS && s == 0) {
                        p.out_feasible[c] = cand_aborted ? 2 : (decided || cand_bad ? 0 : 1);
                        early += (decided && head < n_in) ? 1u : 0u;     // the root had not reached the end of the trace
                    }
                }
                // the group's next candidate
                unsigned long long g = 0;
                if (turn && s == 0) g = atomicAdd(&p.counters[0], 1ull);
                g = __shfl_sync(full, g, root_lane);
                il_stage_config cfg = {0, 1, 1, 0};
                const bool got = turn && g < n_cand;
                if (got) cfg = p.configs[g * S + s];
                const bool bad = got && (cfg.hw >= p.H || cfg.max_batch < 1 || cfg.max_batch > p.Bmax ||
                                         cfg.replicas < 1 || cfg.replicas > IL_MAX_REPLICAS);
                const bool grp_bad = (__ballot_sync(full, bad) & group_mask) != 0u;
                if (turn) {
                    has = got;
                    exhausted = !got;
                    c = (int64_t)g;      // g < n_cand whenever the group got a candidate: rows of the slab, the
                    cand_bad = grp_bad;  // overflow array and the output exist for it
                    uint64_t *slab = FEAS ? nullptr : reinterpret_cast<uint64_t *>(p.slab + (got ? c : 0) * p.slab_stride);
                    if (got && cand_bad) {
                        if (s == 0) atomicCAS(p.status, 0, IL_ERR_BAD_CONFIG);
                        if (!FEAS) for (int i = s; i < p.n; i += S) slab[i] = 0;
                    }
                    live = got && !cand_bad && n_in > 0;
                    R = cfg.replicas;
                    mb = cfg.max_batch;
                    if (live) {
                        const int32_t *row = p.lat + (s * p.H + cfg.hw) * p.Bmax;
                        for (int k = 0; k < p.Bmax; k++) wm.lat[k][lane] = (uint32_t)row[k];
                    }
                    out_a = da < 0 ? slab + exit_off : my_block + p.lane_off[da];
                    out_b = db < 0 ? slab + exit_off : my_block + p.lane_off[db];
                    slab_row = reinterpret_cast<unsigned long long *>(slab);
                    n_left = 0;
                    // the root's stream is complete from the start; a stage nobody visits is finished at once
                    const uint32_t avail0 = (s == 0 || !live) ? (n_in | kDone) : 0u;
                    wm.avail[0][lane] = avail0; wm.avail[1][lane] = avail0;
                    if (RING) wm.freed[lane] = 0u;
                    if (FEAS && s == 0) wm.miss[j] = 0u;
                    epos = 0; lpos = 0; tpos = 0;
                    kfront = kInf; ktail = 0;
                    head = 0; b = 0; tk = 0;
                    e_base = 0; e_idx = 0; e_left = 0; vmask = 0;
                    fx = 0; fx1 = 0; fx2 = 0; fx3 = 0;
                    tail_a = 0; tail_b = 0; nb = 0;
                    done = !live;
                    const unsigned long long limit =
                        iter_limit ? iter_limit : 8ull * (unsigned)p.n * (unsigned)(S + 1) + 4096ull;
                    guard = (uint32_t)(limit & 0xffffffffull) + 1u;
                    guard_hi = (uint32_t)(limit >> 32);
                    if (guard == 0u) guard = 0xffffffffu;
                    lim_a = (RING && lane_a >= 0) ? K : 0xffffffffu;
                    lim_b = (RING && lane_b >= 0) ? K : 0xffffffffu;
                    low_pub = 0; low_new = 0; e_first = 0;
                    low_pending = false; aborted = false;
                    late_fin = 0;
                    miss_local = 0;
                    av = avail0;
                }
                __syncwarp();     // the mailboxes are set before anybody reads them
                if (__all_sync(full, exhausted)) break;
            }
        }
        const uint32_t av_next = wm.avail[par ^ 1][lane];
        if (!done) {
            // the record to hand on in this iteration (requested three iterations ago); its branch bits
            // are fetched here, so that the load runs under the examine step
            const bool h_valid = (vmask & 4u) != 0u;
            const uint32_t h_sl = (it + 1u) & (kStage - 1);
            const uint64_t h_low = wm.stage_e[h_sl][lane] & qmask;       // unused unless h_valid
            const uint32_t h_qid = (uint32_t)h_low & imask;
            const uint64_t h_base = eb3;     // finish << q of the batch of the record requested three iterations ago
            uint32_t h_bits = 0;
            if (BRANCHY && rb > 0) h_bits = (uint32_t)(h_low >> qi);
            else if (BRANCHY && h_valid && bit >= 0 && IL_IN_RANGE(h_qid, p.n, p.status)) h_bits = p.bits[h_qid];
            // feasibility only: the record that left in the previous iteration is tested now, its query's
            // arrival record having had an iteration to come in; the arrival record of a query that may
            // leave in this iteration is requested here
            // (finish << q has no low bits, so finish > arrival + objective holds for the time fields iff it
            // holds with the arrival record's low bits left in; counted in a register, the group's shared
            // count is brought up to date every eighth iteration)
            if (FEAS) miss_local += (late_fin > late_arr + slo_q) ? 1u : 0u;
            // (every lane loads, lanes that hand nothing to the outside the trace's first record: no branch;
            // straight into the register that is carried to the next iteration, so nothing here waits for it)
            if (FEAS) {
                const bool may_leave = h_valid && (da < 0 || (db < 0 && bit >= 0)) && IL_IN_RANGE(h_qid, p.n, p.status);
                late_arr = __ldg(trace + (may_leave ? h_qid : 0u));
            }
            // likewise the next batch to hand on, if the one in hand is used up (a batch handed over in
            // this iteration is picked up in the next), and the table entry a close would need
            const bool f_valid = e_left == 0 && epos != lpos;
            const uint64_t f_key = wm.key[epos & rmask][lane];                      // unused unless f_valid
            const uint32_t f_cnt = wm.cnt[epos & rmask][lane];
            // (latency << q) - qmask: finish key base = dispatch key + that
            const uint64_t latq = ((uint64_t)wm.lat[b > 0 ? b - 1 : 0][lane] << q) - qmask;
            // key of the second slot in use, the front after a hand-over (unused unless there are two)
            uint64_t k2 = wm.key[(lpos + 1u) & rmask][lane];
            const uint32_t written = av & ~kDone;
            const bool pdone = (av & kDone) != 0u;
            // ring streams: may this lane start handing on another record?  Not while a child's ring
            // could be overrun by the records under way (the limits are refreshed every eighth iteration)
            const bool can_emit = !RING || (tail_a + kRingSlack <= lim_a && tail_b + kRingSlack <= lim_b);

            // ---- examine one record of the arrival stream
            const uint32_t i = head + (uint32_t)b;
            const bool known = i < fx3;
            const uint64_t ra = wm.stage_x[i & (kStage - 1)][lane];
            const bool end = pdone && i >= written;
            const bool join = known && b > 0 && b < mb && ra <= tk;
            b += join ? 1 : 0;
            const bool room = tpos - epos < kr;
            const bool close = b > 0 && !join && (known || end || b == mb) && room;
            // close and open as straight-line code under predicates (only the sorted insert branches),
            // so that the hand-on and request steps below can overlap with it
            const uint64_t key = (tk + latq) | head;
            uint32_t pos = tpos;
            const bool sorted_insert = close && tpos != lpos && key < ktail;
            if (sorted_insert) {
                // a batch that finishes before one dispatched earlier
#pragma unroll 1
                while (pos != lpos) {
                    const uint64_t prev = wm.key[(pos - 1) & rmask][lane];
                    if (prev <= key) break;
                    wm.key[pos & rmask][lane] = prev;
                    wm.cnt[pos & rmask][lane] = wm.cnt[(pos - 1) & rmask][lane];
                    pos--;
                }
            }
            if (close) {
                wm.key[pos & rmask][lane] = key;
                wm.cnt[pos & rmask][lane] = (uint8_t)b;
            }
            ktail = (close && !sorted_insert) ? key : ktail;
            const bool at_front = close && pos == lpos;
            k2 = at_front ? kfront : ((close && pos == lpos + 1u) ? key : k2);
            kfront = at_front ? key : kfront;
            tpos += close ? 1u : 0u;
            nb += close ? 1u : 0u;
            head = close ? i : head;
            b = close ? 0 : b;
            // record i opens the next batch on the replica that is free first: one that was never used
            // (free from time 0) while there is one, else the slot with the smallest key
            const bool open = known && !join && b == 0;
            const bool pop = open && tpos - lpos == R;
            const uint64_t kf = pop ? kfront : 0ull;
            lpos += pop ? 1u : 0u;
            kfront = pop ? (lpos != tpos ? k2 : kInf) : kfront;
            tk = open ? (max(kf, ra) | qmask) : tk;
            b = open ? 1 : b;
            if (end && b == 0) lpos = tpos;     // stream exhausted: everything still held leaves, in key order

            // ---- hand on the record picked up at the top of the iteration
            if (FORK) {
                const uint64_t out = h_base | h_low;
                const bool go_a = da >= 0 && (cbit_a < 0 || ((h_bits >> cbit_a) & 1u) == cval_a);
                const bool go_b = db >= 0 && (cbit_b < 0 || ((h_bits >> cbit_b) & 1u) == cval_b);
                if (h_valid) {
                    if (go_a && IL_IN_RANGE(tail_a, size_a, p.status)) out_a[tail_a] = out;
                    if (go_b && IL_IN_RANGE(tail_b, size_b, p.status)) out_b[tail_b] = out;
                    // this copy leaves: the query's slab entry keeps the latest of its copies
                    if (!go_a && !go_b && IL_IN_RANGE(h_qid, p.n, p.status)) atomicMax(slab_row + h_qid, (h_base >> rb) | h_qid);
                }
                tail_a += (h_valid && go_a) ? 1u : 0u;
                tail_b += (h_valid && go_b) ? 1u : 0u;
                n_left += (h_valid && !go_a && !go_b) ? 1u : 0u;
            } else if (BRANCHY) {
                // under predicates: with lanes on both sides of a branch point in one warp this measured
                // 10 % faster than a branch around the block; without routing the branch is the faster form
                const bool to_b = bit >= 0 && ((h_bits >> bit) & 1u);
                const bool leaves = to_b ? db < 0 : da < 0;
                // (slab records are plain (finish, query) records whatever the streams carry)
                const uint64_t out = leaves ? ((h_base >> rb) | h_qid) : (h_base | h_low);
                uint64_t *dst = to_b ? out_b + (tail_b & mask_b) : out_a + (tail_a & mask_a);
                if (FEAS) late_fin = (h_valid && leaves) ? h_base : 0ull;
                if (h_valid && !(FEAS && leaves) &&
                    IL_IN_RANGE(to_b ? (tail_b & mask_b) : (tail_a & mask_a), to_b ? size_b : size_a, p.status))
                    *dst = out;
                tail_b += (h_valid && to_b) ? 1u : 0u;
                tail_a += (h_valid && !to_b) ? 1u : 0u;
            } else {
                if (FEAS) late_fin = (h_valid && da < 0) ? h_base : 0ull;
                if (h_valid) {
                    if (!(FEAS && da < 0) && IL_IN_RANGE(tail_a & mask_a, size_a, p.status))
                        out_a[tail_a & mask_a] = h_base | h_qid;
                    tail_a++;
                }
            }
            // ---- request the next record to hand on
            if (f_valid) {
                e_left = f_cnt;
                e_base = f_key & ~qmask;
                e_idx = (uint32_t)f_key & (uint32_t)qmask;
                if (RING) e_first = e_idx;
                epos++;
            }
            vmask = (vmask << 1) & 7u;
            eb3 = eb2; eb2 = eb1;
            if (e_left > 0 && can_emit) {
                const uint32_t sl = it & (kStage - 1);
                if (IL_IN_RANGE(e_idx & in_mask, in_size, p.status))
                    cp_async8(&wm.stage_e[sl][lane], in + (e_idx & in_mask));
                eb1 = e_base;
                e_idx++; e_left--;
                vmask |= 1u;
            }
            // ---- request the next record to examine: up to kStage records from the one examined
            // next, and (while the parent runs) kLag behind what it has written
            const uint32_t i2 = head + (uint32_t)b;
            if (fx < i2 + (uint32_t)kStage && (pdone ? fx < written : fx + (uint32_t)kLag < written)) {
                if (IL_IN_RANGE(fx & in_mask, in_size, p.status))
                    cp_async8(&wm.stage_x[fx & (kStage - 1)][lane], in + (fx & in_mask));
                fx++;
            }
            done = end && b == 0 && epos == tpos && e_left == 0 && vmask == 0u && !(FEAS && late_fin != 0ull);
            if (--guard == 0) {
                if (guard_hi == 0) { atomicCAS(p.status, 0, IL_ERR_ITER_LIMIT); atomicOr(&p.counters[5], 1ull); done = true; }
                else { guard_hi--; }      // guard wraps to 2^32 - 1 on the next decrement
            }
        }
        fx3 = fx2; fx2 = fx1; fx1 = fx;
        cp_async_commit();
        cp_async_wait<kPending>();
        // every lane publishes every iteration (a finished lane repeats its last words)
        if (lane_a >= 0) wm.avail[par][lane_a] = tail_a | (done ? kDone : 0u);
        if (lane_b >= 0) wm.avail[par][lane_b] = tail_b | (done ? kDone : 0u);
        av = av_next;
        par ^= 1;
        it++;
        __syncwarp();
    }
    cp_async_wait<0>();

    for (int o = 16; o > 0; o >>= 1) {
        batches += __shfl_xor_sync(full, batches, o);
        alg_ops += __shfl_xor_sync(full, alg_ops, o);
        exits_seen += __shfl_xor_sync(full, exits_seen, o);
        exits_due += __shfl_xor_sync(full, exits_due, o);
    }
    if (lane == 0 && exits_seen != exits_due) { atomicCAS(p.status, 0, IL_ERR_ITER_LIMIT); atomicOr(&p.counters[5], 2ull); }
    if (lane == 0 && batches) { atomicAdd(&p.counters[1], batches); atomicAdd(&p.counters[2], alg_ops); }
    if (FEAS) {
        for (int o = 16; o > 0; o >>= 1) early += __shfl_xor_sync(full, early, o);
        if (lane == 0 && early) atomicAdd(&p.counters[6], (unsigned long long)early);
    }
}

namespace {
bool any_branch(const DesParams &p)
{
    for (int s = 0; s < p.S; s++) if (p.bit[s] >= 0) return true;
    return false;
}
}  // namespace

namespace {
template <bool BRANCHY, bool RING, bool FEAS, bool FORK>
cudaError_t launch_one(const DesParams &p, int grid, size_t smem, cudaStream_t stream)
{
    cudaError_t e = cudaFuncSetAttribute(des_lane_kernel<BRANCHY, RING, FEAS, FORK>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    // Shared memory and L1 share 256 KB per SM.  Every stream record reaches a lane through L1 (cp.async),
    // 16 records per line, so the lines of all resident lanes must survive 16 iterations there: ask for
    // no more shared memory than the resident CTAs use (1 KB per CTA is the system's), the rest is L1.
    if (p.lane_ctas_per_sm > 0) {
        const size_t need = (size_t)p.lane_ctas_per_sm * (smem + 1024);
        int pct = (int)((need * 100 + 233472 - 1) / 233472);     // of the 228 KB an SM can give
        pct = pct < 1 ? 1 : (pct > 100 ? 100 : pct);
        e = cudaFuncSetAttribute(des_lane_kernel<BRANCHY, RING, FEAS, FORK>,
                                 cudaFuncAttributePreferredSharedMemoryCarveout, pct);
        if (e != cudaSuccess) return e;
    }
    des_lane_kernel<BRANCHY, RING, FEAS, FORK><<<grid, kLaneWarps * 32, smem, stream>>>(p);
    return cudaGetLastError();
}

template <bool BRANCHY, bool RING>
cudaError_t launch_two(const DesParams &p, int grid, size_t smem, cudaStream_t stream)
{
    return p.out_feasible ? launch_one<BRANCHY, RING, true, false>(p, grid, smem, stream)
                          : launch_one<BRANCHY, RING, false, false>(p, grid, smem, stream);
}
}  // namespace

// Feasibility-only when p.out_feasible is set; the fan-out instantiation when p.fork is (the host
// never combines that with stream rings or feasibility-only).
cudaError_t launch_des_lane(const DesParams &p, int grid, size_t smem, cudaStream_t stream)
{
    if (p.fork) {
        if (p.lane_wrap || p.out_feasible) return cudaErrorInvalidValue;
        return launch_one<true, false, false, true>(p, grid, smem, stream);
    }
    const bool br = any_branch(p);
    if (p.lane_wrap) return br ? launch_two<true, true>(p, grid, smem, stream) : launch_two<false, true>(p, grid, smem, stream);
    return br ? launch_two<true, false>(p, grid, smem, stream) : launch_two<false, false>(p, grid, smem, stream);
}

int des_lane_warps_per_cta() { return kLaneWarps; }

size_t des_lane_smem(int, int Bmax, int ring_slots)
{
    return (size_t)kLaneWarps * warp_mem_bytes(ring_slots, Bmax);
}

int des_lane_max_ctas_per_sm(size_t smem)
{
    int n = 0;
    if (cudaFuncSetAttribute(des_lane_kernel<true, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, des_lane_kernel<true, true, true>, kLaneWarps * 32, smem);
    return e == cudaSuccess ? n : 0;
}

}  // namespace il
