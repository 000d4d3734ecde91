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
// Records and keys are the packed 64-bit words of des_packed_kernel.cu:
// (time << q) | query for stream records, (finish << q) | index of the batch's
// first arrival for replica slots, whose unsigned order is (finish, dispatch
// order).  The host selects this kernel only when every reachable time fits.
#include "il_internal.h"

namespace il {

namespace {

constexpr int kLaneWarps = 2;                  // warps per CTA
constexpr int kRing = 32;                      // ring positions of a lane's slot list (>= IL_MAX_REPLICAS)
constexpr uint32_t kDone = 0x80000000u;
constexpr uint64_t kInf = ~0ull;
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

// Shared memory of one warp.
struct WarpMem {
    // Per lane a ring of batches, [pos][lane].  Positions [epos, lpos): batches whose slot has been
    // taken over, waiting to be handed on, in key order.  Positions [lpos, tpos): the slots in use,
    // sorted by key.
    uint64_t key[kRing][32];     // (finish << q) | index of the batch's first arrival
    uint32_t cnt[kRing][32];     // batch size
    // The lane's row of the profile, [b - 1][lane]: time of a batch of b on the stage's hardware type.
    // One copy per lane, so that lanes with different rows or batch sizes never meet in a bank.
    uint32_t lat[IL_MAX_BATCH][32];
    // Staging rings filled by cp.async, [position][lane]: the next records of the lane's arrival stream
    // (position = record index mod kStage), and the records it is handing on with the finish << q of
    // their batch (position = iteration mod kStage)
    uint64_t stage_x[kStage][32];
    uint64_t stage_e[kStage][32];
    uint64_t stage_b[kStage][32];
    // Mailboxes, double-buffered by iteration parity: what iteration k publishes in buffer k & 1 is read
    // in iteration k + 1, while iteration k + 1 publishes into the other buffer; one warp barrier per
    // iteration then separates every write of a word from the reads of its previous value.
    uint32_t avail[2][32];       // records written so far into the lane's arrival stream (by its parent
                                 // lane); kDone set once that is all of them
};

}  // namespace

// BRANCHY: some stage routes by a branch bit (otherwise every stage has one way out).
template <bool BRANCHY>
__global__ void __launch_bounds__(kLaneWarps * 32)
des_lane_kernel(const __grid_constant__ DesParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    int32_t *s_lat = reinterpret_cast<int32_t *>(smem_raw);      // the profile tables, [S][H][Bmax]
    const int n_tab = p.S * p.H * p.Bmax;
    WarpMem *wm_all = reinterpret_cast<WarpMem *>(smem_raw + ((size_t)n_tab * 4 + 15) / 16 * 16);
    const int q = p.qbits;
    const uint64_t qmask = (1ull << q) - 1ull;
    for (int i = threadIdx.x; i < n_tab; i += blockDim.x)
        s_lat[i] = p.lat[i];
    __syncthreads();

    const unsigned full = 0xffffffffu;
    const int wid = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    WarpMem &wm = wm_all[wid];
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
    const int da = p.dest_a[s], db = p.dest_b[s];
    const int bit = p.bit[s];
    const uint32_t n_in = lane_used ? (uint32_t)p.n_s[s] : 0u;
    const unsigned group_mask = lane_used ? (((1u << S) - 1u) << (j * S)) : 0u;
    // mailbox of the child on either side; a lane without that child writes a word nobody reads
    // (its own entry of a spare row would do as well: lanes j * S + child are always in range)
    const int lane_a = (da < 0 || !lane_used) ? -1 : j * S + da;
    const int lane_b = (db < 0 || db == da || !lane_used) ? -1 : j * S + db;

    const int64_t wslot = (int64_t)blockIdx.x * kLaneWarps + wid;
    uint64_t *my_block = p.lane_ws + (wslot * cpw + (lane_used ? j : 0)) * p.lane_elems;
    const uint64_t *in = s == 0 ? p.ptrace : my_block + p.lane_off[s];
    unsigned long long batches = 0, alg_ops = 0;

    for (;;) {
        unsigned long long g = 0;
        if (lane == 0) g = atomicAdd(&p.counters[0], (unsigned long long)cpw);
        g = __shfl_sync(full, g, 0);
        if (g >= (unsigned long long)p.n_cand) break;
        const int64_t c = (int64_t)g + j;
        const bool has = lane_used && c < p.n_cand;
        il_stage_config cfg = {0, 1, 1, 0};
        if (has) cfg = p.configs[c * S + s];
        const bool bad = has && (cfg.hw >= p.H || cfg.max_batch < 1 || cfg.max_batch > p.Bmax ||
                                 cfg.replicas < 1 || cfg.replicas > IL_MAX_REPLICAS);
        const bool cand_bad = (__ballot_sync(full, bad) & group_mask) != 0u;
        uint64_t *slab = reinterpret_cast<uint64_t *>(p.slab + (has ? c : 0) * p.slab_stride);
        if (has && cand_bad) {
            if (s == 0) atomicCAS(p.status, 0, IL_ERR_BAD_CONFIG);
            for (int i = s; i < p.n; i += S) slab[i] = 0;
        }
        const bool live = has && !cand_bad && n_in > 0;

        const uint32_t R = cfg.replicas;
        const int mb = cfg.max_batch;
        if (live) {
            const int32_t *row = s_lat + (s * p.H + cfg.hw) * p.Bmax;
            for (int k = 0; k < p.Bmax; k++) wm.lat[k][lane] = (uint32_t)row[k];
        }
        uint64_t *out_a = da < 0 ? slab + exit_off : my_block + p.lane_off[da];
        uint64_t *out_b = db < 0 ? slab + exit_off : my_block + p.lane_off[db];

        // the root's stream is complete from the start; a stage nobody visits is finished at once
        const uint32_t avail0 = (s == 0 || !live) ? (n_in | kDone) : 0u;
        wm.avail[0][lane] = avail0; wm.avail[1][lane] = avail0;
        __syncwarp();

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
        // fetch cursor of the arrival stream: records below fx have been requested; fx1..fx3 are its
        // values at the end of the previous three iterations, so records below fx3 have arrived
        uint32_t fx = 0, fx1 = 0, fx2 = 0, fx3 = 0;
        uint32_t tail_a = 0, tail_b = 0;
        unsigned nb = 0;
        bool done = !live;
        const unsigned long long limit = 8ull * (unsigned)p.n * (unsigned)(S + 1) + 4096ull;
        uint32_t guard = limit > 0xffffffffull ? 0xffffffffu : (uint32_t)limit;
        int par = 0;                 // mailbox buffer this iteration publishes into; it reads the other one
        uint32_t av = avail0;        // mailbox word this iteration works with: the one read an iteration ago
        uint32_t it = 0;

        for (;;) {
            const uint32_t av_next = wm.avail[par ^ 1][lane];
            if (!done) {
                // the record to hand on in this iteration (requested three iterations ago); its branch bits
                // are fetched here, so that the load runs under the examine step
                const bool h_valid = (vmask & 4u) != 0u;
                const uint32_t h_sl = (it + 1u) & (kStage - 1);
                const uint32_t h_qid = (uint32_t)wm.stage_e[h_sl][lane] & (uint32_t)qmask;   // unused unless h_valid
                const uint64_t h_base = wm.stage_b[h_sl][lane];
                uint32_t h_bits = 0;
                if (BRANCHY && h_valid && bit >= 0) h_bits = p.bits[h_qid];
                // likewise the next batch to hand on, if the one in hand is used up (a batch handed over in
                // this iteration is picked up in the next), and the table entry a close would need
                const bool f_valid = e_left == 0 && epos != lpos;
                const uint64_t f_key = wm.key[epos & (kRing - 1)][lane];                      // unused unless f_valid
                const uint32_t f_cnt = wm.cnt[epos & (kRing - 1)][lane];
                // (latency << q) - qmask: finish key base = dispatch key + that
                const uint64_t latq = ((uint64_t)wm.lat[b > 0 ? b - 1 : 0][lane] << q) - qmask;
                // key of the second slot in use, the front after a hand-over (unused unless there are two)
                uint64_t k2 = wm.key[(lpos + 1u) & (kRing - 1)][lane];
                const uint32_t written = av & ~kDone;
                const bool pdone = (av & kDone) != 0u;

                // ---- examine one record of the arrival stream
                const uint32_t i = head + (uint32_t)b;
                const bool known = i < fx3;
                const uint64_t ra = wm.stage_x[i & (kStage - 1)][lane];
                const bool end = pdone && i >= written;
                const bool join = known && b > 0 && b < mb && ra <= tk;
                b += join ? 1 : 0;
                const bool room = tpos - epos < (uint32_t)kRing;
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
                        const uint64_t prev = wm.key[(pos - 1) & (kRing - 1)][lane];
                        if (prev <= key) break;
                        wm.key[pos & (kRing - 1)][lane] = prev;
                        wm.cnt[pos & (kRing - 1)][lane] = wm.cnt[(pos - 1) & (kRing - 1)][lane];
                        pos--;
                    }
                }
                if (close) {
                    wm.key[pos & (kRing - 1)][lane] = key;
                    wm.cnt[pos & (kRing - 1)][lane] = (uint32_t)b;
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
                if (BRANCHY) {
                    // under predicates: with lanes on both sides of a branch point in one warp this measured
                    // 10 % faster than a branch around the block; without routing the branch is the faster form
                    const uint64_t out = h_base | h_qid;
                    const bool to_b = bit >= 0 && ((h_bits >> bit) & 1u);
                    uint64_t *dst = to_b ? out_b + tail_b : out_a + tail_a;
                    if (h_valid) *dst = out;
                    tail_b += (h_valid && to_b) ? 1u : 0u;
                    tail_a += (h_valid && !to_b) ? 1u : 0u;
                } else if (h_valid) {
                    out_a[tail_a] = h_base | h_qid;
                    tail_a++;
                }
                // ---- request the next record to hand on
                if (f_valid) {
                    e_left = f_cnt;
                    e_base = f_key & ~qmask;
                    e_idx = (uint32_t)f_key & (uint32_t)qmask;
                    epos++;
                }
                vmask = (vmask << 1) & 7u;
                if (e_left > 0) {
                    const uint32_t sl = it & (kStage - 1);
                    cp_async8(&wm.stage_e[sl][lane], in + e_idx);
                    wm.stage_b[sl][lane] = e_base;
                    e_idx++; e_left--;
                    vmask |= 1u;
                }
                // ---- request the next record to examine: up to kStage records from the one examined
                // next, and (while the parent runs) kLag behind what it has written
                const uint32_t i2 = head + (uint32_t)b;
                if (fx < i2 + (uint32_t)kStage && (pdone ? fx < written : fx + (uint32_t)kLag < written)) {
                    cp_async8(&wm.stage_x[fx & (kStage - 1)][lane], in + fx);
                    fx++;
                }
                done = end && b == 0 && epos == tpos && vmask == 0u;
                if (--guard == 0) { atomicCAS(p.status, 0, IL_ERR_ITER_LIMIT); done = true; }
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
            if (__all_sync(full, done)) break;
        }
        cp_async_wait<0>();

        if (live) {
            batches += nb;
            alg_ops += 3ull * n_in + (unsigned long long)nb * (unsigned)(R + mb + 4);
        }
        // every query of the candidate must have left through exactly one leaf
        int exits = 0;
        if (live) exits = (da < 0 ? (int)tail_a : 0) + ((db < 0 && bit >= 0) ? (int)tail_b : 0);
        for (int o = 16; o > 0; o >>= 1) exits += __shfl_xor_sync(full, exits, o);
        int expect = 0;
        if (has && !cand_bad && s == 0) expect = p.n;
        for (int o = 16; o > 0; o >>= 1) expect += __shfl_xor_sync(full, expect, o);
        if (lane == 0 && exits != expect) atomicCAS(p.status, 0, IL_ERR_ITER_LIMIT);
        __syncwarp();
    }
    for (int o = 16; o > 0; o >>= 1) {
        batches += __shfl_xor_sync(full, batches, o);
        alg_ops += __shfl_xor_sync(full, alg_ops, o);
    }
    if (lane == 0 && batches) { atomicAdd(&p.counters[1], batches); atomicAdd(&p.counters[2], alg_ops); }
}

namespace {
bool any_branch(const DesParams &p)
{
    for (int s = 0; s < p.S; s++) if (p.bit[s] >= 0) return true;
    return false;
}
}  // namespace

cudaError_t launch_des_lane(const DesParams &p, int grid, size_t smem, cudaStream_t stream)
{
    const bool br = any_branch(p);
    cudaError_t e = br
        ? cudaFuncSetAttribute(des_lane_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)
        : cudaFuncSetAttribute(des_lane_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    if (br) des_lane_kernel<true><<<grid, kLaneWarps * 32, smem, stream>>>(p);
    else des_lane_kernel<false><<<grid, kLaneWarps * 32, smem, stream>>>(p);
    return cudaGetLastError();
}

int des_lane_warps_per_cta() { return kLaneWarps; }

size_t des_lane_smem(int n_tab)
{
    return ((size_t)n_tab * 4 + 15) / 16 * 16 + (size_t)kLaneWarps * sizeof(WarpMem);
}

int des_lane_max_ctas_per_sm(size_t smem)
{
    int n = 0;
    if (cudaFuncSetAttribute(des_lane_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, des_lane_kernel<true>, kLaneWarps * 32, smem);
    return e == cudaSuccess ? n : 0;
}

}  // namespace il
