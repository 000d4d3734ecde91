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
// how far its parent has got from two words in shared memory that the parent
// publishes every iteration: the number of records written so far, and a lower
// bound on the time of every record still to come (its watermark).  A batch
// that is not full and has seen all records written so far may only be closed
// once the parent's watermark has passed the batch's dispatch time; until then
// the lane idles for that iteration.  Parents never wait for children, so the
// root always advances and every wait ends.
//
// Records and keys are the packed 64-bit words of des_packed_kernel.cu:
// (time << q) | query for stream records, (finish << q) | index of the batch's
// first arrival for replica slots, whose unsigned order is (finish, dispatch
// order).  The host selects this kernel only when every reachable time fits.
#include "il_internal.h"

namespace il {

namespace {

constexpr int kLaneWarps = 2;                  // warps per CTA
constexpr int kRcap = IL_MAX_REPLICAS;         // ring positions of a lane's slot list
constexpr uint64_t kInf = ~0ull;

// Shared memory of one warp.
struct WarpMem {
    uint64_t key[kRcap][32];     // slot lists, sorted by key from position lhead on (ring); [pos][lane]
    uint32_t cnt[kRcap][32];     // batch size held by the slot (0: replica never used)
    // Mailboxes, double-buffered by iteration parity: what iteration k publishes in buffer k & 1 is read
    // in iteration k + 1, while iteration k + 1 publishes into the other buffer; one warp barrier per
    // iteration then separates every write of a word from the reads of its previous value.
    uint64_t wmark[2][32];       // lane's watermark: (lower bound on the time of records still to come) << q
    uint32_t avail[2][32];       // records written so far into the lane's arrival stream (by its parent lane)
};

}  // namespace

__global__ void __launch_bounds__(kLaneWarps * 32)
des_lane_kernel(const __grid_constant__ DesParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    int32_t *s_lat = reinterpret_cast<int32_t *>(smem_raw);
    const int n_tab = p.S * p.H * p.Bmax;
    WarpMem *wm_all = reinterpret_cast<WarpMem *>(smem_raw + ((size_t)n_tab * 4 + 15) / 16 * 16);
    for (int i = threadIdx.x; i < n_tab; i += blockDim.x) s_lat[i] = p.lat[i];
    __syncthreads();

    const unsigned full = 0xffffffffu;
    const int wid = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    WarpMem &wm = wm_all[wid];
    const int S = p.S, cpw = p.cpw;
    const int j = lane / S, s = lane - j * S;
    const bool lane_used = j < cpw;
    const int q = p.qbits;
    const uint64_t qmask = (1ull << q) - 1ull;

    // static facts of this lane's stage
    int parent = -1;
    int exit_off = 0;
    for (int u = 0; u < S; u++) {
        const int a = p.dest_a[u], b2 = p.dest_b[u];
        if (u != s && (a == s || b2 == s)) parent = u;
        if (u < s) {
            int kids = 0;
            if (a >= 0) kids += p.n_s[a];
            if (b2 >= 0 && b2 != a) kids += p.n_s[b2];
            exit_off += p.n_s[u] - kids;
        }
    }
    const int par_lane = (lane_used && s > 0 && parent >= 0) ? j * S + parent : lane;
    const int da = p.dest_a[s], db = p.dest_b[s];
    const int bit = p.bit[s];
    const uint32_t n_in = lane_used ? (uint32_t)p.n_s[s] : 0u;
    const unsigned group_mask = lane_used ? (((1u << S) - 1u) << (j * S)) : 0u;

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

        const int R = cfg.replicas, mb = cfg.max_batch;
        const int32_t *row = s_lat + (s * p.H + cfg.hw) * p.Bmax;
        uint64_t *out_a = da < 0 ? slab + exit_off : my_block + p.lane_off[da];
        uint64_t *out_b = db < 0 ? slab + exit_off : my_block + p.lane_off[db];
        const int lane_a = (da < 0 || !lane_used) ? -1 : j * S + da;
        const int lane_b = (db < 0 || db == da || !lane_used) ? -1 : j * S + db;

        // slot list: R slots of never-used replicas (key 0 sorts first)
        if (live) for (int r = 0; r < R; r++) { wm.key[r][lane] = 0; wm.cnt[r][lane] = 0; }
        wm.avail[0][lane] = 0; wm.avail[1][lane] = 0;
        wm.wmark[0][lane] = live ? 0 : kInf; wm.wmark[1][lane] = live ? 0 : kInf;
        __syncwarp();

        uint32_t lhead = 0;          // ring position of the list's first slot
        int lcount = R;              // slots in the list (R, or R - 1 while a batch is open)
        int nempty = R;              // never-used slots still at the front of the list
        uint64_t kfront = 0;         // key of the list's first slot (kInf when the list is empty)
        uint32_t head = 0;           // index of the open batch's first record
        int b = 0;                   // size of the open batch (0: none)
        uint64_t tk = 0;             // open batch's dispatch time as (t << q) | qmask
        uint64_t e_base = 0;         // finish << q of the batch being handed on
        uint32_t e_idx = 0;          // its next record in the arrival stream
        int e_left = 0;              // records of it still to hand on
        uint64_t rec_e = 0;          // in[e_idx], loaded ahead
        uint64_t nx = 0;             // in[head + b], loaded ahead when nx_ok
        bool nx_ok = false;
        uint32_t tail_a = 0, tail_b = 0;
        unsigned nb = 0;
        bool done = !live;
        long long guard = 8ll * p.n * (S + 1) + 4096;
        int par = 0;                 // buffer this iteration publishes into; it reads the other one
        uint64_t w_pub = live ? 0 : kInf;

        while (!__all_sync(full, done)) {
            uint32_t avail = n_in;
            uint64_t wp = kInf;
            if (s != 0) { avail = wm.avail[par ^ 1][lane]; wp = wm.wmark[par ^ 1][par_lane]; }
            if (!done) {
                // ---- emit one record of the batch being handed on
                if (e_left > 0) {
                    const uint32_t qid = (uint32_t)(rec_e & qmask);
                    const uint64_t out = e_base | qid;
                    bool to_b = false;
                    if (bit >= 0) to_b = (p.bits[qid] >> bit) & 1;
                    if (to_b) out_b[tail_b++] = out; else out_a[tail_a++] = out;
                    e_idx++; e_left--;
                    if (e_left > 0) rec_e = in[e_idx];
                }
                // ---- examine one record of the arrival stream
                const uint32_t i = head + (uint32_t)b;
                bool close = false, consume = false;
                if (i < avail) {
                    if (!nx_ok) { nx = in[i]; nx_ok = true; }
                    if (b > 0 && b < mb && nx <= tk) { b++; consume = true; }
                    else close = b > 0;
                } else if (i >= n_in) {
                    close = b > 0;
                } else {
                    close = b > 0 && (b == mb || wp > tk);
                }
                if (close) {
                    const uint64_t fk = (tk - qmask) + ((uint64_t)(uint32_t)row[b - 1] << q);
                    const uint64_t key = fk | head;
                    uint32_t pos = lhead + (uint32_t)lcount;
                    while (pos != lhead) {
                        const uint64_t prev = wm.key[(pos - 1) & (kRcap - 1)][lane];
                        if (prev <= key) break;
                        wm.key[pos & (kRcap - 1)][lane] = prev;
                        wm.cnt[pos & (kRcap - 1)][lane] = wm.cnt[(pos - 1) & (kRcap - 1)][lane];
                        pos--;
                    }
                    wm.key[pos & (kRcap - 1)][lane] = key;
                    wm.cnt[pos & (kRcap - 1)][lane] = (uint32_t)b;
                    if (pos == lhead) kfront = key;
                    lcount++;
                    nb++;
                    head = i;
                    b = 0;
                }
                if (b == 0 && e_left == 0) {
                    if (i < avail) {
                        // open the next batch with record i; it takes over the first slot
                        const uint32_t c0 = wm.cnt[lhead & (kRcap - 1)][lane];
                        if (nempty > 0) nempty--;
                        else {
                            e_base = kfront & ~qmask;
                            e_idx = (uint32_t)(kfront & qmask);
                            e_left = (int)c0;
                            rec_e = in[e_idx];
                        }
                        tk = max(kfront, nx) | qmask;
                        lhead++; lcount--;
                        kfront = lcount > 0 ? wm.key[lhead & (kRcap - 1)][lane] : kInf;
                        b = 1;
                        consume = true;
                    } else if (i >= n_in) {
                        // arrival stream exhausted: hand on what the slots still hold, in key order
                        lhead += (uint32_t)nempty; lcount -= nempty; nempty = 0;
                        if (lcount > 0) {
                            const uint64_t k0 = wm.key[lhead & (kRcap - 1)][lane];
                            e_base = k0 & ~qmask;
                            e_idx = (uint32_t)(k0 & qmask);
                            e_left = (int)wm.cnt[lhead & (kRcap - 1)][lane];
                            rec_e = in[e_idx];
                            lhead++; lcount--;
                            kfront = lcount > 0 ? wm.key[lhead & (kRcap - 1)][lane] : kInf;
                        } else {
                            done = true;
                        }
                    }
                }
                if (consume) {
                    nx_ok = i + 1 < avail;
                    if (nx_ok) nx = in[i + 1];
                }
                // ---- publish: records written, and a lower bound on what is still to come
                uint64_t w = kInf;
                if (!done) {
                    if (e_left > 0) w = e_base;
                    else if (lcount > nempty)
                        w = (nempty == 0 ? kfront : wm.key[(lhead + (uint32_t)nempty) & (kRcap - 1)][lane]) & ~qmask;
                    uint64_t nxt;   // (time << q) + 1 unit that every batch still to be closed finishes at or after
                    if (b > 0) nxt = tk + 1;
                    else {
                        const uint32_t i2 = head;      // b == 0: next record to open with
                        uint64_t lb = kInf;
                        if (i2 < avail && nx_ok) lb = nx & ~qmask;
                        else if (i2 < n_in) lb = (i2 < avail) ? 0 : wp;
                        nxt = lb == kInf ? kInf : lb + qmask + 1;
                    }
                    w = min(w, nxt);
                }
                if (--guard < 0) { atomicCAS(p.status, 0, IL_ERR_ITER_LIMIT); done = true; w = kInf; }
                w_pub = w;
            }
            // every lane publishes every iteration (a finished lane repeats its last words)
            wm.wmark[par][lane] = w_pub;
            if (lane_a >= 0) wm.avail[par][lane_a] = tail_a;
            if (lane_b >= 0) wm.avail[par][lane_b] = tail_b;
            par ^= 1;
            __syncwarp();
        }

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

cudaError_t launch_des_lane(const DesParams &p, int grid, size_t smem, cudaStream_t stream)
{
    cudaError_t e = cudaFuncSetAttribute(des_lane_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    des_lane_kernel<<<grid, kLaneWarps * 32, smem, stream>>>(p);
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
    if (cudaFuncSetAttribute(des_lane_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, des_lane_kernel, kLaneWarps * 32, smem);
    return e == cudaSuccess ? n : 0;
}

}  // namespace il
