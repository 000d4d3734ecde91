// Batched discrete-event simulation of the InferLine Estimator (Section 4.2),
// one candidate configuration per warp.
//
// Formulation.  The pipeline is a feed-forward tree with zero delay between
// stages and no back-pressure, so the arrival stream of a stage is fully
// determined by the completion stream of its parent.  A warp therefore
// simulates its candidate stage by stage: it turns the sorted stream of
// (time, query) arrivals of stage s into the sorted stream of completions,
// which is split by the branch bits into the arrival streams of the children
// (or into exit latencies).  Within one stage the centralized batched queue
// (Section 3) is a FIFO, so the queue is always a window [head, tail) of the
// arrival stream, and one step of the simulation is one batch:
//
//     t      = max(earliest time a replica is free, arrival[head])
//     b      = min(max batch, number of arrivals from head on with time <= t)
//     finish = t + latency[stage][hw][b-1]            (Section 4.1 profile)
//
// Replicas are identical, so only the multiset of their free times matters:
// lane r of the warp holds replica r's finish time, the replica with the
// smallest (finish, dispatch order) is the one that is reused, and the batch it
// held is emitted to the next stage at that moment.  Because every later batch
// finishes strictly after the current dispatch time, batches are emitted in
// (finish, dispatch order) order, which is the order in which the next stage's
// queue sees them; batch-mates keep their order.
#include "il_internal.h"

namespace il {

namespace {

constexpr int64_t kNever = INT64_MAX;

__device__ __forceinline__ int64_t warp_min_i64(int64_t v)
{
    // Times are non-negative or -1; compare as (hi signed, lo unsigned).
    const int32_t hi = (int32_t)(v >> 32);
    const int32_t mhi = __reduce_min_sync(0xffffffffu, hi);
    const uint32_t lo = (hi == mhi) ? (uint32_t)v : 0xffffffffu;
    const uint32_t mlo = __reduce_min_sync(0xffffffffu, lo);
    return (int64_t)(((uint64_t)(uint32_t)mhi << 32) | (uint64_t)mlo);
}

// Where one stage's completions go.
struct Route {
    int64_t *a_time; int32_t *a_qid; int32_t a_tail;   // branch bit 0 / unconditional
    int64_t *b_time; int32_t *b_qid; int32_t b_tail;   // branch bit 1
    int bit;                                           // -1: no test
    bool a_exit, b_exit;
};

// Number of leading elements of the sorted array t[0 .. len) that are < key (strict) or <= key.
__device__ __forceinline__ int count_below(const int64_t *t, int len, int64_t key, bool or_equal)
{
    int a = 0, b = len;
    while (a < b) {
        const int m = (a + b) >> 1;
        const int64_t v = t[m];
        if (v < key || (or_equal && v == key)) a = m + 1; else b = m;
    }
    return a;
}

// Arrival stream of a join (a stage with two incoming edges), built by one warp from the two incoming
// streams A (edge from the first parent, na records) and B (edge from the second parent, nb records), both
// sorted by time.  A query is ready at the join when the last of its inputs has arrived, and queries that
// become ready in the same instant queue in the order (delivering stage, that stage's completion order);
// the first parent has the smaller stage index.  So the stream is the merge of
//   Y: the records of A whose query has no record in B, or an earlier one   (made ready by the first parent)
//   X: the records of B whose query has no record in A, or one that is not later (made ready by the second)
// with Y before X at equal times; both halves are subsequences of sorted streams, hence sorted, and an
// element's place in the merge is its index in its own half plus the number of elements of the other half
// that go before it, found by bisection.  Returns the length of the merged stream.
__device__ int build_join_stream(const DesParams &p, int s, int64_t *my_time, int32_t *my_qid, int lane)
{
    const unsigned full = 0xffffffffu;
    const unsigned lt_mask = (1u << lane) - 1u;
    const int na = p.join_na[s], nb = p.join_nb[s];
    const int64_t *ta = my_time + p.join_in_a[s]; const int32_t *qa = my_qid + p.join_in_a[s];
    const int64_t *tb = my_time + p.join_in_b[s]; const int32_t *qb = my_qid + p.join_in_b[s];
    const int64_t n_pad = (p.n + 31) / 32 * 32;
    int64_t *seen_a = my_time + p.join_t_off, *seen_b = seen_a + n_pad;     // time of the query's record, -1: none
    for (int i = lane; i < p.n; i += 32) { seen_a[i] = -1; seen_b[i] = -1; }
    __syncwarp();
    for (int i = lane; i < na; i += 32) { const int32_t q = qa[i]; if (IL_IN_RANGE(q, p.n, p.status)) seen_a[q] = ta[i]; }
    for (int i = lane; i < nb; i += 32) { const int32_t q = qb[i]; if (IL_IN_RANGE(q, p.n, p.status)) seen_b[q] = tb[i]; }
    __syncwarp();
    int64_t *ty = my_time + p.join_tmp_off; int32_t *qy = my_qid + p.join_tmp_off;
    int64_t *tx = ty + (na + 31) / 32 * 32; int32_t *qx = qy + (na + 31) / 32 * 32;
    int ny = 0, nx = 0;
    for (int i0 = 0; i0 < na; i0 += 32) {
        const int i = i0 + lane;
        bool keep = false; int64_t t = 0; int32_t q = 0;
        if (i < na) { t = ta[i]; q = qa[i]; if (IL_IN_RANGE(q, p.n, p.status)) keep = t > seen_b[q]; }   // -1: no record in B
        const unsigned m = __ballot_sync(full, keep);
        if (keep) { const int at = ny + __popc(m & lt_mask); ty[at] = t; qy[at] = q; }
        ny += __popc(m);
    }
    for (int i0 = 0; i0 < nb; i0 += 32) {
        const int i = i0 + lane;
        bool keep = false; int64_t t = 0; int32_t q = 0;
        if (i < nb) { t = tb[i]; q = qb[i]; if (IL_IN_RANGE(q, p.n, p.status)) keep = t >= seen_a[q]; }
        const unsigned m = __ballot_sync(full, keep);
        if (keep) { const int at = nx + __popc(m & lt_mask); tx[at] = t; qx[at] = q; }
        nx += __popc(m);
    }
    __syncwarp();
    int64_t *out_t = my_time + p.buf_off[s]; int32_t *out_q = my_qid + p.buf_off[s];
    const int total = nx + ny;
    if (total != p.n_s[s]) return -1;          // the host counted something else: give up before writing
    for (int i = lane; i < ny; i += 32) {
        const int at = i + count_below(tx, nx, ty[i], false);
        out_t[at] = ty[i]; out_q[at] = qy[i];
    }
    for (int i = lane; i < nx; i += 32) {
        const int at = i + count_below(ty, ny, tx[i], true);
        out_t[at] = tx[i]; out_q[at] = qx[i];
    }
    __syncwarp();
    return total;
}

}  // namespace

__global__ void __launch_bounds__(kWarpsPerCta * 32)
des_kernel(const __grid_constant__ DesParams p)
{
    extern __shared__ int32_t s_lat[];
    const int n_tab = p.S * p.H * p.Bmax;
    for (int i = threadIdx.x; i < n_tab; i += blockDim.x) s_lat[i] = p.lat[i];
    __syncthreads();

    const unsigned full = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const unsigned lt_mask = (1u << lane) - 1u;
    const int64_t slot = (int64_t)blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5);
    int64_t *my_time = p.ws_time + slot * p.slot_elems;
    int32_t *my_qid = p.ws_qid + slot * p.slot_elems;
    unsigned long long batches = 0;
    unsigned long long alg_ops = 0;   // algorithmic integer operations: (R + mb + 4) per batch, 3 per query-event

    for (;;) {
        unsigned long long c = 0;
        if (lane == 0) c = atomicAdd(&p.counters[0], 1ull);
        c = __shfl_sync(full, c, 0);
        if (c >= (unsigned long long)p.n_cand) break;
        c = (unsigned long long)p.order[c];

        // candidate decode: lane s reads stage s
        il_stage_config my_cfg = {0, 1, 1, 0};
        if (lane < p.S) my_cfg = p.configs[c * p.S + lane];
        const bool bad = lane < p.S && (my_cfg.hw >= p.H || my_cfg.max_batch < 1 ||
                                        my_cfg.max_batch > p.Bmax || my_cfg.replicas < 1 ||
                                        my_cfg.replicas > IL_MAX_REPLICAS);
        if (__any_sync(full, bad)) {
            if (lane == 0) atomicCAS(p.status, 0, IL_ERR_BAD_CONFIG);
            for (int i = lane; i < p.n; i += 32) p.slab[c * p.slab_stride + i] = 0;
            continue;
        }

        int64_t *slab = p.slab + c * p.slab_stride;
        if (p.fork) {       // per-query maxima start from zero
            for (int i = lane; i < p.n; i += 32) slab[i] = 0;
            __syncwarp();
        }
        int32_t exits = 0;
        unsigned long long cand_batches = 0;
        bool over = false;      // more batches than the iteration bound allows: the candidate is given up

        for (int s = 0; s < p.S; s++) {
            const int n_in = p.n_s[s];
            if (n_in == 0) continue;
            if (p.fork && p.join_b[s] >= 0 && build_join_stream(p, s, my_time, my_qid, lane) != n_in) {
                if (lane == 0) { atomicCAS(p.status, 0, IL_ERR_ITER_LIMIT); atomicOr(&p.counters[5], 16ull); }
                over = true;
                break;
            }
            const int hw = __shfl_sync(full, (int)my_cfg.hw, s);
            const int mb = __shfl_sync(full, (int)my_cfg.max_batch, s);
            const int R = __shfl_sync(full, (int)my_cfg.replicas, s);
            const int32_t *row = s_lat + (s * p.H + hw) * p.Bmax;
            const int64_t *in_t = (s == 0) ? p.arrival : my_time + p.buf_off[s];
            const int32_t *in_q = (s == 0) ? nullptr : my_qid + p.buf_off[s];

            Route rt;
            rt.bit = p.bit[s];
            const int da = p.dest_a[s], db = p.dest_b[s];
            rt.a_exit = da < 0; rt.b_exit = db < 0;
            rt.a_time = rt.a_exit ? nullptr : my_time + p.buf_off[da];
            rt.a_qid = rt.a_exit ? nullptr : my_qid + p.buf_off[da];
            rt.b_time = rt.b_exit ? nullptr : my_time + p.buf_off[db];
            rt.b_qid = rt.b_exit ? nullptr : my_qid + p.buf_off[db];
            rt.a_tail = 0; rt.b_tail = 0;

            // Emits the batch [start, start + b) of this stage's input stream,
            // finished at time tfin, to the children / the latency slab.
            auto emit = [&](int start, int b, int64_t tfin) {
                for (int j0 = 0; j0 < b; j0 += 32) {
                    const int j = j0 + lane;
                    const bool act = j < b;
                    int32_t q = 0;
                    if (act) q = (s == 0) ? start + j : in_q[start + j];
                    if (p.fork) {
                        // fan-out: every edge whose condition holds; a copy that finds none leaves, and
                        // the slab keeps the largest latency of the query's copies (the stages of a
                        // candidate run one after the other on this warp, so a plain maximum will do)
                        const int ca = p.child_a[s], cb = p.child_b[s];
                        unsigned bits = 0;
                        if (act && (p.cbit_a[s] >= 0 || p.cbit_b[s] >= 0) && IL_IN_RANGE(q, p.n, p.status)) bits = p.bits[q];
                        const bool go_a = act && ca >= 0 && (p.cbit_a[s] < 0 || ((bits >> p.cbit_a[s]) & 1u) == p.cval_a[s]);
                        const bool go_b = act && cb >= 0 && (p.cbit_b[s] < 0 || ((bits >> p.cbit_b[s]) & 1u) == p.cval_b[s]);
                        const bool left = act && !go_a && !go_b;
                        const unsigned fa = __ballot_sync(full, go_a), fb = __ballot_sync(full, go_b);
                        const unsigned fl = __ballot_sync(full, left);
                        if (go_a) {
                            const int at = rt.a_tail + __popc(fa & lt_mask);
                            if (IL_IN_RANGE(p.out_off_a[s] + at, p.slot_elems, p.status)) {
                                (my_time + p.out_off_a[s])[at] = tfin; (my_qid + p.out_off_a[s])[at] = q;
                            }
                        }
                        if (go_b) {
                            const int at = rt.b_tail + __popc(fb & lt_mask);
                            if (IL_IN_RANGE(p.out_off_b[s] + at, p.slot_elems, p.status)) {
                                (my_time + p.out_off_b[s])[at] = tfin; (my_qid + p.out_off_b[s])[at] = q;
                            }
                        }
                        if (left && IL_IN_RANGE(q, p.n, p.status)) {
                            const int64_t l = tfin - p.arrival[q];
                            if (l > slab[q]) slab[q] = l;
                        }
                        rt.a_tail += __popc(fa); rt.b_tail += __popc(fb);
                        exits += __popc(fl);
                        continue;
                    }
                    bool bitv = false;
                    if (act && rt.bit >= 0 && IL_IN_RANGE(q, p.n, p.status)) bitv = (p.bits[q] >> rt.bit) & 1;
                    const unsigned ma = __ballot_sync(full, act && !bitv);
                    const unsigned mb_ = __ballot_sync(full, act && bitv);
                    if (ma) {
                        const bool mine = act && !bitv;
                        const int rank = __popc(ma & lt_mask);
                        if (rt.a_exit) {
                            if (mine && IL_IN_RANGE(q, p.n, p.status)) {
                                const int64_t l = tfin - p.arrival[q];
                                slab[q] = l;   // trace order: the slab doubles as the per-query answer
                            }
                            exits += __popc(ma);
                        } else {
                            if (mine && IL_IN_RANGE(p.buf_off[da] + rt.a_tail + rank, p.slot_elems, p.status)) {
                                rt.a_time[rt.a_tail + rank] = tfin; rt.a_qid[rt.a_tail + rank] = q;
                            }
                            rt.a_tail += __popc(ma);
                        }
                    }
                    if (mb_) {
                        const bool mine = act && bitv;
                        const int rank = __popc(mb_ & lt_mask);
                        if (rt.b_exit) {
                            if (mine && IL_IN_RANGE(q, p.n, p.status)) {
                                const int64_t l = tfin - p.arrival[q];
                                slab[q] = l;   // trace order: the slab doubles as the per-query answer
                            }
                            exits += __popc(mb_);
                        } else {
                            if (mine && IL_IN_RANGE(p.buf_off[db] + rt.b_tail + rank, p.slot_elems, p.status)) {
                                rt.b_time[rt.b_tail + rank] = tfin; rt.b_qid[rt.b_tail + rank] = q;
                            }
                            rt.b_tail += __popc(mb_);
                        }
                    }
                }
            };

            // replica slots: lane r < R holds replica r
            int64_t fin = (lane < R) ? -1 : kNever;   // -1: idle since before the first arrival
            int32_t seq = lane, sl_start = 0, sl_b = 0;
            int32_t seq_ctr = 32;

            // picks the slot with the smallest (finish, dispatch order)
            auto pick = [&](int64_t minfin) -> int {
                const unsigned tie = __ballot_sync(full, fin == minfin);
                if (__popc(tie) == 1) return __ffs(tie) - 1;
                const int32_t myseq = (fin == minfin) ? seq : INT32_MAX;
                const int32_t mseq = __reduce_min_sync(full, myseq);
                return __ffs(__ballot_sync(full, myseq == mseq)) - 1;
            };

            int head = 0;
            int guard = 0;
            const int ops_per_batch = R + mb + 4;
            alg_ops += 3ull * (unsigned)n_in;
            while (head < n_in) {
                const int64_t minfin = warp_min_i64(fin);
                const int sel = pick(minfin);
                // lookahead: how many queued arrivals are there at time t, up to mb
                const int i0 = head + lane;
                const int64_t v0 = (lane < mb && i0 < n_in) ? in_t[i0] : kNever;
                const int64_t a_head = __shfl_sync(full, v0, 0);
                const int64_t t = minfin > a_head ? minfin : a_head;
                int cnt = __popc(__ballot_sync(full, v0 <= t));
                if (mb > 32 && cnt == 32) {
                    const int i1 = head + 32 + lane;
                    const int64_t v1 = (32 + lane < mb && i1 < n_in) ? in_t[i1] : kNever;
                    cnt += __popc(__ballot_sync(full, v1 <= t));
                }
                const int64_t newfin = t + (int64_t)row[cnt - 1];
                // the slot being reused gives up the batch it held
                const int pb = __shfl_sync(full, sl_b, sel);
                const int ps = __shfl_sync(full, sl_start, sel);
                if (pb > 0) emit(ps, pb, minfin);
                if (lane == sel) { fin = newfin; seq = seq_ctr; sl_start = head; sl_b = cnt; }
                seq_ctr++;
                head += cnt;
                batches++;
                alg_ops += ops_per_batch;
                if (++guard > n_in) {   // cannot happen: every batch takes >= 1 query
                    if (lane == 0) atomicCAS(p.status, 0, IL_ERR_ITER_LIMIT);
                    break;
                }
            }
            // drain what is still in flight, in (finish, dispatch order) order
            for (int k = 0; k < 32; k++) {
                const int64_t minfin = warp_min_i64(fin);
                if (minfin == kNever) break;
                const int sel = pick(minfin);
                const int pb = __shfl_sync(full, sl_b, sel);
                const int ps = __shfl_sync(full, sl_start, sel);
                if (pb > 0) emit(ps, pb, minfin);
                if (lane == sel) { fin = kNever; sl_b = 0; }
            }
            __syncwarp();   // order this stage's stream writes before the next stage's reads
            // the bound is checked between stages, where nothing is half-written
            cand_batches += (unsigned)guard;
            if (p.iter_limit && cand_batches > p.iter_limit) {
                if (lane == 0) atomicCAS(p.status, 0, IL_ERR_ITER_LIMIT);
                over = true;
                break;
            }
        }

        if (lane == 0) {
            if (!over && (int64_t)exits != (p.fork ? p.total_leaving : (int64_t)p.n)) atomicCAS(p.status, 0, IL_ERR_ITER_LIMIT);
        }
    }
    if (lane == 0 && batches) { atomicAdd(&p.counters[1], batches); atomicAdd(&p.counters[2], alg_ops); }
}

cudaError_t launch_des(const DesParams &p, int grid, size_t smem, cudaStream_t stream)
{
    cudaError_t e = cudaFuncSetAttribute(des_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    des_kernel<<<grid, kWarpsPerCta * 32, smem, stream>>>(p);
    return cudaGetLastError();
}

int des_max_ctas_per_sm(size_t smem)
{
    int n = 0;
    if (cudaFuncSetAttribute(des_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, des_kernel, kWarpsPerCta * 32, smem) != cudaSuccess)
        return 0;
    return n;
}

// Dependency-free integer instruction stream: 8 independent chains per thread,
// half multiply-add and half logic/add so that both integer pipes are fed.
// One inner step is 4 multiply-adds + 4 x (xor, add) = 12 instructions.
__global__ void __launch_bounds__(256) int_issue_kernel(unsigned *sink, int iters)
{
    unsigned a0 = threadIdx.x, a1 = a0 + 1, a2 = a0 + 2, a3 = a0 + 3,
             a4 = a0 + 4, a5 = a0 + 5, a6 = a0 + 6, a7 = a0 + 7;
    const unsigned k = blockIdx.x | 1u;
    for (int i = 0; i < iters; i++) {
#pragma unroll
        for (int u = 0; u < 16; u++) {
            a0 = a0 * k + 1u; a1 = a1 * k + 2u; a2 = a2 * k + 3u; a3 = a3 * k + 4u;
            a4 = (a4 ^ k) + 5u; a5 = (a5 ^ k) + 6u; a6 = (a6 ^ k) + 7u; a7 = (a7 ^ k) + 8u;
        }
    }
    const unsigned r = a0 ^ a1 ^ a2 ^ a3 ^ a4 ^ a5 ^ a6 ^ a7;
    if (r == 0x12345678u) sink[0] = r;   // keeps the loop alive
}

cudaError_t launch_int_issue(unsigned *sink, int grid, int iters, cudaStream_t stream)
{
    int_issue_kernel<<<grid, 256, 0, stream>>>(sink, iters);
    return cudaGetLastError();
}

}  // namespace il
