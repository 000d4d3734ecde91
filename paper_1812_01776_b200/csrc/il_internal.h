// Internal declarations shared by the host API and the kernels of the batched
// Estimator.  Nothing here is part of the C ABI.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "il_estimator.h"

// Checked build (-DIL_CHECKED): every index into a stream, ring, slab or bound input that a kernel
// computes is compared with the size of its array first; an index outside is recorded as
// IL_ERR_BOUNDS in the status word and the access is skipped, so that a wrong index shows up as an
// error code and never as a fault.  In the normal build the macro is the constant true.
#ifdef IL_CHECKED
#define IL_IN_RANGE(idx, size, status) \
    ((unsigned long long)(idx) < (unsigned long long)(size) ? true : (atomicCAS((status), 0, IL_ERR_BOUNDS), false))
#else
#define IL_IN_RANGE(idx, size, status) true
#endif

namespace il {

constexpr int kWarpsPerCta = 4;
constexpr int kSelectThreads = 256;

// Everything the simulation kernel needs, passed by value as a kernel parameter.
struct DesParams {
    // bound inputs (device)
    const int64_t *arrival;       // [n]
    const uint8_t *bits;          // [n]
    const int32_t *lat;           // [S][H][Bmax]
    const uint64_t *ptrace;       // [n] packed root stream (arrival << qbits) | index; packed kernel only
    // Lane kernel, pipelines with branch points: when rec_bits > 0 a stream record also carries the
    // query's branch bits, (time << (qbits + rec_bits)) | (bits << qbits) | query, and ptrace_b is the
    // trace in that form, so no stage looks the bits up.  Slab records keep the plain form.
    const uint64_t *ptrace_b;
    int32_t rec_bits;
    int32_t qbits;                // bits of a packed record that hold the query index
    int32_t S, H, Bmax;
    int32_t n;                    // queries
    int32_t n_s[IL_MAX_STAGES];   // queries visiting stage s
    int32_t buf_off[IL_MAX_STAGES];  // element offset of stage s's input stream inside a warp slot
    int8_t  dest_a[IL_MAX_STAGES];   // next stage for branch bit 0 (or unconditional); -1 = leave
    int8_t  dest_b[IL_MAX_STAGES];   // next stage for branch bit 1; -1 = leave
    int8_t  bit[IL_MAX_STAGES];      // branch bit tested after stage s, -1 = none
    // Fan-out (fork != 0): some stage has two children that one query can enter both, so the three
    // arrays above do not describe the routing; these do.  A query goes down every edge whose
    // condition holds; where none holds that copy of it leaves, and the slab keeps per query the
    // record of the copy that left last.
    int32_t fork;
    int8_t  child_a[IL_MAX_STAGES], child_b[IL_MAX_STAGES];   // children of stage s, -1 = none
    int8_t  cbit_a[IL_MAX_STAGES], cbit_b[IL_MAX_STAGES];     // branch bit guarding the edge, -1 = always taken
    uint8_t cval_a[IL_MAX_STAGES], cval_b[IL_MAX_STAGES];     // the edge is taken iff the bit has this value
    int64_t total_leaving;           // copies that leave the pipeline, all stages together (n without fan-out)
    int32_t out_off_a[IL_MAX_STAGES], out_off_b[IL_MAX_STAGES];   // fan-out, separate streams: where stage s writes
                                     // the records for child_a / child_b inside a warp slot
    // Joins (kernel with separate streams only): stage s with join_b[s] >= 0 has two incoming edges.  Its
    // parents write to in_a[s] (edge parent -> s, na[s] records) and in_b[s] (edge join_b[s] -> s, nb[s]
    // records); before the stage is simulated the warp merges them into the stage's arrival stream at
    // buf_off[s], one record per query at the time its last input arrived.
    int8_t  join_b[IL_MAX_STAGES];   // second parent, -1 = none
    int32_t join_in_a[IL_MAX_STAGES], join_in_b[IL_MAX_STAGES];
    int32_t join_na[IL_MAX_STAGES], join_nb[IL_MAX_STAGES];
    int32_t join_tmp_off;            // scratch for the two sorted halves of a merge
    int32_t join_t_off;              // scratch: per query the times of its two inputs, 2 x n_pad elements
    // this launch
    const il_stage_config *configs;  // [n_cand][S], already offset to the chunk
    int64_t n_cand;
    const int32_t *order;         // [n_cand] candidates in the order warps should take them (costliest first)
    int64_t slot_elems;           // stream elements per warp slot
    int64_t *ws_time;             // [slots][slot_elems]
    int32_t *ws_qid;              // [slots][slot_elems]
    int64_t *slab;                // [n_cand][slab_stride] exit latencies
    int64_t slab_stride;          // n rounded up to 32
    unsigned long long *counters; // [0] next candidate, [1] batches dispatched, [2] algorithmic ops
    int *status;                  // first error seen by any warp (0 = none)
    // lane-parallel kernel only (des_lane_kernel.cu)
    uint64_t *lane_ws;            // [warp slots][cpw][lane_elems] inter-stage streams of packed records
    int64_t lane_elems;           // stream records per candidate: every stage's arrival stream but the root's
    int32_t lane_off[IL_MAX_STAGES]; // record offset of stage s's arrival stream inside a candidate's block
    int32_t cpw;                  // candidates per warp, floor(32 / S)
    int32_t lane_slots;           // positions of a lane's batch ring in shared memory: 16 or 32, at least the
                                  // largest replica count among the launch's candidates
    int32_t lane_ctas_per_sm;     // CTAs the host keeps resident per SM (sizes the shared-memory carve-out); 0: unknown
    int32_t lane_ring_log2;       // a stream ring holds 2^this records
    int32_t lane_wrap;            // the rings are shorter than the longest stream: positions wrap
    uint8_t *ovf;                 // [n_cand] set to 1 for a candidate given up on ring overflow (lane_wrap only)
    // lane kernel, feasibility only: set out_feasible to select that instantiation
    uint8_t *out_feasible;        // [n_cand] 1: P99 <= slo_us, 0: not, 2: given up on ring overflow (see ovf)
    int64_t slo_us;               // the objective, clamped by the host to 0 .. 2^(62 - qbits)
    uint32_t miss_allow;          // n - ceil(0.99 n): a candidate with more misses than this is infeasible
    // all simulation kernels
    unsigned long long iter_limit;   // iteration bound of a device loop; 0 = the bound the loop derives itself
    const unsigned long long *n_cand_dev;   // if set, the number of candidates is read from here (device
                                            // memory) instead of n_cand: the list in `order` was built on the device
};

struct SelectParams {
    int64_t *slab;                // [n_cand][slab_stride]: latencies, or packed (finish, query) records
    int64_t slab_stride;
    const int64_t *arrival;       // [n], to turn packed records into latencies
    int32_t qbits;
    int32_t packed;               // slab holds packed records (from a packed-record simulation kernel)
    int *status;                  // checked build: where an index out of range is recorded
    int32_t n;
    int64_t n_cand;
    int64_t slo_us;
    int64_t *out_p99;             // [n_cand], already offset to the chunk
    int64_t *out_miss;
};

// Read-only view of what a handle has bound, for translation units that do not
// see the handle's definition.
struct BoundView {
    DesParams base;        // bound-input part of the kernel parameters
    int kernel;            // SimKernel the handle uses
    int32_t S;
    int64_t n, n_pad, slot_elems;
    size_t smem;
    float span_us;
    int device;
    cudaStream_t stream;
};
void bound_view(const il_estimator *est, BoundView *out);
// Records a failing CUDA call for il_last_cuda_error (thread-local).
void set_last_cuda_error(int cuda_error);

cudaError_t launch_des(const DesParams &p, int grid, size_t smem, cudaStream_t stream);
// staged: the root stage reads the trace through a shared-memory tile ring filled by bulk copies
cudaError_t launch_des_packed(const DesParams &p, bool staged, int grid, size_t smem, cudaStream_t stream);
int des_packed_max_ctas_per_sm(bool staged, size_t smem);
int trace_tile_records();     // the packed trace is padded to a multiple of this many records
// lane-parallel kernel: one lane per (candidate, stage); smem from des_lane_smem
cudaError_t launch_des_lane(const DesParams &p, int grid, size_t smem, cudaStream_t stream);
int des_lane_warps_per_cta();
size_t des_lane_smem(int n_tab, int Bmax, int ring_slots);   // ring_slots: 16 or 32 batch ring positions per lane
int des_lane_max_ctas_per_sm(size_t smem);
enum SimKernel { kSimWide = 0, kSimPacked = 1, kSimPackedStaged = 2, kSimLane = 3 };
inline cudaError_t launch_simulation(const DesParams &p, int kernel, int grid, size_t smem,
                                     cudaStream_t stream)
{
    if (kernel == kSimLane) return launch_des_lane(p, grid, smem, stream);
    if (kernel == kSimWide) return launch_des(p, grid, smem, stream);
    return launch_des_packed(p, kernel == kSimPackedStaged, grid, smem, stream);
}
cudaError_t launch_select(const SelectParams &p, cudaStream_t stream);
cudaError_t launch_scatter_latency(const int64_t *slab_row, const int64_t *arrival, int n, int qbits,
                                   int64_t *out, cudaStream_t stream);

// ---- shared-prefix evaluation (prefix_kernel.cu) ----------------------------------------------
// One stage of the node simulation: node k of the stage reads the stream of node node_parent[k] of
// the parent stage (or the trace) and writes its own streams at k * stride.
struct NodeStageParams {
    const int32_t *lat_stage;     // [H][Bmax] profile of this stage
    const uint8_t *bits;          // [n] branch bits
    const uint64_t *ptrace;       // packed trace (root stage)
    int32_t qbits, H, Bmax;
    int32_t n_queries;            // length of the trace (and of bits)
    int32_t n_in;                 // queries visiting the stage
    int32_t bit;                  // branch bit tested after the stage, -1 = none
    int64_t n_nodes;
    const uint32_t *node_cfg;     // [n_nodes] hw | max batch << 8 | replicas << 16
    const int32_t *node_parent;   // [n_nodes] node of the parent stage
    const uint64_t *in;           // parent stage's streams for this stage, nullptr at the root
    int64_t stride_in;
    uint64_t *out_a, *out_b;      // this stage's streams per side: to a child stage, or the leaving records
    int64_t stride_a, stride_b;
    unsigned long long *work;     // work counter (zero at launch)
    unsigned long long *counters; // the handle's counter block
    int *status;
};
cudaError_t launch_node_stage(const NodeStageParams &p, int grid, cudaStream_t stream);
cudaError_t launch_prefix_stage(const il_stage_config *configs, int64_t n_cand, int S, int s, int H, int Bmax,
                                const int32_t *parent_node, uint64_t *keys, uint32_t cap, int32_t *vals,
                                int32_t *slot_of, int *count, uint32_t *node_cfg, int32_t *node_parent,
                                int32_t *node_of, int *status, cudaStream_t stream);
// Largest latencies of every node of a stage that queries leave after (select_kernel.cu).
struct NodeTopParams {
    uint64_t *records;            // [rows][stride] leaving records (finish << qbits | query); overwritten
    int64_t stride;
    const int32_t *row_of;        // row of node k (nullptr: row k)
    int64_t offset;               // a node's records start this far into its row
    int32_t len;                  // records per node
    const int64_t *arrival;
    int32_t qbits;
    int64_t slo_us;
    int32_t top_len;              // T + 1 entries kept per node, T = queries allowed above the P99
    int64_t *top;                 // [n_nodes][top_len] descending, zero-filled beyond the node's count
    int64_t *miss;                // [n_nodes]
    int64_t n_nodes;
};
cudaError_t launch_node_top(const NodeTopParams &p, cudaStream_t stream);
size_t node_top_smem(int top_len);
struct CombineParams {
    int64_t n_cand;
    const int32_t *node_of;       // [S][n_cand]
    int32_t n_exit;               // stages that queries leave after
    int32_t exit_stage[IL_MAX_STAGES];
    const int64_t *top[IL_MAX_STAGES];
    const int64_t *miss[IL_MAX_STAGES];
    int32_t top_len;
    int64_t allowed;              // T = n - k
    int64_t *out_p99, *out_miss;
};
cudaError_t launch_prefix_combine(const CombineParams &p, cudaStream_t stream);
// Covering candidates (prefix_kernel.cu): per node of a stage the smallest candidate that contains it
// (marked in flags), the list of marked candidates with their positions, and per node its candidate's position.
cudaError_t launch_cover_rep(const int32_t *node_of, int64_t n_cand, int32_t *rep, int64_t n_nodes, uint8_t *flags,
                             cudaStream_t stream);
cudaError_t launch_cover_list(const uint8_t *flags, int64_t n_cand, int32_t *list, int32_t *pos, int *count,
                              cudaStream_t stream);
cudaError_t launch_cover_rows(const int32_t *rep, const int32_t *pos, int64_t n_nodes, int32_t *row, cudaStream_t stream);

// Fills order[0..n_cand) with the chunk's candidate indices, costliest first
// (longest-processing-time-first scheduling over the warps).
struct OrderParams {
    const il_stage_config *configs;  // [n_cand][S]
    int64_t n_cand;
    const int32_t *lat;              // [S][H][Bmax]
    int32_t S, H, Bmax;
    int32_t n_s[IL_MAX_STAGES];
    float span_us;                   // last arrival - first arrival (at least 1)
    int32_t *order;                  // [n_cand] out
};
cudaError_t launch_order(const OrderParams &p, cudaStream_t stream);
cudaError_t launch_max_replicas(const il_stage_config *configs, int64_t count, int *out, cudaStream_t stream);
cudaError_t launch_gather_configs(const il_stage_config *configs, const int32_t *list, int64_t count, int S,
                                  il_stage_config *out, cudaStream_t stream);
cudaError_t launch_feasible_from_p99(const int64_t *p99, const int32_t *list, int64_t count, int64_t slo_us,
                                     uint8_t *out, cudaStream_t stream);
cudaError_t launch_overflow_list(const uint8_t *ovf, int64_t n_cand, int32_t *order, unsigned long long *counters,
                                 cudaStream_t stream);
int des_max_ctas_per_sm(size_t smem);
cudaError_t launch_envelope(const int64_t *d_arrival, int n, const int64_t *h_windows, int n_windows,
                            int *d_out, int num_sms, cudaStream_t stream);
int envelope_max_windows();
cudaError_t launch_int_issue(unsigned *sink, int grid, int iters, cudaStream_t stream);

}  // namespace il
