// Host side of the library: layer-list validation, partition / micro-batch bookkeeping, the memory
// plan, the gradient-flow plan, the stream/event (or captured-graph) pipeline scheduler, and the C ABI.
#include "../../include/hpf.h"
#include "conv_tc.h"
#include "hpf_kernels.h"

#include <algorithm>
#include <chrono>
#include <cstdlib>
#include <cstdio>
#include <cstring>
#include <string>
#include <thread>
#include <vector>

using namespace hpf;

namespace {
thread_local std::string g_last_error;
}

int hpf::api_fail(int status, const char* what)
{
    g_last_error = what ? what : "";
    return status;
}

int hpf::api_cuda_fail(cudaError_t e, const char* where)
{
    char buf[512];
    snprintf(buf, sizeof buf, "%s: %s", where, cudaGetErrorString(e));
    g_last_error = buf;
    return HPF_ERR_CUDA;
}

namespace {

int fail(int status, const char* what) { return hpf::api_fail(status, what); }
int cuda_fail(cudaError_t e, const char* where) { return hpf::api_cuda_fail(e, where); }

#define CU(call)                                                   \
    do {                                                           \
        cudaError_t e__ = (call);                                  \
        if (e__ != cudaSuccess) return cuda_fail(e__, #call);      \
    } while (0)

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

enum Phase { PH_FWD = 0, PH_BWD = 1, PH_AVG = 2, PH_COUNT = 3, PH_FB = 4 };
enum State { ST_CREATED = 0, ST_BOUND = 1, ST_FWD = 2, ST_BWD = 3 };

struct OpInfo {
    hpf_op op;
    int H, W, C;            // output
    int iH, iW, iC;         // input (src0)
    int64_t w_off, w_cnt, b_off, b_cnt;
    int part;
    std::vector<int> consumers;   // ascending, with multiplicity
};

// How the backward of op `op` treats its contribution to one source tensor.
struct GradEdge {
    int accumulate = 0;     // the kernel adds to what the gradient buffer already holds
    int addend = -1;        // tensor whose gradient buffer is added on the fly (a residual ADD's output)
};
struct AccumAction {        // explicit dst (+)= src over gradient buffers, run at op `at`'s place in the sweep
    int at, dst, src, accumulate;
};
struct MessagePlan {        // how the partial error of a boundary tensor is assembled (debug messages)
    int tensor;
    int from_buffer;        // the tensor's own gradient buffer holds contributions of consumers >= cut
    int pending;            // plus this ADD output's gradient (not folded yet), or -1
};

}  // namespace

struct hpf_model {
    std::vector<OpInfo> ops;
    int n_ops = 0, B = 0, M = 0, b = 0, P = 1;
    int inH = 0, inW = 0, inC = 0;
    std::vector<int> cuts;                    // P-1
    std::vector<int> part_lo, part_hi;        // P
    std::vector<std::vector<int>> live;       // per cut
    int64_t G = 0;
    // options
    int opt_graph = 1, opt_conv_path = 0, opt_single = 0, opt_messages = 0, opt_fuse_add = 1, opt_wgrad_passes = 1;
    // gradient-flow plan
    std::vector<int> grad_alias;              // tensor -> ADD op whose gradient buffer it shares, or -1
    std::vector<int> fused_into;              // conv -> residual ADD computed in its epilogue (its own output is not stored), or -1
    std::vector<int> add_done_by;             // ADD -> the conv that computes it, or -1
    std::vector<int> bn_fwd_from;              // BN -> conv whose forward kernel also produces the statistics of the BN (its input), or -1
    std::vector<int> conv_fwd_bn;              // the inverse map
    std::vector<int> bn_into, conv_in_bn;      // BN -> the convolution that applies it to its own input operand (no BN kernel), and the inverse
    std::vector<int> bn_late;                  // BN -> 1: the applying convolution derives the statistics from the per-tile sums itself
    std::vector<int> bn_buf;                   // BN -> which of the stream's two per-tile-sum buffers carries its sums
    std::vector<size_t> bn_part_bytes;         // per partition: size of one per-tile-sum buffer
    int opt_bn_late_floats = 8192;             // largest [tiles][2][C] block of per-tile sums a reading convolution adds itself
    bool opt_pdl = true;       // programmatic dependent launch for this model's kernels
    bool opt_bn_cluster = true; // BN backward of micro-batch sized tensors as one thread-block-cluster launch
    int opt_cell_times = 0;    // record a device timestamp at the start and end of every (partition, micro-batch) cell
    size_t cell_times_off = 0;
    // persistent cell kernels: maximal runs of tensor-core forward convolutions of a partition with nothing but
    // kernel-less ops between them (BN+ReLU applied by the reading convolution, residual adds fused into the producer)
    struct CellRun {
        int part = 0;
        std::vector<int> convs;               // ops of the run, ascending; the kernel is enqueued at convs[0]'s place
        std::vector<size_t> ops_off;          // per micro-batch: device records (conv_tc_cell_op) in the workspace
        unsigned int smem = 0, tmem = 0, smem_budget = 0;
        int ctas = 0;
        bool ready = false;
    };
    int opt_cell = 0;          // CTAs of a persistent forward cell kernel; 0: every convolution is its own launch
    // Stage lanes: a stage keeps up to `lanes` of its micro-batches under way at once, micro-batch m on lane m % lanes; every
    // lane has its own streams and its own scratch, so cells of different lanes share nothing but the parameters.  One
    // lane is the paper's schedule (a stage works through its micro-batches one after the other).
    int opt_wgrad_direct = 1;   // weight gradients read their TMA tiles as MN-major operands (0: the kernel that transposes them)
    int opt_lanes = 1;
    int lanes() const { return opt_lanes < M ? opt_lanes : M; }
    int n_slots() const { return P * lanes(); }
    int slot_of(int p, int m) const { return p * lanes() + m % lanes(); }
    int opt_pdl_late_from = 8;   // forward cells that run while at least this many cells are under way trigger their successors late
    std::vector<CellRun> cell_runs;
    std::vector<int> cell_of_op;              // conv -> run, or -1
    std::vector<size_t> cell_bar_off;         // per partition: the grid barrier's two words (zeroed at bind)
    int opt_fuse_bn = 3;       // bit 0: BN statistics in the producing convolution's write-out, bit 1: BN+ReLU applied by the reading convolution
    std::vector<GradEdge> edge0;              // per op: contribution to src0
    std::vector<AccumAction> accums;
    std::vector<std::vector<MessagePlan>> msg_plan;   // per cut
    // memory plan (byte offsets into the workspace)
    std::vector<size_t> act_off, grad_off, stats_off;   // [m * n_ops + op]
    std::vector<size_t> bn_scratch_off, conv_scratch_off;   // per stream slot (partition, lane)
    std::vector<size_t> splitk_off, splitk_bytes;            // per stream: tickets + partial tiles of K-split convolutions (zeroed at bind)
    // the backward kernels of a partition have scratch of their own: in the one-graph schedule (hpf_forward_backward) a
    // partition's backward cells run while its forward cells of later micro-batches are still under way
    std::vector<size_t> bn_scratch_bwd_off, splitk_bwd_off;
    std::vector<size_t> pooled_off, persample_off;      // per m
    std::vector<std::vector<size_t>> fmsg_off, bmsg_off;  // [cut][i*M + m]
    size_t loss_slots_off = 0, loss_avg_off = 0, wprep_off = 0, stage_x_off = 0, stage_lab_off = 0, status_off = 0;
    std::vector<size_t> prep_table_off;       // per partition: WeightPrepEntry[] in the workspace
    std::vector<std::vector<WeightPrepEntry>> prep_table;   // host copies
    size_t zero_lo = 0, zero_hi = 0;          // region that must start zeroed (tickets, status)
    size_t ws_bytes = 0;
    bool planned = false;
    // bound resources
    float *params = nullptr, *gslots = nullptr, *gavg = nullptr;
    char* ws = nullptr;
    std::vector<cudaStream_t> streams;
    std::vector<cudaEvent_t> ev_fwd, ev_bwd;  // [cut * M + m]
    std::vector<cudaEvent_t> ev_join;         // per stream slot
    std::vector<cudaEvent_t> ev_prep;         // per partition: prepared weights ready (the other lanes wait for lane 0)
    std::vector<cudaStream_t> side;           // per partition: weight-gradient stream (empty: none)
    std::vector<cudaStream_t> bwd_streams;    // per partition: the backward cells' stream in the one-graph schedule (empty: none)
    std::vector<cudaEvent_t> ev_fdone, ev_bjoin;   // forward (P-1, m) done; backward stream p done
    std::vector<cudaEvent_t> ev_side, ev_side_join;   // per partition: gradient ready -> side stream; side stream done
    cudaEvent_t ev_fork = nullptr, ev_sync = nullptr;
    // tensor-core plans [m * n_ops + op] per pass
    std::vector<ConvTcPlan> tc_plan[3];
    std::vector<char> use_tc[3];              // per op
    // graphs
    struct FwdGraph { const float* x = nullptr; const int32_t* labels = nullptr; cudaGraphExec_t exec = nullptr; int64_t nodes = 0; };
    FwdGraph fwd_graph[2];
    int fwd_graph_next = 0;
    FwdGraph fb_graph[2];                     // forward + backward as one graph (hpf_forward_backward)
    int fb_graph_next = 0;
    cudaGraphExec_t graph[PH_COUNT] = {nullptr, nullptr, nullptr};
    int64_t graph_nodes[PH_COUNT] = {0, 0, 0};
    const float* cur_x = nullptr;
    const int32_t* cur_labels = nullptr;
    const int32_t* bwd_labels = nullptr;
    const float* bwd_x = nullptr;
    int state = ST_CREATED;
    int64_t launches = 0;

    float* act(int op, int m) const { return reinterpret_cast<float*>(ws + act_off[(size_t)m * n_ops + op]); }
    float* grad(int op, int m) const { return reinterpret_cast<float*>(ws + grad_off[(size_t)m * n_ops + op]); }
    float* stats(int op, int m) const { return reinterpret_cast<float*>(ws + stats_off[(size_t)m * n_ops + op]); }
    float* bn_partials(int bn, int m) const
    {
        const int p = ops[bn].part;
        return reinterpret_cast<float*>(ws + bn_scratch_off[slot_of(p, m)] + 256 + (size_t)bn_buf[bn] * bn_part_bytes[p]);
    }
    unsigned long long* cell_time_slot(int phase, int p, int m) const
    {
        return reinterpret_cast<unsigned long long*>(ws + cell_times_off) + 2 * (((size_t)(phase == PH_BWD) * P + p) * M + m);
    }
    int64_t numel(int op) const { const OpInfo& o = ops[op]; return (int64_t)b * o.H * o.W * o.C; }
    cudaStream_t stream_of(int p, int m = 0) const { return opt_single ? streams[0] : streams[slot_of(p, m)]; }
    DeviceStatus* status() const { return reinterpret_cast<DeviceStatus*>(ws + status_off); }
};

namespace {

// ------------------------------------------------------------------------------------------------
// validation + bookkeeping (Section 5.1)
// ------------------------------------------------------------------------------------------------
int build_ops(hpf_model* mdl, const hpf_op* ops, int n_ops)
{
    mdl->ops.resize(n_ops);
    int64_t at = 0;
    for (int i = 0; i < n_ops; ++i) {
        OpInfo& o = mdl->ops[i];
        o.op = ops[i];
        const hpf_op& q = ops[i];
        if (q.src0 < -1 || q.src0 >= i) return fail(HPF_ERR_INVALID, "op source must be an earlier op or -1");
        if (q.src0 >= 0 && ops[q.src0].kind == HPF_OP_HEAD) return fail(HPF_ERR_INVALID, "the head has no output tensor to read");
        if (q.src0 < 0) { o.iH = mdl->inH; o.iW = mdl->inW; o.iC = mdl->inC; }
        else { o.iH = mdl->ops[q.src0].H; o.iW = mdl->ops[q.src0].W; o.iC = mdl->ops[q.src0].C; }
        int64_t wc = 0, bc = 0;
        switch (q.kind) {
        case HPF_OP_CONV:
        case HPF_OP_MAXPOOL:
            if (q.c_in != o.iC || q.ksize < 1 || q.stride < 1 || q.pad < 0 || q.c_out < 1)
                return fail(HPF_ERR_INVALID, "bad convolution / pooling geometry");
            if (q.kind == HPF_OP_MAXPOOL && q.c_out != o.iC) return fail(HPF_ERR_INVALID, "pooling keeps the channel count");
            if (o.iH + 2 * q.pad < q.ksize || o.iW + 2 * q.pad < q.ksize) return fail(HPF_ERR_INVALID, "window larger than the padded input");
            if (q.pad >= q.ksize) return fail(HPF_ERR_UNSUPPORTED, "padding must be smaller than the window");
            o.H = (o.iH + 2 * q.pad - q.ksize) / q.stride + 1;
            o.W = (o.iW + 2 * q.pad - q.ksize) / q.stride + 1;
            o.C = q.c_out;
            if (q.kind == HPF_OP_CONV) wc = (int64_t)q.c_out * q.ksize * q.ksize * q.c_in;
            break;
        case HPF_OP_RELU:
            if (q.c_in != o.iC || q.c_out != o.iC) return fail(HPF_ERR_INVALID, "RELU channel count mismatch");
            if (q.src0 < 0) return fail(HPF_ERR_UNSUPPORTED, "RELU directly on the network input");
            o.H = o.iH; o.W = o.iW; o.C = o.iC;
            break;
        case HPF_OP_BNRELU:
        case HPF_OP_BN:
            if (q.c_in != o.iC || q.c_out != o.iC) return fail(HPF_ERR_INVALID, "BN channel count mismatch");
            if (o.iC % 4) return fail(HPF_ERR_UNSUPPORTED, "BN channel count must be a multiple of 4");
            if (q.src0 < 0) return fail(HPF_ERR_UNSUPPORTED, "BN directly on the network input");
            if (!(q.eps > 0.f)) return fail(HPF_ERR_INVALID, "BN eps must be positive");
            o.H = o.iH; o.W = o.iW; o.C = o.iC;
            wc = bc = o.iC;
            break;
        case HPF_OP_ADD: {
            if (q.src1 < 0 || q.src1 >= i || q.src0 < 0) return fail(HPF_ERR_INVALID, "ADD needs two earlier ops as sources");
            if (ops[q.src1].kind == HPF_OP_HEAD) return fail(HPF_ERR_INVALID, "the head has no output tensor to read");
            const OpInfo& t = mdl->ops[q.src1];
            if (t.H != o.iH || t.W != o.iW || t.C != o.iC || q.c_out != o.iC) return fail(HPF_ERR_INVALID, "ADD shape mismatch");
            o.H = o.iH; o.W = o.iW; o.C = o.iC;
            break;
        }
        case HPF_OP_HEAD:
            if (i != n_ops - 1) return fail(HPF_ERR_INVALID, "the head must be the last op");
            if (q.c_in != o.iC || q.c_out < 1 || q.src0 < 0) return fail(HPF_ERR_INVALID, "bad head");
            o.H = 1; o.W = 1; o.C = q.c_out;
            wc = (int64_t)q.c_out * q.c_in; bc = q.c_out;
            break;
        default:
            return fail(HPF_ERR_INVALID, "unknown op kind");
        }
        if (q.kind != HPF_OP_ADD && q.src1 != -1) return fail(HPF_ERR_INVALID, "src1 is only for ADD");
        o.w_off = at; o.w_cnt = wc; at += wc;
        o.b_off = at; o.b_cnt = bc; at += bc;
        if (q.src0 >= 0) mdl->ops[q.src0].consumers.push_back(i);
        if (q.kind == HPF_OP_ADD) mdl->ops[q.src1].consumers.push_back(i);
    }
    if (ops[n_ops - 1].kind != HPF_OP_HEAD) return fail(HPF_ERR_INVALID, "the last op must be the head");
    for (int i = 0; i < n_ops - 1; ++i)
        if (mdl->ops[i].consumers.empty()) return fail(HPF_ERR_INVALID, "an op's output is never read");
    mdl->G = at;
    return HPF_OK;
}

int build_partitions(hpf_model* mdl, const int32_t* cuts, int n_cuts)
{
    const int n = mdl->n_ops;
    if (n_cuts < 0 || n_cuts > n - 1) return fail(HPF_ERR_INVALID, "more partitions than ops");
    if (n_cuts > 0 && !cuts) return fail(HPF_ERR_INVALID, "null cut list");
    for (int j = 0; j < n_cuts; ++j) {
        if (cuts[j] < 1 || cuts[j] > n - 1) return fail(HPF_ERR_INVALID, "cut out of range");
        if (j && cuts[j] <= cuts[j - 1]) return fail(HPF_ERR_INVALID, "cuts must be strictly increasing");
    }
    mdl->cuts.assign(cuts, cuts + n_cuts);
    mdl->P = n_cuts + 1;
    mdl->part_lo.resize(mdl->P); mdl->part_hi.resize(mdl->P);
    for (int p = 0; p < mdl->P; ++p) {
        mdl->part_lo[p] = p == 0 ? 0 : cuts[p - 1];
        mdl->part_hi[p] = p == mdl->P - 1 ? n : cuts[p];
        for (int i = mdl->part_lo[p]; i < mdl->part_hi[p]; ++i) mdl->ops[i].part = p;
    }
    // only the first partition may read the network input
    for (int i = mdl->part_hi[0]; i < n; ++i)
        if (mdl->ops[i].op.src0 < 0) return fail(HPF_ERR_INVALID, "the network input is read beyond the first partition");
    // live sets (Section 5.3: what crosses each cut)
    mdl->live.assign(n_cuts, {});
    for (int j = 0; j < n_cuts; ++j)
        for (int t = 0; t < cuts[j]; ++t)
            if (!mdl->ops[t].consumers.empty() && mdl->ops[t].consumers.back() >= cuts[j]) mdl->live[j].push_back(t);
    return HPF_OK;
}

// Gradient flow: a tensor with several consumers sums their contributions in descending consumer
// order (the order of the reverse sweep).  A residual ADD contributes its own output gradient
// unchanged, so it costs no kernel: either the source simply shares the ADD's gradient buffer
// (sole consumer), or the next consumer's kernel adds it on the fly.
int build_grad_plan(hpf_model* mdl)
{
    const int n = mdl->n_ops;
    mdl->grad_alias.assign(n, -1);
    mdl->edge0.assign(n, GradEdge());
    mdl->accums.clear();
    for (int t = 0; t < n - 1; ++t) {
        const std::vector<int>& cs = mdl->ops[t].consumers;
        if (cs.size() == 1 && mdl->ops[cs[0]].op.kind == HPF_OP_ADD) mdl->grad_alias[t] = cs[0];
    }
    std::vector<char> written(n, 0);
    std::vector<int> pending(n, -1);
    for (int i = n - 1; i >= 0; --i) {
        const hpf_op& q = mdl->ops[i].op;
        const int srcs[2] = {q.src0, q.kind == HPF_OP_ADD ? q.src1 : -1};
        for (int k = 0; k < 2; ++k) {
            const int t = srcs[k];
            if (t < 0) continue;
            if (q.kind == HPF_OP_ADD) {
                if (mdl->grad_alias[t] == i) continue;
                bool lower_kernel = false;
                for (int c : mdl->ops[t].consumers)
                    if (c < i && mdl->ops[c].op.kind != HPF_OP_ADD && mdl->ops[c].op.kind != HPF_OP_HEAD &&
                        mdl->ops[c].op.kind != HPF_OP_MAXPOOL) lower_kernel = true;
                if (lower_kernel && pending[t] < 0) { pending[t] = i; continue; }
                mdl->accums.push_back(AccumAction{i, t, i, written[t]});
                written[t] = 1;
            } else {
                if (q.kind == HPF_OP_HEAD || q.kind == HPF_OP_MAXPOOL) {
                    if (pending[t] >= 0) {      // these kernels take no addend: fold it first
                        mdl->accums.push_back(AccumAction{i, t, pending[t], written[t]});
                        written[t] = 1; pending[t] = -1;
                    }
                    if (q.kind == HPF_OP_HEAD && written[t]) return fail(HPF_ERR_UNSUPPORTED, "the head's input has a later consumer");
                }
                mdl->edge0[i].accumulate = written[t];
                mdl->edge0[i].addend = pending[t];
                written[t] = 1; pending[t] = -1;
            }
        }
    }
    // partial-error assembly per cut (for the optional message copies)
    mdl->msg_plan.assign(mdl->cuts.size(), {});
    for (size_t j = 0; j < mdl->cuts.size(); ++j) {
        const int cut = mdl->cuts[j];
        for (int t : mdl->live[j]) {
            MessagePlan mp{t, 0, -1};
            if (mdl->grad_alias[t] >= 0) { mp.from_buffer = 1; mdl->msg_plan[j].push_back(mp); continue; }
            // replay the plan for consumers >= cut
            int pend = -1;
            std::vector<int> cs(mdl->ops[t].consumers.rbegin(), mdl->ops[t].consumers.rend());
            for (int c : cs) {
                if (c < cut) break;
                const hpf_op& q = mdl->ops[c].op;
                if (q.kind == HPF_OP_ADD) {
                    bool explicit_acc = false;
                    for (const AccumAction& a : mdl->accums) if (a.at == c && a.dst == t && a.src == c) explicit_acc = true;
                    if (explicit_acc) mp.from_buffer = 1; else pend = c;
                } else {
                    mp.from_buffer = 1; pend = -1;   // the kernel folded any pending addend
                }
            }
            mp.pending = pend;
            mdl->msg_plan[j].push_back(mp);
        }
    }
    return HPF_OK;
}

// Residual ADD fused into the epilogue of the later of its two producers when that producer is a
// convolution read by nothing else and sits in the same partition: the sum is written straight into the
// ADD's output tensor and the convolution's own output is never stored.
void build_fusion_plan(hpf_model* mdl)
{
    const int n = mdl->n_ops;
    mdl->fused_into.assign(n, -1);
    mdl->add_done_by.assign(n, -1);
    if (!mdl->opt_fuse_add) return;
    for (int i = 0; i < n; ++i) {
        const hpf_op& q = mdl->ops[i].op;
        if (q.kind != HPF_OP_ADD || q.src0 == q.src1) continue;
        const int late = q.src0 > q.src1 ? q.src0 : q.src1;
        const OpInfo& c = mdl->ops[late];
        if (c.op.kind != HPF_OP_CONV || c.consumers.size() != 1 || c.part != mdl->ops[i].part) continue;
        if (mdl->opt_messages) continue;      // message copies want every tensor materialised
        mdl->fused_into[late] = i;
        mdl->add_done_by[i] = late;
    }
}

ConvShape conv_shape_of(const hpf_model* mdl, int i);
bool op_uses_tc(const hpf_model* mdl, int i, int pass);

ConvShape conv_shape_of(const hpf_model* mdl, int i)
{
    const OpInfo& o = mdl->ops[i];
    return make_conv_shape(mdl->b, o.iH, o.iW, o.iC, o.op.c_out, o.op.ksize, o.op.stride, o.op.pad);
}

// Which convolutions run on the tensor cores, and which BN work rides inside them: the statistics of a BN in the
// forward kernel that produces its input (only when producer and BN run back to back on the same stream: same
// partition, nothing but a fused residual add between them, so that the per-stream scratch can carry the per-tile
// sums), and the BN+ReLU itself on the operand path of the convolution that reads it.
void build_kernel_plan(hpf_model* mdl)
{
    const int n = mdl->n_ops;
    for (int pass = 0; pass < 3; ++pass) {
        mdl->use_tc[pass].assign(n, 0);
        for (int i = 0; i < n; ++i) mdl->use_tc[pass][i] = op_uses_tc(mdl, i, pass) ? 1 : 0;
    }
    mdl->bn_fwd_from.assign(n, -1);
    mdl->conv_fwd_bn.assign(n, -1);
    mdl->bn_into.assign(n, -1); mdl->conv_in_bn.assign(n, -1); mdl->bn_late.assign(n, 0); mdl->bn_buf.assign(n, 0);
    std::vector<int> n_fused(mdl->P, 0);
    if (!mdl->opt_fuse_bn) return;
    for (int j = 0; j < n; ++j) {
        const OpInfo& bn = mdl->ops[j];
        if (bn.op.kind != HPF_OP_BNRELU || bn.C > 2048) continue;
        // forward: the kernel that writes the BN's input
        int t = bn.op.src0, prod = -1;
        if (mdl->ops[t].op.kind == HPF_OP_CONV && mdl->fused_into[t] < 0) prod = t;
        else if (mdl->ops[t].op.kind == HPF_OP_ADD && mdl->add_done_by[t] >= 0) prod = mdl->add_done_by[t];
        if ((mdl->opt_fuse_bn & 1) && prod >= 0 && mdl->use_tc[PASS_FWD][prod] && mdl->ops[prod].part == bn.part && mdl->conv_fwd_bn[prod] < 0 &&
            conv_tc_can_fuse_bn(conv_shape_of(mdl, prod), PASS_FWD)) {
            bool adjacent = true;
            for (int k = prod + 1; k < j; ++k)
                if (!(mdl->ops[k].op.kind == HPF_OP_ADD && mdl->add_done_by[k] >= 0)) adjacent = false;
            if (adjacent) {
                mdl->bn_fwd_from[j] = prod; mdl->conv_fwd_bn[prod] = j;
                // A convolution that reads BN j's sums may still be reading them while its own write-out already
                // produces the next BN's: successive fused BNs of a stream alternate between two buffers.
                mdl->bn_buf[j] = n_fused[bn.part]++ & 1;
            }
        }
        // the BN+ReLU itself: applied by its only reader, the next op, a stride-1 tensor-core convolution
        if ((mdl->opt_fuse_bn & 2) && mdl->bn_fwd_from[j] >= 0 && bn.consumers.size() == 1 && bn.consumers[0] == j + 1) {
            const int i = j + 1;
            if (mdl->ops[i].op.kind == HPF_OP_CONV && mdl->ops[i].op.src0 == j && mdl->use_tc[PASS_FWD][i] &&
                mdl->ops[i].part == bn.part && conv_tc_can_fuse_bn_input(conv_shape_of(mdl, i))) {
                mdl->bn_into[j] = i; mdl->conv_in_bn[i] = j;
                // Few per-tile sums: the reading convolution adds them under the latency of its first copy and the
                // producer ends without a ticket.  Many: the producer's last CTA adds them once.
                const long long floats = (long long)conv_tc_tiles(conv_shape_of(mdl, mdl->bn_fwd_from[j]), PASS_FWD) * 2 * bn.C;
                mdl->bn_late[j] = floats <= mdl->opt_bn_late_floats ? 1 : 0;
            }
        }
    }
}

// Which forward convolutions share a persistent cell kernel: consecutive tensor-core convolutions of one partition
// between which the op list holds only ops that launch nothing.
void build_cell_runs(hpf_model* mdl)
{
    const int n = mdl->n_ops;
    mdl->cell_runs.clear();
    mdl->cell_of_op.assign(n, -1);
    if (mdl->opt_cell <= 0) return;
    for (int p = 0; p < mdl->P; ++p) {
        hpf_model::CellRun run;
        run.part = p;
        auto close = [&]() {
            if (run.convs.size() >= 2) {
                for (int i : run.convs) mdl->cell_of_op[i] = (int)mdl->cell_runs.size();
                mdl->cell_runs.push_back(run);
            }
            run.convs.clear();
        };
        for (int i = mdl->part_lo[p]; i < mdl->part_hi[p]; ++i) {
            const int kind = mdl->ops[i].op.kind;
            if (kind == HPF_OP_CONV && mdl->use_tc[PASS_FWD][i]) run.convs.push_back(i);
            else if (kind == HPF_OP_BNRELU && mdl->bn_into[i] >= 0) continue;
            else if (kind == HPF_OP_ADD && mdl->add_done_by[i] >= 0) continue;
            else close();
        }
        close();
    }
}

// ------------------------------------------------------------------------------------------------
// memory plan
// ------------------------------------------------------------------------------------------------
void build_memory_plan(hpf_model* mdl)
{
    build_fusion_plan(mdl);
    build_kernel_plan(mdl);
    const int n = mdl->n_ops, M = mdl->M, P = mdl->P;
    size_t at = 0;
    auto take = [&](size_t bytes) { size_t o = at; at = align_up(at + bytes, 256); return o; };
    // region that must start as zeros: status word and BN tickets (with their partials)
    mdl->zero_lo = at;
    mdl->status_off = take(sizeof(DeviceStatus));
    const int L = mdl->lanes(), S = P * L;
    mdl->bn_scratch_off.assign(S, 0);
    mdl->conv_scratch_off.assign(S, 0);
    mdl->bn_part_bytes.assign(P, 0);
    for (int p = 0; p < P; ++p) {
        size_t bn = 256, part = 0;
        for (int i = mdl->part_lo[p]; i < mdl->part_hi[p]; ++i)
            if (mdl->ops[i].op.kind == HPF_OP_BNRELU || mdl->ops[i].op.kind == HPF_OP_BN) {
                const OpInfo& o = mdl->ops[i];
                size_t need = bn_scratch_bytes((int64_t)mdl->b * o.H * o.W, o.C);
                if (need > bn) bn = need;
                const int from = mdl->bn_fwd_from[i];
                if (from >= 0) {
                    need = align_up((size_t)conv_tc_tiles(conv_shape_of(mdl, from), PASS_FWD) * 2 * o.C * sizeof(float), 256);
                    if (need > part) part = need;
                }
            }
        mdl->bn_part_bytes[p] = part;
        if (256 + 2 * part > bn) bn = 256 + 2 * part;
        for (int l = 0; l < L; ++l) mdl->bn_scratch_off[p * L + l] = take(bn);
    }
    mdl->splitk_off.assign(S, 0); mdl->splitk_bytes.assign(P, 0);
    for (int p = 0; p < P; ++p) {
        size_t need = 0;
        if (mdl->opt_conv_path != 1)
            for (int i = mdl->part_lo[p]; i < mdl->part_hi[p]; ++i)
                if (mdl->ops[i].op.kind == HPF_OP_CONV) {
                    const ConvShape s = conv_shape_of(mdl, i);
                    need = std::max(need, std::max(conv_tc_splitk_bytes(s, PASS_FWD, 3), conv_tc_splitk_bytes(s, PASS_DGRAD, 3)));
                }
        mdl->splitk_bytes[p] = need;
        for (int l = 0; l < L; ++l) mdl->splitk_off[p * L + l] = take(need ? need : 16);
    }
    mdl->bn_scratch_bwd_off.assign(S, 0); mdl->splitk_bwd_off.assign(S, 0);
    for (int p = 0; p < P; ++p) {
        size_t bn = 256;
        for (int i = mdl->part_lo[p]; i < mdl->part_hi[p]; ++i)
            if (mdl->ops[i].op.kind == HPF_OP_BNRELU || mdl->ops[i].op.kind == HPF_OP_BN)
                bn = std::max(bn, bn_scratch_bytes((int64_t)mdl->b * mdl->ops[i].H * mdl->ops[i].W, mdl->ops[i].C));
        for (int l = 0; l < L; ++l) {
            mdl->bn_scratch_bwd_off[p * L + l] = take(bn);
            mdl->splitk_bwd_off[p * L + l] = take(mdl->splitk_bytes[p] ? mdl->splitk_bytes[p] : 16);
        }
    }
    mdl->cell_bar_off.assign(S, 0);
    for (int k = 0; k < S; ++k) mdl->cell_bar_off[k] = take(16);
    mdl->zero_hi = at;
    build_cell_runs(mdl);
    for (auto& run : mdl->cell_runs) {
        run.ops_off.assign(M, 0);
        for (int m = 0; m < M; ++m) run.ops_off[m] = take(conv_tc_cell_op_bytes() * run.convs.size());
    }
    for (int p = 0; p < P; ++p) {
        size_t cv = 256;
        for (int i = mdl->part_lo[p]; i < mdl->part_hi[p]; ++i)
            if (mdl->ops[i].op.kind == HPF_OP_CONV) {
                const ConvShape s = conv_shape_of(mdl, i);
                size_t need = conv_simt_scratch_bytes(s);
                size_t need2 = conv_tc_scratch_bytes(s);
                if (need2 > need) need = need2;
                if (need > cv) cv = need;
            }
        for (int l = 0; l < L; ++l) mdl->conv_scratch_off[p * L + l] = take(cv);
    }
    mdl->cell_times_off = take(sizeof(unsigned long long) * 2 * 2 * (size_t)P * M);
    mdl->loss_slots_off = take(sizeof(float) * M);
    mdl->loss_avg_off = take(sizeof(float));
    mdl->wprep_off = take(sizeof(float) * 4 * (size_t)((mdl->G + 3) / 4 * 4));   // w_hi | w_lo | wt_hi | wt_lo, parameter offsets
    mdl->prep_table_off.assign(P, 0);
    for (int p = 0; p < P; ++p) mdl->prep_table_off[p] = take(sizeof(WeightPrepEntry) * (size_t)(mdl->part_hi[p] - mdl->part_lo[p] + 1));
    mdl->stage_x_off = take(sizeof(float) * (size_t)mdl->B * mdl->inH * mdl->inW * mdl->inC);
    mdl->stage_lab_off = take(sizeof(int32_t) * (size_t)mdl->B);
    const int headC = mdl->ops[n - 1].op.c_in;
    mdl->pooled_off.resize(M); mdl->persample_off.resize(M);
    for (int m = 0; m < M; ++m) {
        mdl->pooled_off[m] = take(sizeof(float) * (size_t)mdl->b * headC);
        mdl->persample_off[m] = take(sizeof(float) * (size_t)mdl->b);
    }
    mdl->act_off.assign((size_t)n * M, 0); mdl->grad_off.assign((size_t)n * M, 0); mdl->stats_off.assign((size_t)n * M, 0);
    for (int m = 0; m < M; ++m) {
        for (int i = n - 1; i >= 0; --i) {
            const int f = mdl->fused_into[i];
            if (f >= 0) mdl->act_off[(size_t)m * n + i] = mdl->act_off[(size_t)m * n + f];   // f > i: already placed
            else mdl->act_off[(size_t)m * n + i] = take(sizeof(float) * (size_t)mdl->numel(i));
        }
        for (int i = n - 1; i >= 0; --i) {
            const int a = mdl->grad_alias[i];
            if (a >= 0) mdl->grad_off[(size_t)m * n + i] = mdl->grad_off[(size_t)m * n + a];   // a > i: already placed
            else mdl->grad_off[(size_t)m * n + i] = take(sizeof(float) * (size_t)mdl->numel(i));
        }
        for (int i = 0; i < n; ++i)
            if (mdl->ops[i].op.kind == HPF_OP_BNRELU || mdl->ops[i].op.kind == HPF_OP_BN)
                mdl->stats_off[(size_t)m * n + i] = take(sizeof(float) * 2 * (size_t)mdl->ops[i].C);
    }
    mdl->fmsg_off.assign(mdl->cuts.size(), {}); mdl->bmsg_off.assign(mdl->cuts.size(), {});
    if (mdl->opt_messages)
        for (size_t j = 0; j < mdl->cuts.size(); ++j) {
            mdl->fmsg_off[j].resize(mdl->live[j].size() * M); mdl->bmsg_off[j].resize(mdl->live[j].size() * M);
            for (size_t k = 0; k < mdl->live[j].size(); ++k)
                for (int m = 0; m < M; ++m) {
                    mdl->fmsg_off[j][k * M + m] = take(sizeof(float) * (size_t)mdl->numel(mdl->live[j][k]));
                    mdl->bmsg_off[j][k * M + m] = take(sizeof(float) * (size_t)mdl->numel(mdl->live[j][k]));
                }
        }
    mdl->ws_bytes = at;
    mdl->planned = true;
}

bool op_uses_tc(const hpf_model* mdl, int i, int pass)
{
    if (mdl->opt_conv_path == 1) return false;
    if (mdl->ops[i].op.kind != HPF_OP_CONV) return false;
    if (mdl->ops[i].op.src0 < 0) return false;          // the network input pointer is not known at bind time
    if (mdl->ops[i].w_off % 4) return false;            // the weight tensor map needs a 16-byte aligned base
    // a strided data gradient zero-fills between its samples, so it cannot also add to what is there
    if (pass == PASS_DGRAD && mdl->ops[i].op.stride > 1 && (mdl->edge0[i].accumulate || mdl->edge0[i].addend >= 0)) return false;
    return conv_tc_supported(conv_shape_of(mdl, i), pass);
}

// ------------------------------------------------------------------------------------------------
// enqueue: the pipeline (Section 5.3)
// ------------------------------------------------------------------------------------------------
const float* src_act(const hpf_model* mdl, int src, int m)
{
    if (src < 0) return mdl->cur_x + (int64_t)m * mdl->b * mdl->inH * mdl->inW * mdl->inC;
    return mdl->act(src, m);
}

// sl: the stream slot (partition, lane) whose scratch and side stream the op uses
int forward_op(hpf_model* mdl, int i, int m, cudaStream_t st, int sl)
{
    const OpInfo& o = mdl->ops[i];
    const hpf_op& q = o.op;
    const float* in0 = src_act(mdl, q.src0, m);
    float* out = mdl->act(i, m);
    switch (q.kind) {
    case HPF_OP_CONV: {
        // with a fused residual ADD, `out` is the ADD's output tensor and the other addend rides in the epilogue
        const float* residual = nullptr;
        if (mdl->fused_into[i] >= 0) {
            const hpf_op& a = mdl->ops[mdl->fused_into[i]].op;
            residual = mdl->act(a.src0 == i ? a.src1 : a.src0, m);
        }
        if (mdl->cell_of_op[i] >= 0 && mdl->cell_runs[mdl->cell_of_op[i]].ready) {
            // the whole run of convolutions is one resident grid, enqueued where its first convolution stands
            const hpf_model::CellRun& run = mdl->cell_runs[mdl->cell_of_op[i]];
            if (run.convs[0] == i)
                CU(conv_tc_cell_launch(mdl->ws + run.ops_off[m], (int)run.convs.size(), run.ctas, run.smem, run.tmem,
                                       reinterpret_cast<unsigned int*>(mdl->ws + mdl->cell_bar_off[sl]), mdl->status(), st, &mdl->launches));
        } else if (mdl->use_tc[PASS_FWD][i]) {
            CU(conv_tc_launch(&mdl->tc_plan[PASS_FWD][(size_t)m * mdl->n_ops + i], mdl->status(), st, &mdl->launches));
        } else {
            CU(conv_fwd_simt(in0, mdl->params + o.w_off, out, residual, conv_shape_of(mdl, i), st, &mdl->launches));
        }
        break;
    }
    case HPF_OP_BNRELU:
        if (mdl->bn_into[i] >= 0) break;   // the convolution that reads this BN applies it (and stores `out` and the statistics)
        if (mdl->bn_fwd_from[i] >= 0)      // the producing convolution left mean and 1/sigma
            CU(bnrelu_fwd_apply(in0, mdl->params + o.w_off, mdl->params + o.b_off, mdl->stats(i, m), out,
                                (int64_t)mdl->b * o.H * o.W, o.C, st, &mdl->launches));
        else
            CU(bnrelu_fwd(in0, mdl->params + o.w_off, mdl->params + o.b_off, q.eps, out, mdl->stats(i, m),
                          (int64_t)mdl->b * o.H * o.W, o.C, mdl->ws + mdl->bn_scratch_off[sl], st, &mdl->launches));
        break;
    case HPF_OP_BN:                        // batch normalisation without the activation
        CU(bnrelu_fwd(in0, mdl->params + o.w_off, mdl->params + o.b_off, q.eps, out, mdl->stats(i, m),
                      (int64_t)mdl->b * o.H * o.W, o.C, mdl->ws + mdl->bn_scratch_off[sl], st, &mdl->launches, false));
        break;
    case HPF_OP_RELU:
        CU(relu_fwd(in0, out, mdl->numel(i), st, &mdl->launches));
        break;
    case HPF_OP_ADD:
        if (mdl->add_done_by[i] < 0) CU(add_fwd(in0, mdl->act(q.src1, m), out, mdl->numel(i), st, &mdl->launches));
        break;
    case HPF_OP_MAXPOOL:
        CU(maxpool_fwd(in0, out, conv_shape_of(mdl, i), st, &mdl->launches));
        break;
    case HPF_OP_HEAD:
        CU(head_fwd(in0, mdl->params + o.w_off, mdl->params + o.b_off, mdl->cur_labels + (int64_t)m * mdl->b, out,
                    reinterpret_cast<float*>(mdl->ws + mdl->pooled_off[m]),
                    reinterpret_cast<float*>(mdl->ws + mdl->persample_off[m]),
                    reinterpret_cast<float*>(mdl->ws + mdl->loss_slots_off) + m, mdl->b, o.iH * o.iW, o.iC, q.c_out, st,
                    &mdl->launches));
        break;
    }
    return HPF_OK;
}

int backward_op(hpf_model* mdl, int i, int m, cudaStream_t st, int sl)
{
    const OpInfo& o = mdl->ops[i];
    const hpf_op& q = o.op;
    const GradEdge& e = mdl->edge0[i];
    // explicit accumulations scheduled at this op
    for (const AccumAction& a : mdl->accums)
        if (a.at == i) CU(grad_accumulate(mdl->grad(a.dst, m), mdl->grad(a.src, m), mdl->numel(a.dst), a.accumulate != 0, st, &mdl->launches));
    const float* in0 = src_act(mdl, q.src0, m);
    float* dout = mdl->grad(i, m);
    float* slot = mdl->gslots + (int64_t)m * mdl->G;
    const float* addend = e.addend >= 0 ? mdl->grad(e.addend, m) : nullptr;
    switch (q.kind) {
    case HPF_OP_CONV: {
        const ConvShape s = conv_shape_of(mdl, i);
        // The weight gradient feeds nothing but the final average, so it leaves the chain of dependent kernels:
        // it runs on the partition's side stream once dL/d(output) is ready (everything before this point on st).
        cudaStream_t wst = st;
        if (!mdl->side.empty() && !mdl->opt_single) {
            wst = mdl->side[sl];
            CU(cudaEventRecord(mdl->ev_side[sl], st));
            CU(cudaStreamWaitEvent(wst, mdl->ev_side[sl], 0));
        }
        if (mdl->use_tc[PASS_WGRAD][i]) {
            CU(conv_tc_launch(&mdl->tc_plan[PASS_WGRAD][(size_t)m * mdl->n_ops + i], mdl->status(), wst, &mdl->launches));
        } else {
            CU(conv_wgrad_simt(in0, dout, slot + o.w_off, s, mdl->ws + mdl->conv_scratch_off[sl], wst, &mdl->launches));
        }
        if (q.src0 >= 0) {
            if (mdl->use_tc[PASS_DGRAD][i]) {
                CU(conv_tc_launch(&mdl->tc_plan[PASS_DGRAD][(size_t)m * mdl->n_ops + i], mdl->status(), st, &mdl->launches));
            } else {
                CU(conv_dgrad_simt(dout, mdl->params + o.w_off, mdl->grad(q.src0, m), addend, e.accumulate != 0, s, st, &mdl->launches));
            }
        }
        break;
    }
    case HPF_OP_BNRELU:
        CU(bnrelu_bwd(in0, dout, mdl->params + o.w_off, mdl->params + o.b_off, mdl->stats(i, m), mdl->grad(q.src0, m), addend,
                      e.accumulate != 0, slot + o.w_off, slot + o.b_off, (int64_t)mdl->b * o.H * o.W, o.C,
                      mdl->ws + mdl->bn_scratch_bwd_off[sl], st, &mdl->launches, true, true));
        break;
    case HPF_OP_BN:
        CU(bnrelu_bwd(in0, dout, mdl->params + o.w_off, mdl->params + o.b_off, mdl->stats(i, m), mdl->grad(q.src0, m), addend,
                      e.accumulate != 0, slot + o.w_off, slot + o.b_off, (int64_t)mdl->b * o.H * o.W, o.C,
                      mdl->ws + mdl->bn_scratch_bwd_off[sl], st, &mdl->launches, false, true));
        break;
    case HPF_OP_RELU:
        CU(relu_bwd(in0, dout, mdl->grad(q.src0, m), addend, e.accumulate != 0, mdl->numel(i), st, &mdl->launches));
        break;
    case HPF_OP_ADD:
        break;   // its contributions are aliases, on-the-fly addends, or the explicit accumulations above
    case HPF_OP_MAXPOOL:
        if (q.src0 >= 0)
            CU(maxpool_bwd(in0, dout, mdl->grad(q.src0, m), e.accumulate != 0, conv_shape_of(mdl, i), st, &mdl->launches));
        break;
    case HPF_OP_HEAD:
        CU(head_bwd(mdl->params + o.w_off, mdl->cur_labels + (int64_t)m * mdl->b, mdl->act(i, m),
                    reinterpret_cast<float*>(mdl->ws + mdl->pooled_off[m]), dout, mdl->grad(q.src0, m), slot + o.w_off,
                    slot + o.b_off, mdl->b, o.iH * o.iW, o.iC, q.c_out, st, &mdl->launches));
        break;
    }
    return HPF_OK;
}

// phase PH_FWD / PH_BWD / PH_AVG: one phase, forked from and joined into stream 0.  PH_FB: forward and backward as ONE
// set of dependencies (hpf_forward_backward): the backward cell (p, m) runs on partition p's backward stream as soon as
// the cell that feeds it has finished - backward (p+1, m), or forward (P-1, m) for the last partition - while the
// partition's forward stream may still be busy with later micro-batches.  Same kernels on the same data as the two
// phases, so the results are bit-identical; only the idle slots of the forward drain and the backward fill get used.
// Cells under way, roughly, while cell (p, m) of the forward (bwd = false) or backward phase runs in the one-graph schedule:
// the stages busy at its own tick plus those of the other phase at the tick that runs at the same time (the backward
// pipeline starts when the first micro-batch has passed all P stages).
int cells_under_way(int P, int M, int p, int m, bool bwd)
{
    auto busy = [&](int t) {
        if (t < 0 || t > P + M - 2) return 0;
        int n = t + 1;
        if (n > P) n = P;
        if (n > M) n = M;
        if (n > P + M - 1 - t) n = P + M - 1 - t;
        return n;
    };
    const int t = bwd ? (P - 1 - p) + m : p + m;
    return bwd ? busy(t) + busy(t + P) : busy(t) + busy(t - P);
}

int enqueue_phase(hpf_model* mdl, int phase)
{
    const PdlScope pdl_scope(mdl->opt_pdl);
    const BnClusterScope bn_cluster_scope(mdl->opt_bn_cluster);
    const int P = mdl->P, M = mdl->M;
    cudaStream_t s0 = mdl->streams[0];
    const bool merged = phase == PH_FB;
    const bool do_fwd = phase == PH_FWD || merged, do_bwd = phase == PH_BWD || merged;
    const int S = mdl->n_slots();
    const bool multi = !mdl->opt_single && S > 1;
    const bool own_bwd_streams = merged && !mdl->bwd_streams.empty() && !mdl->opt_single;
    auto bwd_stream = [&](int p, int m) { return own_bwd_streams ? mdl->bwd_streams[mdl->slot_of(p, m)] : mdl->stream_of(p, m); };
    if (multi || own_bwd_streams) {
        CU(cudaEventRecord(mdl->ev_fork, s0));
        if (multi) for (int k = 1; k < S; ++k) CU(cudaStreamWaitEvent(mdl->streams[k], mdl->ev_fork, 0));
        if (own_bwd_streams) for (int k = 0; k < S; ++k) CU(cudaStreamWaitEvent(mdl->bwd_streams[k], mdl->ev_fork, 0));
    }
    if (do_fwd) {
        // the tensor-core convolutions read split (and, for the data gradient, rearranged) weights: once per step
        for (int p = 0; p < P; ++p)
            if (!mdl->prep_table[p].empty()) {
                float* wp = reinterpret_cast<float*>(mdl->ws + mdl->wprep_off);
                const int64_t G4 = (mdl->G + 3) / 4 * 4;      // keeps every array 16-byte aligned
                int max_tiles = 1;
                for (const WeightPrepEntry& e : mdl->prep_table[p]) max_tiles = std::max(max_tiles, conv_weight_prep_tiles(e.C, e.K, e.R));
                CU(conv_weight_prep(mdl->params, wp, wp + G4, wp + 2 * G4, wp + 3 * G4,
                                    reinterpret_cast<const WeightPrepEntry*>(mdl->ws + mdl->prep_table_off[p]),
                                    (int)mdl->prep_table[p].size(), max_tiles, mdl->stream_of(p), &mdl->launches));
                // the partition's other lanes read the same prepared weights
                if (multi && mdl->lanes() > 1) {
                    CU(cudaEventRecord(mdl->ev_prep[p], mdl->stream_of(p)));
                    for (int l = 1; l < mdl->lanes(); ++l) CU(cudaStreamWaitEvent(mdl->streams[p * mdl->lanes() + l], mdl->ev_prep[p], 0));
                }
            }
        // tick t: every (p, m) with p + m = t
        for (int t = 0; t < P + M - 1; ++t)
            for (int p = 0; p < P; ++p) {
                const int m = t - p;
                if (m < 0 || m >= M) continue;
                cudaStream_t st = mdl->stream_of(p, m);
                if (p > 0) {
                    if (multi) CU(cudaStreamWaitEvent(st, mdl->ev_fwd[(size_t)(p - 1) * M + m], 0));     // recv
                    if (mdl->opt_messages)
                        for (size_t k = 0; k < mdl->live[p - 1].size(); ++k)
                            CU(grad_accumulate(reinterpret_cast<float*>(mdl->ws + mdl->fmsg_off[p - 1][k * M + m]),
                                               mdl->act(mdl->live[p - 1][k], m), mdl->numel(mdl->live[p - 1][k]), false, st, &mdl->launches));
                }
                if (mdl->opt_cell_times) CU(stamp_time(mdl->cell_time_slot(PH_FWD, p, m), st, &mdl->launches));
                for (int i = mdl->part_lo[p]; i < mdl->part_hi[p]; ++i) {
                    int rc = forward_op(mdl, i, m, st, mdl->slot_of(p, m));
                    if (rc) return rc;
                }
                if (mdl->opt_cell_times) CU(stamp_time(mdl->cell_time_slot(PH_FWD, p, m) + 1, st, &mdl->launches));
                if (p < P - 1 && multi) CU(cudaEventRecord(mdl->ev_fwd[(size_t)p * M + m], st));          // send
                if (p == P - 1 && own_bwd_streams) CU(cudaEventRecord(mdl->ev_fdone[m], st));            // the loss of micro-batch m stands
            }
    }
    if (do_bwd) {
        for (int t = 0; t < P + M - 1; ++t)
            for (int p = P - 1; p >= 0; --p) {
                const int m = t - (P - 1 - p);
                if (m < 0 || m >= M) continue;
                cudaStream_t st = bwd_stream(p, m);
                if (p < P - 1) {
                    if (multi || own_bwd_streams) CU(cudaStreamWaitEvent(st, mdl->ev_bwd[(size_t)p * M + m], 0));           // recv partial errors
                    if (mdl->opt_messages)
                        for (size_t k = 0; k < mdl->msg_plan[p].size(); ++k) {
                            const MessagePlan& mp = mdl->msg_plan[p][k];
                            float* dst = reinterpret_cast<float*>(mdl->ws + mdl->bmsg_off[p][k * M + m]);
                            if (mp.from_buffer) CU(grad_accumulate(dst, mdl->grad(mp.tensor, m), mdl->numel(mp.tensor), false, st, &mdl->launches));
                            if (mp.pending >= 0) CU(grad_accumulate(dst, mdl->grad(mp.pending, m), mdl->numel(mp.tensor), mp.from_buffer != 0, st, &mdl->launches));
                        }
                } else if (own_bwd_streams) {
                    CU(cudaStreamWaitEvent(st, mdl->ev_fdone[m], 0));      // the last partition turns around: forward (P-1, m) is done
                }
                if (mdl->opt_cell_times) CU(stamp_time(mdl->cell_time_slot(PH_BWD, p, m), st, &mdl->launches));
                for (int i = mdl->part_hi[p] - 1; i >= mdl->part_lo[p]; --i) {
                    int rc = backward_op(mdl, i, m, st, mdl->slot_of(p, m));
                    if (rc) return rc;
                }
                if (mdl->opt_cell_times) CU(stamp_time(mdl->cell_time_slot(PH_BWD, p, m) + 1, st, &mdl->launches));
                if (p > 0 && (multi || own_bwd_streams)) CU(cudaEventRecord(mdl->ev_bwd[(size_t)(p - 1) * M + m], st));       // send partial errors
            }
    }
    if (do_bwd && !mdl->side.empty() && !mdl->opt_single)
        for (int k = 0; k < S; ++k) {
            // the side stream holds work only if it was forked during this phase; joining an unforked stream is harmless
            cudaStream_t from = own_bwd_streams ? mdl->bwd_streams[k] : mdl->streams[k];
            CU(cudaEventRecord(mdl->ev_side[k], from));
            CU(cudaStreamWaitEvent(mdl->side[k], mdl->ev_side[k], 0));
            CU(cudaEventRecord(mdl->ev_side_join[k], mdl->side[k]));
            CU(cudaStreamWaitEvent(s0, mdl->ev_side_join[k], 0));
        }
    if (own_bwd_streams)
        for (int k = 0; k < S; ++k) {
            CU(cudaEventRecord(mdl->ev_bjoin[k], mdl->bwd_streams[k]));
            CU(cudaStreamWaitEvent(s0, mdl->ev_bjoin[k], 0));
        }
    if (multi)
        for (int k = 1; k < S; ++k) {
            CU(cudaEventRecord(mdl->ev_join[k], mdl->streams[k]));
            CU(cudaStreamWaitEvent(s0, mdl->ev_join[k], 0));
        }
    if (do_fwd)
        CU(loss_average(reinterpret_cast<float*>(mdl->ws + mdl->loss_slots_off), reinterpret_cast<float*>(mdl->ws + mdl->loss_avg_off), M, s0, &mdl->launches));
    if (phase == PH_AVG)
        CU(grad_average(mdl->gslots, mdl->gavg, M, mdl->G, s0, &mdl->launches));
    return HPF_OK;
}

int capture_phase(hpf_model* mdl, int phase, cudaGraphExec_t* exec, int64_t* nodes)
{
    cudaStream_t s0 = mdl->streams[0];
    const int64_t before = mdl->launches;
    CU(cudaStreamBeginCapture(s0, cudaStreamCaptureModeThreadLocal));
    int rc = enqueue_phase(mdl, phase);
    cudaGraph_t graph = nullptr;
    cudaError_t e = cudaStreamEndCapture(s0, &graph);
    *nodes = mdl->launches - before;
    mdl->launches = before;
    if (rc) { if (graph) cudaGraphDestroy(graph); return rc; }
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamEndCapture");
    e = cudaGraphInstantiate(exec, graph, 0);
    cudaGraphDestroy(graph);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGraphInstantiate");
    return HPF_OK;
}

int run_phase(hpf_model* mdl, int phase)
{
    if (!mdl->opt_graph) return enqueue_phase(mdl, phase);
    cudaGraphExec_t exec = nullptr;
    int64_t nodes = 0;
    if (phase == PH_FWD || phase == PH_FB) {
        // the captured graph reads the input and the labels it was captured with: one graph per (x, labels) pair, two kept
        hpf_model::FwdGraph* slots = phase == PH_FWD ? mdl->fwd_graph : mdl->fb_graph;
        int& next = phase == PH_FWD ? mdl->fwd_graph_next : mdl->fb_graph_next;
        hpf_model::FwdGraph* slot = nullptr;
        for (int k = 0; k < 2; ++k)
            if (slots[k].exec && slots[k].x == mdl->cur_x && slots[k].labels == mdl->cur_labels) slot = &slots[k];
        if (!slot) {
            slot = &slots[next];
            next ^= 1;
            if (slot->exec) { cudaGraphExecDestroy(slot->exec); slot->exec = nullptr; }
            int rc = capture_phase(mdl, phase, &slot->exec, &slot->nodes);
            if (rc) return rc;
            slot->x = mdl->cur_x; slot->labels = mdl->cur_labels;
        }
        exec = slot->exec; nodes = slot->nodes;
    } else {
        if (phase == PH_BWD && mdl->graph[PH_BWD] && (mdl->bwd_labels != mdl->cur_labels || mdl->bwd_x != mdl->cur_x)) {
            // the captured backward reads the input and the labels it was captured with
            cudaGraphExecDestroy(mdl->graph[PH_BWD]); mdl->graph[PH_BWD] = nullptr;
        }
        if (!mdl->graph[phase]) {
            int rc = capture_phase(mdl, phase, &mdl->graph[phase], &mdl->graph_nodes[phase]);
            if (rc) return rc;
            if (phase == PH_BWD) { mdl->bwd_labels = mdl->cur_labels; mdl->bwd_x = mdl->cur_x; }
        }
        exec = mdl->graph[phase]; nodes = mdl->graph_nodes[phase];
    }
    CU(cudaGraphLaunch(exec, mdl->streams[0]));
    mdl->launches += nodes;
    return HPF_OK;
}

void release_device_objects(hpf_model* mdl)
{
    for (auto& g : mdl->fwd_graph) if (g.exec) { cudaGraphExecDestroy(g.exec); g.exec = nullptr; }
    for (auto& g : mdl->fb_graph) if (g.exec) { cudaGraphExecDestroy(g.exec); g.exec = nullptr; }
    for (auto e : mdl->ev_fdone) if (e) cudaEventDestroy(e);
    for (auto e : mdl->ev_bjoin) if (e) cudaEventDestroy(e);
    mdl->ev_fdone.clear(); mdl->ev_bjoin.clear();
    for (auto& g : mdl->graph) if (g) { cudaGraphExecDestroy(g); g = nullptr; }
    for (auto e : mdl->ev_fwd) cudaEventDestroy(e);
    for (auto e : mdl->ev_bwd) cudaEventDestroy(e);
    for (auto e : mdl->ev_join) if (e) cudaEventDestroy(e);
    for (auto e : mdl->ev_prep) if (e) cudaEventDestroy(e);
    mdl->ev_prep.clear();
    for (auto e : mdl->ev_side) if (e) cudaEventDestroy(e);
    for (auto e : mdl->ev_side_join) if (e) cudaEventDestroy(e);
    mdl->ev_side.clear(); mdl->ev_side_join.clear();
    if (mdl->ev_fork) cudaEventDestroy(mdl->ev_fork);
    if (mdl->ev_sync) cudaEventDestroy(mdl->ev_sync);
    mdl->ev_fwd.clear(); mdl->ev_bwd.clear(); mdl->ev_join.clear();
    mdl->ev_fork = mdl->ev_sync = nullptr;
}

}  // namespace

// ================================================================================================
// C ABI
// ================================================================================================
extern "C" {

int hpf_model_create(const hpf_op* ops, int32_t n_ops, const int32_t in_shape[4], const int32_t* cuts, int32_t n_cuts,
                     int32_t n_microbatches, hpf_model** out)
{
    if (!ops || !in_shape || !out) return fail(HPF_ERR_INVALID, "null argument");
    if (n_ops < 1) return fail(HPF_ERR_INVALID, "empty op list");
    for (int k = 0; k < 4; ++k) if (in_shape[k] < 1) return fail(HPF_ERR_INVALID, "bad input shape");
    const int B = in_shape[0], M = n_microbatches;
    if (M < 1 || M > B || B % M) return fail(HPF_ERR_INVALID, "the micro-batch count must divide the batch");
    hpf_model* mdl = new hpf_model();
    mdl->n_ops = n_ops; mdl->B = B; mdl->M = M; mdl->b = B / M;
    mdl->inH = in_shape[1]; mdl->inW = in_shape[2]; mdl->inC = in_shape[3];
    int rc = build_ops(mdl, ops, n_ops);
    if (!rc) rc = build_partitions(mdl, cuts, n_cuts);
    if (!rc) rc = build_grad_plan(mdl);
    if (rc) { delete mdl; return rc; }
    *out = mdl;
    return HPF_OK;
}

int hpf_model_destroy(hpf_model* mdl)
{
    if (!mdl) return fail(HPF_ERR_INVALID, "null model");
    release_device_objects(mdl);
    delete mdl;
    return HPF_OK;
}

int hpf_set_option(hpf_model* mdl, int32_t option, int32_t value)
{
    if (!mdl) return fail(HPF_ERR_INVALID, "null model");
    if (mdl->state != ST_CREATED) return fail(HPF_ERR_STATE, "options must be set before hpf_bind");
    switch (option) {
    case HPF_OPT_GRAPH: mdl->opt_graph = value != 0; break;
    case HPF_OPT_CONV_PATH: if (value < 0 || value > 2) return fail(HPF_ERR_INVALID, "bad conv path"); mdl->opt_conv_path = value; break;
    case HPF_OPT_SINGLE_STREAM: mdl->opt_single = value != 0; break;
    case HPF_OPT_KEEP_MESSAGES: mdl->opt_messages = value != 0; break;
    case HPF_OPT_FUSE_ADD: mdl->opt_fuse_add = value != 0; break;
    case HPF_OPT_PDL: mdl->opt_pdl = value != 0; break;
    case HPF_OPT_FUSE_BN: if (value < 0 || value > 3) return fail(HPF_ERR_INVALID, "0..3"); mdl->opt_fuse_bn = value; break;
    case HPF_OPT_CELL_TIMES: mdl->opt_cell_times = value != 0; break;
    case HPF_OPT_BN_CLUSTER: mdl->opt_bn_cluster = value != 0; break;
    case HPF_OPT_WGRAD_DIRECT: mdl->opt_wgrad_direct = value != 0; break;
    case HPF_OPT_STAGE_LANES: if (value < 1 || value > 64) return fail(HPF_ERR_INVALID, "1..64 lanes"); mdl->opt_lanes = value; break;
    case HPF_OPT_PDL_LATE_FROM: if (value < 0) return fail(HPF_ERR_INVALID, ">= 0"); mdl->opt_pdl_late_from = value; break;
    case HPF_OPT_CELL_CTAS: if (value < 0 || value > 148) return fail(HPF_ERR_INVALID, "0..148 CTAs"); mdl->opt_cell = value; break;
    case HPF_OPT_WGRAD_PASSES: if (value != 1 && value != 3) return fail(HPF_ERR_INVALID, "1 or 3 passes"); mdl->opt_wgrad_passes = value; break;
    default: return fail(HPF_ERR_INVALID, "unknown option");
    }
    mdl->planned = false;
    return HPF_OK;
}

int hpf_num_ops(const hpf_model* mdl, int32_t* n) { if (!mdl || !n) return fail(HPF_ERR_INVALID, "null"); *n = mdl->n_ops; return HPF_OK; }
int hpf_num_partitions(const hpf_model* mdl, int32_t* P) { if (!mdl || !P) return fail(HPF_ERR_INVALID, "null"); *P = mdl->P; return HPF_OK; }
int hpf_num_stream_slots(const hpf_model* mdl, int32_t* S) { if (!mdl || !S) return fail(HPF_ERR_INVALID, "null"); *S = mdl->n_slots(); return HPF_OK; }
int hpf_num_params(const hpf_model* mdl, int64_t* G) { if (!mdl || !G) return fail(HPF_ERR_INVALID, "null"); *G = mdl->G; return HPF_OK; }

int hpf_param_layout(const hpf_model* mdl, int32_t op, int64_t* w_off, int64_t* w_cnt, int64_t* b_off, int64_t* b_cnt)
{
    if (!mdl || !w_off || !w_cnt || !b_off || !b_cnt) return fail(HPF_ERR_INVALID, "null");
    if (op < 0 || op >= mdl->n_ops) return fail(HPF_ERR_INVALID, "op out of range");
    const OpInfo& o = mdl->ops[op];
    *w_off = o.w_off; *w_cnt = o.w_cnt; *b_off = o.b_off; *b_cnt = o.b_cnt;
    return HPF_OK;
}

int hpf_op_shape(const hpf_model* mdl, int32_t op, int32_t hwc[3])
{
    if (!mdl || !hwc) return fail(HPF_ERR_INVALID, "null");
    if (op < 0 || op >= mdl->n_ops) return fail(HPF_ERR_INVALID, "op out of range");
    hwc[0] = mdl->ops[op].H; hwc[1] = mdl->ops[op].W; hwc[2] = mdl->ops[op].C;
    return HPF_OK;
}

int hpf_partition_of_op(const hpf_model* mdl, int32_t op, int32_t* p)
{
    if (!mdl || !p) return fail(HPF_ERR_INVALID, "null");
    if (op < 0 || op >= mdl->n_ops) return fail(HPF_ERR_INVALID, "op out of range");
    *p = mdl->ops[op].part;
    return HPF_OK;
}

int hpf_partition_range(const hpf_model* mdl, int32_t p, int32_t* first_op, int32_t* end_op)
{
    if (!mdl || !first_op || !end_op) return fail(HPF_ERR_INVALID, "null");
    if (p < 0 || p >= mdl->P) return fail(HPF_ERR_INVALID, "partition out of range");
    *first_op = mdl->part_lo[p]; *end_op = mdl->part_hi[p];
    return HPF_OK;
}

int hpf_microbatch_range(const hpf_model* mdl, int32_t m, int32_t* first, int32_t* end)
{
    if (!mdl || !first || !end) return fail(HPF_ERR_INVALID, "null");
    if (m < 0 || m >= mdl->M) return fail(HPF_ERR_INVALID, "micro-batch out of range");
    *first = m * mdl->b; *end = (m + 1) * mdl->b;
    return HPF_OK;
}

int hpf_boundary_count(const hpf_model* mdl, int32_t cut, int32_t* n)
{
    if (!mdl || !n) return fail(HPF_ERR_INVALID, "null");
    if (cut < 0 || cut >= (int)mdl->cuts.size()) return fail(HPF_ERR_INVALID, "cut out of range");
    *n = (int32_t)mdl->live[cut].size();
    return HPF_OK;
}

int hpf_boundary_desc(const hpf_model* mdl, int32_t cut, int32_t i, int32_t* producer_op, int32_t shape[4])
{
    if (!mdl || !producer_op || !shape) return fail(HPF_ERR_INVALID, "null");
    if (cut < 0 || cut >= (int)mdl->cuts.size()) return fail(HPF_ERR_INVALID, "cut out of range");
    if (i < 0 || i >= (int)mdl->live[cut].size()) return fail(HPF_ERR_INVALID, "boundary tensor out of range");
    const int t = mdl->live[cut][i];
    *producer_op = t;
    shape[0] = mdl->b; shape[1] = mdl->ops[t].H; shape[2] = mdl->ops[t].W; shape[3] = mdl->ops[t].C;
    return HPF_OK;
}

int hpf_schedule_tick(const hpf_model* mdl, int32_t p, int32_t m, int32_t* fwd_tick, int32_t* bwd_tick)
{
    if (!mdl || !fwd_tick || !bwd_tick) return fail(HPF_ERR_INVALID, "null");
    if (p < 0 || p >= mdl->P || m < 0 || m >= mdl->M) return fail(HPF_ERR_INVALID, "out of range");
    *fwd_tick = p + m; *bwd_tick = (mdl->P - 1 - p) + m;
    return HPF_OK;
}

int hpf_estimate_op_costs(const hpf_op* ops, int32_t n_ops, const int32_t in_shape[4], double* cost_us)
{
    if (!ops || !in_shape || !cost_us || n_ops < 1) return fail(HPF_ERR_INVALID, "null argument");
    // shapes through a throw-away model (validates the list as well)
    hpf_model* tmp = nullptr;
    int rc = hpf_model_create(ops, n_ops, in_shape, nullptr, 0, 1, &tmp);
    if (rc) return rc;
    // Calibration (B200, micro-batch 16, one stream): a bottleneck block costs 113 / 115 / 149 us at 32x32 / 16x16 / 8x8,
    // which a fixed cost per kernel, 0.39 us per tensor-core K step (8 channels of one tap, forward plus data
    // gradient) and 1.4 TB/s of effective bandwidth reproduce.
    const double us_per_k8 = 0.39, bytes_per_us = 1.4e6;
    for (int i = 0; i < n_ops; ++i) {
        const OpInfo& o = tmp->ops[i];
        const double in_el = (double)in_shape[0] * o.iH * o.iW * o.iC, out_el = (double)in_shape[0] * o.H * o.W * o.C;
        double c = 0.0;
        switch (o.op.kind) {
        case HPF_OP_CONV: {
            const int taps = o.op.ksize * o.op.ksize;
            const double k8 = taps * (o.op.c_in / 8.0) + (o.op.src0 >= 0 ? taps * (o.op.c_out / 8.0) : 0.0);
            c = 8.0 + us_per_k8 * k8 + 4.0 * 2.0 * (in_el + out_el) / bytes_per_us;
            break;
        }
        case HPF_OP_BNRELU: c = 9.0 + 20.0 * out_el / bytes_per_us; break;
        case HPF_OP_BN: c = 18.0 + 20.0 * out_el / bytes_per_us; break;        // its own reduce + apply kernels, both ways
        case HPF_OP_RELU: c = 6.0 + 20.0 * out_el / bytes_per_us; break;
        case HPF_OP_ADD: c = 0.0; break;                       // fused into the producing convolution
        case HPF_OP_MAXPOOL: c = 6.0 + 4.0 * 2.0 * (in_el + out_el) / bytes_per_us; break;
        default: c = 20.0; break;                               // head: a handful of tiny kernels
        }
        cost_us[i] = c;
    }
    hpf_model_destroy(tmp);
    return HPF_OK;
}

int hpf_balance_cuts(const double* cost, int32_t n_ops, int32_t P, int32_t* cuts)
{
    if (!cost || n_ops < 1 || P < 1 || P > n_ops || (P > 1 && !cuts)) return fail(HPF_ERR_INVALID, "bad argument");
    double total = 0.0, biggest = 0.0;
    for (int i = 0; i < n_ops; ++i) {
        if (!(cost[i] >= 0.0)) return fail(HPF_ERR_INVALID, "costs must be non-negative");
        total += cost[i];
        if (cost[i] > biggest) biggest = cost[i];
    }
    // smallest bottleneck B such that a greedy left-to-right fill needs at most P partitions (bisection on B)
    auto parts_needed = [&](double B) {
        int parts = 1; double acc = 0.0;
        for (int i = 0; i < n_ops; ++i) {
            if (acc + cost[i] > B && acc > 0.0) { ++parts; acc = 0.0; }
            acc += cost[i];
        }
        return parts;
    };
    double lo = biggest, hi = total > biggest ? total : biggest;
    for (int it = 0; it < 100; ++it) {
        const double mid = 0.5 * (lo + hi);
        if (parts_needed(mid) <= P) hi = mid; else lo = mid;
    }
    // cut greedily at bottleneck hi, but never leave fewer ops than partitions still to be filled
    int made = 0; double acc = 0.0; int start = 0;
    for (int i = 0; i < n_ops && made < P - 1; ++i) {
        const int remaining_parts = P - 1 - made;                // partitions still to open after the current one
        const bool must = n_ops - i == remaining_parts;          // every remaining op has to open a partition
        if (i > start && ((acc + cost[i] > hi * (1.0 + 1e-12)) || must)) { cuts[made++] = i; acc = 0.0; start = i; }
        acc += cost[i];
    }
    // if the costs ran out early (zero-cost tail), spread the remaining cuts over the last ops
    for (int k = made; k < P - 1; ++k) cuts[k] = n_ops - (P - 1 - k);
    for (int k = P - 2; k > 0; --k) if (cuts[k - 1] >= cuts[k]) cuts[k - 1] = cuts[k] - 1;
    return HPF_OK;
}

int hpf_workspace_bytes(const hpf_model* mdl_c, size_t* bytes)
{
    if (!mdl_c || !bytes) return fail(HPF_ERR_INVALID, "null");
    hpf_model* mdl = const_cast<hpf_model*>(mdl_c);
    if (!mdl->planned) build_memory_plan(mdl);
    *bytes = mdl->ws_bytes;
    return HPF_OK;
}

int hpf_bind(hpf_model* mdl, float* d_params, float* d_grad_slots, float* d_grad_avg, void* d_workspace, size_t ws_bytes,
             void* const* cuda_streams, int32_t n_streams)
{
    if (!mdl || !d_params || !d_grad_slots || !d_grad_avg || !d_workspace || !cuda_streams) return fail(HPF_ERR_INVALID, "null argument");
    if (mdl->state != ST_CREATED) return fail(HPF_ERR_STATE, "already bound");
    const int S = mdl->n_slots();
    if (n_streams < S) return fail(HPF_ERR_INVALID, "one stream per partition and stage lane is required");
    if (!mdl->planned) build_memory_plan(mdl);
    if (ws_bytes < mdl->ws_bytes) return fail(HPF_ERR_WORKSPACE, "workspace too small");
    if (reinterpret_cast<uintptr_t>(d_workspace) % 256) return fail(HPF_ERR_WORKSPACE, "workspace must be 256-byte aligned");
    if (reinterpret_cast<uintptr_t>(d_params) % 16 || reinterpret_cast<uintptr_t>(d_grad_slots) % 16 ||
        reinterpret_cast<uintptr_t>(d_grad_avg) % 16) return fail(HPF_ERR_INVALID, "parameter / gradient buffers must be 16-byte aligned");
    int ndev = 0;
    cudaError_t e = cudaGetDeviceCount(&ndev);
    if (e != cudaSuccess || ndev < 1) { cudaGetLastError(); return cuda_fail(e != cudaSuccess ? e : cudaErrorNoDevice, "cudaGetDeviceCount"); }
    mdl->params = d_params; mdl->gslots = d_grad_slots; mdl->gavg = d_grad_avg;
    mdl->ws = reinterpret_cast<char*>(d_workspace);
    mdl->streams.resize(S);
    for (int k = 0; k < S; ++k) mdl->streams[k] = reinterpret_cast<cudaStream_t>(cuda_streams[k]);
    mdl->side.clear();
    if (n_streams >= 2 * S) {
        mdl->side.resize(S);
        for (int k = 0; k < S; ++k) mdl->side[k] = reinterpret_cast<cudaStream_t>(cuda_streams[S + k]);
        mdl->ev_side.assign(S, nullptr); mdl->ev_side_join.assign(S, nullptr);
        for (int k = 0; k < S; ++k) {
            CU(cudaEventCreateWithFlags(&mdl->ev_side[k], cudaEventDisableTiming));
            CU(cudaEventCreateWithFlags(&mdl->ev_side_join[k], cudaEventDisableTiming));
        }
    }
    mdl->bwd_streams.clear();
    if (n_streams >= 3 * S) {
        mdl->bwd_streams.resize(S);
        for (int k = 0; k < S; ++k) mdl->bwd_streams[k] = reinterpret_cast<cudaStream_t>(cuda_streams[2 * S + k]);
        mdl->ev_fdone.assign(mdl->M, nullptr); mdl->ev_bjoin.assign(S, nullptr);
        for (auto& ev : mdl->ev_fdone) CU(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
        for (auto& ev : mdl->ev_bjoin) CU(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
    }
    const int M = mdl->M, n = mdl->n_ops;
    CU(cudaEventCreateWithFlags(&mdl->ev_fork, cudaEventDisableTiming));
    CU(cudaEventCreateWithFlags(&mdl->ev_sync, cudaEventDisableTiming));
    mdl->ev_join.assign(S, nullptr);
    for (int k = 1; k < S; ++k) CU(cudaEventCreateWithFlags(&mdl->ev_join[k], cudaEventDisableTiming));
    mdl->ev_prep.assign(mdl->P, nullptr);
    for (auto& ev : mdl->ev_prep) CU(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
    mdl->ev_fwd.resize(mdl->cuts.size() * M); mdl->ev_bwd.resize(mdl->cuts.size() * M);
    for (auto& ev : mdl->ev_fwd) CU(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
    for (auto& ev : mdl->ev_bwd) CU(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
    CU(cudaMemsetAsync(mdl->ws + mdl->zero_lo, 0, mdl->zero_hi - mdl->zero_lo, mdl->streams[0]));
    // tensor-core plans
    bool any_tc = false;
    for (int pass = 0; pass < 3; ++pass)
        for (int i = 0; i < n; ++i) if (mdl->use_tc[pass][i]) any_tc = true;
    mdl->prep_table.assign(mdl->P, {});
    if (any_tc) {
        CU(conv_tc_init());
        const int passes = mdl->opt_conv_path == 2 ? 1 : 3;
        float* wp = reinterpret_cast<float*>(mdl->ws + mdl->wprep_off);
        const int64_t G = (mdl->G + 3) / 4 * 4;       // stride between the four prepared-weight arrays
        for (int i = 0; i < n; ++i)
            if (mdl->use_tc[PASS_FWD][i] || mdl->use_tc[PASS_DGRAD][i]) {
                const OpInfo& o = mdl->ops[i];
                mdl->prep_table[o.part].push_back(WeightPrepEntry{o.w_off, o.op.c_in, o.op.c_out, o.op.ksize, 0});
            }
        for (int p = 0; p < mdl->P; ++p)
            if (!mdl->prep_table[p].empty())
                CU(cudaMemcpyAsync(mdl->ws + mdl->prep_table_off[p], mdl->prep_table[p].data(),
                                   sizeof(WeightPrepEntry) * mdl->prep_table[p].size(), cudaMemcpyHostToDevice, mdl->streams[0]));
        for (int pass = 0; pass < 3; ++pass) mdl->tc_plan[pass].resize((size_t)n * M);
        // the forward launch of convolution i on micro-batch m (prepared again when its cell's shared-memory budget changes)
        auto prepare_fwd = [&](int i, int m) -> int {
            const OpInfo& o = mdl->ops[i];
            const int src = o.op.src0;
            const ConvShape s = conv_shape_of(mdl, i);
            ConvTcPlan* pl = &mdl->tc_plan[PASS_FWD][(size_t)m * n + i];
            const int sl = mdl->slot_of(o.part, m);
            void* scratch = mdl->ws + mdl->conv_scratch_off[sl];
            const int pass = PASS_FWD;
            const float* residual = nullptr;
                    if (mdl->fused_into[i] >= 0) {
                        const hpf_op& a = mdl->ops[mdl->fused_into[i]].op;
                        residual = mdl->act(a.src0 == i ? a.src1 : a.src0, m);
                    }
                    ConvBnFuse fuse;
                    if (mdl->splitk_bytes[o.part]) { fuse.splitk = mdl->ws + mdl->splitk_off[sl]; fuse.splitk_bytes = mdl->splitk_bytes[o.part]; }
                    fuse.pdl_late = cells_under_way(mdl->P, M, o.part, m, false) * mdl->lanes() >= mdl->opt_pdl_late_from;
                    if (mdl->cell_of_op[i] >= 0) {
                        fuse.cell_ctas = mdl->opt_cell;
                        fuse.cell_smem = mdl->cell_runs[mdl->cell_of_op[i]].smem_budget;
                    }
                    if (mdl->conv_fwd_bn[i] >= 0) {
                        const int jn = mdl->conv_fwd_bn[i];
                        const OpInfo& bn = mdl->ops[jn];
                        fuse.mode = mdl->bn_late[jn] ? 3 : 1;
                        fuse.ticket = reinterpret_cast<unsigned int*>(mdl->ws + mdl->bn_scratch_off[sl]);
                        fuse.partials = mdl->bn_partials(jn, m);
                        fuse.stats_out = mdl->stats(jn, m);
                        fuse.rows = (long long)mdl->b * bn.H * bn.W;
                        fuse.eps = bn.op.eps;
                    }
                    const float* in = mdl->act(src, m);
                    const int jb = mdl->conv_in_bn[i];
                    if (jb >= 0) {
                        const OpInfo& bn = mdl->ops[jb];
                        in = mdl->act(bn.op.src0, m);          // the BN's input; its output is a by-product of this kernel
                        fuse.in_mode = mdl->bn_late[jb] ? 2 : 1;
                        fuse.in_partials = mdl->bn_partials(jb, m);
                        fuse.in_tiles = conv_tc_tiles(conv_shape_of(mdl, mdl->bn_fwd_from[jb]), PASS_FWD);
                        fuse.in_rows = (long long)mdl->b * bn.H * bn.W;
                        fuse.in_eps = bn.op.eps;
                        fuse.in_gamma = mdl->params + bn.w_off; fuse.in_beta = mdl->params + bn.b_off;
                        fuse.in_stats = mdl->stats(jb, m); fuse.in_y = mdl->act(jb, m);
                    }
                    CU(conv_tc_prepare(pl, s, pass, passes, in, nullptr, wp + o.w_off, wp + G + o.w_off,
                                       mdl->act(i, m), residual, false, scratch, &fuse));
            return HPF_OK;
        };
        for (int pass = 0; pass < 3; ++pass) {
            for (int m = 0; m < M; ++m)
                for (int i = 0; i < n; ++i) {
                    if (!mdl->use_tc[pass][i]) continue;
                    const OpInfo& o = mdl->ops[i];
                    const int src = o.op.src0;
                    const ConvShape s = conv_shape_of(mdl, i);
                    const GradEdge& ed = mdl->edge0[i];
                    ConvTcPlan* pl = &mdl->tc_plan[pass][(size_t)m * n + i];
                    const int sl = mdl->slot_of(o.part, m);
                    void* scratch = mdl->ws + mdl->conv_scratch_off[sl];
                    if (pass == PASS_FWD) {
                        int rc = prepare_fwd(i, m);
                        if (rc) return rc;
                    }
                    else if (pass == PASS_DGRAD) {
                        ConvBnFuse dsplit;
                        if (mdl->splitk_bytes[o.part]) { dsplit.splitk = mdl->ws + mdl->splitk_bwd_off[sl]; dsplit.splitk_bytes = mdl->splitk_bytes[o.part]; }
                        CU(conv_tc_prepare(pl, s, pass, passes, mdl->grad(i, m), nullptr, wp + 2 * G + o.w_off, wp + 3 * G + o.w_off,
                                           mdl->grad(src, m), ed.addend >= 0 ? mdl->grad(ed.addend, m) : nullptr, ed.accumulate != 0, scratch,
                                           &dsplit));
                    }
                    else {
                        // Weight gradients run on the side streams, beside the stages' chains of dependent kernels and feeding
                        // nothing but the final average.  With many stages busy the SM time a launch takes counts, not its
                        // duration: about 32 CTAs is the measured optimum for eight stages (fewer and the weight gradients
                        // fall behind the chain; with four stages the uncapped launch measured faster).
                        ConvBnFuse hint;
                        hint.wgrad_max_ctas = (mdl->n_slots() >= 6 && !mdl->side.empty()) ? 32 : 0;
                        hint.wgrad_transposing = mdl->opt_wgrad_direct ? 0 : 1;
                        CU(conv_tc_prepare(pl, s, pass, mdl->opt_conv_path == 2 ? 1 : mdl->opt_wgrad_passes, mdl->grad(i, m), mdl->act(src, m), nullptr, nullptr,
                                           mdl->gslots + (int64_t)m * mdl->G + o.w_off, nullptr, false, scratch, &hint));
                    }
                }
        }
        // persistent forward cells: records of every run's launches, per micro-batch
        for (auto& run : mdl->cell_runs) {
            // a launch whose operand pipeline came out shallower than it wants (wide channels: large stages) gets the
            // shared memory of a whole SM; such a cell's CTAs then sit one per SM
            bool shallow = false;
            for (int i : run.convs) {
                int stages = 0, iters = 0;
                conv_tc_plan_pipeline(&mdl->tc_plan[PASS_FWD][i], &stages, &iters);
                if (stages < (iters < 3 ? iters : 3)) shallow = true;
            }
            if (shallow) {
                run.smem_budget = 200u * 1024u;
                for (int m = 0; m < M; ++m)
                    for (int i : run.convs) { int rc = prepare_fwd(i, m); if (rc) return rc; }
            }
            const size_t rec = conv_tc_cell_op_bytes();
            std::vector<unsigned char> host(rec * run.convs.size());
            bool ok = true;
            unsigned int most_ctas = 0;
            for (int m = 0; m < M && ok; ++m) {
                for (size_t k = 0; k < run.convs.size() && ok; ++k) {
                    unsigned int smem = 0, tmem = 0, ctas = 0;
                    cudaError_t e = conv_tc_cell_op(&mdl->tc_plan[PASS_FWD][(size_t)m * n + run.convs[k]], mdl->status(), host.data() + k * rec, &smem, &tmem, &ctas);
                    if (e == cudaErrorNotSupported) { ok = false; break; }
                    CU(e);
                    if (smem > run.smem) run.smem = smem;
                    if (tmem > run.tmem) run.tmem = tmem;
                    if (ctas > most_ctas) most_ctas = ctas;
                }
                if (ok) CU(cudaMemcpyAsync(mdl->ws + run.ops_off[m], host.data(), host.size(), cudaMemcpyHostToDevice, mdl->streams[0]));
                CU(cudaStreamSynchronize(mdl->streams[0]));          // `host` is reused for the next micro-batch
            }
            run.ctas = (int)most_ctas < mdl->opt_cell ? (int)most_ctas : mdl->opt_cell;
            run.ready = ok && run.ctas >= 1;
        }
        // All cells that can run at the same time (one per partition) must be resident together, or their grid barriers
        // would wait for CTAs that cannot start: the grids have to fit the GPU side by side.
        {
            std::vector<double> share(mdl->P, 0.0);
            for (const auto& run : mdl->cell_runs) {
                if (!run.ready) continue;
                const int cap = conv_tc_cell_max_ctas(run.smem);
                if (cap < run.ctas) return fail(HPF_ERR_UNSUPPORTED, "a persistent cell kernel does not fit the GPU");
                share[run.part] = std::max(share[run.part], (double)run.ctas / cap);
            }
            double total = 0.0;
            for (double v : share) total += v;
            if (total > 0.92) return fail(HPF_ERR_UNSUPPORTED, "the persistent cell kernels of all partitions do not fit the GPU together: lower HPF_OPT_CELL_CTAS");
        }
    }
    CU(cudaStreamSynchronize(mdl->streams[0]));
    mdl->state = ST_BOUND;
    return HPF_OK;
}

int hpf_forward(hpf_model* mdl, const float* d_x, const int32_t* d_labels)
{
    if (!mdl || !d_x || !d_labels) return fail(HPF_ERR_INVALID, "null argument");
    if (mdl->state < ST_BOUND) return fail(HPF_ERR_STATE, "hpf_bind first");
    mdl->cur_x = d_x; mdl->cur_labels = d_labels;
    int rc = run_phase(mdl, PH_FWD);
    if (rc) return rc;
    mdl->state = ST_FWD;
    return HPF_OK;
}

int hpf_forward_backward(hpf_model* mdl, const float* d_x, const int32_t* d_labels)
{
    if (!mdl || !d_x || !d_labels) return fail(HPF_ERR_INVALID, "null argument");
    if (mdl->state < ST_BOUND) return fail(HPF_ERR_STATE, "hpf_bind first");
    mdl->cur_x = d_x; mdl->cur_labels = d_labels;
    int rc = run_phase(mdl, PH_FB);
    if (rc) return rc;
    mdl->state = ST_BWD;
    return HPF_OK;
}

// ---- one cell at a time: the building blocks of a stage-per-GPU run (each GPU owns one partition) ----------------
int hpf_prepare_partition(hpf_model* mdl, int32_t p)
{
    if (!mdl) return fail(HPF_ERR_INVALID, "null model");
    if (mdl->state < ST_BOUND) return fail(HPF_ERR_STATE, "hpf_bind first");
    if (p < 0 || p >= mdl->P) return fail(HPF_ERR_INVALID, "partition out of range");
    if (mdl->prep_table[p].empty()) return HPF_OK;
    float* wp = reinterpret_cast<float*>(mdl->ws + mdl->wprep_off);
    const int64_t G4 = (mdl->G + 3) / 4 * 4;
    int max_tiles = 1;
    for (const WeightPrepEntry& e : mdl->prep_table[p]) max_tiles = std::max(max_tiles, conv_weight_prep_tiles(e.C, e.K, e.R));
    CU(conv_weight_prep(mdl->params, wp, wp + G4, wp + 2 * G4, wp + 3 * G4,
                        reinterpret_cast<const WeightPrepEntry*>(mdl->ws + mdl->prep_table_off[p]),
                        (int)mdl->prep_table[p].size(), max_tiles, mdl->stream_of(p), &mdl->launches));
    if (mdl->lanes() > 1 && !mdl->opt_single) {
        CU(cudaEventRecord(mdl->ev_prep[p], mdl->stream_of(p)));
        for (int l = 1; l < mdl->lanes(); ++l) CU(cudaStreamWaitEvent(mdl->streams[p * mdl->lanes() + l], mdl->ev_prep[p], 0));
    }
    return HPF_OK;
}

int hpf_forward_cell(hpf_model* mdl, int32_t p, int32_t m, const float* d_x, const int32_t* d_labels)
{
    if (!mdl) return fail(HPF_ERR_INVALID, "null model");
    if (mdl->state < ST_BOUND) return fail(HPF_ERR_STATE, "hpf_bind first");
    if (p < 0 || p >= mdl->P || m < 0 || m >= mdl->M) return fail(HPF_ERR_INVALID, "cell out of range");
    if (p == 0 && !d_x) return fail(HPF_ERR_INVALID, "the first partition reads the network input");
    if (p == mdl->P - 1 && !d_labels) return fail(HPF_ERR_INVALID, "the last partition reads the labels");
    if (d_x) mdl->cur_x = d_x;
    if (d_labels) mdl->cur_labels = d_labels;
    const PdlScope pdl_scope(mdl->opt_pdl);
    const BnClusterScope bn_cluster_scope(mdl->opt_bn_cluster);
    for (int i = mdl->part_lo[p]; i < mdl->part_hi[p]; ++i) {
        int rc = forward_op(mdl, i, m, mdl->stream_of(p, m), mdl->slot_of(p, m));
        if (rc) return rc;
    }
    if (mdl->state < ST_FWD) mdl->state = ST_FWD;
    return HPF_OK;
}

int hpf_backward_cell(hpf_model* mdl, int32_t p, int32_t m)
{
    if (!mdl) return fail(HPF_ERR_INVALID, "null model");
    if (mdl->state < ST_FWD) return fail(HPF_ERR_STATE, "the cell's forward has not run");
    if (p < 0 || p >= mdl->P || m < 0 || m >= mdl->M) return fail(HPF_ERR_INVALID, "cell out of range");
    if (p == mdl->P - 1 && !mdl->cur_labels) return fail(HPF_ERR_STATE, "the last partition needs the labels of its forward cell");
    const PdlScope pdl_scope(mdl->opt_pdl);
    const BnClusterScope bn_cluster_scope(mdl->opt_bn_cluster);
    for (int i = mdl->part_hi[p] - 1; i >= mdl->part_lo[p]; --i) {
        int rc = backward_op(mdl, i, m, mdl->stream_of(p, m), mdl->slot_of(p, m));
        if (rc) return rc;
    }
    mdl->state = ST_BWD;
    return HPF_OK;
}

int hpf_join_partition(hpf_model* mdl, int32_t p)
{
    if (!mdl) return fail(HPF_ERR_INVALID, "null model");
    if (mdl->state < ST_BOUND) return fail(HPF_ERR_STATE, "hpf_bind first");
    if (p < 0 || p >= mdl->P) return fail(HPF_ERR_INVALID, "partition out of range");
    if (!mdl->side.empty() && !mdl->opt_single) {
        // every lane's weight gradients and cells join the partition's first stream
        cudaStream_t st = mdl->stream_of(p);
        for (int l = 0; l < mdl->lanes(); ++l) {
            const int k = p * mdl->lanes() + l;
            CU(cudaEventRecord(mdl->ev_side[k], mdl->streams[k]));
            CU(cudaStreamWaitEvent(mdl->side[k], mdl->ev_side[k], 0));
            CU(cudaEventRecord(mdl->ev_side_join[k], mdl->side[k]));
            CU(cudaStreamWaitEvent(st, mdl->ev_side_join[k], 0));
        }
    }
    return HPF_OK;
}

int hpf_partition_param_range(const hpf_model* mdl, int32_t p, int64_t* first, int64_t* count)
{
    if (!mdl || !first || !count) return fail(HPF_ERR_INVALID, "null");
    if (p < 0 || p >= mdl->P) return fail(HPF_ERR_INVALID, "partition out of range");
    const OpInfo& a = mdl->ops[mdl->part_lo[p]];
    const OpInfo& z = mdl->ops[mdl->part_hi[p] - 1];
    *first = a.w_off;
    *count = z.b_off + z.b_cnt - a.w_off;
    return HPF_OK;
}

int hpf_backward_message_count(const hpf_model* mdl, int32_t cut, int32_t* n)
{
    if (!mdl || !n) return fail(HPF_ERR_INVALID, "null");
    if (cut < 0 || cut >= (int)mdl->cuts.size()) return fail(HPF_ERR_INVALID, "cut out of range");
    int k = 0;
    for (const MessagePlan& mp : mdl->msg_plan[cut]) k += (mp.from_buffer ? 1 : 0) + (mp.pending >= 0 ? 1 : 0);
    *n = k;
    return HPF_OK;
}

int hpf_backward_message_desc(const hpf_model* mdl, int32_t cut, int32_t j, int32_t* op, int32_t shape[4])
{
    if (!mdl || !op || !shape) return fail(HPF_ERR_INVALID, "null");
    if (cut < 0 || cut >= (int)mdl->cuts.size()) return fail(HPF_ERR_INVALID, "cut out of range");
    int k = 0;
    for (const MessagePlan& mp : mdl->msg_plan[cut]) {
        const int cand[2] = {mp.from_buffer ? mp.tensor : -1, mp.pending};
        for (int c = 0; c < 2; ++c) {
            if (cand[c] < 0) continue;
            if (k++ == j) {
                *op = cand[c];
                shape[0] = mdl->b; shape[1] = mdl->ops[cand[c]].H; shape[2] = mdl->ops[cand[c]].W; shape[3] = mdl->ops[cand[c]].C;
                return HPF_OK;
            }
        }
    }
    return fail(HPF_ERR_INVALID, "message out of range");
}

int hpf_backward(hpf_model* mdl)
{
    if (!mdl) return fail(HPF_ERR_INVALID, "null model");
    if (mdl->state != ST_FWD) return fail(HPF_ERR_STATE, "hpf_backward needs a fresh hpf_forward");
    int rc = run_phase(mdl, PH_BWD);
    if (rc) return rc;
    mdl->state = ST_BWD;
    return HPF_OK;
}

int hpf_grad_average(hpf_model* mdl)
{
    if (!mdl) return fail(HPF_ERR_INVALID, "null model");
    if (mdl->state != ST_BWD) return fail(HPF_ERR_STATE, "hpf_grad_average needs hpf_backward");
    return run_phase(mdl, PH_AVG);
}

int hpf_sgd_momentum_step(hpf_model* mdl, float* d_velocity, float lr, float momentum, float weight_decay)
{
    if (!mdl || !d_velocity) return fail(HPF_ERR_INVALID, "null argument");
    if (mdl->state != ST_BWD) return fail(HPF_ERR_STATE, "hpf_sgd_momentum_step needs hpf_backward");
    if (!(lr >= 0.f) || !(momentum >= 0.f) || !(weight_decay >= 0.f)) return fail(HPF_ERR_INVALID, "negative or NaN hyper-parameter");
    // stream 0 carries the tail of the backward phase: the update is ordered behind every gradient
    CU(sgd_momentum(mdl->gslots, mdl->gavg, mdl->params, d_velocity, mdl->M, mdl->G, lr, momentum, weight_decay,
                    mdl->streams[0], &mdl->launches));
    return HPF_OK;
}

int hpf_loss(hpf_model* mdl, float* h_loss)
{
    if (!mdl || !h_loss) return fail(HPF_ERR_INVALID, "null argument");
    if (mdl->state < ST_FWD) return fail(HPF_ERR_STATE, "hpf_loss needs hpf_forward");
    CU(cudaMemcpyAsync(h_loss, mdl->ws + mdl->loss_avg_off, sizeof(float), cudaMemcpyDeviceToHost, mdl->streams[0]));
    CU(cudaStreamSynchronize(mdl->streams[0]));
    return HPF_OK;
}

int hpf_step_host(hpf_model* mdl, const float* h_x, const int32_t* h_labels, float* h_loss)
{
    if (!mdl || !h_x || !h_labels || !h_loss) return fail(HPF_ERR_INVALID, "null argument");
    if (mdl->state < ST_BOUND) return fail(HPF_ERR_STATE, "hpf_bind first");
    cudaStream_t s0 = mdl->streams[0];
    float* dx = reinterpret_cast<float*>(mdl->ws + mdl->stage_x_off);
    int32_t* dl = reinterpret_cast<int32_t*>(mdl->ws + mdl->stage_lab_off);
    CU(cudaMemcpyAsync(dx, h_x, sizeof(float) * (size_t)mdl->B * mdl->inH * mdl->inW * mdl->inC, cudaMemcpyHostToDevice, s0));
    CU(cudaMemcpyAsync(dl, h_labels, sizeof(int32_t) * (size_t)mdl->B, cudaMemcpyHostToDevice, s0));
    int rc = hpf_forward_backward(mdl, dx, dl);
    if (!rc) rc = hpf_grad_average(mdl);
    if (rc) return rc;
    return hpf_loss(mdl, h_loss);
}

int hpf_synchronize(hpf_model* mdl, int32_t timeout_ms)
{
    if (!mdl) return fail(HPF_ERR_INVALID, "null model");
    if (mdl->state < ST_BOUND) return fail(HPF_ERR_STATE, "hpf_bind first");
    // every phase joins into stream 0, so its tail covers all stages
    CU(cudaEventRecord(mdl->ev_sync, mdl->streams[0]));
    const auto t0 = std::chrono::steady_clock::now();
    for (;;) {
        cudaError_t e = cudaEventQuery(mdl->ev_sync);
        if (e == cudaSuccess) break;
        if (e != cudaErrorNotReady) return cuda_fail(e, "cudaEventQuery");
        if (timeout_ms > 0 &&
            std::chrono::duration_cast<std::chrono::milliseconds>(std::chrono::steady_clock::now() - t0).count() > timeout_ms)
            return fail(HPF_ERR_TIMEOUT, "hpf_synchronize: deadline passed");
        std::this_thread::sleep_for(std::chrono::microseconds(50));
    }
    DeviceStatus hs{0, 0};
    CU(cudaMemcpy(&hs, mdl->status(), sizeof hs, cudaMemcpyDeviceToHost));
    if (hs.code) {
        char buf[128];
        snprintf(buf, sizeof buf, "a bounded device-side wait gave up (code %u, detail %u)", hs.code, hs.detail);
        return fail(HPF_ERR_TIMEOUT, buf);
    }
    return HPF_OK;
}

int hpf_tensor_ptr(const hpf_model* mdl, int32_t op, int32_t m, int32_t want_grad, const float** d_ptr, int32_t shape[4])
{
    if (!mdl || !d_ptr || !shape) return fail(HPF_ERR_INVALID, "null");
    if (mdl->state < ST_BOUND) return fail(HPF_ERR_STATE, "hpf_bind first");
    if (op < 0 || op >= mdl->n_ops || m < 0 || m >= mdl->M) return fail(HPF_ERR_INVALID, "out of range");
    if (!want_grad && mdl->fused_into[op] >= 0) return fail(HPF_ERR_STATE, "not stored: this convolution's output is fused into the residual add");
    *d_ptr = want_grad ? mdl->grad(op, m) : mdl->act(op, m);
    shape[0] = mdl->b; shape[1] = mdl->ops[op].H; shape[2] = mdl->ops[op].W; shape[3] = mdl->ops[op].C;
    return HPF_OK;
}

int hpf_message_ptr(const hpf_model* mdl, int32_t cut, int32_t i, int32_t m, int32_t want_grad, const float** d_ptr)
{
    if (!mdl || !d_ptr) return fail(HPF_ERR_INVALID, "null");
    if (mdl->state < ST_BOUND || !mdl->opt_messages) return fail(HPF_ERR_STATE, "needs HPF_OPT_KEEP_MESSAGES and hpf_bind");
    if (cut < 0 || cut >= (int)mdl->cuts.size() || m < 0 || m >= mdl->M || i < 0 || i >= (int)mdl->live[cut].size())
        return fail(HPF_ERR_INVALID, "out of range");
    const size_t off = want_grad ? mdl->bmsg_off[cut][(size_t)i * mdl->M + m] : mdl->fmsg_off[cut][(size_t)i * mdl->M + m];
    *d_ptr = reinterpret_cast<const float*>(mdl->ws + off);
    return HPF_OK;
}

int hpf_loss_slots_ptr(const hpf_model* mdl, const float** d_ptr)
{
    if (!mdl || !d_ptr) return fail(HPF_ERR_INVALID, "null");
    if (mdl->state < ST_BOUND) return fail(HPF_ERR_STATE, "hpf_bind first");
    *d_ptr = reinterpret_cast<const float*>(mdl->ws + mdl->loss_slots_off);
    return HPF_OK;
}

int hpf_cell_times(hpf_model* mdl, int32_t phase, int64_t* h_ns)
{
    if (!mdl || !h_ns) return fail(HPF_ERR_INVALID, "null");
    if (phase != 0 && phase != 1) return fail(HPF_ERR_INVALID, "phase is 0 (forward) or 1 (backward)");
    if (mdl->state < ST_FWD || (phase == 1 && mdl->state < ST_BWD)) return fail(HPF_ERR_STATE, "run the phase first");
    if (!mdl->opt_cell_times) return fail(HPF_ERR_STATE, "HPF_OPT_CELL_TIMES is off");
    int rc = hpf_synchronize(mdl, 0);
    if (rc) return rc;
    static_assert(sizeof(unsigned long long) == sizeof(int64_t), "timestamp width");
    CU(cudaMemcpy(h_ns, mdl->cell_time_slot(phase ? PH_BWD : PH_FWD, 0, 0), sizeof(int64_t) * 2 * (size_t)mdl->P * mdl->M, cudaMemcpyDeviceToHost));
    return HPF_OK;
}

int hpf_step_bytes(const hpf_model* mdl_c, double* fused_bytes)
{
    if (!mdl_c || !fused_bytes) return fail(HPF_ERR_INVALID, "null");
    hpf_model* mdl = const_cast<hpf_model*>(mdl_c);
    if (!mdl->planned) build_memory_plan(mdl);
    double total = 0.0;
    double conv_weights = 0.0;
    for (int i = 0; i < mdl->n_ops; ++i) {
        const OpInfo& o = mdl->ops[i];
        const hpf_op& q = o.op;
        const double out_el = (double)mdl->b * o.H * o.W * o.C, in_el = (double)mdl->b * o.iH * o.iW * o.iC;
        const GradEdge& e = mdl->edge0[i];
        const double extra_in = (e.addend >= 0 ? in_el : 0.0) + (e.accumulate ? in_el : 0.0);
        double f = 0.0, bw = 0.0;
        switch (q.kind) {
        case HPF_OP_CONV: {
            const double w = (double)q.c_out * q.ksize * q.ksize * q.c_in;
            const double read_in = q.stride > 1 && q.ksize == 1 ? (double)mdl->b * o.H * o.W * o.iC : in_el;   // a strided 1x1 samples
            conv_weights += w;
            f = read_in + w + out_el;
            if (mdl->fused_into[i] >= 0) f += out_el;                       // the residual rides in the write-out
            if (mdl->conv_in_bn[i] >= 0) f += in_el;                        // the BN+ReLU output is stored as a by-product
            if (q.src0 >= 0) bw += out_el + w + in_el + extra_in;           // data gradient
            bw += read_in + out_el + w;                                     // weight gradient
            break;
        }
        case HPF_OP_BNRELU:
        case HPF_OP_BN:
            f = mdl->bn_into[i] >= 0 ? 0.0 : 2.0 * out_el;                 // applied by the reading convolution: no traffic of its own
            bw = 3.0 * out_el + extra_in;
            break;
        case HPF_OP_RELU: f = 2.0 * out_el; bw = 3.0 * out_el + extra_in; break;
        case HPF_OP_ADD: f = mdl->add_done_by[i] >= 0 ? 0.0 : 3.0 * out_el; break;   // its gradient is an alias or an on-the-fly addend
        case HPF_OP_MAXPOOL: f = in_el + out_el; bw = in_el + out_el + in_el + (e.accumulate ? in_el : 0.0); break;
        case HPF_OP_HEAD: f = in_el; bw = in_el; break;
        }
        total += 4.0 * (f + bw);
    }
    for (const AccumAction& a : mdl->accums) total += 4.0 * 3.0 * (double)mdl->numel(a.dst);
    total *= mdl->M;
    total += 4.0 * 5.0 * conv_weights;                                      // once per step: weights read, four prepared copies written
    total += 4.0 * (mdl->M + 1.0) * (double)mdl->G;                         // the gradient average
    *fused_bytes = total;
    return HPF_OK;
}

int hpf_launch_count(const hpf_model* mdl, int64_t* n)
{
    if (!mdl || !n) return fail(HPF_ERR_INVALID, "null");
    *n = mdl->launches;
    return HPF_OK;
}

int hpf_conv_path_counts(const hpf_model* mdl, int64_t* n_tensor, int64_t* n_cuda_core)
{
    if (!mdl || !n_tensor || !n_cuda_core) return fail(HPF_ERR_INVALID, "null");
    if (mdl->state < ST_BOUND) return fail(HPF_ERR_STATE, "hpf_bind first");
    int64_t t = 0, c = 0;
    for (int i = 0; i < mdl->n_ops; ++i) {
        if (mdl->ops[i].op.kind != HPF_OP_CONV) continue;
        for (int pass = 0; pass < 3; ++pass) {
            if (pass == PASS_DGRAD && mdl->ops[i].op.src0 < 0) continue;
            if (mdl->use_tc[pass][i]) ++t; else ++c;
        }
    }
    *n_tensor = t; *n_cuda_core = c;
    return HPF_OK;
}

// ---- single kernels -----------------------------------------------------------------------------
static int check_conv_args(int32_t N, int32_t H, int32_t W, int32_t C, int32_t K, int32_t R, int32_t stride, int32_t pad)
{
    if (N < 1 || H < 1 || W < 1 || C < 1 || K < 1 || R < 1 || stride < 1 || pad < 0 || pad >= R) return fail(HPF_ERR_INVALID, "bad convolution geometry");
    if (H + 2 * pad < R || W + 2 * pad < R) return fail(HPF_ERR_INVALID, "window larger than the padded input");
    return HPF_OK;
}

int hpf_conv_scratch_bytes(int32_t N, int32_t H, int32_t W, int32_t C, int32_t K, int32_t R, int32_t stride, int32_t pad, size_t* bytes)
{
    if (!bytes) return fail(HPF_ERR_INVALID, "null");
    int rc = check_conv_args(N, H, W, C, K, R, stride, pad);
    if (rc) return rc;
    const ConvShape s = make_conv_shape(N, H, W, C, K, R, stride, pad);
    size_t a = conv_simt_scratch_bytes(s), b = conv_tc_scratch_bytes(s);
    // [weight-gradient partials | K-split tickets and partial tiles | device status (256 bytes)]
    *bytes = align_up(a > b ? a : b, 256) + align_up(std::max(conv_tc_splitk_bytes(s, PASS_FWD, 3), conv_tc_splitk_bytes(s, PASS_DGRAD, 3)), 256) + 256;
    return HPF_OK;
}

static int conv_single(int pass, const float* in, const float* in2, const float* w, const float* wprep, float* out,
                       int32_t N, int32_t H, int32_t W, int32_t C, int32_t K, int32_t R, int32_t stride, int32_t pad,
                       int32_t path, void* d_scratch, void* stream)
{
    int rc = check_conv_args(N, H, W, C, K, R, stride, pad);
    if (rc) return rc;
    if (!in || !out || !d_scratch) return fail(HPF_ERR_INVALID, "null argument");
    const ConvShape s = make_conv_shape(N, H, W, C, K, R, stride, pad);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (path == 1) {
        if (pass != PASS_WGRAD && !w) return fail(HPF_ERR_INVALID, "null argument");
        if (pass == PASS_FWD) CU(conv_fwd_simt(in, w, out, nullptr, s, st, nullptr));
        else if (pass == PASS_DGRAD) CU(conv_dgrad_simt(in, w, out, nullptr, false, s, st, nullptr));
        else CU(conv_wgrad_simt(in2, in, out, s, d_scratch, st, nullptr));
        return HPF_OK;
    }
    const bool transposing = pass == PASS_WGRAD && (path == 3 || path == 4);
    if (transposing) path = path == 3 ? 0 : 2;
    if (path != 0 && path != 2) return fail(HPF_ERR_INVALID, "bad path");
    if (pass != PASS_WGRAD && !wprep) return fail(HPF_ERR_INVALID, "the tensor-core paths need prepared weights");
    if (!conv_tc_supported(s, pass)) return fail(HPF_ERR_UNSUPPORTED, "shape outside the tensor-core kernels' reach");
    CU(conv_tc_init());
    ConvTcPlan plan;
    // The last 256 bytes of the scratch hold the device status word.  The caller zeroes it once; the kernels only ever
    // set it (first failure wins), so a call adds no memset to the stream and back-to-back calls stay kernel after kernel.
    size_t sb = 0;
    hpf_conv_scratch_bytes(N, H, W, C, K, R, stride, pad, &sb);
    DeviceStatus* status = reinterpret_cast<DeviceStatus*>(reinterpret_cast<char*>(d_scratch) + sb - 256);
    const int64_t nw = (int64_t)K * R * R * C;
    const float* hi = wprep ? wprep + (pass == PASS_DGRAD ? 2 * nw : 0) : nullptr;
    ConvBnFuse split;
    split.wgrad_transposing = transposing ? 1 : 0;
    if (pass != PASS_WGRAD) {
        const size_t a = conv_simt_scratch_bytes(s), b = conv_tc_scratch_bytes(s);
        split.splitk_bytes = conv_tc_splitk_bytes(s, pass, 3);
        if (split.splitk_bytes) split.splitk = reinterpret_cast<char*>(d_scratch) + align_up(a > b ? a : b, 256);
    }
    CU(conv_tc_prepare(&plan, s, pass, path == 2 ? 1 : 3, in, in2, hi, hi ? hi + nw : nullptr, out, nullptr, false, d_scratch, &split));
    CU(conv_tc_launch(&plan, status, st, nullptr));
    return HPF_OK;
}

int hpf_conv_prepare_weights(const float* d_w, float* d_wprep, int32_t C, int32_t K, int32_t R, void* stream)
{
    if (!d_w || !d_wprep || C < 1 || K < 1 || R < 1) return fail(HPF_ERR_INVALID, "bad argument");
    const int64_t nw = (int64_t)K * R * R * C;
    CU(conv_weight_prep_single(d_w, d_wprep, d_wprep + nw, d_wprep + 2 * nw, d_wprep + 3 * nw, C, K, R,
                               reinterpret_cast<cudaStream_t>(stream), nullptr));
    return HPF_OK;
}

int hpf_conv_fwd(const float* d_x, const float* d_w, const float* d_wprep, float* d_y, int32_t N, int32_t H, int32_t W, int32_t C,
                 int32_t K, int32_t R, int32_t stride, int32_t pad, int32_t path, void* d_scratch, void* stream)
{
    return conv_single(PASS_FWD, d_x, nullptr, d_w, d_wprep, d_y, N, H, W, C, K, R, stride, pad, path, d_scratch, stream);
}

int hpf_conv_dgrad(const float* d_dy, const float* d_w, const float* d_wprep, float* d_dx, int32_t N, int32_t H, int32_t W,
                   int32_t C, int32_t K, int32_t R, int32_t stride, int32_t pad, int32_t path, void* d_scratch, void* stream)
{
    return conv_single(PASS_DGRAD, d_dy, nullptr, d_w, d_wprep, d_dx, N, H, W, C, K, R, stride, pad, path, d_scratch, stream);
}

int hpf_conv_wgrad(const float* d_x, const float* d_dy, float* d_dw, int32_t N, int32_t H, int32_t W, int32_t C, int32_t K,
                   int32_t R, int32_t stride, int32_t pad, int32_t path, void* d_scratch, void* stream)
{
    if (!d_x) return fail(HPF_ERR_INVALID, "null argument");
    return conv_single(PASS_WGRAD, d_dy, d_x, nullptr, nullptr, d_dw, N, H, W, C, K, R, stride, pad, path, d_scratch, stream);
}

int hpf_bnrelu_scratch_bytes(int64_t rows, int32_t C, size_t* bytes)
{
    if (!bytes || rows < 1 || C < 4 || C % 4) return fail(HPF_ERR_INVALID, "bad argument");
    *bytes = align_up(bn_scratch_bytes(rows, C), 256);
    return HPF_OK;
}

// HPF_BN_RESIDENT=0 in the environment keeps single-op BN calls on the two-kernel path (comparison runs).
static const bool g_bn_resident = [] { const char* v = getenv("HPF_BN_RESIDENT"); return !v || atoi(v) != 0; }();

int hpf_bnrelu_fwd(const float* d_x, const float* d_gamma, const float* d_beta, float eps, float* d_y, float* d_stats,
                   int64_t rows, int32_t C, void* d_scratch, void* stream)
{
    if (!d_x || !d_gamma || !d_beta || !d_y || !d_stats || !d_scratch) return fail(HPF_ERR_INVALID, "null argument");
    if (rows < 1 || C < 4 || C % 4) return fail(HPF_ERR_UNSUPPORTED, "channel count must be a multiple of 4");
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    // a single-op call has the GPU to itself: tensors that fit the chip are read once and held between the two steps
    const cudaError_t res = g_bn_resident ? bnrelu_fwd_resident(d_x, d_gamma, d_beta, eps, d_y, d_stats, rows, C, d_scratch, st, nullptr)
                                          : cudaErrorNotSupported;
    if (res == cudaSuccess) return HPF_OK;
    if (res != cudaErrorNotSupported) CU(res);
    (void)cudaGetLastError();
    CU(bnrelu_fwd(d_x, d_gamma, d_beta, eps, d_y, d_stats, rows, C, d_scratch, st, nullptr));
    return HPF_OK;
}

int hpf_bnrelu_bwd(const float* d_x, const float* d_dy, const float* d_gamma, const float* d_beta, const float* d_stats,
                   float* d_dx, const float* d_addend, int32_t accumulate, float* d_dgamma, float* d_dbeta, int64_t rows,
                   int32_t C, void* d_scratch, void* stream)
{
    if (!d_x || !d_dy || !d_gamma || !d_beta || !d_stats || !d_dx || !d_dgamma || !d_dbeta || !d_scratch) return fail(HPF_ERR_INVALID, "null argument");
    if (rows < 1 || C < 4 || C % 4) return fail(HPF_ERR_UNSUPPORTED, "channel count must be a multiple of 4");
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const cudaError_t res = g_bn_resident ? bnrelu_bwd_resident(d_x, d_dy, d_gamma, d_beta, d_stats, d_dx, d_addend, accumulate != 0,
                                                                 d_dgamma, d_dbeta, rows, C, d_scratch, st, nullptr)
                                          : cudaErrorNotSupported;
    if (res == cudaSuccess) return HPF_OK;
    if (res != cudaErrorNotSupported) CU(res);
    (void)cudaGetLastError();
    CU(bnrelu_bwd(d_x, d_dy, d_gamma, d_beta, d_stats, d_dx, d_addend, accumulate != 0, d_dgamma, d_dbeta, rows, C, d_scratch, st, nullptr));
    return HPF_OK;
}

int hpf_bnrelu_status(const void* d_scratch, int32_t* h_gave_up)
{
    if (!d_scratch || !h_gave_up) return fail(HPF_ERR_INVALID, "null argument");
    unsigned int words[3] = {0, 0, 0};
    CU(cudaMemcpy(words, d_scratch, sizeof words, cudaMemcpyDeviceToHost));
    *h_gave_up = words[2] != 0u;
    return HPF_OK;
}

int hpf_sgd_momentum_flat(const float* d_slots, float* d_grad_avg, float* d_params, float* d_velocity, int32_t M, int64_t G,
                          float lr, float momentum, float weight_decay, void* stream)
{
    if (!d_slots || !d_params || !d_velocity || M < 1 || G < 1) return fail(HPF_ERR_INVALID, "bad argument");
    CU(sgd_momentum(d_slots, d_grad_avg, d_params, d_velocity, M, G, lr, momentum, weight_decay, reinterpret_cast<cudaStream_t>(stream), nullptr));
    return HPF_OK;
}

int hpf_grad_average_flat(const float* d_slots, float* d_out, int32_t M, int64_t G, void* stream)
{
    if (!d_slots || !d_out || M < 1 || G < 1) return fail(HPF_ERR_INVALID, "bad argument");
    CU(grad_average(d_slots, d_out, M, G, reinterpret_cast<cudaStream_t>(stream), nullptr));
    return HPF_OK;
}

const char* hpf_strerror(int status)
{
    switch (status) {
    case HPF_OK: return "ok";
    case HPF_ERR_INVALID: return "invalid argument";
    case HPF_ERR_UNSUPPORTED: return "unsupported shape";
    case HPF_ERR_STATE: return "call out of order";
    case HPF_ERR_WORKSPACE: return "workspace too small or misaligned";
    case HPF_ERR_CUDA: return "CUDA error";
    case HPF_ERR_TIMEOUT: return "timeout";
    default: return "unknown status";
    }
}

const char* hpf_last_error(void) { return g_last_error.c_str(); }

}  // extern "C"
