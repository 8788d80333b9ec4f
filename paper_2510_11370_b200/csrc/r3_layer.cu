// The whole replayed layer as one enqueue: logits -> replay gate -> permute -> experts ->
// combine -> dgates -> dlogits (Section 4.1, Eqs. replay_gate / replay_output and the
// router-logit gradient), plus a variant whose per-step tensors live in host memory.
#include <mutex>

#include "r3_common.cuh"
#include "r3_internal.h"

namespace r3 {

// The router logits depend only on x and W_r, the permutation only on the record: the layer runs
// the former on a helper stream beside the latter.  One non-blocking helper stream and two events
// per device, created at the first call on that device and kept until the process exits; the
// helper is forked from and joined back into the caller's stream with the events, so the call as
// a whole is still ordered on the caller's stream (and can be captured with it).
constexpr int kHostChunksMax = 16;       // host-buffer entry point: token chunks in flight
constexpr int kHostChunkTokens = 8192;   // ... and their least size
struct SideStream {
    cudaStream_t stream = nullptr;
    cudaStream_t copy = nullptr;      // host-buffer entry point: inputs travel here beside the compute
    cudaStream_t copy_out = nullptr;  // ... and results back on this one
    cudaEvent_t fork = nullptr, join = nullptr, copy_fork = nullptr, copied = nullptr;
    cudaEvent_t in_ready[kHostChunksMax] = {}, done[kHostChunksMax] = {}, out_done = nullptr;
    int state = 0;                 // 0 = not tried, 1 = ready, -1 = unavailable
};
static SideStream* side_stream() {
    static SideStream per_device[64];
    static std::mutex mu;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    SideStream& ss = per_device[dev];
    if (ss.state == 0) {
        bool ok =
            cudaStreamCreateWithFlags(&ss.stream, cudaStreamNonBlocking) == cudaSuccess &&
            cudaStreamCreateWithFlags(&ss.copy, cudaStreamNonBlocking) == cudaSuccess &&
            cudaStreamCreateWithFlags(&ss.copy_out, cudaStreamNonBlocking) == cudaSuccess &&
            cudaEventCreateWithFlags(&ss.out_done, cudaEventDisableTiming) == cudaSuccess &&
            cudaEventCreateWithFlags(&ss.copy_fork, cudaEventDisableTiming) == cudaSuccess &&
            cudaEventCreateWithFlags(&ss.copied, cudaEventDisableTiming) == cudaSuccess &&
            cudaEventCreateWithFlags(&ss.fork, cudaEventDisableTiming) == cudaSuccess &&
            cudaEventCreateWithFlags(&ss.join, cudaEventDisableTiming) == cudaSuccess;
        for (int c = 0; ok && c < kHostChunksMax; ++c)
            ok = cudaEventCreateWithFlags(&ss.in_ready[c], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&ss.done[c], cudaEventDisableTiming) == cudaSuccess;
        ss.state = ok ? 1 : -1;
        if (!ok) cudaGetLastError();
    }
    return ss.state == 1 ? &ss : nullptr;
}

struct LayerWs {
    float* logits;
    float* gates;
    float* dgates;
    int32_t* counts;
    int32_t* offsets;
    int32_t* row_of_slot;
    int32_t* slot_of_row;
    void* xp;
    void* o;
    void* permute_ws;
    size_t permute_bytes;
    void* swiglu_ws;
    size_t swiglu_bytes;
    void* router_ws;
    size_t router_bytes;
    size_t total;
};

// Carves the workspace; with base == nullptr only the total size is meaningful.
static LayerWs carve(const r3_shape* s, void* base) {
    LayerWs w;
    size_t off = 0;
    char* b = static_cast<char*>(base);
    auto take = [&](size_t bytes) {
        void* p = b ? b + off : nullptr;
        off += round_up(bytes ? bytes : 1, 256);
        return p;
    };
    const size_t T = s->T, K = s->K, E = s->E, R = T * K;
    w.logits = static_cast<float*>(take(T * E * 4));
    w.gates = static_cast<float*>(take(R * 4));
    w.dgates = static_cast<float*>(take(R * 4));
    w.counts = static_cast<int32_t*>(take(E * 4));
    w.offsets = static_cast<int32_t*>(take((E + 1) * 4));
    w.row_of_slot = static_cast<int32_t*>(take(R * 4));
    w.slot_of_row = static_cast<int32_t*>(take(R * 4));
    w.xp = take(R * s->d * act_bytes(s));
    w.o = take(R * s->d * act_bytes(s));
    w.permute_bytes = r3_permute_workspace_bytes(s);
    w.permute_ws = take(w.permute_bytes);
    w.swiglu_bytes = r3_grouped_swiglu_workspace_bytes(s);
    w.swiglu_ws = take(w.swiglu_bytes);
    w.router_bytes = r3_capture_topk_workspace_bytes(s, 1);
    w.router_ws = w.router_bytes ? take(w.router_bytes) : nullptr;
    w.total = off;
    return w;
}

}  // namespace r3

extern "C" size_t r3_replay_layer_workspace_bytes(const r3_shape* shape) {
    if (r3::check_shape(shape) != R3_OK) return 0;
    return r3::carve(shape, nullptr).total;
}

namespace r3 {
// One replayed layer; `residual` (may be null) is added to the combined output.
static r3_status run_layer(const r3_shape* shape, const void* x, const void* w_router,
                           const void* idx, const void* w_gate, const void* w_up,
                           const void* w_down, const void* dy, const void* residual, void* y,
                           float* dlogits, float* gates_out, void* workspace,
                           int32_t* dev_status, void* stream, cudaEvent_t dy_ready = nullptr,
                           void* pre_gate = nullptr, void* pre_up = nullptr,
                           bool same_record = false) {
    // the helper stream's fork and join events are per device: one layer is enqueued at a time,
    // so that host threads calling at once cannot pair a wait with another call's record
    static std::mutex layer_mu;
    std::lock_guard<std::mutex> layer_lock(layer_mu);
    const LayerWs w = carve(shape, workspace);
    float* gates = gates_out ? gates_out : w.gates;
    r3_status st;
    // s_train = x W_r (only the logits are needed on the training side, and only by the last
    // kernel): on the helper stream, beside the permutation
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    SideStream* side = side_stream();
    if (side && (cudaEventRecord(side->fork, cs) != cudaSuccess ||
                 cudaStreamWaitEvent(side->stream, side->fork, 0) != cudaSuccess))
        return R3_ERR_CUDA;
    if ((st = r3_capture_topk_ws(shape, 1, x, w_router, nullptr, w.logits, w.router_ws,
                                 w.router_bytes, side ? side->stream : cs)) != R3_OK)
        return st;
    if (side && cudaEventRecord(side->join, side->stream) != cudaSuccess) return R3_ERR_CUDA;
    // K <= 8: gate, combine and both gradients in one pass over the expert outputs; wider records
    // take the four separate kernels (same results).
    const bool fused = shape->K <= 8;
    if (!fused) {
        if (side && cudaStreamWaitEvent(cs, side->join, 0) != cudaSuccess) return R3_ERR_CUDA;
        if ((st = r3_replay_gate_fwd(shape, w.logits, idx, gates, dev_status, stream)) != R3_OK)
            return st;
    }
    if (same_record) {
        // the maps and the GEMM work lists of the previous call on this workspace still hold:
        // only the rows are copied again
        if ((st = launch_permute_rows(shape, x, w.row_of_slot, w.xp, cs, dev_status)) != R3_OK) return st;
        st = grouped_swiglu_keep_lists(shape, w.xp, w.offsets, w_gate, w_up, w_down, w.o, pre_gate,
                                       pre_up, w.swiglu_ws, w.swiglu_bytes, dev_status, stream);
    } else {
        // a small batch is dispatched by one cluster launch, which then builds the experts' work
        // lists as well (one launch fewer in front of the GEMMs)
        WorkListSpec lists;
        const bool want = grouped_swiglu_list_spec(shape, w.swiglu_ws, &lists);
        bool built = false;
        if ((st = permute_impl(shape, idx, x, w.counts, w.offsets, w.row_of_slot, w.slot_of_row,
                               w.xp, w.permute_ws, w.permute_bytes, dev_status, stream,
                               want ? &lists : nullptr, &built)) != R3_OK)
            return st;
        if (built)
            st = grouped_swiglu_keep_lists(shape, w.xp, w.offsets, w_gate, w_up, w_down, w.o,
                                           pre_gate, pre_up, w.swiglu_ws, w.swiglu_bytes,
                                           dev_status, stream);
        else
            st = pre_gate ? r3_grouped_swiglu_train(shape, w.xp, w.offsets, w_gate, w_up, w_down,
                                                    w.o, pre_gate, pre_up, w.swiglu_ws,
                                                    w.swiglu_bytes, dev_status, stream)
                          : r3_grouped_swiglu(shape, w.xp, w.offsets, w_gate, w_up, w_down, w.o,
                                              w.swiglu_ws, w.swiglu_bytes, dev_status, stream);
    }
    if (st != R3_OK) return st;
    if (fused && side && cudaStreamWaitEvent(cs, side->join, 0) != cudaSuccess) return R3_ERR_CUDA;
    // dy is first needed here (host-buffer entry point: it may still be on its way)
    if (dy_ready && cudaStreamWaitEvent(cs, dy_ready, 0) != cudaSuccess) return R3_ERR_CUDA;
    if (fused)
        return r3_replay_finish(shape, w.logits, idx, w.o, w.row_of_slot, dy, residual, y,
                                gates_out, dlogits, dev_status, stream);
    if ((st = r3_combine_residual(shape, w.o, w.row_of_slot, gates, residual, y, stream)) != R3_OK)
        return st;
    if ((st = r3_combine_bwd_gates(shape, dy, w.o, w.row_of_slot, w.dgates, stream)) != R3_OK)
        return st;
    return r3_replay_gate_bwd(shape, gates, w.dgates, idx, dlogits, stream);
}
}  // namespace r3

extern "C" r3_status r3_replay_layer(const r3_shape* shape, const void* x, const void* w_router,
                                     const void* idx, const void* w_gate, const void* w_up,
                                     const void* w_down, const void* dy, void* y, float* dlogits,
                                     float* gates_out, void* workspace, size_t ws_bytes,
                                     int32_t* dev_status, void* stream) {
    r3_status st = r3::check_shape(shape);
    if (st != R3_OK) return st;
    if (shape->T == 0) return R3_OK;
    if (!x || !w_router || !idx || !w_gate || !w_up || !w_down || !dy || !y || !dlogits)
        return R3_ERR_INVALID_ARG;
    if (!workspace || !r3::aligned(workspace, 256) ||
        ws_bytes < r3_replay_layer_workspace_bytes(shape))
        return R3_ERR_WORKSPACE;
    return r3::run_layer(shape, x, w_router, idx, w_gate, w_up, w_down, dy, nullptr, y, dlogits,
                         gates_out, workspace, dev_status, stream);
}

extern "C" r3_status r3_replay_layer_same_record(const r3_shape* shape, const void* x,
                                                 const void* w_router, const void* idx,
                                                 const void* w_gate, const void* w_up,
                                                 const void* w_down, const void* dy, void* y,
                                                 float* dlogits, float* gates_out, void* workspace,
                                                 size_t ws_bytes, int32_t* dev_status,
                                                 void* stream) {
    r3_status st = r3::check_shape(shape);
    if (st != R3_OK) return st;
    if (shape->T == 0) return R3_OK;
    if (!x || !w_router || !idx || !w_gate || !w_up || !w_down || !dy || !y || !dlogits)
        return R3_ERR_INVALID_ARG;
    if (!workspace || !r3::aligned(workspace, 256) ||
        ws_bytes < r3_replay_layer_workspace_bytes(shape))
        return R3_ERR_WORKSPACE;
    return r3::run_layer(shape, x, w_router, idx, w_gate, w_up, w_down, dy, nullptr, y, dlogits,
                         gates_out, workspace, dev_status, stream, nullptr, nullptr, nullptr, true);
}

// ---- forward plus the backward to the layer input and the router weight ------------------------
namespace r3 {
struct TrainWs {
    void* inner; size_t inner_bytes;
    float* gates; void* pre_gate; void* pre_up; void* dxp; void* bwd_ws; size_t bwd_bytes;
    size_t total;
};
static TrainWs carve_train(const r3_shape* s, void* base) {
    TrainWs t;
    size_t off = 0;
    char* b = static_cast<char*>(base);
    auto take = [&](size_t bytes) {
        void* p = b ? b + off : nullptr;
        off += round_up(bytes ? bytes : 1, 256);
        return p;
    };
    const size_t R = (size_t)s->T * s->K;
    t.inner_bytes = r3_replay_layer_workspace_bytes(s);
    t.inner = take(t.inner_bytes);
    t.gates = static_cast<float*>(take(R * 4));
    t.pre_gate = take(R * s->F * act_bytes(s));
    t.pre_up = take(R * s->F * act_bytes(s));
    t.dxp = take(R * s->d * act_bytes(s));
    t.bwd_bytes = r3_grouped_swiglu_bwd_workspace_bytes(s);
    t.bwd_ws = take(t.bwd_bytes);
    t.total = off;
    return t;
}
}  // namespace r3

extern "C" size_t r3_replay_layer_train_workspace_bytes(const r3_shape* shape) {
    if (r3::check_shape(shape) != R3_OK || shape->act_dtype != R3_BF16) return 0;
    return r3::carve_train(shape, nullptr).total;
}

namespace r3 {
// Forward of one layer (pre-activations kept), then its backward.  `dres` (may be null) is the
// gradient that reaches x around the layer; the expert-weight outputs may all be null.
static r3_status run_layer_train(const r3_shape* shape, const void* x, const void* w_router,
                                 const void* idx, const void* w_gate, const void* w_up,
                                 const void* w_down, const void* dy, const void* dres, void* y,
                                 float* dlogits, void* dx, float* dw_router, float* dw_gate,
                                 float* dw_up, float* dw_down, void* workspace,
                                 int32_t* dev_status, void* stream) {
    const TrainWs t = carve_train(shape, workspace);
    const LayerWs w = carve(shape, t.inner);
    r3_status st = run_layer(shape, x, w_router, idx, w_gate, w_up, w_down, dy, nullptr, y,
                             dlogits, t.gates, t.inner, dev_status, stream, nullptr, t.pre_gate,
                             t.pre_up);
    if (st != R3_OK) return st;
    // the expert outputs are no longer needed: their buffer takes dout = g dy
    if ((st = r3_scale_rows(shape, dy, t.gates, w.row_of_slot, w.o, stream)) != R3_OK) return st;
    st = dw_gate ? r3_grouped_swiglu_bwd(shape, w.xp, w.o, t.pre_gate, t.pre_up, w.offsets, w_gate,
                                         w_up, w_down, t.dxp, dw_gate, dw_up, dw_down, t.bwd_ws,
                                         t.bwd_bytes, dev_status, stream)
                 : r3_grouped_swiglu_bwd_input(shape, w.o, t.pre_gate, t.pre_up, w.offsets, w_gate,
                                               w_up, w_down, t.dxp, t.bwd_ws, t.bwd_bytes,
                                               dev_status, stream);
    if (st != R3_OK) return st;
    return r3_input_grad_finish(shape, t.dxp, w.row_of_slot, w.slot_of_row, w.offsets, dlogits,
                                idx, x, w_router, dres, dx, dw_router, stream);
}
}  // namespace r3

extern "C" r3_status r3_replay_layer_train(const r3_shape* shape, const void* x,
                                           const void* w_router, const void* idx,
                                           const void* w_gate, const void* w_up,
                                           const void* w_down, const void* dy, void* y,
                                           float* dlogits, void* dx, float* dw_router,
                                           float* dw_gate, float* dw_up, float* dw_down,
                                           void* workspace, size_t ws_bytes, int32_t* dev_status,
                                           void* stream) {
    r3_status st = r3::check_shape(shape);
    if (st != R3_OK) return st;
    if (shape->act_dtype != R3_BF16) return R3_ERR_UNSUPPORTED;
    if (shape->T == 0) return R3_OK;
    if (!x || !w_router || !idx || !w_gate || !w_up || !w_down || !dy || !y || !dlogits || !dx ||
        !dw_router)
        return R3_ERR_INVALID_ARG;
    const bool weights = dw_gate || dw_up || dw_down;
    if (weights && (!dw_gate || !dw_up || !dw_down)) return R3_ERR_INVALID_ARG;
    if (!workspace || !r3::aligned(workspace, 256) ||
        ws_bytes < r3_replay_layer_train_workspace_bytes(shape))
        return R3_ERR_WORKSPACE;
    return r3::run_layer_train(shape, x, w_router, idx, w_gate, w_up, w_down, dy, nullptr, y,
                               dlogits, dx, dw_router, dw_gate, dw_up, dw_down, workspace,
                               dev_status, stream);
}

// ---- L residual blocks: forward, then the exact backward chain ---------------------------------
extern "C" size_t r3_replay_stack_train_workspace_bytes(const r3_shape* shape, int32_t L) {
    if (r3::check_shape(shape) != R3_OK || shape->act_dtype != R3_BF16 || L <= 0) return 0;
    const size_t xb = r3::round_up((size_t)shape->T * shape->d * r3::act_bytes(shape), 256);
    return ((size_t)L + 3) * xb + r3_replay_layer_train_workspace_bytes(shape);
}

extern "C" r3_status r3_replay_stack_train(const r3_shape* shape, int32_t L, const void* x0,
                                           const void* w_router, const void* idx,
                                           const void* w_gate, const void* w_up,
                                           const void* w_down, const void* dy, void* x_out,
                                           float* dlogits, void* dx0, float* dw_router,
                                           float* dw_gate, float* dw_up, float* dw_down,
                                           void* workspace, size_t ws_bytes, int32_t* dev_status,
                                           void* stream) {
    r3_status st = r3::check_shape(shape);
    if (st != R3_OK) return st;
    if (shape->act_dtype != R3_BF16) return R3_ERR_UNSUPPORTED;
    if (L <= 0) return R3_ERR_INVALID_ARG;
    if (shape->T == 0) return R3_OK;
    if (!x0 || !w_router || !idx || !w_gate || !w_up || !w_down || !dy || !x_out || !dlogits ||
        !dx0 || !dw_router || dx0 == dy)
        return R3_ERR_INVALID_ARG;
    const bool weights = dw_gate || dw_up || dw_down;
    if (weights && (!dw_gate || !dw_up || !dw_down)) return R3_ERR_INVALID_ARG;
    if (!workspace || !r3::aligned(workspace, 256) ||
        ws_bytes < r3_replay_stack_train_workspace_bytes(shape, L))
        return R3_ERR_WORKSPACE;
    const size_t T = shape->T, d = shape->d, E = shape->E, F = shape->F, K = shape->K;
    const size_t es = r3::act_bytes(shape);
    const size_t xb = r3::round_up(T * d * es, 256);
    char* ws = static_cast<char*>(workspace);
    // x_1 .. x_{L-1} are kept for the backward pass (x_0 is the caller's, x_L goes to x_out)
    auto kept = [&](int32_t l) { return static_cast<void*>(ws + (size_t)l * xb); };
    void* grad[2] = {ws + (size_t)L * xb, ws + ((size_t)L + 1) * xb};
    void* y_scratch = ws + ((size_t)L + 2) * xb;
    void* inner = ws + ((size_t)L + 3) * xb;
    const size_t rw = E * d * (shape->router_w_dtype == R3_BF16 ? 2 : 4);
    const size_t ew = E * F * d * es, rec = T * K * r3::idx_bytes(shape);
    auto at = [](const void* p, size_t off) { return static_cast<const char*>(p) + off; };
    const void* cur = x0;
    for (int32_t l = 0; l < L; ++l) {
        void* nxt = (l == L - 1) ? x_out : kept(l + 1);
        st = r3::run_layer(shape, cur, at(w_router, l * rw), at(idx, l * rec), at(w_gate, l * ew),
                           at(w_up, l * ew), at(w_down, l * ew), dy, cur, nxt,
                           dlogits + (size_t)l * T * E, nullptr, inner, dev_status, stream);
        if (st != R3_OK) return st;
        cur = nxt;
    }
    // g_L = dy;  g_l = g_{l+1} + (gradient through block l at x_l), block l's forward recomputed
    const void* g = dy;
    for (int32_t l = L - 1; l >= 0; --l) {
        const void* xl = l == 0 ? x0 : kept(l);
        void* g_out = l == 0 ? dx0 : grad[l & 1];
        st = r3::run_layer_train(shape, xl, at(w_router, l * rw), at(idx, l * rec),
                                 at(w_gate, l * ew), at(w_up, l * ew), at(w_down, l * ew), g, g,
                                 y_scratch, dlogits + (size_t)l * T * E, g_out,
                                 dw_router + (size_t)l * E * d,
                                 weights ? dw_gate + (size_t)l * E * F * d : nullptr,
                                 weights ? dw_up + (size_t)l * E * F * d : nullptr,
                                 weights ? dw_down + (size_t)l * E * F * d : nullptr, inner,
                                 dev_status, stream);
        if (st != R3_OK) return st;
        g = g_out;
    }
    return R3_OK;
}

// ---- a stack of L replayed MoE blocks with residual connections ------------------------------
extern "C" size_t r3_replay_stack_workspace_bytes(const r3_shape* shape) {
    if (r3::check_shape(shape) != R3_OK) return 0;
    const size_t xb = r3::round_up((size_t)shape->T * shape->d * r3::act_bytes(shape), 256);
    return 2 * xb + r3_replay_layer_workspace_bytes(shape);
}

extern "C" r3_status r3_replay_stack(const r3_shape* shape, int32_t L, const void* x0,
                                     const void* w_router, const void* idx, const void* w_gate,
                                     const void* w_up, const void* w_down, const void* dy,
                                     void* x_out, float* dlogits, void* workspace, size_t ws_bytes,
                                     int32_t* dev_status, void* stream) {
    r3_status st = r3::check_shape(shape);
    if (st != R3_OK) return st;
    if (L <= 0) return R3_ERR_INVALID_ARG;
    if (shape->T == 0) return R3_OK;
    if (!x0 || !w_router || !idx || !w_gate || !w_up || !w_down || !dy || !x_out || !dlogits)
        return R3_ERR_INVALID_ARG;
    if (!workspace || !r3::aligned(workspace, 256) ||
        ws_bytes < r3_replay_stack_workspace_bytes(shape))
        return R3_ERR_WORKSPACE;
    const size_t T = shape->T, d = shape->d, E = shape->E, F = shape->F, K = shape->K;
    const size_t es = r3::act_bytes(shape);
    const size_t xb = r3::round_up(T * d * es, 256);
    char* ws = static_cast<char*>(workspace);
    void* ping[2] = {ws, ws + xb};
    void* inner = ws + 2 * xb;
    const size_t rw = E * d * (shape->router_w_dtype == R3_BF16 ? 2 : 4);
    const char* wr = static_cast<const char*>(w_router);
    const char* wg = static_cast<const char*>(w_gate);
    const char* wu = static_cast<const char*>(w_up);
    const char* wd = static_cast<const char*>(w_down);
    const char* rec = static_cast<const char*>(idx);
    const void* cur = x0;
    for (int32_t l = 0; l < L; ++l) {
        void* nxt = (l == L - 1) ? x_out : ping[l & 1];
        // x_{l+1} = x_l + y_l : the block input is also the residual
        st = r3::run_layer(shape, cur, wr + (size_t)l * rw, rec + (size_t)l * T * K * r3::idx_bytes(shape),
                           wg + (size_t)l * E * F * d * es, wu + (size_t)l * E * F * d * es,
                           wd + (size_t)l * E * d * F * es, dy, cur, nxt,
                           dlogits + (size_t)l * T * E, nullptr, inner, dev_status, stream);
        if (st != R3_OK) return st;
        cur = nxt;
    }
    return R3_OK;
}

// ---- L independent replayed MoE blocks (each with its own input) -----------------------------
extern "C" r3_status r3_replay_blocks(const r3_shape* shape, int32_t L, const void* x,
                                      const void* w_router, const void* idx, const void* w_gate,
                                      const void* w_up, const void* w_down, const void* dy,
                                      void* y, float* dlogits, void* workspace, size_t ws_bytes,
                                      int32_t* dev_status, void* stream) {
    r3_status st = r3::check_shape(shape);
    if (st != R3_OK) return st;
    if (L <= 0) return R3_ERR_INVALID_ARG;
    if (shape->T == 0) return R3_OK;
    if (!x || !w_router || !idx || !w_gate || !w_up || !w_down || !dy || !y || !dlogits)
        return R3_ERR_INVALID_ARG;
    if (!workspace || !r3::aligned(workspace, 256) ||
        ws_bytes < r3_replay_layer_workspace_bytes(shape))
        return R3_ERR_WORKSPACE;
    const size_t T = shape->T, d = shape->d, E = shape->E, F = shape->F, K = shape->K;
    const size_t es = r3::act_bytes(shape);
    const size_t rw = E * d * (shape->router_w_dtype == R3_BF16 ? 2 : 4);
    const size_t act = T * d * es, ew = E * F * d * es;
    for (int32_t l = 0; l < L; ++l) {
        st = r3::run_layer(shape, static_cast<const char*>(x) + l * act,
                           static_cast<const char*>(w_router) + l * rw,
                           static_cast<const char*>(idx) + l * T * K * r3::idx_bytes(shape),
                           static_cast<const char*>(w_gate) + l * ew,
                           static_cast<const char*>(w_up) + l * ew,
                           static_cast<const char*>(w_down) + l * ew,
                           static_cast<const char*>(dy) + l * act, nullptr,
                           static_cast<char*>(y) + l * act, dlogits + l * T * E, nullptr,
                           workspace, dev_status, stream);
        if (st != R3_OK) return st;
    }
    return R3_OK;
}

namespace r3 {
struct HostWs {
    void* x; void* idx; void* dy; void* y; float* dlogits; void* inner; size_t inner_bytes;
    size_t total;
};
static HostWs carve_host(const r3_shape* s, void* base) {
    HostWs h;
    size_t off = 0;
    char* b = static_cast<char*>(base);
    auto take = [&](size_t bytes) {
        void* p = b ? b + off : nullptr;
        off += round_up(bytes ? bytes : 1, 256);
        return p;
    };
    const size_t T = s->T, row = (size_t)s->d * act_bytes(s);
    h.x = take(T * row);
    h.idx = take(T * s->K * idx_bytes(s));
    h.dy = take(T * row);
    h.y = take(T * row);
    h.dlogits = static_cast<float*>(take(T * s->E * 4));
    h.inner_bytes = r3_replay_layer_workspace_bytes(s);
    h.inner = take(h.inner_bytes);
    h.total = off;
    return h;
}
// Token chunks of the host-buffer call: starts[0..n] with starts[n] = T; n = 1 below
// 2 * kHostChunkTokens tokens.  Equal chunks of at least kHostChunkTokens tokens (a multiple of
// 256, at most 12 of them), except that the last one is cut into a half and two quarters: what the
// call cannot hide is the compute and the result copy of its LAST chunk, so that one is small.
static int host_chunks(int64_t T, int64_t* starts) {
    starts[0] = 0;
    if (T < 2 * (int64_t)kHostChunkTokens) {
        starts[1] = T;
        return 1;
    }
    int64_t chunk = ((T + 11) / 12 + 255) / 256 * 256;
    if (chunk < kHostChunkTokens) chunk = kHostChunkTokens;
    int n = 0;
    int64_t t = 0;
    while (T - t > chunk) {
        t += chunk;
        starts[++n] = t;
    }
    const int64_t rest = T - t;                      // 1 .. chunk tokens
    if (rest >= 4096) {
        const int64_t half = rest / 2 / 256 * 256, quarter = rest / 4 / 256 * 256;
        starts[++n] = t + half;
        starts[++n] = t + half + quarter;
    }
    starts[++n] = T;
    return n;
}
}  // namespace r3

extern "C" int32_t r3_replay_layer_host_chunks(const r3_shape* shape, int64_t* starts) {
    if (r3::check_shape(shape) != R3_OK || !starts) return 0;
    return r3::host_chunks(shape->T, starts);
}

extern "C" size_t r3_replay_layer_host_workspace_bytes(const r3_shape* shape) {
    if (r3::check_shape(shape) != R3_OK) return 0;
    return r3::carve_host(shape, nullptr).total;
}

extern "C" r3_status r3_replay_layer_host_enqueue(const r3_shape* shape, const void* x_host,
                                                  const void* w_router, const void* idx_host,
                                                  const void* w_gate, const void* w_up,
                                                  const void* w_down, const void* dy_host,
                                                  void* y_host, float* dlogits_host,
                                                  void* workspace, size_t ws_bytes,
                                                  int32_t* dev_status, void* stream) {
    r3_status st = r3::check_shape(shape);
    if (st != R3_OK) return st;
    if (shape->T == 0) return R3_OK;
    if (!x_host || !idx_host || !dy_host || !y_host || !dlogits_host) return R3_ERR_INVALID_ARG;
    if (!workspace || !r3::aligned(workspace, 256) ||
        ws_bytes < r3_replay_layer_host_workspace_bytes(shape))
        return R3_ERR_WORKSPACE;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const r3::HostWs h = r3::carve_host(shape, workspace);
    const size_t T = shape->T, row = (size_t)shape->d * r3::act_bytes(shape);
    if (!x_host || !w_router || !w_gate || !w_up || !w_down) return R3_ERR_INVALID_ARG;
    r3::SideStream* side = r3::side_stream();
    if (side && T >= 2 * (size_t)r3::kHostChunkTokens) {
        // A large batch goes through in chunks of tokens (every step of the layer is per token once
        // the record is given, so the chunks are layers of their own): chunk c + 1 crosses the link
        // while chunk c computes and chunk c - 1 returns, so the call takes about the time of its
        // host-to-device bytes instead of the sum of copies and compute.
        // the events below belong to the device, not to the call: one enqueue at a time, so that
        // every wait is paired with the record of its own call
        static std::mutex enqueue_mu;
        std::lock_guard<std::mutex> lock(enqueue_mu);
        int64_t starts[r3::kHostChunksMax + 1];
        const int n_chunks = r3::host_chunks((int64_t)T, starts);
        const size_t idx_row = (size_t)shape->K * r3::idx_bytes(shape);
        if (cudaEventRecord(side->copy_fork, cs) != cudaSuccess ||
            cudaStreamWaitEvent(side->copy, side->copy_fork, 0) != cudaSuccess ||
            cudaStreamWaitEvent(side->copy_out, side->copy_fork, 0) != cudaSuccess)
            return R3_ERR_CUDA;
        for (int c = 0; c < n_chunks; ++c) {
            const size_t t0 = (size_t)starts[c], n = (size_t)(starts[c + 1] - starts[c]);
            if (cudaMemcpyAsync(static_cast<char*>(h.x) + t0 * row,
                                static_cast<const char*>(x_host) + t0 * row, n * row,
                                cudaMemcpyHostToDevice, side->copy) != cudaSuccess ||
                cudaMemcpyAsync(static_cast<char*>(h.idx) + t0 * idx_row,
                                static_cast<const char*>(idx_host) + t0 * idx_row, n * idx_row,
                                cudaMemcpyHostToDevice, side->copy) != cudaSuccess ||
                cudaMemcpyAsync(static_cast<char*>(h.dy) + t0 * row,
                                static_cast<const char*>(dy_host) + t0 * row, n * row,
                                cudaMemcpyHostToDevice, side->copy) != cudaSuccess ||
                cudaEventRecord(side->in_ready[c], side->copy) != cudaSuccess)
                return R3_ERR_CUDA;
        }
        for (int c = 0; c < n_chunks; ++c) {
            const size_t t0 = (size_t)starts[c], n = (size_t)(starts[c + 1] - starts[c]);
            r3_shape part = *shape;
            part.T = (int32_t)n;
            if (cudaStreamWaitEvent(cs, side->in_ready[c], 0) != cudaSuccess) return R3_ERR_CUDA;
            st = r3::run_layer(&part, static_cast<char*>(h.x) + t0 * row, w_router,
                               static_cast<char*>(h.idx) + t0 * idx_row, w_gate, w_up, w_down,
                               static_cast<char*>(h.dy) + t0 * row, nullptr,
                               static_cast<char*>(h.y) + t0 * row, h.dlogits + t0 * shape->E,
                               nullptr, h.inner, dev_status, stream);
            if (st != R3_OK) return st;
            if (cudaEventRecord(side->done[c], cs) != cudaSuccess ||
                cudaStreamWaitEvent(side->copy_out, side->done[c], 0) != cudaSuccess ||
                cudaMemcpyAsync(static_cast<char*>(y_host) + t0 * row,
                                static_cast<char*>(h.y) + t0 * row, n * row,
                                cudaMemcpyDeviceToHost, side->copy_out) != cudaSuccess ||
                cudaMemcpyAsync(dlogits_host + t0 * shape->E, h.dlogits + t0 * shape->E,
                                n * shape->E * 4, cudaMemcpyDeviceToHost, side->copy_out) !=
                    cudaSuccess)
                return R3_ERR_CUDA;
        }
        // the caller's stream ends behind the last result copy
        if (cudaEventRecord(side->out_done, side->copy_out) != cudaSuccess ||
            cudaStreamWaitEvent(cs, side->out_done, 0) != cudaSuccess)
            return R3_ERR_CUDA;
        return R3_OK;
    }
    if (cudaMemcpyAsync(h.x, x_host, T * row, cudaMemcpyHostToDevice, cs) != cudaSuccess ||
        cudaMemcpyAsync(h.idx, idx_host, T * shape->K * r3::idx_bytes(shape),
                        cudaMemcpyHostToDevice, cs) != cudaSuccess)
        return R3_ERR_CUDA;
    // x and the record are needed at once; dy only by the last kernel: it follows x over the
    // link on a copy stream of its own while the layer computes
    cudaEvent_t dy_ready = nullptr;
    if (side) {
        if (cudaEventRecord(side->copy_fork, cs) != cudaSuccess ||
            cudaStreamWaitEvent(side->copy, side->copy_fork, 0) != cudaSuccess ||
            cudaMemcpyAsync(h.dy, dy_host, T * row, cudaMemcpyHostToDevice, side->copy) !=
                cudaSuccess ||
            cudaEventRecord(side->copied, side->copy) != cudaSuccess)
            return R3_ERR_CUDA;
        dy_ready = side->copied;
    } else if (cudaMemcpyAsync(h.dy, dy_host, T * row, cudaMemcpyHostToDevice, cs) != cudaSuccess) {
        return R3_ERR_CUDA;
    }
    st = r3::run_layer(shape, h.x, w_router, h.idx, w_gate, w_up, w_down, h.dy, nullptr, h.y,
                       h.dlogits, nullptr, h.inner, dev_status, stream, dy_ready);
    if (st != R3_OK) return st;
    if (cudaMemcpyAsync(y_host, h.y, T * row, cudaMemcpyDeviceToHost, cs) != cudaSuccess ||
        cudaMemcpyAsync(dlogits_host, h.dlogits, T * shape->E * 4, cudaMemcpyDeviceToHost, cs) !=
            cudaSuccess)
        return R3_ERR_CUDA;
    return R3_OK;
}

extern "C" r3_status r3_replay_layer_host(const r3_shape* shape, const void* x_host,
                                          const void* w_router, const void* idx_host,
                                          const void* w_gate, const void* w_up,
                                          const void* w_down, const void* dy_host, void* y_host,
                                          float* dlogits_host, void* workspace, size_t ws_bytes,
                                          int32_t* dev_status, void* stream) {
    const r3_status st = r3_replay_layer_host_enqueue(shape, x_host, w_router, idx_host, w_gate,
                                                      w_up, w_down, dy_host, y_host, dlogits_host,
                                                      workspace, ws_bytes, dev_status, stream);
    if (st != R3_OK || shape->T == 0) return st;
    return cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) == cudaSuccess ? R3_OK
                                                                                   : R3_ERR_CUDA;
}

extern "C" const char* r3_status_string(r3_status s) {
    switch (s) {
        case R3_OK: return "R3_OK";
        case R3_ERR_INVALID_ARG: return "R3_ERR_INVALID_ARG: null pointer, bad size or dtype code";
        case R3_ERR_UNSUPPORTED: return "R3_ERR_UNSUPPORTED: no kernel for this shape";
        case R3_ERR_WORKSPACE: return "R3_ERR_WORKSPACE: workspace missing, too small or misaligned";
        case R3_ERR_CUDA: return "R3_ERR_CUDA: a CUDA call failed";
        case R3_ERR_OUT_OF_PAGES: return "R3_ERR_OUT_OF_PAGES: not enough free record pages";
        case R3_ERR_SCRATCH_LIMIT:
            return "R3_ERR_SCRATCH_LIMIT: E * ceil(T/256) exceeds the 262144 counters of the "
                   "library's fixed scratch; use r3_permute with a caller workspace";
    }
    return "unknown r3_status";
}
