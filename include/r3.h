/*
 * r3.h - C ABI of the replayed-routing MoE layer (Rollout Routing Replay, "R3") for NVIDIA B200.
 *
 * The library evaluates one Mixture-of-Experts layer whose expert selection is REPLAYED from a
 * record made by an inference engine, as defined in Section 4.1 of the paper
 * "Stabilizing MoE Reinforcement Learning by Aligning Training and Inference Routers":
 *
 *   s        = x W_r                                            (router logits, first equation)
 *   I        = TopKMask(s, K)                                   (second equation; capture side)
 *   g_i      = I_infer,i exp(s_train,i) / sum_j I_infer,j exp(s_train,j)      (Eq. replay_gate)
 *   y        = sum_i g_i E_i(x_train)                                          (Eq. replay_output)
 *
 * plus the gradient of a loss with respect to s_train through the replayed gate (the mask is a
 * constant; Section 4.1, purpose (b)).  The expert network E_i is a bias-free SwiGLU feed-forward
 * network of width F:  E_i(x) = W_down,i ( silu(W_gate,i x) * (W_up,i x) ).
 *
 * Notation: T tokens, d hidden size, E (= M) experts, K experts per token, R = T*K rows.
 *
 * General rules
 *  - Every pointer is a DEVICE pointer owned by the caller unless the parameter is documented as
 *    "host".  The library never allocates, frees or synchronises (except r3_replay_layer_host,
 *    which synchronises the stream before it returns); each call enqueues its kernels on
 *    `stream` (a cudaStream_t passed as void*; NULL = the legacy default stream) and returns.
 *    r3_replay_layer and the entry points built on it (_host, _blocks, _stack) also use one
 *    internal non-blocking helper stream per device, created at the first such call on that
 *    device and kept until the process exits: the router logits run there beside the
 *    permutation.  The helper is forked from and joined back into `stream` with events, so the
 *    call as a whole is ordered on `stream` exactly as if everything had been enqueued there.
 *    Host threads may call at once: the enqueue of a layer takes a process-wide lock for its
 *    few microseconds, because the helper streams and their events belong to the device.
 *  - Matrices are row-major and dense.  Weights are stored output-major: W_r [E, d],
 *    W_gate/W_up [E, F, d], W_down [E, d, F].
 *  - Activations and expert weights have dtype `act_dtype` (R3_F32 or R3_BF16); W_r has dtype
 *    `router_w_dtype`; logits, gates and their gradients are always float32.  All accumulation is
 *    float32.
 *  - The routing record holds K expert indices per token, `idx_type` R3_IDX_U8 (E <= 256) or
 *    R3_IDX_I16 (E <= 32767), laid out [layer][token][slot].  Replay accepts the K indices of a
 *    token in any order; gates are returned in the same slot order.
 *  - Alignment: all base pointers 16-byte aligned, workspaces 256-byte aligned; d and F
 *    multiples of 8.
 *  - Errors the host can see (null pointer, bad shape, workspace too small, failed launch) are
 *    returned as r3_status and nothing is launched.  Data-dependent problems (index out of range,
 *    duplicate index within a token, an internal wait that ran out) are written to the optional
 *    device word `dev_status` (first error wins; 0 = clean; the caller zeroes it); kernels never
 *    trap, and skip the offending element.
 *  - T = 0 returns R3_OK without launching.  Experts with no rows are legal.
 *  - Results are bit-reproducible from run to run: no floating-point atomics are used anywhere.
 *  - Host threads: the library keeps small host-side caches (encoded tensor maps, per-kernel
 *    attributes, the helper stream).  Calls from several host threads must be serialised by the
 *    caller; one process per GPU with one calling thread is the intended use.
 */
#ifndef R3_H_
#define R3_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    R3_OK = 0,
    R3_ERR_INVALID_ARG = 1,   /* null pointer, non-positive size, K > E, index type too narrow */
    R3_ERR_UNSUPPORTED = 2,   /* a legal shape the library has no kernel for */
    R3_ERR_WORKSPACE = 3,     /* workspace missing, too small or misaligned */
    R3_ERR_CUDA = 4,          /* a CUDA runtime/driver call failed (launch, tensor-map encode) */
    R3_ERR_SCRATCH_LIMIT = 5, /* the problem needs more than the library's fixed on-device scratch */
    R3_ERR_OUT_OF_PAGES = 6   /* r3_pagepool_alloc: fewer free pages than asked for */
} r3_status;

enum { R3_F32 = 0, R3_BF16 = 1 };
enum { R3_IDX_U8 = 1, R3_IDX_I16 = 2 };

/* values written to *dev_status by kernels */
enum { R3_DEV_OK = 0, R3_DEV_BAD_INDEX = 1, R3_DEV_DUP_INDEX = 2, R3_DEV_TIMEOUT = 3 };

typedef struct {
    int32_t T, d, E, K, F;
    int32_t act_dtype;        /* R3_F32 | R3_BF16 : x, dy, xp, h, o, y, expert weights */
    int32_t router_w_dtype;   /* R3_F32 | R3_BF16 : W_r */
    int32_t idx_type;         /* R3_IDX_U8 | R3_IDX_I16 */
} r3_shape;

const char* r3_status_string(r3_status s);

/* Section 4.1, first and second equations: router logits and TopKMask, fused.
 *   s[t,i] = sum_c x[t,c] W_r[i,c];  idx_out[t, 0..K) = the K experts with the largest s[t,.],
 *   slot order = descending logit, exact ties to the lower expert index.
 * x [T,d] act_dtype; w_router [E,d] router_w_dtype; idx_out [T,K] idx_type (may be NULL when only
 * logits are wanted); logits_out [T,E] float32 or NULL.  At least one output must be non-NULL.
 * Used on the inference side to make the record, and on the training side (logits_out set) for
 * s_train.  bf16 activations with bf16 router weights (E a multiple of 16 up to 256, K <= 16)
 * run on the tensor cores; other combinations use a float32 FMA kernel (E <= 512). */
r3_status r3_capture_topk(const r3_shape* shape, const void* x, const void* w_router,
                          void* idx_out, float* logits_out, void* stream);

/* The same for L independent layers in one launch sequence: x [L,T,d], w_router [L,E,d],
 * idx_out [L,T,K], logits_out [L,T,E] or NULL. */
r3_status r3_capture_topk_batched(const r3_shape* shape, int32_t L, const void* x,
                                  const void* w_router, void* idx_out, float* logits_out,
                                  void* stream);

/* The same with caller scratch, which lets float32 router weights use the tensor cores too: the
 * weights are split into three bf16 planes (hi + mid + lo = all 24 mantissa bits) in the
 * workspace and the three products are accumulated in fp32, so the logits keep float32-level
 * accuracy.  workspace: r3_capture_topk_workspace_bytes(shape, L) bytes (0 when none is needed:
 * bf16 router weights, or a shape the tensor-core kernel does not cover).  Without a workspace
 * (or through r3_capture_topk / _batched) float32 router weights take the float32 FMA kernel.
 * Tensor-core kernel: bf16 activations, E a multiple of 16 up to 256, K <= 16. */
size_t r3_capture_topk_workspace_bytes(const r3_shape* shape, int32_t L);
r3_status r3_capture_topk_ws(const r3_shape* shape, int32_t L, const void* x,
                             const void* w_router, void* idx_out, float* logits_out,
                             void* workspace, size_t ws_bytes, void* stream);

/* Eq. (replay_gate): softmax of the TRAINING logits over the K RECORDED experts.
 *   gates[t,j] = exp(s[t,e_j] - m) / sum_j' exp(s[t,e_j'] - m),  e_j = idx[t,j], m = max_j s[t,e_j]
 * logits [T,E] f32; idx [T,K]; gates [T,K] f32 (slot-aligned with idx).
 * dev_status (optional): R3_DEV_BAD_INDEX / R3_DEV_DUP_INDEX if a token's record is invalid; the
 * gates of such a token are written as 0. */
r3_status r3_replay_gate_fwd(const r3_shape* shape, const float* logits, const void* idx,
                             float* gates, int32_t* dev_status, void* stream);

/* Gradient through Eq. (replay_gate) with the mask held constant:
 *   c = sum_j g[t,j] dg[t,j];  dlogits[t,e_j] = g[t,j] (dg[t,j] - c);  dlogits[t,i] = 0 elsewhere.
 * gates, dgates [T,K] f32; idx [T,K]; dlogits [T,E] f32, every element written; a dlogits that is
 * not 16-byte aligned returns R3_ERR_INVALID_ARG. */
r3_status r3_replay_gate_bwd(const r3_shape* shape, const float* gates, const float* dgates,
                             const void* idx, float* dlogits, void* stream);

/* Token dispatch implied by Eq. (replay_output): expert i is evaluated only on tokens whose
 * recorded mask has I_i = 1.  The R (token, slot) pairs are grouped by expert, stably (within an
 * expert, ascending token).
 *   counts[e]        = number of pairs with idx = e                       [E]   int32
 *   offsets          = exclusive scan of counts, offsets[E] = R           [E+1] int32
 *   row_of_slot[t,j] = destination row of pair (t,j)                      [T,K] int32
 *   slot_of_row[r]   = t*K + j of the pair stored in row r                [R]   int32
 *   xp[r]            = x[slot_of_row[r] / K]                              [R,d] act_dtype
 * x / xp may both be NULL to compute the maps only.  Integer outputs are exact and independent of
 * scheduling.  workspace: r3_permute_workspace_bytes(shape) bytes.  Supported: E <= 1024.
 * dev_status (optional): R3_DEV_BAD_INDEX for an index >= E (that pair is dropped). */
size_t r3_permute_workspace_bytes(const r3_shape* shape);
r3_status r3_permute(const r3_shape* shape, const void* idx, const void* x, int32_t* counts,
                     int32_t* offsets, int32_t* row_of_slot, int32_t* slot_of_row, void* xp,
                     void* workspace, size_t ws_bytes, int32_t* dev_status, void* stream);

/* r3_permute without a caller-supplied workspace (the paper has no counterpart; this exists for
 * the integration, not for the method).  Meant for callers that cannot allocate device memory at
 * the point of the call: for example a host process whose whole device-memory budget belongs to
 * another component's pool, where a fresh driver allocation may fail or stall the device, or a
 * step whose memory plan was fixed in advance.  The scratch (per-expert, per-256-token-chunk
 * counters) lives in a fixed array inside the library, 1 MiB on every GPU that loads the library,
 * held until the process exits.  Inputs and outputs are the caller's, exactly as for r3_permute,
 * and the results are identical to r3_permute's.
 *  - Limit: E * ceil(T / 256) <= 262144 (e.g. E = 128 up to T = 524288); beyond it the call
 *    returns R3_ERR_SCRATCH_LIMIT and launches nothing.  E <= 1024 as for r3_permute.
 *  - The call itself allocates and frees nothing, on the host or on the device.
 *  - The first call on each device looks up the array's device address (with that device
 *    current) and caches it; make that first call outside any stream capture.
 *  - Every call uses the same array, and it keeps the previous call's contents (no part of it
 *    has to be cleared: each call overwrites all the counters it later reads).  Calls that may
 *    overlap on the GPU - different streams or host threads - race on it; serialise them. */
r3_status r3_permute_static(const r3_shape* shape, const void* idx, const void* x, int32_t* counts,
                            int32_t* offsets, int32_t* row_of_slot, int32_t* slot_of_row,
                            void* xp, int32_t* dev_status, void* stream);

/* Expert networks E_i on the grouped rows: for expert e and rows r in [offsets[e], offsets[e+1])
 *   h[r] = silu(xp[r] W_gate,e^T) * (xp[r] W_up,e^T);   o[r] = h[r] W_down,e^T.
 * xp [R,d]; offsets [E+1]; w_gate, w_up [E,F,d]; w_down [E,d,F]; o [R,d]; all act_dtype.
 * bf16: tcgen05 tensor-core grouped GEMMs with fp32 accumulation, h and o rounded to bf16.
 * f32:  plain fp32 FMA kernels.
 * workspace: r3_grouped_swiglu_workspace_bytes(shape) bytes (holds h [R,F] and the tile list).
 * dev_status (optional): R3_DEV_TIMEOUT if an internal bounded wait ran out (outputs invalid). */
size_t r3_grouped_swiglu_workspace_bytes(const r3_shape* shape);
r3_status r3_grouped_swiglu(const r3_shape* shape, const void* xp, const int32_t* offsets,
                            const void* w_gate, const void* w_up, const void* w_down, void* o,
                            void* workspace, size_t ws_bytes, int32_t* dev_status, void* stream);

/* r3_grouped_swiglu without the permuted copy of the activations: the token operand of the up
 * projection is read in place from x [T,d], row slot_of_row[r] / K for grouped row r (Eq.
 * (replay_output): expert i sees exactly the tokens whose recorded mask has I_i = 1), so
 * r3_permute can be called with x = xp = NULL and the R x d buffer never exists.  Results are
 * bit-identical to r3_grouped_swiglu on xp[r] = x[slot_of_row[r] / K].  The rows arrive through
 * four-row TMA gather copies, which on B200 run well below the rate of the tiled copies of the
 * permuted form (measured: the up projection takes about 2.8x as long), so this form is for
 * callers short of memory, not of time; r3_replay_layer uses the permuted copy.  bf16 only
 * (R3_ERR_UNSUPPORTED for float32).  slot_of_row [R] and offsets [E+1] as written by r3_permute;
 * workspace and dev_status as for r3_grouped_swiglu. */
r3_status r3_grouped_swiglu_gather(const r3_shape* shape, const void* x, const int32_t* slot_of_row,
                                   const int32_t* offsets, const void* w_gate, const void* w_up,
                                   const void* w_down, void* o, void* workspace, size_t ws_bytes,
                                   int32_t* dev_status, void* stream);

/* The two halves of r3_grouped_swiglu as separate calls (same kernels, same workspace), so that a
 * caller can place other work, or timing events, between them:
 *   r3_expert_up_swiglu : builds the tile list from offsets and writes h = silu(xp Wg^T)*(xp Wu^T)
 *                         into the workspace;
 *   r3_expert_down      : o = h W_down^T, reading h and the tile list that the preceding
 *                         r3_expert_up_swiglu call left in the SAME workspace.
 * Expert network E_i of Eq. (replay_output); argument rules as for r3_grouped_swiglu. */
r3_status r3_expert_up_swiglu(const r3_shape* shape, const void* xp, const int32_t* offsets,
                              const void* w_gate, const void* w_up, void* workspace,
                              size_t ws_bytes, int32_t* dev_status, void* stream);
r3_status r3_expert_down(const r3_shape* shape, const void* w_down, void* o, void* workspace,
                         size_t ws_bytes, int32_t* dev_status, void* stream);

/* Eq. (replay_output): y[t] = sum_{j=0..K-1} gates[t,j] * o[row_of_slot[t,j]], added in slot
 * order in fp32 (no atomics), rounded once to act_dtype.  o [R,d]; y [T,d].
 * r3_combine, r3_combine_residual and r3_combine_bwd_gates take no dev_status word: should one of
 * their internal bounded waits ever run out, the affected token's output is left unwritten without
 * a report.  r3_replay_finish (what the layer runs) computes the same values and reports
 * R3_DEV_TIMEOUT. */
r3_status r3_combine(const r3_shape* shape, const void* o, const int32_t* row_of_slot,
                     const float* gates, void* y, void* stream);

/* The same with a residual: y[t] = residual[t] + sum_j gates[t,j] * o[row_of_slot[t,j]] (the sum is
 * formed first, the residual added last, all in fp32, one rounding).  residual [T,d] act_dtype or
 * NULL (then identical to r3_combine).  Used by r3_replay_stack for x_{l+1} = x_l + y_l. */
r3_status r3_combine_residual(const r3_shape* shape, const void* o, const int32_t* row_of_slot,
                              const float* gates, const void* residual, void* y, void* stream);

/* Chain rule on Eq. (replay_output): dgates[t,j] = sum_c dy[t,c] * o[row_of_slot[t,j], c].
 * dy [T,d] act_dtype; dgates [T,K] f32. */
r3_status r3_combine_bwd_gates(const r3_shape* shape, const void* dy, const void* o,
                               const int32_t* row_of_slot, float* dgates, void* stream);

/* Everything that follows the expert networks, in one pass over the expert outputs: the replay
 * gate of Eq. (replay_gate), the combine of Eq. (replay_output), the gate gradient and the
 * router-logit gradient (Section 4.1, purpose (b): the mask is a constant).  Per token,
 *   g      = softmax of logits[t, idx[t, .]]                       (as r3_replay_gate_fwd)
 *   y[t]   = residual[t] + sum_j g_j o[row_of_slot[t,j]]           (as r3_combine_residual)
 *   dg_j   = <dy[t], o[row_of_slot[t,j]]>                          (as r3_combine_bwd_gates)
 *   dlogits[t, idx[t,j]] = g_j (dg_j - sum_j' g_j' dg_j'), 0 elsewhere   (as r3_replay_gate_bwd)
 * with the same arithmetic and summation orders as those four calls, so y, gates and dlogits are
 * bit-identical to theirs, but each expert-output row is read once instead of twice.
 * logits [T,E] f32; idx [T,K]; o [R,d]; row_of_slot [T,K]; dy [T,d]; residual [T,d] or NULL;
 * outputs y [T,d], gates_out [T,K] f32 or NULL, dlogits [T,E] f32 (every element written).
 * Supported for K <= 8 (R3_ERR_UNSUPPORTED beyond; use the four calls).  dev_status as for
 * r3_replay_gate_fwd. */
r3_status r3_replay_finish(const r3_shape* shape, const float* logits, const void* idx,
                           const void* o, const int32_t* row_of_slot, const void* dy,
                           const void* residual, void* y, float* gates_out, float* dlogits,
                           int32_t* dev_status, void* stream);

/* The whole replayed layer, forward and router-logit backward, enqueued back to back on one
 * stream: logits -> replay gate -> permute -> experts -> combine -> dgates -> dlogits.
 * Inputs x [T,d], w_router [E,d], idx [T,K], expert weights, dy [T,d];
 * outputs y [T,d] act_dtype and dlogits [T,E] f32.  Intermediates live in `workspace`
 * (r3_replay_layer_workspace_bytes).  Optional outputs (may be NULL): gates_out [T,K] f32. */
size_t r3_replay_layer_workspace_bytes(const r3_shape* shape);
r3_status r3_replay_layer(const r3_shape* shape, const void* x, const void* w_router,
                          const void* idx, const void* w_gate, const void* w_up,
                          const void* w_down, const void* dy, void* y, float* dlogits,
                          float* gates_out, void* workspace, size_t ws_bytes,
                          int32_t* dev_status, void* stream);
/* The same layer for another pass over the SAME record: the rollout's record is replayed in the
 * Recompute stage and again in the Update stage (Section 5.1, settings of the method; Section 6.3),
 * so the dispatch (counts, offsets, both maps) and the expert
 * work lists that the preceding r3_replay_layer call left in `workspace` still hold; this call
 * copies the rows of the new x with those maps and skips the dispatch.  `workspace` must be the
 * one that call used, untouched since, with the same shape and the same idx (idx is still read:
 * the gate needs it); x, the weights and dy may differ.  Results are bit-identical to
 * r3_replay_layer on the same arguments.  Passing a workspace that holds no such dispatch gives
 * undefined results (rows are copied to whatever row numbers it holds: call r3_replay_layer
 * first). */
r3_status r3_replay_layer_same_record(const r3_shape* shape, const void* x, const void* w_router,
                          const void* idx, const void* w_gate, const void* w_up,
                          const void* w_down, const void* dy, void* y, float* dlogits,
                          float* gates_out, void* workspace, size_t ws_bytes,
                          int32_t* dev_status, void* stream);

/* L independent replayed MoE blocks enqueued back to back: block l is r3_replay_layer on its own
 * input x[l], record idx[l], weights and upstream gradient dy[l] (a model's MoE blocks with the
 * sublayers between them left out, so that every block's input is given).  All tensors carry a
 * leading layer axis: x, dy, y [L,T,d]; w_router [L,E,d]; idx [L,T,K]; w_gate/w_up [L,E,F,d];
 * w_down [L,E,d,F]; dlogits [L,T,E] f32.  workspace: r3_replay_layer_workspace_bytes(shape). */
r3_status r3_replay_blocks(const r3_shape* shape, int32_t L, const void* x, const void* w_router,
                           const void* idx, const void* w_gate, const void* w_up,
                           const void* w_down, const void* dy, void* y, float* dlogits,
                           void* workspace, size_t ws_bytes, int32_t* dev_status, void* stream);

/* A stack of L replayed MoE blocks (no attention) with residual connections,
 *   x_{l+1} = x_l + y_replay,l(x_l),   l = 0..L-1,
 * each block being Eq. (replay_output) with its own weights and its own record, plus the
 * router-logit gradient of every block for one upstream gradient dy [T,d] shared by all blocks
 * (the gradient that reaches a block's output through the identity path of the later blocks).
 * Per-layer tensors are stacked on a leading layer axis: w_router [L,E,d], idx [L,T,K],
 * w_gate/w_up [L,E,F,d], w_down [L,E,d,F]; x0 [T,d]; outputs x_out [T,d] = x_L and
 * dlogits [L,T,E] f32.  workspace: r3_replay_stack_workspace_bytes(shape) (independent of L). */
size_t r3_replay_stack_workspace_bytes(const r3_shape* shape);
r3_status r3_replay_stack(const r3_shape* shape, int32_t L, const void* x0, const void* w_router,
                          const void* idx, const void* w_gate, const void* w_up,
                          const void* w_down, const void* dy, void* x_out, float* dlogits,
                          void* workspace, size_t ws_bytes, int32_t* dev_status, void* stream);

/* As r3_replay_layer, with the per-step tensors in HOST memory (pinned memory recommended):
 * x_host, idx_host, dy_host are copied to the device, y_host and dlogits_host are copied back,
 * and the stream is synchronised before returning.  Weights stay on the device.  The workspace
 * must hold r3_replay_layer_host_workspace_bytes(shape) bytes (device staging included).
 * From 16384 tokens on the batch goes through in chunks of tokens (r3_replay_layer_host_chunks),
 * each a layer of its own: the copies travel on two library-owned streams beside the kernels on
 * `stream`, which ends behind the last result copy.  Every token's result is what a layer of its
 * chunk alone gives; against one launch over the whole batch it may differ in the last bits (the
 * router kernel sums d in another order for another token count). */
size_t r3_replay_layer_host_workspace_bytes(const r3_shape* shape);
/* How r3_replay_layer_host cuts shape->T tokens: writes starts[0..n] (host memory, room for 17
 * values; starts[0] = 0, starts[n] = T, chunk c holds tokens [starts[c], starts[c+1])) and returns
 * n; 0 for a bad shape or a null pointer.  Equal chunks of at least 8192 tokens, multiples of
 * 256, the last one cut into a half and two quarters (the compute and the result copy of the last
 * chunk are what the call cannot hide under its input copies).  A host-side schedule: the paper
 * has no counterpart. */
int32_t r3_replay_layer_host_chunks(const r3_shape* shape, int64_t* starts);
r3_status r3_replay_layer_host(const r3_shape* shape, const void* x_host, const void* w_router,
                               const void* idx_host, const void* w_gate, const void* w_up,
                               const void* w_down, const void* dy_host, void* y_host,
                               float* dlogits_host, void* workspace, size_t ws_bytes,
                               int32_t* dev_status, void* stream);
/* The same without the final synchronisation: copies in, layer and copies out are enqueued on
 * `stream` and the call returns.  y_host and dlogits_host hold the result once the caller has
 * synchronised the stream; the host buffers and the workspace must stay untouched until then
 * (pageable host memory makes the copies synchronous: use pinned memory).  A caller that feeds a
 * sequence of batches keeps two or more of them in flight, each with its own stream, workspace and
 * host buffers: the copies of one batch then run beside the kernels of another.  Errors as
 * r3_replay_layer_host. */
r3_status r3_replay_layer_host_enqueue(const r3_shape* shape, const void* x_host,
                                       const void* w_router, const void* idx_host,
                                       const void* w_gate, const void* w_up, const void* w_down,
                                       const void* dy_host, void* y_host, float* dlogits_host,
                                       void* workspace, size_t ws_bytes, int32_t* dev_status,
                                       void* stream);

/* ---- Update-stage backward to the layer input (Section 4.1, purpose (b)) ------------------------ */

/* Input gradient of the expert networks on the grouped rows.  With a = xp W_gate,e^T,
 * b = xp W_up,e^T (the forward's pre-activations), h = silu(a) * b, o = h W_down,e^T and a
 * gradient dout = dL/do:
 *   dh  = dout W_down,e ;  da = dh * b * silu'(a) ;  db = dh * silu(a) ;
 *   dxp = da W_gate,e + db W_up,e                                   (= dL/dxp)
 * dout, dxp [R,d]; pre_gate, pre_up [R,F] (as stored by the forward, bf16); weights as in
 * r3_grouped_swiglu (read transposed in place, no transposed copy is made).  bf16 only
 * (R3_ERR_UNSUPPORTED for float32).  dh, da, db are rounded to bf16 once each.
 * workspace: r3_grouped_swiglu_bwd_workspace_bytes(shape). */
size_t r3_grouped_swiglu_bwd_workspace_bytes(const r3_shape* shape);
r3_status r3_grouped_swiglu_bwd_input(const r3_shape* shape, const void* dout, const void* pre_gate,
                                      const void* pre_up, const int32_t* offsets,
                                      const void* w_gate, const void* w_up, const void* w_down,
                                      void* dxp, void* workspace, size_t ws_bytes,
                                      int32_t* dev_status, void* stream);

/* The whole backward of the grouped experts: dxp as r3_grouped_swiglu_bwd_input, and the
 * gradients of the expert weights, for each expert e over its rows [offsets[e], offsets[e+1]):
 *   dW_down[e] = dout_e^T h_e     dW_gate[e] = da_e^T xp_e     dW_up[e] = db_e^T xp_e
 * xp [R,d] are the permuted rows the forward saw.  dw_gate, dw_up [E,F,d] and dw_down [E,d,F] are
 * float32 and are OVERWRITTEN (an expert without rows gets zeros); products of bf16 operands
 * (h, da, db rounded to bf16 once each) accumulate in float32 in a fixed order.  bf16 only.
 * workspace: r3_grouped_swiglu_bwd_workspace_bytes(shape). */
r3_status r3_grouped_swiglu_bwd(const r3_shape* shape, const void* xp, const void* dout,
                                const void* pre_gate, const void* pre_up, const int32_t* offsets,
                                const void* w_gate, const void* w_up, const void* w_down,
                                void* dxp, float* dw_gate, float* dw_up, float* dw_down,
                                void* workspace, size_t ws_bytes, int32_t* dev_status,
                                void* stream);

/* r3_grouped_swiglu that also keeps what its backward needs: besides o it stores the
 * pre-activations pre_gate = xp W_gate,e^T and pre_up = xp W_up,e^T ([R,F] each, rounded to bf16
 * from the float32 accumulator; h is formed from the unrounded values, so o is bit-identical to
 * r3_grouped_swiglu's).  bf16 only (R3_ERR_UNSUPPORTED for float32).  Same workspace. */
r3_status r3_grouped_swiglu_train(const r3_shape* shape, const void* xp, const int32_t* offsets,
                                  const void* w_gate, const void* w_up, const void* w_down,
                                  void* o, void* pre_gate, void* pre_up, void* workspace,
                                  size_t ws_bytes, int32_t* dev_status, void* stream);

/* Gradient of the expert outputs under Eq. (replay_output), y_t = sum_j g[t,j] o[row(t,j)]:
 *   dout[row_of_slot[t,j], :] = gates[t,j] * dy[t, :]
 * dy [T,d], gates [T,K] float32, row_of_slot [T,K], dout [R,d] (every row written once; slots
 * with row_of_slot < 0 are skipped).  No workspace. */
r3_status r3_scale_rows(const r3_shape* shape, const void* dy, const float* gates,
                        const int32_t* row_of_slot, void* dout, void* stream);

/* Last step of the backward to the layer input.  The input x_t reaches the loss through its K
 * experts and through the training logits s = x W_r^T that feed the replay gate (the recorded
 * mask is a constant, Section 4.1):
 *   dx[t,:]        = dx_residual[t,:] + sum_j dxp[row_of_slot[t,j], :]
 *                    + sum_j dlogits[t, e_j] * W_r[e_j, :]
 *   dw_router[e,:] = sum over tokens t whose record holds e of dlogits[t,e] * x[t,:]
 * (dlogits is zero outside the record, so these are the full products dlogits W_r and
 * dlogits^T x.)  dxp [R,d], dlogits [T,E] float32, idx [T,K], x [T,d], w_router [E,d]
 * (router_w_dtype), dx [T,d], dw_router [E,d] float32; dx_residual [T,d] (the gradient that
 * reaches x around the layer, e.g. through a residual connection) or null for none, never the
 * same buffer as dx; row_of_slot / slot_of_row / offsets from
 * r3_permute.  Sums run in float32 in a fixed order (dx: slot order; dw_router: eight interleaved
 * partial sums over the expert's rows, added in order): reproducible.  An
 * expert that appears twice in a token's record contributes its term twice to dx, as the
 * gradient of the gate does.  K <= 64 (R3_ERR_UNSUPPORTED beyond).  No workspace. */
r3_status r3_input_grad_finish(const r3_shape* shape, const void* dxp, const int32_t* row_of_slot,
                               const int32_t* slot_of_row, const int32_t* offsets,
                               const float* dlogits, const void* idx, const void* x,
                               const void* w_router, const void* dx_residual, void* dx,
                               float* dw_router, void* stream);

/* r3_replay_layer followed by its backward to the layer input and to the router weight, one
 * enqueue: y, dlogits as in r3_replay_layer, then dout = g dy, the expert input gradient
 * (r3_grouped_swiglu_bwd) and r3_input_grad_finish.  dx [T,d], dw_router [E,d] float32.
 * dw_gate, dw_up [E,F,d], dw_down [E,d,F] float32 receive the expert-weight gradients
 * (overwritten); pass all three null to skip them.  bf16 only
 * (R3_ERR_UNSUPPORTED for float32; r3_replay_layer_train_workspace_bytes returns 0 then).
 * workspace: r3_replay_layer_train_workspace_bytes(shape), 256-byte aligned. */
size_t r3_replay_layer_train_workspace_bytes(const r3_shape* shape);
r3_status r3_replay_layer_train(const r3_shape* shape, const void* x, const void* w_router,
                                const void* idx, const void* w_gate, const void* w_up,
                                const void* w_down, const void* dy, void* y, float* dlogits,
                                void* dx, float* dw_router, float* dw_gate, float* dw_up,
                                float* dw_down, void* workspace, size_t ws_bytes,
                                int32_t* dev_status, void* stream);

/* L residual blocks x_{l+1} = x_l + y_replay,l(x_l) (as r3_replay_stack), then the exact backward
 * chain of <dy, x_L>:  g_L = dy,  g_l = g_{l+1} + dx_l(g_{l+1}),  where block l's backward is
 * r3_replay_layer_train's at its own input x_l with upstream gradient g_{l+1} and the residual
 * path carries g_{l+1} through unchanged.  Block inputs are kept (L activations of [T,d]); each
 * block's forward is run again in the backward pass instead of keeping its intermediates.
 * Per-block tensors are stacked along a leading L: w_router [L,E,d], idx [L,T,K], w_gate / w_up
 * [L,E,F,d], w_down [L,E,d,F]; dy [T,d] = dL/dx_L.  Outputs: x_out [T,d] = x_L, dlogits [L,T,E]
 * (the exact router-logit gradients), dx0 [T,d] = dL/dx_0 (not the same buffer as dy),
 * dw_router [L,E,d] float32, and dw_gate / dw_up [L,E,F,d], dw_down [L,E,d,F] float32 or all
 * three null.  Activations and the gradients g_l are stored in bf16 between blocks.  bf16 only.
 * workspace: r3_replay_stack_train_workspace_bytes(shape, L). */
size_t r3_replay_stack_train_workspace_bytes(const r3_shape* shape, int32_t L);
r3_status r3_replay_stack_train(const r3_shape* shape, int32_t L, const void* x0,
                                const void* w_router, const void* idx, const void* w_gate,
                                const void* w_up, const void* w_down, const void* dy, void* x_out,
                                float* dlogits, void* dx0, float* dw_router, float* dw_gate,
                                float* dw_up, float* dw_down, void* workspace, size_t ws_bytes,
                                int32_t* dev_status, void* stream);

/* ---- expert parallelism: bookkeeping of the row exchange (an extension; the paper describes
 * no parallelism) ------------------------------------------------------------------------------
 *
 * With the E experts split over N ranks (rank q owns the experts [q E/N, (q+1) E/N)) every rank
 * runs r3_permute on its own tokens with GLOBAL expert numbers; the grouped rows bound for one rank
 * are then a contiguous block, the blocks are exchanged with an all-to-all (the caller's:
 * torch.distributed / NCCL), and the receiver holds [source rank][local expert][row].  The library
 * supplies the reordering into the [local expert][source rank][row] order that r3_grouped_swiglu
 * takes (with T = received rows, K = 1, E = E/N), and its inverse for the way back.
 *
 * r3_ep_regroup_map: recv_counts [n_src, e_local] int32 = rows received from each source for each
 * local expert; rows = their sum (known to the host from the split sizes; a table that does not
 * add up to it sets dev_status and writes nothing).  Writes perm [rows] (position in the new
 * order -> arrival index) and offsets [e_local + 1] (first row of each local expert in the new
 * order).  n_src * e_local <= 4096 (R3_ERR_UNSUPPORTED beyond).
 * r3_ep_move_rows: inverse = 0: dst[j] = src[perm[j]];  inverse = 1: dst[perm[j]] = src[j], for
 * rows of row_bytes bytes (a multiple of 16).  src and dst must not be the same buffer. */
r3_status r3_ep_regroup_map(const int32_t* recv_counts, int32_t n_src, int32_t e_local,
                            int32_t rows, int32_t* perm, int32_t* offsets, int32_t* dev_status,
                            void* stream);
r3_status r3_ep_move_rows(const void* src, void* dst, const int32_t* perm, int32_t rows,
                          size_t row_bytes, int32_t inverse, void* stream);

/* The same exchange without a collective for the rows: every rank writes its rows straight
 * into the owners' buffers (plain stores to memory this GPU can address: its own, or a peer's
 * mapped with peer access / symmetric memory, over NVLink), at the place they have in the owner's
 * [local expert][source][row] order, and later fetches the expert outputs of its rows from the
 * owners' output buffers by address.  No multicast load is involved anywhere.
 *
 * r3_ep_dest_table: counts_all [n_ranks, E] int32 (device; the ranks' `counts` of r3_permute after
 * an all-gather).  Writes dst_base [E] (row, in the owner's buffer, of THIS rank's first row of
 * every expert) and offsets_local [E / n_ranks + 1] (the offsets r3_grouped_swiglu takes for this
 * rank's own experts).  n_ranks <= 64.
 * r3_ep_dispatch_rows: copies x[t] to its K places; idx, row_of_slot and my_offsets (= offsets) are
 * those of this rank's r3_permute (called without x); peer_buffers_host [n_ranks] is a HOST array
 * of device addresses, entry q = base of rank q's receive buffer [capacity_rows, d] (the same
 * capacity on every rank).  A row whose place lies at or beyond capacity_rows is NOT stored and
 * dev_status (optional) receives R3_DEV_BAD_INDEX: a peer's memory is never written out of
 * bounds.  The owners must not read the buffers before every rank's call has completed (a barrier
 * of the job's own).
 * r3_ep_slot_rows: row_ptr [T, K] (device, 64-bit addresses) = where the expert-output row of each
 * (token, slot) pair will stand in the owners' OUTPUT buffers (peer_buffers_host: their bases,
 * capacity_rows as above); 0 for a pair that r3_permute dropped or whose place is beyond the
 * capacity (then dev_status receives R3_DEV_BAD_INDEX).
 * r3_replay_finish_rows: r3_replay_finish with the rows given by address (row_ptr) instead of
 * (o, row_of_slot).  K <= 8 and the rows of one token must fit in shared memory
 * ((K + 2) d elements, else R3_ERR_UNSUPPORTED). */
r3_status r3_ep_dest_table(const int32_t* counts_all, int32_t n_ranks, int32_t E, int32_t rank,
                           int32_t* dst_base, int32_t* offsets_local, void* stream);
r3_status r3_ep_dispatch_rows(const r3_shape* shape, int32_t n_ranks, const void* x,
                              const void* idx, const int32_t* row_of_slot,
                              const int32_t* my_offsets, const int32_t* dst_base,
                              const unsigned long long* peer_buffers_host, int64_t capacity_rows,
                              int32_t* dev_status, void* stream);
r3_status r3_ep_slot_rows(const r3_shape* shape, int32_t n_ranks, const void* idx,
                          const int32_t* row_of_slot, const int32_t* my_offsets,
                          const int32_t* dst_base, const unsigned long long* peer_buffers_host,
                          int64_t capacity_rows, unsigned long long* row_ptr, int32_t* dev_status,
                          void* stream);
r3_status r3_replay_finish_rows(const r3_shape* shape, const float* logits, const void* idx,
                                const unsigned long long* row_ptr, const void* dy,
                                const void* residual, void* y, float* gates_out, float* dlogits,
                                int32_t* dev_status, void* stream);

/* ---- training/inference discrepancy measures (Sections 3.1 and 3.2) -------------------------- */

/* Eq. (kl), the k3 estimate of KL(pi_train || pi_infer), and Eq. (etdf), the Extreme Token
 * Distribution Function, over n response tokens:
 *   *kl_out       = (1/n) sum_t [ r_t - 1 - log r_t ],   r_t = p_train[t] / p_infer[t]   (float64)
 *   counts_out[i] = #{ t : max(r_t, 1/r_t) > taus[i] }   (so F(taus[i]) = counts_out[i] / n)
 * p_train, p_infer [n] float32 probabilities of the sampled tokens (positive); taus [n_tau]
 * float32 (device), n_tau <= 16; kl_out [1] float64 and counts_out [n_tau] int64 (device).
 * Each k3 term is formed in float32 by a cancellation-free expression of (p_train - p_infer) /
 * p_infer (relative error below 1e-5, typically 1e-7) and the terms are summed in float64 in a
 * fixed order (reproducible); the threshold decision is taken on float32 ratios.  workspace: r3_prob_discrepancy_workspace_bytes(n). */
size_t r3_prob_discrepancy_workspace_bytes(int64_t n);
r3_status r3_prob_discrepancy(const float* p_train, const float* p_infer, int64_t n,
                              const float* taus, int32_t n_tau, double* kl_out,
                              int64_t* counts_out, void* workspace, size_t ws_bytes, void* stream);

/* Section 3.2, router-level and token-level comparison of two routing records rec_a, rec_b
 * [L, T, K] (shape->T, K, E, idx_type; K <= 32; each (layer, token) holds K distinct experts, in
 * any slot order):
 *   diff[l,t]        = K - |{rec_a[l,t,.]} & {rec_b[l,t,.]}|   differing expert choices of a router
 *   hist[v]          = number of routers (l,t) with diff = v                 [K+1] int64
 *   token_choices[t] = sum_l diff[l,t]                                       [T]   int32
 *   token_routers[t] = number of layers l with diff[l,t] > 0                 [T]   int32
 * diff_out [L,T] uint8 may be NULL.  All outputs are exact integers. */
r3_status r3_record_diff(const r3_shape* shape, int32_t L, const void* rec_a, const void* rec_b,
                         uint8_t* diff_out, int32_t* token_choices, int32_t* token_routers,
                         int64_t* hist, void* stream);

/* Section 3.2, sequence-level comparison: seq_sum[s] = sum of token_routers over the tokens
 * [cu_seqlens[s], cu_seqlens[s+1]) of sequence s; the paper's mean difference per token of a
 * sequence is seq_sum[s] / length.  cu_seqlens [S+1] int32 (device), seq_sum [S] int64. */
r3_status r3_sequence_diff(const int32_t* token_routers, const int32_t* cu_seqlens, int32_t S,
                           int64_t* seq_sum, void* stream);

/* ---- routing-record store (Section 4.2: router masks cached with the prefix KV cache) --------- */

/* Records are kept in pages of `page_tokens` tokens, laid out [page][layer][token in page][slot]
 * (r3_record_page_bytes per page) in a device buffer `pages` of n_pages pages owned by the
 * caller.  A sequence is the list of its page numbers: row b of block_table [B, max_pages] int32
 * (device).  Two sequences that share a prefix list the same pages for it, which is how cached
 * masks are reused without recomputation (Section 4.2).  shape gives K and idx_type.
 *
 * r3_record_append (inference side): rec_new [L, N, K] holds the records of N new tokens, packed
 * sequence after sequence (cu_new [B+1]); the tokens of sequence b go to positions seq_pos0[b],
 * seq_pos0[b]+1, ... of that sequence.  Multi-turn use appends again to the same sequence.
 * r3_record_gather (training side): out [L, T, K] receives the records of positions 0 ..
 * len_b - 1 of every sequence, packed in the order of cu_seqlens [B+1] - the record that
 * r3_replay_layer / r3_replay_blocks take.
 * Both copy bytes (bit-exact).  dev_status (optional): R3_DEV_BAD_INDEX when a position has no
 * page (table entry < 0, >= n_pages, or beyond max_pages); that record is skipped. */
size_t r3_record_page_bytes(const r3_shape* shape, int32_t L, int32_t page_tokens);
r3_status r3_record_append(const r3_shape* shape, int32_t L, int32_t page_tokens, int32_t n_pages,
                           void* pages, const int32_t* block_table, int32_t max_pages,
                           const int32_t* seq_pos0, const int32_t* cu_new, int32_t B,
                           const void* rec_new, int32_t N, int32_t* dev_status, void* stream);
r3_status r3_record_gather(const r3_shape* shape, int32_t L, int32_t page_tokens, int32_t n_pages,
                           const void* pages, const int32_t* block_table, int32_t max_pages,
                           const int32_t* cu_seqlens, int32_t B, void* out, int32_t T,
                           int32_t* dev_status, void* stream);

/* Host-side bookkeeping of the pages (no device work; all pointers are HOST pointers; the pool
 * allocates host memory only, freed by r3_pagepool_destroy).  Not thread-safe.
 *   match   : the pages of the longest already stored whole-page prefix of token_ids (use counts
 *             go up); returns how many pages matched - their records need not be produced again
 *   alloc   : n unused pages (use count 1), R3_ERR_OUT_OF_PAGES if fewer are free
 *   publish : makes every full page of a sequence (token_ids = the n_tokens ids whose records the
 *             table's pages hold) findable by later match calls; a prefix is indexed once
 *   release : use counts go down; a page nobody uses leaves the index and becomes free
 * A page is identified by a chained 64-bit hash of all token ids up to its end, and a match also
 * compares the page's own ids: distinct prefixes are confused only on a hash collision. */
typedef struct r3_pagepool r3_pagepool;
r3_pagepool* r3_pagepool_create(int32_t n_pages, int32_t page_tokens);
void r3_pagepool_destroy(r3_pagepool* pool);
int32_t r3_pagepool_free_pages(const r3_pagepool* pool);
int32_t r3_pagepool_match(r3_pagepool* pool, const int32_t* token_ids, int32_t n_tokens,
                          int32_t* pages_out, int32_t max_pages);
r3_status r3_pagepool_alloc(r3_pagepool* pool, int32_t n, int32_t* pages_out);
r3_status r3_pagepool_publish(r3_pagepool* pool, const int32_t* token_ids, int32_t n_tokens,
                              const int32_t* table, int32_t n_table);
r3_status r3_pagepool_release(r3_pagepool* pool, const int32_t* table, int32_t n);

/* ---- self-test of the error path (the paper has no counterpart) ---------------------------------
 *
 * The tensor-core kernels wait on shared-memory barriers for their copies and MMAs; every such
 * wait is bounded, and a wait that runs out raises an abort flag in its CTA, writes
 * R3_DEV_TIMEOUT to dev_status and lets the kernel drain and return (see "General rules").  In a
 * healthy run that path never executes.  r3_selftest_bounded_wait runs it on purpose in a
 * harmless form: one 32-thread CTA waits, with the library's own wait routine and a limit of
 * `limit_clocks` SM clocks (1 .. 2e9, else R3_ERR_INVALID_ARG), on a barrier of its own that nothing
 * signals - no copy is in flight and no tensor memory is held.  Afterwards dev_status (optional)
 * holds R3_DEV_TIMEOUT and out [4] int32 (device) = {the wait's return value (0 = gave up), the
 * abort flag (1), clocks spent waiting (saturated), the return value of a second wait entered
 * while the CTA was already aborting (0)}.  The context stays usable: the next call is an
 * ordinary one. */
r3_status r3_selftest_bounded_wait(int64_t limit_clocks, int32_t* dev_status, int32_t* out,
                                   void* stream);

#ifdef __cplusplus
}
#endif
#endif /* R3_H_ */
