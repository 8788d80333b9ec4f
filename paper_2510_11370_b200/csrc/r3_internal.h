// Internal (non-exported) interfaces between the translation units of the library.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "r3.h"

namespace r3 {

// Device-side tile list of the grouped GEMMs: int32 header[4] = {number of M tiles, BM, 0, 0}
// followed by one int32[4] entry per M tile = {expert, first row, valid rows, 0}.  Tiles are
// listed expert by expert, rows ascending; an M tile never spans two experts.
constexpr int kTileHeaderInts = 4;
inline size_t tile_list_bytes(long long R, int E, int BM) {
    const long long max_tiles = R / BM + E + 1;
    return (size_t)(kTileHeaderInts + 4 * max_tiles) * sizeof(int32_t);
}
inline int max_m_tiles(long long R, int E, int BM) {
    const long long by_rows = R / BM + E;          // each expert adds at most one partial tile
    const long long by_pairs = R < by_rows ? R : by_rows;   // and no more tiles than rows
    return (int)(by_pairs > 0 ? by_pairs : 0);
}

// Builds the tile list from offsets [E+1] (one small kernel).
r3_status launch_build_tiles(const int32_t* offsets, int E, int BM, int32_t* tiles,
                             cudaStream_t stream);

// bf16 grouped SwiGLU on the tcgen05 tensor cores (sm_100a, two CTAs per MMA).  `work` is
// tc_work_bytes() of scratch for the two device-built work lists (the up phase builds both from
// `offsets`; the down phase reads the list the up phase left there).
size_t tc_work_bytes(const r3_shape* shape);
// phases: bit 0 = gate/up projections + SwiGLU (xp -> h), bit 1 = down projection (h -> o),
// bit 2 = the work lists in `work` were built by an earlier call from the same offsets: the up
// phase does not build them again.
enum { kPhaseUp = 1, kPhaseDown = 2, kPhaseKeepLists = 4 };
// pre_gate / pre_up (optional, [R,F] bf16): the up phase also stores xp W_gate^T and xp W_up^T.
// Token operand of the up projection: either the permuted rows `xp` [R, d], or (xp == nullptr) the
// un-permuted activations `x` [T, d] gathered in place through `slot_of_row` [R].
r3_status launch_grouped_swiglu_tc(const r3_shape* shape, const void* xp, const void* x,
                                   const int32_t* slot_of_row, const int32_t* offsets,
                                   const void* w_gate, const void* w_up, const void* w_down,
                                   void* h, void* o, void* work, int32_t* dev_status, int phases,
                                   cudaStream_t stream, void* pre_gate = nullptr,
                                   void* pre_up = nullptr);

// Input gradient of the grouped SwiGLU experts on the tensor cores (bf16): dout [R,d] -> dxp [R,d]
// with the forward's pre-activations pre_gate, pre_up [R,F].  `work`: tc_bwd_work_bytes().
// With dw_gate non-null (then xp, dw_up, dw_down too) the expert-weight gradients follow.
size_t tc_bwd_work_bytes(const r3_shape* shape);
r3_status launch_grouped_swiglu_bwd_tc(const r3_shape* shape, const void* dout, const void* pre_gate,
                                       const void* pre_up, const int32_t* offsets,
                                       const void* w_gate, const void* w_up, const void* w_down,
                                       void* dxp, void* work, int32_t* dev_status,
                                       cudaStream_t stream, const void* xp = nullptr,
                                       float* dw_gate = nullptr, float* dw_up = nullptr,
                                       float* dw_down = nullptr);
// dW_down[e] = dout_e^T h_e, dW_gate[e] = da_e^T xp_e, dW_up[e] = db_e^T xp_e (float32 [E,d,F],
// [E,F,d], [E,F,d]); all operands bf16, [R, .] row-major.
r3_status launch_wgrad_tc(const r3_shape* shape, const void* xp, const void* dout, const void* h,
                          const void* da, const void* db, const int32_t* offsets, float* dw_gate,
                          float* dw_up, float* dw_down, int32_t* dev_status, cudaStream_t stream);

// Router logits + top-K on the tensor cores (bf16 activations, E a multiple of 16 up to 256,
// K <= 16).  float32 router weights need router_tc_workspace_bytes() of scratch for their three
// bf16 planes; bf16 router weights need none.
bool router_tc_supported(const r3_shape* shape);
size_t router_tc_workspace_bytes(const r3_shape* shape, int L);
r3_status launch_router_tc(const r3_shape* shape, int L, const void* x, const void* w_router,
                           void* idx_out, float* logits_out, void* workspace, cudaStream_t stream);

// Where the up phase of the bf16 experts expects its two work lists inside a
// r3_grouped_swiglu workspace, and their parameters (feature tiles per list, resident clusters).
// false: this shape does not use such lists (float32), or the device query failed.
struct WorkListSpec {
    int32_t* list0;
    int32_t* list1;
    int nf0, nf1, pairs;
};
bool grouped_swiglu_list_spec(const r3_shape* shape, void* workspace, WorkListSpec* spec);
bool tc_work_lists(const r3_shape* shape, void* work, WorkListSpec* spec);

// r3_permute; with `lists` the one-cluster form of the dispatch also builds the expert GEMMs'
// work lists (then *lists_built = true and the experts run with kPhaseKeepLists).
r3_status permute_impl(const r3_shape* shape, const void* idx, const void* x, int32_t* counts,
                       int32_t* offsets, int32_t* row_of_slot, int32_t* slot_of_row, void* xp,
                       void* workspace, size_t ws_bytes, int32_t* dev_status, void* stream,
                       const WorkListSpec* lists, bool* lists_built);

// r3_grouped_swiglu (with pre_gate / pre_up: r3_grouped_swiglu_train) on a workspace whose work
// lists an earlier call built from the same offsets.
r3_status grouped_swiglu_keep_lists(const r3_shape* shape, const void* xp, const int32_t* offsets,
                                    const void* w_gate, const void* w_up, const void* w_down,
                                    void* o, void* pre_gate, void* pre_up, void* workspace,
                                    size_t ws_bytes, int32_t* dev_status, void* stream);

// The row copy of the dispatch alone: xp[row_of_slot[t, j]] = x[t] (maps from an earlier r3_permute).
// x_early = true only when the kernel launched just before on the stream does not write x and
// cannot let this one start before everything in front of it has completed (the dispatch kernels):
// the token rows are then fetched before the dependency wait.
r3_status launch_permute_rows(const r3_shape* shape, const void* x, const int32_t* row_of_slot,
                              void* xp, cudaStream_t stream, int32_t* dev_status,
                              bool x_early = false);

// Number of SMs of the current device (cached).
int sm_count();

}  // namespace r3
