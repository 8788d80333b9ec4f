// Expert networks on the grouped rows: entry point, tile-list builder and the float32 kernels.
//   h[r] = silu(xp[r] W_gate,e^T) * (xp[r] W_up,e^T),   o[r] = h[r] W_down,e^T
// bf16 goes to the tcgen05 kernels (r3_swiglu_tc.cu); float32 uses the plain FMA kernels below
// (tf32 tensor cores would not hold the 1e-5 tolerance of the float32 configuration).
#include "r3_common.cuh"
#include "r3_internal.h"

namespace r3 {

int sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

// One CTA of 1024 threads; thread e owns expert e (E <= 1024).
__global__ void __launch_bounds__(1024)
build_tiles_kernel(const int32_t* __restrict__ offsets, int E, int BM, int32_t* __restrict__ tiles) {
    __shared__ int32_t warp_sum[32];
    const int e = threadIdx.x, lane = e & 31, warp = e >> 5;
    const int32_t lo = e < E ? offsets[e] : 0;
    const int32_t cnt = e < E ? offsets[e + 1] - lo : 0;
    const int32_t nt = (cnt + BM - 1) / BM;
    int32_t inc = nt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int32_t n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
    }
    if (lane == 31) warp_sum[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        int32_t w = warp_sum[lane], winc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int32_t n = __shfl_up_sync(0xffffffffu, winc, o);
            if (lane >= o) winc += n;
        }
        warp_sum[lane] = winc - w;
        if (lane == 31) {
            tiles[0] = winc;      // total number of M tiles
            tiles[1] = BM;
            tiles[2] = 0;
            tiles[3] = 0;
        }
    }
    __syncthreads();
    const int32_t base = warp_sum[warp] + inc - nt;
    int4* ent = reinterpret_cast<int4*>(tiles + kTileHeaderInts);
    for (int32_t i = 0; i < nt; ++i)
        ent[base + i] = make_int4(e, lo + i * BM, min(BM, cnt - i * BM), 0);
}

r3_status launch_build_tiles(const int32_t* offsets, int E, int BM, int32_t* tiles,
                             cudaStream_t stream) {
    build_tiles_kernel<<<1, 1024, 0, stream>>>(offsets, E, BM, tiles);
    return launch_status();
}

// ---------------------------------------------------------------------------------------------
// float32 grouped GEMM, C[r, n] = sum_k A[r, k] * B_e[n, k]  (B output-major).  64x64 tile,
// 16-wide k steps, 256 threads with 4x4 outputs each.  DUAL: two B matrices (gate, up) and the
// SwiGLU epilogue; otherwise a plain store.
// ---------------------------------------------------------------------------------------------
constexpr int SBM = 64, SBN = 64, SBK = 16;

template <bool DUAL>
__global__ void __launch_bounds__(256)
simt_grouped_gemm_kernel(const float* __restrict__ A, const float* __restrict__ B0,
                         const float* __restrict__ B1, float* __restrict__ C,
                         const int32_t* __restrict__ tiles, int Kdim, int N) {
    const int m_tile = blockIdx.x;
    if (m_tile >= tiles[0]) return;
    const int4 ent = reinterpret_cast<const int4*>(tiles + kTileHeaderInts)[m_tile];
    const int e = ent.x, row0 = ent.y, rows = ent.z;
    const int n0 = blockIdx.y * SBN;
    __shared__ float as[SBK][SBM + 4];
    __shared__ float b0s[SBK][SBN + 4];
    __shared__ float b1s[DUAL ? SBK : 1][SBN + 4];
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const float* Be0 = B0 + (size_t)e * N * Kdim;
    const float* Be1 = DUAL ? B1 + (size_t)e * N * Kdim : nullptr;
    float acc0[4][4] = {}, acc1[4][4] = {};
    const int lr = tid >> 2, lk = (tid & 3) * 4;       // loader: row lr (0..63), k offset lk
    for (int k0 = 0; k0 < Kdim; k0 += SBK) {
        float4 va = make_float4(0, 0, 0, 0), vb0 = va, vb1 = va;
        const bool kin = k0 + lk < Kdim;               // Kdim is a multiple of 8, lk of 4
        if (kin && lr < rows)
            va = *reinterpret_cast<const float4*>(A + (size_t)(row0 + lr) * Kdim + k0 + lk);
        if (kin && n0 + lr < N) {
            vb0 = *reinterpret_cast<const float4*>(Be0 + (size_t)(n0 + lr) * Kdim + k0 + lk);
            if (DUAL) vb1 = *reinterpret_cast<const float4*>(Be1 + (size_t)(n0 + lr) * Kdim + k0 + lk);
        }
        __syncthreads();
        as[lk + 0][lr] = va.x; as[lk + 1][lr] = va.y; as[lk + 2][lr] = va.z; as[lk + 3][lr] = va.w;
        b0s[lk + 0][lr] = vb0.x; b0s[lk + 1][lr] = vb0.y; b0s[lk + 2][lr] = vb0.z; b0s[lk + 3][lr] = vb0.w;
        if (DUAL) {
            b1s[lk + 0][lr] = vb1.x; b1s[lk + 1][lr] = vb1.y; b1s[lk + 2][lr] = vb1.z; b1s[lk + 3][lr] = vb1.w;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < SBK; ++kk) {
            const float4 a = *reinterpret_cast<const float4*>(&as[kk][ty * 4]);
            const float4 b = *reinterpret_cast<const float4*>(&b0s[kk][tx * 4]);
            const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc0[i][j] = fmaf(av[i], bv[j], acc0[i][j]);
            if (DUAL) {
                const float4 c = *reinterpret_cast<const float4*>(&b1s[kk][tx * 4]);
                const float cv[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc1[i][j] = fmaf(av[i], cv[j], acc1[i][j]);
            }
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = ty * 4 + i;
        if (r >= rows) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n >= N) continue;
            float v = acc0[i][j];
            if (DUAL) v = v / (1.f + expf(-v)) * acc1[i][j];
            C[(size_t)(row0 + r) * N + n] = v;
        }
    }
}

static r3_status launch_grouped_swiglu_f32(const r3_shape* s, const void* xp, const int32_t* tiles,
                                           const void* w_gate, const void* w_up,
                                           const void* w_down, void* h, void* o,
                                           int phases, cudaStream_t cs) {
    const long long R = (long long)s->T * s->K;
    const int mt = max_m_tiles(R, s->E, SBM);
    if (mt == 0) return R3_OK;
    dim3 g1(mt, (s->F + SBN - 1) / SBN), g2(mt, (s->d + SBN - 1) / SBN);
    if (phases & kPhaseUp)
        simt_grouped_gemm_kernel<true><<<g1, 256, 0, cs>>>(
            static_cast<const float*>(xp), static_cast<const float*>(w_gate),
            static_cast<const float*>(w_up), static_cast<float*>(h), tiles, s->d, s->F);
    if (phases & kPhaseDown)
        simt_grouped_gemm_kernel<false><<<g2, 256, 0, cs>>>(
            static_cast<const float*>(h), static_cast<const float*>(w_down), nullptr,
            static_cast<float*>(o), tiles, s->F, s->d);
    return launch_status();
}

static size_t h_bytes(const r3_shape* s) {
    return round_up((size_t)s->T * s->K * s->F * act_bytes(s), 256);
}
// scratch after h: the tensor-core work lists (bf16) or the row-tile list (float32)
static size_t list_bytes(const r3_shape* s) {
    if (s->act_dtype == R3_BF16) return tc_work_bytes(s);
    return round_up(tile_list_bytes((long long)s->T * s->K, s->E, SBM), 256);
}

}  // namespace r3

extern "C" size_t r3_grouped_swiglu_workspace_bytes(const r3_shape* shape) {
    if (r3::check_shape(shape) != R3_OK) return 0;
    return r3::h_bytes(shape) + r3::list_bytes(shape);
}

namespace r3 {
// Shared body of the three expert entry points.
static r3_status run_experts(const r3_shape* shape, const void* xp, const void* x,
                             const int32_t* slot_of_row, const int32_t* offsets,
                             const void* w_gate, const void* w_up, const void* w_down, void* o,
                             void* workspace, size_t ws_bytes, int32_t* dev_status, int phases,
                             void* stream, void* pre_gate = nullptr, void* pre_up = nullptr) {
    r3_status st = check_shape(shape);
    if (st != R3_OK) return st;
    if (shape->E > 1024) return R3_ERR_UNSUPPORTED;
    if (shape->T == 0) return R3_OK;
    const bool up = phases & kPhaseUp, down = phases & kPhaseDown;
    const bool gather = up && !xp;             // token rows read in place from x
    if ((gather || pre_gate || pre_up) && shape->act_dtype != R3_BF16) return R3_ERR_UNSUPPORTED;
    if ((pre_gate != nullptr) != (pre_up != nullptr) || !aligned(pre_gate, 16) ||
        !aligned(pre_up, 16))
        return R3_ERR_INVALID_ARG;
    if ((up && (!offsets || !w_gate || !w_up || (gather ? (!x || !slot_of_row) : !xp))) ||
        (down && (!w_down || !o)))
        return R3_ERR_INVALID_ARG;
    if ((up && (!aligned(xp, 16) || !aligned(x, 16) || !aligned(w_gate, 16) ||
                !aligned(w_up, 16))) ||
        (down && (!aligned(o, 16) || !aligned(w_down, 16))))
        return R3_ERR_INVALID_ARG;
    if (!workspace || ws_bytes < r3_grouped_swiglu_workspace_bytes(shape) ||
        !aligned(workspace, 256))
        return R3_ERR_WORKSPACE;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    void* h = workspace;
    int32_t* tiles = reinterpret_cast<int32_t*>(static_cast<char*>(workspace) + h_bytes(shape));
    if (shape->act_dtype == R3_BF16)
        return launch_grouped_swiglu_tc(shape, xp, x, slot_of_row, offsets, w_gate, w_up, w_down,
                                        h, o, tiles, dev_status, phases, cs, pre_gate, pre_up);
    if (up && !(phases & kPhaseKeepLists)) {
        st = launch_build_tiles(offsets, shape->E, SBM, tiles, cs);
        if (st != R3_OK) return st;
    }
    return launch_grouped_swiglu_f32(shape, xp, tiles, w_gate, w_up, w_down, h, o, phases, cs);
}

bool grouped_swiglu_list_spec(const r3_shape* shape, void* workspace, WorkListSpec* spec) {
    if (shape->act_dtype != R3_BF16 || shape->E > 1024 || !workspace) return false;
    return tc_work_lists(shape, static_cast<char*>(workspace) + h_bytes(shape), spec);
}

r3_status grouped_swiglu_keep_lists(const r3_shape* shape, const void* xp, const int32_t* offsets,
                                    const void* w_gate, const void* w_up, const void* w_down,
                                    void* o, void* pre_gate, void* pre_up, void* workspace,
                                    size_t ws_bytes, int32_t* dev_status, void* stream) {
    return run_experts(shape, xp, nullptr, nullptr, offsets, w_gate, w_up, w_down, o, workspace,
                       ws_bytes, dev_status, kPhaseUp | kPhaseDown | kPhaseKeepLists, stream,
                       pre_gate, pre_up);
}
}  // namespace r3

extern "C" r3_status r3_grouped_swiglu(const r3_shape* shape, const void* xp,
                                       const int32_t* offsets, const void* w_gate,
                                       const void* w_up, const void* w_down, void* o,
                                       void* workspace, size_t ws_bytes, int32_t* dev_status,
                                       void* stream) {
    return r3::run_experts(shape, xp, nullptr, nullptr, offsets, w_gate, w_up, w_down, o, workspace,
                           ws_bytes, dev_status, r3::kPhaseUp | r3::kPhaseDown, stream);
}

extern "C" r3_status r3_grouped_swiglu_train(const r3_shape* shape, const void* xp,
                                             const int32_t* offsets, const void* w_gate,
                                             const void* w_up, const void* w_down, void* o,
                                             void* pre_gate, void* pre_up, void* workspace,
                                             size_t ws_bytes, int32_t* dev_status, void* stream) {
    if (shape && shape->T > 0 && (!pre_gate || !pre_up)) return R3_ERR_INVALID_ARG;
    return r3::run_experts(shape, xp, nullptr, nullptr, offsets, w_gate, w_up, w_down, o, workspace,
                           ws_bytes, dev_status, r3::kPhaseUp | r3::kPhaseDown, stream, pre_gate,
                           pre_up);
}

extern "C" r3_status r3_grouped_swiglu_gather(const r3_shape* shape, const void* x,
                                              const int32_t* slot_of_row, const int32_t* offsets,
                                              const void* w_gate, const void* w_up,
                                              const void* w_down, void* o, void* workspace,
                                              size_t ws_bytes, int32_t* dev_status, void* stream) {
    if (!x || !slot_of_row) return R3_ERR_INVALID_ARG;
    return r3::run_experts(shape, nullptr, x, slot_of_row, offsets, w_gate, w_up, w_down, o,
                           workspace, ws_bytes, dev_status, r3::kPhaseUp | r3::kPhaseDown, stream);
}

extern "C" r3_status r3_expert_up_swiglu(const r3_shape* shape, const void* xp,
                                         const int32_t* offsets, const void* w_gate,
                                         const void* w_up, void* workspace, size_t ws_bytes,
                                         int32_t* dev_status, void* stream) {
    return r3::run_experts(shape, xp, nullptr, nullptr, offsets, w_gate, w_up, nullptr, nullptr,
                           workspace, ws_bytes, dev_status, r3::kPhaseUp, stream);
}

extern "C" r3_status r3_expert_down(const r3_shape* shape, const void* w_down, void* o,
                                    void* workspace, size_t ws_bytes, int32_t* dev_status,
                                    void* stream) {
    return r3::run_experts(shape, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, w_down, o,
                           workspace, ws_bytes, dev_status, r3::kPhaseDown, stream);
}

extern "C" size_t r3_grouped_swiglu_bwd_workspace_bytes(const r3_shape* shape) {
    if (r3::check_shape(shape) != R3_OK || shape->act_dtype != R3_BF16) return 0;
    return r3::tc_bwd_work_bytes(shape);
}

extern "C" r3_status r3_grouped_swiglu_bwd_input(const r3_shape* shape, const void* dout,
                                                 const void* pre_gate, const void* pre_up,
                                                 const int32_t* offsets, const void* w_gate,
                                                 const void* w_up, const void* w_down, void* dxp,
                                                 void* workspace, size_t ws_bytes,
                                                 int32_t* dev_status, void* stream) {
    r3_status st = r3::check_shape(shape);
    if (st != R3_OK) return st;
    if (shape->act_dtype != R3_BF16 || shape->E > 1024) return R3_ERR_UNSUPPORTED;
    if (shape->T == 0) return R3_OK;
    if (!dout || !pre_gate || !pre_up || !offsets || !w_gate || !w_up || !w_down || !dxp)
        return R3_ERR_INVALID_ARG;
    if (!r3::aligned(dout, 16) || !r3::aligned(pre_gate, 16) || !r3::aligned(pre_up, 16) ||
        !r3::aligned(dxp, 16) || !r3::aligned(w_gate, 16) || !r3::aligned(w_up, 16) ||
        !r3::aligned(w_down, 16))
        return R3_ERR_INVALID_ARG;
    if (!workspace || !r3::aligned(workspace, 256) ||
        ws_bytes < r3_grouped_swiglu_bwd_workspace_bytes(shape))
        return R3_ERR_WORKSPACE;
    return r3::launch_grouped_swiglu_bwd_tc(shape, dout, pre_gate, pre_up, offsets, w_gate, w_up,
                                            w_down, dxp, workspace, dev_status,
                                            static_cast<cudaStream_t>(stream));
}

extern "C" r3_status r3_grouped_swiglu_bwd(const r3_shape* shape, const void* xp, const void* dout,
                                           const void* pre_gate, const void* pre_up,
                                           const int32_t* offsets, const void* w_gate,
                                           const void* w_up, const void* w_down, void* dxp,
                                           float* dw_gate, float* dw_up, float* dw_down,
                                           void* workspace, size_t ws_bytes, int32_t* dev_status,
                                           void* stream) {
    r3_status st = r3::check_shape(shape);
    if (st != R3_OK) return st;
    if (shape->act_dtype != R3_BF16 || shape->E > 1024) return R3_ERR_UNSUPPORTED;
    if (shape->T == 0) return R3_OK;
    if (!xp || !dout || !pre_gate || !pre_up || !offsets || !w_gate || !w_up || !w_down || !dxp ||
        !dw_gate || !dw_up || !dw_down)
        return R3_ERR_INVALID_ARG;
    if (!r3::aligned(xp, 16) || !r3::aligned(dout, 16) || !r3::aligned(pre_gate, 16) ||
        !r3::aligned(pre_up, 16) || !r3::aligned(dxp, 16) || !r3::aligned(w_gate, 16) ||
        !r3::aligned(w_up, 16) || !r3::aligned(w_down, 16) || !r3::aligned(dw_gate, 16) ||
        !r3::aligned(dw_up, 16) || !r3::aligned(dw_down, 16))
        return R3_ERR_INVALID_ARG;
    if (!workspace || !r3::aligned(workspace, 256) ||
        ws_bytes < r3_grouped_swiglu_bwd_workspace_bytes(shape))
        return R3_ERR_WORKSPACE;
    return r3::launch_grouped_swiglu_bwd_tc(shape, dout, pre_gate, pre_up, offsets, w_gate, w_up,
                                            w_down, dxp, workspace, dev_status,
                                            static_cast<cudaStream_t>(stream), xp, dw_gate, dw_up,
                                            dw_down);
}
