// Router logits and TopKMask, fused (Section 4.1, first and second equations):
//   s[t,i] = sum_c x[t,c] W_r[i,c];   record[t, 0..K) = the K largest experts of row t,
// descending logit, exact ties to the lower expert index.
//
// A CTA computes the logits of 64 tokens against all E experts (float32 accumulation, operands
// widened exactly), keeps that tile in shared memory, optionally streams it out, and selects the
// top K of each row with warp-wide argmax rounds.
#include "r3_common.cuh"
#include "r3_internal.h"

namespace r3 {

constexpr int CT = 64;      // tokens per CTA
constexpr int CE = 128;     // experts per accumulation pass
constexpr int CK = 16;      // k per shared-memory step
constexpr int kMaxPerLane = kMaxExpertsCapture / 32;

__device__ __forceinline__ void load4(const float* p, float* f) {
    const float4 v = *reinterpret_cast<const float4*>(p);
    f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
}
__device__ __forceinline__ void load4(const __nv_bfloat16* p, float* f) {
    const uint2 v = *reinterpret_cast<const uint2*>(p);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
    const float2 a = __bfloat1622float2(h[0]), b = __bfloat1622float2(h[1]);
    f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y;
}

template <typename XT, typename WT, typename IdxT>
__global__ void __launch_bounds__(256)
capture_topk_kernel(const XT* __restrict__ x, const WT* __restrict__ w, IdxT* __restrict__ idx_out,
                    float* __restrict__ logits_out, int T, int d, int E, int K, int Epad) {
    extern __shared__ float lg[];                 // [CT][Epad] logits of this CTA's tokens
    __shared__ float xs[CK][CT + 4];
    __shared__ float ws[CK][CE + 4];
    const int layer = blockIdx.y;
    x += (size_t)layer * T * d;
    w += (size_t)layer * E * d;
    if (idx_out) idx_out += (size_t)layer * T * K;
    if (logits_out) logits_out += (size_t)layer * T * E;

    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const int t0 = blockIdx.x * CT;
    const int xr = tid >> 2, xk = (tid & 3) * 4;          // x loader: token xr, k offset xk
    const int wr = tid >> 1, wk = (tid & 1) * 8;          // w loader: expert wr, k offset wk

    for (int e0 = 0; e0 < E; e0 += CE) {
        float acc[4][8] = {};
        for (int k0 = 0; k0 < d; k0 += CK) {
            float xv[4] = {0.f, 0.f, 0.f, 0.f}, wv[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            if (t0 + xr < T && k0 + xk < d) load4(x + (size_t)(t0 + xr) * d + k0 + xk, xv);
            if (e0 + wr < E && k0 + wk < d) {
                load4(w + (size_t)(e0 + wr) * d + k0 + wk, wv);
                load4(w + (size_t)(e0 + wr) * d + k0 + wk + 4, wv + 4);
            }
            __syncthreads();
#pragma unroll
            for (int i = 0; i < 4; ++i) xs[xk + i][xr] = xv[i];
#pragma unroll
            for (int i = 0; i < 8; ++i) ws[wk + i][wr] = wv[i];
            __syncthreads();
#pragma unroll
            for (int kk = 0; kk < CK; ++kk) {
                const float4 a = *reinterpret_cast<const float4*>(&xs[kk][ty * 4]);
                const float4 b0 = *reinterpret_cast<const float4*>(&ws[kk][tx * 8]);
                const float4 b1 = *reinterpret_cast<const float4*>(&ws[kk][tx * 8 + 4]);
                const float av[4] = {a.x, a.y, a.z, a.w};
                const float bv[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int e = e0 + tx * 8 + j;
                if (e < Epad) lg[(ty * 4 + i) * Epad + e] = e < E ? acc[i][j] : -INFINITY;
            }
    }
    __syncthreads();

    if (logits_out) {
        const int rows = min(CT, T - t0);
        for (int i = tid; i < rows * E; i += 256) {
            const int r = i / E, e = i - r * E;
            logits_out[(size_t)(t0 + r) * E + e] = lg[r * Epad + e];
        }
    }
    if (!idx_out) return;

    // top-K: one warp per token, each lane holds the logits of experts lane, lane+32, ...
    const int lane = tid & 31, warp = tid >> 5;
    for (int r = warp; r < CT && t0 + r < T; r += 8) {
        float v[kMaxPerLane];
#pragma unroll
        for (int i = 0; i < kMaxPerLane; ++i)
            v[i] = lane + 32 * i < Epad ? lg[r * Epad + lane + 32 * i] : -INFINITY;
        for (int j = 0; j < K; ++j) {
            float best = -INFINITY;
            int bi = 0x7fffffff;
#pragma unroll
            for (int i = 0; i < kMaxPerLane; ++i)
                if (v[i] > best) { best = v[i]; bi = lane + 32 * i; }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ob = __shfl_xor_sync(0xffffffffu, best, o);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                if (ob > best || (ob == best && oi < bi)) { best = ob; bi = oi; }
            }
#pragma unroll
            for (int i = 0; i < kMaxPerLane; ++i)
                if (lane + 32 * i == bi) v[i] = -INFINITY;
            if (lane == 0) idx_out[(size_t)(t0 + r) * K + j] = (IdxT)(bi < E ? bi : 0);
        }
    }
}

template <typename XT, typename WT, typename IdxT>
static r3_status launch_capture(const r3_shape* s, int L, const void* x, const void* w,
                                void* idx_out, float* logits_out, cudaStream_t cs) {
    const int Epad = (s->E + 31) / 32 * 32;
    const size_t smem = (size_t)CT * Epad * sizeof(float);
    auto kern = capture_topk_kernel<XT, WT, IdxT>;
    if (smem > 32 * 1024) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
            cudaSuccess)
            return R3_ERR_CUDA;
    }
    dim3 grid((s->T + CT - 1) / CT, L);
    kern<<<grid, 256, smem, cs>>>(static_cast<const XT*>(x), static_cast<const WT*>(w),
                                  static_cast<IdxT*>(idx_out), logits_out, s->T, s->d, s->E, s->K,
                                  Epad);
    return launch_status();
}

static r3_status capture_dispatch(const r3_shape* s, int L, const void* x, const void* w,
                                  void* idx_out, float* logits_out, cudaStream_t cs) {
    const bool xb = s->act_dtype == R3_BF16, wb = s->router_w_dtype == R3_BF16;
    const bool u8 = s->idx_type == R3_IDX_U8;
#define R3_CAP(XT, WT)                                                                        \
    (u8 ? launch_capture<XT, WT, uint8_t>(s, L, x, w, idx_out, logits_out, cs)                \
        : launch_capture<XT, WT, int16_t>(s, L, x, w, idx_out, logits_out, cs))
    if (xb && wb) return R3_CAP(__nv_bfloat16, __nv_bfloat16);
    if (xb) return R3_CAP(__nv_bfloat16, float);
    if (wb) return R3_CAP(float, __nv_bfloat16);
    return R3_CAP(float, float);
#undef R3_CAP
}

}  // namespace r3

namespace r3 {
// Shared body: tensor-core kernel when the shape allows it (and, for float32 router weights, when
// the caller supplied scratch for the bf16 planes), otherwise the float32 FMA kernel.
static r3_status capture_any(const r3_shape* shape, int32_t L, const void* x, const void* w_router,
                             void* idx_out, float* logits_out, void* workspace, size_t ws_bytes,
                             void* stream) {
    r3_status st = check_shape(shape);
    if (st != R3_OK) return st;
    if (L < 0 || L > 65535) return R3_ERR_INVALID_ARG;
    if (shape->T == 0 || L == 0) return R3_OK;
    if (!x || !w_router || (!idx_out && !logits_out)) return R3_ERR_INVALID_ARG;
    if (!aligned(x, 16) || !aligned(w_router, 16)) return R3_ERR_INVALID_ARG;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (router_tc_supported(shape)) {
        const size_t need = router_tc_workspace_bytes(shape, L);
        if (need == 0) return launch_router_tc(shape, L, x, w_router, idx_out, logits_out, nullptr, cs);
        if (workspace) {
            if (ws_bytes < need || !aligned(workspace, 256)) return R3_ERR_WORKSPACE;
            return launch_router_tc(shape, L, x, w_router, idx_out, logits_out, workspace, cs);
        }
    }
    if (shape->E > kMaxExpertsCapture) return R3_ERR_UNSUPPORTED;
    return capture_dispatch(shape, L, x, w_router, idx_out, logits_out, cs);
}
}  // namespace r3

extern "C" size_t r3_capture_topk_workspace_bytes(const r3_shape* shape, int32_t L) {
    if (r3::check_shape(shape) != R3_OK || L <= 0) return 0;
    return r3::router_tc_workspace_bytes(shape, L);
}

extern "C" r3_status r3_capture_topk_ws(const r3_shape* shape, int32_t L, const void* x,
                                        const void* w_router, void* idx_out, float* logits_out,
                                        void* workspace, size_t ws_bytes, void* stream) {
    return r3::capture_any(shape, L, x, w_router, idx_out, logits_out, workspace, ws_bytes, stream);
}

extern "C" r3_status r3_capture_topk_batched(const r3_shape* shape, int32_t L, const void* x,
                                             const void* w_router, void* idx_out,
                                             float* logits_out, void* stream) {
    return r3::capture_any(shape, L, x, w_router, idx_out, logits_out, nullptr, 0, stream);
}

extern "C" r3_status r3_capture_topk(const r3_shape* shape, const void* x, const void* w_router,
                                     void* idx_out, float* logits_out, void* stream) {
    return r3::capture_any(shape, 1, x, w_router, idx_out, logits_out, nullptr, 0, stream);
}
