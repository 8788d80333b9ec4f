// Update-stage backward of the replayed layer to its input and to the router weight (Section 4.1,
// purpose (b): the recorded mask is a constant, everything else is differentiated).  With
// g = replay gate, o_j = E_{e_j}(x_t), y_t = sum_j g_j o_j and dy = dL/dy:
//   dout[r]  = g[t,j] dy[t]                      for the grouped row r of pair (t, j)
//   dxp      = expert input gradient of dout      (r3_grouped_swiglu_bwd_input)
//   dx[t]    = sum_j dxp[row_of_slot[t,j]] + sum_j ds[t,e_j] W_r[e_j,:]
//   dW_r[e]  = sum over the tokens t whose record holds e of ds[t,e] x[t,:]
// where ds = dlogits is the router-logit gradient.  The memory-bound pieces live here; sums run in
// a fixed order in fp32 (no atomics).
#include "r3_common.cuh"
#include "r3_internal.h"

namespace r3 {

// One warp per token: dy[t] is read once and written, scaled by the token's K gates, to its K
// grouped rows.
template <typename ActT>
__global__ void __launch_bounds__(256)
scale_rows_kernel(const ActT* __restrict__ dy, const float* __restrict__ gates,
                  const int32_t* __restrict__ row_of_slot, ActT* __restrict__ dout, int T, int K,
                  int d) {
    using V = Vec16<ActT>;
    constexpr int N = V::N;
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (t >= T) return;
    const int row_vecs = d / N;
    const V* src = reinterpret_cast<const V*>(dy) + (size_t)t * row_vecs;
    V* dst = reinterpret_cast<V*>(dout);
    for (int c = lane; c < row_vecs; c += 32) {
        float f[N];
        src[c].unpack(f);
        for (int j = 0; j < K; ++j) {
            const int32_t r = row_of_slot[(size_t)t * K + j];
            if (r < 0) continue;
            const float g = gates[(size_t)t * K + j];
            float s[N];
#pragma unroll
            for (int i = 0; i < N; ++i) s[i] = g * f[i];
            V out;
            out.pack(s);
            dst[(size_t)r * row_vecs + c] = out;
        }
    }
}

// N consecutive router-weight elements (N = 4 or 8, the address a multiple of 16 bytes) as floats.
template <typename WrT, int N>
__device__ __forceinline__ void load_row_piece(const WrT* p, float* out);
template <> __device__ __forceinline__ void load_row_piece<float, 4>(const float* p, float* out) {
    const float4 v = *reinterpret_cast<const float4*>(p);
    out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
}
template <> __device__ __forceinline__ void load_row_piece<float, 8>(const float* p, float* out) {
    load_row_piece<float, 4>(p, out);
    load_row_piece<float, 4>(p + 4, out + 4);
}
template <>
__device__ __forceinline__ void load_row_piece<__nv_bfloat16, 8>(const __nv_bfloat16* p,
                                                                 float* out) {
    Vec16<__nv_bfloat16> v = *reinterpret_cast<const Vec16<__nv_bfloat16>*>(p);
    v.unpack(out);
}
template <>
__device__ __forceinline__ void load_row_piece<__nv_bfloat16, 4>(const __nv_bfloat16* p,
                                                                 float* out) {
    const uint2 raw = *reinterpret_cast<const uint2*>(p);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
    const float2 a = __bfloat1622float2(h[0]), b = __bfloat1622float2(h[1]);
    out[0] = a.x; out[1] = a.y; out[2] = b.x; out[3] = b.y;
}

// One CTA per token, a thread per 16-byte column piece: starting from the residual-path gradient
// (if any), the K expert-path rows are added in slot order, then the K router-path rows
// ds_j W_r[e_j] in slot order.  The token's K rows, experts and logit gradients are fetched once
// into shared memory, so the row loads of the sums are independent of each other.
constexpr int kDxMaxK = 64;
template <typename ActT, typename IdxT, typename WrT>
__global__ void __launch_bounds__(256)
dx_kernel(const ActT* __restrict__ dxp, const int32_t* __restrict__ row_of_slot,
          const float* __restrict__ dlogits, const IdxT* __restrict__ idx,
          const WrT* __restrict__ w_r, const ActT* __restrict__ dres, ActT* __restrict__ dx, int T,
          int E, int K, int d) {
    using V = Vec16<ActT>;
    constexpr int N = V::N;
    __shared__ int32_t s_row[kDxMaxK];
    __shared__ int32_t s_e[kDxMaxK];
    __shared__ float s_ds[kDxMaxK];
    const int t = blockIdx.x;
    if (threadIdx.x < K) {
        const int j = threadIdx.x;
        s_row[j] = row_of_slot[(size_t)t * K + j];
        const int e = idx_to_int(idx[(size_t)t * K + j]);
        const bool ok = e >= 0 && e < E;
        s_e[j] = ok ? e : -1;
        s_ds[j] = ok ? dlogits[(size_t)t * E + e] : 0.f;
    }
    __syncthreads();
    const int row_vecs = d / N;
    const V* pv = reinterpret_cast<const V*>(dxp);
    for (int c = threadIdx.x; c < row_vecs; c += blockDim.x) {
        float acc[N];
#pragma unroll
        for (int i = 0; i < N; ++i) acc[i] = 0.f;
        if (dres) reinterpret_cast<const V*>(dres)[(size_t)t * row_vecs + c].unpack(acc);
#pragma unroll 8
        for (int j = 0; j < K; ++j) {
            const int32_t r = s_row[j];
            if (r < 0) continue;
            float f[N];
            pv[(size_t)r * row_vecs + c].unpack(f);
#pragma unroll
            for (int i = 0; i < N; ++i) acc[i] += f[i];
        }
#pragma unroll 4
        for (int j = 0; j < K; ++j) {
            const int e = s_e[j];
            if (e < 0) continue;
            const float ds = s_ds[j];
            float wv[N];
            load_row_piece<WrT, N>(w_r + (size_t)e * d + (size_t)c * N, wv);
#pragma unroll
            for (int i = 0; i < N; ++i) acc[i] = fmaf(ds, wv[i], acc[i]);
        }
        V out;
        out.pack(acc);
        reinterpret_cast<V*>(dx)[(size_t)t * row_vecs + c] = out;
    }
}

// dW_r[e, c] = sum over the rows r of expert e of ds[token(r), e] * x[token(r), c].  Grid
// (E, blocks of 32 x N columns); each of the 8 warps takes the rows r = lo + warp, lo + warp + 8,
// ... (four in flight at a time), a lane owns one 16-byte piece of the row; the 8 partial sums are
// added in warp order.
template <typename ActT>
__global__ void __launch_bounds__(256)
dwr_kernel(const ActT* __restrict__ x, const float* __restrict__ dlogits,
           const int32_t* __restrict__ offsets, const int32_t* __restrict__ slot_of_row,
           float* __restrict__ dw_r, int E, int K, int d) {
    using V = Vec16<ActT>;
    constexpr int N = V::N;
    __shared__ float part[8][32][N + 1];
    const int e = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int c = (blockIdx.y * 32 + lane) * N;
    const bool in = c < d;                       // d is a multiple of 8
    const int lo = offsets[e], hi = offsets[e + 1];
    float acc[N];
#pragma unroll
    for (int i = 0; i < N; ++i) acc[i] = 0.f;
    for (int r = lo + warp; r < hi; r += 32) {
        float ds[4];
        V xv[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int ru = r + 8 * u;
            ds[u] = 0.f;
            if (ru < hi) {
                const int t = slot_of_row[ru] / K;
                ds[u] = dlogits[(size_t)t * E + e];
                if (in) xv[u] = *reinterpret_cast<const V*>(x + (size_t)t * d + c);
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (r + 8 * u < hi && in) {
                float f[N];
                xv[u].unpack(f);
#pragma unroll
                for (int i = 0; i < N; ++i) acc[i] = fmaf(ds[u], f[i], acc[i]);
            }
        }
    }
#pragma unroll
    for (int i = 0; i < N; ++i) part[warp][lane][i] = acc[i];
    __syncthreads();
    // thread (warp, lane) finishes column piece `lane`, elements warp, warp + 8, ... (< N)
    if (in) {
        for (int i = warp; i < N; i += 8) {
            float sum = part[0][lane][i];
#pragma unroll
            for (int wv = 1; wv < 8; ++wv) sum += part[wv][lane][i];
            dw_r[(size_t)e * d + c + i] = sum;
        }
    }
}

}  // namespace r3

extern "C" r3_status r3_scale_rows(const r3_shape* shape, const void* dy, const float* gates,
                                   const int32_t* row_of_slot, void* dout, void* stream) {
    r3_status st = r3::check_shape(shape);
    if (st != R3_OK) return st;
    if (shape->T == 0) return R3_OK;
    if (!dy || !gates || !row_of_slot || !dout) return R3_ERR_INVALID_ARG;
    if (!r3::aligned(dy, 16) || !r3::aligned(dout, 16)) return R3_ERR_INVALID_ARG;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const int wpb = 8;
    const unsigned grid = (unsigned)((shape->T + wpb - 1) / wpb);
    R3_DISPATCH_ACT(shape, ActT,
        r3::scale_rows_kernel<ActT><<<grid, wpb * 32, 0, cs>>>(
            static_cast<const ActT*>(dy), gates, row_of_slot, static_cast<ActT*>(dout), shape->T,
            shape->K, shape->d));
    return r3::launch_status();
}

extern "C" r3_status r3_input_grad_finish(const r3_shape* shape, const void* dxp,
                                          const int32_t* row_of_slot, const int32_t* slot_of_row,
                                          const int32_t* offsets, const float* dlogits,
                                          const void* idx, const void* x, const void* w_router,
                                          const void* dx_residual, void* dx, float* dw_router,
                                          void* stream) {
    r3_status st = r3::check_shape(shape);
    if (st != R3_OK) return st;
    if (shape->T == 0) return R3_OK;
    if (!dxp || !row_of_slot || !slot_of_row || !offsets || !dlogits || !idx || !x || !w_router ||
        !dx || !dw_router)
        return R3_ERR_INVALID_ARG;
    if (shape->K > r3::kDxMaxK) return R3_ERR_UNSUPPORTED;
    if (!r3::aligned(dxp, 16) || !r3::aligned(dx, 16) || !r3::aligned(dx_residual, 16) ||
        !r3::aligned(w_router, 16) ||
        dx_residual == dx)
        return R3_ERR_INVALID_ARG;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const int T = shape->T, E = shape->E, K = shape->K, d = shape->d;
    const bool wr_bf16 = shape->router_w_dtype == R3_BF16;
    R3_DISPATCH_ACT(shape, ActT, R3_DISPATCH_IDX(shape, IdxT, {
        if (wr_bf16)
            r3::dx_kernel<ActT, IdxT, __nv_bfloat16><<<T, 256, 0, cs>>>(
                static_cast<const ActT*>(dxp), row_of_slot, dlogits, static_cast<const IdxT*>(idx),
                static_cast<const __nv_bfloat16*>(w_router),
                static_cast<const ActT*>(dx_residual), static_cast<ActT*>(dx), T, E, K, d);
        else
            r3::dx_kernel<ActT, IdxT, float><<<T, 256, 0, cs>>>(
                static_cast<const ActT*>(dxp), row_of_slot, dlogits, static_cast<const IdxT*>(idx),
                static_cast<const float*>(w_router), static_cast<const ActT*>(dx_residual),
                static_cast<ActT*>(dx), T, E, K, d);
    }));
    R3_DISPATCH_ACT(shape, ActT,
        r3::dwr_kernel<ActT><<<dim3(E, (d + 32 * r3::Vec16<ActT>::N - 1) / (32 * r3::Vec16<ActT>::N)), 256, 0,
                              cs>>>(
            static_cast<const ActT*>(x), dlogits, offsets, slot_of_row, dw_router, E, K, d));
    return r3::launch_status();
}
