// Gate-weighted combine (Eq. replay_output) and its gradient with respect to the gates.
// Memory-bound gathers of K expert-output rows per token; fixed summation order, no atomics.
#include "r3_common.cuh"

namespace r3 {

constexpr int kSlotBatch = 8;     // slots gathered together (their loads are issued back to back)

// A team of TPT threads serves one token; 256/TPT tokens per CTA.
template <typename ActT, int TPT>
__global__ void __launch_bounds__(256)
combine_kernel(const ActT* __restrict__ o, const int32_t* __restrict__ row_of_slot,
               const float* __restrict__ gates, const ActT* __restrict__ residual,
               ActT* __restrict__ y, int T, int K, int d) {
    using V = Vec16<ActT>;
    constexpr int N = V::N;
    const int team = threadIdx.x / TPT, tl = threadIdx.x % TPT;
    const int t = blockIdx.x * (256 / TPT) + team;
    if (t >= T) return;
    const int row_vecs = d / N;
    const int32_t* rows = row_of_slot + (size_t)t * K;
    const float* g = gates + (size_t)t * K;
    const V* ov = reinterpret_cast<const V*>(o);
    V* yv = reinterpret_cast<V*>(y) + (size_t)t * row_vecs;
    for (int c = tl; c < row_vecs; c += TPT) {
        float acc[N];
#pragma unroll
        for (int i = 0; i < N; ++i) acc[i] = 0.f;
        for (int j0 = 0; j0 < K; j0 += kSlotBatch) {
            int32_t r[kSlotBatch];
            float gj[kSlotBatch];
            V v[kSlotBatch];
#pragma unroll
            for (int u = 0; u < kSlotBatch; ++u) {
                const int j = j0 + u;
                r[u] = j < K ? rows[j] : -1;
                gj[u] = j < K ? g[j] : 0.f;
            }
#pragma unroll
            for (int u = 0; u < kSlotBatch; ++u)
                if (r[u] >= 0) v[u] = ov[(size_t)r[u] * row_vecs + c];
#pragma unroll
            for (int u = 0; u < kSlotBatch; ++u) {
                if (r[u] >= 0) {
                    float f[N];
                    v[u].unpack(f);
#pragma unroll
                    for (int i = 0; i < N; ++i) acc[i] = fmaf(gj[u], f[i], acc[i]);
                }
            }
        }
        if (residual) {                      // y = residual + sum (one extra fp32 add per element)
            float f[N];
            reinterpret_cast<const V*>(residual)[(size_t)t * row_vecs + c].unpack(f);
#pragma unroll
            for (int i = 0; i < N; ++i) acc[i] += f[i];
        }
        V out;
        out.pack(acc);
        yv[c] = out;
    }
}

template <typename ActT, int TPT>
__global__ void __launch_bounds__(256)
combine_bwd_gates_kernel(const ActT* __restrict__ dy, const ActT* __restrict__ o,
                         const int32_t* __restrict__ row_of_slot, float* __restrict__ dgates,
                         int T, int K, int d) {
    using V = Vec16<ActT>;
    constexpr int N = V::N;
    constexpr int WPT = TPT / 32;                      // warps per team
    __shared__ float part[256 / 32][kSlotBatch];
    const int team = threadIdx.x / TPT, tl = threadIdx.x % TPT;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int t = blockIdx.x * (256 / TPT) + team;
    const bool live = t < T;                           // no early exit: block-wide barriers below
    const int tt = live ? t : T - 1;
    const int row_vecs = d / N;
    const int32_t* rows = row_of_slot + (size_t)tt * K;
    const V* dyv = reinterpret_cast<const V*>(dy) + (size_t)tt * row_vecs;
    const V* ov = reinterpret_cast<const V*>(o);
    for (int j0 = 0; j0 < K; j0 += kSlotBatch) {
        int32_t r[kSlotBatch];
        float acc[kSlotBatch];
#pragma unroll
        for (int u = 0; u < kSlotBatch; ++u) {
            const int j = j0 + u;
            r[u] = j < K ? rows[j] : -1;
            acc[u] = 0.f;
        }
        for (int c = tl; c < row_vecs; c += TPT) {
            float g[N];
            dyv[c].unpack(g);
            V v[kSlotBatch];
#pragma unroll
            for (int u = 0; u < kSlotBatch; ++u)
                if (r[u] >= 0) v[u] = ov[(size_t)r[u] * row_vecs + c];
#pragma unroll
            for (int u = 0; u < kSlotBatch; ++u) {
                if (r[u] >= 0) {
                    float f[N];
                    v[u].unpack(f);
#pragma unroll
                    for (int i = 0; i < N; ++i) acc[u] = fmaf(g[i], f[i], acc[u]);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kSlotBatch; ++u) {
#pragma unroll
            for (int s = 16; s > 0; s >>= 1) acc[u] += __shfl_xor_sync(0xffffffffu, acc[u], s);
        }
        if (lane == 0) {
#pragma unroll
            for (int u = 0; u < kSlotBatch; ++u) part[warp][u] = acc[u];
        }
        __syncthreads();
        if (live && tl < kSlotBatch && j0 + tl < K) {
            float s = 0.f;
            for (int w = 0; w < WPT; ++w) s += part[team * WPT + w][tl];   // fixed order
            dgates[(size_t)t * K + j0 + tl] = s;
        }
        __syncthreads();
    }
}

static int pick_team(int row_vecs) {
    int tpt = 32;
    while (tpt < 256 && tpt < row_vecs) tpt <<= 1;
    return tpt;
}

template <typename ActT>
static void launch_combine(const r3_shape* s, const void* o, const int32_t* row_of_slot,
                           const float* gates, const void* residual, void* y, cudaStream_t cs) {
    const int T = s->T, K = s->K, d = s->d;
    const int tpt = pick_team(d / Vec16<ActT>::N);
    const unsigned grid = (unsigned)((T + 256 / tpt - 1) / (256 / tpt));
    const ActT* op = static_cast<const ActT*>(o);
    ActT* yp = static_cast<ActT*>(y);
    const ActT* rp = static_cast<const ActT*>(residual);
    switch (tpt) {
        case 32: combine_kernel<ActT, 32><<<grid, 256, 0, cs>>>(op, row_of_slot, gates, rp, yp, T, K, d); break;
        case 64: combine_kernel<ActT, 64><<<grid, 256, 0, cs>>>(op, row_of_slot, gates, rp, yp, T, K, d); break;
        case 128: combine_kernel<ActT, 128><<<grid, 256, 0, cs>>>(op, row_of_slot, gates, rp, yp, T, K, d); break;
        default: combine_kernel<ActT, 256><<<grid, 256, 0, cs>>>(op, row_of_slot, gates, rp, yp, T, K, d); break;
    }
}

template <typename ActT>
static void launch_combine_bwd(const r3_shape* s, const void* dy, const void* o,
                               const int32_t* row_of_slot, float* dgates, cudaStream_t cs) {
    const int T = s->T, K = s->K, d = s->d;
    const int tpt = pick_team(d / Vec16<ActT>::N);
    const unsigned grid = (unsigned)((T + 256 / tpt - 1) / (256 / tpt));
    const ActT* dp = static_cast<const ActT*>(dy);
    const ActT* op = static_cast<const ActT*>(o);
    switch (tpt) {
        case 32: combine_bwd_gates_kernel<ActT, 32><<<grid, 256, 0, cs>>>(dp, op, row_of_slot, dgates, T, K, d); break;
        case 64: combine_bwd_gates_kernel<ActT, 64><<<grid, 256, 0, cs>>>(dp, op, row_of_slot, dgates, T, K, d); break;
        case 128: combine_bwd_gates_kernel<ActT, 128><<<grid, 256, 0, cs>>>(dp, op, row_of_slot, dgates, T, K, d); break;
        default: combine_bwd_gates_kernel<ActT, 256><<<grid, 256, 0, cs>>>(dp, op, row_of_slot, dgates, T, K, d); break;
    }
}

}  // namespace r3

extern "C" r3_status r3_combine_residual(const r3_shape* shape, const void* o,
                                         const int32_t* row_of_slot, const float* gates,
                                         const void* residual, void* y, void* stream) {
    r3_status st = r3::check_shape(shape);
    if (st != R3_OK) return st;
    if (shape->T == 0) return R3_OK;
    if (!o || !row_of_slot || !gates || !y) return R3_ERR_INVALID_ARG;
    if (!r3::aligned(o, 16) || !r3::aligned(y, 16) || !r3::aligned(residual, 16))
        return R3_ERR_INVALID_ARG;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    R3_DISPATCH_ACT(shape, ActT,
                    r3::launch_combine<ActT>(shape, o, row_of_slot, gates, residual, y, cs));
    return r3::launch_status();
}

extern "C" r3_status r3_combine(const r3_shape* shape, const void* o, const int32_t* row_of_slot,
                                const float* gates, void* y, void* stream) {
    return r3_combine_residual(shape, o, row_of_slot, gates, nullptr, y, stream);
}

extern "C" r3_status r3_combine_bwd_gates(const r3_shape* shape, const void* dy, const void* o,
                                          const int32_t* row_of_slot, float* dgates,
                                          void* stream) {
    r3_status st = r3::check_shape(shape);
    if (st != R3_OK) return st;
    if (shape->T == 0) return R3_OK;
    if (!dy || !o || !row_of_slot || !dgates) return R3_ERR_INVALID_ARG;
    if (!r3::aligned(o, 16) || !r3::aligned(dy, 16)) return R3_ERR_INVALID_ARG;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    R3_DISPATCH_ACT(shape, ActT, r3::launch_combine_bwd<ActT>(shape, dy, o, row_of_slot, dgates, cs));
    return r3::launch_status();
}
