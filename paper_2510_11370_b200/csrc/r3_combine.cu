// Gate-weighted combine (Eq. replay_output) and its gradient with respect to the gates.
// Memory-bound gathers of K expert-output rows per token; fixed summation order, no atomics.
#include "r3_common.cuh"
#include "r3_tc.cuh"

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

// ---------------------------------------------------------------------------------------------
// Shared-memory-staged form of both kernels for K <= 8: one CTA of 4 warps per token.  The CTA
// first asks for the token's K expert-output rows (and its dy / residual row) with bulk
// asynchronous copies, one lane and one copy per row, completion counted on an mbarrier; the data
// in flight lives in shared memory rather than in registers, so six CTAs fit on an SM and keep
// about 200 KB of copies per SM in flight.  DO_Y: y = residual + sum_j g_j o_j in slot order (the
// same per-element order as combine_kernel).  DO_DG: dg_j = <dy, o_j>, summed per lane over the
// columns, across the warp, then over the four warps (fixed order).
// ---------------------------------------------------------------------------------------------
constexpr int kStageWarps = 4;
constexpr int kStageThreads = kStageWarps * 32;
constexpr int kStageHeader = 256;         // mbarrier, flags, row mask, partial sums
constexpr int kStageMaxK = 8;
constexpr int kStageSmemLimit = 113 * 1024;

__device__ __forceinline__ void bulk_row_load(uint32_t dst, const void* src, uint32_t bytes,
                                              uint32_t bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

template <typename ActT, bool DO_Y, bool DO_DG>
__global__ void __launch_bounds__(kStageThreads)
gather_staged_kernel(const ActT* __restrict__ o, const int32_t* __restrict__ row_of_slot,
                     const float* __restrict__ gates, const ActT* __restrict__ residual,
                     const ActT* __restrict__ dy, ActT* __restrict__ y,
                     float* __restrict__ dgates, int K, int d) {
    using V = Vec16<ActT>;
    constexpr int N = V::N;
    extern __shared__ __align__(128) uint8_t smem_g[];
    const uint32_t bar = tc::smem_u32(smem_g);
    volatile int* flags = reinterpret_cast<volatile int*>(smem_g + 8);      // [0] abort [1] ready
    unsigned* have_s = reinterpret_cast<unsigned*>(smem_g + 16);
    float* part = reinterpret_cast<float*>(smem_g + 128);                    // [4 warps][8]
    const V* orow = reinterpret_cast<const V*>(smem_g + kStageHeader);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int t = blockIdx.x;
    const int row_vecs = d / N;
    const uint32_t row_bytes = (uint32_t)d * sizeof(ActT);
    const bool has_res = DO_Y && residual != nullptr;
    const int extra_dy = K, extra_res = K + (DO_DG ? 1 : 0);     // row slots after the K rows

    // the token's gates are read while the copies fly, not after them
    float gj[kStageMaxK];
#pragma unroll
    for (int u = 0; u < kStageMaxK; ++u) gj[u] = (DO_Y && u < K) ? gates[(size_t)t * K + u] : 0.f;

    if (warp == 0) {
        int32_t r = -1;
        if (lane < K) r = row_of_slot[(size_t)t * K + lane];
        if (lane == 0) {
            tc::mbar_init(bar, 1);
            flags[0] = 0;
            tc::fence_barrier_init();
        }
        __syncwarp();
        const uint32_t s_rows = tc::smem_u32(orow);
        // dy and the residual row do not wait for the row numbers (bytes may land before the
        // barrier is told how many to expect: its one pending arrival keeps the phase open)
        if (DO_DG && lane == K) {
            bulk_row_load(s_rows + (uint32_t)extra_dy * row_bytes, dy + (size_t)t * d, row_bytes, bar);
        } else if (lane == K + 1) {
            if (has_res)
                bulk_row_load(s_rows + (uint32_t)extra_res * row_bytes, residual + (size_t)t * d,
                              row_bytes, bar);
        }
        const unsigned have = __ballot_sync(0xffffffffu, r >= 0);
        if (lane == 0) {
            *have_s = have;
            tc::mbar_expect_tx(bar, row_bytes * (uint32_t)(__popc(have) + (DO_DG ? 1 : 0) +
                                                           (has_res ? 1 : 0)));
        }
        __syncwarp();
        if (lane < K && r >= 0)
            bulk_row_load(s_rows + (uint32_t)lane * row_bytes, o + (size_t)r * d, row_bytes, bar);
        // one thread waits for the copies; the others sleep at the barrier below
        if (lane == 0) flags[1] = tc::mbar_wait(bar, 0u, flags, nullptr) ? 1 : 0;
    }
    __syncthreads();
    const bool ready = flags[1] != 0;

    float dacc[kStageMaxK];
#pragma unroll
    for (int u = 0; u < kStageMaxK; ++u) dacc[u] = 0.f;
    if (ready) {
        const unsigned have = *have_s;
        for (int c = tid; c < row_vecs; c += kStageThreads) {
            float gr[N], acc[N];
            if (DO_DG) orow[(size_t)extra_dy * row_vecs + c].unpack(gr);
#pragma unroll
            for (int k2 = 0; k2 < N; ++k2) acc[k2] = 0.f;
#pragma unroll
            for (int u = 0; u < kStageMaxK; ++u) {
                if (have >> u & 1u) {
                    float f[N];
                    orow[(size_t)u * row_vecs + c].unpack(f);
                    if (DO_Y) {
#pragma unroll
                        for (int k2 = 0; k2 < N; ++k2) acc[k2] = fmaf(gj[u], f[k2], acc[k2]);
                    }
                    if (DO_DG) {
#pragma unroll
                        for (int k2 = 0; k2 < N; ++k2) dacc[u] = fmaf(gr[k2], f[k2], dacc[u]);
                    }
                }
            }
            if (DO_Y) {
                if (has_res) {
                    float f[N];
                    orow[(size_t)extra_res * row_vecs + c].unpack(f);
#pragma unroll
                    for (int k2 = 0; k2 < N; ++k2) acc[k2] += f[k2];
                }
                V out;
                out.pack(acc);
                reinterpret_cast<V*>(y)[(size_t)t * row_vecs + c] = out;
            }
        }
    }
    if (DO_DG) {
#pragma unroll
        for (int u = 0; u < kStageMaxK; ++u) {
#pragma unroll
            for (int sft = 16; sft > 0; sft >>= 1)
                dacc[u] += __shfl_xor_sync(0xffffffffu, dacc[u], sft);
        }
        if (lane == 0) {
#pragma unroll
            for (int u = 0; u < kStageMaxK; ++u) part[warp * kStageMaxK + u] = dacc[u];
        }
        __syncthreads();
        if (ready && tid < K) {
            float sum = 0.f;
            for (int w2 = 0; w2 < kStageWarps; ++w2) sum += part[w2 * kStageMaxK + tid];
            dgates[(size_t)t * K + tid] = sum;
        }
    }
    if (!ready) {
        // the wait ran out: copies may still be in flight into this CTA's shared memory
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    }
}

// Launches the staged kernel when the token's rows fit; returns false otherwise.
template <typename ActT, bool DO_Y, bool DO_DG>
static bool launch_staged(const r3_shape* s, const void* o, const int32_t* row_of_slot,
                          const float* gates, const void* residual, const void* dy, void* y,
                          float* dgates, cudaStream_t cs) {
    if (s->K > kStageMaxK) return false;
    const int rows = s->K + (DO_DG ? 1 : 0) + ((DO_Y && residual) ? 1 : 0);
    const size_t smem = kStageHeader + (size_t)rows * s->d * sizeof(ActT);
    if (smem > (size_t)kStageSmemLimit) return false;
    auto kern = gather_staged_kernel<ActT, DO_Y, DO_DG>;
    static PerDevice attr_set;                 // one set of flags per instantiation
    if (!attr_set.done()) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kStageSmemLimit) != cudaSuccess) {
            cudaGetLastError();
            return false;                      // the register kernel takes over
        }
        attr_set.mark();
    }
    kern<<<s->T, kStageThreads, smem, cs>>>(
        static_cast<const ActT*>(o), row_of_slot, gates, static_cast<const ActT*>(residual),
        static_cast<const ActT*>(dy), static_cast<ActT*>(y), dgates, s->K, s->d);
    return true;
}

static int pick_team(int row_vecs) {
    int tpt = 32;
    while (tpt < 256 && tpt < row_vecs) tpt <<= 1;
    return tpt;
}

template <typename ActT>
static void launch_combine(const r3_shape* s, const void* o, const int32_t* row_of_slot,
                           const float* gates, const void* residual, void* y, cudaStream_t cs) {
    if (launch_staged<ActT, true, false>(s, o, row_of_slot, gates, residual, nullptr, y, nullptr, cs))
        return;
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
    if (launch_staged<ActT, false, true>(s, o, row_of_slot, nullptr, nullptr, dy, nullptr, dgates, cs))
        return;
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
