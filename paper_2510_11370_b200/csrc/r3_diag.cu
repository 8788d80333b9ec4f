// Training/inference discrepancy measures (Sections 3.1 and 3.2 of the paper): reductions over
// per-token probabilities of the two engines and over two routing records.  All memory-bound.
//   Eq. (kl):    k3 estimate  (1/|T|) sum_t [ r_t - 1 - log r_t ],  r_t = p_train[t] / p_infer[t]
//   Eq. (etdf):  F(tau) |T| = number of tokens with max(r_t, 1/r_t) > tau
//   Section 3.2: per router (layer, token) the number of differing expert choices between two
//                records, K - |set_a & set_b|; per token its sum over the layers and the number of
//                layers that differ; per sequence the sum over its tokens of the latter.
// Determinism: floating-point sums are formed per thread, per warp, per CTA and then over the
// CTAs in a fixed order (two kernels, no floating-point atomics); counts are integers.
#include "r3_common.cuh"
#include "r3_internal.h"

namespace r3 {

constexpr int kMaxTaus = 16;
constexpr int kDiagThreads = 256;
constexpr int kFinalThreads = 1024;
constexpr int kMaxDiffK = 32;

// r - 1 - log r for r = a / b, in float32 without the cancellation of the literal form (for r
// near 1 the result is (r-1)^2 / 2, far below the rounding of r - 1 and log r taken separately):
// with u = (a - b) / b,  u - log(1 + u) = u^2 (1/2 - u/3 + u^2/4 - ...) for |u| < 1/4 (twelve
// terms: truncation below 2^-26 relative), the literal form otherwise (the result is then at
// least 0.026 and float32 rounding of its three parts stays below 1e-5 of it).  float64 would be
// exact to 1e-16 but runs at a small fraction of the float32 rate: the kernel would be bound by
// the float64 pipe, not by memory.
__device__ __forceinline__ float k3_term(float a, float b) {
    // a - b is exact for values within a factor of two; the quotient may be two units off in its
    // last place (the fast division), which is 2^-22 of the term: far inside its tolerance
    const float u = __fdividef(a - b, b);
    if (fabsf(u) < 0.25f) {
        float p = 1.f / 13.f;
#pragma unroll
        for (int k = 12; k >= 2; --k) p = fmaf(-u, p, 1.f / (float)k);
        return u * u * p;
    }
    return u - log1pf(u);
}

// NT = the number of thresholds rounded up to 4, 8 or 16 (unused ones are +inf: never exceeded).
// A thread takes 16-byte pieces (four tokens of each array), two pieces per round so that 64
// bytes per thread are in flight; the four k3 terms of a piece are added in float32 (a rounding of
// 2^-24 of their sum, far inside the 1e-5 that the estimate is compared within) and the piece
// sums in float64.  Arrays that do not start on a 16-byte boundary take the scalar loop.
template <int NT>
__global__ void __launch_bounds__(kDiagThreads)
prob_partial_kernel(const float* __restrict__ pt, const float* __restrict__ pi, long long n,
                    const float* __restrict__ taus, int n_tau, double* __restrict__ part_kl,
                    long long* __restrict__ part_cnt) {
    __shared__ double s_kl[kDiagThreads / 32];
    __shared__ long long s_cnt[kDiagThreads / 32][kMaxTaus];
    float tau[NT];
    int cnt[NT];
#pragma unroll
    for (int i = 0; i < NT; ++i) {
        tau[i] = i < n_tau ? taus[i] : INFINITY;
        cnt[i] = 0;
    }
    double acc = 0.0;
    auto one = [&](float a, float b) -> float {
        // the threshold decision is taken on float32 ratios, the precision of the inputs:
        // max(a / b, b / a) is the correctly rounded quotient of the larger by the smaller (one of
        // the two quotients is at least 1, the other at most 1, and rounding keeps that order)
        const float big = fmaxf(a, b) / fminf(a, b);
#pragma unroll
        for (int i = 0; i < NT; ++i) cnt[i] += big > tau[i] ? 1 : 0;
        return k3_term(a, b);
    };
    auto four = [&](const float4& a, const float4& b) {
        const float s0 = one(a.x, b.x), s1 = one(a.y, b.y), s2 = one(a.z, b.z), s3 = one(a.w, b.w);
        acc += (double)((s0 + s1) + (s2 + s3));
    };
    const long long stride = (long long)gridDim.x * blockDim.x;
    const long long gtid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const bool vec = ((reinterpret_cast<uintptr_t>(pt) | reinterpret_cast<uintptr_t>(pi)) & 15u) == 0;
    const long long n4 = vec ? n >> 2 : 0;
    const float4* pt4 = reinterpret_cast<const float4*>(pt);
    const float4* pi4 = reinterpret_cast<const float4*>(pi);
    long long v = gtid;
    for (; v + stride < n4; v += 2 * stride) {
        const float4 a0 = pt4[v], b0 = pi4[v], a1 = pt4[v + stride], b1 = pi4[v + stride];
        four(a0, b0);
        four(a1, b1);
    }
    if (v < n4) four(pt4[v], pi4[v]);
    for (long long t = 4 * n4 + gtid; t < n; t += stride) acc += (double)one(pt[t], pi[t]);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, s);
#pragma unroll
    for (int i = 0; i < NT; ++i) {
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) cnt[i] += __shfl_xor_sync(0xffffffffu, cnt[i], s);
    }
    if (lane == 0) {
        s_kl[warp] = acc;
#pragma unroll
        for (int i = 0; i < NT; ++i) s_cnt[warp][i] = cnt[i];
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        double k = 0.0;
        for (int w = 0; w < kDiagThreads / 32; ++w) k += s_kl[w];           // fixed order
        part_kl[blockIdx.x] = k;
    }
    if (threadIdx.x < n_tau) {
        long long c = 0;
        for (int w = 0; w < kDiagThreads / 32; ++w) c += s_cnt[w][threadIdx.x];
        part_cnt[(size_t)blockIdx.x * kMaxTaus + threadIdx.x] = c;
    }
}

// Sums the per-CTA partials: thread i takes partials i, i + 1024, ... (fixed), then the same warp
// and CTA reduction as above (one CTA of kFinalThreads threads).
__global__ void __launch_bounds__(kFinalThreads)
prob_final_kernel(const double* __restrict__ part_kl, const long long* __restrict__ part_cnt,
                  int parts, long long n, int n_tau, double* __restrict__ kl_out,
                  long long* __restrict__ counts_out) {
    __shared__ double s_kl[kFinalThreads / 32];
    __shared__ long long s_cnt[kFinalThreads / 32][kMaxTaus];
    double k = 0.0;
    long long c[kMaxTaus];
#pragma unroll
    for (int i = 0; i < kMaxTaus; ++i) c[i] = 0;
    for (int p = threadIdx.x; p < parts; p += kFinalThreads) {
        k += part_kl[p];
#pragma unroll
        for (int i = 0; i < kMaxTaus; ++i)
            if (i < n_tau) c[i] += part_cnt[(size_t)p * kMaxTaus + i];
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) k += __shfl_xor_sync(0xffffffffu, k, s);
#pragma unroll
    for (int i = 0; i < kMaxTaus; ++i) {
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) c[i] += __shfl_xor_sync(0xffffffffu, c[i], s);
    }
    if (lane == 0) {
        s_kl[warp] = k;
#pragma unroll
        for (int i = 0; i < kMaxTaus; ++i) s_cnt[warp][i] = c[i];
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        double tot = 0.0;
        for (int w = 0; w < kFinalThreads / 32; ++w) tot += s_kl[w];         // fixed order
        *kl_out = n > 0 ? tot / (double)n : 0.0;
    }
    if (threadIdx.x < n_tau) {
        long long tot = 0;
        for (int w = 0; w < kFinalThreads / 32; ++w) tot += s_cnt[w][threadIdx.x];
        counts_out[threadIdx.x] = tot;
    }
}

// One thread per token, looping over the layers (a warp reads 32 consecutive records of a layer).
template <typename IdxT>
__global__ void __launch_bounds__(kDiagThreads)
record_diff_kernel(const IdxT* __restrict__ ra, const IdxT* __restrict__ rb, int L, int T, int K,
                   uint8_t* __restrict__ diff_out, int32_t* __restrict__ token_choices,
                   int32_t* __restrict__ token_routers, unsigned long long* __restrict__ hist) {
    __shared__ unsigned int s_hist[kMaxDiffK + 1];
    for (int i = threadIdx.x; i <= K; i += blockDim.x) s_hist[i] = 0u;
    __syncthreads();
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t < T) {
        int choices = 0, routers = 0;
        for (int l = 0; l < L; ++l) {
            const IdxT* a = ra + ((size_t)l * T + t) * K;
            const IdxT* b = rb + ((size_t)l * T + t) * K;
            int same = 0;
            for (int i = 0; i < K; ++i) {
                const int ea = idx_to_int(a[i]);
                bool hit = false;
                for (int j = 0; j < K; ++j) hit |= idx_to_int(b[j]) == ea;
                same += hit ? 1 : 0;
            }
            const int dlt = K - same;
            choices += dlt;
            routers += dlt > 0 ? 1 : 0;
            atomicAdd(&s_hist[dlt], 1u);                         // integer: order-independent
            if (diff_out) diff_out[(size_t)l * T + t] = (uint8_t)dlt;
        }
        token_choices[t] = choices;
        token_routers[t] = routers;
    }
    __syncthreads();
    for (int i = threadIdx.x; i <= K; i += blockDim.x)
        if (s_hist[i]) atomicAdd(&hist[i], (unsigned long long)s_hist[i]);
}

// The common case K = 8 with one-byte ids: both records of a router are one 8-byte load each, and
// membership of an id in the other record is a zero-byte test on packed words.  A CTA takes 32
// tokens: lane = token (a warp reads 256 consecutive bytes of a layer), warp w the layers w,
// w + 8, ...; the per-token sums of the eight warps meet in shared memory.
__global__ void __launch_bounds__(kDiagThreads)
record_diff_k8_kernel(const uint2* __restrict__ ra, const uint2* __restrict__ rb, int L, int T,
                      uint8_t* __restrict__ diff_out, int32_t* __restrict__ token_choices,
                      int32_t* __restrict__ token_routers, unsigned long long* __restrict__ hist) {
    constexpr int W = kDiagThreads / 32;
    __shared__ unsigned int s_hist[9];
    __shared__ int s_choices[W][32], s_routers[W][32];
    if (threadIdx.x < 9) s_hist[threadIdx.x] = 0u;
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int t = blockIdx.x * 32 + lane;
    int choices = 0, routers = 0;
    if (t < T) {
        unsigned int local[9] = {0, 0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll 2
        for (int l = warp; l < L; l += W) {
            const uint2 a = ra[(size_t)l * T + t], b = rb[(size_t)l * T + t];
            int same = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const unsigned int ea = ((i < 4 ? a.x : a.y) >> (8 * (i & 3))) & 0xffu;
                const unsigned int rep = ea * 0x01010101u;
                // a byte of x is zero where the ids are equal; (x - 01..01) & ~x has the top bit of
                // a byte set if that byte is zero (and possibly of bytes above a zero one, which
                // does not matter for "any")
                const unsigned int x0 = rep ^ b.x, x1 = rep ^ b.y;
                const unsigned int z = ((x0 - 0x01010101u) & ~x0) | ((x1 - 0x01010101u) & ~x1);
                same += (z & 0x80808080u) != 0u ? 1 : 0;
            }
            const int dlt = 8 - same;
            choices += dlt;
            routers += dlt > 0 ? 1 : 0;
#pragma unroll
            for (int v = 0; v < 9; ++v) local[v] += dlt == v ? 1u : 0u;
            if (diff_out) diff_out[(size_t)l * T + t] = (uint8_t)dlt;
        }
#pragma unroll
        for (int v = 0; v < 9; ++v)
            if (local[v]) atomicAdd(&s_hist[v], local[v]);       // integer: order-independent
    }
    s_choices[warp][lane] = choices;
    s_routers[warp][lane] = routers;
    __syncthreads();
    if (warp == 0 && t < T) {
        int c = 0, r = 0;
#pragma unroll
        for (int w = 0; w < W; ++w) {
            c += s_choices[w][lane];
            r += s_routers[w][lane];
        }
        token_choices[t] = c;
        token_routers[t] = r;
    }
    if (threadIdx.x < 9 && s_hist[threadIdx.x])
        atomicAdd(&hist[threadIdx.x], (unsigned long long)s_hist[threadIdx.x]);
}

// One warp per sequence.
__global__ void __launch_bounds__(kDiagThreads)
sequence_sum_kernel(const int32_t* __restrict__ token_routers, const int32_t* __restrict__ cu, int S,
                    long long* __restrict__ seq_sum) {
    const int lane = threadIdx.x & 31;
    const int s = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (s >= S) return;
    const int lo = cu[s], hi = cu[s + 1];
    long long acc = 0;
    for (int t = lo + lane; t < hi; t += 32) acc += token_routers[t];
#pragma unroll
    for (int sft = 16; sft > 0; sft >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, sft);
    if (lane == 0) seq_sum[s] = acc;
}

static int prob_parts(long long n) {
    const long long want = (n + kDiagThreads * 8LL - 1) / (kDiagThreads * 8LL);
    const long long cap = 4LL * sm_count();
    const long long g = want < cap ? want : cap;
    return (int)(g > 0 ? g : 1);
}

}  // namespace r3

extern "C" size_t r3_prob_discrepancy_workspace_bytes(int64_t n) {
    if (n < 0) return 0;
    const size_t parts = (size_t)r3::prob_parts(n);
    return r3::round_up(parts * (sizeof(double) + r3::kMaxTaus * sizeof(long long)), 256);
}

extern "C" r3_status r3_prob_discrepancy(const float* p_train, const float* p_infer, int64_t n,
                                         const float* taus, int32_t n_tau, double* kl_out,
                                         int64_t* counts_out, void* workspace, size_t ws_bytes,
                                         void* stream) {
    if (n < 0 || n_tau < 0 || n_tau > r3::kMaxTaus) return R3_ERR_INVALID_ARG;
    if (!kl_out || (n_tau > 0 && (!taus || !counts_out)) || (n > 0 && (!p_train || !p_infer)))
        return R3_ERR_INVALID_ARG;
    if (!workspace || !r3::aligned(workspace, 256) ||
        ws_bytes < r3_prob_discrepancy_workspace_bytes(n))
        return R3_ERR_WORKSPACE;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const int parts = r3::prob_parts(n);
    double* part_kl = static_cast<double*>(workspace);
    long long* part_cnt = reinterpret_cast<long long*>(part_kl + parts);
    if (n_tau <= 4)
        r3::prob_partial_kernel<4><<<parts, r3::kDiagThreads, 0, cs>>>(p_train, p_infer, n, taus,
                                                                      n_tau, part_kl, part_cnt);
    else if (n_tau <= 8)
        r3::prob_partial_kernel<8><<<parts, r3::kDiagThreads, 0, cs>>>(p_train, p_infer, n, taus,
                                                                      n_tau, part_kl, part_cnt);
    else
        r3::prob_partial_kernel<16><<<parts, r3::kDiagThreads, 0, cs>>>(p_train, p_infer, n, taus,
                                                                       n_tau, part_kl, part_cnt);
    r3::prob_final_kernel<<<1, r3::kFinalThreads, 0, cs>>>(part_kl, part_cnt, parts, n, n_tau, kl_out,
                                            reinterpret_cast<long long*>(counts_out));
    return r3::launch_status();
}

extern "C" r3_status r3_record_diff(const r3_shape* shape, int32_t L, const void* rec_a,
                                    const void* rec_b, uint8_t* diff_out, int32_t* token_choices,
                                    int32_t* token_routers, int64_t* hist, void* stream) {
    r3_status st = r3::check_shape(shape);
    if (st != R3_OK) return st;
    if (L <= 0 || !hist) return R3_ERR_INVALID_ARG;
    if (shape->K > r3::kMaxDiffK) return R3_ERR_UNSUPPORTED;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(hist, 0, sizeof(int64_t) * (shape->K + 1), cs) != cudaSuccess)
        return R3_ERR_CUDA;
    if (shape->T == 0) return R3_OK;
    if (!rec_a || !rec_b || !token_choices || !token_routers) return R3_ERR_INVALID_ARG;
    const unsigned grid = (unsigned)((shape->T + r3::kDiagThreads - 1) / r3::kDiagThreads);
    if (shape->K == 8 && shape->idx_type == R3_IDX_U8 && r3::aligned(rec_a, 8) &&
        r3::aligned(rec_b, 8)) {
        r3::record_diff_k8_kernel<<<(unsigned)((shape->T + 31) / 32), r3::kDiagThreads, 0, cs>>>(
            static_cast<const uint2*>(rec_a), static_cast<const uint2*>(rec_b), L, shape->T,
            diff_out, token_choices, token_routers, reinterpret_cast<unsigned long long*>(hist));
        return r3::launch_status();
    }
    R3_DISPATCH_IDX(shape, IdxT,
        r3::record_diff_kernel<IdxT><<<grid, r3::kDiagThreads, 0, cs>>>(
            static_cast<const IdxT*>(rec_a), static_cast<const IdxT*>(rec_b), L, shape->T, shape->K,
            diff_out, token_choices, token_routers, reinterpret_cast<unsigned long long*>(hist)));
    return r3::launch_status();
}

extern "C" r3_status r3_sequence_diff(const int32_t* token_routers, const int32_t* cu_seqlens,
                                      int32_t S, int64_t* seq_sum, void* stream) {
    if (S < 0) return R3_ERR_INVALID_ARG;
    if (S == 0) return R3_OK;
    if (!token_routers || !cu_seqlens || !seq_sum) return R3_ERR_INVALID_ARG;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const int wpb = r3::kDiagThreads / 32;
    r3::sequence_sum_kernel<<<(S + wpb - 1) / wpb, r3::kDiagThreads, 0, cs>>>(
        token_routers, cu_seqlens, S, reinterpret_cast<long long*>(seq_sum));
    return r3::launch_status();
}
