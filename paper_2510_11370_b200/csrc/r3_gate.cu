// Replay gate (Eq. replay_gate) and its backward: softmax of the training logits over the K
// recorded experts.  Memory-bound; reductions are warp shuffles in float32.
#include "r3_common.cuh"

namespace r3 {

// A group of W lanes (W = power of two, >= min(K,32)) serves one token; 32/W tokens per warp.
template <typename IdxT, int W>
__global__ void __launch_bounds__(256)
replay_gate_fwd_kernel(const float* __restrict__ logits, const IdxT* __restrict__ idx,
                       float* __restrict__ gates, int T, int E, int K, int32_t* dev_status) {
    const int l = threadIdx.x & (W - 1);
    const long long group = ((long long)blockIdx.x * blockDim.x + threadIdx.x) / W;
    // No early exit: every lane of the warp takes part in the shuffles; stores are predicated.
    const bool live = group < T;
    const int t = live ? (int)group : T - 1;
    const IdxT* rec = idx + (size_t)t * K;
    const float* row = logits + (size_t)t * E;

    // validity of the record: range and duplicates
    int bad = 0;
    for (int j = l; j < K; j += W) {
        const int e = idx_to_int(rec[j]);
        if (e < 0 || e >= E) bad |= 1;
        for (int j2 = 0; j2 < j; ++j2)
            if (idx_to_int(rec[j2]) == e) bad |= 2;
    }
#pragma unroll
    for (int o = W / 2; o > 0; o >>= 1) bad |= __shfl_xor_sync(0xffffffffu, bad, o, W);
    if (bad && live && l == 0)
        report(dev_status, (bad & 1) ? R3_DEV_BAD_INDEX : R3_DEV_DUP_INDEX);

    // out-of-range indices are clamped for the loads only; such a token's gates are written as 0
    float m = -INFINITY;
    for (int j = l; j < K; j += W) m = fmaxf(m, row[min(max(idx_to_int(rec[j]), 0), E - 1)]);
#pragma unroll
    for (int o = W / 2; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o, W));

    float sum = 0.f;
    for (int j = l; j < K; j += W)
        sum += expf(row[min(max(idx_to_int(rec[j]), 0), E - 1)] - m);
#pragma unroll
    for (int o = W / 2; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o, W);

    const float inv = bad ? 0.f : 1.f / sum;
    if (live)
        for (int j = l; j < K; j += W)
            gates[(size_t)t * K + j] =
                expf(row[min(max(idx_to_int(rec[j]), 0), E - 1)] - m) * inv;
}

// K <= 8: one lane per token.  The lane reads its record, fetches the K recorded logits (K
// independent loads in flight per lane) and forms the softmax in registers.  The sums are taken in
// the order of the W-lane butterfly above (W = K rounded up to a power of two, missing slots add
// 0), so both kernels give the same bits.
template <typename IdxT>
__global__ void __launch_bounds__(128)
replay_gate_fwd_lane_kernel(const float* __restrict__ logits, const IdxT* __restrict__ idx,
                            float* __restrict__ gates, int T, int E, int K, int W,
                            int32_t* dev_status) {
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    const IdxT* rec = idx + (size_t)t * K;
    const float* row = logits + (size_t)t * E;
    int e[8];
    int bad = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) e[j] = j < K ? idx_to_int(rec[j]) : -1 - j;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        if (j < K) {
            if (e[j] < 0 || e[j] >= E) bad |= 1;
#pragma unroll
            for (int j2 = 0; j2 < j; ++j2)
                if (e[j2] == e[j]) bad |= 2;
        }
    }
    if (bad) report(dev_status, (bad & 1) ? R3_DEV_BAD_INDEX : R3_DEV_DUP_INDEX);
    float sv[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) sv[j] = j < K ? row[min(max(e[j], 0), E - 1)] : -INFINITY;
    float m = sv[0];
#pragma unroll
    for (int j = 1; j < 8; ++j) m = fmaxf(m, sv[j]);
    float ex[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) ex[j] = j < K ? expf(sv[j] - m) : 0.f;
    float sum;
    if (W == 8) sum = ((ex[0] + ex[4]) + (ex[2] + ex[6])) + ((ex[1] + ex[5]) + (ex[3] + ex[7]));
    else if (W == 4) sum = (ex[0] + ex[2]) + (ex[1] + ex[3]);
    else if (W == 2) sum = ex[0] + ex[1];
    else sum = ex[0];
    const float inv = bad ? 0.f : 1.f / sum;
#pragma unroll
    for (int j = 0; j < 8; ++j)
        if (j < K) gates[(size_t)t * K + j] = ex[j] * inv;
}

// One warp per NT tokens, taken together so that their loads are in flight at once.  Per token
// the lanes hold up to 32 slots (e_j, v_j = g_j (dg_j - c)); every lane then assembles its 4-float
// pieces of the dense row from those slots and writes them, zeros included, so the row is written
// exactly once.
constexpr int kGateBwdTokens = 4;
template <typename IdxT>
__global__ void __launch_bounds__(256)
replay_gate_bwd_kernel(const float* __restrict__ gates, const float* __restrict__ dgates,
                       const IdxT* __restrict__ idx, float* __restrict__ dlogits,
                       int T, int E, int K, bool staged) {
    constexpr int NT = kGateBwdTokens;
    const int lane = threadIdx.x & 31;
    const long long t0 = ((long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * NT;
    if (t0 >= T) return;
    const int nchunk = (E + 3) >> 2;
    if (K <= 32) {
        float gl[NT], dl[NT];
        int e[NT];
#pragma unroll
        for (int a = 0; a < NT; ++a) {
            gl[a] = 0.f;
            dl[a] = 0.f;
            e[a] = -1;
            if (t0 + a < T && lane < K) {
                const size_t at = (size_t)(t0 + a) * K + lane;
                gl[a] = gates[at];
                dl[a] = dgates[at];
                e[a] = idx_to_int(idx[at]);
            }
        }
        float v[NT];
#pragma unroll
        for (int a = 0; a < NT; ++a) {
            float c = gl[a] * dl[a];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
            v[a] = gl[a] * (dl[a] - c);
        }
        if (staged) {
            // dense rows built in shared memory (zeros, then the K values) and written out in
            // 16-byte pieces: a dozen instructions per lane and token, where the scan below of
            // the K slots by every lane made the kernel issue-bound
            extern __shared__ __align__(16) float stage_all[];
            float* stage = stage_all + (size_t)(threadIdx.x >> 5) * NT * E;
#pragma unroll
            for (int a = 0; a < NT; ++a)
                for (int ch = lane; ch < nchunk; ch += 32)
                    reinterpret_cast<float4*>(stage + a * E)[ch] = make_float4(0.f, 0.f, 0.f, 0.f);
            __syncwarp();
#pragma unroll
            for (int a = 0; a < NT; ++a)
                if (e[a] >= 0 && e[a] < E) stage[a * E + e[a]] = v[a];
            __syncwarp();
#pragma unroll
            for (int a = 0; a < NT; ++a) {
                if (t0 + a >= T) break;                   // uniform across the warp
                float4* out = reinterpret_cast<float4*>(dlogits + (size_t)(t0 + a) * E);
                for (int ch = lane; ch < nchunk; ch += 32)
                    out[ch] = reinterpret_cast<const float4*>(stage + a * E)[ch];
            }
            return;
        }
#pragma unroll
        for (int a = 0; a < NT; ++a) {
            if (t0 + a >= T) break;                       // uniform across the warp
            float* out = dlogits + (size_t)(t0 + a) * E;
            for (int ch = lane; ch < ((nchunk + 31) & ~31); ch += 32) {
                // selects, no branches: the kernel is bound by instruction issue otherwise
                float r0 = 0.f, r1 = 0.f, r2 = 0.f, r3 = 0.f;
                auto place = [&](int j) {
                    const int ej = __shfl_sync(0xffffffffu, e[a], j);
                    const float vj = __shfl_sync(0xffffffffu, v[a], j);
                    const int q = (ej >> 2) == ch ? (ej & 3) : -1;
                    r0 = q == 0 ? vj : r0;
                    r1 = q == 1 ? vj : r1;
                    r2 = q == 2 ? vj : r2;
                    r3 = q == 3 ? vj : r3;
                };
                if (K <= 8) {
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        if (j < K) place(j);
                } else {
                    for (int j = 0; j < K; ++j) place(j);
                }
                if (ch < nchunk) {
                    const int e0 = ch << 2;
                    if (e0 + 3 < E && (E & 3) == 0) {
                        *reinterpret_cast<float4*>(out + e0) = make_float4(r0, r1, r2, r3);
                    } else {
                        const float r[4] = {r0, r1, r2, r3};
                        for (int q = 0; q < 4 && e0 + q < E; ++q) out[e0 + q] = r[q];
                    }
                }
            }
        }
    } else {
        // rare wide-K case: zero the row, then scatter (same warp, ordered by __syncwarp)
        for (int a = 0; a < NT && t0 + a < T; ++a) {
            const size_t base = (size_t)(t0 + a) * K;
            float* out = dlogits + (size_t)(t0 + a) * E;
            float c = 0.f;
            for (int j = lane; j < K; j += 32) c += gates[base + j] * dgates[base + j];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
            for (int i = lane; i < E; i += 32) out[i] = 0.f;
            __syncwarp();
            for (int j = lane; j < K; j += 32) {
                const int e = idx_to_int(idx[base + j]);
                if (e >= 0 && e < E) out[e] = gates[base + j] * (dgates[base + j] - c);
            }
        }
    }
}

template <typename IdxT>
static void launch_gate_fwd(const r3_shape* s, const float* logits, const void* idx, float* gates,
                            int32_t* dev_status, cudaStream_t st) {
    int W = 1;
    while (W < s->K && W < 32) W <<= 1;
    const long long threads = (long long)s->T * W;
    const int block = 256;
    const unsigned grid = (unsigned)((threads + block - 1) / block);
    const IdxT* ip = static_cast<const IdxT*>(idx);
    if (s->K <= 8) {
        replay_gate_fwd_lane_kernel<IdxT><<<(unsigned)((s->T + 127) / 128), 128, 0, st>>>(
            logits, ip, gates, s->T, s->E, s->K, W, dev_status);
        return;
    }
#define R3_GF(WW) replay_gate_fwd_kernel<IdxT, WW><<<grid, block, 0, st>>>( \
        logits, ip, gates, s->T, s->E, s->K, dev_status)
    switch (W) {
        case 1: R3_GF(1); break;
        case 2: R3_GF(2); break;
        case 4: R3_GF(4); break;
        case 8: R3_GF(8); break;
        case 16: R3_GF(16); break;
        default: R3_GF(32); break;
    }
#undef R3_GF
}

}  // namespace r3

extern "C" r3_status r3_replay_gate_fwd(const r3_shape* shape, const float* logits,
                                        const void* idx, float* gates, int32_t* dev_status,
                                        void* stream) {
    r3_status st = r3::check_shape(shape);
    if (st != R3_OK) return st;
    if (shape->T == 0) return R3_OK;
    if (!logits || !idx || !gates) return R3_ERR_INVALID_ARG;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    R3_DISPATCH_IDX(shape, IdxT, r3::launch_gate_fwd<IdxT>(shape, logits, idx, gates, dev_status, cs));
    return r3::launch_status();
}

extern "C" r3_status r3_replay_gate_bwd(const r3_shape* shape, const float* gates,
                                        const float* dgates, const void* idx, float* dlogits,
                                        void* stream) {
    r3_status st = r3::check_shape(shape);
    if (st != R3_OK) return st;
    if (shape->T == 0) return R3_OK;
    if (!gates || !dgates || !idx || !dlogits) return R3_ERR_INVALID_ARG;
    // rows are written in 16-byte pieces whenever E is a multiple of 4
    if (!r3::aligned(dlogits, 16)) return R3_ERR_INVALID_ARG;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const int wpb = 8;
    const int tpb = wpb * r3::kGateBwdTokens;               // tokens per block
    const unsigned grid = (unsigned)((shape->T + tpb - 1) / tpb);
    // rows staged in shared memory when they are 16-byte pieces and a block's rows fit 32 KB
    const size_t stage_bytes = (size_t)tpb * shape->E * sizeof(float);
    const bool staged = shape->K <= 32 && (shape->E & 3) == 0 && stage_bytes <= 32 * 1024;
    R3_DISPATCH_IDX(shape, IdxT,
        r3::replay_gate_bwd_kernel<IdxT><<<grid, wpb * 32, staged ? stage_bytes : 0, cs>>>(
            gates, dgates, static_cast<const IdxT*>(idx), dlogits, shape->T, shape->E, shape->K,
            staged));
    return r3::launch_status();
}
