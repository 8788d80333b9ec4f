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

// One warp per token.  Lanes hold up to 32 slots at a time (e_j, v_j = g_j (dg_j - c)); every lane
// then assembles its 4-float pieces of the dense row from those slots and writes them, zeros
// included, so the row is written exactly once.
template <typename IdxT>
__global__ void __launch_bounds__(256)
replay_gate_bwd_kernel(const float* __restrict__ gates, const float* __restrict__ dgates,
                       const IdxT* __restrict__ idx, float* __restrict__ dlogits,
                       int T, int E, int K) {
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (t >= T) return;
    const size_t base = (size_t)t * K;

    float c = 0.f;
    for (int j = lane; j < K; j += 32) c += gates[base + j] * dgates[base + j];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);

    float* out = dlogits + (size_t)t * E;
    const int nchunk = (E + 3) >> 2;
    if (K <= 32) {
        int e = -1;
        float v = 0.f;
        if (lane < K) {
            e = idx_to_int(idx[base + lane]);
            v = gates[base + lane] * (dgates[base + lane] - c);
        }
        for (int ch = lane; ch < ((nchunk + 31) & ~31); ch += 32) {
            float r[4] = {0.f, 0.f, 0.f, 0.f};
            for (int j = 0; j < K; ++j) {
                const int ej = __shfl_sync(0xffffffffu, e, j);
                const float vj = __shfl_sync(0xffffffffu, v, j);
                if ((ej >> 2) == ch) r[ej & 3] = vj;
            }
            if (ch < nchunk) {
                const int e0 = ch << 2;
                if (e0 + 3 < E && (E & 3) == 0) {
                    *reinterpret_cast<float4*>(out + e0) = make_float4(r[0], r[1], r[2], r[3]);
                } else {
                    for (int q = 0; q < 4 && e0 + q < E; ++q) out[e0 + q] = r[q];
                }
            }
        }
    } else {
        // rare wide-K case: zero the row, then scatter (same warp, ordered by __syncwarp)
        for (int i = lane; i < E; i += 32) out[i] = 0.f;
        __syncwarp();
        for (int j = lane; j < K; j += 32) {
            const int e = idx_to_int(idx[base + j]);
            if (e >= 0 && e < E) out[e] = gates[base + j] * (dgates[base + j] - c);
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
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const int wpb = 8;
    const unsigned grid = (unsigned)((shape->T + wpb - 1) / wpb);
    R3_DISPATCH_IDX(shape, IdxT,
        r3::replay_gate_bwd_kernel<IdxT><<<grid, wpb * 32, 0, cs>>>(
            gates, dgates, static_cast<const IdxT*>(idx), dlogits, shape->T, shape->E, shape->K));
    return r3::launch_status();
}
