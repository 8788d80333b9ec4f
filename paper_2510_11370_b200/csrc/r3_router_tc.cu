// Router logits + TopKMask on the tcgen05 tensor cores (Section 4.1, first two equations), for
// bf16 activations.
//
//   s[t, i] = sum_c x[t, c] W_r[i, c]
//
// bf16 router weights are used as they are (one MMA pass).  float32 router weights are first
// split into three bf16 planes  w = hi + mid + lo  (hi = bf16(w), mid = bf16(w - hi),
// lo = bf16(w - hi - mid); 24 mantissa bits in all), and the three products are accumulated into
// the same fp32 TMEM accumulator: x is exact in bf16, so the logits keep float32-level accuracy
// while the contraction runs on the tensor pipe.
//
// When the tiles are few (a single layer's decode batch, or the training logits of a few thousand
// tokens: at most half as many tiles as SMs), two CTAs of a cluster share a tile: each contracts
// half of the k blocks into its own accumulator and finishes half of the tile's tokens, reading
// the other CTA's partial logits through distributed shared memory (the sum of the two partials is
// the same number in both CTAs).
//
// One CTA of 12 warps per 128-token tile: warp 0 lane 0 = TMA producer, warp 1 lane 0 = MMA
// issuer, warps 2-5 read the finished accumulator out of TMEM into a [128][E + 1] float tile in
// shared memory (the copy ring is free by then).  All 12 warps then finish tokens out of that
// tile, four at a time per warp: the lanes write the token's logits out coalesced and pick the K
// largest with K rounds of warp reductions on order-preserving integer keys (exact ties go to the
// lower expert).  A per-thread sorted insertion list, one thread per token, took 12 us of
// dependent compare-and-swaps per tile; this takes about a third of that.
#include "r3_common.cuh"
#include "r3_internal.h"
#include "r3_tc.cuh"

namespace r3 {
namespace rt {

using namespace tc;

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int UK = 16;
constexpr int A_BYTES = BM * BK * 2;
constexpr int THREADS = 12 * 32;           // producer, MMA issuer, 4 TMEM readers; all 12 pick top-K
constexpr int BAR_BYTES = 256;
constexpr int MAX_STAGES = 7;
constexpr int KMAX = 16;                 // longest record the register top-K list supports
constexpr int SMEM_LIMIT = 227 * 1024;

__global__ void __launch_bounds__(256)
split_router_weight_kernel(const float* __restrict__ w, __nv_bfloat16* __restrict__ planes,
                           long long per_layer, long long total) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    const long long l = i / per_layer, r = i - l * per_layer;
    const float v = w[i];
    const __nv_bfloat16 hi = __float2bfloat16_rn(v);
    const float r1 = v - __bfloat162float(hi);
    const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
    const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
    __nv_bfloat16* base = planes + l * 3 * per_layer + r;
    base[0] = hi;
    base[per_layer] = mid;
    base[2 * per_layer] = lo;
}

// One warp finishes NT tokens at a time out of the shared-memory logits tile: lane l holds the
// logits of experts l + 32 s (slot s), writes them out (coalesced) and, if a record is wanted,
// picks the K largest by K rounds of warp reductions on order-preserving integer keys; exact ties
// go to the lower expert.  NT tokens are interleaved so that their reduction chains overlap.
template <typename IdxT, int SLOTS, int NT>
__device__ __forceinline__ void finish_tokens(const float* tile, int LD, const int* rows, int n_rows,
                                              int lane, int E, int K, size_t out_row0,
                                              IdxT* idx_out, float* logits_out,
                                              uint32_t peer_tile) {
    uint32_t key[NT][SLOTS];
    float val[NT][SLOTS];
    // all reads of the tile(s) first: the global stores below might alias them for the compiler
#pragma unroll
    for (int a = 0; a < NT; ++a) {
#pragma unroll
        for (int sl = 0; sl < SLOTS; ++sl) {
            const int e = lane + 32 * sl;
            val[a][sl] = 0.f;
            if (a < n_rows && e < E) {
                float v = tile[(size_t)rows[a] * LD + e];
                if (peer_tile) {                         // the other half of the contraction
                    float w;
                    asm volatile("ld.shared::cluster.f32 %0, [%1];"
                                 : "=f"(w) : "r"(peer_tile + 4u * (uint32_t)(rows[a] * LD + e)));
                    v += w;
                }
                val[a][sl] = v;
            }
        }
    }
#pragma unroll
    for (int a = 0; a < NT; ++a) {
#pragma unroll
        for (int sl = 0; sl < SLOTS; ++sl) {
            const int e = lane + 32 * sl;
            key[a][sl] = 0u;                             // 0 = no candidate (below every real key)
            if (a < n_rows && e < E) {
                const float v = val[a][sl];
                if (logits_out) logits_out[(out_row0 + rows[a]) * E + e] = v;
                // order-preserving key; -0.0 and +0.0 are one value (a tie: lower expert wins)
                uint32_t u = __float_as_uint(v);
                if (u == 0x80000000u) u = 0u;
                const uint32_t k2 = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
                key[a][sl] = k2 ? k2 : 1u;
            }
        }
    }
    if (!idx_out) return;
    int mine[NT];
#pragma unroll
    for (int a = 0; a < NT; ++a) mine[a] = 0;
    for (int j = 0; j < K; ++j) {
#pragma unroll
        for (int a = 0; a < NT; ++a) {
            uint32_t best = 0u;
#pragma unroll
            for (int sl = 0; sl < SLOTS; ++sl) best = max(best, key[a][sl]);
            const uint32_t top = __reduce_max_sync(0xffffffffu, best);
            uint32_t cand = 0xffffffffu;                 // lowest expert of this lane with that key
#pragma unroll
            for (int sl = SLOTS - 1; sl >= 0; --sl)
                if (key[a][sl] == top) cand = (uint32_t)(lane + 32 * sl);
            const uint32_t win = __reduce_min_sync(0xffffffffu, cand);
#pragma unroll
            for (int sl = 0; sl < SLOTS; ++sl)
                if (win == (uint32_t)(lane + 32 * sl)) key[a][sl] = 0u;
            if (lane == j) mine[a] = (int)win;
        }
    }
#pragma unroll
    for (int a = 0; a < NT; ++a)
        if (a < n_rows && lane < K) idx_out[(out_row0 + rows[a]) * K + lane] = (IdxT)mine[a];
}

template <typename IdxT, int KM>
__global__ void __launch_bounds__(THREADS, 1)
router_tc_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW,
                 IdxT* __restrict__ idx_out, float* __restrict__ logits_out, int T, int d, int E,
                 int K, int planes, int stages, uint32_t tmem_cols, int ksplit) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const int b_bytes = planes * E * BK * 2;
    const int stage_bytes = A_BYTES + b_bytes;
    const uint32_t bar0 = base + stages * stage_bytes;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (MAX_STAGES + s); };
    const uint32_t acc_bar = bar0 + 8u * (2 * MAX_STAGES);
    volatile uint32_t* tmem_slot =
        reinterpret_cast<volatile uint32_t*>(base_ptr + stages * stage_bytes + 128);
    volatile int* abort_flag =
        reinterpret_cast<volatile int*>(base_ptr + stages * stage_bytes + 132);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int layer = blockIdx.y;
    // ksplit = 2: the two CTAs of a cluster (consecutive blockIdx.x) share a tile
    const int rank = ksplit == 2 ? (int)cluster_ctarank() : 0;
    const int t0 = (ksplit == 2 ? (int)(blockIdx.x >> 1) : (int)blockIdx.x) * BM;
    const int kblocks = (d + BK - 1) / BK;
    const int kb_per = (kblocks + ksplit - 1) / ksplit;
    const int kb0 = rank * kb_per, kb1 = min(kblocks, kb0 + kb_per);    // this CTA's k blocks

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(acc_bar, 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            for (int kb = kb0; kb < kb1; ++kb) {
                if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, nullptr)) break;
                const uint32_t sa = base + stage * stage_bytes, sb = sa + A_BYTES;
                mbar_expect_tx(full_bar(stage), (uint32_t)stage_bytes);
                tma_load_2d(sa, &tmX, kb * BK, layer * T + t0, full_bar(stage));
                for (int p = 0; p < planes; ++p)
                    tma_load_2d(sb + p * E * BK * 2, &tmW, kb * BK, (layer * planes + p) * E,
                                full_bar(stage));
                if (++stage == stages) { stage = 0; phase ^= 1u; }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = instr_desc_bf16(BM, E);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int kb = kb0; kb < kb1 && ok; ++kb) {
                if (!mbar_wait(full_bar(stage), phase, abort_flag, nullptr)) { ok = false; break; }
                tc_fence_after();
                const uint32_t sa = base + stage * stage_bytes, sb = sa + A_BYTES;
                const uint64_t da = smem_desc_sw128(sa);
                for (int p = 0; p < planes; ++p) {
                    const uint64_t db = smem_desc_sw128(sb + p * E * BK * 2);
#pragma unroll
                    for (int kk = 0; kk < BK / UK; ++kk)
                        tc_mma_bf16(tmem_base, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2),
                                    idesc, ((kb - kb0) | p | kk) != 0 ? 1u : 0u);
                }
                tc_commit(empty_bar(stage));
                if (++stage == stages) { stage = 0; phase ^= 1u; }
            }
            if (ok && kb1 > kb0) tc_commit(acc_bar);
        }
        __syncwarp();
    } else if (warp < 6) {
        // ------------------------------ epilogue, part 1 --------------------------------------
        // every epilogue warp dumps its 32 tokens' logits from tensor memory into a [128][E + 1]
        // float tile in shared memory (the copy ring is free once the accumulator is complete)
        const int q = warp & 3;
        float* tile = reinterpret_cast<float*>(base_ptr);
        float* trow = tile + (size_t)(q * 32 + lane) * (E + 1);
        if (kb1 <= kb0) {
            for (int c = 0; c < E; ++c) trow[c] = 0.f;      // no k block fell to this CTA
        } else if (__all_sync(0xffffffffu, mbar_wait(acc_bar, 0u, abort_flag, nullptr))) {
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
            for (int c = 0; c < E; c += 32) {
                float v[32];
                tc_ld32(taddr + c, v);
                tc_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (c + i < E) trow[c + i] = v[i];
            }
        }
    }
    // ------------------------------ epilogue, part 2: all twelve warps, a few tokens each -------
    tc_fence_before();
    __syncthreads();
    if (ksplit == 2) cluster_sync_all();       // the other CTA's partial logits are in its tile
    if (!*abort_flag) {
        const float* tile = reinterpret_cast<const float*>(base_ptr);
        const uint32_t peer_tile = ksplit == 2 ? mapa_shared(smem_u32(tile), (uint32_t)(rank ^ 1)) : 0u;
        // with a shared tile each CTA finishes half of its tokens
        const int n_all = min(BM, T - t0);
        const int tok_lo = ksplit == 2 ? rank * (BM / 2) : 0;
        const int n_tok = ksplit == 2 ? min(n_all, tok_lo + BM / 2) : n_all;
        constexpr int NT = 4, NW = THREADS / 32;
        for (int r0 = tok_lo + warp * NT; r0 < n_tok; r0 += NW * NT) {
            int rows[NT];
#pragma unroll
            for (int a = 0; a < NT; ++a) rows[a] = min(r0 + a, n_tok - 1);
            const int n_rows = min(NT, n_tok - r0);
            const size_t out_row0 = (size_t)layer * T + t0;
            if (E <= 128)
                finish_tokens<IdxT, 4, NT>(tile, E + 1, rows, n_rows, lane, E, K, out_row0, idx_out,
                                           logits_out, peer_tile);
            else
                finish_tokens<IdxT, 8, NT>(tile, E + 1, rows, n_rows, lane, E, K, out_row0, idx_out,
                                           logits_out, peer_tile);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (ksplit == 2) cluster_sync_all();       // the other CTA may still be reading this tile
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, tmem_cols);
    }
}

}  // namespace rt

bool router_tc_supported(const r3_shape* s) {
    return s->act_dtype == R3_BF16 && s->E % 16 == 0 && s->E >= 16 && s->E <= 256 &&
           s->K <= rt::KMAX;
}

size_t router_tc_workspace_bytes(const r3_shape* s, int L) {
    if (!router_tc_supported(s) || s->router_w_dtype == R3_BF16) return 0;
    return round_up((size_t)L * 3 * s->E * s->d * sizeof(__nv_bfloat16), 256);
}

r3_status launch_router_tc(const r3_shape* s, int L, const void* x, const void* w_router,
                           void* idx_out, float* logits_out, void* workspace, cudaStream_t cs) {
    using namespace rt;
    const int planes = s->router_w_dtype == R3_BF16 ? 1 : 3;
    const void* wplanes = w_router;
    if (planes == 3) {
        const long long per_layer = (long long)s->E * s->d, total = per_layer * L;
        split_router_weight_kernel<<<(unsigned)((total + 255) / 256), 256, 0, cs>>>(
            static_cast<const float*>(w_router), static_cast<__nv_bfloat16*>(workspace), per_layer,
            total);
        wplanes = workspace;
    }
    const int stage_bytes = A_BYTES + planes * s->E * BK * 2;
    const int tiles = (s->T + BM - 1) / BM;
    const int kblocks = (s->d + BK - 1) / BK;
    // Few enough tiles that twice as many CTAs still get an SM each: two CTAs of a cluster share
    // a tile (half of the k blocks and half of the tokens each).  With more tiles than that the
    // shared form needs two CTAs per SM with half the ring each, which measured slower on the
    // 48-layer decode batch (29.4 us against 24.7 us).
    const int ksplit = ((long long)2 * tiles * L <= sm_count() && kblocks >= 2) ? 2 : 1;
    int stages = (SMEM_LIMIT - BAR_BYTES - 1024) / stage_bytes;
    if (stages > MAX_STAGES) stages = MAX_STAGES;
    if (stages < 2) return R3_ERR_UNSUPPORTED;
    const int tile_bytes = BM * (s->E + 1) * 4;        // the logits tile re-uses the ring
    int ring = stages * stage_bytes;
    if (ring < tile_bytes) ring = (tile_bytes + 1023) & ~1023;
    if (ring + BAR_BYTES + 1024 > SMEM_LIMIT) return R3_ERR_UNSUPPORTED;
    const int smem = ring + BAR_BYTES + 1024;
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < s->E) tmem_cols <<= 1;

    CUtensorMap mx, mw;
    if (!make_map_2d(&mx, x, (uint64_t)L * s->T, (uint64_t)s->d, BM) ||
        !make_map_2d(&mw, wplanes, (uint64_t)L * planes * s->E, (uint64_t)s->d, (uint32_t)s->E))
        return R3_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)ksplit;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.gridDim = dim3((unsigned)(tiles * ksplit), (unsigned)L);
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = cs;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
#define R3_RT(IDX, KM)                                                                          \
    do {                                                                                        \
        auto kern = router_tc_kernel<IDX, KM>;                                                  \
        static int attr_smem = 0;              /* largest size set so far, per instantiation */ \
        if (smem > attr_smem) {                                                                 \
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,         \
                                     SMEM_LIMIT) != cudaSuccess)                                \
                return R3_ERR_CUDA;                                                             \
            attr_smem = SMEM_LIMIT;                                                             \
        }                                                                                       \
        if (cudaLaunchKernelEx(&cfg, kern, mx, mw, static_cast<IDX*>(idx_out), logits_out,      \
                               (int)s->T, (int)s->d, (int)s->E, (int)s->K, planes, stages,      \
                               tmem_cols, ksplit) != cudaSuccess)                               \
            return R3_ERR_CUDA;                                                                 \
    } while (0)
    const bool u8 = s->idx_type == R3_IDX_U8;
    if (s->K <= 8) { if (u8) R3_RT(uint8_t, 8); else R3_RT(int16_t, 8); }
    else { if (u8) R3_RT(uint8_t, 16); else R3_RT(int16_t, 16); }
#undef R3_RT
    return launch_status();
}

}  // namespace r3
