// bf16 grouped SwiGLU expert GEMMs on the Blackwell tensor cores (sm_100a).
//
// Two persistent, warp-specialised kernels share one template:
//   MODE 0:  h[r, f]  = silu(xp[r] . W_gate,e[f]) * (xp[r] . W_up,e[f])      (K = d, N = F)
//   MODE 1:  o[r, c]  = h[r] . W_down,e[c]                                    (K = F, N = d)
// A CTA owns output tiles of 128 rows x 256 accumulator columns.  In MODE 0 the 256 columns are
// 128 gate columns followed by the 128 up columns of the same F slice (two TMA loads into one
// B tile), so the SwiGLU product is formed in the epilogue without repacking weights.
//
// Roles (320 threads): warp 0 lane 0 = TMA producer (cp.async.bulk.tensor into a 4-stage ring of
// 128B-swizzled tiles), warp 1 lane 0 = tcgen05.mma issuer (accumulators in TMEM, two stages of
// 256 columns so the epilogue of a tile overlaps the main loop of the next), warps 2..9 =
// epilogue (tcgen05.ld -> registers -> bf16 -> global).  Rows that belong to the next expert or
// lie beyond R are computed but never stored.
//
// Every mbarrier wait is bounded by a clock limit; when a wait runs out the CTA raises a shared
// abort flag, reports R3_DEV_TIMEOUT, lets the other roles drain, frees its TMEM and returns.
#include "r3_common.cuh"
#include "r3_internal.h"
#include "r3_tc.cuh"

namespace r3 {
namespace tc {

constexpr int BM = 128;            // rows per tile (UMMA M)
constexpr int BN = 256;            // accumulator columns per tile (UMMA N)
constexpr int BK = 64;             // k per stage: 64 bf16 = one 128-byte swizzle row
constexpr int UK = 16;             // k per tcgen05.mma (bf16)
constexpr int STAGES = 4;
constexpr int ACC_STAGES = 2;
constexpr int TMEM_COLS = ACC_STAGES * BN;       // 512 = all of tensor memory
constexpr int A_BYTES = BM * BK * 2;             // 16 KB
constexpr int B_BYTES = BN * BK * 2;             // 32 KB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int EPI_WARPS = 8;
constexpr int THREADS = (2 + EPI_WARPS) * 32;
constexpr int BAR_BYTES = 256;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + BAR_BYTES + 1024;   // + alignment slack

constexpr uint32_t kInstrDesc = instr_desc_bf16(BM, BN);

__device__ __forceinline__ void store8(__nv_bfloat16* dst, const float* f) {
    uint4 v;
    __nv_bfloat162* p = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) p[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
    *reinterpret_cast<uint4*>(dst) = v;
}

template <int MODE>
__global__ void __launch_bounds__(THREADS, 1)
grouped_gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA,
                       const __grid_constant__ CUtensorMap tmB0,
                       const __grid_constant__ CUtensorMap tmB1,
                       const int32_t* __restrict__ tiles, __nv_bfloat16* __restrict__ out,
                       int Kdim, int Nout, int n_blocks, int32_t* dev_status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bar0 = base + STAGES * STAGE_BYTES;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
    auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + ACC_STAGES + a); };
    volatile uint32_t* tmem_slot =
        reinterpret_cast<volatile uint32_t*>(base_ptr + STAGES * STAGE_BYTES + 128);
    volatile int* abort_flag =
        reinterpret_cast<volatile int*>(base_ptr + STAGES * STAGE_BYTES + 132);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_mtiles = tiles[0];
    const int total = num_mtiles * n_blocks;
    const int kblocks = (Kdim + BK - 1) / BK;
    const int4* ents = reinterpret_cast<const int4*>(tiles + kTileHeaderInts);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < ACC_STAGES; ++a) {
            mbar_init(tfull_bar(a), 1);
            mbar_init(tempty_bar(a), EPI_WARPS);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))), "r"((uint32_t)TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------ TMA producer ------------------------------------------
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int w = blockIdx.x; ok && w < total; w += gridDim.x) {
                const int4 ent = ents[w / n_blocks];
                const int n_blk = w % n_blocks;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, dev_status)) {
                        ok = false;
                        break;
                    }
                    const uint32_t sa = base + stage * STAGE_BYTES, sb = sa + A_BYTES;
                    mbar_expect_tx(full_bar(stage), STAGE_BYTES);
                    tma_load_2d(sa, &tmA, kb * BK, ent.y, full_bar(stage));
                    if (MODE == 0) {
                        tma_load_3d(sb, &tmB0, kb * BK, n_blk * (BN / 2), ent.x, full_bar(stage));
                        tma_load_3d(sb + B_BYTES / 2, &tmB1, kb * BK, n_blk * (BN / 2), ent.x,
                                    full_bar(stage));
                    } else {
                        tma_load_3d(sb, &tmB0, kb * BK, n_blk * BN, ent.x, full_bar(stage));
                    }
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ---------------------------------------------
        if (lane == 0) {
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int w = blockIdx.x; ok && w < total; w += gridDim.x) {
                if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, dev_status)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase, abort_flag, dev_status)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t sa = base + stage * STAGE_BYTES, sb = sa + A_BYTES;
                    const uint64_t da = smem_desc_sw128(sa), db = smem_desc_sw128(sb);
#pragma unroll
                    for (int kk = 0; kk < BK / UK; ++kk) {
                        // 16 bf16 = 32 bytes further along k inside the swizzled row
                        tc_mma_bf16(d_tmem, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2),
                                    kInstrDesc, (kb | kk) != 0 ? 1u : 0u);
                    }
                    tc_commit(empty_bar(stage));      // frees the stage when these MMAs retire
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                tc_commit(tfull_bar(acc));            // accumulator complete
                if (++acc == ACC_STAGES) { acc = 0; acc_phase ^= 1u; }
            }
        }
    } else {
        // ------------------------------ epilogue -----------------------------------------------
        const int q = warp & 3;                       // TMEM lane quadrant this warp may read
        const int half = (warp - 2) >> 2;             // which half of the columns it handles
        int acc = 0;
        uint32_t acc_phase = 0;
        for (int w = blockIdx.x; w < total; w += gridDim.x) {
            const int4 ent = ents[w / n_blocks];
            const int n_blk = w % n_blocks;
            if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag, dev_status)) break;
            tc_fence_after();
            const int r_in = q * 32 + lane;
            const bool row_ok = r_in < ent.z;
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN);
            __nv_bfloat16* orow = out + (size_t)(ent.y + r_in) * Nout;
            if (MODE == 0) {
                constexpr int HALF_N = BN / 2;        // 128 h columns per tile
#pragma unroll 1
                for (int c = 0; c < HALF_N / 2; c += 32) {
                    const int col = half * (HALF_N / 2) + c;
                    float g[32], u[32];
                    tc_ld32(taddr + col, g);
                    tc_ld32(taddr + HALF_N + col, u);
                    tc_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        g[i] = __fdividef(g[i], 1.f + __expf(-g[i])) * u[i];
                    const int n0 = n_blk * HALF_N + col;
                    if (row_ok) {
#pragma unroll
                        for (int i = 0; i < 32; i += 8)
                            if (n0 + i + 8 <= Nout) store8(orow + n0 + i, g + i);
                    }
                }
            } else {
#pragma unroll 1
                for (int c = 0; c < BN / 2; c += 32) {
                    const int col = half * (BN / 2) + c;
                    float v[32];
                    tc_ld32(taddr + col, v);
                    tc_wait_ld();
                    const int n0 = n_blk * BN + col;
                    if (row_ok) {
#pragma unroll
                        for (int i = 0; i < 32; i += 8)
                            if (n0 + i + 8 <= Nout) store8(orow + n0 + i, v + i);
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(acc));
            if (++acc == ACC_STAGES) { acc = 0; acc_phase ^= 1u; }
        }
    }

    // ------------------------------ teardown ---------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // copies may still be in flight into this CTA's shared memory: give them time to land
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
    }
}

}  // namespace tc

int tc_block_m() { return tc::BM; }

r3_status launch_grouped_swiglu_tc(const r3_shape* s, const void* xp, const int32_t* tiles,
                                   const void* w_gate, const void* w_up, const void* w_down,
                                   void* h, void* o, int32_t* dev_status, int phases,
                                   cudaStream_t cs) {
    using namespace tc;
    const long long R = (long long)s->T * s->K;
    const int mt = max_m_tiles(R, s->E, BM);
    if (mt == 0) return R3_OK;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(grouped_gemm_tc_kernel<0>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess ||
            cudaFuncSetAttribute(grouped_gemm_tc_kernel<1>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess)
            return R3_ERR_CUDA;
        attr_set = true;
    }
    const int sms = sm_count();
    if (phases & kPhaseUp) {
        CUtensorMap m_xp, m_g, m_u;
        if (!make_map_2d(&m_xp, xp, (uint64_t)R, (uint64_t)s->d, BM) ||
            !make_map_3d(&m_g, w_gate, s->E, s->F, s->d, BN / 2) ||
            !make_map_3d(&m_u, w_up, s->E, s->F, s->d, BN / 2))
            return R3_ERR_CUDA;
        const int nb1 = (s->F + BN / 2 - 1) / (BN / 2);
        const long long t1 = (long long)mt * nb1;
        const int g1 = (int)(t1 < sms ? t1 : sms);
        grouped_gemm_tc_kernel<0><<<g1, THREADS, SMEM_BYTES, cs>>>(
            m_xp, m_g, m_u, tiles, static_cast<__nv_bfloat16*>(h), s->d, s->F, nb1, dev_status);
    }
    if (phases & kPhaseDown) {
        CUtensorMap m_h, m_d;
        if (!make_map_2d(&m_h, h, (uint64_t)R, (uint64_t)s->F, BM) ||
            !make_map_3d(&m_d, w_down, s->E, s->d, s->F, BN))
            return R3_ERR_CUDA;
        const int nb2 = (s->d + BN - 1) / BN;
        const long long t2 = (long long)mt * nb2;
        const int g2 = (int)(t2 < sms ? t2 : sms);
        grouped_gemm_tc_kernel<1><<<g2, THREADS, SMEM_BYTES, cs>>>(
            m_h, m_d, m_d, tiles, static_cast<__nv_bfloat16*>(o), s->F, s->d, nb2, dev_status);
    }
    return launch_status();
}

}  // namespace r3
