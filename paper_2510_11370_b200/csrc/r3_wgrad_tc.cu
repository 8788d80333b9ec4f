// Expert-weight gradients of the grouped SwiGLU experts on the tensor cores (bf16 operands, float32
// result).  For expert e with grouped rows [offsets[e], offsets[e+1]):
//   dW_down[e] [d,F] = dout_e^T h_e      dW_gate[e] [F,d] = da_e^T xp_e      dW_up[e] [F,d] = db_e^T xp_e
// Every product contracts over the expert's token rows, so both operands are read "MN-major": a
// TMA box of 64 consecutive columns x 64 token rows lands as 64 swizzled 128-byte rows, and the
// tcgen05 descriptors walk the rows as the k dimension.  One CTA per SM (cta_group::1), float32
// accumulators in tensor memory, items (expert, problem, m tile, n tile) dealt round-robin.  Two
// tile shapes:
//   MT = 1: 128 x 256 outputs, two accumulator stages (a tile's epilogue runs under the next tile's
//           MMAs), 4 ring stages of 48 KB.  For few rows per expert, where the float32 result
//           written to HBM is the bound and the epilogue must never wait.
//   MT = 2: 256 x 256 outputs as two 128-row MMAs that share the B boxes, one accumulator stage
//           (all 512 columns), 3 ring stages of 64 KB.  For many rows per expert, where the bound
//           is the operand bytes each SM can draw from L2: 32 KB per SM and 64 token rows for
//           2 x 128 x 256 x 64 products, against 48 KB for half of that with MT = 1.
//
// The token count of an expert is ragged.  Rows of the last 64-row block that belong to the next
// expert must not contribute: whole 16-row MMA steps beyond the expert's end are not issued, and
// inside the last partial step the surplus rows are overwritten with zeros in shared memory (both
// operands) before the MMA reads them.
#include "r3_tc.cuh"
#include "r3_internal.h"

namespace r3 {
namespace wg {

using namespace tc;

constexpr int WM = 128;                 // output rows per tile (MMA M)
constexpr int WN = 256;                 // output columns per tile (MMA N)
constexpr int WK = 64;                  // token rows per pipeline stage
constexpr int UK = 16;                  // token rows per MMA
constexpr int BOX_BYTES = 64 * WK * 2;  // one TMA box: 64 columns x 64 rows of bf16
constexpr int EPI_WARPS = 8;                            // two per TMEM lane quadrant
constexpr int EPI_PER_Q = EPI_WARPS / 4;
constexpr int EPI_BYTES = EPI_WARPS * 32 * 32 * 4;      // a 32 x 32 float block per warp
constexpr int THREADS = 32 * (2 + EPI_WARPS);
constexpr int TMEM_COLS = 512;
constexpr int MAX_STAGES = 4;
template <int MT>
struct Shape {
    static constexpr int TILE_M = MT * WM;
    static constexpr int STAGES = MT == 1 ? 4 : 3;
    static constexpr int ACC_STAGES = 2 / MT;
    static constexpr int A_BYTES = (TILE_M / 64) * BOX_BYTES;
    static constexpr int B_BYTES = (WN / 64) * BOX_BYTES;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;          // 48 KB / 64 KB
    static constexpr int SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + EPI_BYTES + 256;
};
constexpr uint32_t kInstrDescBothMN = (1u << 15) | (1u << 16);
constexpr int MAX_PROBLEMS = 3;
constexpr int TALL_TILE_MIN_ROWS = 1024;   // average rows per expert from which MT = 2 is used

struct Problem {
    CUtensorMap a;      // [R, M] bf16, box 64 x 64
    CUtensorMap b;      // [R, N] bf16, box 64 x 64
    float* out;         // [E, M, N]
    int M, N;
    int mt, nt;         // tiles along M and N
    int tile0;          // first tile of this problem among an expert's tiles
};
struct Params {
    Problem p[MAX_PROBLEMS];
    int n_problems;
    int tiles_per_expert;   // over all problems
    int total_items;
};

struct Item {
    int q, e, m0, n0;
};
// Items run expert by expert (all tiles of all problems of an expert are neighbours, so the CTAs
// that run at the same time share that expert's operand rows in L2), then problem, m tile, n tile
// (neighbouring CTAs write neighbouring 1 KB pieces of the same gradient rows).
template <int MT>
__device__ __forceinline__ Item decode(const Params& P, int i) {
    const int e = i / P.tiles_per_expert, t = i - e * P.tiles_per_expert;
    int q = 0;
#pragma unroll
    for (int k = 1; k < MAX_PROBLEMS; ++k)
        if (k < P.n_problems && t >= P.p[k].tile0) q = k;
    const int rem = t - P.p[q].tile0;
    const int m = rem / P.p[q].nt, n = rem - m * P.p[q].nt;     // n fastest: neighbours fill a row
    return Item{q, e, m * (MT * WM), n * WN};
}

template <int MT>
__global__ void __launch_bounds__(THREADS, 1)
wgrad_kernel(const __grid_constant__ Params P, const int32_t* __restrict__ offsets,
             int32_t* dev_status) {
    using S = Shape<MT>;
    constexpr int STAGES = S::STAGES, ACC_STAGES = S::ACC_STAGES, STAGE_BYTES = S::STAGE_BYTES;
    constexpr int A_BYTES = S::A_BYTES;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    uint8_t* epi_ptr = base_ptr + STAGES * STAGE_BYTES;
    const uint32_t bar0 = base + STAGES * STAGE_BYTES + EPI_BYTES;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
    auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * MAX_STAGES + a); };
    auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * MAX_STAGES + 2 + a); };
    uint8_t* misc = epi_ptr + EPI_BYTES + 128;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(misc);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int w_begin = blockIdx.x, w_step = gridDim.x, w_end = P.total_items;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < ACC_STAGES; ++a) {
            mbar_init(tfull_bar(a), 1);
            mbar_init(tempty_bar(a), EPI_WARPS);
        }
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------ TMA producer -------------------------------------------
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int w = w_begin; ok && w < w_end; w += w_step) {
                const Item it = decode<MT>(P, w);
                const CUtensorMap* amap = &P.p[it.q].a;
                const CUtensorMap* bmap = &P.p[it.q].b;
                const int lo = offsets[it.e], hi = offsets[it.e + 1];
                for (int row = lo; row < hi; row += WK) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, dev_status)) {
                        ok = false;
                        break;
                    }
                    const uint32_t sa = base + stage * STAGE_BYTES, sb = sa + A_BYTES;
                    mbar_expect_tx(full_bar(stage), (uint32_t)STAGE_BYTES);
#pragma unroll
                    for (int bx = 0; bx < S::TILE_M / 64; ++bx)
                        tma_load_2d(sa + bx * BOX_BYTES, amap, it.m0 + 64 * bx, row,
                                    full_bar(stage));
#pragma unroll
                    for (int bx = 0; bx < WN / 64; ++bx)
                        tma_load_2d(sb + bx * BOX_BYTES, bmap, it.n0 + 64 * bx, row,
                                    full_bar(stage));
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            // every stage's release has landed before this CTA may leave
            for (int s = 0; ok && s < STAGES; ++s) {
                ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, dev_status);
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer (whole warp: it also clears ragged rows) -----
        int stage = 0, acc = 0;
        uint32_t phase = 0, acc_phase = 0;
        bool ok = true;
        constexpr uint32_t idesc = instr_desc_bf16(WM, WN) | kInstrDescBothMN;
        constexpr int HALF_A = (WM / 64) * BOX_BYTES;     // the A boxes of one 128-row half
        for (int w = w_begin; ok && w < w_end; w += w_step) {
            const Item it = decode<MT>(P, w);
            const int lo = offsets[it.e], hi = offsets[it.e + 1];
            int go = 1;
            if (lane == 0)
                go = mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, dev_status) ? 1 : 0;
            if (!__shfl_sync(0xffffffffu, go, 0)) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(acc * MT * WN);
            for (int row = lo; row < hi; row += WK) {
                if (lane == 0)
                    go = mbar_wait(full_bar(stage), phase, abort_flag, dev_status) ? 1 : 0;
                if (!__shfl_sync(0xffffffffu, go, 0)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint32_t sa = base + stage * STAGE_BYTES, sb = sa + A_BYTES;
                const int valid = min(WK, hi - row);
                const int ksteps = (valid + UK - 1) / UK;
                if (valid < ksteps * UK) {
                    // rows valid .. ksteps*16-1 of every box: 8 x 16 bytes per row and box
                    uint8_t* tile = base_ptr + stage * STAGE_BYTES;
                    const int n_rows = ksteps * UK - valid;
                    const int n_vec = n_rows * (STAGE_BYTES / BOX_BYTES) * 8;
                    for (int v = lane; v < n_vec; v += 32) {
                        const int piece = v & 7, rb = v >> 3;
                        const int r = valid + rb % n_rows, bx = rb / n_rows;
                        *reinterpret_cast<uint4*>(tile + bx * BOX_BYTES + r * 128 + piece * 16) =
                            make_uint4(0u, 0u, 0u, 0u);
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                }
                __syncwarp();
                if (lane == 0) {
                    const uint64_t db = smem_desc_mn_sw128(sb, BOX_BYTES);
#pragma unroll
                    for (int half = 0; half < MT; ++half) {
                        const uint64_t da = smem_desc_mn_sw128(sa + half * HALF_A, BOX_BYTES);
                        for (int kk = 0; kk < ksteps; ++kk)
                            tc_mma_bf16(d_tmem + (uint32_t)(half * WN),
                                        da + (uint64_t)(kk * (2048 >> 4)),
                                        db + (uint64_t)(kk * (2048 >> 4)), idesc,
                                        (row != lo || kk != 0) ? 1u : 0u);
                    }
                    tc_commit(empty_bar(stage));
                }
                __syncwarp();
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
            if (!ok) break;
            if (lane == 0) tc_commit(tfull_bar(acc));
            __syncwarp();
            if (++acc == ACC_STAGES) { acc = 0; acc_phase ^= 1u; }
        }
    } else {
        // ------------------------------ epilogue: TMEM -> float32 rows --------------------------
        // Two warps per TMEM lane quadrant; the chunks of 32 columns of a tile alternate between
        // them.  The TMEM load of a warp's next chunk is in flight while it stores the current one.
        const int q = warp & 3;                       // TMEM lane quadrant this warp may read
        const int grp = (warp - 2) >> 2;              // which of the quadrant's two warps
        float4* tbuf = reinterpret_cast<float4*>(epi_ptr + (warp - 2) * 4096);
        int acc = 0;
        uint32_t acc_phase = 0;
        bool alive = true;
        for (int w = w_begin; w < w_end; w += w_step) {
            const Item it = decode<MT>(P, w);
            const int M = P.p[it.q].M, N = P.p[it.q].N;
            float* out = P.p[it.q].out + (size_t)it.e * M * N;
            const bool empty = offsets[it.e + 1] == offsets[it.e];   // no MMA ran: gradient 0
            if (alive) {
                const bool ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag, dev_status);
                alive = __all_sync(0xffffffffu, ok);
            }
            tc_fence_after();
            // chunk u = (128-row half, 32 columns): only those that hold outputs of the problem
            const int cols_ok = min(WN / 32, (N - it.n0 + 31) / 32);
            const int halves_ok = min(MT, (M - it.m0 + WM - 1) / WM);
            const int n_u = alive ? halves_ok * cols_ok : 0;
            const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * MT * WN);
            auto load = [&](int u, float(&v)[32]) {
                const int half = u / cols_ok, c = (u - half * cols_ok) * 32;
                tc_ld32(tacc + (uint32_t)(half * WN + c), v);
            };
            auto store = [&](int u, float(&v)[32]) {
                const int half = u / cols_ok, c = (u - half * cols_ok) * 32;
                // the lane's row goes to shared memory in 16-byte pieces, piece j at slot
                // j ^ (row & 7): conflict-free both for these stores and for the row reads below
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    tbuf[lane * 8 + (j ^ (lane & 7))] =
                        make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                __syncwarp();
                float4 val[8];                     // all reads before the first store (the
#pragma unroll                                     // stores might alias them for the compiler)
                for (int rr = 0; rr < 8; ++rr) {
                    const int r = rr * 4 + (lane >> 3), j = lane & 7;
                    val[rr] = tbuf[r * 8 + (j ^ (r & 7))];
                }
#pragma unroll
                for (int rr = 0; rr < 8; ++rr) {
                    const int r = rr * 4 + (lane >> 3), j = lane & 7;
                    const int m = it.m0 + half * WM + q * 32 + r, n = it.n0 + c + 4 * j;
                    if (m < M && n + 4 <= N)
                        *reinterpret_cast<float4*>(out + (size_t)m * N + n) = val[rr];
                }
                __syncwarp();
            };
            float va[32], vb[32];
            if (empty) {
#pragma unroll
                for (int i = 0; i < 32; ++i) va[i] = vb[i] = 0.f;
            }
            int u = grp;
            if (u < n_u && !empty) load(u, va);
#pragma unroll 1
            while (u < n_u) {
                tc_wait_ld();
                if (u + EPI_PER_Q < n_u && !empty) load(u + EPI_PER_Q, vb);
                store(u, va);
                u += EPI_PER_Q;
                if (u >= n_u) break;
                tc_wait_ld();
                if (u + EPI_PER_Q < n_u && !empty) load(u + EPI_PER_Q, va);
                store(u, vb);
                u += EPI_PER_Q;
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0 && alive) mbar_arrive(tempty_bar(acc));
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
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace wg

// bf16 matrix [rows, cols] as an MN-major operand: boxes of 64 columns x 64 rows.
static bool operand_map(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t cols) {
    return tc::make_map_2d(m, ptr, rows, cols, wg::WK);
}

r3_status launch_wgrad_tc(const r3_shape* s, const void* xp, const void* dout, const void* h,
                          const void* da, const void* db, const int32_t* offsets, float* dw_gate,
                          float* dw_up, float* dw_down, int32_t* dev_status, cudaStream_t cs) {
    using namespace wg;
    const uint64_t R = (uint64_t)s->T * s->K;
    if (R == 0) return R3_OK;
    static PerDevice attr_set;
    if (!attr_set.done()) {
        if (cudaFuncSetAttribute(wgrad_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 Shape<1>::SMEM_BYTES) != cudaSuccess ||
            cudaFuncSetAttribute(wgrad_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 Shape<2>::SMEM_BYTES) != cudaSuccess)
            return R3_ERR_CUDA;
        attr_set.mark();
    }
    // the tall tile once an expert holds enough rows for its operand traffic to matter more than
    // an epilogue that the next tile's MMAs do not hide
    const int MT = R / (uint64_t)s->E >= (uint64_t)TALL_TILE_MIN_ROWS ? 2 : 1;
    Params P;
    const void* a_ptr[3] = {dout, da, db};
    const void* b_ptr[3] = {h, xp, xp};
    float* out[3] = {dw_down, dw_gate, dw_up};
    const int Ms[3] = {s->d, s->F, s->F}, Ns[3] = {s->F, s->d, s->d};
    int tiles = 0;
    for (int q = 0; q < 3; ++q) {
        Problem& p = P.p[q];
        if (!operand_map(&p.a, a_ptr[q], R, (uint64_t)Ms[q]) ||
            !operand_map(&p.b, b_ptr[q], R, (uint64_t)Ns[q]))
            return R3_ERR_CUDA;
        p.out = out[q];
        p.M = Ms[q];
        p.N = Ns[q];
        p.mt = (Ms[q] + MT * WM - 1) / (MT * WM);
        p.nt = (Ns[q] + WN - 1) / WN;
        p.tile0 = tiles;
        tiles += p.mt * p.nt;
    }
    P.n_problems = 3;
    P.tiles_per_expert = tiles;
    const int items = s->E * tiles;
    P.total_items = items;
    const int grid = items < sm_count() ? items : sm_count();
    if (MT == 2)
        wgrad_kernel<2><<<grid, THREADS, Shape<2>::SMEM_BYTES, cs>>>(P, offsets, dev_status);
    else
        wgrad_kernel<1><<<grid, THREADS, Shape<1>::SMEM_BYTES, cs>>>(P, offsets, dev_status);
    return launch_status();
}

}  // namespace r3
