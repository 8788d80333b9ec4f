// bf16 grouped SwiGLU expert GEMMs on the Blackwell tensor cores (sm_100a), two CTAs per MMA.
//
//   MODE 0:  h[r, f]  = silu(xp[r] . W_gate,e[f]) * (xp[r] . W_up,e[f])      (K = d, out = F)
//   MODE 1:  o[r, c]  = h[r] . W_down,e[c]                                    (K = F, out = d)
// and the two input-gradient GEMMs of the Update stage, whose weight operand is read TRANSPOSED
// (MN-major shared-memory tiles straight from the forward layout, no transposed copy):
//   MODE 2:  dh[r, f] = sum_c do[r, c] W_down,e[c, f]                         (K = d, out = F)
//   MODE 3:  dxp[r, c] = sum_f da[r, f] W_gate,e[f, c] + db[r, f] W_up,e[f, c] (K = 2F, out = d;
//            k blocks alternate between (W_gate, da) and (W_up, db); da, db = planes 0, 1 of one
//            [2, R, F] array)
//
// Orientation.  The WEIGHT rows are the M side of the MMA and the TOKEN rows are the N side, so
// the accumulator holds out^T: tensor-memory lane = output feature, column = token.  M is fixed
// by the hardware (256 per CTA pair) while N may be any multiple of 16 up to 256, so the token
// rows of a tile are padded to 16, not to a fixed row tile: a short tile copies and stores fewer
// rows and its MMAs are shorter (a 256 x N x 16 MMA measures max(58, N/2) clocks).  The weight
// tile is copied once per token tile whatever its N.
//
// A work item is (expert, token tile of N <= 256 rows, feature tile).  The two CTAs of a cluster
// share it (tcgen05 cta_group::2, UMMA 256 x N x 16): each CTA loads 128 weight rows and N/2
// token rows per 64-wide k block (32 KB per stage instead of the 48 KB a single-CTA 128x256 tile
// needs for the same MMA time), and receives 128 features x N tokens in its own tensor memory.
// In MODE 0 the 128 weight rows of a CTA are 64 gate rows followed by the 64 up rows of the same
// features, so lanes 0-63 hold the gate pre-activations and lanes 64-127 the up projections; the
// epilogue exchanges them through shared memory to form the SwiGLU product.
//
// Items are ordered (expert, feature tile, token tile).  Every cluster takes three items by
// position (cluster c: c, c + C, c + 2C for C clusters) and claims the rest in list order from a
// device counter, so the clusters running at any moment work on neighbouring items (their copies
// of a shared weight or token tile meet in L2 and the weights stream from HBM once) and no
// cluster idles while another still holds a queue.  Claims run three items ahead of the copies:
// the leader CTA's producer thread issues the atomic for item s + 4 when it starts item s, hands
// item s + 3 to the peer CTA's producer through distributed shared memory, and both producers
// publish each item's descriptor to the other warps of their CTA through a tagged ring in shared
// memory, so nobody waits on a claim.  The last cluster to finish re-arms the counter.
//
// Roles (224 threads per CTA): warp 0 lane 0 = TMA producer of the weight boxes and warp 6 lane 0
// = TMA producer of the token box (both CTAs, into a 6-stage ring of 128B-swizzled tiles; two
// issuing threads per stage), warp 1 of the leader CTA = MMA issuer (the warp walks the barriers, one
// elected lane issues; two accumulator stages of 256 columns, so the epilogue of an item overlaps
// the main loop of the next), warps 2..5 = epilogue (tcgen05.ld -> transpose through shared
// memory -> 16-byte global stores).
//
// Every mbarrier wait is bounded by a clock limit; when a wait runs out the CTA raises a shared
// abort flag, reports R3_DEV_TIMEOUT, lets the other roles drain (they keep their barrier
// protocol but skip the work), frees its tensor memory and returns.
#include "r3_common.cuh"
#include "r3_internal.h"
#include "r3_tc.cuh"
#include "r3_worklist.cuh"

namespace r3 {
namespace tc {

constexpr int BMF = 128;           // weight rows (output features) per CTA; UMMA M = 2 * BMF
constexpr int BK = 64;             // k per stage: 64 bf16 = one 128-byte swizzle row
constexpr int UK = 16;             // k per tcgen05.mma (bf16)
constexpr int STAGES = 6;
constexpr int ACC_STAGES = 2;
constexpr int TMEM_COLS = ACC_STAGES * BNT;      // 512 = all of tensor memory
constexpr int A_BYTES = BMF * BK * 2;            // 16 KB of weights per CTA and stage
constexpr int B_BYTES = (BNT / 2) * BK * 2;      // up to 16 KB of tokens per CTA and stage
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int EPI_WARPS = 4;
constexpr int THREADS = (3 + EPI_WARPS) * 32;    // + warp 6: token-tile copies
constexpr int EPI_BYTES = 28 * 1024;             // transpose / exchange buffers of the epilogue
constexpr int BAR_BYTES = 256;
constexpr int RING = 16;                         // item descriptors / claims in flight per CTA
constexpr int SCHED_BYTES = RING * 32 + RING * 8;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_BYTES + BAR_BYTES + SCHED_BYTES + 1024;
constexpr int FEAT0 = BMF;         // h features per item in MODE 0 (64 per CTA, gate + up rows)
constexpr int FEAT1 = 2 * BMF;     // o features per item in MODE 1

// Tensor maps of one launch.  b[i] loads a token box of 8 * (i + 1) rows.
struct alignas(64) PairMaps {
    CUtensorMap a0, a1;
    CUtensorMap b[BNT / 16];
    CUtensorMap g;                 // gather form: the un-permuted activations, box 64 x 1
};

// ---- work list (layout and builder: r3_worklist.cuh) ------------------------------------------
// One CTA per list (blockIdx.x = 0: up projection with nf0 feature tiles, 1: down with nf1).
__global__ void __launch_bounds__(1024)
build_work_kernel(const int32_t* __restrict__ offsets, int E, int nf0, int nf1,
                  int32_t* __restrict__ list0, int32_t* __restrict__ list1, int pairs) {
    __shared__ int32_t s_items[1025];
    grid_launch_dependents();
    grid_dependency_wait();                // the offsets come from the dispatch before
    build_work_list(offsets, E, blockIdx.x == 0 ? nf0 : nf1, blockIdx.x == 0 ? list0 : list1, pairs,
                    s_items);
}

// ---- item hand-over inside a CTA pair ---------------------------------------------------------
// Descriptor ring (shared memory of one CTA): slot = sequence number % RING, 32 bytes = the item
// (n = 0: no more items) and a tag = sequence number + 1 written last.  Written by the CTA's
// producer thread when it starts the item, read by the MMA and epilogue warps.
__device__ __forceinline__ void desc_put(uint8_t* ring, int seq, const int4& d) {
    volatile int32_t* slot = reinterpret_cast<volatile int32_t*>(ring + (seq % RING) * 32);
    slot[0] = d.x;
    slot[1] = d.y;
    slot[2] = d.z;
    slot[3] = d.w;
    __threadfence_block();
    slot[4] = seq + 1;
}
__device__ __forceinline__ bool desc_get(uint8_t* ring, int seq, int4* d, volatile int* abort_flag,
                                         int32_t* dev_status) {
    volatile int32_t* slot = reinterpret_cast<volatile int32_t*>(ring + (seq % RING) * 32);
    if (slot[4] != seq + 1) {
        const long long t0 = clock64();
        while (slot[4] != seq + 1) {
            if (*abort_flag) return false;
            if (clock64() - t0 > WAIT_CLOCKS) {
                *abort_flag = 1;
                report(dev_status, R3_DEV_TIMEOUT);
                return false;
            }
        }
    }
    __threadfence_block();
    *d = make_int4(slot[0], slot[1], slot[2], slot[3]);
    return true;
}
// Claim ring (shared memory of the peer CTA, written by the leader's producer through the
// cluster's distributed shared memory): one 64-bit word per slot = tag (sequence + 1) << 32 | item.
__device__ __forceinline__ void claim_post(uint32_t peer_ring, int seq, int item) {
    const unsigned long long v = ((unsigned long long)(uint32_t)(seq + 1) << 32) | (uint32_t)item;
    asm volatile("st.volatile.shared::cluster.u64 [%0], %1;"
                 ::"r"(peer_ring + (uint32_t)(seq % RING) * 8u), "l"(v) : "memory");
}
__device__ __forceinline__ bool claim_get(uint8_t* ring, int seq, int* item, volatile int* abort_flag,
                                          int32_t* dev_status) {
    volatile unsigned long long* slot =
        reinterpret_cast<volatile unsigned long long*>(ring) + (seq % RING);
    unsigned long long v = *slot;
    if ((uint32_t)(v >> 32) != (uint32_t)(seq + 1)) {
        const long long t0 = clock64();
        for (;;) {
            v = *slot;
            if ((uint32_t)(v >> 32) == (uint32_t)(seq + 1)) break;
            if (*abort_flag) return false;
            if (clock64() - t0 > WAIT_CLOCKS) {
                *abort_flag = 1;
                report(dev_status, R3_DEV_TIMEOUT);
                return false;
            }
        }
    }
    *item = (int)(uint32_t)v;
    return true;
}

// ---- the GEMM kernel --------------------------------------------------------------------------
// GATHER (up projection only): the token operand is read from the un-permuted activations
// x [T, d], row slot_of_row[r] / K for grouped row r, with TMA gather4 copies (each lane of the
// producer warp owns four rows of the CTA's half of the token tile and issues one copy per k
// block), so the permuted copy of x never has to exist.
template <int MODE, bool GATHER>
__global__ void __launch_bounds__(THREADS, 1)
grouped_gemm_pair_kernel(const __grid_constant__ PairMaps maps, int32_t* list,
                         const int32_t* __restrict__ slot_of_row, int K,
                         __nv_bfloat16* __restrict__ out, __nv_bfloat16* __restrict__ pre_gate,
                         __nv_bfloat16* __restrict__ pre_up, int Kdim, int Nout,
                         int32_t* dev_status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    uint8_t* epi_ptr = base_ptr + STAGES * STAGE_BYTES;
    const uint32_t bar0 = base + STAGES * STAGE_BYTES + EPI_BYTES;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
    auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + ACC_STAGES + a); };
    uint8_t* misc = epi_ptr + EPI_BYTES + 128;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(misc);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 4);
    uint8_t* desc_ring = epi_ptr + EPI_BYTES + BAR_BYTES;
    uint8_t* claim_ring = desc_ring + RING * 32;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();          // 0 = leader of the CTA pair
    const int pair = blockIdx.x >> 1;
    const int w_step = gridDim.x >> 1;
    const int4* __restrict__ items = reinterpret_cast<const int4*>(list + kHeaderInts);
    const int4 kNone = make_int4(0, 0, 0, 0);          // n = 0 ends the item stream
    // MODE 3 walks the k blocks of both weight matrices alternately
    const int kblocks = (MODE == 3 ? 2 : 1) * ((Kdim + BK - 1) / BK);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < ACC_STAGES; ++a) {
            mbar_init(tfull_bar(a), 1);
            mbar_init(tempty_bar(a), 2 * EPI_WARPS);       // epilogue warps of both CTAs
        }
        *abort_flag = 0;
        for (int i = 0; i < SCHED_BYTES / 4; ++i) reinterpret_cast<volatile int32_t*>(desc_ring)[i] = 0;
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_slot)), TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();            // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // Nothing above touched global memory: it may have run while the kernel before this one in
    // the stream was draining.  The work list, the operands and the outputs come after the wait.
    grid_launch_dependents();
    grid_dependency_wait();
    const int w_begin = pair, w_end = list[0];

    if (warp == 0 && GATHER) {
        // ------------------------------ TMA producer, gather form (the whole warp) -------------
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        int seq = 0;
        // token (row of x) of rows 4*lane .. 4*lane+3 of this CTA's half of item `it`
        auto load_tokens = [&](const int4& it, int* tok) {
            const int half = it.z >> 1;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int in_half = 4 * lane + i, in_item = (int)rank * half + in_half;
                tok[i] = (in_half < half && in_item < it.w) ? slot_of_row[it.y + in_item] / K : 0;
            }
        };
        // item descriptors run two items ahead of the copies, token numbers one item ahead
        int4 it_cur = w_begin < w_end ? items[w_begin] : kNone;
        int4 it_nxt = w_begin + w_step < w_end ? items[w_begin + w_step] : kNone;
        int cur[4], nxt[4];
        load_tokens(it_cur, nxt);
        for (int w = w_begin; ok && w < w_end; w += w_step) {
#pragma unroll
            for (int i = 0; i < 4; ++i) cur[i] = nxt[i];
            const int4 it = it_cur;
            it_cur = it_nxt;
            it_nxt = w + 2 * w_step < w_end ? items[w + 2 * w_step] : kNone;
            load_tokens(it_cur, nxt);             // lands while this item's copies are issued
            if (lane == 0) desc_put(desc_ring, seq, it);
            ++seq;
            const int e = it.x & 0xffff, f = it.x >> 16, n = it.z, half = n >> 1;
            for (int kb = 0; kb < kblocks; ++kb) {
                int free_ok = 1;
                if (lane == 0)
                    free_ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, dev_status) ? 1 : 0;
                if (!__shfl_sync(0xffffffffu, free_ok, 0)) {
                    ok = false;
                    break;
                }
                const uint32_t sa = base + stage * STAGE_BYTES, sb = sa + A_BYTES;
                const uint32_t lead_full = mapa_shared(full_bar(stage), 0);
                if (lane == 0) {
                    if (rank == 0)                      // bytes of both CTAs: 2 x (A + n/2 rows)
                        mbar_expect_tx(full_bar(stage), (uint32_t)(2 * A_BYTES + n * BK * 2));
                    const int f0 = f * FEAT0 + (int)rank * (BMF / 2);
                    tma_load_3d_pair(sa, &maps.a0, kb * BK, f0, e, lead_full);
                    tma_load_3d_pair(sa + A_BYTES / 2, &maps.a1, kb * BK, f0, e, lead_full);
                }
                if (4 * lane < half)
                    tma_gather4_pair(sb + (uint32_t)lane * 512u, &maps.g, kb * BK, cur[0], cur[1],
                                     cur[2], cur[3], lead_full);
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
        }
        if (lane == 0) {
            desc_put(desc_ring, seq, kNone);
            for (int s = 0; ok && s < STAGES; ++s) {
                ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, dev_status);
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 0) {
        // ------------------------------ TMA producer (each CTA loads its own halves) -----------
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            const int I = w_end, P = w_step;
            int32_t* counter = list + 1;
            const uint32_t peer_claims = mapa_shared(smem_u32(claim_ring), 1);
            int seq = 0;
            int idx_cur = pair;
            int4 it_cur = idx_cur < I ? items[idx_cur] : kNone;
            // leader only: items seq + 1 and seq + 2, the descriptor of seq + 1, and the claim in
            // flight (it becomes item seq + 3 when the next item starts)
            int idx_n1 = pair + P, idx_n2 = pair + 2 * P;
            int4 it_n1 = kNone;
            int pending = I;
            if (rank == 0) {
                if (idx_n1 < I) it_n1 = items[idx_n1];
                if (idx_n2 < I) pending = atomicAdd(counter, 1);
            }
            while (ok && idx_cur < I) {
                const int4 it = it_cur;
                desc_put(desc_ring, seq, it);
                int idx_next;
                if (rank == 0) {
                    const int claimed = pending;                     // item seq + 3
                    claim_post(peer_claims, seq + 3, claimed);
                    pending = claimed < I ? atomicAdd(counter, 1) : I;
                    idx_next = idx_n1;
                    it_cur = it_n1;
                    it_n1 = idx_n2 < I ? items[idx_n2] : kNone;      // lands during this item
                    idx_n1 = idx_n2;
                    idx_n2 = claimed;
                } else {
                    if (seq + 1 < STATIC_ITEMS) {
                        idx_next = pair + (seq + 1) * P;
                    } else if (!claim_get(claim_ring, seq + 1, &idx_next, abort_flag, dev_status)) {
                        ok = false;
                        break;
                    }
                    it_cur = idx_next < I ? items[idx_next] : kNone; // lands during this item
                }
                idx_cur = idx_next;
                ++seq;
                const int e = it.x & 0xffff, f = it.x >> 16, n = it.z;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, dev_status)) {
                        ok = false;
                        break;
                    }
                    const uint32_t sa = base + stage * STAGE_BYTES;
                    const uint32_t lead_full = mapa_shared(full_bar(stage), 0);
                    if (rank == 0)                      // bytes of both CTAs: 2 x (A + n/2 rows)
                        mbar_expect_tx(full_bar(stage), (uint32_t)(2 * A_BYTES + n * BK * 2));
                    if (MODE == 0) {
                        const int f0 = f * FEAT0 + (int)rank * (BMF / 2);
                        tma_load_3d_pair(sa, &maps.a0, kb * BK, f0, e, lead_full);
                        tma_load_3d_pair(sa + A_BYTES / 2, &maps.a1, kb * BK, f0, e, lead_full);
                    } else if (MODE == 1) {
                        tma_load_3d_pair(sa, &maps.a0, kb * BK, f * FEAT1 + (int)rank * BMF, e,
                                         lead_full);
                    } else {
                        // transposed weights: two boxes of 64 output features x 64 k rows
                        const int which = MODE == 3 ? (kb & 1) : 0;
                        const int kk = MODE == 3 ? (kb >> 1) : kb;
                        const CUtensorMap* amap = which ? &maps.a1 : &maps.a0;
                        const int m0 = f * FEAT1 + (int)rank * BMF;
                        tma_load_3d_pair(sa, amap, m0, kk * BK, e, lead_full);
                        tma_load_3d_pair(sa + A_BYTES / 2, amap, m0 + 64, kk * BK, e, lead_full);
                    }
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            desc_put(desc_ring, seq, kNone);
            if (rank == 0) {
                // all of this cluster's claims have returned; the last cluster re-arms the counter
                __threadfence();
                if (atomicAdd(list + 2, 1) == P - 1) {
                    atomicExch(counter, STATIC_ITEMS * P);
                    atomicExch(list + 2, 0);
                }
            }
            // Tail: every stage's release (signalled from the leader's tensor core, also into the
            // peer CTA) must have landed before this CTA may leave.
            for (int s = 0; ok && s < STAGES; ++s) {
                ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, dev_status);
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer (leader CTA only) ---------------------------
        // The whole warp of the leader CTA walks the barriers; one elected lane issues the MMAs
        // and commits (the compiler then sees a warp-uniform loop around a single-thread region).
        if (rank == 0) {
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int seq = 0; ok; ++seq) {
                int4 it;
                if (!desc_get(desc_ring, seq, &it, abort_flag, dev_status)) break;
                const int n = it.z;
                if (n == 0) break;
                const uint32_t idesc = instr_desc_bf16(2 * BMF, n) | (MODE >= 2 ? kInstrDescAMajorMN : 0u);
                if (!__all_sync(0xffffffffu, mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag,
                                                       dev_status)))
                    break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BNT);
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!__all_sync(0xffffffffu, mbar_wait(full_bar(stage), phase, abort_flag,
                                                           dev_status))) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    if (elect_one()) {
                        const uint32_t sa = base + stage * STAGE_BYTES, sb = sa + A_BYTES;
                        const uint64_t da = MODE >= 2 ? smem_desc_mn_sw128(sa, A_BYTES / 2)
                                                      : smem_desc_sw128(sa);
                        const uint64_t db = smem_desc_sw128(sb);
                        // per MMA (16 along k): K-major tiles move 32 bytes inside the swizzled
                        // row, the MN-major tile moves two groups of 8 k rows = 2048 bytes
                        constexpr uint64_t a_step = MODE >= 2 ? (2048 >> 4) : 2;
#pragma unroll
                        for (int kk = 0; kk < BK / UK; ++kk) {
                            tc_mma_bf16_pair(d_tmem, da + a_step * kk, db + (uint64_t)(kk * 2), idesc,
                                             (kb | kk) != 0 ? 1u : 0u);
                        }
                        tc_commit_pair(empty_bar(stage), 3);   // frees the stage in both CTAs
                    }
                    __syncwarp();
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                if (elect_one()) tc_commit_pair(tfull_bar(acc), 3);   // accumulator complete, both CTAs
                __syncwarp();
                if (++acc == ACC_STAGES) { acc = 0; acc_phase ^= 1u; }
            }
        }
    } else if (warp == 6) {
        // ------------------------------ token-tile copies (each CTA its own half) --------------
        // A second issuing thread: the weight boxes and the token box of a stage are asked for
        // by two threads at once.  It follows the items through the descriptor ring and walks
        // the same stages as warp 0; its bytes may land before warp 0 has told the barrier how
        // many to expect (the pending arrival keeps the phase open).  The gather form copies the
        // token rows in warp 0.
        if (lane == 0 && !GATHER) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int seq = 0; ok; ++seq) {
                int4 it;
                if (!desc_get(desc_ring, seq, &it, abort_flag, dev_status)) break;
                const int n = it.z, half = n >> 1;
                if (n == 0) break;
                const CUtensorMap* bmap = &maps.b[(half >> 3) - 1];
                const int brow = it.y + (int)rank * half;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, dev_status)) {
                        ok = false;
                        break;
                    }
                    const uint32_t sb = base + stage * STAGE_BYTES + A_BYTES;
                    const uint32_t lead_full = mapa_shared(full_bar(stage), 0);
                    if (MODE == 3)
                        tma_load_3d_pair(sb, bmap, (kb >> 1) * BK, brow, kb & 1, lead_full);
                    else
                        tma_load_2d_pair(sb, bmap, kb * BK, brow, lead_full);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else {
        // ------------------------------ epilogue -----------------------------------------------
        const int q = warp & 3;                       // TMEM lane quadrant this warp may read
        int acc = 0;
        uint32_t acc_phase = 0;
        int chunk_no = 0;
        bool alive = true;                            // false after a wait ran out: the barrier
                                                      // protocol goes on, the work is skipped
        for (int seq = 0;; ++seq) {
            int4 it;
            if (!desc_get(desc_ring, seq, &it, abort_flag, dev_status)) break;
            if (it.z == 0) break;
            const int f = it.x >> 16, row0 = it.y, n = it.z, valid = it.w;
            if (alive) {
                const bool ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag, dev_status);
                alive = __all_sync(0xffffffffu, ok);
            }
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BNT);
            if (MODE == 0) {
                // Quadrants 0,1 hold the gate rows of features p*32 + lane, quadrants 2,3 the up
                // rows of the same features.  Per chunk of 32 tokens the two warps swap halves
                // through shared memory (two buffers, one named barrier per chunk): the gate warp
                // finishes tokens 0-15, the up warp tokens 16-31.
                const int p = q & 1;
                const bool gate = q < 2;
                float* xpair = reinterpret_cast<float*>(epi_ptr + p * 8192);      // 2 x [2][16][32]
                __nv_bfloat16* hb = reinterpret_cast<__nv_bfloat16*>(epi_ptr + 16384 + q * 1024);
                // training: the pre-activations are kept for the backward pass
                __nv_bfloat16* gb = reinterpret_cast<__nv_bfloat16*>(epi_ptr + 20480 + q * 2048);
                __nv_bfloat16* ub = gb + 512;
                const bool keep = pre_gate != nullptr;
                const int feat = f * FEAT0 + (int)rank * (BMF / 2) + p * 32 + (lane & 3) * 8;
                const int own = gate ? 0 : 16;        // first of the 16 tokens this warp finishes
#pragma unroll 1
                for (int c = 0; c < n; c += 32, ++chunk_no) {
                    float v[32];
                    if (alive) {
                        tc_ld32(taddr + c, v);
                        tc_wait_ld();
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = 0.f;
                    }
                    float* xb = xpair + (chunk_no & 1) * 1024;
                    float* send = xb + (gate ? 0 : 512);
                    const float* recv = xb + (gate ? 512 : 0);
#pragma unroll
                    for (int i = 0; i < 16; ++i) send[i * 32 + lane] = gate ? v[16 + i] : v[i];
                    named_bar_sync(1 + p, 64);
                    // all loads first, then the arithmetic, then the stores: written as one loop
                    // the stores to hb may alias the loads from recv as far as the compiler knows,
                    // and the 16 load - exp - divide - store chains run one after the other
                    // (measured: 2000 of the 2700 clocks of a chunk)
                    float other[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) other[i] = recv[i * 32 + lane];
                    float hv[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const float g = gate ? v[i] : other[i];
                        const float u = gate ? other[i] : v[16 + i];
                        hv[i] = __fdividef(g, 1.f + __expf(-g)) * u;
                    }
#pragma unroll
                    for (int i = 0; i < 16; ++i) hb[i * 32 + lane] = __float2bfloat16_rn(hv[i]);
                    if (keep) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            gb[i * 32 + lane] = __float2bfloat16_rn(gate ? v[i] : other[i]);
                            ub[i * 32 + lane] = __float2bfloat16_rn(gate ? other[i] : v[16 + i]);
                        }
                    }
                    __syncwarp();
                    uint4 hq[2], gq[2], uq[2];         // all reads before the first store
#pragma unroll
                    for (int rr = 0; rr < 2; ++rr) {
                        const int in_tile = ((lane >> 2) + 8 * rr) * 32 + (lane & 3) * 8;
                        hq[rr] = *reinterpret_cast<const uint4*>(hb + in_tile);
                        if (keep) {
                            gq[rr] = *reinterpret_cast<const uint4*>(gb + in_tile);
                            uq[rr] = *reinterpret_cast<const uint4*>(ub + in_tile);
                        }
                    }
#pragma unroll
                    for (int rr = 0; rr < 2; ++rr) {
                        const int tl = (lane >> 2) + 8 * rr;
                        const int tok = c + own + tl;
                        if (alive && tok < valid && feat + 8 <= Nout) {
                            const size_t at = (size_t)(row0 + tok) * Nout + feat;
                            *reinterpret_cast<uint4*>(out + at) = hq[rr];
                            if (keep) {
                                *reinterpret_cast<uint4*>(pre_gate + at) = gq[rr];
                                *reinterpret_cast<uint4*>(pre_up + at) = uq[rr];
                            }
                        }
                    }
                    __syncwarp();
                }
            } else {
                __nv_bfloat16* tbuf = reinterpret_cast<__nv_bfloat16*>(epi_ptr + q * 2048);
                const int feat0 = f * FEAT1 + (int)rank * BMF + q * 32;
#pragma unroll 1
                for (int c = 0; c < n; c += 32) {
                    if (alive) {
                        float v[32];
                        tc_ld32(taddr + c, v);
                        tc_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) tbuf[i * 32 + lane] = __float2bfloat16_rn(v[i]);
                        __syncwarp();
                        uint4 val[4];                  // all reads before the first store
#pragma unroll
                        for (int rr = 0; rr < 4; ++rr)
                            val[rr] = *reinterpret_cast<const uint4*>(
                                tbuf + ((lane >> 2) + 8 * rr) * 32 + (lane & 3) * 8);
#pragma unroll
                        for (int rr = 0; rr < 4; ++rr) {
                            const int tok = (lane >> 2) + 8 * rr;
                            const int feat = feat0 + (lane & 3) * 8;
                            if (c + tok < valid && feat + 8 <= Nout)
                                *reinterpret_cast<uint4*>(out + (size_t)(row0 + c + tok) * Nout +
                                                          feat) = val[rr];
                        }
                        __syncwarp();
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0 && alive) mbar_arrive_cluster(mapa_shared(tempty_bar(acc), 0));
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
    cluster_sync_all();            // neither CTA leaves while the other may still signal it
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

// ---- host side --------------------------------------------------------------------------------
// Tensor maps of the token operand are encoded once per (pointer, shape) and re-used.
struct TokenMapCache {
    const void* ptr = nullptr;
    uint64_t rows = 0, cols = 0;
    CUtensorMap b[BNT / 16];
};

static bool token_maps(TokenMapCache* c, const void* ptr, uint64_t rows, uint64_t cols,
                       PairMaps* out) {
    if (c->ptr != ptr || c->rows != rows || c->cols != cols) {
        for (int i = 0; i < BNT / 16; ++i)
            if (!make_map_2d(&c->b[i], ptr, rows, cols, 8u * (i + 1))) return false;
        c->ptr = ptr;
        c->rows = rows;
        c->cols = cols;
    }
    for (int i = 0; i < BNT / 16; ++i) out->b[i] = c->b[i];
    return true;
}

// Number of CTA pairs that can be resident at once (one CTA per SM), cached per device.
template <typename Kern>
static int resident_pairs(Kern kern) {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (cached[dev] == 0) {
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.gridDim = dim3(2 * (sm_count() / 2));
        cfg.blockDim = dim3(THREADS);
        cfg.dynamicSmemBytes = SMEM_BYTES;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n <= 0) return 0;
        const int by_sm = sm_count() / 2;
        n = n < by_sm ? n : by_sm;
        cached[dev] = n;
    }
    return cached[dev];
}

template <int MODE, bool GATHER>
static r3_status launch_pair(const PairMaps& maps, int pairs, int32_t* list,
                             const int32_t* slot_of_row, int K, void* out, int Kdim, int Nout,
                             int32_t* dev_status, cudaStream_t cs, void* pre_gate = nullptr,
                             void* pre_up = nullptr) {
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = dim3(2 * pairs);
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = cs;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, grouped_gemm_pair_kernel<MODE, GATHER>, maps, list, slot_of_row, K,
                              static_cast<__nv_bfloat16*>(out), static_cast<__nv_bfloat16*>(pre_gate),
                              static_cast<__nv_bfloat16*>(pre_up), Kdim, Nout,
                              dev_status) == cudaSuccess ? R3_OK : R3_ERR_CUDA;
}

// Backward of h = silu(a) * b:  da = dh * b * silu'(a),  db = dh * silu(a), written as planes 0
// and 1 of dab [2, R, F].  16-byte vectors; F is a multiple of 8.  With `h` non-null the forward's
// h = silu(a) * b is formed again (the weight gradient of the down projection needs it).
__global__ void __launch_bounds__(256)
swiglu_bwd_kernel(const uint4* __restrict__ dh, const uint4* __restrict__ a,
                  const uint4* __restrict__ b, uint4* __restrict__ dab, uint4* __restrict__ h,
                  long long n_vec) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_vec) return;
    const uint4 vd = dh[i], va = a[i], vb = b[i];
    uint4 oa, ob, oh;
    __nv_bfloat162* qh = reinterpret_cast<__nv_bfloat162*>(&oh);
    const __nv_bfloat162* pd = reinterpret_cast<const __nv_bfloat162*>(&vd);
    const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&va);
    const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&vb);
    __nv_bfloat162* qa = reinterpret_cast<__nv_bfloat162*>(&oa);
    __nv_bfloat162* qb = reinterpret_cast<__nv_bfloat162*>(&ob);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float2 fd = __bfloat1622float2(pd[k]), fa = __bfloat1622float2(pa[k]),
                     fb = __bfloat1622float2(pb[k]);
        const float s0 = 1.f / (1.f + __expf(-fa.x)), s1 = 1.f / (1.f + __expf(-fa.y));
        qa[k] = __floats2bfloat162_rn(fd.x * fb.x * s0 * (1.f + fa.x * (1.f - s0)),
                                      fd.y * fb.y * s1 * (1.f + fa.y * (1.f - s1)));
        qb[k] = __floats2bfloat162_rn(fd.x * fa.x * s0, fd.y * fa.y * s1);
        qh[k] = __floats2bfloat162_rn(fa.x * s0 * fb.x, fa.y * s1 * fb.y);
    }
    dab[i] = oa;
    dab[n_vec + i] = ob;
    if (h) h[i] = oh;
}

}  // namespace tc

static long long max_items(long long R, int E, int nf) {
    return (R / tc::BNT + E) * (long long)nf;       // each expert adds at most one partial tile
}
static int feat_tiles_up(const r3_shape* s) { return (s->F + tc::FEAT0 - 1) / tc::FEAT0; }
static int feat_tiles_down(const r3_shape* s) { return (s->d + tc::FEAT1 - 1) / tc::FEAT1; }
static size_t list_bytes(long long R, int E, int nf) {
    return round_up(sizeof(int32_t) * tc::kHeaderInts + 16 * (size_t)max_items(R, E, nf), 256);
}

size_t tc_work_bytes(const r3_shape* s) {
    const long long R = (long long)s->T * s->K;
    return list_bytes(R, s->E, feat_tiles_up(s)) + list_bytes(R, s->E, feat_tiles_down(s));
}

static bool forward_attrs() {
    using namespace tc;
    static PerDevice attr_set;
    if (!attr_set.done()) {
        if (cudaFuncSetAttribute(grouped_gemm_pair_kernel<0, false>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess ||
            cudaFuncSetAttribute(grouped_gemm_pair_kernel<0, true>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess ||
            cudaFuncSetAttribute(grouped_gemm_pair_kernel<1, false>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess)
            return false;
        attr_set.mark();
    }
    return true;
}

bool tc_work_lists(const r3_shape* s, void* work, WorkListSpec* spec) {
    using namespace tc;
    if (!forward_attrs()) return false;
    const int pairs = resident_pairs(grouped_gemm_pair_kernel<0, false>);
    if (pairs <= 0) return false;
    const long long R = (long long)s->T * s->K;
    spec->nf0 = feat_tiles_up(s);
    spec->nf1 = feat_tiles_down(s);
    spec->pairs = pairs;
    spec->list0 = static_cast<int32_t*>(work);
    spec->list1 = reinterpret_cast<int32_t*>(static_cast<char*>(work) + list_bytes(R, s->E, spec->nf0));
    return true;
}

r3_status launch_grouped_swiglu_tc(const r3_shape* s, const void* xp, const void* x,
                                   const int32_t* slot_of_row, const int32_t* offsets,
                                   const void* w_gate, const void* w_up, const void* w_down,
                                   void* h, void* o, void* work, int32_t* dev_status, int phases,
                                   cudaStream_t cs, void* pre_gate, void* pre_up) {
    using namespace tc;
    const long long R = (long long)s->T * s->K;
    if (R == 0) return R3_OK;
    if (!forward_attrs()) return R3_ERR_CUDA;
    const int pairs = resident_pairs(grouped_gemm_pair_kernel<0, false>);
    if (pairs <= 0) return R3_ERR_CUDA;
    const int nf0 = feat_tiles_up(s), nf1 = feat_tiles_down(s);
    int32_t* list0 = static_cast<int32_t*>(work);
    int32_t* list1 = reinterpret_cast<int32_t*>(static_cast<char*>(work) +
                                                list_bytes(R, s->E, nf0));
    static TokenMapCache cache_xp, cache_h;
    if (phases & kPhaseUp) {
        if (!(phases & kPhaseKeepLists))
            launch_dependent(build_work_kernel, dim3(2), dim3(1024), 0, cs, offsets, (int)s->E, nf0,
                             nf1, list0, list1, pairs);
        PairMaps m;
        if (!make_map_3d(&m.a0, w_gate, s->E, s->F, s->d, BMF / 2) ||
            !make_map_3d(&m.a1, w_up, s->E, s->F, s->d, BMF / 2))
            return R3_ERR_CUDA;
        r3_status st;
        if (xp) {
            if (!token_maps(&cache_xp, xp, (uint64_t)R, (uint64_t)s->d, &m)) return R3_ERR_CUDA;
            m.g = m.b[0];
            st = launch_pair<0, false>(m, pairs, list0, nullptr, 0, h, s->d, s->F, dev_status, cs,
                                       pre_gate, pre_up);
        } else {
            if (!make_map_2d(&m.g, x, (uint64_t)s->T, (uint64_t)s->d, 1)) return R3_ERR_CUDA;
            for (int i = 0; i < BNT / 16; ++i) m.b[i] = m.g;
            st = launch_pair<0, true>(m, pairs, list0, slot_of_row, s->K, h, s->d, s->F,
                                      dev_status, cs, pre_gate, pre_up);
        }
        if (st != R3_OK) return st;
    }
    if (phases & kPhaseDown) {
        PairMaps m;
        if (!make_map_3d(&m.a0, w_down, s->E, s->d, s->F, BMF) ||
            !token_maps(&cache_h, h, (uint64_t)R, (uint64_t)s->F, &m))
            return R3_ERR_CUDA;
        m.a1 = m.a0;
        m.g = m.b[0];
        const r3_status st = launch_pair<1, false>(m, pairs, list1, nullptr, 0, o, s->F, s->d,
                                                   dev_status, cs);
        if (st != R3_OK) return st;
    }
    return launch_status();
}

// ---- input gradient of the expert networks (Update stage) ------------------------------------
size_t tc_bwd_work_bytes(const r3_shape* s) {
    const long long R = (long long)s->T * s->K;
    const int nf_h = (s->F + tc::FEAT1 - 1) / tc::FEAT1;
    return 2 * round_up((size_t)R * s->F * 2, 256) + round_up(2 * (size_t)R * s->F * 2, 256) +
           list_bytes(R, s->E, nf_h) + list_bytes(R, s->E, feat_tiles_down(s));
}

r3_status launch_grouped_swiglu_bwd_tc(const r3_shape* s, const void* dout, const void* pre_gate,
                                       const void* pre_up, const int32_t* offsets,
                                       const void* w_gate, const void* w_up, const void* w_down,
                                       void* dxp, void* work, int32_t* dev_status,
                                       cudaStream_t cs, const void* xp, float* dw_gate,
                                       float* dw_up, float* dw_down) {
    using namespace tc;
    const long long R = (long long)s->T * s->K;
    if (R == 0) return R3_OK;
    static PerDevice attr_set;
    if (!attr_set.done()) {
        if (cudaFuncSetAttribute(grouped_gemm_pair_kernel<2, false>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess ||
            cudaFuncSetAttribute(grouped_gemm_pair_kernel<3, false>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess)
            return R3_ERR_CUDA;
        attr_set.mark();
    }
    const int pairs = resident_pairs(grouped_gemm_pair_kernel<2, false>);
    if (pairs <= 0) return R3_ERR_CUDA;
    const int nf_h = (s->F + FEAT1 - 1) / FEAT1, nf_x = feat_tiles_down(s);
    char* w = static_cast<char*>(work);
    void* dh = w;
    w += round_up((size_t)R * s->F * 2, 256);
    void* dab = w;
    w += round_up(2 * (size_t)R * s->F * 2, 256);
    void* h = w;
    w += round_up((size_t)R * s->F * 2, 256);
    const bool weights = dw_gate != nullptr;
    int32_t* list_h = reinterpret_cast<int32_t*>(w);
    int32_t* list_x = reinterpret_cast<int32_t*>(w + list_bytes(R, s->E, nf_h));
    build_work_kernel<<<2, 1024, 0, cs>>>(offsets, s->E, nf_h, nf_x, list_h, list_x, pairs);

    // dh = dout W_down   (weights transposed: contraction over d)
    static TokenMapCache cache_do;
    PairMaps m;
    if (!make_map_3d(&m.a0, w_down, s->E, s->d, s->F, BK) ||
        !token_maps(&cache_do, dout, (uint64_t)R, (uint64_t)s->d, &m))
        return R3_ERR_CUDA;
    m.a1 = m.a0;
    m.g = m.b[0];
    r3_status st = launch_pair<2, false>(m, pairs, list_h, nullptr, 0, dh, s->d, s->F, dev_status, cs);
    if (st != R3_OK) return st;

    // through the SwiGLU
    const long long n_vec = R * s->F / 8;
    swiglu_bwd_kernel<<<(unsigned)((n_vec + 255) / 256), 256, 0, cs>>>(
        static_cast<const uint4*>(dh), static_cast<const uint4*>(pre_gate),
        static_cast<const uint4*>(pre_up), static_cast<uint4*>(dab),
        weights ? static_cast<uint4*>(h) : nullptr, n_vec);

    // dxp = da W_gate + db W_up   (weights transposed: contraction over F, both matrices)
    PairMaps m2;
    if (!make_map_3d(&m2.a0, w_gate, s->E, s->F, s->d, BK) ||
        !make_map_3d(&m2.a1, w_up, s->E, s->F, s->d, BK))
        return R3_ERR_CUDA;
    for (int i = 0; i < BNT / 16; ++i)
        if (!make_map_3d(&m2.b[i], dab, 2, (uint64_t)R, (uint64_t)s->F, 8u * (i + 1)))
            return R3_ERR_CUDA;
    m2.g = m2.b[0];
    st = launch_pair<3, false>(m2, pairs, list_x, nullptr, 0, dxp, s->F, s->d, dev_status, cs);
    if (st != R3_OK) return st;
    if (weights) {
        const char* db = static_cast<const char*>(dab) + (size_t)R * s->F * 2;
        return launch_wgrad_tc(s, xp, dout, h, dab, db, offsets, dw_gate, dw_up, dw_down,
                               dev_status, cs);
    }
    return launch_status();
}

}  // namespace r3
