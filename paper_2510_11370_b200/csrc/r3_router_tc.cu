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
// Orientation.  The EXPERT rows of W_r are the M side of the MMA (128 per M tile, up to two M
// tiles) and the TOKENS are the N side (a tile of up to 256 tokens, any multiple of 16), so the
// accumulator holds s^T: tensor-memory lane = expert, column = token.  A whole decode batch of a
// layer (256 tokens) is then ONE tile whose router weights are fetched once.
//
// K split.  The kernel is bound by bytes (4 KB of x per token for 0.5 MFLOP), so the bytes of a
// tile are spread over several SMs whenever the tiles are fewer than the SMs: the CTAs of a
// cluster share a tile, each contracting its own range of the k blocks into its own accumulator,
// and each finishes its share of the tile's tokens.  The partial logits travel between the CTAs
// in one of two ways:
//   two CTAs   every CTA moves its whole accumulator into its own shared memory [token][experts+1]
//              and PUSHES the rows of the other CTA's tokens to it with one bulk asynchronous copy
//              (shared memory to the peer's shared memory, completion on the peer's barrier); no
//              cluster barrier is needed after the start;
//   3..8 CTAs  (one layer's decode batch) every CTA stores each token's values straight into the
//              shared memory of the CTA that finishes the token (st.shared::cluster, 32 consecutive
//              words per instruction) into the slot of its own rank, between two cluster barriers.
// Measured on one layer's decode batch split 8 ways: reading the partials with ld.shared::cluster
// cost about 1.6 us per dependent round trip (13 us of 21), the remote stores cost 6 us.  The
// partial sums are added in rank order (a fixed order: reproducible).
//
// One CTA of 12 warps per (tile, k range): warp 0 lane 0 = TMA producer, warp 1 lane 0 = MMA
// issuer; then all 12 warps move the finished accumulator out of TMEM (transposed on the way:
// tensor-memory lane = expert, but a token's experts must lie next to each other), and TopKMask
// is taken by two or four lanes per token on packed candidates in registers (group_topk below), with a
// warp-wide exact selection for the few tokens that the packed form cannot decide.
//
// The kernel is launched with programmatic stream serialisation: everything up to its first
// access to global memory (barrier set-up, tensor-memory allocation) may run while the previous
// kernel of the stream drains, and it lets its own successor do the same once its copies are done.
#include <type_traits>

#include "r3_common.cuh"
#include "r3_internal.h"
#include "r3_tc.cuh"

namespace r3 {
namespace rt {

using namespace tc;

constexpr int BME = 128;                 // expert rows per M tile (UMMA M)
constexpr int BK = 64;
constexpr int UK = 16;
constexpr int A_BYTES = BME * BK * 2;    // one M tile of one weight plane per stage
constexpr int THREADS = 12 * 32;         // producer, MMA issuer, 4 TMEM readers; all 12 pick top-K
constexpr int BAR_BYTES = 256;
constexpr int MAX_STAGES = 7;
constexpr int KMAX = 16;                 // longest record the warp top-K supports (one lane per slot)
constexpr int SMEM_LIMIT = 227 * 1024;
constexpr int MAX_SPLIT = 8;             // portable cluster size

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

// Order-preserving integer key of a logit: a < b as floats  <=>  key(a) < key(b) as unsigned.
// -0.0 and +0.0 are one value (a tie); 0 is reserved for "no candidate".
__device__ __forceinline__ uint32_t logit_key(float v) {
    const uint32_t u = __float_as_uint(v + 0.0f);        // -0.0 + 0.0 = +0.0
    // negative: all bits flipped; positive: sign bit set
    const uint32_t k = u ^ ((uint32_t)((int32_t)u >> 31) | 0x80000000u);
    return k ? k : 1u;
}

// Where the partial logits of the tokens a CTA finishes lie in its shared memory: the value of
// (row, expert) is the sum over the ranks r = 0 .. n - 1, in that order, of the words at
// p0 (rank 0), p1 (rank 1), p1 + stride (rank 2), ..., each at offset row * LD + e.
struct Partials {
    const float* p0;
    const float* p1;
    int stride, n;
    // CNT values at offsets off + i * STEP: all loads of a rank are issued together (a loop over
    // the ranks inside a loop over the values made every load wait for the one before it)
    template <int CNT, int STEP>
    __device__ __forceinline__ void sum(int off, float* v) const {
#pragma unroll
        for (int i = 0; i < CNT; ++i) v[i] = p0[off + i * STEP];
        if (n > 1) {
#pragma unroll
            for (int i = 0; i < CNT; ++i) v[i] += p1[off + i * STEP];
            for (int r = 2; r < n; ++r) {
                const float* q = p1 + (r - 1) * stride;
#pragma unroll
                for (int i = 0; i < CNT; ++i) v[i] += q[off + i * STEP];
            }
        }
    }
};

// Exact TopKMask of one token by the whole warp: lane l holds the keys of experts l + 32 s; K
// rounds of two warp reductions pick the largest key and, among equal keys, the lowest expert.
// About 30 instructions per round and token: used only for the few tokens the packed selection
// below cannot decide.
template <typename IdxT, int SLOTS>
__device__ __forceinline__ void warp_topk_exact(const Partials& ps, int LD, int row, int lane, int E,
                                                int K, IdxT* out) {
    uint32_t key[SLOTS];
    float v[SLOTS];
    ps.sum<SLOTS, 32>(row * LD + lane, v);               // 32 * SLOTS < LD: inside the row
#pragma unroll
    for (int sl = 0; sl < SLOTS; ++sl) key[sl] = lane + 32 * sl < E ? logit_key(v[sl]) : 0u;
    int mine = 0;
    for (int j = 0; j < K; ++j) {
        uint32_t best = 0u;
#pragma unroll
        for (int sl = 0; sl < SLOTS; ++sl) best = max(best, key[sl]);
        const uint32_t top = __reduce_max_sync(0xffffffffu, best);
        uint32_t cand = 0xffffffffu;                     // lowest expert of this lane with that key
#pragma unroll
        for (int sl = SLOTS - 1; sl >= 0; --sl)
            if (key[sl] == top) cand = (uint32_t)(lane + 32 * sl);
        const uint32_t win = __reduce_min_sync(0xffffffffu, cand);
#pragma unroll
        for (int sl = 0; sl < SLOTS; ++sl)
            if (win == (uint32_t)(lane + 32 * sl)) key[sl] = 0u;
        if (lane == j) mine = (int)win;
    }
    if (lane < K) out[lane] = (IdxT)mine;
}

// A packed candidate is the logit itself (a float, after -0.0 -> +0.0) with its low 8 mantissa
// bits replaced by a tag of the expert e (E <= 256): 255 - e for a positive logit, e for a
// negative one.  Compared as FLOATS, a larger candidate has the larger logit truncated to 24 bits
// (sign, exponent, 15 mantissa bits) and, among equal truncated logits, the LOWER expert (for a
// negative number a smaller tag means a smaller magnitude, i.e. a larger value).  A
// compare-exchange is one fminf and one fmaxf.  -inf = no candidate.
__device__ __forceinline__ float pack_candidate(float v, int e) {
    const uint32_t u = __float_as_uint(v + 0.0f);                       // -0.0 + 0.0 = +0.0
    const uint32_t tag = (uint32_t)(255 - e) ^ ((uint32_t)((int32_t)u >> 31) & 255u);
    return __uint_as_float((u & 0xffffff00u) | tag);
}
__device__ __forceinline__ int candidate_expert(float c) {
    const uint32_t u = __float_as_uint(c);
    return (int)(((u & 255u) ^ ((uint32_t)((int32_t)u >> 31) & 255u)) ^ 255u);
}
__device__ __forceinline__ void ce_desc(float& a, float& b) {           // a keeps the larger
    const float hi = fmaxf(a, b), lo = fminf(a, b);
    a = hi;
    b = lo;
}
constexpr float kNoCandidate = -__builtin_huge_valf();

// Sorts KM candidates in descending order: the 19-comparator network for 8, a bitonic network
// for 16.
template <int KM>
__device__ __forceinline__ void sort_desc(float* c) {
    if (KM == 8) {
        ce_desc(c[0], c[2]); ce_desc(c[1], c[3]); ce_desc(c[4], c[6]); ce_desc(c[5], c[7]);
        ce_desc(c[0], c[4]); ce_desc(c[1], c[5]); ce_desc(c[2], c[6]); ce_desc(c[3], c[7]);
        ce_desc(c[0], c[1]); ce_desc(c[2], c[3]); ce_desc(c[4], c[5]); ce_desc(c[6], c[7]);
        ce_desc(c[2], c[4]); ce_desc(c[3], c[5]);
        ce_desc(c[1], c[4]); ce_desc(c[3], c[6]);
        ce_desc(c[1], c[2]); ce_desc(c[3], c[4]); ce_desc(c[5], c[6]);
    } else {
#pragma unroll
        for (int k = 2; k <= KM; k <<= 1) {
#pragma unroll
            for (int j = k >> 1; j > 0; j >>= 1) {
#pragma unroll
                for (int i = 0; i < KM; ++i) {
                    const int l = i ^ j;
                    if (l > i) {
                        if ((i & k) == 0) ce_desc(c[i], c[l]); else ce_desc(c[l], c[i]);
                    }
                }
            }
        }
    }
}

// A sorted list of the KM largest candidates seen so far, plus the largest one dropped
// (`runner` = the (KM+1)-th largest).
template <int KM>
struct TopList {
    float top[KM];
    float runner;
    __device__ __forceinline__ void clear() {
#pragma unroll
        for (int i = 0; i < KM; ++i) top[i] = kNoCandidate;
        runner = kNoCandidate;
    }
    // Merges a list sorted in descending order (and its runner) into this one: max(a_i, b_{KM-1-i})
    // are the KM largest of both (a bitonic sequence), a bitonic merge sorts them again.
    __device__ __forceinline__ void merge(const float* b, float b_runner) {
        float dropped[KM];
#pragma unroll
        for (int i = 0; i < KM; ++i) {
            const float x = top[i], y = b[KM - 1 - i];
            top[i] = fmaxf(x, y);
            dropped[i] = fminf(x, y);
        }
#pragma unroll
        for (int w = KM >> 1; w > 0; w >>= 1)                // a tree, not a chain
#pragma unroll
            for (int i = 0; i < w; ++i) dropped[i] = fmaxf(dropped[i], dropped[i + w]);
        runner = fmaxf(fmaxf(runner, b_runner), dropped[0]);
#pragma unroll
        for (int j = KM >> 1; j > 0; j >>= 1) {
#pragma unroll
            for (int i = 0; i < KM; ++i) {
                const int l = i ^ j;
                if (l > i) ce_desc(top[i], top[l]);
            }
        }
    }
};

// TopKMask of the tokens of one warp task: GROUP (2 or 4) lanes share a token (lane = GROUP *
// token + part); each takes every GROUP-th block of KM experts, sorts the block with a sorting network
// and merges it into its list; the GROUP lists of a token are then merged through shuffles.  The
// result is exact unless two candidates next to each other in the final order (down to the first
// one left out) share their 24 leading bits while the full logits might differ; such a token is
// flagged and repeated with warp_topk_exact (random logits: a few tokens in a thousand; planted
// exact ties: every such token, still correct).  Returns the flags of the warp's tokens (bit =
// lane of the token's first lane).
// Measured for the 128 tokens that a CTA of the 48-layer decode batch finishes: K rounds of two
// warp reductions per token 9.6 us; one reduction per round on packed candidates 6.3 us (a warp
// reduction costs this SM about ten cycles whoever issues it); this form 4.2 us with four lanes
// per token (16 warp tasks for 12 warps) and 3.3 us with two (8 tasks): about 1400 fminf / fmaxf
// per token, which issue at half rate.  With few tokens per CTA four lanes are faster.
template <typename IdxT, int KM, int GROUP>
__device__ __forceinline__ uint32_t group_topk(const Partials& ps, int LD, int row, bool valid,
                                               int part, int E, int K, IdxT* out) {
    TopList<KM> list;
    list.clear();
    if (valid) {
        for (int e0 = part * KM; e0 < E; e0 += GROUP * KM) {
            float c[KM];
            ps.sum<KM, 1>(row * LD + e0, c);
#pragma unroll
            for (int i = 0; i < KM; ++i) c[i] = pack_candidate(c[i], e0 + i);
            sort_desc<KM>(c);
            list.merge(c, kNoCandidate);
        }
    }
    // the lists of the GROUP lanes of a token, merged pairwise (every lane ends with the result)
#pragma unroll
    for (int m = 1; m < GROUP; m <<= 1) {
        float other[KM];
#pragma unroll
        for (int i = 0; i < KM; ++i) other[i] = __shfl_xor_sync(0xffffffffu, list.top[i], m);
        const float other_runner = __shfl_xor_sync(0xffffffffu, list.runner, m);
        list.merge(other, other_runner);
    }
    bool sure = true;
    if (valid && part == 0) {
#pragma unroll
        for (int j = 0; j < KM; ++j) {
            const float next = j + 1 < KM ? list.top[j + 1 < KM ? j + 1 : j] : list.runner;
            if (j < K) {
                if ((__float_as_uint(list.top[j]) >> 8) == (__float_as_uint(next) >> 8)) sure = false;
                out[j] = (IdxT)candidate_expert(list.top[j]);
            }
        }
    }
    return __ballot_sync(0xffffffffu, !sure);
}

// grid = (token tiles of a layer * ksplit, L), cluster = (ksplit, 1, 1).  N = tokens per tile
// (multiple of 16), MT = M tiles of 128 experts (1 or 2).  Shared memory: [ring_bytes: the copy
// ring, later the logits of the accumulator / the slots of the partial logits and, from recv_off
// on, the rows pushed by the other CTA of a pair][barriers].
template <typename IdxT>
__global__ void __launch_bounds__(THREADS, 1)
router_tc_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW,
                 IdxT* __restrict__ idx_out, float* __restrict__ logits_out, int T, int d, int E,
                 int K, int planes, int stages, uint32_t tmem_cols, int ksplit, int N, int MT,
                 int ring_bytes, int recv_off) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const int a_bytes = planes * MT * A_BYTES;
    const int stage_bytes = a_bytes + N * BK * 2;
    const int LD = MT * BME + 1;                         // odd: rows start in different banks
    const uint32_t recv0 = base + (uint32_t)recv_off;
    const uint32_t bar0 = base + (uint32_t)ring_bytes;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (MAX_STAGES + s); };
    const uint32_t acc_bar = bar0 + 8u * (2 * MAX_STAGES);
    const uint32_t push_bar = bar0 + 8u * (2 * MAX_STAGES + 1);
    const uint32_t ready_bar = bar0 + 8u * (2 * MAX_STAGES + 2);
    uint8_t* misc = base_ptr + ring_bytes + 128;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(misc);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int layer = blockIdx.y;
    const int rank = ksplit > 1 ? (int)cluster_ctarank() : 0;
    const int t0 = (int)(blockIdx.x / (unsigned)ksplit) * N;
    const int kblocks = (d + BK - 1) / BK;
    // this CTA's k blocks (ranges differ by at most one block)
    const int kb0 = (int)((long long)rank * kblocks / ksplit);
    const int kb1 = (int)((long long)(rank + 1) * kblocks / ksplit);
    // Token c of the tile is finished by CTA c / per as its row c % per; `per` is a multiple of 32,
    // so the 32 tokens of one tensor-memory read go to one CTA.
    const int n_all = max(0, min(N, T - t0));
    const int per = ((n_all + ksplit - 1) / ksplit + 31) & ~31;
    const int tok_lo = rank * per;
    const int n_mine = max(0, min(per, n_all - tok_lo));
    const bool pair = ksplit == 2;             // partial logits pushed with a bulk copy
    const uint32_t push_bytes = (uint32_t)(per * LD * 4);

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(acc_bar, 1);
        mbar_init(push_bar, 1);
        mbar_init(ready_bar, 1);
        *abort_flag = 0;
        fence_barrier_init();
        // the rows the other CTA of the pair will push here
        if (pair && n_mine > 0) mbar_expect_tx(push_bar, push_bytes);
    }
    if (warp == 1) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), tmem_cols);
    tc_fence_before();
    __syncthreads();
    if (ksplit > 1) cluster_sync_all();        // the peers' barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // nothing above touched global memory: it may have run beside the previous kernel of the stream
    grid_dependency_wait();

    if (warp == 0) {
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            for (int kb = kb0; kb < kb1; ++kb) {
                if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, nullptr)) break;
                const uint32_t sa = base + stage * stage_bytes, sb = sa + a_bytes;
                mbar_expect_tx(full_bar(stage), (uint32_t)stage_bytes);
                tma_load_2d(sb, &tmX, kb * BK, layer * T + t0, full_bar(stage));
                for (int p = 0; p < planes; ++p)
                    for (int m = 0; m < MT; ++m)       // rows beyond E are filled with zeros
                        tma_load_3d(sa + (p * MT + m) * A_BYTES, &tmW, kb * BK, m * BME,
                                    layer * planes + p, full_bar(stage));
                if (++stage == stages) { stage = 0; phase ^= 1u; }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = instr_desc_bf16(BME, N);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int kb = kb0; kb < kb1 && ok; ++kb) {
                if (!mbar_wait(full_bar(stage), phase, abort_flag, nullptr)) { ok = false; break; }
                tc_fence_after();
                const uint32_t sa = base + stage * stage_bytes, sb = sa + a_bytes;
                const uint64_t db = smem_desc_sw128(sb);
                for (int m = 0; m < MT; ++m) {
                    for (int p = 0; p < planes; ++p) {
                        const uint64_t da = smem_desc_sw128(sa + (p * MT + m) * A_BYTES);
#pragma unroll
                        for (int kk = 0; kk < BK / UK; ++kk)
                            tc_mma_bf16(tmem_base + (uint32_t)(m * N), da + (uint64_t)(kk * 2),
                                        db + (uint64_t)(kk * 2), idesc,
                                        ((kb - kb0) | p | kk) != 0 ? 1u : 0u);
                    }
                }
                tc_commit(empty_bar(stage));
                if (++stage == stages) { stage = 0; phase ^= 1u; }
            }
            if (ok && kb1 > kb0) tc_commit(acc_bar);
        }
        __syncwarp();
    } else if (warp < 6) {
        // the accumulator is complete: every copy has landed and every MMA has read its operands
        if (kb1 > kb0) __all_sync(0xffffffffu, mbar_wait(acc_bar, 0u, abort_flag, nullptr));
    }
    tc_fence_before();
    __syncthreads();
    // this grid has fetched its inputs: the next kernel of the stream may begin its set-up
    grid_launch_dependents();
    // a pair: this CTA has left its copy ring, the peer may push rows into it (the signal travels
    // while the accumulator is moved out); 3..8 CTAs store into each other's rings right away:
    // every CTA of the cluster must have left its ring first
    if (pair && threadIdx.x == 0) mbar_arrive_cluster(mapa_shared(ready_bar, (uint32_t)(rank ^ 1)));
    if (ksplit > 2) cluster_sync_all();

    // ------------------------------ epilogue, part 1 ------------------------------------------
    // Every warp moves 32 experts' partial logits of 32 tokens at a time out of tensor memory
    // (one store instruction writes 32 consecutive words of a token's row):
    //   one or two CTAs: into this CTA's own [token][LD] tile, all tokens of the tile;
    //   more CTAs: into slot [this rank][row] of the CTA that finishes the token.
    const int nchunk = (n_all + 31) >> 5;
    auto store_chunks = [&](int chunk_lo, int chunk_hi) {
        const int q = warp & 3;                // the tensor-memory lanes this warp may read
        const int span = chunk_hi - chunk_lo;
        // (M tile, 32-token chunk) pairs are dealt to the three warps of a lane quadrant
        for (int p = warp >> 2; p < MT * span; p += 3) {
            const int m = p / span, c = (chunk_lo + p - m * span) << 5;
            float v[32];
            if (kb1 > kb0) {
                tc_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(m * N + c), v);
                tc_wait_ld();
            } else {                                        // no k block fell to this CTA
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = 0.f;
            }
            const int e_off = m * BME + q * 32 + lane;
            uint32_t dst;
            if (ksplit <= 2) {
                dst = base + 4u * (uint32_t)(c * LD + e_off);
            } else {
                const int owner = c / per, row0 = c - owner * per;
                dst = mapa_shared(base + 4u * (uint32_t)((rank * per + row0) * LD + e_off),
                                  (uint32_t)owner);
            }
            const int n_here = min(32, n_all - c);
#pragma unroll
            for (int i = 0; i < 32; ++i)
                if (i < n_here)
                    asm volatile("st.shared::cluster.f32 [%0], %1;"
                                 ::"r"(dst + 4u * (uint32_t)(i * LD)), "f"(v[i]) : "memory");
        }
    };
    tc_fence_after();
    if (pair) {
        // the peer's tokens first: their rows leave with one bulk copy while this CTA's own rows
        // are still being moved out of tensor memory
        const int peer = rank ^ 1;
        const int peer_lo = min(nchunk, (peer * per) >> 5), peer_hi = min(nchunk, ((peer + 1) * per) >> 5);
        if (!*abort_flag) store_chunks(peer_lo, peer_hi);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncthreads();
        if (threadIdx.x == 0 && peer_hi > peer_lo && !*abort_flag &&
            mbar_wait(ready_bar, 0u, abort_flag, nullptr)) {
            asm volatile(
                "cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                ::"r"(mapa_shared(recv0, (uint32_t)peer)),
                  "r"(base + (uint32_t)(peer * per) * (uint32_t)(LD * 4)), "r"(push_bytes),
                  "r"(mapa_shared(push_bar, (uint32_t)peer)) : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
        const int own_lo = min(nchunk, tok_lo >> 5), own_hi = min(nchunk, (tok_lo + per) >> 5);
        if (!*abort_flag) store_chunks(own_lo, own_hi);
        tc_fence_before();
        __syncthreads();
        if (n_mine > 0) mbar_wait(push_bar, 0u, abort_flag, nullptr);
    } else {
        if (!*abort_flag) store_chunks(0, nchunk);
        tc_fence_before();
        __syncthreads();
        if (ksplit > 2) cluster_sync_all();    // the partial logits of this CTA's tokens have landed
    }

    // ------------------------------ epilogue, part 2 --------------------------------------------
    Partials ps;
    {
        const float* tile = reinterpret_cast<const float*>(base_ptr);
        const float* recv = reinterpret_cast<const float*>(base_ptr + recv_off);
        const float* own = tile + (size_t)tok_lo * LD;
        ps.n = ksplit;
        ps.stride = per * LD;
        ps.p0 = tile;
        ps.p1 = tile + (size_t)per * LD;
        if (pair) {                            // rank order: the lower rank's partial first
            ps.p0 = rank == 0 ? own : recv;
            ps.p1 = rank == 0 ? recv : own;
        }
    }
    const size_t out_row0 = (size_t)layer * T + t0 + tok_lo;
    if (!*abort_flag && logits_out) {
        // one warp per token, lane l writes the experts l, l + 32, ... (coalesced)
        for (int row = warp; row < n_mine; row += THREADS / 32) {
            float v[8];                                  // experts lane, lane + 32, ...
            if (E <= 128) ps.sum<4, 32>(row * LD + lane, v); else ps.sum<8, 32>(row * LD + lane, v);
#pragma unroll
            for (int i = 0; i < 8; ++i)
                if (lane + 32 * i < E) logits_out[(out_row0 + row) * E + lane + 32 * i] = v[i];
        }
    }
    if (!*abort_flag && idx_out) {
        // TopKMask: two lanes per token (16 tokens per warp task), four when the tokens are few
        auto select = [&](auto group_tag) {
            constexpr int GROUP = decltype(group_tag)::value;
            constexpr int TPW = 32 / GROUP;
            for (int task = warp; task * TPW < n_mine; task += THREADS / 32) {
                const int row = task * TPW + (lane / GROUP);
                const bool valid = row < n_mine;
                IdxT* out = idx_out + (out_row0 + (valid ? row : 0)) * K;
                uint32_t redo = K <= 8
                    ? group_topk<IdxT, 8, GROUP>(ps, LD, row, valid, lane % GROUP, E, K, out)
                    : group_topk<IdxT, 16, GROUP>(ps, LD, row, valid, lane % GROUP, E, K, out);
                while (redo) {
                    const int r2 = task * TPW + (__ffs(redo) - 1) / GROUP;
                    redo &= redo - 1;
                    if (E <= 128)
                        warp_topk_exact<IdxT, 4>(ps, LD, r2, lane, E, K, idx_out + (out_row0 + r2) * K);
                    else
                        warp_topk_exact<IdxT, 8>(ps, LD, r2, lane, E, K, idx_out + (out_row0 + r2) * K);
                }
            }
        };
        if (n_mine > 6 * (THREADS / 32)) select(std::integral_constant<int, 2>{});
        else select(std::integral_constant<int, 4>{});
    }

    // ------------------------------ teardown ---------------------------------------------------
    if (pair && threadIdx.x == 0)              // the peer has read the pushed rows out of this CTA
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (ksplit > 1) cluster_sync_all();        // no CTA leaves while a peer may still address it
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, tmem_cols);
    }
}


// ---- CTA-pair form: tokens on the M side, one tile of 256 tokens per pair of SMs ---------------
// tcgen05.mma cta_group::2 with M = 256: CTA r of the pair holds tokens [128 r, 128 r + 128) of
// the tile as its 128 tensor-memory lanes, all E experts as columns.  Per k block it copies its own
// 128 token rows and only HALF of the router rows (experts [r E/2, (r+1) E/2)): the tensor cores of
// the two SMs exchange the halves themselves.  A layer's 256-token decode batch then costs a CTA
// 512 KB of x and 256 KB of W_r (bf16, d = 2048), the bytes of the two-way k split, but every CTA
// ends with the COMPLETE logits of its tokens: no partial sums travel, and lane = token means that
// a thread reads a token's logits straight out of tensor memory, 32 experts at a time.
// 16 warps: warp 0 lane 0 copies, warp 1 lane 0 of the leader issues the MMAs, then warp w takes
// lane quadrant w % 4 and the experts 32 (w / 4), 32 (w / 4) + 128: a thread sorts its 32 (or 64)
// packed candidates into a list of 8 (the networks of group_topk), the lists of a token's four
// threads meet in shared memory and the thread of the first chunk merges them.  A token whose
// packed order is not certain is done again from its full-precision logits (moved to a row buffer
// by the threads that hold them) by one warp with warp_topk_exact, 16 tokens per round.
namespace pairm {
constexpr int TM = 128;                  // tokens per CTA
constexpr int THREADS = 16 * 32;
constexpr int PSTAGES = 8;               // most ring stages
constexpr int X_BYTES = TM * BK * 2;     // 16 KB
constexpr int LIST = 9;                  // 8 candidates + runner
constexpr int REDO_ROWS = 16;
constexpr int EPI_BYTES = 4 * TM * LIST * 4 + REDO_ROWS * 256 * 4 + (TM + 4) * 4;
}  // namespace pairm

template <typename IdxT>
__global__ void __launch_bounds__(pairm::THREADS, 1)
router_pair_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW,
                   IdxT* __restrict__ idx_out, float* __restrict__ logits_out, int T, int d, int E,
                   int K, int planes, int stages, uint32_t tmem_cols, int ring_bytes) {
    using namespace pairm;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const int w_bytes = (E >> 1) * BK * 2;               // half of the router rows, one plane
    const int stage_bytes = X_BYTES + planes * w_bytes;
    const uint32_t bar0 = base + (uint32_t)ring_bytes;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (PSTAGES + s); };
    const uint32_t acc_bar = bar0 + 8u * (2 * PSTAGES);
    uint8_t* misc = base_ptr + ring_bytes + 8 * (2 * PSTAGES + 1);
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(misc);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 4);
    // after the k loop the ring's place holds the lists, the row buffer and the redo list
    float* lists = reinterpret_cast<float*>(base_ptr);                   // [4][TM][LIST]
    float* rowbuf = lists + 4 * TM * LIST;                               // [REDO_ROWS][256]
    int* redo_n = reinterpret_cast<int*>(rowbuf + REDO_ROWS * 256);      // count, then tokens
    int* redo_tok = redo_n + 4;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int layer = blockIdx.y;
    const uint32_t rank = cluster_ctarank();
    const int t0 = (int)(blockIdx.x >> 1) * 2 * TM + (int)rank * TM;   // this CTA's first token
    const int n_mine = max(0, min(TM, T - t0));
    const int kblocks = (d + BK - 1) / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(acc_bar, 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_slot)), tmem_cols);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();            // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // nothing above touched global memory: it may have run beside the previous kernel of the stream
    grid_dependency_wait();

    if (warp == 0) {
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int kb = 0; kb < kblocks; ++kb) {
                if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, nullptr)) { ok = false; break; }
                const uint32_t sx = base + stage * stage_bytes, sw = sx + X_BYTES;
                const uint32_t lead_full = mapa_shared(full_bar(stage), 0);
                if (rank == 0) mbar_expect_tx(full_bar(stage), (uint32_t)(2 * stage_bytes));
                tma_load_2d_pair(sx, &tmX, kb * BK, layer * T + t0, lead_full);
                for (int p = 0; p < planes; ++p)
                    tma_load_3d_pair(sw + p * w_bytes, &tmW, kb * BK, (int)rank * (E >> 1),
                                     layer * planes + p, lead_full);
                if (++stage == stages) { stage = 0; phase ^= 1u; }
            }
            // every stage's release (signalled from the leader's tensor core) has landed
            for (int s = 0; ok && s < stages && s < kblocks; ++s) {
                ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, nullptr);
                if (++stage == stages) { stage = 0; phase ^= 1u; }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = instr_desc_bf16(2 * TM, E);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int kb = 0; kb < kblocks && ok; ++kb) {
                if (!mbar_wait(full_bar(stage), phase, abort_flag, nullptr)) { ok = false; break; }
                tc_fence_after();
                const uint32_t sx = base + stage * stage_bytes, sw = sx + X_BYTES;
                const uint64_t da = smem_desc_sw128(sx);
                for (int p = 0; p < planes; ++p) {
                    const uint64_t db = smem_desc_sw128(sw + p * w_bytes);
#pragma unroll
                    for (int kk = 0; kk < BK / UK; ++kk)
                        tc_mma_bf16_pair(tmem_base, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2),
                                         idesc, (kb | p | kk) != 0 ? 1u : 0u);
                }
                tc_commit_pair(empty_bar(stage), 3);       // frees the stage in both CTAs
                if (++stage == stages) { stage = 0; phase ^= 1u; }
            }
            if (ok) tc_commit_pair(acc_bar, 3);            // accumulators complete, both CTAs
        }
        __syncwarp();
    } else if (warp < 6) {
        // the accumulator is complete: every copy has landed and every MMA has read its operands
        __all_sync(0xffffffffu, mbar_wait(acc_bar, 0u, abort_flag, nullptr));
    }
    tc_fence_before();
    __syncthreads();
    // this grid has fetched its inputs: the next kernel of the stream may begin its set-up
    grid_launch_dependents();
    tc_fence_after();

    // ------------------------------ epilogue -----------------------------------------------------
    const int q = warp & 3, cg = warp >> 2;              // lane quadrant, chunk group
    const int row = q * 32 + lane;                       // token of this thread within the CTA
    const bool valid = row < n_mine && !*abort_flag;
    const size_t out_row = (size_t)layer * T + t0 + row;
    if (threadIdx.x == 0) *redo_n = 0;
    TopList<8> list;
    list.clear();
    for (int c = cg * 32; c < E; c += 128) {             // uniform in the warp
        float v[32];
        tc_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c, v);
        tc_wait_ld();
        if (valid && logits_out) {
            float4* dst = reinterpret_cast<float4*>(logits_out + out_row * E + c);
#pragma unroll
            for (int i = 0; i < 8; ++i)
                if (c + 4 * i < E)                        // E is a multiple of 16
                    dst[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
        }
        if (idx_out) {
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                if (c + 8 * b < E) {
                    float cand[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) cand[i] = pack_candidate(v[8 * b + i], c + 8 * b + i);
                    sort_desc<8>(cand);
                    list.merge(cand, kNoCandidate);
                }
            }
        }
    }
    if (idx_out) {
        float* mine = lists + ((size_t)cg * TM + row) * LIST;
#pragma unroll
        for (int i = 0; i < 8; ++i) mine[i] = list.top[i];
        mine[8] = list.runner;
        __syncthreads();
        if (cg == 0 && valid) {
            for (int g = 1; g < 4 && g * 32 < E; ++g) {
                const float* other = lists + ((size_t)g * TM + row) * LIST;
                float o8[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) o8[i] = other[i];
                list.merge(o8, other[8]);
            }
            bool sure = true;
            IdxT* out = idx_out + out_row * K;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float next = j + 1 < 8 ? list.top[j + 1 < 8 ? j + 1 : j] : list.runner;
                if (j < K) {
                    if ((__float_as_uint(list.top[j]) >> 8) == (__float_as_uint(next) >> 8)) sure = false;
                    out[j] = (IdxT)candidate_expert(list.top[j]);
                }
            }
            if (!sure) redo_tok[atomicAdd(redo_n, 1)] = row;
        }
        __syncthreads();
        // tokens whose packed order was not certain: full-precision rows, one warp each
        const int n_redo = *redo_n;
        for (int r0 = 0; r0 < n_redo; r0 += REDO_ROWS) {
            const int nb = min(REDO_ROWS, n_redo - r0);
            for (int c = cg * 32; c < E; c += 128) {
                float v[32];
                tc_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c, v);
                tc_wait_ld();
                for (int b = 0; b < nb; ++b) {
                    if (redo_tok[r0 + b] == row) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) rowbuf[b * 256 + c + i] = v[i];
                    }
                }
            }
            __syncthreads();
            if (warp < nb) {
                Partials ps;
                ps.p0 = rowbuf;
                ps.p1 = rowbuf;
                ps.stride = 0;
                ps.n = 1;
                const int tok = redo_tok[r0 + warp];
                IdxT* out = idx_out + ((size_t)layer * T + t0 + tok) * K;
                if (E <= 128) warp_topk_exact<IdxT, 4>(ps, 256, warp, lane, E, K, out);
                else warp_topk_exact<IdxT, 8>(ps, 256, warp, lane, E, K, out);
            }
            __syncthreads();
        }
    }

    // ------------------------------ teardown ---------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
        __syncthreads();
    }
    cluster_sync_all();            // neither CTA leaves while the other may still signal it
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, tmem_cols);
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

namespace rt {
// Largest cluster size c <= want such that `units` clusters of c CTAs can all be resident at once
// on the current device (a cluster lives inside one GPC, whose SM count need not be a multiple of
// c: a B200 with 148 SMs holds 74 pairs but only 45 triples).  Cached per (device, c).
template <typename Kern>
static int usable_split(Kern kern, int want, long long units) {
    static int max_clusters[64][MAX_SPLIT + 1] = {};        // 0 = not asked yet, -1 = failed
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 1;
    for (int c = want; c >= 2; --c) {
        if (max_clusters[dev][c] == 0) {
            cudaLaunchConfig_t cfg = {};
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = (unsigned)c;
            attr[0].val.clusterDim.y = 1;
            attr[0].val.clusterDim.z = 1;
            cfg.gridDim = dim3((unsigned)c * 64);
            cfg.blockDim = dim3(THREADS);
            cfg.dynamicSmemBytes = (size_t)SMEM_LIMIT;      // the most a CTA of this kernel asks for
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n <= 0) {
                cudaGetLastError();
                n = -1;
            }
            max_clusters[dev][c] = n;
        }
        if ((long long)max_clusters[dev][c] >= units) return c;
    }
    return 1;
}
}  // namespace rt

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
    // The CTA-pair form (records of up to 8 experts; it writes the logits in 16-byte pieces).  It
    // is taken below where the k-split form would put exactly two CTAs on a tile: with more CTAs
    // per tile the split form is faster (one layer's decode batch: 16.5 us against 20.3 us), with
    // one CTA per tile (many tiles) its coalesced logits stores are (65536 tokens: 0.075 against
    // 0.10 ms).
    // Returns R3_OK after a launch, R3_ERR_UNSUPPORTED when this device cannot run the pair form.
    auto launch_pair_form = [&]() -> r3_status {
        using namespace pairm;
        const int stage_bytes = X_BYTES + planes * (s->E / 2) * BK * 2;
        const int fixed = BAR_BYTES + 1024;
        int stages = (SMEM_LIMIT - fixed) / stage_bytes;
        if (stages > PSTAGES) stages = PSTAGES;
        int ring = stages * stage_bytes;
        if (ring < EPI_BYTES) ring = (EPI_BYTES + 127) & ~127;
        uint32_t cols = 32;
        while ((int)cols < s->E) cols <<= 1;
        CUtensorMap px, pw;
        if (!make_map_2d(&px, x, (uint64_t)L * s->T, (uint64_t)s->d, TM) ||
            !make_map_3d(&pw, wplanes, (uint64_t)L * planes, (uint64_t)s->E, (uint64_t)s->d,
                         (uint32_t)(s->E / 2)))
            return R3_ERR_CUDA;
        cudaLaunchConfig_t pc = {};
        cudaLaunchAttribute pa[2];
        pa[0].id = cudaLaunchAttributeClusterDimension;
        pa[0].val.clusterDim.x = 2;
        pa[0].val.clusterDim.y = 1;
        pa[0].val.clusterDim.z = 1;
        pa[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        pa[1].val.programmaticStreamSerializationAllowed = 1;
        const int tiles = (s->T + 2 * TM - 1) / (2 * TM);
        pc.gridDim = dim3((unsigned)(2 * tiles), (unsigned)L);
        pc.blockDim = dim3(pairm::THREADS);
        pc.dynamicSmemBytes = (size_t)(ring + fixed);
        pc.stream = cs;
        pc.attrs = pa;
        pc.numAttrs = 2;
        static int pair_ok[64][2] = {};         // per device and index type: 0 untested, 1 yes, -1 no
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return R3_ERR_CUDA;
        const int ti = s->idx_type == R3_IDX_U8 ? 0 : 1;
        cudaError_t le = cudaSuccess;
#define R3_RP(IDX)                                                                              \
        do {                                                                                    \
            auto kern = router_pair_kernel<IDX>;                                                \
            if (pair_ok[dev][ti] == 0) {                                                        \
                int n = 0;                                                                      \
                cudaLaunchConfig_t probe = pc;                                                  \
                probe.numAttrs = 1;                                                             \
                probe.dynamicSmemBytes = (size_t)SMEM_LIMIT;                                    \
                pair_ok[dev][ti] =                                                              \
                    (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,    \
                                          SMEM_LIMIT) == cudaSuccess &&                         \
                     cudaOccupancyMaxActiveClusters(&n, kern, &probe) == cudaSuccess && n >= 1) \
                        ? 1 : -1;                                                               \
                if (pair_ok[dev][ti] < 0) cudaGetLastError();                                   \
            }                                                                                   \
            if (pair_ok[dev][ti] == 1)                                                          \
                le = cudaLaunchKernelEx(&pc, kern, px, pw, static_cast<IDX*>(idx_out),          \
                                        logits_out, (int)s->T, (int)s->d, (int)s->E, (int)s->K, \
                                        planes, stages, cols, ring);                            \
        } while (0)
        if (ti == 0) R3_RP(uint8_t); else R3_RP(int16_t);
#undef R3_RP
        if (pair_ok[dev][ti] == 1) return le == cudaSuccess ? launch_status() : R3_ERR_CUDA;
        return R3_ERR_UNSUPPORTED;
    };
    const bool pair_form_fits = s->K <= 8 && aligned(logits_out, 16);
    // token tiles of a layer: as few as possible, of equal size (a multiple of 16); with two M
    // tiles (E > 128) the logits of 256 tokens would not fit in shared memory
    const int MT = (s->E + BME - 1) / BME;
    const int n_max = MT == 1 ? 256 : 128;
    const int tiles = (s->T + n_max - 1) / n_max;
    const int N = (((s->T + tiles - 1) / tiles) + 15) & ~15;
    const int kblocks = (s->d + BK - 1) / BK;
    const int LD = MT * BME + 1;
    const int stage_bytes = planes * MT * A_BYTES + N * BK * 2;
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < MT * N) tmem_cols <<= 1;

    CUtensorMap mx, mw;
    if (!make_map_2d(&mx, x, (uint64_t)L * s->T, (uint64_t)s->d, (uint32_t)N) ||
        !make_map_3d(&mw, wplanes, (uint64_t)L * planes, (uint64_t)s->E, (uint64_t)s->d, BME))
        return R3_ERR_CUDA;
    const long long units = (long long)tiles * L;
    // What a cluster of c CTAs keeps in the ring's place once the ring is free: per = tokens
    // finished by one CTA (a multiple of 32).  c <= 2: the whole tile [c * per][LD] and, for
    // c = 2, behind it the rows pushed by the peer [per][LD].  c > 2: the slots [c][per][LD].
    auto per_of = [&](int c) { return (((N + c - 1) / c) + 31) & ~31; };
    auto tile_of = [&](int c) { return (c * per_of(c) * LD * 4 + 127) & ~127; };
    auto recv_of = [&](int c) { return c == 2 ? per_of(c) * LD * 4 : 0; };
    const int fixed = BAR_BYTES + 1024;
    auto fits = [&](int c) {
        const int after = tile_of(c) + recv_of(c);
        return (after > 2 * stage_bytes ? after : 2 * stage_bytes) + fixed <= SMEM_LIMIT;
    };
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.blockDim = dim3(THREADS);
    cfg.stream = cs;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
#define R3_RT(IDX)                                                                              \
    do {                                                                                        \
        auto kern = router_tc_kernel<IDX>;                                                      \
        static bool attr_set[64] = {};         /* per device */                                 \
        int dev = 0;                                                                            \
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return R3_ERR_CUDA;     \
        if (!attr_set[dev]) {                                                                   \
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,         \
                                     SMEM_LIMIT) != cudaSuccess)                                \
                return R3_ERR_CUDA;                                                             \
            attr_set[dev] = true;                                                               \
        }                                                                                       \
        /* few tiles: the CTAs of a cluster share a tile's k blocks, as many as give every CTA  \
           an SM of its own and at least two k blocks, and whose slots fit in shared memory */  \
        int want = (int)(sm_count() / (units > 0 ? units : 1));                                 \
        if (want > MAX_SPLIT) want = MAX_SPLIT;                                                 \
        if (want > kblocks / 2) want = kblocks / 2;                                             \
        while (want > 1 && !fits(want)) --want;                                                 \
        int ksplit = want >= 2 ? usable_split(kern, want, units) : 1;                           \
        while (ksplit > 1 && !fits(ksplit)) --ksplit;                                           \
        if (!fits(ksplit)) return R3_ERR_UNSUPPORTED;                                           \
        if (ksplit == 2 && pair_form_fits) {                                                    \
            const r3_status ps = launch_pair_form();                                            \
            if (ps != R3_ERR_UNSUPPORTED) return ps;                                            \
        }                                                                                       \
        int stages = (SMEM_LIMIT - fixed) / stage_bytes;                                        \
        if (stages > MAX_STAGES) stages = MAX_STAGES;                                           \
        int ring = stages * stage_bytes;                                                        \
        const int after = tile_of(ksplit) + recv_of(ksplit);                                    \
        if (ring < after) ring = (after + 127) & ~127;                                          \
        attr[0].val.clusterDim.x = (unsigned)ksplit;                                            \
        cfg.gridDim = dim3((unsigned)(tiles * ksplit), (unsigned)L);                            \
        cfg.dynamicSmemBytes = (size_t)(ring + fixed);                                          \
        if (cudaLaunchKernelEx(&cfg, kern, mx, mw, static_cast<IDX*>(idx_out), logits_out,      \
                               (int)s->T, (int)s->d, (int)s->E, (int)s->K, planes, stages,      \
                               tmem_cols, ksplit, N, MT, ring, tile_of(ksplit)) != cudaSuccess) \
            return R3_ERR_CUDA;                                                                 \
    } while (0)
    if (s->idx_type == R3_IDX_U8) R3_RT(uint8_t); else R3_RT(int16_t);
#undef R3_RT
    return launch_status();
}

}  // namespace r3
