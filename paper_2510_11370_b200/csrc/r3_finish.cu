// One pass over the expert outputs that does everything after the expert networks:
//   replay gate (Eq. replay_gate)            g[t,j]  = softmax over the K recorded logits
//   combine     (Eq. replay_output)          y[t]    = sum_j g[t,j] o[row_of_slot[t,j]] (+ residual)
//   gate gradient                            dg[t,j] = <dy[t], o[row_of_slot[t,j]]>
//   router-logit gradient                    ds[t,e_j] = g_j (dg_j - sum_j' g_j' dg_j'), 0 elsewhere
// The separate kernels (r3_replay_gate_fwd, r3_combine, r3_combine_bwd_gates, r3_replay_gate_bwd)
// read every expert-output row twice and need four launches; here a team of threads owns a token,
// gathers its K rows once, and keeps the same arithmetic and the same summation orders as those
// kernels, so the results are bit-identical to theirs.  No atomics.
#include <algorithm>

#include "r3_common.cuh"
#include "r3_internal.h"
#include "r3_tc.cuh"

namespace r3 {

constexpr int kFusedMaxK = 8;     // slots held in registers per thread

template <typename ActT, typename IdxT, int TPT>
__global__ void __launch_bounds__(256, 3)
replay_finish_kernel(const float* __restrict__ logits, const IdxT* __restrict__ idx,
                     const ActT* __restrict__ o, const int32_t* __restrict__ row_of_slot,
                     const ActT* __restrict__ dy, const ActT* __restrict__ residual,
                     ActT* __restrict__ y, float* __restrict__ gates_out,
                     float* __restrict__ dlogits, int T, int E, int K, int d, int W,
                     int32_t* dev_status) {
    using V = Vec16<ActT>;
    constexpr int N = V::N;
    constexpr int TEAMS = 256 / TPT;
    constexpr int WPT = TPT / 32;                      // warps per team
    __shared__ float g_s[TEAMS][kFusedMaxK];
    __shared__ float dg_s[TEAMS][kFusedMaxK];
    __shared__ float part[256 / 32][kFusedMaxK];

    const int team = threadIdx.x / TPT, tl = threadIdx.x % TPT;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int t = blockIdx.x * TEAMS + team;
    const bool live = t < T;                           // no early exit: block-wide barriers below
    const int tt = live ? t : T - 1;
    const IdxT* rec = idx + (size_t)tt * K;

    // The K row gathers of the first column piece do not depend on the gates: they are issued
    // first, so that they are in flight while the team's first warp works out the gates.
    const int row_vecs = d / N;
    const int32_t* rows = row_of_slot + (size_t)tt * K;
    const V* ov = reinterpret_cast<const V*>(o);
    const V* dyv = reinterpret_cast<const V*>(dy) + (size_t)tt * row_vecs;
    V* yv = reinterpret_cast<V*>(y) + (size_t)tt * row_vecs;
    unsigned have = 0;                                  // bit u: slot u has a row
    V v[kFusedMaxK], dv;
    {
        int32_t r[kFusedMaxK];
#pragma unroll
        for (int u = 0; u < kFusedMaxK; ++u) {
            r[u] = u < K ? rows[u] : -1;
            if (r[u] >= 0) have |= 1u << u;
        }
        if (tl < row_vecs) {
#pragma unroll
            for (int u = 0; u < kFusedMaxK; ++u)
                if (r[u] >= 0) v[u] = ov[(size_t)r[u] * row_vecs + tl];
            dv = dyv[tl];
        }
    }

    // ---- replay gate: the first W lanes of the team, one slot each (K <= W <= 32) ------------
    int my_e = -1;
    if (tl < 32) {
        const float* row = logits + (size_t)tt * E;
        int bad = 0;
        float s = -INFINITY;
        if (tl < K) {
            my_e = idx_to_int(rec[tl]);
            if (my_e < 0 || my_e >= E) bad |= 1;
            for (int j2 = 0; j2 < tl; ++j2)
                if (idx_to_int(rec[j2]) == my_e) bad |= 2;
            s = row[min(max(my_e, 0), E - 1)];
        }
        for (int ofs = W / 2; ofs > 0; ofs >>= 1) bad |= __shfl_xor_sync(0xffffffffu, bad, ofs, W);
        if (bad && live && tl == 0)
            report(dev_status, (bad & 1) ? R3_DEV_BAD_INDEX : R3_DEV_DUP_INDEX);
        float m = s;
        for (int ofs = W / 2; ofs > 0; ofs >>= 1)
            m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, ofs, W));
        const float ex = tl < K ? expf(s - m) : 0.f;
        float sum = ex;
        for (int ofs = W / 2; ofs > 0; ofs >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, ofs, W);
        const float inv = bad ? 0.f : 1.f / sum;
        if (tl < K) {
            const float g = ex * inv;
            g_s[team][tl] = g;
            if (gates_out && live) gates_out[(size_t)t * K + tl] = g;
        }
    }
    __syncthreads();

    // ---- combine and <dy, o_j> from the gathered rows -------------------------------------------
    float dacc[kFusedMaxK];
#pragma unroll
    for (int u = 0; u < kFusedMaxK; ++u) dacc[u] = 0.f;
    for (int c = tl; c < row_vecs; c += TPT) {
        if (c != tl) {                       // later column pieces (d wider than one pass)
#pragma unroll
            for (int u = 0; u < kFusedMaxK; ++u)
                if (have >> u & 1u) v[u] = ov[(size_t)rows[u] * row_vecs + c];
            dv = dyv[c];
        }
        float gr[N];
        dv.unpack(gr);
        float acc[N];
#pragma unroll
        for (int i = 0; i < N; ++i) acc[i] = 0.f;
#pragma unroll
        for (int u = 0; u < kFusedMaxK; ++u) {
            if (have >> u & 1u) {
                const float gu = g_s[team][u];
                float f[N];
                v[u].unpack(f);
#pragma unroll
                for (int i = 0; i < N; ++i) acc[i] = fmaf(gu, f[i], acc[i]);
#pragma unroll
                for (int i = 0; i < N; ++i) dacc[u] = fmaf(gr[i], f[i], dacc[u]);
            }
        }
        if (residual) {                      // y = residual + sum (one extra fp32 add per element)
            float f[N];
            reinterpret_cast<const V*>(residual)[(size_t)tt * row_vecs + c].unpack(f);
#pragma unroll
            for (int i = 0; i < N; ++i) acc[i] += f[i];
        }
        if (live) {
            V out;
            out.pack(acc);
            yv[c] = out;
        }
    }

    // ---- dg: warp shuffles, then the team's warps in a fixed order ------------------------------
#pragma unroll
    for (int u = 0; u < kFusedMaxK; ++u) {
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) dacc[u] += __shfl_xor_sync(0xffffffffu, dacc[u], s);
    }
    if (lane == 0) {
#pragma unroll
        for (int u = 0; u < kFusedMaxK; ++u) part[warp][u] = dacc[u];
    }
    __syncthreads();
    if (tl < kFusedMaxK) {
        float s = 0.f;
        for (int w = 0; w < WPT; ++w) s += part[team * WPT + w][tl];   // fixed order
        dg_s[team][tl] = s;
    }
    __syncthreads();

    // ---- router-logit gradient: the team's first warp writes the dense row once ----------------
    if (tl < 32 && live) {
        const float g = tl < K ? g_s[team][tl] : 0.f;
        const float dg = tl < K ? dg_s[team][tl] : 0.f;
        float c = g * dg;
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) c += __shfl_xor_sync(0xffffffffu, c, s);
        const float v = g * (dg - c);
        float* out = dlogits + (size_t)t * E;
        const int nchunk = (E + 3) >> 2;
        for (int ch = tl; ch < ((nchunk + 31) & ~31); ch += 32) {
            float q[4] = {0.f, 0.f, 0.f, 0.f};
            for (int j = 0; j < K; ++j) {
                const int ej = __shfl_sync(0xffffffffu, my_e, j);
                const float vj = __shfl_sync(0xffffffffu, v, j);
                if ((ej >> 2) == ch) q[ej & 3] = vj;
            }
            if (ch < nchunk) {
                const int e0 = ch << 2;
                if (e0 + 3 < E && (E & 3) == 0) {
                    *reinterpret_cast<float4*>(out + e0) = make_float4(q[0], q[1], q[2], q[3]);
                } else {
                    for (int i = 0; i < 4 && e0 + i < E; ++i) out[e0 + i] = q[i];
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// The same computation with the token's rows staged in shared memory: one CTA of 4 warps per
// token.  At its start the CTA asks for the token's K expert-output rows, its dy row and its
// residual row with bulk asynchronous copies (one lane and one copy per row, completion counted on
// an mbarrier); the data in flight lives in shared memory instead of registers, so six CTAs fit
// on an SM and keep about 200 KB of copies per SM in flight while the first warp works out the
// gates from the logits.  The four warps then split the columns.
// y and the gates are bit-identical to the separate kernels (same per-element order); the gate
// gradient is summed per lane over the columns, across the warp and then over the four warps,
// a different (fixed) order than r3_combine_bwd_gates, so dlogits agrees with the separate
// kernels to rounding.
// ---------------------------------------------------------------------------------------------
constexpr int kTokWarps = 4;
constexpr int kTokThreads = kTokWarps * 32;
constexpr int kTokHeader = 128;           // mbarrier, flags, gates, partial sums
constexpr int kTokSmemLimit = 227 * 1024;

__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes,
                                          uint32_t bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// PTR: the expert-output row of slot (t, j) is given by its address row_ptr[t, j] (0 = no row)
// instead of by a row number into `o` - the rows may then live in several buffers, also in another
// GPU's memory that this GPU can address (plain bulk copies, no multicast).
template <typename ActT, typename IdxT, bool PTR>
__global__ void __launch_bounds__(kTokThreads)
replay_finish_staged_kernel(const float* __restrict__ logits, const IdxT* __restrict__ idx,
                            const ActT* __restrict__ o, const int32_t* __restrict__ row_of_slot,
                            const unsigned long long* __restrict__ row_ptr,
                            const ActT* __restrict__ dy, const ActT* __restrict__ residual,
                            ActT* __restrict__ y, float* __restrict__ gates_out,
                            float* __restrict__ dlogits, int E, int K, int d, int W,
                            int32_t* dev_status) {
    using V = Vec16<ActT>;
    constexpr int N = V::N;
    extern __shared__ __align__(128) uint8_t smem_tok[];
    const uint32_t bar = tc::smem_u32(smem_tok);                       // 8 bytes
    volatile int* flags = reinterpret_cast<volatile int*>(smem_tok + 8);   // [0] abort [1] ready
    unsigned* have_s = reinterpret_cast<unsigned*>(smem_tok + 16);
    float* g_s = reinterpret_cast<float*>(smem_tok + 32);               // [8]
    const V* orow = reinterpret_cast<const V*>(smem_tok + kTokHeader + 128);
    float* part2 = reinterpret_cast<float*>(smem_tok + kTokHeader);     // [kTokWarps][8] = 128 bytes

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int t = blockIdx.x;
    const int row_vecs = d / N;
    const uint32_t row_bytes = (uint32_t)d * sizeof(ActT);

    int my_e = -1;
    float g = 0.f;
    tc::grid_launch_dependents();
    tc::grid_dependency_wait();            // everything this kernel reads may come from the one before
    if (warp == 0) {
        // ---- the token's record and row numbers first (independent loads), then the logit of
        // each recorded expert, so that only two memory latencies precede the copies ------------
        const IdxT* rec = idx + (size_t)t * K;
        const float* lrow = logits + (size_t)t * E;
        int32_t r = -1;
        const ActT* src_row = nullptr;
        if (lane < K) {
            my_e = idx_to_int(rec[lane]);
            if (PTR) {
                src_row = reinterpret_cast<const ActT*>(row_ptr[(size_t)t * K + lane]);
                r = src_row ? 0 : -1;
            } else {
                r = row_of_slot[(size_t)t * K + lane];
                if (r >= 0) src_row = o + (size_t)r * d;
            }
        }
        // ---- ask for the rows ---------------------------------------------------------------------
        // dy and the residual row do not wait for the row numbers: their copies start at once
        // (bytes may land before the barrier is told how many to expect; its one pending
        // arrival, the expect_tx below, keeps the phase open until then)
        if (lane == 0) {
            tc::mbar_init(bar, 1);
            flags[0] = 0;
            tc::fence_barrier_init();
        }
        __syncwarp();
        const uint32_t s_rows = tc::smem_u32(orow);
        if (lane == K) {
            bulk_load(s_rows + (uint32_t)K * row_bytes, dy + (size_t)t * d, row_bytes, bar);
        } else if (lane == K + 1) {
            if (residual)
                bulk_load(s_rows + (uint32_t)(K + 1) * row_bytes, residual + (size_t)t * d,
                          row_bytes, bar);
        }
        float s = -INFINITY;
        if (lane < K) s = lrow[min(max(my_e, 0), E - 1)];      // in flight while the rows are asked for
        const unsigned have = __ballot_sync(0xffffffffu, r >= 0);
        if (lane == 0) {
            *have_s = have;
            tc::mbar_expect_tx(bar, row_bytes * (uint32_t)(__popc(have) + 1 + (residual ? 1 : 0)));
        }
        __syncwarp();
        if (lane < K && r >= 0)
            bulk_load(s_rows + (uint32_t)lane * row_bytes, src_row, row_bytes, bar);
        // ---- replay gate while the copies fly: the first W lanes, one slot each -----------------
        int bad = 0;
        if (lane < K && (my_e < 0 || my_e >= E)) bad |= 1;
        for (int j2 = 0; j2 < K; ++j2) {
            const int e2 = __shfl_sync(0xffffffffu, my_e, j2);
            if (j2 < lane && lane < K && e2 == my_e) bad |= 2;
        }
        for (int ofs = W / 2; ofs > 0; ofs >>= 1) bad |= __shfl_xor_sync(0xffffffffu, bad, ofs, W);
        if (bad && lane == 0)
            report(dev_status, (bad & 1) ? R3_DEV_BAD_INDEX : R3_DEV_DUP_INDEX);
        float m = s;
        for (int ofs = W / 2; ofs > 0; ofs >>= 1)
            m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, ofs, W));
        const float ex = lane < K ? expf(s - m) : 0.f;
        float sum = ex;
        for (int ofs = W / 2; ofs > 0; ofs >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, ofs, W);
        const float inv = bad ? 0.f : 1.f / sum;
        if (lane < K) {
            g = ex * inv;
            if (gates_out) gates_out[(size_t)t * K + lane] = g;
        }
        if (lane < kFusedMaxK) g_s[lane] = g;
        // ---- one thread waits for the copies; the others sleep at the barrier below -----------
        if (lane == 0) flags[1] = tc::mbar_wait(bar, 0u, flags, dev_status) ? 1 : 0;
    }
    __syncthreads();
    const bool ready = flags[1] != 0;

    // ---- combine and <dy, o_j> out of shared memory: the warps split the columns ------------------
    float dacc[kFusedMaxK];
#pragma unroll
    for (int u = 0; u < kFusedMaxK; ++u) dacc[u] = 0.f;
    if (ready) {
        const unsigned have = *have_s;
        float gj[kFusedMaxK];
#pragma unroll
        for (int u = 0; u < kFusedMaxK; ++u) gj[u] = g_s[u];
        V* yv = reinterpret_cast<V*>(y) + (size_t)t * row_vecs;
        for (int c = tid; c < row_vecs; c += kTokThreads) {
            float gr[N];
            orow[(size_t)K * row_vecs + c].unpack(gr);
            float acc[N];
#pragma unroll
            for (int k2 = 0; k2 < N; ++k2) acc[k2] = 0.f;
#pragma unroll
            for (int u = 0; u < kFusedMaxK; ++u) {
                if (have >> u & 1u) {
                    float f[N];
                    orow[(size_t)u * row_vecs + c].unpack(f);
#pragma unroll
                    for (int k2 = 0; k2 < N; ++k2) acc[k2] = fmaf(gj[u], f[k2], acc[k2]);
#pragma unroll
                    for (int k2 = 0; k2 < N; ++k2) dacc[u] = fmaf(gr[k2], f[k2], dacc[u]);
                }
            }
            if (residual) {
                float f[N];
                orow[(size_t)(K + 1) * row_vecs + c].unpack(f);
#pragma unroll
                for (int k2 = 0; k2 < N; ++k2) acc[k2] += f[k2];
            }
            V out;
            out.pack(acc);
            yv[c] = out;
        }
    }
    // ---- dg: across the warp, then the four warps in a fixed order -------------------------------
#pragma unroll
    for (int u = 0; u < kFusedMaxK; ++u) {
#pragma unroll
        for (int sft = 16; sft > 0; sft >>= 1) dacc[u] += __shfl_xor_sync(0xffffffffu, dacc[u], sft);
    }
    if (lane == 0) {
#pragma unroll
        for (int u = 0; u < kFusedMaxK; ++u) part2[warp * kFusedMaxK + u] = dacc[u];
    }
    __syncthreads();
    if (warp == 0 && ready) {
        float dg = 0.f;
        if (lane < kFusedMaxK) {
            for (int w2 = 0; w2 < kTokWarps; ++w2) dg += part2[w2 * kFusedMaxK + lane];
        }
        float cs = g * dg;                                        // lanes >= K hold g = 0
#pragma unroll
        for (int sft = 16; sft > 0; sft >>= 1) cs += __shfl_xor_sync(0xffffffffu, cs, sft);
        const float val = g * (dg - cs);
        float* out = dlogits + (size_t)t * E;
        const int nchunk = (E + 3) >> 2;
        if ((E & 3) == 0 && (size_t)E * sizeof(float) <= (size_t)(K + 1) * row_bytes) {
            // the row buffers are free now: build the dense row there (zeros, then the K values)
            // and write it out in 16-byte pieces - a dozen instructions per lane instead of a scan
            // of the K slots by every lane
            float* stage = reinterpret_cast<float*>(smem_tok + kTokHeader + 128);
            for (int ch = lane; ch < nchunk; ch += 32)
                reinterpret_cast<float4*>(stage)[ch] = make_float4(0.f, 0.f, 0.f, 0.f);
            __syncwarp();
            if (lane < K && my_e >= 0 && my_e < E) stage[my_e] = val;
            __syncwarp();
            for (int ch = lane; ch < nchunk; ch += 32)
                reinterpret_cast<float4*>(out)[ch] = reinterpret_cast<const float4*>(stage)[ch];
        } else
        for (int ch = lane; ch < ((nchunk + 31) & ~31); ch += 32) {
            float q0 = 0.f, q1 = 0.f, q2 = 0.f, q3 = 0.f;          // selects, no branches
#pragma unroll
            for (int j = 0; j < kFusedMaxK; ++j) {
                if (j < K) {
                    const int ej = __shfl_sync(0xffffffffu, my_e, j);
                    const float vj = __shfl_sync(0xffffffffu, val, j);
                    const int w = (ej >> 2) == ch ? (ej & 3) : -1;
                    q0 = w == 0 ? vj : q0;
                    q1 = w == 1 ? vj : q1;
                    q2 = w == 2 ? vj : q2;
                    q3 = w == 3 ? vj : q3;
                }
            }
            if (ch < nchunk) {
                const int e0 = ch << 2;
                if ((E & 3) == 0) {
                    *reinterpret_cast<float4*>(out + e0) = make_float4(q0, q1, q2, q3);
                } else {
                    const float q[4] = {q0, q1, q2, q3};
                    for (int k2 = 0; k2 < 4 && e0 + k2 < E; ++k2) out[e0 + k2] = q[k2];
                }
            }
        }
    }
    if (!ready) {
        // the wait ran out: copies may still be in flight into this CTA's shared memory
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    }
}

static int pick_team_fused(int row_vecs) {
    int tpt = 32;
    while (tpt < 256 && tpt < row_vecs) tpt <<= 1;
    return tpt;
}

template <typename ActT, typename IdxT>
static r3_status launch_finish(const r3_shape* s, const float* logits, const void* idx,
                               const void* o, const int32_t* row_of_slot,
                               const unsigned long long* row_ptr, const void* dy,
                               const void* residual, void* y, float* gates_out, float* dlogits,
                               int32_t* dev_status, cudaStream_t cs) {
    const int T = s->T, K = s->K, d = s->d, E = s->E;
    int W = 1;
    while (W < K && W < 32) W <<= 1;
    // staged kernel: one CTA per token, its K + 2 rows in shared memory (when they fit)
    const size_t smem = kTokHeader + 128 + (size_t)(K + 1 + (residual ? 1 : 0)) * d * sizeof(ActT);
    if (smem <= (size_t)kTokSmemLimit / 2 && row_ptr) {
        auto kern = replay_finish_staged_kernel<ActT, IdxT, true>;
        static PerDevice attr_set;             // one set of flags per instantiation
        if (!attr_set.done()) {
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     kTokSmemLimit / 2) != cudaSuccess)
                return R3_ERR_CUDA;
            attr_set.mark();
        }
        if (tc::launch_dependent(kern, dim3(T), dim3(kTokThreads), smem, cs, logits,
                                 static_cast<const IdxT*>(idx), nullptr, nullptr, row_ptr,
                                 static_cast<const ActT*>(dy), static_cast<const ActT*>(residual),
                                 static_cast<ActT*>(y), gates_out, dlogits, E, K, d, W,
                                 dev_status) != cudaSuccess)
            return R3_ERR_CUDA;
        return R3_OK;
    }
    if (row_ptr) return R3_ERR_UNSUPPORTED;    // rows by address need the staged kernel
    if (smem <= (size_t)kTokSmemLimit / 2) {
        auto kern = replay_finish_staged_kernel<ActT, IdxT, false>;
        static PerDevice attr_set;             // one set of flags per instantiation
        if (!attr_set.done()) {
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     kTokSmemLimit / 2) != cudaSuccess)
                return R3_ERR_CUDA;
            attr_set.mark();
        }
        if (tc::launch_dependent(kern, dim3(T), dim3(kTokThreads), smem, cs, logits,
                                 static_cast<const IdxT*>(idx), static_cast<const ActT*>(o),
                                 row_of_slot, nullptr, static_cast<const ActT*>(dy),
                                 static_cast<const ActT*>(residual), static_cast<ActT*>(y),
                                 gates_out, dlogits, E, K, d, W, dev_status) != cudaSuccess)
            return R3_ERR_CUDA;
        return R3_OK;
    }
    const int tpt = pick_team_fused(d / Vec16<ActT>::N);
    const unsigned grid = (unsigned)((T + 256 / tpt - 1) / (256 / tpt));
#define R3_FIN(TPT)                                                                              \
    replay_finish_kernel<ActT, IdxT, TPT><<<grid, 256, 0, cs>>>(                                 \
        logits, static_cast<const IdxT*>(idx), static_cast<const ActT*>(o), row_of_slot,         \
        static_cast<const ActT*>(dy), static_cast<const ActT*>(residual), static_cast<ActT*>(y), \
        gates_out, dlogits, T, E, K, d, W, dev_status)
    switch (tpt) {
        case 32: R3_FIN(32); break;
        case 64: R3_FIN(64); break;
        case 128: R3_FIN(128); break;
        default: R3_FIN(256); break;
    }
#undef R3_FIN
    return R3_OK;
}

}  // namespace r3

extern "C" r3_status r3_replay_finish(const r3_shape* shape, const float* logits, const void* idx,
                                      const void* o, const int32_t* row_of_slot, const void* dy,
                                      const void* residual, void* y, float* gates_out,
                                      float* dlogits, int32_t* dev_status, void* stream) {
    r3_status st = r3::check_shape(shape);
    if (st != R3_OK) return st;
    if (shape->K > r3::kFusedMaxK) return R3_ERR_UNSUPPORTED;
    if (shape->T == 0) return R3_OK;
    if (!logits || !idx || !o || !row_of_slot || !dy || !y || !dlogits) return R3_ERR_INVALID_ARG;
    if (!r3::aligned(o, 16) || !r3::aligned(dy, 16) || !r3::aligned(y, 16) ||
        !r3::aligned(residual, 16))
        return R3_ERR_INVALID_ARG;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    R3_DISPATCH_ACT(shape, ActT, R3_DISPATCH_IDX(shape, IdxT,
        (st = r3::launch_finish<ActT, IdxT>(shape, logits, idx, o, row_of_slot, nullptr, dy,
                                            residual, y, gates_out, dlogits, dev_status, cs))));
    return st != R3_OK ? st : r3::launch_status();
}

extern "C" r3_status r3_replay_finish_rows(const r3_shape* shape, const float* logits,
                                           const void* idx, const unsigned long long* row_ptr,
                                           const void* dy, const void* residual, void* y,
                                           float* gates_out, float* dlogits, int32_t* dev_status,
                                           void* stream) {
    r3_status st = r3::check_shape(shape);
    if (st != R3_OK) return st;
    if (shape->K > r3::kFusedMaxK) return R3_ERR_UNSUPPORTED;
    if (shape->T == 0) return R3_OK;
    if (!logits || !idx || !row_ptr || !dy || !y || !dlogits) return R3_ERR_INVALID_ARG;
    if (!r3::aligned(dy, 16) || !r3::aligned(y, 16) || !r3::aligned(residual, 16))
        return R3_ERR_INVALID_ARG;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    R3_DISPATCH_ACT(shape, ActT, R3_DISPATCH_IDX(shape, IdxT,
        (st = r3::launch_finish<ActT, IdxT>(shape, logits, idx, nullptr, nullptr, row_ptr, dy,
                                            residual, y, gates_out, dlogits, dev_status, cs))));
    return st != R3_OK ? st : r3::launch_status();
}
