// Token dispatch for the replayed layer: group the R = T*K (token, slot) pairs by recorded
// expert, stably, and copy each token's row to its K destination rows.
//
// Determinism: ranks never depend on the arrival order of atomics.  A CTA owns a chunk of 256
// consecutive tokens; (1) it counts its pairs per expert (integer atomics on shared counters -
// the sum does not depend on order), (2) one CTA turns the [expert][chunk] counts into exclusive
// prefixes and the expert offsets, (3) each CTA marks, per expert, the bitmap of its tokens that
// chose the expert; the rank of a pair inside the chunk is the number of lower set bits.
// A pair whose index is out of range, or repeats an earlier slot of the same token, is dropped
// (row_of_slot = -1) and reported through dev_status.
#include <cooperative_groups.h>

#include "r3_common.cuh"
#include "r3_internal.h"
#include "r3_tc.cuh"
#include "r3_worklist.cuh"

namespace r3 {

constexpr int kChunk = 256;               // tokens per CTA in the counting / ranking kernels
constexpr int kWords = kChunk / 32;

template <typename IdxT>
__device__ __forceinline__ bool pair_ok(const IdxT* rec, int j, int E, int& e, int32_t* dev_status) {
    e = idx_to_int(rec[j]);
    if (e < 0 || e >= E) { report(dev_status, R3_DEV_BAD_INDEX); return false; }
    for (int j2 = 0; j2 < j; ++j2)
        if (idx_to_int(rec[j2]) == e) { report(dev_status, R3_DEV_DUP_INDEX); return false; }
    return true;
}

template <typename IdxT>
__global__ void __launch_bounds__(kChunk)
permute_count_kernel(const IdxT* __restrict__ idx, int32_t* __restrict__ chunk_counts,
                     int T, int E, int K, int NB, int32_t* dev_status) {
    extern __shared__ int32_t hist[];
    for (int e = threadIdx.x; e < E; e += kChunk) hist[e] = 0;
    __syncthreads();
    const int t = blockIdx.x * kChunk + threadIdx.x;
    if (t < T) {
        const IdxT* rec = idx + (size_t)t * K;
        for (int j = 0; j < K; ++j) {
            int e;
            if (pair_ok(rec, j, E, e, dev_status)) atomicAdd(&hist[e], 1);
        }
    }
    __syncthreads();
    for (int e = threadIdx.x; e < E; e += kChunk)
        chunk_counts[(size_t)e * NB + blockIdx.x] = hist[e];
}

// One CTA.  In place: chunk_counts[e][b] becomes the number of expert-e pairs in chunks < b.
// Also writes counts[E] and offsets[E+1].
__global__ void __launch_bounds__(1024)
permute_scan_kernel(int32_t* __restrict__ chunk_counts, int32_t* __restrict__ counts,
                    int32_t* __restrict__ offsets, int E, int NB) {
    __shared__ int32_t total[kMaxExpertsPermute];
    __shared__ int32_t warp_sum[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int e = warp; e < E; e += 32) {
        int32_t* row = chunk_counts + (size_t)e * NB;
        int32_t carry = 0;
        for (int b0 = 0; b0 < NB; b0 += 256) {
            int32_t v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int b = b0 + u * 32 + lane;
                v[u] = b < NB ? row[b] : 0;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                int32_t inc = v[u];
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int32_t n = __shfl_up_sync(0xffffffffu, inc, o);
                    if (lane >= o) inc += n;
                }
                const int b = b0 + u * 32 + lane;
                if (b < NB) row[b] = carry + inc - v[u];
                carry += __shfl_sync(0xffffffffu, inc, 31);
            }
        }
        if (lane == 0) total[e] = carry;
    }
    __syncthreads();
    // exclusive scan of total[0..E) over the block (E <= 1024 = blockDim)
    const int e = threadIdx.x;
    const int32_t mine = e < E ? total[e] : 0;
    int32_t inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int32_t n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
    }
    if (lane == 31) warp_sum[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        int32_t w = warp_sum[lane], winc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int32_t n = __shfl_up_sync(0xffffffffu, winc, o);
            if (lane >= o) winc += n;
        }
        warp_sum[lane] = winc - w;
    }
    __syncthreads();
    const int32_t excl = warp_sum[warp] + inc - mine;
    if (e < E) {
        counts[e] = mine;
        offsets[e] = excl;
        if (e == E - 1) offsets[E] = excl + mine;
    }
}

template <typename IdxT>
__global__ void __launch_bounds__(kChunk)
permute_rank_kernel(const IdxT* __restrict__ idx, const int32_t* __restrict__ chunk_base,
                    const int32_t* __restrict__ offsets, int32_t* __restrict__ row_of_slot,
                    int32_t* __restrict__ slot_of_row, int T, int E, int K, int NB) {
    extern __shared__ uint32_t bits[];            // [E][kWords]
    for (int i = threadIdx.x; i < E * kWords; i += kChunk) bits[i] = 0u;
    __syncthreads();
    const int lt = threadIdx.x;
    const int t = blockIdx.x * kChunk + lt;
    const IdxT* rec = idx + (size_t)(t < T ? t : 0) * K;
    if (t < T) {
        for (int j = 0; j < K; ++j) {
            int e;
            if (pair_ok(rec, j, E, e, nullptr)) atomicOr(&bits[e * kWords + (lt >> 5)], 1u << (lt & 31));
        }
    }
    __syncthreads();
    if (t < T) {
        // slots in batches of 8: the (independent) table reads of a batch are issued together
        for (int j0 = 0; j0 < K; j0 += 8) {
            int32_t row[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int j = j0 + u;
                int e;
                row[u] = -1;
                if (j < K && pair_ok(rec, j, E, e, nullptr)) {
                    const uint32_t* m = bits + e * kWords;
                    int rank = __popc(m[lt >> 5] & ((1u << (lt & 31)) - 1u));
                    for (int w = 0; w < (lt >> 5); ++w) rank += __popc(m[w]);
                    row[u] = offsets[e] + chunk_base[(size_t)e * NB + blockIdx.x] + rank;
                }
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int j = j0 + u;
                if (j < K) {
                    if (row[u] >= 0) slot_of_row[row[u]] = t * K + j;
                    row_of_slot[(size_t)t * K + j] = row[u];
                }
            }
        }
    }
}

// The three steps above as ONE cooperative launch (all chunk CTAs resident, two grid-wide
// barriers): at a few thousand tokens the three separate launches cost more in launch and drain
// time than in work.  Same arithmetic, same results; used whenever all the chunk CTAs fit on the
// device at once.
//   step 1  per-chunk counts -> chunk_counts[e][chunk]
//   step 2  one warp per expert: exclusive scan along the chunks, total -> counts[e]
//   step 3  every CTA scans counts[] into the expert offsets (shared memory), CTA 0 writes them
//           out; then ranks and maps exactly as permute_rank_kernel
template <typename IdxT>
__global__ void __launch_bounds__(kChunk)
permute_maps_coop_kernel(const IdxT* __restrict__ idx, int32_t* chunk_counts, int32_t* counts,
                         int32_t* offsets, int32_t* __restrict__ row_of_slot,
                         int32_t* __restrict__ slot_of_row, int T, int E, int K, int NB,
                         int32_t* dev_status) {
    namespace cg = cooperative_groups;
    cg::grid_group grid = cg::this_grid();
    extern __shared__ int32_t sm[];
    int32_t* hist = sm;                                   // [E], later the expert offsets
    uint32_t* bits = reinterpret_cast<uint32_t*>(sm + E); // [E][kWords]
    __shared__ int32_t warp_sum[kChunk / 32];
    const int lt = threadIdx.x, lane = lt & 31, warp = lt >> 5;
    const int t = blockIdx.x * kChunk + lt;
    const IdxT* rec = idx + (size_t)(t < T ? t : 0) * K;

    // ---- step 1 -----------------------------------------------------------------------------
    for (int e = lt; e < E; e += kChunk) hist[e] = 0;
    for (int i = lt; i < E * kWords; i += kChunk) bits[i] = 0u;
    __syncthreads();
    if (t < T) {
        for (int j = 0; j < K; ++j) {
            int e;
            if (pair_ok(rec, j, E, e, dev_status)) {
                atomicAdd(&hist[e], 1);
                atomicOr(&bits[e * kWords + (lt >> 5)], 1u << (lt & 31));
            }
        }
    }
    __syncthreads();
    for (int e = lt; e < E; e += kChunk) chunk_counts[(size_t)e * NB + blockIdx.x] = hist[e];
    grid.sync();

    // ---- step 2 -----------------------------------------------------------------------------
    const int warps_total = gridDim.x * (kChunk / 32);
    for (int e = blockIdx.x * (kChunk / 32) + warp; e < E; e += warps_total) {
        int32_t* row = chunk_counts + (size_t)e * NB;
        int32_t carry = 0;
        for (int b0 = 0; b0 < NB; b0 += 32) {
            const int b = b0 + lane;
            const int32_t v = b < NB ? row[b] : 0;
            int32_t inc = v;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int32_t n = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += n;
            }
            if (b < NB) row[b] = carry + inc - v;
            carry += __shfl_sync(0xffffffffu, inc, 31);
        }
        if (lane == 0) counts[e] = carry;
    }
    grid.sync();

    // ---- step 3: offsets (each thread owns a run of experts), then ranks -----------------------
    const int per = (E + kChunk - 1) / kChunk;
    int32_t mine = 0;
    for (int i = 0; i < per; ++i) {
        const int e = lt * per + i;
        if (e < E) mine += counts[e];
    }
    int32_t inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int32_t n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
    }
    if (lane == 31) warp_sum[warp] = inc;
    __syncthreads();
    int32_t run = inc - mine;
    for (int w = 0; w < warp; ++w) run += warp_sum[w];
    for (int i = 0; i < per; ++i) {
        const int e = lt * per + i;
        if (e < E) {
            hist[e] = run;                                // exclusive offset of expert e
            if (blockIdx.x == 0) offsets[e] = run;
            run += counts[e];
            if (blockIdx.x == 0 && e == E - 1) offsets[E] = run;
        }
    }
    __syncthreads();
    if (t < T) {
        for (int j0 = 0; j0 < K; j0 += 8) {
            int32_t row[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int j = j0 + u;
                int e;
                row[u] = -1;
                if (j < K && pair_ok(rec, j, E, e, nullptr)) {
                    const uint32_t* m = bits + e * kWords;
                    int rank = __popc(m[lt >> 5] & ((1u << (lt & 31)) - 1u));
                    for (int w = 0; w < (lt >> 5); ++w) rank += __popc(m[w]);
                    row[u] = hist[e] + chunk_counts[(size_t)e * NB + blockIdx.x] + rank;
                }
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int j = j0 + u;
                if (j < K) {
                    if (row[u] >= 0) slot_of_row[row[u]] = t * K + j;
                    row_of_slot[(size_t)t * K + j] = row[u];
                }
            }
        }
    }
}

// The same maps for at most kClusterMax chunks, all in ONE thread-block cluster: the per-chunk
// counts stay in shared memory and are read across the cluster (distributed shared memory), and
// the two grid-wide syncs become hardware cluster barriers.  CTA b owns tokens [256 b, 256 b + 256);
// CTAs beyond the last chunk only take part in the barriers.
constexpr int kClusterMax = 16;
__device__ __forceinline__ void cluster_barrier() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\t"
                 "barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ int32_t ld_cluster_s32(const int32_t* own, uint32_t rank) {
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(own);
    uint32_t ra;
    int32_t v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(a), "r"(rank));
    asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(v) : "r"(ra) : "memory");
    return v;
}

template <typename IdxT>
__global__ void __launch_bounds__(kChunk)
permute_maps_cluster_kernel(const IdxT* __restrict__ idx, int32_t* __restrict__ counts,
                            int32_t* __restrict__ offsets, int32_t* __restrict__ row_of_slot,
                            int32_t* __restrict__ slot_of_row, int T, int E, int K,
                            int32_t* dev_status, WorkListSpec lists) {
    extern __shared__ int32_t sm[];
    int32_t* hist = sm;                                       // [E] this chunk's counts
    int32_t* total = sm + E;                                  // [E] all chunks
    int32_t* first = sm + 2 * E;                              // [E] first row of (expert, chunk)
    uint32_t* bits = reinterpret_cast<uint32_t*>(sm + 3 * E); // [E][kWords]
    int32_t* eoff = sm + (3 + kWords) * E;                    // [E + 1] expert offsets
    int32_t* s_items = eoff + E + 1;                          // [E + 1] scratch of the list builder
    __shared__ int32_t warp_sum[kChunk / 32];
    const int lt = threadIdx.x, lane = lt & 31, warp = lt >> 5;
    const int nb = gridDim.x, b = blockIdx.x;                 // one cluster: rank = blockIdx.x
    const int t = b * kChunk + lt;
    const IdxT* rec = idx + (size_t)(t < T ? t : 0) * K;

    for (int e = lt; e < E; e += kChunk) hist[e] = 0;
    for (int i = lt; i < E * kWords; i += kChunk) bits[i] = 0u;
    __syncthreads();
    // The wait comes first here: once this grid lets its dependent start, everything before it
    // in the stream has completed, so the row copy launched right behind it may fetch the token
    // rows (which this kernel does not write) before its own wait.
    tc::grid_dependency_wait();                    // the record may come from the kernel before
    tc::grid_launch_dependents();
    int kept[8];                                   // slots 0..7: the expert, or -1 for a dropped pair
#pragma unroll
    for (int u = 0; u < 8; ++u) kept[u] = -1;
    if (t < T) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            int e;
            if (u < K && pair_ok(rec, u, E, e, dev_status)) {
                kept[u] = e;
                atomicAdd(&hist[e], 1);
                atomicOr(&bits[e * kWords + (lt >> 5)], 1u << (lt & 31));
            }
        }
        for (int j = 8; j < K; ++j) {
            int e;
            if (pair_ok(rec, j, E, e, dev_status)) {
                atomicAdd(&hist[e], 1);
                atomicOr(&bits[e * kWords + (lt >> 5)], 1u << (lt & 31));
            }
        }
    }
    cluster_barrier();                      // every chunk's counts are final and visible

    for (int e = lt; e < E; e += kChunk) {
        int32_t v[kClusterMax];
#pragma unroll
        for (int c = 0; c < kClusterMax; ++c)                 // all loads in flight together
            v[c] = c < nb ? ld_cluster_s32(hist + e, (uint32_t)c) : 0;
        int32_t before = 0, all = 0;
#pragma unroll
        for (int c = 0; c < kClusterMax; ++c) {
            all += v[c];
            if (c < b) before += v[c];
        }
        total[e] = all;
        first[e] = before;
    }
    __syncthreads();
    cluster_barrier();                      // nobody reads this CTA's counts after this point

    // offsets: each thread owns a run of experts
    const int per = (E + kChunk - 1) / kChunk;
    int32_t mine = 0;
    for (int i = 0; i < per; ++i) {
        const int e = lt * per + i;
        if (e < E) mine += total[e];
    }
    int32_t inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int32_t n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
    }
    if (lane == 31) warp_sum[warp] = inc;
    __syncthreads();
    int32_t run = inc - mine;
    for (int w = 0; w < warp; ++w) run += warp_sum[w];
    for (int i = 0; i < per; ++i) {
        const int e = lt * per + i;
        if (e < E) {
            const int32_t cnt = total[e];
            first[e] += run;                               // expert offset + rows of earlier chunks
            eoff[e] = run;
            if (e == E - 1) eoff[E] = run + cnt;
            if (b == 0) {
                offsets[e] = run;
                counts[e] = cnt;
                if (e == E - 1) offsets[E] = run + cnt;
            }
            run += cnt;
        }
    }
    __syncthreads();
    if (t < T) {
        for (int j0 = 0; j0 < K; j0 += 8) {
            int32_t row[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int j = j0 + u;
                int e = kept[u];
                row[u] = -1;
                if (j < K && (j0 == 0 ? e >= 0 : pair_ok(rec, j, E, e, nullptr))) {
                    const uint32_t* m = bits + e * kWords;
                    int rank = __popc(m[lt >> 5] & ((1u << (lt & 31)) - 1u));
                    for (int w = 0; w < (lt >> 5); ++w) rank += __popc(m[w]);
                    row[u] = first[e] + rank;
                }
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int j = j0 + u;
                if (j < K) {
                    if (row[u] >= 0) slot_of_row[row[u]] = t * K + j;
                    row_of_slot[(size_t)t * K + j] = row[u];
                }
            }
        }
    }
    // The work lists of the expert GEMMs, when the caller wants them from this launch: the last
    // CTA builds the up-projection list, the one before it (if there is one) the other.
    if (lists.list0) {
        if (b == nb - 1) tc::build_work_list(eoff, E, lists.nf0, lists.list0, lists.pairs, s_items);
        if (b == (nb >= 2 ? nb - 2 : 0))
            tc::build_work_list(eoff, E, lists.nf1, lists.list1, lists.pairs, s_items);
    }
}

// One warp per token: read x[t] once (16-byte pieces), write it to the token's K rows.
template <int VEC_BYTES>
__global__ void __launch_bounds__(256)
permute_rows_kernel(const uint4* __restrict__ x, const int32_t* __restrict__ row_of_slot,
                    uint4* __restrict__ xp, int T, int K, int row_vecs) {
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (t >= T) return;
    const uint4* src = x + (size_t)t * row_vecs;
    const int32_t* rows = row_of_slot + (size_t)t * K;
    for (int c0 = 0; c0 < row_vecs; c0 += 128) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int c = c0 + u * 32 + lane;
            if (c < row_vecs) v[u] = src[c];
        }
        for (int j = 0; j < K; ++j) {
            const int32_t r = rows[j];
            if (r < 0) continue;
            uint4* dst = xp + (size_t)r * row_vecs;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int c = c0 + u * 32 + lane;
                if (c < row_vecs) dst[c] = v[u];
            }
        }
    }
}


// The same copy staged through shared memory with bulk asynchronous copies: a CTA of one warp
// takes kRowTokens tokens; lane i brings token i's row in (one copy, completion counted on an
// mbarrier) and, once it has landed, sends it to the token's K destination rows (one bulk store
// each).  Nothing passes through registers, each copy is a whole row, and seven CTAs per SM keep
// about 200 KB in flight.
constexpr int kRowTokens = 8;

__global__ void __launch_bounds__(32)
permute_rows_staged_kernel(const uint8_t* __restrict__ x, const int32_t* __restrict__ row_of_slot,
                           uint8_t* __restrict__ xp, int T, int K, uint32_t row_bytes,
                           int x_early, int32_t* dev_status) {
    extern __shared__ __align__(128) uint8_t smem_p[];
    const uint32_t bar = tc::smem_u32(smem_p);
    volatile int* flags = reinterpret_cast<volatile int*>(smem_p + 8);
    const uint32_t rows0 = tc::smem_u32(smem_p + 128);
    const int lane = threadIdx.x;
    const int t0 = blockIdx.x * kRowTokens;
    const int nt = min(kRowTokens, T - t0);
    if (lane == 0) {
        tc::mbar_init(bar, 1);
        flags[0] = 0;
        tc::fence_barrier_init();
        tc::mbar_expect_tx(bar, row_bytes * (uint32_t)nt);
    }
    __syncwarp();
    auto fetch_rows = [&]() {
        if (lane < nt)
            asm volatile(
                "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                ::"r"(rows0 + (uint32_t)lane * row_bytes), "l"(x + (size_t)(t0 + lane) * row_bytes),
                  "r"(row_bytes), "r"(bar) : "memory");
    };
    // x_early: the kernel before this one in the stream does not write x and lets this grid start
    // only after everything before IT has completed (the dispatch kernels), so the token rows are
    // fetched while the dispatch is still computing the maps.
    if (x_early) fetch_rows();
    tc::grid_launch_dependents();
    tc::grid_dependency_wait();            // the maps (and, unless x_early, x) come from before
    if (!x_early) fetch_rows();
    int32_t r[8];
    // destination rows of this lane's token, fetched while the copy flies; K > 8 goes in rounds
    const int32_t* rows = row_of_slot + (size_t)(t0 + (lane < nt ? lane : 0)) * K;
#pragma unroll
    for (int u = 0; u < 8; ++u) r[u] = (lane < nt && u < K) ? rows[u] : -1;
    // a wait that runs out leaves these tokens' rows unwritten and says so in dev_status
    const bool ok = __all_sync(0xffffffffu, tc::mbar_wait(bar, 0u, flags, dev_status));
    if (ok && lane < nt) {
        for (int j0 = 0; j0 < K; j0 += 8) {
            if (j0 > 0) {
#pragma unroll
                for (int u = 0; u < 8; ++u) r[u] = j0 + u < K ? rows[j0 + u] : -1;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u)
                if (r[u] >= 0)
                    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                                 ::"l"(xp + (size_t)r[u] * row_bytes),
                                   "r"(rows0 + (uint32_t)lane * row_bytes), "r"(row_bytes)
                                 : "memory");
        }
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        // shared memory must outlive the stores that read it
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
    }
    if (!ok) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    }
}

r3_status launch_permute_rows(const r3_shape* shape, const void* x, const int32_t* row_of_slot,
                              void* xp, cudaStream_t cs, int32_t* dev_status, bool x_early) {
    const int T = shape->T, K = shape->K;
    const size_t row_bytes = (size_t)shape->d * act_bytes(shape);
    if (row_bytes * kRowTokens <= 96 * 1024) {
        const size_t smem = 128 + row_bytes * kRowTokens;
        static PerDevice attr_set;
        if (!attr_set.done()) {
            if (cudaFuncSetAttribute(permute_rows_staged_kernel,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     128 + 96 * 1024) != cudaSuccess)
                return R3_ERR_CUDA;
            attr_set.mark();
        }
        if (tc::launch_dependent(permute_rows_staged_kernel, dim3((T + kRowTokens - 1) / kRowTokens),
                                 dim3(32), smem, cs, static_cast<const uint8_t*>(x), row_of_slot,
                                 static_cast<uint8_t*>(xp), T, K, (uint32_t)row_bytes,
                                 x_early ? 1 : 0, dev_status) != cudaSuccess)
            return R3_ERR_CUDA;
        return launch_status();
    }
    const int row_vecs = (int)(row_bytes / 16);
    const int wpb = 8;
    permute_rows_kernel<16><<<(T + wpb - 1) / wpb, wpb * 32, 0, cs>>>(
        static_cast<const uint4*>(x), row_of_slot, static_cast<uint4*>(xp), T, K, row_vecs);
    return launch_status();
}

}  // namespace r3

extern "C" size_t r3_permute_workspace_bytes(const r3_shape* shape) {
    if (r3::check_shape(shape) != R3_OK) return 0;
    const size_t NB = (shape->T + r3::kChunk - 1) / r3::kChunk;
    return r3::round_up((size_t)shape->E * (NB ? NB : 1) * sizeof(int32_t), 256);
}

// `lists` (may be null): the expert GEMMs' work lists are wanted from the dispatch launch itself;
// *lists_built tells whether this call could do that (only the one-cluster form does).
r3_status r3::permute_impl(const r3_shape* shape, const void* idx, const void* x, int32_t* counts,
                           int32_t* offsets, int32_t* row_of_slot, int32_t* slot_of_row, void* xp,
                           void* workspace, size_t ws_bytes, int32_t* dev_status, void* stream,
                           const WorkListSpec* lists, bool* lists_built) {
    if (lists_built) *lists_built = false;
    r3_status st = r3::check_shape(shape);
    if (st != R3_OK) return st;
    if (shape->E > r3::kMaxExpertsPermute) return R3_ERR_UNSUPPORTED;
    if (!counts || !offsets) return R3_ERR_INVALID_ARG;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (shape->T == 0) {
        // nothing to group: counts and offsets are still defined (all zero)
        if (cudaMemsetAsync(counts, 0, sizeof(int32_t) * shape->E, cs) != cudaSuccess ||
            cudaMemsetAsync(offsets, 0, sizeof(int32_t) * (shape->E + 1), cs) != cudaSuccess)
            return R3_ERR_CUDA;
        return R3_OK;
    }
    if (!idx || !row_of_slot || !slot_of_row) return R3_ERR_INVALID_ARG;
    if ((x == nullptr) != (xp == nullptr)) return R3_ERR_INVALID_ARG;
    if (x && (!r3::aligned(x, 16) || !r3::aligned(xp, 16))) return R3_ERR_INVALID_ARG;
    if (!workspace || ws_bytes < r3_permute_workspace_bytes(shape) || !r3::aligned(workspace, 256))
        return R3_ERR_WORKSPACE;

    const int T = shape->T, E = shape->E, K = shape->K;
    const int NB = (T + r3::kChunk - 1) / r3::kChunk;
    int32_t* chunk_counts = static_cast<int32_t*>(workspace);
    // up to 16 chunks: one thread-block cluster, counts exchanged through shared memory
    bool coop_done = false;
    if (NB <= r3::kClusterMax) {
        int cl = 1;
        while (cl < NB) cl <<= 1;
        const size_t smem = ((size_t)E * (5 + r3::kWords) + 2) * sizeof(int32_t);
        // per device, index type and cluster size: 0 = untested, 1 = ok, -1 = no
        static int usable_dev[64][2][r3::kClusterMax + 1] = {};
        int (*usable)[r3::kClusterMax + 1] = usable_dev[r3::PerDevice::current()];
        const int ti = shape->idx_type == R3_IDX_U8 ? 0 : 1;
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)cl;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.gridDim = dim3((unsigned)cl);
        cfg.blockDim = dim3(r3::kChunk);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = cs;
        cfg.attrs = attr;
        cfg.numAttrs = 2;
        if (usable[ti][cl] == 0) {
            usable[ti][cl] = -1;
            if (smem <= 200 * 1024) {
                cudaError_t a1 = cudaErrorUnknown, a2 = cudaErrorUnknown, q = cudaErrorUnknown;
                int n = 0;
                R3_DISPATCH_IDX(shape, IdxT, {
                    auto kern = r3::permute_maps_cluster_kernel<IdxT>;
                    a1 = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              200 * 1024);
                    a2 = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
                    q = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
                });
                if (a1 == cudaSuccess && a2 == cudaSuccess && q == cudaSuccess && n >= 1)
                    usable[ti][cl] = 1;
                else
                    cudaGetLastError();
            }
        }
        if (usable[ti][cl] == 1) {
            r3::WorkListSpec wl = {nullptr, nullptr, 0, 0, 0};
            if (lists && E <= 1024) wl = *lists;
            cudaError_t le = cudaErrorUnknown;
            R3_DISPATCH_IDX(shape, IdxT, le = cudaLaunchKernelEx(
                &cfg, r3::permute_maps_cluster_kernel<IdxT>, static_cast<const IdxT*>(idx), counts,
                offsets, row_of_slot, slot_of_row, T, E, K, dev_status, wl));
            if (le != cudaSuccess) return R3_ERR_CUDA;
            coop_done = true;
            if (lists_built && wl.list0) *lists_built = true;
        }
    }
    // one cooperative launch when all the chunk CTAs can be resident together
    if (!coop_done) {
        const size_t smem = (size_t)E * (1 + r3::kWords) * sizeof(int32_t);
        int per_sm = 0;
        cudaError_t qe = cudaErrorUnknown;
        R3_DISPATCH_IDX(shape, IdxT, qe = cudaOccupancyMaxActiveBlocksPerMultiprocessor(
            &per_sm, r3::permute_maps_coop_kernel<IdxT>, r3::kChunk, smem));
        if (qe == cudaSuccess && smem <= 48 * 1024 && (long long)per_sm * r3::sm_count() >= NB) {
            int Tn = T, En = E, Kn = K, NBn = NB;
            void* args[] = {(void*)&idx, (void*)&chunk_counts, (void*)&counts, (void*)&offsets,
                            (void*)&row_of_slot, (void*)&slot_of_row, (void*)&Tn, (void*)&En,
                            (void*)&Kn, (void*)&NBn, (void*)&dev_status};
            cudaError_t le = cudaErrorUnknown;
            R3_DISPATCH_IDX(shape, IdxT, le = cudaLaunchCooperativeKernel(
                (const void*)r3::permute_maps_coop_kernel<IdxT>, dim3(NB), dim3(r3::kChunk), args,
                smem, cs));
            if (le != cudaSuccess) return R3_ERR_CUDA;
            coop_done = true;
        } else {
            cudaGetLastError();
        }
    }
    if (!coop_done) {
    R3_DISPATCH_IDX(shape, IdxT,
        r3::permute_count_kernel<IdxT><<<NB, r3::kChunk, E * sizeof(int32_t), cs>>>(
            static_cast<const IdxT*>(idx), chunk_counts, T, E, K, NB, dev_status));
    r3::permute_scan_kernel<<<1, 1024, 0, cs>>>(chunk_counts, counts, offsets, E, NB);
    R3_DISPATCH_IDX(shape, IdxT,
        r3::permute_rank_kernel<IdxT><<<NB, r3::kChunk, E * r3::kWords * sizeof(uint32_t), cs>>>(
            static_cast<const IdxT*>(idx), chunk_counts, offsets, row_of_slot, slot_of_row,
            T, E, K, NB));
    }
    // The kernel in front of the row copy is one of the dispatch kernels above: none writes x,
    // the one-cluster form lets its dependent start only after its own wait and the others not
    // before they end, so everything earlier in the stream has completed when the row copy starts
    // and it may fetch the token rows before its wait.
    if (x) return r3::launch_permute_rows(shape, x, row_of_slot, xp, cs, dev_status, true);
    return r3::launch_status();
}

extern "C" r3_status r3_permute(const r3_shape* shape, const void* idx, const void* x,
                                int32_t* counts, int32_t* offsets, int32_t* row_of_slot,
                                int32_t* slot_of_row, void* xp, void* workspace, size_t ws_bytes,
                                int32_t* dev_status, void* stream) {
    return r3::permute_impl(shape, idx, x, counts, offsets, row_of_slot, slot_of_row, xp, workspace,
                            ws_bytes, dev_status, stream, nullptr, nullptr);
}

// ---------------------------------------------------------------------------------------------
// r3_permute_static: the same dispatch with its scratch in a fixed device array of this library.
//
// For callers that have no way to hand over scratch memory: a host whose device memory is owned
// entirely by another component's pool (asking the driver for more would fail, fragment the pool
// or stall the device, since a driver allocation synchronises it), or a step that must not touch
// the allocator because its memory budget was fixed up front.  They still pass inputs and outputs;
// only the [expert][chunk] counters live here.
//
// The array is part of the loaded library image: every GPU that loads the library carries these
// kStaticScratchInts * 4 bytes until the process exits.  All calls share it and it keeps whatever
// the last call left; nothing in it needs to start at zero because the counting kernel overwrites
// every counter the later kernels read.  Two calls that overlap on the GPU (different streams, or
// different host threads) would race on it.
// ---------------------------------------------------------------------------------------------
namespace r3 {
constexpr int kStaticScratchInts = 1 << 18;            // 1 MiB: E * ceil(T / 256) <= 262144
static __device__ __align__(256) int32_t g_permute_scratch[kStaticScratchInts];

// In host code the array's name only stands for the symbol; the device address has to be asked
// for, per device, with that device current.  Cached after the first call on each device.
static r3_status static_scratch_ptr(int32_t** out) {
    constexpr int kMaxDevices = 64;
    static int32_t* cached[kMaxDevices] = {nullptr};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return R3_ERR_CUDA;
    if (!cached[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_permute_scratch) != cudaSuccess || !p) return R3_ERR_CUDA;
        cached[dev] = static_cast<int32_t*>(p);
    }
    *out = cached[dev];
    return R3_OK;
}
}  // namespace r3

extern "C" r3_status r3_permute_static(const r3_shape* shape, const void* idx, const void* x,
                                       int32_t* counts, int32_t* offsets, int32_t* row_of_slot,
                                       int32_t* slot_of_row, void* xp, int32_t* dev_status,
                                       void* stream) {
    r3_status st = r3::check_shape(shape);
    if (st != R3_OK) return st;
    if (shape->E > r3::kMaxExpertsPermute) return R3_ERR_UNSUPPORTED;
    const long long NB = ((long long)shape->T + r3::kChunk - 1) / r3::kChunk;
    if ((long long)shape->E * NB > r3::kStaticScratchInts) return R3_ERR_SCRATCH_LIMIT;
    int32_t* scratch = nullptr;
    if ((st = r3::static_scratch_ptr(&scratch)) != R3_OK) return st;
    return r3_permute(shape, idx, x, counts, offsets, row_of_slot, slot_of_row, xp, scratch,
                      sizeof(int32_t) * r3::kStaticScratchInts, dev_status, stream);
}
