// Expert-parallel bookkeeping around the replayed layer (an extension: the paper describes no
// parallelism).  With the experts split over N ranks, every rank groups its (token, slot) rows by
// global expert as usual; the rows bound for one rank are then one contiguous block, and after an
// all-to-all a rank holds the blocks of all sources one after the other: [source][local expert]
// [row].  The grouped expert GEMM wants [local expert][source][row].  The two kernels here build
// that reordering from the table of received row counts and apply it (and its inverse, for the
// way back) - index work, bit-exact.
#include "r3_common.cuh"

namespace r3 {

constexpr int kEpMaxSegments = 4096;     // sources x local experts

// One CTA.  recv_counts [n_src][el] -> perm [rows] (position in [expert][source][row] order ->
// arrival index), offsets [el + 1].  `rows_expected` is checked against the table.
__global__ void __launch_bounds__(1024)
ep_regroup_map_kernel(const int32_t* __restrict__ recv_counts, int n_src, int el,
                      int rows_expected, int32_t* __restrict__ perm,
                      int32_t* __restrict__ offsets, int32_t* dev_status) {
    __shared__ int32_t arrive_start[kEpMaxSegments];   // by arrival id  s * el + k
    __shared__ int32_t place_start[kEpMaxSegments];    // by placed id   k * n_src + s
    __shared__ int32_t total_s;
    const int tid = threadIdx.x, nseg = n_src * el;
    // two exclusive scans of the same counts in two orders; the table is small, one thread each
    if (tid == 0) {
        int32_t run = 0;
        for (int a = 0; a < nseg; ++a) {
            arrive_start[a] = run;
            run += max(recv_counts[a], 0);
        }
        total_s = run;
    } else if (tid == 32) {
        int32_t run = 0;
        for (int k = 0; k < el; ++k) {
            offsets[k] = run;
            for (int s = 0; s < n_src; ++s) {
                place_start[k * n_src + s] = run;
                run += max(recv_counts[s * el + k], 0);
            }
        }
        offsets[el] = run;
    }
    __syncthreads();
    if (total_s != rows_expected) {
        if (tid == 0) report(dev_status, R3_DEV_BAD_INDEX);
        return;
    }
    const int warp = tid >> 5, lane = tid & 31;
    for (int b = warp; b < nseg; b += 32) {
        const int k = b / n_src, s = b - k * n_src;
        const int cnt = max(recv_counts[s * el + k], 0);
        const int32_t from = arrive_start[s * el + k], to = place_start[b];
        for (int i = lane; i < cnt; i += 32) perm[to + i] = from + i;
    }
}

// One warp per row: forward dst[j] = src[perm[j]], inverse dst[perm[j]] = src[j].
__global__ void __launch_bounds__(256)
ep_move_rows_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst,
                    const int32_t* __restrict__ perm, int rows, int row_vecs, int inverse) {
    const int lane = threadIdx.x & 31;
    const int j = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (j >= rows) return;
    const int p = perm[j];
    if (p < 0 || p >= rows) return;
    const uint4* from = src + (size_t)(inverse ? j : p) * row_vecs;
    uint4* to = dst + (size_t)(inverse ? p : j) * row_vecs;
    for (int c = lane; c < row_vecs; c += 32) to[c] = from[c];
}

}  // namespace r3

namespace r3 {

constexpr int kEpMaxRanks = 64;
struct EpPeers {
    unsigned long long base[kEpMaxRanks];   // one buffer address per rank
};

// One CTA.  counts_all [n][E] = rows of every expert on every rank (after an all-gather).  For
// rank `me`:  dst_base[e] = row, in the owner's [local expert][source][row] buffer, of this
// rank's first row of expert e;  offsets_local [el + 1] = first row of each of this rank's own
// experts in that buffer (what the grouped GEMM of this rank takes).
__global__ void __launch_bounds__(1024)
ep_dest_table_kernel(const int32_t* __restrict__ counts_all, int n, int E, int me,
                     int32_t* __restrict__ dst_base, int32_t* __restrict__ offsets_local) {
    const int el = E / n;
    for (int e = threadIdx.x; e < E; e += blockDim.x) {
        const int q = e / el, k = e - q * el;
        int32_t before = 0;                       // rows of the owner's earlier experts, all sources
        for (int k2 = 0; k2 < k; ++k2)
            for (int s = 0; s < n; ++s) before += counts_all[s * E + q * el + k2];
        int32_t mine = before;
        for (int s = 0; s < me; ++s) mine += counts_all[s * E + e];
        dst_base[e] = mine;
        if (q == me) {
            offsets_local[k] = before;
            if (k == el - 1) {
                int32_t total = before;
                for (int s = 0; s < n; ++s) total += counts_all[s * E + e];
                offsets_local[el] = total;
            }
        }
    }
}

// One warp per token: x[t] goes straight to its K places in the owners' expert-major buffers.
template <typename IdxT>
__global__ void __launch_bounds__(256)
ep_dispatch_rows_kernel(const uint4* __restrict__ x, const IdxT* __restrict__ idx,
                        const int32_t* __restrict__ row_of_slot,
                        const int32_t* __restrict__ my_offsets,
                        const int32_t* __restrict__ dst_base, const __grid_constant__ EpPeers peers,
                        int T, int E, int K, int el, int row_vecs, long long capacity_rows,
                        int32_t* dev_status) {
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (t >= T) return;
    const uint4* src = x + (size_t)t * row_vecs;
    for (int j = 0; j < K; ++j) {
        const int32_t r = row_of_slot[(size_t)t * K + j];
        if (r < 0) continue;
        const int e = idx_to_int(idx[(size_t)t * K + j]);
        const size_t row = (size_t)dst_base[e] + (size_t)(r - my_offsets[e]);
        if ((long long)row >= capacity_rows) {        // beyond the owner's buffer: never stored
            if (lane == 0) report(dev_status, R3_DEV_BAD_INDEX);
            continue;
        }
        uint4* dst = reinterpret_cast<uint4*>(peers.base[e / el]) + row * row_vecs;
        for (int c = lane; c < row_vecs; c += 32) dst[c] = src[c];
    }
}

// Address of the expert-output row of every (token, slot) pair in the owners' output buffers.
template <typename IdxT>
__global__ void __launch_bounds__(256)
ep_slot_rows_kernel(const IdxT* __restrict__ idx, const int32_t* __restrict__ row_of_slot,
                    const int32_t* __restrict__ my_offsets, const int32_t* __restrict__ dst_base,
                    const __grid_constant__ EpPeers peers, unsigned long long* __restrict__ row_ptr,
                    long long pairs, int el, unsigned long long row_bytes, long long capacity_rows,
                    int32_t* dev_status) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= pairs) return;
    const int32_t r = row_of_slot[i];
    unsigned long long p = 0;
    if (r >= 0) {
        const int e = idx_to_int(idx[i]);
        const unsigned long long row = (unsigned long long)dst_base[e] + (r - my_offsets[e]);
        if ((long long)row < capacity_rows)
            p = peers.base[e / el] + row * row_bytes;
        else
            report(dev_status, R3_DEV_BAD_INDEX);     // beyond the owner's buffer: no address
    }
    row_ptr[i] = p;
}

}  // namespace r3

extern "C" r3_status r3_ep_dest_table(const int32_t* counts_all, int32_t n_ranks, int32_t E,
                                      int32_t rank, int32_t* dst_base, int32_t* offsets_local,
                                      void* stream) {
    if (n_ranks <= 0 || n_ranks > r3::kEpMaxRanks || E <= 0 || E % n_ranks || rank < 0 ||
        rank >= n_ranks || !counts_all || !dst_base || !offsets_local)
        return R3_ERR_INVALID_ARG;
    r3::ep_dest_table_kernel<<<1, 1024, 0, static_cast<cudaStream_t>(stream)>>>(
        counts_all, n_ranks, E, rank, dst_base, offsets_local);
    return r3::launch_status();
}

extern "C" r3_status r3_ep_dispatch_rows(const r3_shape* shape, int32_t n_ranks, const void* x,
                                         const void* idx, const int32_t* row_of_slot,
                                         const int32_t* my_offsets, const int32_t* dst_base,
                                         const unsigned long long* peer_buffers_host,
                                         int64_t capacity_rows, int32_t* dev_status,
                                         void* stream) {
    r3_status st = r3::check_shape(shape);
    if (st != R3_OK) return st;
    if (n_ranks <= 0 || n_ranks > r3::kEpMaxRanks || shape->E % n_ranks || capacity_rows < 0)
        return R3_ERR_INVALID_ARG;
    if (shape->T == 0) return R3_OK;
    if (!x || !idx || !row_of_slot || !my_offsets || !dst_base || !peer_buffers_host ||
        !r3::aligned(x, 16))
        return R3_ERR_INVALID_ARG;
    r3::EpPeers peers = {};
    for (int q = 0; q < n_ranks; ++q) {
        if (!peer_buffers_host[q] || (peer_buffers_host[q] & 15)) return R3_ERR_INVALID_ARG;
        peers.base[q] = peer_buffers_host[q];
    }
    const int row_vecs = (int)((size_t)shape->d * r3::act_bytes(shape) / 16);
    const int wpb = 8;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    R3_DISPATCH_IDX(shape, IdxT,
        r3::ep_dispatch_rows_kernel<IdxT><<<(shape->T + wpb - 1) / wpb, wpb * 32, 0, cs>>>(
            static_cast<const uint4*>(x), static_cast<const IdxT*>(idx), row_of_slot, my_offsets,
            dst_base, peers, shape->T, shape->E, shape->K, shape->E / n_ranks, row_vecs,
            (long long)capacity_rows, dev_status));
    return r3::launch_status();
}

extern "C" r3_status r3_ep_slot_rows(const r3_shape* shape, int32_t n_ranks, const void* idx,
                                     const int32_t* row_of_slot, const int32_t* my_offsets,
                                     const int32_t* dst_base,
                                     const unsigned long long* peer_buffers_host,
                                     int64_t capacity_rows, unsigned long long* row_ptr,
                                     int32_t* dev_status, void* stream) {
    r3_status st = r3::check_shape(shape);
    if (st != R3_OK) return st;
    if (n_ranks <= 0 || n_ranks > r3::kEpMaxRanks || shape->E % n_ranks || capacity_rows < 0)
        return R3_ERR_INVALID_ARG;
    if (shape->T == 0) return R3_OK;
    if (!idx || !row_of_slot || !my_offsets || !dst_base || !peer_buffers_host || !row_ptr)
        return R3_ERR_INVALID_ARG;
    r3::EpPeers peers = {};
    for (int q = 0; q < n_ranks; ++q) {
        if (!peer_buffers_host[q] || (peer_buffers_host[q] & 15)) return R3_ERR_INVALID_ARG;
        peers.base[q] = peer_buffers_host[q];
    }
    const long long pairs = (long long)shape->T * shape->K;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    R3_DISPATCH_IDX(shape, IdxT,
        r3::ep_slot_rows_kernel<IdxT><<<(unsigned)((pairs + 255) / 256), 256, 0, cs>>>(
            static_cast<const IdxT*>(idx), row_of_slot, my_offsets, dst_base, peers, row_ptr, pairs,
            shape->E / n_ranks, (unsigned long long)shape->d * r3::act_bytes(shape),
            (long long)capacity_rows, dev_status));
    return r3::launch_status();
}

extern "C" r3_status r3_ep_regroup_map(const int32_t* recv_counts, int32_t n_src, int32_t e_local,
                                       int32_t rows, int32_t* perm, int32_t* offsets,
                                       int32_t* dev_status, void* stream) {
    if (n_src <= 0 || e_local <= 0 || rows < 0) return R3_ERR_INVALID_ARG;
    if ((long long)n_src * e_local > r3::kEpMaxSegments) return R3_ERR_UNSUPPORTED;
    if (!recv_counts || !offsets || (rows > 0 && !perm)) return R3_ERR_INVALID_ARG;
    r3::ep_regroup_map_kernel<<<1, 1024, 0, static_cast<cudaStream_t>(stream)>>>(
        recv_counts, n_src, e_local, rows, perm, offsets, dev_status);
    return r3::launch_status();
}

extern "C" r3_status r3_ep_move_rows(const void* src, void* dst, const int32_t* perm,
                                     int32_t rows, size_t row_bytes, int32_t inverse,
                                     void* stream) {
    if (rows < 0 || row_bytes == 0 || (row_bytes % 16) != 0) return R3_ERR_INVALID_ARG;
    if (rows == 0) return R3_OK;
    if (!src || !dst || !perm || src == dst) return R3_ERR_INVALID_ARG;
    if (!r3::aligned(src, 16) || !r3::aligned(dst, 16)) return R3_ERR_INVALID_ARG;
    const int wpb = 8;
    r3::ep_move_rows_kernel<<<(rows + wpb - 1) / wpb, wpb * 32, 0,
                              static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4*>(src), static_cast<uint4*>(dst), perm, rows,
        (int)(row_bytes / 16), inverse ? 1 : 0);
    return r3::launch_status();
}
