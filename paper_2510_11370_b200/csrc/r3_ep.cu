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
