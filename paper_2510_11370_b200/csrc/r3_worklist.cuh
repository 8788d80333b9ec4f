// Work lists of the tensor-core grouped GEMMs (csrc/r3_swiglu_tc.cu): layout, the cut of an
// expert's rows into token tiles, and the routine that builds a list with the threads of one CTA.
// Shared by the list kernel of the GEMM file and by the dispatch kernel, which builds the lists at
// its end when the layer asks for them (one launch fewer in front of the GEMMs).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace r3 {
namespace tc {

constexpr int BNT = 256;           // most token rows per item (UMMA N)
// Per list: int32 header[kHeaderInts] = {number of items, claim counter, clusters finished, 0},
// then one int4 per item = {expert | feature tile << 16, first row, N (multiple of 16),
// valid rows}, ordered (expert, feature tile, token tile).  An expert with cnt rows is cut into
// nt = ceil(cnt / 256) token tiles of equal size q (rounded up to 16; the last one holds what is
// left).
constexpr int kHeaderInts = 4;
constexpr int STATIC_ITEMS = 3;    // items per cluster taken by position, the rest by the counter

__host__ __device__ inline int split_tiles(int cnt) { return (cnt + BNT - 1) / BNT; }
__host__ __device__ inline int split_rows(int cnt, int nt) {      // rows per tile, multiple of 16
    return (((cnt + nt - 1) / nt) + 15) & ~15;
}

// Builds one list from the row offsets [E + 1] of the experts (shared or global memory) for nf
// feature tiles.  Called by every thread of the CTA (it synchronises the CTA); s_items is shared
// scratch of E + 1 words; E <= 1024.
__device__ inline void build_work_list(const int32_t* offsets, int E, int nf, int32_t* list,
                                       int pairs, int32_t* s_items) {
    const int tid = threadIdx.x, nthr = blockDim.x;
    for (int e = tid; e < E; e += nthr)
        s_items[e + 1] = split_tiles(offsets[e + 1] - offsets[e]) * nf;
    if (tid == 0) s_items[0] = 0;
    __syncthreads();
    if (tid < 32) {                                   // s_items[e] = items of the experts before e
        const int per = (E + 31) / 32;
        const int lo = min(E, tid * per), hi = min(E, lo + per);
        int32_t sum = 0;
        for (int e = lo; e < hi; ++e) sum += s_items[e + 1];
        int32_t inc = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int32_t a = __shfl_up_sync(0xffffffffu, inc, o);
            if (tid >= o) inc += a;
        }
        int32_t run = inc - sum;
        for (int e = lo; e < hi; ++e) {
            run += s_items[e + 1];
            s_items[e + 1] = run;
        }
    }
    __syncthreads();
    const int32_t I = s_items[E];
    if (tid == 0) {
        list[0] = I;
        list[1] = STATIC_ITEMS * pairs;               // first item handed out by the counter
        list[2] = 0;
    }
    int4* items = reinterpret_cast<int4*>(list + kHeaderInts);
    for (int32_t i = tid; i < I; i += nthr) {
        int lo = 0, hi = E;                           // last e with s_items[e] <= i
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (s_items[mid] <= i) lo = mid; else hi = mid;
        }
        const int e = lo;
        const int row_lo = offsets[e], cnt = offsets[e + 1] - row_lo;
        const int nt = split_tiles(cnt), q = split_rows(cnt, nt);
        const int k = i - s_items[e];
        const int f = k / nt, j = k - f * nt;
        const int valid = min(q, cnt - j * q);
        items[i] = make_int4(e | (f << 16), row_lo + j * q, (valid + 15) & ~15, valid);
    }
    __syncthreads();
}

}  // namespace tc
}  // namespace r3
