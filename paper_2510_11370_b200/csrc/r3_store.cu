// Routing-record store (Section 4.2 of the paper: router masks cached with the prefix KV cache and
// reused across turns).  Records live in fixed-size pages of `page_tokens` tokens, laid out
// [page][layer][token in page][slot]; a sequence is a list of page numbers (its block table), and
// a shared prefix is two sequences listing the same pages.
//   r3_record_append   inference side: the records of newly decoded / prefilled tokens go into the
//                      pages of their sequences
//   r3_record_gather   training side: the packed [layer][token][slot] record of a variable-length
//                      batch is assembled from the pages
//   r3_pagepool_*      host-side page bookkeeping: free list, use counts, and the index from a
//                      token prefix to the page that holds its records
// The device side copies bytes (bit-exact); the host side allocates host memory only.
#include <cstring>
#include <unordered_map>
#include <vector>

#include "r3_common.cuh"
#include "r3_internal.h"

namespace r3 {

// Sequence of packed token n: the b with cu[b] <= n < cu[b+1] (empty sequences are skipped).
__device__ __forceinline__ int seq_of(const int32_t* __restrict__ cu, int B, int n) {
    int lo = 0, hi = B;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (cu[mid] <= n) lo = mid; else hi = mid;
    }
    return lo;
}

template <int RB>     // record bytes per (layer, token): K * sizeof(index); 0 = any
__device__ __forceinline__ void copy_record(uint8_t* dst, const uint8_t* src, int rb) {
    if (RB == 8) {
        *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(src);
    } else if (RB == 16) {
        *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
    } else {
        for (int i = 0; i < rb; ++i) dst[i] = src[i];
    }
}

// APPEND: packed [L, N, rb] -> pages.  !APPEND: pages -> packed [L, N, rb].
// One thread per token: it finds the token's page once and moves the records of all layers (for a
// fixed layer a warp touches 32 consecutive records of the packed array and whole runs of a page).
template <int RB, bool APPEND>
__global__ void __launch_bounds__(256)
record_move_kernel(uint8_t* __restrict__ pages, uint8_t* __restrict__ packed,
                   const int32_t* __restrict__ block_table, int max_pages,
                   const int32_t* __restrict__ pos0, const int32_t* __restrict__ cu, int B, int N,
                   int L, int page_tokens, int n_pages, int rb, int32_t* dev_status) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= N) return;
    const int b = seq_of(cu, B, n);
    const int pos = (pos0 ? pos0[b] : 0) + (n - cu[b]);
    const int slot = pos / page_tokens;
    const int page = slot < max_pages ? block_table[(size_t)b * max_pages + slot] : -1;
    if (page < 0 || page >= n_pages) {
        report(dev_status, R3_DEV_BAD_INDEX);       // no such page: the records are skipped
        return;
    }
    uint8_t* in_page = pages + ((size_t)page * L * page_tokens + pos % page_tokens) * rb;
    uint8_t* in_pack = packed + (size_t)n * rb;
    const size_t page_step = (size_t)page_tokens * rb, pack_step = (size_t)N * rb;
#pragma unroll 8                 // 8 records in flight per thread: 4 gave 0.63, 16 gave 0.51 of the copy bandwidth
    for (int l = 0; l < L; ++l) {
        if (APPEND) copy_record<RB>(in_page + l * page_step, in_pack + l * pack_step, rb);
        else copy_record<RB>(in_pack + l * pack_step, in_page + l * page_step, rb);
    }
}

template <bool APPEND>
static r3_status launch_move(const r3_shape* s, int L, int page_tokens, int n_pages, void* pages,
                             const int32_t* block_table, int max_pages, const int32_t* pos0,
                             const int32_t* cu, int B, void* packed, int N, int32_t* dev_status,
                             cudaStream_t cs) {
    const int rb = s->K * (int)idx_bytes(s);
    const unsigned grid = (unsigned)((N + 255) / 256);
    uint8_t* pg = static_cast<uint8_t*>(pages);
    uint8_t* pk = static_cast<uint8_t*>(packed);
    const bool a8 = rb == 8 && aligned(pages, 8) && aligned(packed, 8);
    const bool a16 = rb == 16 && aligned(pages, 16) && aligned(packed, 16);
    if (a8)
        record_move_kernel<8, APPEND><<<grid, 256, 0, cs>>>(pg, pk, block_table, max_pages, pos0, cu,
                                                            B, N, L, page_tokens, n_pages, rb,
                                                            dev_status);
    else if (a16)
        record_move_kernel<16, APPEND><<<grid, 256, 0, cs>>>(pg, pk, block_table, max_pages, pos0,
                                                             cu, B, N, L, page_tokens, n_pages, rb,
                                                             dev_status);
    else
        record_move_kernel<0, APPEND><<<grid, 256, 0, cs>>>(pg, pk, block_table, max_pages, pos0, cu,
                                                            B, N, L, page_tokens, n_pages, rb,
                                                            dev_status);
    return launch_status();
}

static r3_status check_move(const r3_shape* s, int L, int page_tokens, int n_pages, int max_pages,
                            int B, int N) {
    r3_status st = check_shape(s);
    if (st != R3_OK) return st;
    if (L <= 0 || page_tokens <= 0 || n_pages <= 0 || max_pages <= 0 || B < 0 || N < 0)
        return R3_ERR_INVALID_ARG;
    return R3_OK;
}

}  // namespace r3

extern "C" size_t r3_record_page_bytes(const r3_shape* shape, int32_t L, int32_t page_tokens) {
    if (r3::check_shape(shape) != R3_OK || L <= 0 || page_tokens <= 0) return 0;
    return (size_t)L * page_tokens * shape->K * r3::idx_bytes(shape);
}

extern "C" r3_status r3_record_append(const r3_shape* shape, int32_t L, int32_t page_tokens,
                                      int32_t n_pages, void* pages, const int32_t* block_table,
                                      int32_t max_pages, const int32_t* seq_pos0,
                                      const int32_t* cu_new, int32_t B, const void* rec_new,
                                      int32_t N, int32_t* dev_status, void* stream) {
    r3_status st = r3::check_move(shape, L, page_tokens, n_pages, max_pages, B, N);
    if (st != R3_OK) return st;
    if (B == 0 || N == 0) return R3_OK;
    if (!pages || !block_table || !seq_pos0 || !cu_new || !rec_new) return R3_ERR_INVALID_ARG;
    return r3::launch_move<true>(shape, L, page_tokens, n_pages, pages, block_table, max_pages,
                                 seq_pos0, cu_new, B, const_cast<void*>(rec_new), N, dev_status,
                                 static_cast<cudaStream_t>(stream));
}

extern "C" r3_status r3_record_gather(const r3_shape* shape, int32_t L, int32_t page_tokens,
                                      int32_t n_pages, const void* pages,
                                      const int32_t* block_table, int32_t max_pages,
                                      const int32_t* cu_seqlens, int32_t B, void* out, int32_t T,
                                      int32_t* dev_status, void* stream) {
    r3_status st = r3::check_move(shape, L, page_tokens, n_pages, max_pages, B, T);
    if (st != R3_OK) return st;
    if (B == 0 || T == 0) return R3_OK;
    if (!pages || !block_table || !cu_seqlens || !out) return R3_ERR_INVALID_ARG;
    return r3::launch_move<false>(shape, L, page_tokens, n_pages, const_cast<void*>(pages),
                                  block_table, max_pages, nullptr, cu_seqlens, B, out, T,
                                  dev_status, static_cast<cudaStream_t>(stream));
}

// ---- host-side page bookkeeping ---------------------------------------------------------------
// A page of the index is identified by the chained 64-bit hash of every token id up to its end
// (hash of the previous page's hash and its own ids); a lookup also compares the page's own ids
// and the previous hash, so a false match needs a collision of the 64-bit chain.
struct r3_pagepool {
    int page_tokens = 0;
    std::vector<int32_t> free_list;                 // free_list[head..) = pages not in use
    size_t head = 0;
    std::vector<int32_t> use;                       // use count per page
    std::vector<uint8_t> indexed;                   // page is in the index
    std::vector<uint64_t> chain, prev_chain;        // hash up to the page's end / its start
    std::vector<int32_t> tokens;                    // [n_pages][page_tokens] ids of indexed pages
    std::unordered_multimap<uint64_t, int32_t> index;   // chain hash -> page

    uint64_t extend(uint64_t h, const int32_t* tok) const {
        for (int i = 0; i < page_tokens; ++i) {
            h ^= (uint64_t)(uint32_t)tok[i] + 0x9E3779B97F4A7C15ull + (h << 6) + (h >> 2);
            h *= 0xBF58476D1CE4E5B9ull;
            h ^= h >> 31;
        }
        return h;
    }
    int32_t find(uint64_t prev, uint64_t now, const int32_t* tok) const {
        auto range = index.equal_range(now);
        for (auto it = range.first; it != range.second; ++it) {
            const int32_t p = it->second;
            if (prev_chain[p] == prev &&
                std::memcmp(&tokens[(size_t)p * page_tokens], tok, sizeof(int32_t) * page_tokens) == 0)
                return p;
        }
        return -1;
    }
    void unindex(int32_t p) {
        if (!indexed[p]) return;
        auto range = index.equal_range(chain[p]);
        for (auto it = range.first; it != range.second; ++it)
            if (it->second == p) { index.erase(it); break; }
        indexed[p] = 0;
    }
};

constexpr uint64_t kChainSeed = 0x243F6A8885A308D3ull;

extern "C" r3_pagepool* r3_pagepool_create(int32_t n_pages, int32_t page_tokens) {
    if (n_pages <= 0 || page_tokens <= 0) return nullptr;
    r3_pagepool* pool = new (std::nothrow) r3_pagepool();
    if (!pool) return nullptr;
    pool->page_tokens = page_tokens;
    pool->free_list.resize(n_pages);
    for (int32_t i = 0; i < n_pages; ++i) pool->free_list[i] = i;
    pool->use.assign(n_pages, 0);
    pool->indexed.assign(n_pages, 0);
    pool->chain.assign(n_pages, 0);
    pool->prev_chain.assign(n_pages, 0);
    pool->tokens.assign((size_t)n_pages * page_tokens, 0);
    return pool;
}

extern "C" void r3_pagepool_destroy(r3_pagepool* pool) { delete pool; }

extern "C" int32_t r3_pagepool_free_pages(const r3_pagepool* pool) {
    return pool ? (int32_t)(pool->free_list.size() - pool->head) : 0;
}

extern "C" int32_t r3_pagepool_match(r3_pagepool* pool, const int32_t* token_ids, int32_t n_tokens,
                                     int32_t* pages_out, int32_t max_pages) {
    if (!pool || !token_ids || !pages_out || n_tokens < 0) return 0;
    int32_t matched = 0;
    uint64_t h = kChainSeed;
    while (matched < max_pages && (matched + 1) * pool->page_tokens <= n_tokens) {
        const int32_t* tok = token_ids + (size_t)matched * pool->page_tokens;
        const uint64_t now = pool->extend(h, tok);
        const int32_t p = pool->find(h, now, tok);
        if (p < 0) break;
        pages_out[matched++] = p;
        h = now;
    }
    for (int32_t i = 0; i < matched; ++i) ++pool->use[pages_out[i]];
    return matched;
}

extern "C" r3_status r3_pagepool_alloc(r3_pagepool* pool, int32_t n, int32_t* pages_out) {
    if (!pool || n < 0 || (n > 0 && !pages_out)) return R3_ERR_INVALID_ARG;
    if ((size_t)n > pool->free_list.size() - pool->head) return R3_ERR_OUT_OF_PAGES;
    for (int32_t i = 0; i < n; ++i) {
        const int32_t p = pool->free_list[pool->head++];
        pool->use[p] = 1;
        pages_out[i] = p;
    }
    if (pool->head > 4096 && pool->head * 2 > pool->free_list.size()) {   // compact now and then
        pool->free_list.erase(pool->free_list.begin(), pool->free_list.begin() + pool->head);
        pool->head = 0;
    }
    return R3_OK;
}

extern "C" r3_status r3_pagepool_publish(r3_pagepool* pool, const int32_t* token_ids,
                                         int32_t n_tokens, const int32_t* table, int32_t n_table) {
    if (!pool || !token_ids || !table || n_tokens < 0 || n_table < 0) return R3_ERR_INVALID_ARG;
    const int32_t n_pages = (int32_t)pool->use.size();
    uint64_t h = kChainSeed;
    for (int32_t i = 0; i < n_table && (i + 1) * pool->page_tokens <= n_tokens; ++i) {
        const int32_t p = table[i];
        if (p < 0 || p >= n_pages || pool->use[p] <= 0) return R3_ERR_INVALID_ARG;
        const int32_t* tok = token_ids + (size_t)i * pool->page_tokens;
        const uint64_t now = pool->extend(h, tok);
        // a prefix is indexed once: a second page with the same content stays private
        if (!pool->indexed[p] && pool->find(h, now, tok) < 0) {
            pool->indexed[p] = 1;
            pool->chain[p] = now;
            pool->prev_chain[p] = h;
            std::memcpy(&pool->tokens[(size_t)p * pool->page_tokens], tok,
                        sizeof(int32_t) * pool->page_tokens);
            pool->index.emplace(now, p);
        }
        h = now;
    }
    return R3_OK;
}

extern "C" r3_status r3_pagepool_release(r3_pagepool* pool, const int32_t* table, int32_t n) {
    if (!pool || n < 0 || (n > 0 && !table)) return R3_ERR_INVALID_ARG;
    const int32_t n_pages = (int32_t)pool->use.size();
    for (int32_t i = 0; i < n; ++i)
        if (table[i] < 0 || table[i] >= n_pages || pool->use[table[i]] <= 0)
            return R3_ERR_INVALID_ARG;
    for (int32_t i = 0; i < n; ++i) {
        const int32_t p = table[i];
        if (--pool->use[p] == 0) {
            pool->unindex(p);
            pool->free_list.push_back(p);
        }
    }
    return R3_OK;
}
