// Receive and send schedules (arXiv 2205.10072, Algorithms 2-5 and the lookup of Algorithm 9):
// kernels and the entry points bcs_build, bcs_build_to_host, bcs_build_batch.
//
// Two constructions, bit-identical in their results:
//
//  * workspace path (three kernels).  codes_kernel writes the skip code (bcs_common.cuh) of every
//    rank x of a p once.  recv_codes_kernel then reads, per rank r and round i, the codes of the
//    two ranks that bound the window of Algorithm 4 (r - skips[i+1], r - skips[i]; consecutive
//    threads read consecutive words) and finds the largest new block of the window from the two
//    codes alone: walking down from the first level where they differ, every step yields one
//    "head" (a rank whose baseblock is that level) and a run of low blocks.  It writes the rows
//    rank-major and a round-major copy from which send_rm_kernel reads
//    sendsched[r][k] = recvsched[(r+skips[k]) mod p][k] with unit stride.
//
//  * self-contained path (no workspace).  One thread per rank runs Algorithm 4 with the range
//    search done by descending the homeranges; the send schedule is looked up in the rank-major
//    receive table where the to-processor is inside the call's range and recomputed
//    (Algorithm 5) where it is not.
#include <mutex>

#include "bcs_common.cuh"

namespace bcs {
namespace {

// Scratch of bcs_build_static: lives in the library's device image, so every GPU that loads
// the library sets these bytes aside until the process ends.  In host code this name is only a
// handle for cudaGetSymbolAddress, never an address a kernel may be given.
static __device__ __align__(256) unsigned char g_static_scratch[BCS_STATIC_WORKSPACE_BYTES];

// ================================================================ self-contained path
// Algorithm 2: peel off the head of the homerange until r is a skip itself.
__device__ __forceinline__ int base_block(const uint32_t *s, uint32_t r)
{
    for (;;) {
        int k = home_of(s, r);
        uint32_t v = s[k];
        if (r == v) return k;
        r -= v;
    }
}

// Baseblocks of the ranks a..b (1 <= a, b < p; empty when a > b) as a bit set: what
// Algorithm 3 is described to return.  A homerange without its head repeats the ranks
// 1.., and the ranks 1..y hold exactly the blocks 0..home(y).
__device__ __forceinline__ uint32_t range_mask(const uint32_t *s, uint32_t a, uint32_t b)
{
    uint32_t set = 0;
    while (a <= b) {
        int k = home_of(s, b);
        uint32_t v = s[k];
        if (a > v) {
            a -= v;
            b -= v;
        } else {
            set |= 1u << k;
            uint32_t y = b - v;
            if (y) set |= (2u << home_of(s, y)) - 1u;
            b = v - 1;
        }
    }
    return set;
}

// The same for a cyclic range lo..hi of signed rank numbers (taken mod p); the root has
// no baseblock.  Only the second window of Algorithm 4 needs this generality.
__device__ __noinline__ uint32_t cyclic_mask(const uint32_t *s, uint32_t p, int q,
                                             long long lo, long long hi)
{
    long long len = hi - lo + 1;
    if (len <= 0) return 0;
    if (len >= (long long)p) return q >= 32 ? 0xffffffffu : (1u << q) - 1u;
    long long a = lo % (long long)p;
    if (a < 0) a += p;
    long long b = a + len - 1;
    uint32_t set = 0;
    if (b < (long long)p) {
        if (a == 0) a = 1;
        set = range_mask(s, (uint32_t)a, (uint32_t)b);
    } else {
        if (a == 0) a = 1;
        set = range_mask(s, (uint32_t)a, p - 1);
        b -= p;
        if (b >= 1) set |= range_mask(s, 1, (uint32_t)b);
    }
    return set;
}

// Algorithm 4: receive blocks of rounds 0..last of rank r; rounds are written to
// row[0..last] when row != nullptr; the entry of round `last` is returned.
// B starts as {baseblock(r)} for r > 0 so that the row holds the baseblock once and
// q-1 different other blocks (text after Theorem 1).  Round i looks for the largest new
// block among ranks r-skips[i+1]+1 .. r-skips[i]; that window never contains the root
// outside the home round, it lies entirely below r (i < home) or entirely wrapped
// (i > home).
__device__ __forceinline__ int recv_rounds(const uint32_t *s, uint32_t p, int q, uint32_t r,
                                           int last, uint8_t *row)
{
    int h = -1, bb = 0;
    uint32_t B = 0;
    if (r > 0) {
        h = home_of(s, r);
        bb = base_block(s, r);
        B = 1u << bb;
    }
    unsigned long long sum = 0;
    int entry = 0;
    for (int i = 0; i <= last; ++i) {
        uint32_t lo_skip = s[i], hi_skip = s[i + 1];
        sum += lo_skip;
        if (i == h) {
            entry = bb;
        } else {
            uint32_t wrap = i > h ? p : 0u;      // r - skip + p stays below 2^32
            uint32_t a = r + wrap - hi_skip + 1u;
            uint32_t b = r + wrap - lo_skip;
            uint32_t U = range_mask(s, a, b) & ~B;
            if (U == 0)
                U = cyclic_mask(s, p, q, (long long)r - (long long)sum,
                                (long long)r - (long long)hi_skip) & ~B;
            if (U == 0) {
                entry = BCS_BAD_ENTRY;
            } else {
                int blk = 31 - __clz(U);
                B |= 1u << blk;
                entry = blk - q;
            }
        }
        if (row) row[i] = (uint8_t)entry;
    }
    return entry;
}

template <bool kBatch>
__global__ void __launch_bounds__(kTile)
recv_kernel(PTable tab, uint64_t r_begin, uint64_t r_end, BatchArgs ba, int8_t *recv_out)
{
    __shared__ TileShared sh;
    RankCtx c = resolve_rank<kBatch>(sh, tab, r_begin, r_end, ba);
    const uint32_t shift = (uint32_t)(sh.span_begin & 15u);
    if (c.valid && c.q > 0)
        recv_rounds(c.s, c.p, c.q, c.r, c.q - 1, sh.stage + shift + (c.entry - sh.span_begin));
    __syncthreads();
    flush_span(sh.stage, shift, (uint32_t)(sh.span_end - sh.span_begin), recv_out, sh.span_begin);
}

// Send schedule: sendsched[r][k] = recvsched[(r+skips[k]) mod p][k] (Algorithm 9); where
// that row is not in `recv` the entry is recomputed as Algorithm 5 does.
template <bool kBatch>
__global__ void __launch_bounds__(kTile)
send_kernel(PTable tab, uint64_t r_begin, uint64_t r_end, BatchArgs ba,
            const int8_t *__restrict__ recv, int8_t *send_out)
{
    __shared__ TileShared sh;
    RankCtx c = resolve_rank<kBatch>(sh, tab, r_begin, r_end, ba);
    const uint32_t shift = (uint32_t)(sh.span_begin & 15u);
    if (c.valid) {
        uint8_t *row = sh.stage + shift + (c.entry - sh.span_begin);
        const uint64_t table0 = kBatch ? ba.entry_off[c.pj] : 0;
        for (int k = 0; k < c.q; ++k) {
            uint32_t t = c.r + c.s[k];          // < 2^32 since r, skips[k] < 2^31
            if (t >= c.p) t -= c.p;
            int v;
            if (kBatch) {
                v = recv[table0 + (uint64_t)t * c.q + k];
            } else if (recv != nullptr && t >= r_begin && t < r_end) {
                v = recv[(t - r_begin) * (uint64_t)c.q + k];
            } else {
                v = recv_rounds(c.s, c.p, c.q, t, k, nullptr);
            }
            row[k] = (uint8_t)v;
        }
    }
    __syncthreads();
    flush_span(sh.stage, shift, (uint32_t)(sh.span_end - sh.span_begin), send_out, sh.span_begin);
}

// ================================================================ workspace path
// Skip code of every rank: codes[g] for the flattened rank g (single p: g = x).
template <bool kBatch>
__global__ void __launch_bounds__(kTile)
codes_kernel(PTable tab, BatchArgs ba, uint32_t *__restrict__ codes)
{
    __shared__ TileShared sh;
    RankCtx c = resolve_rank<kBatch>(sh, tab, 0, tab.p, ba);
    if (c.valid) codes[c.rank0 + c.r] = skip_code(c.s, c.q, c.r);
}

// Largest block among the baseblocks of the ranks x+1..y that is not in B, or -1; X and F
// are the skip codes of x and y (x <= y, F = code of y).  Let d be the highest level at which
// the codes differ: y has the term skips[d], x does not, the ranks share everything above.
// Then rank (common part) + skips[d] lies in the range and has baseblock d, the largest of
// the range; behind it come the ranks (head)+1..y, a copy of the ranks 1..(rest of y), which
// hold the blocks 0..m, m the next term of y; before it come the ranks x+1..(head)-1, i.e.
// the range from (rest of x) to skips[d]-1 inside the copy of 1..skips[d]-1, which is
// handled the same way with y replaced by skips[d]-1 (code full[d]).  Heads come out in
// falling order, so the first head outside B, or the point where a head drops to the run of
// low blocks already collected, ends the search.
__device__ __forceinline__ int pick_block(uint32_t X, uint32_t F, uint32_t B,
                                          const uint32_t *full)
{
    uint32_t low = 0;                       // blocks 0..m collected so far, as 2^(m+1)-1
    for (;;) {
        const uint32_t diff = X ^ F;
        if (diff == 0) break;
        const int d = 31 - __clz(diff);
        const uint32_t bit = 1u << d;
        if (bit <= low) break;              // this head and all later ones are inside `low`
        if (!(B & bit)) return d;
        const uint32_t rest = F & (bit - 1u);
        if (rest) low |= (2u << (31 - __clz(rest))) - 1u;
        X &= bit - 1u;
        F = full[d];
    }
    const uint32_t U = low & ~B;
    return U ? 31 - __clz(U) : -1;
}

// Second window of Algorithm 4, ranks r - sum_{j<=i} skips[j] .. r - skips[i+1] (cyclic, the
// root contributes nothing): largest block not in B, or -1.
__device__ __noinline__ int pick_second_window(const uint32_t *codes, const uint32_t *full,
                                               uint32_t p, int q, uint32_t r,
                                               unsigned long long sum, uint32_t hi_skip,
                                               uint32_t B)
{
    const long long lo = (long long)r - (long long)sum, hi = (long long)r - (long long)hi_skip;
    const long long len = hi - lo + 1;
    if (len <= 0) return -1;
    if (len >= (long long)p) {
        const uint32_t U = (q >= 32 ? 0xffffffffu : (1u << q) - 1u) & ~B;
        return U ? 31 - __clz(U) : -1;
    }
    long long a = lo % (long long)p;
    if (a < 0) a += p;
    long long e = a + len - 1;
    if (a == 0) a = 1;
    if (e < (long long)p)
        return a <= e ? pick_block(codes[a - 1], codes[e], B, full) : -1;
    const int b1 = pick_block(codes[a - 1], full[q], B, full);     // a .. p-1 (code of p-1)
    e -= p;
    const int b2 = e >= 1 ? pick_block(0u, codes[e], B, full) : -1;  // 1 .. e
    return b1 > b2 ? b1 : b2;
}

// Algorithm 4 on skip codes: rounds 0..last of rank r of a p whose codes start at `codes`.
// row (shared memory, q bytes) and col (round-major copy, element k at col[k * col_stride])
// receive the entries when not null; the entry of round `last` is returned.
__device__ __forceinline__ int recv_rounds_codes(const uint32_t *__restrict__ codes,
                                                 const uint32_t *s, const uint32_t *full,
                                                 uint32_t p, int q, uint32_t r, int last,
                                                 uint8_t *row, int8_t *col, uint64_t col_stride)
{
    const uint32_t own = codes[r];
    int h = -1, bb = 0;
    uint32_t B = 0;
    if (r > 0) {
        h = 31 - __clz(own);          // homerange: highest term
        bb = __ffs(own) - 1;          // baseblock: lowest term (Algorithm 2)
        B = 1u << bb;
    }
    unsigned long long sum = 0;
    int entry = 0;
    uint32_t upper = codes[r >= 1u ? r - 1u : p - 1u];      // code of r - skips[0]
    for (int i = 0; i <= last; ++i) {
        const uint32_t lo_skip = s[i], hi_skip = s[i + 1];
        sum += lo_skip;
        const uint32_t below = r >= hi_skip ? r - hi_skip : r + p - hi_skip;
        const uint32_t lower = codes[below];                 // code of r - skips[i+1] (mod p)
        if (i == h) {
            entry = bb;
        } else {
            int blk = pick_block(lower, upper, B, full);
            if (blk < 0) blk = pick_second_window(codes, full, p, q, r, sum, hi_skip, B);
            if (blk < 0) {
                entry = BCS_BAD_ENTRY;
            } else {
                B |= 1u << blk;
                entry = blk - q;
            }
        }
        upper = lower;
        if (row) row[i] = (uint8_t)entry;
        if (col) col[(uint64_t)i * col_stride] = (int8_t)entry;
    }
    return entry;
}

// recv_t: round-major copy.  Single p: recv_t[k * t_stride + (r - r_begin)].
// Batch: recv_t[entry_off[j] + k * p_j + r].
template <bool kBatch>
__global__ void __launch_bounds__(kTile)
recv_codes_kernel(PTable tab, uint64_t r_begin, uint64_t r_end, BatchArgs ba,
                  const uint32_t *__restrict__ codes, int8_t *recv_out, int8_t *recv_t,
                  uint64_t t_stride)
{
    __shared__ TileShared sh;
    RankCtx c = resolve_rank<kBatch>(sh, tab, r_begin, r_end, ba);
    const uint32_t shift = (uint32_t)(sh.span_begin & 15u);
    if (c.valid && c.q > 0) {
        int8_t *col = nullptr;
        uint64_t stride = 0;
        if (recv_t != nullptr) {
            col = kBatch ? recv_t + ba.entry_off[c.pj] + c.r : recv_t + (c.r - r_begin);
            stride = kBatch ? (uint64_t)c.p : t_stride;
        }
        uint8_t *row = recv_out ? sh.stage + shift + (c.entry - sh.span_begin) : nullptr;
        recv_rounds_codes(codes + c.rank0, c.s, c.full, c.p, c.q, c.r, c.q - 1, row, col, stride);
    }
    if (recv_out != nullptr) {
        __syncthreads();
        flush_span(sh.stage, shift, (uint32_t)(sh.span_end - sh.span_begin), recv_out,
                   sh.span_begin);
    }
}

// Send rows from the round-major receive copy; to-processors outside the call's range
// (single p, sub-range) are recomputed from the codes (Algorithm 5).
template <bool kBatch>
__global__ void __launch_bounds__(kTile)
send_rm_kernel(PTable tab, uint64_t r_begin, uint64_t r_end, BatchArgs ba,
               const uint32_t *__restrict__ codes, const int8_t *__restrict__ recv_t,
               uint64_t t_stride, int8_t *send_out)
{
    __shared__ TileShared sh;
    RankCtx c = resolve_rank<kBatch>(sh, tab, r_begin, r_end, ba);
    const uint32_t shift = (uint32_t)(sh.span_begin & 15u);
    if (c.valid) {
        uint8_t *row = sh.stage + shift + (c.entry - sh.span_begin);
        const int8_t *tbl = kBatch ? recv_t + ba.entry_off[c.pj] : recv_t;
        const uint64_t stride = kBatch ? (uint64_t)c.p : t_stride;
        for (int k = 0; k < c.q; ++k) {
            uint32_t t = c.r + c.s[k];
            if (t >= c.p) t -= c.p;
            int v;
            if (kBatch) {
                v = tbl[(uint64_t)k * stride + t];
            } else if (t >= r_begin && t < r_end) {
                v = tbl[(uint64_t)k * stride + (t - r_begin)];
            } else {
                v = recv_rounds_codes(codes, c.s, c.full, c.p, c.q, t, k, nullptr, nullptr, 0);
            }
            row[k] = (uint8_t)v;
        }
    }
    __syncthreads();
    flush_span(sh.stage, shift, (uint32_t)(sh.span_end - sh.span_begin), send_out, sh.span_begin);
}

struct Workspace {
    uint32_t *codes;
    int8_t *recv_t;
    uint64_t t_stride;
};

}  // namespace

bcs_status make_table(uint32_t p, PTable *tab)
{
    if (p == 0) return BCS_ERR_RANGE;
    if (p > 0x7fffffffu) return BCS_ERR_UNSUPPORTED;
    const int q = ceil_log2_u32(p);
    for (int k = 0; k < kRow; ++k) tab->s[k] = tab->full[k] = 0;
    uint32_t v = p;
    for (int k = q; k >= 0; --k) {   // Algorithm 1: successive ceil-halving
        tab->s[k] = v;
        v = (v + 1u) / 2u;
    }
    for (int d = 0; d <= q; ++d) tab->full[d] = skip_code(tab->s, q, tab->s[d] - 1u);
    tab->p = p;
    tab->q = q;
    return BCS_OK;
}

}  // namespace bcs

using namespace bcs;

extern "C" {

size_t bcs_build_workspace_bytes(uint32_t p, uint64_t r_begin, uint64_t r_end)
{
    if (check_range(p, r_begin, r_end) != BCS_OK) return 0;
    const int q = ceil_log2_u32(p);
    const uint64_t count = r_end - r_begin;
    if (q == 0 || count == 0) return 0;
    return (size_t)(align_up(4ull * p, 256) + (uint64_t)q * align_up(count, 16));
}

bcs_status bcs_build(uint32_t p, uint64_t r_begin, uint64_t r_end, int8_t *recv_out,
                     int8_t *send_out, void *workspace, size_t workspace_bytes,
                     void *cuda_stream)
{
    bcs_status st = check_range(p, r_begin, r_end);
    if (st != BCS_OK) return st;
    PTable tab;
    make_table(p, &tab);
    const uint64_t count = r_end - r_begin;
    if (count == 0 || tab.q == 0) return BCS_OK;
    if (recv_out == nullptr && send_out == nullptr) return BCS_ERR_ARG;
    if (!aligned16(recv_out) || !aligned16(send_out) || !aligned16(workspace)) return BCS_ERR_ALIGN;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const unsigned blocks = (unsigned)((count + kTile - 1) / kTile);
    BatchArgs none = {};
    if (workspace != nullptr && workspace_bytes >= bcs_build_workspace_bytes(p, r_begin, r_end)) {
        Workspace ws;
        ws.codes = static_cast<uint32_t *>(workspace);
        ws.recv_t = static_cast<int8_t *>(workspace) + align_up(4ull * p, 256);
        ws.t_stride = align_up(count, 16);
        codes_kernel<false><<<(unsigned)((p + kTile - 1) / kTile), kTile, 0, stream>>>(tab, none,
                                                                                      ws.codes);
        if ((st = launch_status()) != BCS_OK) return st;
        recv_codes_kernel<false><<<blocks, kTile, 0, stream>>>(
            tab, r_begin, r_end, none, ws.codes, recv_out, send_out ? ws.recv_t : nullptr,
            ws.t_stride);
        if ((st = launch_status()) != BCS_OK) return st;
        if (send_out != nullptr) {
            send_rm_kernel<false><<<blocks, kTile, 0, stream>>>(tab, r_begin, r_end, none, ws.codes,
                                                                ws.recv_t, ws.t_stride, send_out);
            if ((st = launch_status()) != BCS_OK) return st;
        }
        return BCS_OK;
    }
    if (recv_out != nullptr) {
        recv_kernel<false><<<blocks, kTile, 0, stream>>>(tab, r_begin, r_end, none, recv_out);
        if ((st = launch_status()) != BCS_OK) return st;
    }
    if (send_out != nullptr) {
        send_kernel<false><<<blocks, kTile, 0, stream>>>(tab, r_begin, r_end, none, recv_out,
                                                         send_out);
        if ((st = launch_status()) != BCS_OK) return st;
    }
    return BCS_OK;
}

bcs_status bcs_build_to_host(uint32_t p, uint64_t r_begin, uint64_t r_end, int8_t *recv_host,
                             int8_t *send_host, void *stage_dev, size_t stage_bytes,
                             void *cuda_stream)
{
    bcs_status st = check_range(p, r_begin, r_end);
    if (st != BCS_OK) return st;
    const int q = ceil_log2_u32(p);
    const uint64_t bytes = (r_end - r_begin) * (uint64_t)q;
    if (bytes == 0) return BCS_OK;
    if (recv_host == nullptr && send_host == nullptr) return BCS_ERR_ARG;
    if (stage_dev == nullptr) return BCS_ERR_ARG;
    if (!aligned16(stage_dev)) return BCS_ERR_ALIGN;
    const uint64_t half = align_up(bytes, 256);
    if ((uint64_t)stage_bytes < 2 * half) return BCS_ERR_ARG;
    int8_t *recv_dev = static_cast<int8_t *>(stage_dev);
    int8_t *send_dev = recv_dev + half;
    // what is left of the staging buffer serves as workspace (fast path when large enough)
    void *ws = recv_dev + 2 * half;
    const size_t ws_bytes = stage_bytes - (size_t)(2 * half);
    // the receive table is built even when only the send table is wanted: the send
    // rows are looked up in it.
    st = bcs_build(p, r_begin, r_end, recv_dev, send_host ? send_dev : nullptr,
                   ws_bytes ? ws : nullptr, ws_bytes, cuda_stream);
    if (st != BCS_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (recv_host &&
        cudaMemcpyAsync(recv_host, recv_dev, bytes, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return BCS_ERR_CUDA;
    if (send_host &&
        cudaMemcpyAsync(send_host, send_dev, bytes, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return BCS_ERR_CUDA;
    return BCS_OK;
}

size_t bcs_build_batch_workspace_bytes(uint64_t total_ranks, uint64_t total_entries)
{
    if (total_ranks == 0 || total_entries == 0) return 0;
    return (size_t)(align_up(4ull * total_ranks, 256) + total_entries);
}

bcs_status bcs_build_batch(const uint32_t *p_list_dev, const uint64_t *rank_off_dev,
                           const uint64_t *entry_off_dev, const uint32_t *skips_tab_dev,
                           const uint32_t *full_tab_dev, uint32_t num_p, uint64_t total_ranks,
                           uint64_t total_entries, int8_t *recv_out, int8_t *send_out,
                           void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (num_p == 0 || total_ranks == 0) return BCS_OK;
    if (p_list_dev == nullptr || rank_off_dev == nullptr || entry_off_dev == nullptr ||
        skips_tab_dev == nullptr || full_tab_dev == nullptr)
        return BCS_ERR_ARG;
    if (total_entries == 0) return BCS_OK;   // only p == 1 in the list
    if (recv_out == nullptr) return BCS_ERR_ARG;
    if (!aligned16(recv_out) || !aligned16(send_out) || !aligned16(workspace)) return BCS_ERR_ALIGN;
    const uint64_t blocks64 = (total_ranks + kTile - 1) / kTile;
    if (blocks64 > 0x7fffffffull) return BCS_ERR_UNSUPPORTED;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    BatchArgs ba = {p_list_dev, rank_off_dev, entry_off_dev, skips_tab_dev, full_tab_dev, num_p,
                    total_ranks};
    PTable none = {};
    const unsigned blocks = (unsigned)blocks64;
    bcs_status st;
    if (workspace != nullptr &&
        workspace_bytes >= bcs_build_batch_workspace_bytes(total_ranks, total_entries)) {
        uint32_t *codes = static_cast<uint32_t *>(workspace);
        int8_t *recv_t = static_cast<int8_t *>(workspace) + align_up(4ull * total_ranks, 256);
        codes_kernel<true><<<blocks, kTile, 0, stream>>>(none, ba, codes);
        if ((st = launch_status()) != BCS_OK) return st;
        recv_codes_kernel<true><<<blocks, kTile, 0, stream>>>(none, 0, 0, ba, codes, recv_out,
                                                              send_out ? recv_t : nullptr, 0);
        if ((st = launch_status()) != BCS_OK) return st;
        if (send_out != nullptr) {
            send_rm_kernel<true><<<blocks, kTile, 0, stream>>>(none, 0, 0, ba, codes, recv_t, 0,
                                                               send_out);
            if ((st = launch_status()) != BCS_OK) return st;
        }
        return BCS_OK;
    }
    recv_kernel<true><<<blocks, kTile, 0, stream>>>(none, 0, 0, ba, recv_out);
    if ((st = launch_status()) != BCS_OK) return st;
    if (send_out != nullptr) {
        send_kernel<true><<<blocks, kTile, 0, stream>>>(none, 0, 0, ba, recv_out, send_out);
        if ((st = launch_status()) != BCS_OK) return st;
    }
    return BCS_OK;
}

// Device address of g_static_scratch on the current device, looked up once per device (with that
// device current) and remembered; nullptr if the runtime refuses.
static void *static_scratch_address()
{
    constexpr int kMaxDevices = 64;
    static std::mutex lock;
    static void *known[kMaxDevices] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) return nullptr;
    std::lock_guard<std::mutex> guard(lock);
    if (dev < kMaxDevices && known[dev] != nullptr) return known[dev];
    void *ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess) {
        (void)cudaGetLastError();
        return nullptr;
    }
    if (dev < kMaxDevices) known[dev] = ptr;
    return ptr;
}

bcs_status bcs_build_static(uint32_t p, uint64_t r_begin, uint64_t r_end, int8_t *recv_out,
                            int8_t *send_out, void *cuda_stream)
{
    bcs_status st = check_range(p, r_begin, r_end);
    if (st != BCS_OK) return st;
    if (bcs_build_workspace_bytes(p, r_begin, r_end) > (size_t)BCS_STATIC_WORKSPACE_BYTES)
        return BCS_ERR_UNSUPPORTED;          // needs more scratch than the library carries
    const uint64_t count = r_end - r_begin;
    if (count == 0 || ceil_log2_u32(p) == 0) return BCS_OK;
    void *scratch = static_scratch_address();
    if (scratch == nullptr) return BCS_ERR_CUDA;
    // Nothing in the scratch has to start at zero: the codes of all p ranks and the round-major
    // rows of the range are written by this call before anything reads them, so whatever an
    // earlier call left behind is simply overwritten or never looked at.
    return bcs_build(p, r_begin, r_end, recv_out, send_out, scratch, BCS_STATIC_WORKSPACE_BYTES,
                     cuda_stream);
}

}  // extern "C"
