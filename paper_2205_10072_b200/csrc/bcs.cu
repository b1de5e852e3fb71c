// Construction of round-optimal circulant-graph broadcast schedules on the GPU
// (arXiv 2205.10072, Section 2) -- kernels and the C ABI declared in include/bcs.h.
//
// Work decomposition: one thread per rank for the receive schedule (Algorithm 4),
// one thread per rank for the send schedule (lookup of Algorithm 9, with Algorithm 5's
// recomputation where the to-processor's row is not available), one thread per output
// record for the round tables (Algorithm 6).  A CTA covers a run of consecutive ranks;
// its rows are assembled in shared memory and leave as one contiguous, 16-byte
// vectorised span because the tables are rank-major and unpadded.
#include <cuda_runtime.h>
#include <stdint.h>

#include "bcs.h"

namespace {

constexpr int kTile = 256;                    // ranks (= threads) per CTA of the schedule kernels
constexpr int kStageBytes = kTile * 32 + 16;  // room for kTile rows of <= 31 bytes + alignment shift
constexpr int kCachedRows = 8;                // skips rows a batch CTA keeps in shared memory

struct SkipTable {      // kernel parameter of the single-p kernels
    uint32_t s[32];     // skips[0..q], q <= 31
    uint32_t p;
    int q;
};

struct BatchArgs {
    const uint32_t *p_list;
    const uint64_t *rank_off;
    const uint64_t *entry_off;
    const uint32_t *skips_tab;
    uint32_t num_p;
    uint64_t total_ranks;
};

__host__ __device__ inline int ceil_log2_u32(uint32_t p)
{
    int q = 0;
    while (q < 32 && (uint64_t(1) << q) < p) ++q;
    return q;
}

__device__ __forceinline__ int ceil_log2_fast(uint32_t p) { return p > 1u ? 32 - __clz(p - 1u) : 0; }

// ---------------------------------------------------------------- Section 2 primitives
// Largest k with skips[k] <= x (the homerange of x), 1 <= x < p.  Algorithm 1 gives
// 2^(k-1) < skips[k] <= 2^k, so k is floor(log2 x) or one more.
__device__ __forceinline__ int home_of(const uint32_t *s, uint32_t x)
{
    int m = 31 - __clz(x);
    return m + (s[m + 1] <= x ? 1 : 0);
}

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

// ---------------------------------------------------------------- tile bookkeeping
struct RankCtx {
    const uint32_t *s;   // skips of this rank's p (shared or global memory)
    uint32_t p;
    int q;
    uint32_t r;
    uint32_t pj;         // index of p in the batch (0 for the single-p kernels)
    uint64_t entry;      // byte offset of the rank's row in the output
    bool valid;
};

// Copies stage[shift, shift+len) to out[byte0, byte0+len); (byte0 & 15) == shift and `out`
// is 16-byte aligned, so all but the ragged ends go out as 16-byte vectors.
__device__ __forceinline__ void flush_span(const uint8_t *stage, uint32_t shift, uint32_t len,
                                           int8_t *out, uint64_t byte0)
{
    uint8_t *dst = reinterpret_cast<uint8_t *>(out) + (byte0 - shift);
    const uint32_t end = shift + len;
    const uint32_t nvec = (end + 15u) >> 4;
    for (uint32_t v = threadIdx.x; v < nvec; v += blockDim.x) {
        uint32_t lo = v << 4, hi = lo + 16u;
        if (lo >= shift && hi <= end) {
            *reinterpret_cast<uint4 *>(dst + lo) = *reinterpret_cast<const uint4 *>(stage + lo);
        } else {
            uint32_t from = lo < shift ? shift : lo, to = hi > end ? end : hi;
            for (uint32_t e = from; e < to; ++e) dst[e] = stage[e];
        }
    }
}

// Largest j with off[j] <= g, searched in [lo, hi].
__device__ __forceinline__ uint32_t find_segment(const uint64_t *off, uint32_t lo, uint32_t hi,
                                                 uint64_t g)
{
    while (lo < hi) {
        uint32_t mid = (lo + hi + 1) >> 1;
        if (off[mid] <= g) lo = mid; else hi = mid - 1;
    }
    return lo;
}

struct TileShared {
    uint32_t skips[kCachedRows][BCS_SKIPS_STRIDE];
    uint64_t span_begin, span_end;
    uint32_t j_first, j_last;
    __align__(16) uint8_t stage[kStageBytes];
};

// Resolves the rank this thread works on.  Single p: consecutive ranks from r_begin.
// Batch: flattened index g over all (p_j, r); the CTA looks up the first and last p it
// touches once, keeps the first few skips rows in shared memory, and each thread finds
// its own p between the two.
template <bool kBatch>
__device__ __forceinline__ RankCtx resolve_rank(TileShared &sh, const SkipTable &tab,
                                                uint64_t r_begin, uint64_t r_end,
                                                const BatchArgs &ba)
{
    RankCtx c;
    const uint64_t g0 = (uint64_t)blockIdx.x * kTile;
    if (!kBatch) {
        if (threadIdx.x <= (unsigned)tab.q) sh.skips[0][threadIdx.x] = tab.s[threadIdx.x];
        const uint64_t count = r_end - r_begin;
        const uint64_t g1 = g0 + kTile < count ? g0 + kTile : count;
        if (threadIdx.x == 0) {
            sh.span_begin = g0 * (uint64_t)tab.q;
            sh.span_end = g1 * (uint64_t)tab.q;
        }
        __syncthreads();
        const uint64_t g = g0 + threadIdx.x;
        c.s = sh.skips[0];
        c.p = tab.p;
        c.q = tab.q;
        c.pj = 0;
        c.valid = g < count;
        c.r = (uint32_t)(r_begin + g);
        c.entry = g * (uint64_t)tab.q;
        return c;
    }
    const uint64_t g1 = g0 + kTile < ba.total_ranks ? g0 + kTile : ba.total_ranks;
    if (threadIdx.x == 0) {
        uint32_t jf = find_segment(ba.rank_off, 0, ba.num_p - 1, g0);
        uint32_t jl = find_segment(ba.rank_off, jf, ba.num_p - 1, g1 - 1);
        sh.j_first = jf;
        sh.j_last = jl;
        int qf = ceil_log2_fast(ba.p_list[jf]);
        int ql = ceil_log2_fast(ba.p_list[jl]);
        sh.span_begin = ba.entry_off[jf] + (g0 - ba.rank_off[jf]) * (uint64_t)qf;
        sh.span_end = ba.entry_off[jl] + (g1 - ba.rank_off[jl]) * (uint64_t)ql;
    }
    __syncthreads();
    const uint32_t jf = sh.j_first, jl = sh.j_last;
    {
        const uint32_t row = threadIdx.x / BCS_SKIPS_STRIDE, col = threadIdx.x % BCS_SKIPS_STRIDE;
        if (row < kCachedRows && jf + row <= jl)
            sh.skips[row][col] = ba.skips_tab[(size_t)(jf + row) * BCS_SKIPS_STRIDE + col];
    }
    __syncthreads();
    const uint64_t g = g0 + threadIdx.x;
    c.valid = g < g1;
    const uint32_t j = c.valid ? find_segment(ba.rank_off, jf, jl, g) : jf;
    c.s = (j - jf < (uint32_t)kCachedRows) ? sh.skips[j - jf]
                                           : ba.skips_tab + (size_t)j * BCS_SKIPS_STRIDE;
    c.pj = j;
    c.p = ba.p_list[j];
    c.q = ceil_log2_fast(c.p);
    c.r = (uint32_t)(g - ba.rank_off[j]);
    c.entry = ba.entry_off[j] + (uint64_t)c.r * (uint64_t)c.q;
    return c;
}

// ---------------------------------------------------------------- schedule kernels
template <bool kBatch>
__global__ void __launch_bounds__(kTile)
recv_kernel(SkipTable tab, uint64_t r_begin, uint64_t r_end, BatchArgs ba, int8_t *recv_out)
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
send_kernel(SkipTable tab, uint64_t r_begin, uint64_t r_end, BatchArgs ba,
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

// ---------------------------------------------------------------- Algorithm 6: round tables
constexpr int kExpandThreads = 256;
constexpr int kExpandRanks = 8;   // ranks per CTA

__global__ void __launch_bounds__(kExpandThreads)
expand_kernel(SkipTable tab, uint32_t n, uint64_t r_begin, uint64_t r_end,
              const int8_t *__restrict__ recv, const int8_t *__restrict__ send,
              int4 *__restrict__ table_out)
{
    // per rank of the CTA and per round k of a phase: {send entry - x, recv entry - x, to, from}.
    // Algorithm 6 adds q to an entry after each use and starts entries k < x at +q because
    // their first use is in the second phase; both are covered by adding q * floor(i / q).
    __shared__ int4 base[kExpandRanks][32];
    const int q = tab.q;
    const uint32_t p = tab.p;
    const uint32_t rounds = n - 1u + (uint32_t)q;
    const int x = (int)(((uint32_t)q - rounds % (uint32_t)q) % (uint32_t)q);
    const uint64_t j0 = (uint64_t)blockIdx.x * kExpandRanks;
    const uint64_t count = r_end - r_begin;
    {
        const int g = threadIdx.x / 32, k = threadIdx.x % 32;
        if (g < kExpandRanks && k < q && j0 + g < count) {
            const uint64_t row = (j0 + g) * (uint64_t)q;
            const uint32_t r = (uint32_t)(r_begin + j0 + g);
            const uint32_t sk = tab.s[k];
            const int adj = -x;
            uint32_t to = r + sk;
            if (to >= p) to -= p;
            uint32_t from = r >= sk ? r - sk : r + p - sk;
            base[g][k] = make_int4((int)send[row + k] + adj, (int)recv[row + k] + adj, (int)to,
                                   (int)from);
        }
    }
    __syncthreads();
    // round j uses i = j + x: entry k = i mod q of phase i / q.
    const uint32_t step_k = kExpandThreads % (uint32_t)q, step_ph = kExpandThreads / (uint32_t)q;
    const int last = (int)n - 1;
    for (int g = 0; g < kExpandRanks; ++g) {
        if (j0 + g >= count) break;
        int4 *out = table_out + (j0 + g) * (uint64_t)rounds;
        uint32_t i = threadIdx.x + (uint32_t)x;
        uint32_t k = i % (uint32_t)q, ph = i / (uint32_t)q;
        for (uint32_t j = threadIdx.x; j < rounds; j += kExpandThreads) {
            int4 rec = base[g][k];
            const int add = (int)(ph * (uint32_t)q);
            int sb = rec.x + add, rb = rec.y + add;
            sb = sb < 0 ? -1 : (sb > last ? last : sb);
            rb = rb < 0 ? -1 : (rb > last ? last : rb);
            __stcs(out + j, make_int4(sb, rb, rec.z, rec.w));
            k += step_k;
            ph += step_ph;
            if (k >= (uint32_t)q) { k -= (uint32_t)q; ++ph; }
        }
    }
}

// ---------------------------------------------------------------- checksum
__device__ __forceinline__ uint32_t fmix32(uint32_t h)
{
    h ^= h >> 16; h *= 0x85ebca6bu;
    h ^= h >> 13; h *= 0xc2b2ae35u;
    h ^= h >> 16;
    return h;
}

__device__ __forceinline__ uint32_t word_weight(uint64_t g)
{
    return fmix32((uint32_t)g ^ (0x9E3779B9u * (uint32_t)(g >> 32))) | 1u;
}

constexpr int kSumThreads = 256;

__global__ void __launch_bounds__(kSumThreads)
checksum_kernel(const uint32_t *__restrict__ words, uint64_t n_words, uint32_t tail_bytes,
                uint64_t first_word, unsigned long long *sum)
{
    // n_words full words, then tail_bytes (0..3) bytes of one more, zero-padded.
    unsigned long long acc = 0;
    const uint64_t stride = (uint64_t)gridDim.x * kSumThreads;
    for (uint64_t w = (uint64_t)blockIdx.x * kSumThreads + threadIdx.x; w < n_words; w += stride)
        acc += (unsigned long long)words[w] * word_weight(first_word + w);
    if (tail_bytes && blockIdx.x == 0 && threadIdx.x == 0) {
        const uint8_t *b = reinterpret_cast<const uint8_t *>(words + n_words);
        uint32_t v = 0;
        for (uint32_t t = 0; t < tail_bytes; ++t) v |= (uint32_t)b[t] << (8 * t);
        acc += (unsigned long long)v * word_weight(first_word + n_words);
    }
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, o);
    __shared__ unsigned long long part[kSumThreads / 32];
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long t = 0;
        for (int w = 0; w < kSumThreads / 32; ++w) t += part[w];
        atomicAdd(sum, t);
    }
}

// ---------------------------------------------------------------- host side
bcs_status make_table(uint32_t p, SkipTable *tab)
{
    if (p == 0) return BCS_ERR_RANGE;
    if (p > 0x7fffffffu) return BCS_ERR_UNSUPPORTED;
    const int q = ceil_log2_u32(p);
    for (int k = 0; k < 32; ++k) tab->s[k] = 0;
    uint32_t v = p;
    for (int k = q; k >= 0; --k) {   // Algorithm 1: successive ceil-halving
        tab->s[k] = v;
        v = (v + 1u) / 2u;
    }
    tab->p = p;
    tab->q = q;
    return BCS_OK;
}

inline bool aligned16(const void *ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15u) == 0; }

inline bcs_status launch_status()
{
    return cudaGetLastError() == cudaSuccess ? BCS_OK : BCS_ERR_CUDA;
}

bcs_status check_range(uint32_t p, uint64_t r_begin, uint64_t r_end)
{
    if (p == 0) return BCS_ERR_RANGE;
    if (p > 0x7fffffffu) return BCS_ERR_UNSUPPORTED;
    if (r_begin > r_end || r_end > p) return BCS_ERR_RANGE;
    return BCS_OK;
}

}  // namespace

extern "C" {

const char *bcs_status_str(bcs_status st)
{
    switch (st) {
        case BCS_OK: return "BCS_OK";
        case BCS_ERR_ARG: return "BCS_ERR_ARG";
        case BCS_ERR_RANGE: return "BCS_ERR_RANGE";
        case BCS_ERR_ALIGN: return "BCS_ERR_ALIGN";
        case BCS_ERR_UNSUPPORTED: return "BCS_ERR_UNSUPPORTED";
        case BCS_ERR_CUDA: return "BCS_ERR_CUDA";
    }
    return "BCS_ERR_UNKNOWN";
}

int bcs_q(uint32_t p) { return p == 0 ? -1 : ceil_log2_u32(p); }

bcs_status bcs_skips(uint32_t p, uint32_t *skips_host)
{
    SkipTable tab;
    bcs_status st = make_table(p, &tab);
    if (st != BCS_OK) return st;
    if (skips_host == nullptr) return BCS_ERR_ARG;
    for (int k = 0; k <= tab.q; ++k) skips_host[k] = tab.s[k];
    return BCS_OK;
}

bcs_status bcs_build(uint32_t p, uint64_t r_begin, uint64_t r_end, int8_t *recv_out,
                     int8_t *send_out, void *cuda_stream)
{
    bcs_status st = check_range(p, r_begin, r_end);
    if (st != BCS_OK) return st;
    SkipTable tab;
    make_table(p, &tab);
    const uint64_t count = r_end - r_begin;
    if (count == 0 || tab.q == 0) return BCS_OK;
    if (recv_out == nullptr && send_out == nullptr) return BCS_ERR_ARG;
    if (!aligned16(recv_out) || !aligned16(send_out)) return BCS_ERR_ALIGN;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const unsigned blocks = (unsigned)((count + kTile - 1) / kTile);
    BatchArgs none = {};
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
    const uint64_t half = (bytes + 255u) & ~uint64_t(255);
    if ((uint64_t)stage_bytes < 2 * half) return BCS_ERR_ARG;
    int8_t *recv_dev = static_cast<int8_t *>(stage_dev);
    int8_t *send_dev = recv_dev + half;
    // the receive table is built even when only the send table is wanted: the send
    // rows are looked up in it.
    st = bcs_build(p, r_begin, r_end, recv_dev, send_host ? send_dev : nullptr, cuda_stream);
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

bcs_status bcs_batch_plan(const uint32_t *p_list_host, uint32_t num_p, uint64_t *rank_off_host,
                          uint64_t *entry_off_host, uint32_t *skips_tab_host)
{
    if (p_list_host == nullptr || rank_off_host == nullptr || entry_off_host == nullptr ||
        skips_tab_host == nullptr)
        return BCS_ERR_ARG;
    uint64_t ranks = 0, entries = 0;
    for (uint32_t j = 0; j < num_p; ++j) {
        SkipTable tab;
        bcs_status st = make_table(p_list_host[j], &tab);
        if (st != BCS_OK) return st;
        rank_off_host[j] = ranks;
        entry_off_host[j] = entries;
        uint32_t *row = skips_tab_host + (size_t)j * BCS_SKIPS_STRIDE;
        for (int k = 0; k < BCS_SKIPS_STRIDE; ++k) row[k] = tab.s[k];
        ranks += tab.p;
        entries += (uint64_t)tab.p * (uint64_t)tab.q;
    }
    rank_off_host[num_p] = ranks;
    entry_off_host[num_p] = entries;
    return BCS_OK;
}

bcs_status bcs_build_batch(const uint32_t *p_list_dev, const uint64_t *rank_off_dev,
                           const uint64_t *entry_off_dev, const uint32_t *skips_tab_dev,
                           uint32_t num_p, uint64_t total_ranks, uint64_t total_entries,
                           int8_t *recv_out, int8_t *send_out, void *cuda_stream)
{
    if (num_p == 0 || total_ranks == 0) return BCS_OK;
    if (p_list_dev == nullptr || rank_off_dev == nullptr || entry_off_dev == nullptr ||
        skips_tab_dev == nullptr)
        return BCS_ERR_ARG;
    if (total_entries == 0) return BCS_OK;   // only p == 1 in the list
    if (recv_out == nullptr) return BCS_ERR_ARG;
    if (!aligned16(recv_out) || !aligned16(send_out)) return BCS_ERR_ALIGN;
    const uint64_t blocks64 = (total_ranks + kTile - 1) / kTile;
    if (blocks64 > 0x7fffffffull) return BCS_ERR_UNSUPPORTED;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    BatchArgs ba = {p_list_dev, rank_off_dev, entry_off_dev, skips_tab_dev, num_p, total_ranks};
    SkipTable none = {};
    const unsigned blocks = (unsigned)blocks64;
    bcs_status st;
    recv_kernel<true><<<blocks, kTile, 0, stream>>>(none, 0, 0, ba, recv_out);
    if ((st = launch_status()) != BCS_OK) return st;
    if (send_out != nullptr) {
        send_kernel<true><<<blocks, kTile, 0, stream>>>(none, 0, 0, ba, recv_out, send_out);
        if ((st = launch_status()) != BCS_OK) return st;
    }
    return BCS_OK;
}

bcs_status bcs_expand(uint32_t p, uint32_t n, uint64_t r_begin, uint64_t r_end,
                      const int8_t *recv, const int8_t *send, int32_t *table_out,
                      void *cuda_stream)
{
    bcs_status st = check_range(p, r_begin, r_end);
    if (st != BCS_OK) return st;
    if (n == 0) return BCS_ERR_ARG;
    if (n > 0x7fffff00u) return BCS_ERR_UNSUPPORTED;   // block numbers and n-1+q stay in int32
    SkipTable tab;
    make_table(p, &tab);
    const uint64_t count = r_end - r_begin;
    if (count == 0 || tab.q == 0) return BCS_OK;
    if (recv == nullptr || send == nullptr || table_out == nullptr) return BCS_ERR_ARG;
    if (!aligned16(table_out)) return BCS_ERR_ALIGN;
    const unsigned blocks = (unsigned)((count + kExpandRanks - 1) / kExpandRanks);
    expand_kernel<<<blocks, kExpandThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        tab, n, r_begin, r_end, recv, send, reinterpret_cast<int4 *>(table_out));
    return launch_status();
}

bcs_status bcs_checksum(const int8_t *buf_dev, uint64_t n_entries, uint64_t first_entry_index,
                        uint64_t *sum_dev, void *cuda_stream)
{
    if (sum_dev == nullptr) return BCS_ERR_ARG;
    if (n_entries != 0 && buf_dev == nullptr) return BCS_ERR_ARG;
    if ((first_entry_index & 3u) != 0 || (reinterpret_cast<uintptr_t>(buf_dev) & 3u) != 0)
        return BCS_ERR_ALIGN;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemsetAsync(sum_dev, 0, sizeof(uint64_t), stream) != cudaSuccess) return BCS_ERR_CUDA;
    if (n_entries == 0) return BCS_OK;
    const uint64_t n_words = n_entries / 4;
    uint64_t blocks = (n_words / 4 + kSumThreads - 1) / kSumThreads;   // ~4 words per thread
    if (blocks < 1) blocks = 1;
    if (blocks > 148u * 16u) blocks = 148u * 16u;
    checksum_kernel<<<(unsigned)blocks, kSumThreads, 0, stream>>>(
        reinterpret_cast<const uint32_t *>(buf_dev), n_words, (uint32_t)(n_entries & 3u),
        first_entry_index / 4, reinterpret_cast<unsigned long long *>(sum_dev));
    return launch_status();
}

}  // extern "C"
