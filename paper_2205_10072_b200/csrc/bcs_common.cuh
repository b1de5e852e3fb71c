// Shared pieces of the schedule, round-table and checksum translation units: per-p tables,
// the Section 2 primitives of arXiv 2205.10072 as device functions, and the tile bookkeeping
// that turns per-rank rows into contiguous, 16-byte vectorised output spans.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "bcs.h"

namespace bcs {

constexpr int kTile = 256;                    // ranks (= threads) per CTA of the schedule kernels
constexpr int kStageBytes = kTile * 32 + 16;  // kTile rows of <= 31 bytes + alignment shift
constexpr uint32_t kFusedMaxP = 1024;         // batch: a p up to here is built by one CTA of the fused kernel
constexpr int kFusedMaxQ = 10;                //        (q <= 10)
constexpr int kCachedRows = 4;                // per-p table rows a batch CTA keeps in shared memory
constexpr int kRow = BCS_SKIPS_STRIDE;        // words per table row

// Per-p constants (kernel parameter of the single-p kernels).
//   s[k]    = skips[k] of Algorithm 1, k = 0..q (q <= 31)
//   full[d] = skip code of rank skips[d]-1, d = 0..q (see skip_code below)
struct PTable {
    uint32_t s[kRow];
    uint32_t full[kRow];
    uint32_t p;
    int q;
};

struct BatchArgs {
    const uint32_t *p_list;
    const uint64_t *rank_off;
    const uint64_t *entry_off;
    const uint32_t *skips_tab;   // [num_p][kRow]
    const uint32_t *full_tab;    // [num_p][kRow]
    uint32_t num_p;
    uint64_t total_ranks;
    // workspace construction only: tiles of 512 ranks that start anew with every p, and where
    // the round-major copy of each p starts (every round padded to a multiple of 16 bytes)
    const uint64_t *tile_off;    // [num_p + 1] prefix sums of ceil(p_j / 512)
    const uint64_t *copy_off;    // [num_p + 1] prefix sums of q_j * align16(p_j)
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

// Skip code of rank x (0 <= x < p): bit k set iff skips[k] is a term of the greedy
// decomposition x = skips[k1] + skips[k2] + ... that Algorithm 2 walks down (largest skip
// not above the remainder first; the remainder after taking skips[k] is below skips[k], so a
// downward scan over the levels finds the same terms).  The baseblock of x is the lowest set
// bit, its homerange the highest.  Codes order like ranks.
__host__ __device__ inline uint32_t skip_code(const uint32_t *s, int q, uint32_t x)
{
    uint32_t code = 0;
    for (int k = q - 1; k >= 0; --k) {
        if (x >= s[k]) {
            x -= s[k];
            code |= 1u << k;
        }
    }
    return code;
}

// ---------------------------------------------------------------- tile bookkeeping
struct RankCtx {
    const uint32_t *s;      // skips of this rank's p (shared or global memory)
    const uint32_t *full;   // full[] of this rank's p
    uint32_t p;
    int q;
    uint32_t r;
    uint32_t pj;            // index of p in the batch (0 for the single-p kernels)
    uint64_t rank0;         // flattened index of rank 0 of this p (0 for single p)
    uint64_t entry;         // byte offset of the rank's row in the output
    bool valid;
};

struct TileShared {
    uint32_t skips[kCachedRows][kRow];
    uint32_t full[kCachedRows][kRow];
    uint64_t span_begin, span_end;
    uint64_t rank0_first, entry0_first;   // batch: rank and entry offset of the CTA's first p
    uint32_t j_first, j_last;
    uint32_t p_first;
    __align__(16) uint8_t stage[kStageBytes];
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

// The same for a staging buffer whose span starts `lag` = 1..3 bytes EARLIER in its 16-byte group
// than the span does in global memory: stage[shift - lag, shift - lag + len) goes to
// out[byte0, byte0 + len) with (byte0 & 15) == shift, shift >= lag.  (Rows that must start on a word
// in shared memory while the table starts at any byte of the output.)  Every 16-byte vector of the
// output is put together from five aligned words of the staging buffer, funnel-shifted by `lag`
// bytes; the ragged ends go out as bytes.  The four bytes before `stage` must be readable.
__device__ __forceinline__ void flush_span_lagging(const uint8_t *stage, uint32_t shift, uint32_t lag, uint32_t len,
                                                   int8_t *out, uint64_t byte0)
{
    uint8_t *dst = reinterpret_cast<uint8_t *>(out) + (byte0 - shift);
    const uint32_t end = shift + len;
    const uint32_t nvec = (end + 15u) >> 4;
    const uint32_t bits = 8u * (4u - lag);
    for (uint32_t v = threadIdx.x; v < nvec; v += blockDim.x) {
        const uint32_t lo = v << 4, hi = lo + 16u;
        if (lo >= shift && hi <= end) {
            // output bytes lo .. lo+15 are staging bytes lo-lag .. lo+15-lag: words at lo-4, lo, ..., lo+12
            const uint32_t *w = reinterpret_cast<const uint32_t *>(stage + lo) - 1;
            const uint32_t w0 = w[0], w1 = w[1], w2 = w[2], w3 = w[3], w4 = w[4];
            *reinterpret_cast<uint4 *>(dst + lo) =
                make_uint4(__funnelshift_r(w0, w1, bits), __funnelshift_r(w1, w2, bits),
                           __funnelshift_r(w2, w3, bits), __funnelshift_r(w3, w4, bits));
        } else {
            const uint32_t from = lo < shift ? shift : lo, to = hi > end ? end : hi;
            for (uint32_t e = from; e < to; ++e) dst[e] = stage[e - lag];
        }
    }
}

// The same for a span that starts 16-byte aligned in shared and global memory and is a multiple
// of 16 bytes long, as one bulk copy of the TMA unit (cp.async.bulk, shared -> global) issued by
// one thread.  Call with all threads of the CTA, after the rows have been written and INSTEAD of
// the barrier that precedes flush_span: every thread makes its shared-memory writes visible to
// the asynchronous proxy, the CTA synchronises, thread 0 issues the copy and waits until the
// unit has read the staging buffer (the global writes complete on their own).
__device__ __forceinline__ void flush_span_bulk(const uint8_t *stage, uint32_t len, int8_t *out,
                                                uint64_t byte0)
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    if (threadIdx.x == 0 && len != 0) {
        const uint32_t src = (uint32_t)__cvta_generic_to_shared(stage);
        const uint64_t dst = reinterpret_cast<uint64_t>(out) + byte0;
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                     :: "l"(dst), "r"(src), "r"(len) : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
    }
}

// Copies in[byte0, byte0+len) to stage[shift, shift+len), (byte0 & 15) == shift, `in` 16-byte
// aligned: the mirror image of flush_span.
__device__ __forceinline__ void load_span(uint8_t *stage, uint32_t shift, uint32_t len,
                                          const int8_t *in, uint64_t byte0)
{
    const uint8_t *src = reinterpret_cast<const uint8_t *>(in) + (byte0 - shift);
    const uint32_t end = shift + len;
    const uint32_t nvec = (end + 15u) >> 4;
    for (uint32_t v = threadIdx.x; v < nvec; v += blockDim.x) {
        const uint32_t lo = v << 4, hi = lo + 16u;
        if (lo >= shift && hi <= end) {
            *reinterpret_cast<uint4 *>(stage + lo) = *reinterpret_cast<const uint4 *>(src + lo);
        } else {
            const uint32_t from = lo < shift ? shift : lo, to = hi > end ? end : hi;
            for (uint32_t e = from; e < to; ++e) stage[e] = src[e];
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

// The same search by a whole warp: 32 probes per step instead of one, so a table of a few
// thousand offsets takes three dependent loads instead of twelve.  All 32 lanes must call.
__device__ __forceinline__ uint32_t find_segment_warp(const uint64_t *off, uint32_t num, uint64_t g)
{
    const uint32_t lane = threadIdx.x & 31u;
    uint32_t lo = 0, hi = num;                       // answer in [lo, hi)
    while (hi - lo > 1u) {
        const uint32_t step = (hi - lo + 31u) / 32u;
        const uint32_t idx = lo + lane * step;
        const bool le = idx < hi && off[idx] <= g;
        const uint32_t hits = __popc(__ballot_sync(0xffffffffu, le));   // lane 0 always hits
        lo += (hits - 1u) * step;
        hi = lo + step < hi ? lo + step : hi;
    }
    return lo;
}

// Resolves the rank this thread works on.  Single p: consecutive ranks from r_begin.
// Batch: flattened index g over all (p_j, r); the CTA looks up the first and last p it
// touches once, keeps the first few table rows in shared memory, and each thread finds
// its own p between the two.
template <bool kBatch>
__device__ __forceinline__ RankCtx resolve_rank(TileShared &sh, const PTable &tab,
                                                uint64_t r_begin, uint64_t r_end,
                                                const BatchArgs &ba)
{
    RankCtx c;
    const uint64_t g0 = (uint64_t)blockIdx.x * kTile;
    if (!kBatch) {
        if (threadIdx.x < kRow) {
            sh.skips[0][threadIdx.x] = tab.s[threadIdx.x];
            sh.full[0][threadIdx.x] = tab.full[threadIdx.x];
        }
        const uint64_t count = r_end - r_begin;
        const uint64_t g1 = g0 + kTile < count ? g0 + kTile : count;
        if (threadIdx.x == 0) {
            sh.span_begin = g0 * (uint64_t)tab.q;
            sh.span_end = g1 * (uint64_t)tab.q;
        }
        __syncthreads();
        const uint64_t g = g0 + threadIdx.x;
        c.s = sh.skips[0];
        c.full = sh.full[0];
        c.p = tab.p;
        c.q = tab.q;
        c.pj = 0;
        c.rank0 = 0;
        c.valid = g < count;
        c.r = (uint32_t)(r_begin + g);
        c.entry = g * (uint64_t)tab.q;
        return c;
    }
    const uint64_t g1 = g0 + kTile < ba.total_ranks ? g0 + kTile : ba.total_ranks;
    if (threadIdx.x < 32) {
        const uint32_t jf = find_segment_warp(ba.rank_off, ba.num_p, g0);
        const uint32_t jl = ba.rank_off[jf + 1] >= g1 ? jf : find_segment_warp(ba.rank_off, ba.num_p, g1 - 1);
        if (threadIdx.x == 0) {
            sh.j_first = jf;
            sh.j_last = jl;
            sh.p_first = ba.p_list[jf];
            sh.rank0_first = ba.rank_off[jf];
            sh.entry0_first = ba.entry_off[jf];
            const int qf = ceil_log2_fast(sh.p_first);
            const int ql = ceil_log2_fast(ba.p_list[jl]);
            sh.span_begin = sh.entry0_first + (g0 - sh.rank0_first) * (uint64_t)qf;
            sh.span_end = ba.entry_off[jl] + (g1 - ba.rank_off[jl]) * (uint64_t)ql;
        }
    }
    __syncthreads();
    const uint32_t jf = sh.j_first, jl = sh.j_last;
    {
        const uint32_t row = threadIdx.x / (2 * kRow), col = threadIdx.x % (2 * kRow);
        if (row < kCachedRows && jf + row <= jl) {
            if (col < kRow)
                sh.skips[row][col] = ba.skips_tab[(size_t)(jf + row) * kRow + col];
            else
                sh.full[row][col - kRow] = ba.full_tab[(size_t)(jf + row) * kRow + col - kRow];
        }
    }
    __syncthreads();
    const uint64_t g = g0 + threadIdx.x;
    c.valid = g < g1;
    if (jf == jl) {                                  // the whole CTA inside one p: no per-thread lookups
        c.s = sh.skips[0];
        c.full = sh.full[0];
        c.pj = jf;
        c.p = sh.p_first;
        c.q = ceil_log2_fast(c.p);
        c.rank0 = sh.rank0_first;
        c.r = (uint32_t)(g - c.rank0);
        c.entry = sh.entry0_first + (uint64_t)c.r * (uint64_t)c.q;
        return c;
    }
    const uint32_t j = c.valid ? find_segment(ba.rank_off, jf, jl, g) : jf;
    const bool cached = j - jf < (uint32_t)kCachedRows;
    c.s = cached ? sh.skips[j - jf] : ba.skips_tab + (size_t)j * kRow;
    c.full = cached ? sh.full[j - jf] : ba.full_tab + (size_t)j * kRow;
    c.pj = j;
    c.p = ba.p_list[j];
    c.q = ceil_log2_fast(c.p);
    c.rank0 = ba.rank_off[j];
    c.r = (uint32_t)(g - c.rank0);
    c.entry = ba.entry_off[j] + (uint64_t)c.r * (uint64_t)c.q;
    return c;
}

// ---------------------------------------------------------------- dependent launches
// The kernels of one construction run back to back on one stream, each a few tens of
// microseconds long, so the time in which one grid drains and the next is brought onto the SMs
// counts.  A kernel launched with launch_dependent() may be made resident as soon as every CTA
// of the kernel before it on the stream has called grid_launch_dependents() (or has exited); it
// runs its set-up and then blocks in grid_dependency_wait() until that kernel has completed and
// its writes are visible.  Both calls do nothing in a kernel that was launched the ordinary way.
__device__ __forceinline__ void grid_dependency_wait()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

__device__ __forceinline__ void grid_launch_dependents()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// ---------------------------------------------------------------- host helpers
bcs_status make_table(uint32_t p, PTable *tab);

// Launch with programmatic stream serialisation (see above); `dependent` false: ordinary launch.
template <class... Params, class... Args>
inline void launch_dependent(bool dependent, void (*kernel)(Params...), unsigned grid, unsigned block,
                             cudaStream_t stream, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 1 : 0;
    cudaLaunchKernelEx(&cfg, kernel, Params(args)...);
}

inline bool aligned16(const void *ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15u) == 0; }

inline bcs_status launch_status()
{
    return cudaGetLastError() == cudaSuccess ? BCS_OK : BCS_ERR_CUDA;
}

inline bcs_status check_range(uint32_t p, uint64_t r_begin, uint64_t r_end)
{
    if (p == 0) return BCS_ERR_RANGE;
    if (p > 0x7fffffffu) return BCS_ERR_UNSUPPORTED;
    if (r_begin > r_end || r_end > p) return BCS_ERR_RANGE;
    return BCS_OK;
}

__host__ __device__ inline uint64_t align_up(uint64_t v, uint64_t a) { return (v + a - 1) / a * a; }

}  // namespace bcs
