// Receive and send schedules (arXiv 2205.10072, Algorithms 2-5 and the lookup of Algorithm 9):
// kernels and the entry points bcs_build, bcs_build_static, bcs_build_to_host, bcs_prepare,
// bcs_prepare_codes, bcs_prepare_rows, bcs_build_prepared, bcs_build_rooted, bcs_build_batch.
//
// Two constructions, bit-identical in their results:
//
//  * workspace path.  codes_single_kernel / codes_batch_kernel write the skip code (bcs_common.cuh) of every rank x of a p
//    once.  The receive kernels (recv_codes_quad_kernel for one p >= 64, recv_quad_batch_kernel
//    for a batch, recv_codes_kernel for tiny p) then read, per rank r and round i, the codes of
//    the two ranks that bound the window of Algorithm 4 (r - skips[i+1], r - skips[i];
//    consecutive threads read consecutive words) and find the largest new block of the window
//    from the two codes alone: walking down from the first level where they differ, every step
//    yields one "head" (a rank whose baseblock is that level) and a run of low blocks; the rounds
//    whose windows reach only a few ranks back read them from a table of the tile's baseblock
//    bits in shared memory.  They write the rows rank-major and a round-major copy, from which
//    send_transpose_kernel / send_batch_kernel produce
//    sendsched[r][k] = recvsched[(r+skips[k]) mod p][k] as a transposition with row k rotated by
//    skips[k] (send_rm_kernel: sub-ranges, byte gathers and recomputation for to-processors
//    outside the range).  The kernels of a build are launched as dependents of one another
//    (bcs_common.cuh), so each is brought onto the SMs while the one before it drains.  In a
//    batch, every p up to 1024 is built by ONE CTA of fused_small_batch_kernel instead: codes,
//    a table of exact window sets over all ranks of the p, both tables, all in shared memory.
//
//  * self-contained path (no workspace).  One thread per rank runs Algorithm 4 with the range
//    search done by descending the homeranges; the send schedule is looked up in the rank-major
//    receive table where the to-processor is inside the call's range and recomputed
//    (Algorithm 5) where it is not.
#include <cstddef>
#include <mutex>
#include <type_traits>

#include "bcs_common.cuh"
#include "paper_path.cuh"

namespace bcs {
namespace {

// Scratch of bcs_build_static: lives in the library's device image, so every GPU that loads
// the library sets these bytes aside until the process ends.  In host code this name is only a
// handle for cudaGetSymbolAddress, never an address a kernel may be given.
static __device__ __align__(256) unsigned char g_static_scratch[BCS_STATIC_WORKSPACE_BYTES];

// ================================================================ self-contained path
// (Algorithms 2-4 per rank: paper_path.cuh)
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
// Skip codes of many consecutive ranks at the price of one scan.  The greedy scan of rank g+e
// (0 < e < 32) decides like that of g at every level until the one where the remainder R of g
// has R < skips[k] <= R + e: there g+e takes skips[k] and keeps R + e - skips[k] < 31, while g
// does not.  From such a level on g takes every level of the scanned range: with R = skips[k] - d,
// 1 <= d <= 31, and skips[k] = 2 skips[k-1] or 2 skips[k-1] - 1, the remainder before level j < k
// is skips[j+1] - d' with d' <= d + (k - 1 - j) < 55 <= skips[j] (the scanned levels are 8 and up,
// skips[8] > 128), which is at least skips[j].  So a block has at most one such level; a second
// one is still recorded as a flag that sends the 32 ranks to the plain scan.  The levels below
// kCodesLow come from a table in shared memory, low[v] = code of v < skips[kCodesLow] over those
// levels, which also holds the codes of the remainders below 31.
constexpr int kCodesThreads = 256;
constexpr int kCodesSub = 32;                                   // consecutive ranks scanned as one
constexpr int kCodesCta = kCodesThreads * kCodesSub;            // ranks per CTA
constexpr int kCodesLow = 8;
// Ranks per scan in the kernel of one p: 32 where the kernel streams (4 million ranks and more:
// fewest instructions per rank), 16 for a smaller p, where its latency counts: twice the threads,
// each with half the quads to write (p = 2^20+1: 1.1 us less).
__host__ __device__ constexpr int codes_sub(int q) { return q <= 22 ? 16 : 32; }

struct BlockScan {
    uint32_t biased;   // remainder of the block's first rank, plus (ranks per block - 1)
    uint32_t code;     // its code so far
    uint32_t stay;     // ranks g .. g+stay-1 decide like g; the whole block while no level has split it
    uint32_t left;     // code, down to the splitting level, of the ranks that left there
    uint32_t plain;    // a second splitting level was met
};

template <int kSub = kCodesSub>
__device__ __forceinline__ void scan_level(BlockScan &b, uint32_t skip, int k)
{
    const uint32_t u = b.biased - skip;
    if (u < (uint32_t)(kSub - 1)) {                   // skip - (kSub - 1) <= remainder < skip: rare
        if (b.stay == kSub) {
            b.stay = (kSub - 1) - u;                  // = skip - remainder
            b.left = b.code | (1u << k);
        } else {
            b.plain = 1;
        }
    }
    if ((int32_t)u >= kSub - 1) {
        b.biased = u;
        b.code |= 1u << k;
    }
}

template <int kSub = kCodesSub>
__device__ __forceinline__ uint4 pack_scan(const BlockScan &b)
{
    return make_uint4(b.biased - (kSub - 1), b.code, b.stay | (b.plain << 8), b.left);
}

// Codes of the four ranks at offset e0 .. e0+3 of a block whose scan is sb (no second split).
__device__ __forceinline__ uint4 quad_codes(const uint4 sb, const uint16_t *low, uint32_t e0)
{
    const uint32_t stay = sb.z;
    uint32_t out[4];
    if (stay >= e0 + 4u || stay <= e0) {              // the four on one side of the split
        const bool with_g = stay > e0;
        const uint16_t *at = low + (with_g ? sb.x + e0 : e0 - stay);
        const uint32_t high = with_g ? sb.y : sb.w;
#pragma unroll
        for (int e = 0; e < 4; ++e) out[e] = high | at[e];
    } else {
#pragma unroll
        for (uint32_t e = 0; e < 4; ++e) {
            const bool with_g = e0 + e < stay;
            out[e] = (with_g ? sb.y : sb.w) | low[(with_g ? sb.x + e0 : e0 - stay) + e];
        }
    }
    return make_uint4(out[0], out[1], out[2], out[3]);
}

// Skip code of every rank of one p: codes[x].  A warp takes 1024 consecutive ranks: lane l
// scans the levels above the table for the 32 ranks from first + 32 l (unrolled for the q at
// hand, every skip an immediate operand from the kernel parameters), then the warp writes its
// 256 quads, lane l the quads l, l+32, ..., one 16-byte store each.
template <int kQ>
__global__ void __launch_bounds__(kCodesThreads)
codes_single_kernel(const __grid_constant__ PTable tab, uint32_t *__restrict__ codes)
{
    constexpr int kLow = kQ < kCodesLow ? kQ : kCodesLow;
    __shared__ uint16_t low[1 << kLow];
    __shared__ uint4 sub[kCodesThreads];
    grid_launch_dependents();
    if (threadIdx.x < (1u << kLow)) {
        uint32_t v = threadIdx.x, c = 0;
#pragma unroll
        for (int k = kLow - 1; k >= 0; --k) {
            if (v >= tab.s[k]) {
                v -= tab.s[k];
                c |= 1u << k;
            }
        }
        low[threadIdx.x] = (uint16_t)c;
    }
    const uint32_t lane = threadIdx.x & 31u;
    constexpr int kSub = codes_sub(kQ);
    constexpr uint32_t kSubQuads = kSub / 4;                       // quads per block: 4 or 8
    const uint32_t first = (blockIdx.x * kCodesThreads + (threadIdx.x & ~31u)) * (uint32_t)kSub;
    {
        const uint32_t g = first + kSub * lane;
        BlockScan b = {g + (kSub - 1), 0, kSub, 0, 0};
        if (g < tab.p) {
#pragma unroll
            for (int k = kQ - 1; k >= kLow; --k) scan_level<kSub>(b, tab.s[k], k);
        }
        sub[threadIdx.x] = pack_scan<kSub>(b);
    }
    __syncthreads();
    const uint32_t e0 = 4u * (lane % kSubQuads);
#pragma unroll 2
    for (uint32_t i = 0; i < kSubQuads; ++i) {
        const uint32_t g = first + 4u * (i * 32u + lane);
        if (g >= tab.p) break;
        const uint4 sb = sub[(threadIdx.x & ~31u) + i * (32u / kSubQuads) + lane / kSubQuads];
        if (sb.z < 256u && g + 4u <= tab.p) {
            *reinterpret_cast<uint4 *>(codes + g) = quad_codes(sb, low, e0);
        } else {
            for (uint32_t e = 0; e < 4 && g + e < tab.p; ++e) codes[g + e] = skip_code(tab.s, kQ, g + e);
        }
    }
}

template <int kQ>
struct CodesLauncher {
    static void launch(int q, const PTable &tab, uint32_t *codes, cudaStream_t stream)
    {
        constexpr unsigned per_cta = kCodesThreads * codes_sub(kQ);
        if (q == kQ)
            codes_single_kernel<kQ><<<(tab.p + per_cta - 1) / per_cta, kCodesThreads, 0, stream>>>(tab, codes);
        else
            CodesLauncher<kQ - 1>::launch(q, tab, codes, stream);
    }
};
template <>
struct CodesLauncher<0> {
    static void launch(int, const PTable &, uint32_t *, cudaStream_t) {}
};

inline void launch_codes(const PTable &tab, uint32_t *codes, cudaStream_t stream)
{
    CodesLauncher<BCS_MAX_Q>::launch(tab.q, tab, codes, stream);
}

// Batch: codes[g] for the flattened rank g, 8192 flattened ranks per CTA, scanned in blocks of
// 32 as above.  The CTA keeps the skips and the table of the first and of the last p it touches;
// a block of 32 that lies inside one of the two is scanned once, every other block (one that
// crosses from one p to the next, or lies in a p between the two) rank by rank.
__global__ void __launch_bounds__(kCodesThreads)
codes_batch_kernel(BatchArgs ba, uint32_t *__restrict__ codes)
{
    __shared__ uint32_t skips_sh[2][kRow];
    __shared__ uint16_t low[2][1 << kCodesLow];
    __shared__ uint4 sub[kCodesThreads];
    __shared__ uint32_t seg[2];
    __shared__ int q_sh[2];
    __shared__ uint64_t edge[3];                 // rank 0 of the first p, its end, rank 0 of the last p
    grid_launch_dependents();
    const uint64_t g0 = (uint64_t)blockIdx.x * kCodesCta;
    const uint64_t g1 = g0 + kCodesCta < ba.total_ranks ? g0 + kCodesCta : ba.total_ranks;
    if (threadIdx.x < 32) {
        const uint32_t jf = find_segment_warp(ba.rank_off, ba.num_p, g0);
        const uint32_t jl = ba.rank_off[jf + 1] >= g1 ? jf : find_segment_warp(ba.rank_off, ba.num_p, g1 - 1);
        skips_sh[0][threadIdx.x] = ba.skips_tab[(size_t)jf * kRow + threadIdx.x];
        skips_sh[1][threadIdx.x] = ba.skips_tab[(size_t)jl * kRow + threadIdx.x];
        if (threadIdx.x == 0) {
            seg[0] = jf;
            seg[1] = jl;
            q_sh[0] = ceil_log2_fast(ba.p_list[jf]);
            q_sh[1] = ceil_log2_fast(ba.p_list[jl]);
            edge[0] = ba.rank_off[jf];
            edge[1] = ba.rank_off[jf + 1];
            edge[2] = ba.rank_off[jl];
        }
    }
    __syncthreads();
    const uint32_t jf = seg[0], jl = seg[1];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        const int levels = q_sh[t] < kCodesLow ? q_sh[t] : kCodesLow;
        if (threadIdx.x < (1u << levels)) {
            low[t][threadIdx.x] = (uint16_t)skip_code(skips_sh[t], levels, threadIdx.x);
        }
    }
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t first = g0 + (uint64_t)(threadIdx.x & ~31u) * kCodesSub;
    {
        const uint64_t g = first + kCodesSub * lane;
        // which of the two p the block lies in: the last one from its rank 0 on (all ranks up to
        // g1 are its), the first one if the block ends inside it; 2 = neither
        const uint32_t which = g >= edge[2] ? 1u : (g + kCodesSub <= edge[1] ? 0u : 2u);
        BlockScan b = {0, 0, kCodesSub, 0, which >> 1};
        if (g < g1 && which < 2u) {
            b.biased = (uint32_t)(g - edge[2 * which]) + (kCodesSub - 1);
            const int q = q_sh[which];
            for (int k = q - 1; k >= kCodesLow; --k) scan_level(b, skips_sh[which][k], k);
        }
        uint4 packed = pack_scan(b);
        packed.z |= which << 9;
        sub[threadIdx.x] = packed;
    }
    __syncthreads();
    const uint32_t e0 = 4u * (lane & 7u);
#pragma unroll 2
    for (uint32_t i = 0; i < 8; ++i) {
        const uint64_t g = first + 4u * (i * 32u + lane);
        if (g >= g1) break;
        uint4 sb = sub[(threadIdx.x & ~31u) + i * 4u + (lane >> 3)];
        if ((sb.z & 256u) == 0 && g + 4 <= g1) {
            const uint16_t *table = low[sb.z >> 9];
            sb.z &= 255u;
            *reinterpret_cast<uint4 *>(codes + g) = quad_codes(sb, table, e0);
        } else {
            for (uint32_t e = 0; e < 4 && g + e < g1; ++e) {
                const uint32_t j = find_segment(ba.rank_off, jf, jl, g + e);
                codes[g + e] = skip_code(ba.skips_tab + (size_t)j * kRow, ceil_log2_fast(ba.p_list[j]),
                                         (uint32_t)(g + e - ba.rank_off[j]));
            }
        }
    }
}

// Batch of small p (a few thousand ranks each or fewer, where most blocks of 32 would cross from
// one p to the next): codes[g] for the flattened rank g, 1024 flattened ranks per CTA.  A CTA
// inside one p scans four consecutive ranks per thread, one shared-memory load of the skip per
// level for the four, and stores their codes as one 16-byte vector; a CTA that straddles several
// p finds the p of every rank.
constexpr int kCodesTile = 4 * kTile;
__global__ void __launch_bounds__(kTile)
codes_batch_flat_kernel(BatchArgs ba, uint32_t *__restrict__ codes)
{
    __shared__ uint32_t skips_sh[kRow];
    __shared__ uint32_t seg[3];                  // first and last p of the CTA, the first p itself
    __shared__ uint64_t rank0_sh;
    grid_launch_dependents();
    const uint64_t g0 = (uint64_t)blockIdx.x * kCodesTile;
    const uint64_t g1 = g0 + kCodesTile < ba.total_ranks ? g0 + kCodesTile : ba.total_ranks;
    if (threadIdx.x < 32) {
        const uint32_t jf = find_segment_warp(ba.rank_off, ba.num_p, g0);
        const uint32_t jl = ba.rank_off[jf + 1] >= g1 ? jf : find_segment_warp(ba.rank_off, ba.num_p, g1 - 1);
        skips_sh[threadIdx.x] = ba.skips_tab[(size_t)jf * kRow + threadIdx.x];
        if (threadIdx.x == 0) {
            seg[0] = jf;
            seg[1] = jl;
            seg[2] = ba.p_list[jf];
            rank0_sh = ba.rank_off[jf];
        }
    }
    __syncthreads();
    const uint32_t jf = seg[0], jl = seg[1];
    if (jf == jl) {
        const uint64_t g = g0 + 4u * threadIdx.x;
        if (g >= g1) return;
        const int q = ceil_log2_fast(seg[2]);
        uint32_t x[4], code[4] = {0, 0, 0, 0};
#pragma unroll
        for (int e = 0; e < 4; ++e) x[e] = (uint32_t)(g - rank0_sh) + e;   // ranks >= p give unused codes
        for (int k = q - 1; k >= 0; --k) {
            const uint32_t skip = skips_sh[k];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if (x[e] >= skip) {
                    x[e] -= skip;
                    code[e] |= 1u << k;
                }
            }
        }
        if (g + 4 <= g1) {
            *reinterpret_cast<uint4 *>(codes + g) = make_uint4(code[0], code[1], code[2], code[3]);
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (g + e < g1) codes[g + e] = code[e];
        }
    } else {
        for (uint64_t g = g0 + threadIdx.x; g < g1; g += kTile) {
            const uint32_t j = find_segment(ba.rank_off, jf, jl, g);
            const uint32_t p = ba.p_list[j];
            codes[g] = skip_code(ba.skips_tab + (size_t)j * kRow, ceil_log2_fast(p), (uint32_t)(g - ba.rank_off[j]));
        }
    }
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

// Second window of Algorithm 4: the ranks r - sum_{j<=i} skips[j] .. r - skips[i+1] (cyclic, the
// root contributes nothing), i.e. the `len` ranks that end at rank `below` = r - skips[i+1]
// mod p, whose code is `lower`.  len = sum_{j<=i} skips[j] - skips[i+1] + 1 is at most q + 1
// (Lemma 1), so apart from the ranks next to the root the window does not wrap and one more
// code, that of the rank just before the window, decides it.  Largest block not in B, or -1.
__device__ __forceinline__ int pick_second_window(const uint32_t *codes, const uint32_t *full,
                                                  uint32_t p, int q, uint32_t below,
                                                  uint32_t lower, uint32_t len, uint32_t B)
{
    if (len == 0) return -1;
    if (len >= p) {
        const uint32_t U = (q >= 32 ? 0xffffffffu : (1u << q) - 1u) & ~B;
        return U ? 31 - __clz(U) : -1;
    }
    if (below >= len)                      // ranks below-len+1 .. below, all >= 1
        return pick_block(codes[below - len], lower, B, full);
    // the window reaches the root: ranks p-(len-below)+1 .. p-1 (if any), then 1 .. below
    const uint32_t over = len - below;     // >= 1 ranks at or before the root
    const int b1 = over >= 2 ? pick_block(codes[p - over], full[q], B, full) : -1;
    const int b2 = below >= 1 ? pick_block(0u, lower, B, full) : -1;
    return b1 > b2 ? b1 : b2;
}

// What a round does when its first head is already in B (or its window is empty): the full
// search of the first window, then the second window.  Kept out of line: a few percent of the
// rounds come here.
__device__ __noinline__ int pick_rest(const uint32_t *codes, const uint32_t *full, uint32_t p,
                                      int q, uint32_t below, uint32_t lower, uint32_t upper,
                                      uint32_t len, uint32_t B)
{
    int blk = pick_block(lower, upper, B, full);
    if (blk < 0) blk = pick_second_window(codes, full, p, q, below, lower, len, B);
    return blk;
}

// One round of Algorithm 4 on skip codes.  The window of round i is bounded by the ranks
// r - skips[i+1] and r - skips[i] (mod p; both wrapped when i is past the home round, neither
// before it), and the first head of pick_block -- the highest level at which their codes
// differ -- is new in all but a few percent of the rounds, so that case is decided here.
struct RoundState {
    uint32_t B, upper, sum, lo_skip;
};

__device__ __forceinline__ int recv_round(const uint32_t *__restrict__ codes, const uint32_t *full,
                                          uint32_t p, int q, uint32_t r, int i, int h, int bb,
                                          uint32_t hi_skip, RoundState &st)
{
    st.sum += st.lo_skip;                                    // sum_{j<=i} skips[j] < p + q
    const uint32_t below = r - hi_skip + (r >= hi_skip ? 0u : p);   // r - skips[i+1] mod p
    const uint32_t lower = codes[below];
    const uint32_t diff = lower ^ st.upper;
    int blk = 31 - __clz(diff);                              // first head; -1 for an empty window
    const bool taken = diff == 0 || ((st.B >> blk) & 1u);
    const uint32_t upper = st.upper;
    st.upper = lower;
    st.lo_skip = hi_skip;
    if (i == h) return bb;
    if (taken) {
        blk = pick_rest(codes, full, p, q, below, lower, upper, st.sum - hi_skip + 1u, st.B);
        if (blk < 0) return BCS_BAD_ENTRY;
    }
    st.B |= 1u << blk;
    return blk - q;
}

// Algorithm 4 on skip codes: rounds 0..last of rank r of a p whose codes start at `codes`.
// kRowOut: entries go to row[0..last] (shared memory); kColOut: entry k also goes to
// col[k * col_stride] (round-major copy).  The entry of round `last` is returned.
template <bool kRowOut, bool kColOut>
__device__ __forceinline__ int recv_rounds_codes(const uint32_t *__restrict__ codes,
                                                 const uint32_t *s, const uint32_t *full,
                                                 uint32_t p, int q, uint32_t r, int last,
                                                 uint8_t *row, int8_t *col, uint64_t col_stride)
{
    const uint32_t own = codes[r];
    int h = -1, bb = 0;
    RoundState st;
    st.B = 0;
    if (r > 0) {
        h = 31 - __clz(own);          // homerange: highest term
        bb = __ffs(own) - 1;          // baseblock: lowest term (Algorithm 2)
        st.B = 1u << bb;
    }
    st.sum = 0;
    st.lo_skip = 1u;                                        // skips[0]
    st.upper = codes[r >= 1u ? r - 1u : p - 1u];          // code of r - skips[0]
    int entry = 0;
    for (int i = 0; i <= last; ++i) {
        entry = recv_round(codes, full, p, q, r, i, h, bb, s[i + 1], st);
        if (kRowOut) row[i] = (uint8_t)entry;
        if (kColOut) {
            *col = (int8_t)entry;
            col += col_stride;
        }
    }
    return entry;
}

// One p, every round searched per lane (used for p < 64, where a warp's 32 predecessors would
// wrap around the ring more than once).  recv_t: round-major copy, recv_t[k * t_stride + (r - r_begin)].
template <bool kRowOut, bool kColOut>
__global__ void __launch_bounds__(kTile)
recv_codes_kernel(PTable tab, uint64_t r_begin, uint64_t r_end,
                  const uint32_t *__restrict__ codes, int8_t *recv_out, int8_t *recv_t,
                  uint64_t t_stride)
{
    __shared__ TileShared sh;
    BatchArgs none = {};
    RankCtx c = resolve_rank<false>(sh, tab, r_begin, r_end, none);
    if (c.valid && c.q > 0) {
        int8_t *col = kColOut ? recv_t + (c.r - r_begin) : nullptr;
        uint8_t *row = kRowOut ? sh.stage + (c.entry - sh.span_begin) : nullptr;
        recv_rounds_codes<kRowOut, kColOut>(codes, c.s, c.full, c.p, c.q, c.r, c.q - 1, row, col,
                                            t_stride);
    }
    if (kRowOut) {
        __syncthreads();
        flush_span(sh.stage, 0, (uint32_t)(sh.span_end - sh.span_begin), recv_out, sh.span_begin);
    }
}

// The run table.  The windows of the rounds with skips[i+1] <= 33 (at most six rounds, i <= 5)
// reach only a few ranks back: the first window ends skips[i+1] - 1 ranks below r, the second at
// sum_{j<=i} skips[j] <= skips[i+1] + i <= 38 (every halving rounds up by at most one), and a run
// of the table adds at most 3 more to the second and none beyond skips[i+1] - 1 to the first.  So
// every baseblock those windows can contain is the lowest code bit of one of the tile's ranks or
// of the 64 ranks before the tile.  The tile keeps, for x = every one of those ranks and
// l = 0..4, the baseblock bits OR-ed over the 2^l ranks that end at x (runs of 2 and 4 from the
// single bits, runs of 8 and 16 from the runs of 4: two barriers after the one that publishes the
// bits); a window of L ranks is the union of two such runs of 2^floor(log2 L) ranks: two
// shared-memory words per window, whatever its length, at offsets that depend on p and the round
// only.  These are the rounds in which neighbouring ranks disagree about which path of the code
// search they take; the later rounds run the code search per lane.
constexpr int kRunBack = 64;                   // ranks before the tile that the run table covers
constexpr int kRunLevels = 5;                  // runs of 1, 2, 4, 8, 16 ranks

// Skips of a p from a table row in shared memory.
struct SharedSkips {
    const uint32_t *s;
    __device__ __forceinline__ uint32_t operator()(int k) const { return s[k]; }
};

// A tile of one p >= 64, four consecutive ranks per thread.  The work of a round that does not depend
// on the rank -- the address of the codes at the window's lower end, the store into the
// round-major copy -- is done once for four ranks: their four codes are four words at one
// address, their four entries one aligned 32-bit word of the copy.  A thread whose four ranks
// lie in the same homerange past the table rounds (all but a few dozen quads of a p) runs the
// rounds for the four together, with the wrap decided per quad: before the home round h every
// window bound is r - skip, after it r + p - skip.  A warp that holds any other quad (around a
// skip, next to the root, at the end of the range: a few dozen warps of a p) runs the general
// code, home round and wrap tested per rank, for all its quads.
//
// The run table of the tile is kept as four sub-tables by position mod 4:
// entry x (x = -64 .. tile-1, counted from the tile's first rank) is word
// ((x + 64) mod 4) * kQuadSub + (x + 64) / 4 of its level, so that the threads of a warp, whose
// ranks are four apart, read consecutive words whatever the distance of the window.
constexpr int kQuadThreads = 128;
constexpr int kQuadTile = 4 * kQuadThreads;                 // ranks per CTA
constexpr int kQuadSub = kQuadThreads + kRunBack / 4;       // words per sub-table
constexpr int kQuadLevelWords = 4 * kQuadSub;               // words per level
constexpr int kQuadTableRounds = 6;                         // at most six rounds have skips[i+1] <= 33

// 1 << k for k = 0..31, 0 for any other k (the hardware shift clamps its count).
__device__ __forceinline__ uint32_t bit_or_none(int k)
{
    uint32_t bit;
    asm("shl.b32 %0, 1, %1;" : "=r"(bit) : "r"(k));
    return bit;
}

// Position of the highest set bit, -1 for 0 (one instruction).
__device__ __forceinline__ int top_bit(uint32_t v)
{
    int d;
    asm("bfind.u32 %0, %1;" : "=r"(d) : "r"(v));
    return d;
}

// byte 0 of a, b, c, d as the four bytes of one word
__device__ __forceinline__ uint32_t pack_bytes(uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    return __byte_perm(__byte_perm(a, b, 0x0040), __byte_perm(c, d, 0x0040), 0x5410);
}

struct QuadConsts {
    // Table round i, word w (0, 1: the two runs that cover the first window; 2, 3: the second
    // window, or the first again), rank j of the quad: byte offset of that word from the thread's
    // word of sub-table 0, level 0.
    int32_t word[kQuadTableRounds][4][4];
    uint32_t len2[kRow];     // length of the second window of round i, or 0
    int table_rounds;        // rounds 0 .. table_rounds-1 are decided from the run table
    // bit k: the four window bounds that a quad loads at its first rank minus skips[k] start on a
    // 16-byte boundary of the codes, so that they can be loaded as one 16-byte word
    uint32_t aligned;
    // tiles that (may) hold a quad for the general code: those of the ranks skips[k], the first
    // and the last of the range; distinct, n_special <= 32 (missing one costs time, not correctness)
    uint32_t special[kRow];
    int n_special;
};

// Length of the second window of round i, sum_{j<=i} skips[j] - skips[i+1] + 1, or 0 if empty.
__host__ __device__ inline uint32_t quad_len2(const uint32_t *skips, int i)
{
    uint32_t sum = 0;
    for (int j = 0; j <= i; ++j) sum += skips[j];
    return sum >= skips[i + 1] ? sum - skips[i + 1] + 1u : 0u;
}

// Rounds 0 .. result-1 have skips[i+1] <= 33 and are decided from the run table.
__host__ __device__ inline int quad_table_rounds(const uint32_t *skips, int q)
{
    int rounds = 0;
    while (rounds < q && rounds < kQuadTableRounds && skips[rounds + 1] <= 33u) ++rounds;
    return rounds;
}

// QuadConsts::word[i][w][j] of a p with these skips.  The len >= 1 ranks that end d ranks below a
// rank are covered by two runs of 2^l ranks, l = floor(log2 len), ending d and d + len - 2^l
// ranks below: words 0, 1 for the first window (d = skips[i], len = skips[i+1] - skips[i]),
// words 2, 3 for the second (d = skips[i+1], len = quad_len2), or the first again if it is empty.
__host__ __device__ inline int32_t quad_word_offset(const uint32_t *skips, int i, int w, int j)
{
    const uint32_t lo = skips[i], hi = skips[i + 1];
    uint32_t d = lo, len = hi - lo;
    const uint32_t len2 = quad_len2(skips, i);
    if (w >= 2 && len2) {
        d = hi;
        len = len2;
    }
    int level = 0;
    while ((2u << level) <= len) ++level;
    const uint32_t back = (w & 1) ? d + len - (1u << level) : d;
    const int rel = j - (int)back;                 // position relative to the quad's first rank
    const int sub = rel & 3;
    const int quad = (rel - sub) / 4;              // exact: rel - sub is a multiple of 4
    return 4 * (level * kQuadLevelWords + sub * kQuadSub + kRunBack / 4 + quad);
}

inline QuadConsts make_quad_consts(const PTable &tab, uint64_t r_begin, uint64_t r_end)
{
    QuadConsts qc = {};
    {
        const uint64_t count = r_end - r_begin;
        auto add = [&](uint64_t tile) {
            for (int m = 0; m < qc.n_special; ++m)
                if (qc.special[m] == tile) return;
            if (qc.n_special < kRow) qc.special[qc.n_special++] = (uint32_t)tile;
        };
        if (count) {
            add(0);
            for (int k = 1; k < tab.q; ++k)
                if (tab.s[k] >= r_begin && tab.s[k] < r_end) add((tab.s[k] - r_begin) / kQuadTile);
            add((count - 1) / kQuadTile);
        }
    }
    for (int i = 0; i < tab.q; ++i) qc.len2[i] = quad_len2(tab.s, i);
    qc.table_rounds = quad_table_rounds(tab.s, tab.q);
    // quads start at ranks r_begin + multiples of 4, the codes at a 16-byte boundary
    for (int k = 0; k <= tab.q; ++k) {
        if ((((uint32_t)r_begin - tab.s[k]) & 3u) == 0) qc.aligned |= 1u << k;
    }
    for (int i = 0; i < qc.table_rounds; ++i)
        for (int w = 0; w < 4; ++w)
            for (int j = 0; j < 4; ++j) qc.word[i][w][j] = quad_word_offset(tab.s, i, w, j);
    return qc;
}

// Where a quad tile reads the constants of its p from: the kernel parameters (single p:
// constant-bank operands) ...
struct ParamEnv {
    const PTable &tab;
    const QuadConsts &qc;
    __device__ __forceinline__ uint32_t skip(int k) const { return tab.s[k]; }
    __device__ __forceinline__ int word(int i, int w, int j) const { return qc.word[i][w][j]; }
    __device__ __forceinline__ uint32_t len2(int i) const { return qc.len2[i]; }
    __device__ __forceinline__ int table_rounds() const { return qc.table_rounds; }
};
// ... or shared memory (batch: the CTA computes them for the p of its tile).
struct SharedEnv {
    const uint32_t *s;
    const QuadConsts *qc;
    __device__ __forceinline__ uint32_t skip(int k) const { return s[k]; }
    __device__ __forceinline__ int word(int i, int w, int j) const { return qc->word[i][w][j]; }
    __device__ __forceinline__ uint32_t len2(int i) const { return qc->len2[i]; }
    __device__ __forceinline__ int table_rounds() const { return qc->table_rounds; }
};

// One tile: the n <= 512 ranks first .. first+n-1 of a p >= 64 (first may exceed p for the
// threads past the end of a range: taken mod p), four per thread; all 128 threads must call.
// codes: skip codes of this p; stage: where the tile's rank-major rows start in shared memory;
// col_tile: byte of the tile's first rank in round 0 of the round-major copy, rounds t_stride
// bytes apart (kPackedCol: both multiples of 4, so that the four entries of a quad and round are
// stored as one word).
template <bool kRowOut, bool kColOut, bool kPackedCol, bool kWideLoads, bool kWordRows, class Env>
__device__ __forceinline__ void quad_tile(const Env env, const uint32_t *full_sh, uint32_t p, int q,
                                          uint64_t first, uint32_t n,
                                          const uint32_t *__restrict__ codes, uint8_t *stage,
                                          int8_t *col_tile, uint64_t t_stride,
                                          uint32_t (&runs)[kRunLevels][kQuadLevelWords])
{
    const uint32_t t = threadIdx.x;
    // ranks of the quad mod p (defined for every thread, also past the end of the range: the
    // table entries of such ranks are never read for a rank of the range)
    uint32_t r[4], c[4], B[4];
    {
        uint64_t wrapped = first + 4u * t;
        while (wrapped >= p) wrapped -= p;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            r[j] = (uint32_t)wrapped + j;
            if (r[j] >= p) r[j] -= p;
            c[j] = codes[r[j]];
            B[j] = c[j] & (0u - c[j]);                         // baseblock as a bit, 0 for the root
            runs[0][j * kQuadSub + kRunBack / 4 + t] = B[j];
        }
        if (t < kRunBack / 4) {                                // the 64 ranks before the tile, mod p (p >= 64)
            uint64_t back = first + 4u * t + p - kRunBack;
            while (back >= p) back -= p;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                uint32_t x = (uint32_t)back + j;
                if (x >= p) x -= p;
                const uint32_t cx = codes[x];
                runs[0][j * kQuadSub + t] = cx & (0u - cx);
            }
        }
    }
    __syncthreads();
    // Runs of 2 and 4 from the single bits, then runs of 8 and 16 from the runs of 4; entry x of
    // level l is complete from x = -64 + 2^l - 1 on, and nothing before x = -41 is ever read.
    // `slot` is the thread's word in the sub-tables: its own quad, or a quad of the ranks before the tile.
    auto build_narrow = [&](uint32_t slot, uint32_t b0, uint32_t b1, uint32_t b2, uint32_t b3) {
        const uint32_t m1 = runs[0][3 * kQuadSub + slot - 1];  // the three ranks before the quad
        const uint32_t m2 = runs[0][2 * kQuadSub + slot - 1];
        const uint32_t m3 = runs[0][1 * kQuadSub + slot - 1];
        runs[1][0 * kQuadSub + slot] = b0 | m1;
        runs[1][1 * kQuadSub + slot] = b1 | b0;
        runs[1][2 * kQuadSub + slot] = b2 | b1;
        runs[1][3 * kQuadSub + slot] = b3 | b2;
        runs[2][0 * kQuadSub + slot] = b0 | m1 | m2 | m3;
        runs[2][1 * kQuadSub + slot] = b1 | b0 | m1 | m2;
        runs[2][2 * kQuadSub + slot] = b2 | b1 | b0 | m1;
        runs[2][3 * kQuadSub + slot] = b3 | b2 | b1 | b0;
    };
    build_narrow(kRunBack / 4 + t, B[0], B[1], B[2], B[3]);
    if (t >= 1u && t < kRunBack / 4)
        build_narrow(t, runs[0][t], runs[0][kQuadSub + t], runs[0][2 * kQuadSub + t], runs[0][3 * kQuadSub + t]);
    __syncthreads();
    auto build_wide = [&](uint32_t slot) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t *four = &runs[2][j * kQuadSub + slot];   // runs of 4 ending at x, x-4, x-8, x-12
            const uint32_t eight = four[0] | four[-1];
            runs[3][j * kQuadSub + slot] = eight;
            runs[4][j * kQuadSub + slot] = eight | four[-2] | four[-3];
        }
    };
    build_wide(kRunBack / 4 + t);
    if (t >= 4u && t < kRunBack / 4) build_wide(t);
    __syncthreads();
    const char *mine = reinterpret_cast<const char *>(&runs[0][t]);
    auto word = [&](int byte_offset) { return *reinterpret_cast<const uint32_t *>(mine + byte_offset); };
    uint8_t *row0 = stage + 4u * t * (uint32_t)q;              // rows of the quad: row0 + j * q
    int8_t *col0 = kColOut ? col_tile + 4u * t : nullptr;      // the quad's four bytes of round 0
    const int first_lane_round = env.table_rounds();
    const int h0 = 31 - __clz(c[0]);                           // -1 for the root
    const bool together = 4u * t + 4u <= n && r[0] != 0u && r[3] == r[0] + 3u &&
                          h0 == 31 - __clz(c[3]) && h0 >= first_lane_round;
    // One path for a whole warp (no divergence inside it): the general one if any of its quads
    // needs it -- in the first tile, the last, and the tiles in which a homerange starts.  Neither
    // path has a barrier, so the other warps of such a tile keep the fast one.
    const bool empty = 4u * t >= n;
    if (__any_sync(0xffffffffu, !empty && !together)) {
        // Four ranks, each with its own homerange, wrap and validity: the table rounds with the
        // home round tested per rank, then recv_round for every rank and round.
        int h[4], bb[4];
        RoundState st[4];
        bool valid[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            valid[j] = 4u * t + j < n;
            h[j] = -1;
            bb[j] = 0;
            st[j].B = 0;
            if (r[j] > 0) {
                h[j] = 31 - __clz(c[j]);
                bb[j] = __ffs(c[j]) - 1;
                st[j].B = B[j];
            }
        }
        uint32_t sum = 0;
        for (int i = 0; i < first_lane_round; ++i) {
            sum += env.skip(i);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t free_blocks = ~st[j].B;
                uint32_t U = (word(env.word(i, 0, j)) | word(env.word(i, 1, j))) & free_blocks;
                const uint32_t U2 = (word(env.word(i, 2, j)) | word(env.word(i, 3, j))) & free_blocks;
                if (U == 0) U = U2;
                const int lead = __clz(U);
                uint32_t bit = U ? 0x80000000u >> lead : 0u;
                int entry = U ? 31 - q - lead : BCS_BAD_ENTRY;
                if (i == h[j]) {
                    entry = bb[j];
                    bit = 0;
                }
                st[j].B |= bit;
                if (kRowOut) row0[j * q + i] = (uint8_t)entry;
                if (kColOut && valid[j]) col0[(uint64_t)i * t_stride + j] = (int8_t)entry;
            }
        }
        if (first_lane_round < q) {
            const uint32_t edge = env.skip(first_lane_round);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                st[j].sum = sum;
                st[j].lo_skip = edge;
                st[j].upper = codes[r[j] - edge + (r[j] >= edge ? 0u : p)];
            }
            for (int i = first_lane_round; i < q; ++i) {
                const uint32_t hi_skip = env.skip(i + 1);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int entry = recv_round(codes, full_sh, p, q, r[j], i, h[j], bb[j], hi_skip, st[j]);
                    if (kRowOut) row0[j * q + i] = (uint8_t)entry;
                    if (kColOut && valid[j]) col0[(uint64_t)i * t_stride + j] = (int8_t)entry;
                }
            }
        }
    } else if (!empty) {
        // ---- the four ranks together: same homerange h0, no home round among the table rounds
        // kPackedCol: col_tile and t_stride are multiples of 4, the four entries of a round are one word
        int8_t *col = col0;
        int i = 0;
        // Row bytes.  A thread's rows are q bytes apart in the staging buffer and its neighbour's
        // 4q bytes further on: for an even q the byte stores of a warp hit only 32 / gcd(q, 32)
        // banks (a quarter of the bandwidth at q = 20 or 28, a sixteenth at q = 16).  Rows of a q
        // that is a multiple of 4 are whole words, so (kWordRows) every row's entries are shifted
        // into a register instead and stored as one word after every fourth round: a quarter of
        // the conflicting stores (q = 28: 32 -> 38 G ranks/s).  The same for q = 4m + 2, where two
        // rows share a word and half the bandwidth is lost, did not pay (30.2 instead of 28.7 ms
        // for the receive rows of p = 2^30-1).  Every round of the quad, in order, goes through
        // put_rows.
        uint32_t acc[4] = {0u, 0u, 0u, 0u};
        auto put_rows = [&](const int round, const uint32_t (&entry)[4]) {
            if (kRowOut) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (kWordRows) {
                        acc[j] = __funnelshift_r(acc[j], entry[j], 8);    // (acc >> 8) | (entry << 24)
                        if ((round & 3) == 3) *reinterpret_cast<uint32_t *>(row0 + j * q + (round - 3)) = acc[j];
                    } else {
                        row0[j * q + round] = (uint8_t)entry[j];
                    }
                }
            }
        };
#pragma unroll
        for (int unrolled = 0; unrolled < kQuadTableRounds; ++unrolled) {
            if (unrolled >= first_lane_round) break;           // uniform over the grid
            i = unrolled;
            uint32_t entry[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t free_blocks = ~B[j];
                uint32_t U = (word(env.word(unrolled, 0, j)) | word(env.word(unrolled, 1, j))) & free_blocks;
                const uint32_t U2 = (word(env.word(unrolled, 2, j)) | word(env.word(unrolled, 3, j))) & free_blocks;
                if (U == 0) U = U2;
                const int lead = top_bit(U);                   // -1 when there is no new block at all
                B[j] |= bit_or_none(lead);
                entry[j] = U ? (uint32_t)(lead - q) : (uint32_t)BCS_BAD_ENTRY;
            }
            put_rows(unrolled, entry);
            if (kColOut) {
                if (kPackedCol) {
                    *reinterpret_cast<uint32_t *>(col) = pack_bytes(entry[0], entry[1], entry[2], entry[3]);
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j) col[j] = (int8_t)entry[j];
                }
                col += t_stride;
            }
            i = unrolled + 1;
        }
        // Per-lane rounds.  upper[j]: code of r[j] - skips[i]; lower[j]: code of r[j] - skips[i+1].
        uint32_t upper[4], lower[4];
        // The four bounds of a quad are four consecutive words.  Where they start in their 16-byte
        // group is the same for all quads of a launch (the ranks of quads are multiples of 4
        // apart); where they fill the group -- skips that are multiples of 4, e.g. the powers of
        // two of a p just below one -- they come as ONE 16-byte load, which touches a quarter of
        // the L1 sectors of four one-word loads with the lanes 16 bytes apart.  kWideLoads: the
        // host has checked that this holds for every round before the home round of any rank of
        // the launch, and those rounds load 16 bytes unconditionally.  (A test per round, for a p
        // with only some such skips, was compiled into both kinds of loads under a predicate: the
        // four one-word loads were issued, switched off, in every round -- 4 % of the kernel's
        // issue slots.)  The rounds past the home round load word by word: p is rarely a multiple
        // of 4 further on.
        auto load4 = [&](uint32_t (&dst)[4], uint32_t from, int k, auto wide) {
            const uint32_t *src = codes + (from - env.skip(k));
            if (decltype(wide)::value) {
                const uint4 v = *reinterpret_cast<const uint4 *>(src);
                dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w;
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) dst[j] = src[j];
            }
        };
        uint8_t *out = row0 + i;
        auto store_round = [&](const int (&entry)[4]) {
            if (kRowOut) {
                if (kWordRows) {
                    const bool full = (reinterpret_cast<uintptr_t>(out) & 3u) == 3u;   // round & 3 == 3: row0 is word-aligned
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        acc[j] = __funnelshift_r(acc[j], (uint32_t)entry[j], 8);
                        if (full) *reinterpret_cast<uint32_t *>(out + j * q - 3) = acc[j];
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j) out[j * q] = (uint8_t)entry[j];
                }
                ++out;
            }
            if (kColOut) {
                if (kPackedCol) {
                    *reinterpret_cast<uint32_t *>(col) = pack_bytes((uint32_t)entry[0], (uint32_t)entry[1],
                                                                    (uint32_t)entry[2], (uint32_t)entry[3]);
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j) col[j] = (int8_t)entry[j];
                }
                col += t_stride;
            }
        };
        // rounds i .. end-1 with the window bounds at from - skip (from = r[0] or r[0] + p)
        auto rounds_until = [&](int end, uint32_t from, auto aligned_skips) {
            if (i >= end) return;
            uint32_t ahead[4];
            load4(ahead, from, i + 1, aligned_skips);
            // (unrolled twice only with the 16-byte loads: with the one-word loads the single
            // body was 2-3 % faster at every size measured)
#pragma unroll(kWideLoads ? 2 : 1)
            for (; i < end; ++i) {
                const uint32_t below = from - env.skip(i + 1);
#pragma unroll
                for (int j = 0; j < 4; ++j) lower[j] = ahead[j];
                if (i + 1 < end) load4(ahead, from, i + 2, aligned_skips);
                // The first head of each of the four windows and B with its bit; B unchanged means
                // that the head is already taken or the window empty.  ONE test whether that holds
                // for any of the four: the four chains stay free of branches.
                int blk[4];
                uint32_t with[4];
                bool taken = false;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    blk[j] = top_bit(lower[j] ^ upper[j]);     // -1 for an empty window
                    with[j] = B[j] | bit_or_none(blk[j]);
                    taken |= with[j] == B[j];
                }
                if (taken) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if (with[j] == B[j]) {
                            // The usual case, decided here: the first head is taken and the search
                            // of pick_block ends at its second step, with a new block in the run
                            // of low blocks behind the head.  Everything else: the full search.
                            const uint32_t diff = lower[j] ^ upper[j];
                            const uint32_t below_head = (1u << (blk[j] & 31)) - 1u;
                            const uint32_t rest = upper[j] & below_head;
                            const uint32_t low = rest ? (2u << (31 - __clz(rest))) - 1u : 0u;
                            const uint32_t diff2 = (lower[j] & below_head) ^ full_sh[blk[j] & 31];
                            const uint32_t fresh = low & ~B[j];
                            int b;
                            if (diff != 0 && fresh != 0 && (diff2 == 0 || (0x80000000u >> __clz(diff2)) <= low))
                                b = 31 - __clz(fresh);
                            else
                                b = pick_rest(codes, full_sh, p, q, below + j, lower[j], upper[j],
                                              env.len2(i), B[j]);
                            blk[j] = b >= 0 ? b : BCS_BAD_ENTRY + q;   // entry BCS_BAD_ENTRY, no bit
                            with[j] = B[j] | bit_or_none(blk[j]);
                        }
                    }
                }
                int entry[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    B[j] = with[j];
                    entry[j] = blk[j] - q;
                    upper[j] = lower[j];
                }
                store_round(entry);
            }
        };
        load4(upper, r[0], i, std::integral_constant<bool, kWideLoads>());   // i <= h0: skips[i] <= r[0]
        rounds_until(h0, r[0], std::integral_constant<bool, kWideLoads>());
        {                                                      // home round: the baseblocks themselves
            int entry[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) entry[j] = __ffs(c[j]) - 1;
            store_round(entry);
            load4(upper, r[0] + p, h0 + 1, std::false_type());    // r[3] < skips[h0+1]
            i = h0 + 1;
        }
        rounds_until(q, r[0] + p, std::false_type());
    }
}

// The quad tile for a range of one p >= 64.  kRowOut: rank-major rows; kColOut: round-major copy;
// kWideLoads, kWordRows: see load4 and put_rows in quad_tile (picked per launch by launch_recv_quad).
template <bool kRowOut, bool kColOut, bool kWideLoads, bool kWordRows>
__global__ void __launch_bounds__(kQuadThreads, 8)
recv_codes_quad_kernel(const __grid_constant__ PTable tab, const __grid_constant__ QuadConsts qc,
                       uint64_t r_begin, uint64_t r_end, const uint32_t *__restrict__ codes,
                       int8_t *recv_out, int8_t *recv_t, uint64_t t_stride)
{
    __shared__ __align__(16) uint8_t stage[kQuadTile * BCS_MAX_Q];
    __shared__ uint32_t full_sh[kRow];
    __shared__ uint32_t runs[kRunLevels][kQuadLevelWords];
    grid_launch_dependents();
    const uint32_t t = threadIdx.x;
    if (t < kRow) full_sh[t] = tab.full[t];                    // read after the first barrier
    const uint32_t p = tab.p;
    const int q = tab.q;
    const uint64_t count = r_end - r_begin;
    // The first CTAs of the grid take the tiles that run the general code (listed by the host):
    // they last longer, so they start first; the others skip a listed tile.
    uint64_t tile = blockIdx.x;
    if (blockIdx.x < (uint32_t)qc.n_special) {
        tile = qc.special[blockIdx.x];
    } else {
        tile -= (uint32_t)qc.n_special;
        if (__syncthreads_or(t < (uint32_t)qc.n_special && qc.special[t] == tile)) return;
    }
    grid_dependency_wait();                                    // the codes are complete from here on
    const uint64_t g0 = tile * kQuadTile;
    const uint32_t n = (uint32_t)(count - g0 < (uint64_t)kQuadTile ? count - g0 : (uint64_t)kQuadTile);
    // g0 and t_stride are multiples of 4 and recv_t is 16-byte aligned: packed column stores
    quad_tile<kRowOut, kColOut, true, kWideLoads, kWordRows>(ParamEnv{tab, qc}, full_sh, p, q, r_begin + g0, n, codes, stage,
                                      kColOut ? recv_t + g0 : nullptr, t_stride, runs);
    if (kRowOut) {
        const uint32_t len = n * (uint32_t)q;                  // the tile's rows start at byte g0 * q: 16-byte aligned
        if ((len & 15u) == 0) {
            flush_span_bulk(stage, len, recv_out, g0 * (uint64_t)q);
        } else {                                               // ragged last tile
            __syncthreads();
            flush_span(stage, 0, len, recv_out, g0 * (uint64_t)q);
        }
    }
}

// Batch: the tiles of 512 ranks start anew with every p (the host's plan gives the prefix sums of
// the tiles per p), so a CTA works inside ONE p: the quad tile with that p's constants computed
// into shared memory when p >= 64, the per-lane search for the ranks of a smaller p.  The round-
// major copy of a p has every round padded to a multiple of 16 bytes, so that the four entries of
// a quad and round are one aligned word there as in the single-p kernel; the tile's rows start at
// any byte of the output (staged shifted by that byte's offset in its 16-byte group).
struct QuadBatchShared {
    uint32_t skips[kRow], full[kRow];
    QuadConsts qc;
    uint32_t j, p;                          // index of the tile's p in the list; the p itself
    uint64_t tile0, rank0, entry0, copy0;   // of that p: first tile, flattened rank 0, first byte, copy
    __align__(16) uint8_t stage_pad[16];    // (readable bytes before the staging buffer)
    __align__(16) uint8_t stage[kQuadTile * BCS_MAX_Q + 16];
    uint32_t runs[kRunLevels][kQuadLevelWords];
};

template <bool kColOut>
__global__ void __launch_bounds__(kQuadThreads, 6)
recv_quad_batch_kernel(BatchArgs ba, const uint32_t *__restrict__ codes, int8_t *recv_out,
                       int8_t *recv_t)
{
    __shared__ QuadBatchShared sh;
    grid_launch_dependents();
    const uint32_t t = threadIdx.x;
    if (t < 32) {
        const uint32_t j = find_segment_warp(ba.tile_off, ba.num_p, blockIdx.x);
        if (t == 0) {
            sh.j = j;
            sh.p = ba.p_list[j];
            sh.tile0 = ba.tile_off[j];
            sh.rank0 = ba.rank_off[j];
            sh.entry0 = ba.entry_off[j];
            sh.copy0 = ba.copy_off[j];
        }
    }
    __syncthreads();
    const uint32_t j = sh.j, p = sh.p;
    const int q = ceil_log2_fast(p);
    if (q == 0) return;                                            // p == 1: a tile without entries
    const uint32_t first = (uint32_t)(blockIdx.x - sh.tile0) * kQuadTile;
    const uint32_t n = p - first < (uint32_t)kQuadTile ? p - first : (uint32_t)kQuadTile;
    const uint64_t span_begin = sh.entry0 + (uint64_t)first * (uint64_t)q;
    const uint32_t shift = (uint32_t)(span_begin & 15u);
    const uint64_t pitch = align_up(p, 16);
    const uint32_t *skips = ba.skips_tab + (size_t)j * kRow;       // the constants of this p
    int8_t *col_tile = kColOut ? recv_t + sh.copy0 + first : nullptr;
    uint32_t lag = 0;                                              // see below
    if (p >= 64u) {                                                // uniform over the CTA
        if (t < kRow) {
            sh.skips[t] = skips[t];
            sh.full[t] = ba.full_tab[(size_t)j * kRow + t];
            if (t < (uint32_t)q) sh.qc.len2[t] = quad_len2(skips, (int)t);
            if (t == 0) sh.qc.table_rounds = quad_table_rounds(skips, q);
        } else if (t < kRow + kQuadTableRounds * 16 && (int)((t - kRow) >> 4) < q) {
            const uint32_t e = t - kRow;                           // round e / 16, word (e / 4) % 4, rank e % 4
            sh.qc.word[e >> 4][(e >> 2) & 3u][e & 3u] = quad_word_offset(skips, (int)(e >> 4), (int)((e >> 2) & 3u), (int)(e & 3u));
        }
        grid_dependency_wait();                                    // the codes are complete from here on
        // (the tile's first barrier comes before anything above is read)
        if ((q & 3) == 0) {
            // rows of whole words are stored word by word (see put_rows): they must start on a
            // word in shared memory, `lag` bytes before their place in the output's 16-byte group
            lag = shift & 3u;
            quad_tile<true, kColOut, true, false, true>(SharedEnv{sh.skips, &sh.qc}, sh.full, p, q, first, n,
                                                        codes + sh.rank0, sh.stage + (shift - lag), col_tile, pitch,
                                                        sh.runs);
        } else {
            quad_tile<true, kColOut, true, false, false>(SharedEnv{sh.skips, &sh.qc}, sh.full, p, q, first, n,
                                                         codes + sh.rank0, sh.stage + shift, col_tile, pitch, sh.runs);
        }
    } else {
        grid_dependency_wait();
        if (t < n)
            recv_rounds_codes<true, kColOut>(codes + sh.rank0, skips, ba.full_tab + (size_t)j * kRow, p, q, t, q - 1,
                                             sh.stage + shift + t * (uint32_t)q, kColOut ? col_tile + t : nullptr, pitch);
    }
    __syncthreads();
    if (lag != 0)
        flush_span_lagging(sh.stage, shift, lag, n * (uint32_t)q, recv_out, span_begin);
    else
        flush_span(sh.stage, shift, n * (uint32_t)q, recv_out, span_begin);
}

// Batch, p <= kFusedMaxP: ONE CTA builds both tables of a p, everything in shared memory.
// With all p ranks on chip the windows of Algorithm 4 are looked up as exact block sets, whatever
// their length: run[l][x] holds the baseblock bits of the 2^l ranks that end at x (cyclically; the
// root contributes no bit), built level by level from the ranks' own bits, and a window of L ranks
// is the union of the two runs of 2^floor(log2 L) ranks at its ends.  So every round of every rank
// is two (or, when the first window holds nothing new, four) 16-bit loads and a leading-bit
// search, with no case for the root, the wrap or the homeranges; the send rows are the lookup
// sendsched[r][k] = recvsched[(r+skips[k]) mod p][k] in the staged receive rows.  No workspace,
// one launch for any number of such p (the plan gives them no tiles, so the tiled kernels never
// see them); CTAs of larger p return at once.  The last p of the list come first: lists are
// often ascending and the largest p take longest.
constexpr int kFusedThreads = 256;
struct FusedShared {
    uint32_t skips[kRow];
    uint32_t len2[kFusedMaxQ];                    // length of the second window of round i
    uint8_t level1[kFusedMaxQ], level2[kFusedMaxQ];   // floor(log2) of the two window lengths
    uint16_t codes[kFusedMaxP];
    union alignas(16) {                           // (the staging buffers go out as 16-byte vectors)
        uint16_t run[kFusedMaxQ][kFusedMaxP];     // levels 0 .. floor(log2(p-1)) <= 9
        uint8_t send_stage[kFusedMaxP * kFusedMaxQ + 16];   // after the last round
    };
    __align__(16) uint8_t recv_stage[kFusedMaxP * kFusedMaxQ + 16];
};
static_assert(offsetof(FusedShared, send_stage) % 16 == 0 && offsetof(FusedShared, recv_stage) % 16 == 0,
              "staging buffers start on a 16-byte boundary");

template <bool kSend>
__global__ void __launch_bounds__(kFusedThreads)
fused_small_batch_kernel(BatchArgs ba, int8_t *recv_out, int8_t *send_out)
{
    __shared__ __align__(16) FusedShared sh;
    grid_launch_dependents();
    const uint32_t t = threadIdx.x;
    const uint32_t j = ba.num_p - 1u - blockIdx.x;
    const uint32_t p = ba.p_list[j];
    const int q = ceil_log2_fast(p);
    if (q == 0 || p > kFusedMaxP) {                                // uniform over the CTA
        grid_dependency_wait();                                    // see the end of the kernel
        return;
    }
    const uint32_t *skips = ba.skips_tab + (size_t)j * kRow;
    if (t < kRow) sh.skips[t] = skips[t];
    if (t < (uint32_t)q) {
        const uint32_t first_len = skips[t + 1] - skips[t];        // >= 1
        const uint32_t second_len = quad_len2(skips, (int)t);
        sh.len2[t] = second_len;
        sh.level1[t] = (uint8_t)(31 - __clz(first_len));
        sh.level2[t] = (uint8_t)(second_len != 0 && second_len < p ? 31 - __clz(second_len) : 0);
    }
    for (uint32_t x = t; x < p; x += kFusedThreads) {
        const uint32_t c = skip_code(skips, q, x);
        sh.codes[x] = (uint16_t)c;
        sh.run[0][x] = (uint16_t)(c & (0u - c));                   // baseblock as a bit, 0 for the root
    }
    __syncthreads();
    const int top_level = 31 - __clz(p - 1u);                      // the longest window has p - 1 ranks
    for (int l = 1; l <= top_level; ++l) {
        const uint32_t half = 1u << (l - 1);
        for (uint32_t x = t; x < p; x += kFusedThreads)
            sh.run[l][x] = sh.run[l - 1][x] | sh.run[l - 1][x >= half ? x - half : x + p - half];
        __syncthreads();
    }
    const uint64_t entry0 = ba.entry_off[j];
    const uint32_t shift = (uint32_t)(entry0 & 15u);
    const uint32_t all = (1u << q) - 1u;
    // A thread has the ranks t, t + 256, ... (at most four); the rounds are the outer loop, so
    // that what a round needs of its skips and window lengths is worked out once for the four.
    constexpr int kMine = (int)(kFusedMaxP / kFusedThreads);
    uint32_t B[kMine];
    int h[kMine], bb[kMine];
#pragma unroll
    for (int m = 0; m < kMine; ++m) {
        const uint32_t r = t + (uint32_t)m * kFusedThreads;
        const uint32_t c = r < p ? sh.codes[r] : 0u;
        h[m] = r < p ? 31 - __clz(c) : -2;                         // homerange; -1 for the root
        bb[m] = __ffs(c) - 1;                                      // baseblock (Algorithm 2)
        B[m] = c & (0u - c);
    }
    uint8_t *const rows = sh.recv_stage + shift + t * (uint32_t)q;
    for (int i = 0; i < q; ++i) {
        const uint32_t lo = sh.skips[i], hi = sh.skips[i + 1];
        const uint32_t len1 = hi - lo, second_len = sh.len2[i];
        const int l1 = sh.level1[i], l2 = sh.level2[i];
        const uint32_t back1 = len1 - (1u << l1), back2 = second_len - (1u << l2);
        const uint16_t *const run1 = sh.run[l1], *const run2 = sh.run[l2];
        const uint32_t hi_back = hi == p ? 0u : hi;                // r - p is rank r
#pragma unroll
        for (int m = 0; m < kMine; ++m) {
            const uint32_t r = t + (uint32_t)m * kFusedThreads;
            if (r >= p) break;
            int entry = bb[m];
            if (i != h[m]) {
                // the baseblock bits of the len1 ranks that end at rank e = r - lo
                const uint32_t e = r >= lo ? r - lo : r + p - lo;
                uint32_t U = ((uint32_t)run1[e] | (uint32_t)run1[e >= back1 ? e - back1 : e + p - back1]) & ~B[m];
                if (U == 0) {
                    if (second_len >= p) {
                        U = all & ~B[m];
                    } else if (second_len != 0) {
                        const uint32_t e2 = r >= hi_back ? r - hi_back : r + p - hi_back;
                        U = ((uint32_t)run2[e2] | (uint32_t)run2[e2 >= back2 ? e2 - back2 : e2 + p - back2]) & ~B[m];
                    }
                }
                const int blk = top_bit(U);
                B[m] |= bit_or_none(blk);
                entry = U ? blk - q : BCS_BAD_ENTRY;
            }
            rows[(uint32_t)m * kFusedThreads * (uint32_t)q + (uint32_t)i] = (uint8_t)entry;
        }
    }
    __syncthreads();                                               // the run table is done with
    flush_span(sh.recv_stage, shift, p * (uint32_t)q, recv_out, entry0);
    if (kSend) {
        uint8_t *const out = sh.send_stage + shift + t * (uint32_t)q;
        for (int k = 0; k < q; ++k) {
            const uint32_t skip = sh.skips[k];
#pragma unroll
            for (int m = 0; m < kMine; ++m) {
                const uint32_t r = t + (uint32_t)m * kFusedThreads;
                if (r >= p) break;
                uint32_t to = r + skip;
                if (to >= p) to -= p;
                out[(uint32_t)m * kFusedThreads * (uint32_t)q + (uint32_t)k] =
                    sh.recv_stage[shift + to * (uint32_t)q + (uint32_t)k];
            }
        }
        __syncthreads();
        flush_span(sh.send_stage, shift, p * (uint32_t)q, send_out, entry0);
    }
    // Launched as a dependent of the tiled kernels (when the list has larger p too), this kernel
    // needs nothing of theirs and starts beside their tail; but it must not END before them, or
    // what follows it on the stream could start while they still write.
    grid_dependency_wait();
}

// Send rows of a sub-range of one p from the round-major receive copy of that range;
// to-processors outside the range are recomputed from the codes (Algorithm 5).
__global__ void __launch_bounds__(kTile)
send_rm_kernel(PTable tab, uint64_t r_begin, uint64_t r_end, const uint32_t *__restrict__ codes,
               const int8_t *__restrict__ recv_t, uint64_t t_stride, int8_t *send_out)
{
    __shared__ TileShared sh;
    BatchArgs none = {};
    RankCtx c = resolve_rank<false>(sh, tab, r_begin, r_end, none);
    if (c.valid) {
        uint8_t *row = sh.stage + (c.entry - sh.span_begin);
        const int8_t *tbl = recv_t;
        const uint32_t first = (uint32_t)r_begin, width = (uint32_t)(r_end - r_begin);
        for (int k = 0; k < c.q; ++k) {
            uint32_t t = c.r + c.s[k];
            if (t >= c.p) t -= c.p;
            const uint32_t rel = t - first;          // index into the round-major row
            int v;
            if (rel < width) {
                v = tbl[rel];
            } else {
                v = recv_rounds_codes<false, false>(codes, c.s, c.full, c.p, c.q, t, k, nullptr,
                                                    nullptr, 0);
            }
            row[k] = (uint8_t)v;
            tbl += t_stride;
        }
    }
    __syncthreads();
    flush_span(sh.stage, 0, (uint32_t)(sh.span_end - sh.span_begin), send_out, sh.span_begin);
}

// Row k of the round-major send table is row k of the round-major receive copy rotated by
// skips[k] (sendsched[r][k] = recvsched[(r+skips[k]) mod p][k]), so the send rows of a run of
// ranks are a transposition with one rotation per row (and the receive rows the same with
// rotation 0).  A tile is up to 256 consecutive ranks of one p.
//   * Thread k < q brings the (rotated) bytes of round k into shared memory with one bulk copy
//     (cp.async.bulk global -> shared, completion counted on an mbarrier); the copy starts at the
//     16-byte boundary at or before the first needed byte and ends at the one at or after the
//     last (up to 15 bytes before and after the needed ones are read as well).  A round whose
//     bytes pass the end of the row (at most q tiles of a table) gets the part after the wrap
//     by plain loads.
//   * Thread j < 64 then takes the four ranks 4j..4j+3: one 32-bit word per round (two aligned
//     words and a funnel shift, as the rotation puts the tile anywhere in the word), and its 4q
//     output bytes -- q words of the rank-major rows -- are put together by byte permutations
//     with selectors known at compile time (one instantiation per q).  Shared memory sees 3 word
//     accesses per four entries instead of 8 byte accesses.
constexpr int kTrPitch = kTile + 32;        // bytes per round in shared memory: 256 + alignment slack
constexpr int kTrThreads = kTile / 4;       // threads that gather
constexpr uint32_t kWaitLimit = 1u << 22;   // polls of the mbarrier before a CTA gives up

// CTAs whose bulk load did not complete within kWaitLimit polls (they leave their tile unwritten).
__device__ unsigned long long g_wait_expired;

template <int kRounds>
struct RoundBuffer {
    __align__(128) uint8_t rounds[kRounds * kTrPitch];
    __align__(8) uint64_t bar;
    uint32_t lead[kRounds];     // offset of the tile's first byte inside its pitch row
    uint32_t wraps;             // rounds whose bytes pass the end of the row
};

// Skips from the kernel parameter (single p).
struct TableSkips {
    const PTable &tab;
    __device__ __forceinline__ uint32_t operator()(int k) const { return tab.s[k]; }
};

// All threads of the CTA call.  tbl: round 0 of the round-major table of this p (rows `stride`
// bytes apart, any alignment); the tile is ranks r0..r0+n-1 (r0 < p, n <= 256, n <= p).
// Returns false, in all threads, if the copies did not arrive within the poll limit.
template <class Skips, class Buffer>
__device__ __forceinline__ bool load_rounds(const Skips skip, uint32_t p, int q,
                                            const int8_t *__restrict__ tbl, uint64_t stride,
                                            uint32_t r0, uint32_t n, bool rotate, Buffer &rb)
{
    const uint32_t bar_addr = (uint32_t)__cvta_generic_to_shared(&rb.bar);
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar_addr), "r"(q) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        rb.wraps = 0;
    }
    grid_launch_dependents();
    __syncthreads();
    grid_dependency_wait();                                    // the round-major copy is complete
    if (threadIdx.x < (uint32_t)q) {
        const int k = threadIdx.x;
        uint32_t start = r0 + (rotate ? skip(k) : 0u);
        if (start >= p) start -= p;
        const uint64_t from = reinterpret_cast<uint64_t>(tbl) + (uint64_t)k * stride + start;
        const uint32_t mis = (uint32_t)(from & 15u);
        const uint32_t run = p - start < n ? p - start : n;    // bytes before the wrap
        const uint32_t bytes = (mis + run + 15u) & ~15u;       // <= 272, inside the row's pitch
        rb.lead[k] = mis;
        if (run < n) atomicOr(&rb.wraps, 1u << k);
        const uint32_t dst = (uint32_t)__cvta_generic_to_shared(rb.rounds + k * kTrPitch);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                     :: "r"(bar_addr), "r"(bytes) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     :: "r"(dst), "l"(from - mis), "r"(bytes), "r"(bar_addr) : "memory");
    }
    uint32_t done = 0;
    for (uint32_t poll = 0; poll < kWaitLimit && !done; ++poll)
        asm volatile("{\n\t.reg .pred ok;\n\t"
                     "mbarrier.try_wait.parity.shared::cta.b64 ok, [%1], 0;\n\t"
                     "selp.u32 %0, 1, 0, ok;\n\t}"
                     : "=r"(done) : "r"(bar_addr) : "memory");
    if (__syncthreads_or(!done)) {                             // uniform: nobody touches the tile
        if (threadIdx.x == 0) atomicAdd(&g_wait_expired, 1ull);
        return false;
    }
    if (rb.wraps) {                                            // the part after the wrap, by bytes
        for (uint32_t left = rb.wraps; left != 0; left &= left - 1u) {
            const int k = __ffs(left) - 1;
            uint32_t start = r0 + (rotate ? skip(k) : 0u);
            if (start >= p) start -= p;
            const uint32_t run = p - start;                    // < n for these rounds
            const uint8_t *src_row = reinterpret_cast<const uint8_t *>(tbl) + (uint64_t)k * stride;
            for (uint32_t j = run + threadIdx.x; j < n; j += blockDim.x)
                rb.rounds[k * kTrPitch + rb.lead[k] + j] = src_row[j - run];
        }
        __syncthreads();
    }
    return true;
}

// W[k]: the entries of round k of the ranks 4j..4j+3 of the tile.
template <int kQ, class Buffer>
__device__ __forceinline__ void load_four_ranks(const Buffer &rb, uint32_t j, uint32_t (&W)[kQ])
{
#pragma unroll
    for (int k = 0; k < kQ; ++k) {
        const uint32_t off = (uint32_t)k * kTrPitch + rb.lead[k] + 4u * j;
        const uint32_t *word = reinterpret_cast<const uint32_t *>(rb.rounds + (off & ~3u));
        W[k] = __funnelshift_r(word[0], word[1], (off & 3u) * 8u);
    }
}

// Word m of the 4q bytes of four consecutive rank-major rows: byte e is rank e / q, round e % q.
template <int kQ>
__device__ __forceinline__ uint32_t row_word(const uint32_t (&W)[kQ], int m)
{
    const int e = 4 * m;
    const uint32_t lo = __byte_perm(W[e % kQ], W[(e + 1) % kQ],
                                    (uint32_t)(e / kQ) | (uint32_t)(4 + (e + 1) / kQ) << 4);
    const uint32_t hi = __byte_perm(W[(e + 2) % kQ], W[(e + 3) % kQ],
                                    (uint32_t)((e + 2) / kQ) | (uint32_t)(4 + (e + 3) / kQ) << 4);
    return __byte_perm(lo, hi, 0x5410u);
}

// Single p: recv_t holds all p ranks of every round (rows 16-byte aligned); the CTA's tile is
// ranks r0..r0+n-1 of the range r_begin..r_begin+count-1.  rotate: send rows; otherwise the
// receive rows themselves.  The rows are written over the round buffer (after a barrier) and
// leave as one bulk store: 64 threads and 6 KB (q = 21) per 256 ranks, so the whole grid of a
// million-rank table is resident at once, and the many small CTAs per SM overlap one another's
// copies.
template <int kQ>
__global__ void __launch_bounds__(kTrThreads)
send_transpose_kernel(const __grid_constant__ PTable tab, const int8_t *__restrict__ recv_t,
                      uint64_t t_stride, int8_t *send_out, uint32_t r_begin, uint32_t count,
                      bool rotate)
{
    __shared__ RoundBuffer<kQ> rb;
    const uint32_t first = blockIdx.x * kTile;
    const uint32_t n = count - first < (uint32_t)kTile ? count - first : (uint32_t)kTile;
    if (!load_rounds(TableSkips{tab}, tab.p, kQ, recv_t, t_stride, r_begin + first, n, rotate, rb))
        return;
    uint32_t W[kQ];
    load_four_ranks(rb, threadIdx.x, W);
    __syncthreads();                                       // everyone has read: the rows take the buffer over
    uint8_t *stage = rb.rounds;
    uint32_t *rows = reinterpret_cast<uint32_t *>(stage) + threadIdx.x * kQ;   // 4q bytes start at a multiple of 4
#pragma unroll
    for (int m = 0; m < kQ; ++m) rows[m] = row_word<kQ>(W, m);
    const uint32_t len = n * (uint32_t)kQ;                 // starts at byte first * q: 16-byte aligned
    if ((len & 15u) == 0) {
        flush_span_bulk(stage, len, send_out, (uint64_t)first * (uint64_t)kQ);
    } else {                                               // ragged last tile
        __syncthreads();
        flush_span(stage, 0, len, send_out, (uint64_t)first * (uint64_t)kQ);
    }
}

// Batch: the same for a tile whose rows start at any byte.  `out` is where the tile's first row
// starts in the staging buffer; with sh = its address mod 4, word m of a thread's rows lies sh
// bytes into an aligned word, so consecutive words are funnel-shifted together and the up to
// three bytes at either end go out one by one.
using BatchRoundBuffer = RoundBuffer<BCS_MAX_Q>;

template <int kQ>
__device__ __forceinline__ void gather_rows_unaligned(const BatchRoundBuffer &rb, uint8_t *out)
{
    uint32_t W[kQ];
    load_four_ranks(rb, threadIdx.x, W);
    __syncthreads();                                          // everyone has read: `out` may lie in the round buffer
    uint8_t *mine = out + 4u * threadIdx.x * kQ;
    const uint32_t sh = (uint32_t)(__cvta_generic_to_shared(mine) & 3u);
    uint32_t *words = reinterpret_cast<uint32_t *>(mine - sh);
    uint32_t prev = 0;
#pragma unroll
    for (int m = 0; m < kQ; ++m) {
        const uint32_t cur = row_word<kQ>(W, m);
        if (m == 0 && sh != 0) {
            for (uint32_t e = 0; e + sh < 4u; ++e) mine[e] = (uint8_t)(cur >> (8u * e));
        } else {
            words[m] = __funnelshift_l(prev, cur, 8u * sh);
        }
        prev = cur;
    }
    for (uint32_t e = 0; e < sh; ++e)                         // the last sh bytes
        mine[4u * kQ - sh + e] = (uint8_t)(prev >> (8u * (4u - sh + e)));
}

template <int kQ>
struct GatherDispatch {
    static __device__ __forceinline__ void run(int q, const BatchRoundBuffer &rb, uint8_t *out)
    {
        if (q == kQ)
            gather_rows_unaligned<kQ>(rb, out);
        else
            GatherDispatch<kQ - 1>::run(q, rb, out);
    }
};
template <>
struct GatherDispatch<0> {
    static __device__ __forceinline__ void run(int, const BatchRoundBuffer &, uint8_t *) {}
};

template <int kQ>
struct TransposeLauncher {
    static void launch(const PTable &tab, const int8_t *recv_t, uint64_t t_stride, int8_t *out,
                       uint32_t r_begin, uint32_t count, bool rotate, bool dependent,
                       cudaStream_t stream)
    {
        if (tab.q == kQ)
            launch_dependent(dependent, send_transpose_kernel<kQ>, (count + kTile - 1) / kTile,
                             kTrThreads, stream, tab, recv_t, t_stride, out, r_begin, count, rotate);
        else
            TransposeLauncher<kQ - 1>::launch(tab, recv_t, t_stride, out, r_begin, count, rotate,
                                              dependent, stream);
    }
};
template <>
struct TransposeLauncher<0> {
    static void launch(const PTable &, const int8_t *, uint64_t, int8_t *, uint32_t, uint32_t, bool,
                       bool, cudaStream_t) {}
};

// dependent: the kernel before this one on the stream calls grid_launch_dependents().
inline void launch_transpose(const PTable &tab, const int8_t *recv_t, uint64_t t_stride, int8_t *out,
                             uint32_t r_begin, uint32_t count, bool rotate, bool dependent,
                             cudaStream_t stream)
{
    TransposeLauncher<BCS_MAX_Q>::launch(tab, recv_t, t_stride, out, r_begin, count, rotate,
                                         dependent, stream);
}

// Batch: 256 ranks and 64 threads per CTA, as in the single-p kernel; two CTAs per tile of the
// plan (512 ranks of one p), the second with nothing to do where a p ends in the first half.
struct SendBatchShared {
    uint32_t skips[kRow];
    uint32_t j, p;
    uint64_t tile0, entry0, copy0;
};
static_assert(BCS_MAX_Q * kTrPitch >= kTile * BCS_MAX_Q + 16, "the rows of a tile fit in its round buffer");

__global__ void __launch_bounds__(kTrThreads, 16)
send_batch_kernel(BatchArgs ba, const int8_t *__restrict__ recv_t, int8_t *send_out)
{
    __shared__ SendBatchShared sh;
    __shared__ BatchRoundBuffer rb;
    const uint32_t t = threadIdx.x;
    const uint64_t tile = blockIdx.x >> 1;
    if (t < 32) {
        const uint32_t j = find_segment_warp(ba.tile_off, ba.num_p, tile);
        sh.skips[t] = ba.skips_tab[(size_t)j * kRow + t];
        if (t == 0) {
            sh.j = j;
            sh.p = ba.p_list[j];
            sh.tile0 = ba.tile_off[j];
            sh.entry0 = ba.entry_off[j];
            sh.copy0 = ba.copy_off[j];
        }
    }
    __syncthreads();
    const uint32_t p = sh.p;
    const int q = ceil_log2_fast(p);
    const uint64_t first64 = (tile - sh.tile0) * kQuadTile + (blockIdx.x & 1u) * kTile;
    if (q == 0 || first64 >= p) return;                            // uniform over the CTA
    const uint32_t first = (uint32_t)first64;
    const uint32_t n = p - first < (uint32_t)kTile ? p - first : (uint32_t)kTile;
    const uint64_t span_begin = sh.entry0 + (uint64_t)first * (uint64_t)q;
    const uint32_t shift = (uint32_t)(span_begin & 15u);
    if (!load_rounds(SharedSkips{sh.skips}, p, q, recv_t + sh.copy0, align_up(p, 16), first, n, true, rb))
        return;
    // the rows take the round buffer over (after a barrier inside the gather): 9 KB per CTA
    GatherDispatch<BCS_MAX_Q>::run(q, rb, rb.rounds + shift);
    __syncthreads();
    flush_span(rb.rounds, shift, n * (uint32_t)q, send_out, span_begin);
}

// Launches the quad receive kernel of one p >= 64 for a range, as a dependent of the kernel
// before it on the stream.  The instantiation that loads the window bounds of the rounds before
// the home round as 16-byte words is taken when all of them are aligned (a p in the top 32nd of
// its octave, whose skips from 32 on are powers of two, and a range that starts at a multiple of
// 4): 10 % fewer L1 wavefronts and 5 % fewer issue slots than the one-word loads.
template <bool kRowOut, bool kColOut>
inline void launch_recv_quad(const PTable &tab, const QuadConsts &qc, uint64_t r_begin, uint64_t r_end,
                             const uint32_t *codes, int8_t *recv_out, int8_t *recv_t, uint64_t t_stride,
                             cudaStream_t stream)
{
    const uint64_t count = r_end - r_begin;
    const unsigned grid = (unsigned)((count + kQuadTile - 1) / kQuadTile) + (unsigned)qc.n_special;
    // bounds of every round from the first per-lane round to the last possible home round
    bool all_wide = true;
    for (int k = qc.table_rounds; k < tab.q; ++k) all_wide = all_wide && ((qc.aligned >> k) & 1u);
    // rows of a q that is a multiple of 4 are stored word by word (see put_rows)
    const bool word_rows = kRowOut && (tab.q & 3) == 0;
    auto go = [&](auto kernel) {
        launch_dependent(true, kernel, grid, kQuadThreads, stream, tab, qc, r_begin, r_end, codes, recv_out, recv_t,
                         t_stride);
    };
    if (all_wide) {
        if (word_rows) go(recv_codes_quad_kernel<kRowOut, kColOut, true, kRowOut>);
        else go(recv_codes_quad_kernel<kRowOut, kColOut, true, false>);
    } else {
        if (word_rows) go(recv_codes_quad_kernel<kRowOut, kColOut, false, kRowOut>);
        else go(recv_codes_quad_kernel<kRowOut, kColOut, false, false>);
    }
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
        launch_codes(tab, ws.codes, stream);
        if ((st = launch_status()) != BCS_OK) return st;
        const bool warp_rounds = p >= 64;      // the table kernel needs 64 distinct ranks back
        const QuadConsts rc = make_quad_consts(tab, r_begin, r_end);
        if (recv_out != nullptr && send_out != nullptr) {
            if (warp_rounds)
                launch_recv_quad<true, true>(tab, rc, r_begin, r_end, ws.codes, recv_out, ws.recv_t, ws.t_stride, stream);
            else
                recv_codes_kernel<true, true><<<blocks, kTile, 0, stream>>>(
                    tab, r_begin, r_end, ws.codes, recv_out, ws.recv_t, ws.t_stride);
        } else if (recv_out != nullptr) {
            if (warp_rounds)
                launch_recv_quad<true, false>(tab, rc, r_begin, r_end, ws.codes, recv_out, nullptr, 0, stream);
            else
                recv_codes_kernel<true, false><<<blocks, kTile, 0, stream>>>(
                    tab, r_begin, r_end, ws.codes, recv_out, nullptr, 0);
        } else {
            if (warp_rounds)
                launch_recv_quad<false, true>(tab, rc, r_begin, r_end, ws.codes, nullptr, ws.recv_t, ws.t_stride, stream);
            else
                recv_codes_kernel<false, true><<<blocks, kTile, 0, stream>>>(
                    tab, r_begin, r_end, ws.codes, nullptr, ws.recv_t, ws.t_stride);
        }
        if ((st = launch_status()) != BCS_OK) return st;
        if (send_out != nullptr) {
            if (count == p)
                launch_transpose(tab, ws.recv_t, ws.t_stride, send_out, 0u, p, true, warp_rounds,
                                 stream);
            else
                send_rm_kernel<<<blocks, kTile, 0, stream>>>(tab, r_begin, r_end, ws.codes,
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

size_t bcs_prepare_workspace_bytes(uint32_t p)
{
    if (p == 0 || p > 0x7fffffffu) return 0;
    const int q = ceil_log2_u32(p);
    if (q == 0) return 0;
    return (size_t)(align_up(4ull * p, 256) + (uint64_t)q * align_up(p, 16));
}

// The two halves of bcs_prepare.  Layout of the workspace: skip codes of all p ranks, then the
// round-major copy recv_t[k * align16(p) + r].
static bcs_status prepare_check(uint32_t p, PTable *tab, const void *workspace, size_t workspace_bytes)
{
    bcs_status st = make_table(p, tab);
    if (st != BCS_OK) return st;
    if (tab->q == 0) return BCS_OK;
    if (workspace == nullptr || workspace_bytes < bcs_prepare_workspace_bytes(p)) return BCS_ERR_ARG;
    if (!aligned16(workspace)) return BCS_ERR_ALIGN;
    return BCS_OK;
}

bcs_status bcs_prepare_codes(uint32_t p, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    PTable tab;
    bcs_status st = prepare_check(p, &tab, workspace, workspace_bytes);
    if (st != BCS_OK || tab.q == 0) return st;
    launch_codes(tab, static_cast<uint32_t *>(workspace), static_cast<cudaStream_t>(cuda_stream));
    return launch_status();
}

bcs_status bcs_prepare_rows(uint32_t p, uint64_t r_begin, uint64_t r_end, int8_t *recv_out,
                            void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    bcs_status st = check_range(p, r_begin, r_end);
    if (st != BCS_OK) return st;
    PTable tab;
    st = prepare_check(p, &tab, workspace, workspace_bytes);
    if (st != BCS_OK || tab.q == 0 || r_begin == r_end) return st;
    if ((r_begin & 15u) != 0 || !aligned16(recv_out)) return BCS_ERR_ALIGN;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const uint32_t *codes = static_cast<const uint32_t *>(workspace);
    const uint64_t t_stride = align_up(p, 16);
    // round k of rank r_begin + j goes to recv_t[k * t_stride + r_begin + j]
    int8_t *recv_t = static_cast<int8_t *>(workspace) + align_up(4ull * p, 256) + r_begin;
    const uint64_t count = r_end - r_begin;
    if (p >= 64) {
        const QuadConsts qc = make_quad_consts(tab, r_begin, r_end);
        // (dependent launch: harmless when the kernel before it on the stream is not the codes kernel)
        if (recv_out != nullptr)
            launch_recv_quad<true, true>(tab, qc, r_begin, r_end, codes, recv_out, recv_t, t_stride, stream);
        else
            launch_recv_quad<false, true>(tab, qc, r_begin, r_end, codes, nullptr, recv_t, t_stride, stream);
    } else {
        const unsigned blocks = (unsigned)((count + kTile - 1) / kTile);
        if (recv_out != nullptr)
            recv_codes_kernel<true, true><<<blocks, kTile, 0, stream>>>(tab, r_begin, r_end, codes, recv_out, recv_t,
                                                                        t_stride);
        else
            recv_codes_kernel<false, true><<<blocks, kTile, 0, stream>>>(tab, r_begin, r_end, codes, nullptr, recv_t,
                                                                         t_stride);
    }
    return launch_status();
}

bcs_status bcs_prepare(uint32_t p, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    bcs_status st = bcs_prepare_codes(p, workspace, workspace_bytes, cuda_stream);
    if (st != BCS_OK) return st;
    return bcs_prepare_rows(p, 0, p, nullptr, workspace, workspace_bytes, cuda_stream);
}

bcs_status bcs_build_prepared(uint32_t p, uint64_t r_begin, uint64_t r_end, int8_t *recv_out,
                              int8_t *send_out, const void *workspace, size_t workspace_bytes,
                              void *cuda_stream)
{
    bcs_status st = check_range(p, r_begin, r_end);
    if (st != BCS_OK) return st;
    PTable tab;
    make_table(p, &tab);
    const uint64_t count = r_end - r_begin;
    if (count == 0 || tab.q == 0) return BCS_OK;
    if (recv_out == nullptr && send_out == nullptr) return BCS_ERR_ARG;
    if (workspace == nullptr || workspace_bytes < bcs_prepare_workspace_bytes(p)) return BCS_ERR_ARG;
    if (!aligned16(recv_out) || !aligned16(send_out) || !aligned16(workspace)) return BCS_ERR_ALIGN;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int8_t *recv_t = static_cast<const int8_t *>(workspace) + align_up(4ull * p, 256);
    const uint64_t t_stride = align_up(p, 16);
    if (recv_out != nullptr) {
        launch_transpose(tab, recv_t, t_stride, recv_out, (uint32_t)r_begin, (uint32_t)count, false,
                         false, stream);
        if ((st = launch_status()) != BCS_OK) return st;
    }
    if (send_out != nullptr) {
        launch_transpose(tab, recv_t, t_stride, send_out, (uint32_t)r_begin, (uint32_t)count, true,
                         recv_out != nullptr, stream);
        if ((st = launch_status()) != BCS_OK) return st;
    }
    return BCS_OK;
}

// The runs of virtual ranks (r - root) mod p of the range [r_begin, r_end): [v0, v0 + len_a) and,
// when the range passes virtual rank p - 1, [0, len_b).
struct RootedRuns {
    uint64_t v0, len_a, len_b;
};

static RootedRuns rooted_runs(uint32_t p, uint32_t root, uint64_t r_begin, uint64_t r_end)
{
    RootedRuns rr;
    const uint64_t count = r_end - r_begin;
    rr.v0 = count ? (r_begin + p - root) % p : 0;
    rr.len_a = count < p - rr.v0 ? count : p - rr.v0;
    rr.len_b = count - rr.len_a;
    return rr;
}

size_t bcs_build_rooted_workspace_bytes(uint32_t p, uint32_t root, uint64_t r_begin, uint64_t r_end)
{
    if (check_range(p, r_begin, r_end) != BCS_OK || root >= p) return 0;
    const int q = ceil_log2_u32(p);
    const RootedRuns rr = rooted_runs(p, root, r_begin, r_end);
    const size_t a = bcs_build_workspace_bytes(p, rr.v0, rr.v0 + rr.len_a);
    const size_t b = bcs_build_workspace_bytes(p, 0, rr.len_b);
    // two staging tables for the second run (used only where it lands off a 16-byte boundary)
    return (size_t)align_up(a > b ? a : b, 256) + 2 * (size_t)align_up(rr.len_b * (uint64_t)q, 256);
}

bcs_status bcs_build_rooted(uint32_t p, uint32_t root, uint64_t r_begin, uint64_t r_end,
                            int8_t *recv_out, int8_t *send_out, void *workspace,
                            size_t workspace_bytes, void *cuda_stream)
{
    bcs_status st = check_range(p, r_begin, r_end);
    if (st != BCS_OK) return st;
    if (root >= p) return BCS_ERR_RANGE;
    const int q = ceil_log2_u32(p);
    if (r_begin == r_end || q == 0) return BCS_OK;
    if (recv_out == nullptr && send_out == nullptr) return BCS_ERR_ARG;
    if (!aligned16(recv_out) || !aligned16(send_out) || !aligned16(workspace)) return BCS_ERR_ALIGN;
    const RootedRuns rr = rooted_runs(p, root, r_begin, r_end);
    const bool fast = workspace != nullptr &&
                      workspace_bytes >= bcs_build_rooted_workspace_bytes(p, root, r_begin, r_end);
    const uint64_t bytes_a = rr.len_a * (uint64_t)q, bytes_b = rr.len_b * (uint64_t)q;
    const bool staged = rr.len_b != 0 && (bytes_a & 15u) != 0;
    if (staged && !fast) return BCS_ERR_ARG;
    // workspace = [construction scratch, a multiple of 256 bytes][recv staging][send staging]
    const size_t need_a = bcs_build_workspace_bytes(p, rr.v0, rr.v0 + rr.len_a);
    const size_t need_b = bcs_build_workspace_bytes(p, 0, rr.len_b);
    const size_t build_ws = fast ? (size_t)align_up(need_a > need_b ? need_a : need_b, 256) : 0;
    st = bcs_build(p, rr.v0, rr.v0 + rr.len_a, recv_out, send_out, fast ? workspace : nullptr, build_ws,
                   cuda_stream);
    if (st != BCS_OK || rr.len_b == 0) return st;
    int8_t *recv_b = recv_out ? recv_out + bytes_a : nullptr;
    int8_t *send_b = send_out ? send_out + bytes_a : nullptr;
    if (!staged)
        return bcs_build(p, 0, rr.len_b, recv_b, send_b, fast ? workspace : nullptr, build_ws, cuda_stream);
    int8_t *stage_recv = static_cast<int8_t *>(workspace) + build_ws;
    int8_t *stage_send = stage_recv + align_up(bytes_b, 256);
    st = bcs_build(p, 0, rr.len_b, recv_out ? stage_recv : nullptr, send_out ? stage_send : nullptr,
                   workspace, build_ws, cuda_stream);
    if (st != BCS_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (recv_out && cudaMemcpyAsync(recv_b, stage_recv, bytes_b, cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
        return BCS_ERR_CUDA;
    if (send_out && cudaMemcpyAsync(send_b, stage_send, bytes_b, cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
        return BCS_ERR_CUDA;
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

size_t bcs_build_batch_workspace_bytes(uint64_t total_ranks, uint64_t total_copy)
{
    if (total_ranks == 0) return 0;
    // no p above kFusedMaxP: the fused kernel needs no scratch, and a token workspace selects it
    if (total_copy == 0) return 256;
    return (size_t)(align_up(4ull * total_ranks, 256) + total_copy);
}

bcs_status bcs_build_batch(const uint32_t *p_list_dev, const uint64_t *rank_off_dev,
                           const uint64_t *entry_off_dev, const uint64_t *tile_off_dev,
                           const uint64_t *copy_off_dev, const uint32_t *skips_tab_dev,
                           const uint32_t *full_tab_dev, uint32_t num_p, uint64_t total_ranks,
                           uint64_t total_entries, uint64_t total_tiles, uint64_t total_copy,
                           int8_t *recv_out, int8_t *send_out, void *workspace, size_t workspace_bytes,
                           void *cuda_stream)
{
    if (num_p == 0 || total_ranks == 0) return BCS_OK;
    if (p_list_dev == nullptr || rank_off_dev == nullptr || entry_off_dev == nullptr ||
        skips_tab_dev == nullptr || full_tab_dev == nullptr)
        return BCS_ERR_ARG;
    if (total_entries == 0) return BCS_OK;   // only p == 1 in the list
    if (recv_out == nullptr) return BCS_ERR_ARG;
    if (!aligned16(recv_out) || !aligned16(send_out) || !aligned16(workspace)) return BCS_ERR_ALIGN;
    const uint64_t blocks64 = (total_ranks + kTile - 1) / kTile;
    if (blocks64 > 0x7fffffffull || total_tiles > 0x3fffffffull) return BCS_ERR_UNSUPPORTED;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    BatchArgs ba = {p_list_dev, rank_off_dev, entry_off_dev, skips_tab_dev, full_tab_dev, num_p,
                    total_ranks, tile_off_dev, copy_off_dev};
    PTable none = {};
    const unsigned blocks = (unsigned)blocks64;
    bcs_status st;
    if (workspace != nullptr && tile_off_dev != nullptr && copy_off_dev != nullptr &&
        workspace_bytes >= bcs_build_batch_workspace_bytes(total_ranks, total_copy)) {
        uint32_t *codes = static_cast<uint32_t *>(workspace);
        int8_t *recv_t = static_cast<int8_t *>(workspace) + align_up(4ull * total_ranks, 256);
        // the p above kFusedMaxP, tile by tile (the plan counts tiles for these only): codes, receive
        // rows, send rows, each launched as a dependent of the kernel before it
        if (total_tiles != 0) {
            // blocks of 32 ranks scanned as one where the p are large enough for most blocks to lie
            // inside one of them
            if (total_ranks / num_p >= (uint64_t)kCodesCta)
                codes_batch_kernel<<<(unsigned)((total_ranks + kCodesCta - 1) / kCodesCta), kCodesThreads, 0, stream>>>(ba, codes);
            else
                codes_batch_flat_kernel<<<(unsigned)((total_ranks + kCodesTile - 1) / kCodesTile), kTile, 0, stream>>>(ba, codes);
            if ((st = launch_status()) != BCS_OK) return st;
            if (send_out != nullptr)
                launch_dependent(true, recv_quad_batch_kernel<true>, (unsigned)total_tiles, kQuadThreads, stream, ba,
                                 (const uint32_t *)codes, recv_out, recv_t);
            else
                launch_dependent(true, recv_quad_batch_kernel<false>, (unsigned)total_tiles, kQuadThreads, stream, ba,
                                 (const uint32_t *)codes, recv_out, (int8_t *)nullptr);
            if ((st = launch_status()) != BCS_OK) return st;
            if (send_out != nullptr) {
                launch_dependent(true, send_batch_kernel, (unsigned)(2 * total_tiles), kTrThreads, stream, ba,
                                 (const int8_t *)recv_t, send_out);
                if ((st = launch_status()) != BCS_OK) return st;
            }
        }
        // the p up to kFusedMaxP, one CTA each; needs nothing of the kernels before it and does not
        // wait for them (the host cannot tell whether the list holds such p: their CTAs return at once
        // where it does not)
        if (send_out != nullptr)
            launch_dependent(total_tiles != 0, fused_small_batch_kernel<true>, num_p, kFusedThreads, stream, ba,
                             recv_out, send_out);
        else
            launch_dependent(total_tiles != 0, fused_small_batch_kernel<false>, num_p, kFusedThreads, stream, ba,
                             recv_out, (int8_t *)nullptr);
        return launch_status();
    }
    recv_kernel<true><<<blocks, kTile, 0, stream>>>(none, 0, 0, ba, recv_out);
    if ((st = launch_status()) != BCS_OK) return st;
    if (send_out != nullptr) {
        send_kernel<true><<<blocks, kTile, 0, stream>>>(none, 0, 0, ba, recv_out, send_out);
        if ((st = launch_status()) != BCS_OK) return st;
    }
    return BCS_OK;
}

bcs_status bcs_wait_expired(uint64_t *count_host)
{
    if (count_host == nullptr) return BCS_ERR_ARG;
    unsigned long long v = 0;
    // every stream of the device, the non-blocking ones included: a copy from a symbol alone
    // would only order itself after the legacy default stream
    if (cudaDeviceSynchronize() != cudaSuccess) return BCS_ERR_CUDA;
    if (cudaMemcpyFromSymbol(&v, g_wait_expired, sizeof(v)) != cudaSuccess) return BCS_ERR_CUDA;
    *count_host = v;
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
    // the argument checks of bcs_build, repeated here so that they come before any runtime call
    if (recv_out == nullptr && send_out == nullptr) return BCS_ERR_ARG;
    if (!aligned16(recv_out) || !aligned16(send_out)) return BCS_ERR_ALIGN;
    void *scratch = static_scratch_address();
    if (scratch == nullptr) return BCS_ERR_CUDA;
    // Nothing in the scratch has to start at zero: the codes of all p ranks and the round-major
    // rows of the range are written by this call before anything reads them, so whatever an
    // earlier call left behind is simply overwritten or never looked at.
    return bcs_build(p, r_begin, r_end, recv_out, send_out, scratch, BCS_STATIC_WORKSPACE_BYTES,
                     cuda_stream);
}

}  // extern "C"
