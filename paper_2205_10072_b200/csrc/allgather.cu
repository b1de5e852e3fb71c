// Index tables of the irregular allgather (arXiv 2205.10072, Algorithm 9 without the data
// movement): for one processor r, which block of buffer[j] is packed and which is unpacked in
// every round.  Processor r treats buffer j as virtual processor (r-j) mod p of a broadcast
// rooted at j, so entry [round][j] is the send resp. receive block of that virtual processor's
// round (Algorithm 6's closed form).  A pure store stream: 8 bytes per (round, buffer).
#include "bcs_common.cuh"

namespace bcs {
namespace {

constexpr int kAgThreads = 256;   // threads per CTA; a CTA writes 256 consecutive buffers of a row
constexpr int kAgLine = 32;       // int32 elements per 128-byte line
constexpr int kAgCols = kAgThreads + kAgLine;   // buffers staged per CTA: its window slides by up to 31 from row to row
constexpr int kAgCtas = 148 * 32; // CTAs that a call aims for: the rounds are cut into as many chunks as that takes
constexpr int kAgRowBytes = kAgCols * BCS_MAX_Q + 48;

// Where the rows of a CTA's columns lie in its copy of a schedule table: column c (buffer j0 + c,
// virtual processor (hi - c) mod p) has its q entries at byte at(c, q) of the copy.
struct StagedRows {
    uint32_t first;      // columns 0..first-1 are the ranks hi, hi-1, ..., hi-first+1
    uint32_t off_a;      // byte of the row of rank hi-first+1 (rows ascend from there)
    uint32_t off_b;      // byte of the row of rank p-(n-first): the columns from `first` on are p-1, p-2, ...
    uint32_t n;
    __device__ __forceinline__ uint32_t at(uint32_t c, int q) const
    {
        return c < first ? off_a + (first - 1u - c) * (uint32_t)q : off_b + (n - 1u - c) * (uint32_t)q;
    }
};

// Rows of `table` ([p][q] int8, 16-byte aligned) for the ranks hi, hi-1, ..., hi-n+1 (mod p), brought into shared
// memory with 16-byte loads: one contiguous run of the table, or two when the ranks pass 0 (the
// second run is placed behind the first at the next 16-byte boundary plus its own alignment).
// No barrier inside: the caller synchronises before reading `rows`.
__device__ __forceinline__ StagedRows load_rows_descending(const int8_t *__restrict__ table, uint32_t p,
                                                           int q, uint32_t hi, uint32_t n,
                                                           uint8_t *rows /* kAgRowBytes, 16-byte aligned */)
{
    StagedRows sr;
    sr.n = n;
    sr.first = n <= hi + 1u ? n : hi + 1u;
    const uint32_t lo = hi + 1u - sr.first;
    const uint64_t byte_a = (uint64_t)lo * q;
    const uint32_t shift_a = (uint32_t)(byte_a & 15u);
    load_span(rows, shift_a, sr.first * (uint32_t)q, table, byte_a);
    sr.off_a = shift_a;
    sr.off_b = 0;
    if (sr.first < n) {                                    // the rest: ranks p-1, p-2, ...
        const uint32_t rest = n - sr.first;
        const uint64_t byte_b = (uint64_t)(p - rest) * q;
        const uint32_t shift_b = (uint32_t)(byte_b & 15u);
        const uint32_t region = (shift_a + sr.first * (uint32_t)q + 15u) & ~15u;
        load_span(rows + region, shift_b, rest * (uint32_t)q, table, byte_b);
        sr.off_b = region + shift_b;
    }
    return sr;
}

// Block number of Algorithm 6's closed form: entry + q * floor(i / q) - x (= entry + add); below
// 0 -> -1 (nothing is packed or unpacked), above n-1 -> n-1.
__device__ __forceinline__ int clamp_block(int b, int last) { return max(min(b, last), -1); }

// Element address (in int32 units) of out[0], of which only the position in its 128-byte line matters.
__device__ __forceinline__ uint32_t line_phase(const int32_t *out)
{
    return (uint32_t)(reinterpret_cast<uintptr_t>(out) >> 2) & (kAgLine - 1u);
}

// A thread's share of one output table.  A row of the output is p * 4 bytes long and starts
// wherever the row before it ended, so the 128-byte lines of memory cut every row at different
// buffers.  Stores that do not cover whole lines (even whole 32-byte sectors) cost the memory
// system up to 40 % of its write bandwidth, so in every row the CTA with first buffer j0 writes
// the eight lines that begin at buffers j0 + hd .. j0 + hd + 255, hd in 0..31 being the distance
// from buffer j0 of this row to the next line boundary: a warp's 32 x 16 bytes are then four whole
// lines.  (The hd buffers before the first line of a row and the up to three after the last whole
// group of four are written by loose_columns.)  Thread t takes the rows jr0 + t / 64, +4, +8, ...
// and in each of them the four buffers j0 + hd + 4 * (t % 64) .. +3.
struct QuadStream {
    const uint32_t *tbl;     // staged entries, round-major, kAgCols bytes per round
    int32_t *row;            // &out[jr * p + j0]
    uint32_t phase;          // (element address of row[0]) mod 32
    uint32_t step;           // 4 * p mod 32: what four rows add to the phase
    uint32_t avail;          // buffers from j0 to the end of the row
    __device__ __forceinline__ void init(const int8_t (*staged)[kAgCols], int32_t *out, uint64_t at,
                                         uint32_t p, uint32_t avail_)
    {
        tbl = reinterpret_cast<const uint32_t *>(&staged[0][0]);
        row = out + at;
        phase = (line_phase(out) + (uint32_t)at) & (kAgLine - 1u);
        step = (4u * p) & (kAgLine - 1u);
        avail = avail_;
    }
    // Round k of a phase: the four entries are four consecutive bytes of the staged round (two
    // aligned words and a funnel shift; the second word of the last group is the next round or
    // the pad); a byte is widened and the round's offset added by one dot-product instruction
    // (the byte times 1, the other three times 0, plus the offset).
    __device__ __forceinline__ void store(uint32_t grp, uint32_t k, int add, bool clamp, int last, uint32_t p)
    {
        const uint32_t c = ((0u - phase) & (kAgLine - 1u)) + 4u * grp;
        if (c + 4u <= avail) {
            const uint32_t *w = tbl + k * (kAgCols / 4) + (c >> 2);
            const int four = (int)__funnelshift_r(w[0], w[1], (c & 3u) * 8u);
            int4 v;
            v.x = __dp4a(four, 0x00000001, add);
            v.y = __dp4a(four, 0x00000100, add);
            v.z = __dp4a(four, 0x00010000, add);
            v.w = __dp4a(four, 0x01000000, add);
            if (clamp) {
                v.x = clamp_block(v.x, last);
                v.y = clamp_block(v.y, last);
                v.z = clamp_block(v.z, last);
                v.w = clamp_block(v.w, last);
            }
            __stcs(reinterpret_cast<int4 *>(row + c), v);
        }
        row += 4ull * p;
        phase = (phase + step) & (kAgLine - 1u);
    }
};

// The buffers of the CTA's rows that the line-aligned groups of four leave out, written one by
// one: in the first CTA of a row the hd buffers before the first line boundary (slots 0..30),
// and, where the row ends inside the CTA's window, the up to three buffers after its last whole
// group (slots 32..34).  Thread t takes slot t % 64 of the rows jr0 + t / 64, +4, ...  With
// everything == true the slot is the buffer itself (used when q < 4, i.e. p <= 8).
__device__ __forceinline__ void loose_columns(const int8_t (*tbl)[kAgCols], int32_t *__restrict__ out,
                                              uint32_t p, int q, int x, int last, uint32_t j0,
                                              uint32_t avail, uint32_t jr0, uint32_t jr1, bool everything)
{
    const uint32_t slot = threadIdx.x & 63u;
    const uint32_t base_phase = line_phase(out);
    for (uint32_t jr = jr0 + (threadIdx.x >> 6); jr < jr1; jr += 4) {
        const uint64_t at = (uint64_t)jr * p + j0;
        const uint32_t hd = (0u - (base_phase + (uint32_t)at)) & (kAgLine - 1u);
        uint32_t col = 0xffffffffu;
        if (everything) {
            col = slot;
        } else if (slot < kAgLine) {
            if (j0 == 0 && slot < hd) col = slot;
        } else if (avail >= hd && avail - hd < (uint32_t)kAgThreads) {   // the row ends in this CTA's window
            const uint32_t j = slot - kAgLine;
            if (j < ((avail - hd) & 3u)) col = hd + ((avail - hd) & ~3u) + j;
        }
        if (col < avail) {
            const uint32_t i = jr + (uint32_t)x;
            const int b = (int)tbl[i % (uint32_t)q][col] + (int)(i / (uint32_t)q) * q - x;
            out[at + col] = clamp_block(b, last);
        }
    }
}

template <bool kPack, bool kUnpack>
__global__ void __launch_bounds__(kAgThreads)
allgather_kernel(PTable tab, uint32_t n, uint32_t r, uint32_t rounds_per_cta,
                 const int8_t *__restrict__ recv, const int8_t *__restrict__ send,
                 int32_t *__restrict__ pack_out, int32_t *__restrict__ unpack_out)
{
    // schedule entries of this CTA's 288 virtual processors, round-major so that the threads of a
    // warp read consecutive bytes (one row of padding: the funnel shift of the last group of the
    // last round reads one word past its row)
    __shared__ __align__(16) int8_t send_k[kPack ? BCS_MAX_Q + 1 : 1][kAgCols];
    __shared__ __align__(16) int8_t recv_k[kUnpack ? BCS_MAX_Q + 1 : 1][kAgCols];
    __shared__ __align__(16) uint8_t send_rows[kPack ? kAgRowBytes : 16];
    __shared__ __align__(16) uint8_t recv_rows[kUnpack ? kAgRowBytes : 16];
    const uint32_t p = tab.p;
    const int q = tab.q;
    const uint32_t rounds = n - 1u + (uint32_t)q;
    const int x = (int)(((uint32_t)q - rounds % (uint32_t)q) % (uint32_t)q);
    const uint32_t j0 = blockIdx.x * kAgThreads;                   // first buffer of the CTA
    const uint32_t avail = p - j0;                                 // buffers from j0 to the end of a row
    const uint32_t cols = avail < (uint32_t)kAgCols ? avail : (uint32_t)kAgCols;   // buffers staged
    uint32_t hi = r + p - j0;                                      // (r - j0) mod p: virtual rank of column 0
    if (hi >= p) hi -= p;
    StagedRows sr = {};
    if (kPack) sr = load_rows_descending(send, p, q, hi, cols, send_rows);
    if (kUnpack) sr = load_rows_descending(recv, p, q, hi, cols, recv_rows);   // same offsets for both tables
    __syncthreads();
    for (uint32_t c = threadIdx.x; c < cols; c += kAgThreads) {    // column c: its row, spread over the rounds
        const uint32_t at = sr.at(c, q);
        const uint8_t *ps = send_rows + at, *pr = recv_rows + at;
        int k = 0;
        for (; k + 4 <= q; k += 4) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (kPack) send_k[k + u][c] = (int8_t)ps[k + u];
                if (kUnpack) recv_k[k + u][c] = (int8_t)pr[k + u];
            }
        }
        for (; k < q; ++k) {
            if (kPack) send_k[k][c] = (int8_t)ps[k];
            if (kUnpack) recv_k[k][c] = (int8_t)pr[k];
        }
    }
    __syncthreads();
    const uint32_t jr0 = blockIdx.y * rounds_per_cta;
    const uint32_t jr1 = rounds - jr0 > rounds_per_cta ? jr0 + rounds_per_cta : rounds;
    const int last = (int)n - 1;
    const bool tiny = q < 4;                                       // the phase bookkeeping below steps by four rounds
    uint32_t jr = jr0 + (threadIdx.x >> 6);
    if (!tiny && jr < jr1) {
        const uint64_t at = (uint64_t)jr * p + j0;                 // element index of the CTA's first buffer in this row
        const uint32_t grp = threadIdx.x & 63u;
        QuadStream ps, us;
        if (kPack) ps.init(send_k, pack_out, at, p, avail);
        if (kUnpack) us.init(recv_k, unpack_out, at, p, avail);
        const uint32_t i0 = jr + (uint32_t)x;
        uint32_t k = i0 % (uint32_t)q;
        int add = (int)(i0 / (uint32_t)q) * q - x;                 // q * floor(i / q) - x
#pragma unroll 2
        for (; jr < jr1; jr += 4) {
            // entries are in [-q, q-1]: only rows of the first two and of the last phases can
            // leave 0..n-1 (the same test for all threads of a warp)
            const bool clamp = add < q || add + q - 1 > last;
            if (kPack) ps.store(grp, k, add, clamp, last, p);
            if (kUnpack) us.store(grp, k, add, clamp, last, p);
            k += 4;
            if (k >= (uint32_t)q) {
                k -= (uint32_t)q;
                add += q;
            }
        }
    }
    if (tiny || j0 == 0 || avail < (uint32_t)kAgCols) {            // the same for all threads of the CTA
        if (kPack) loose_columns(send_k, pack_out, p, q, x, last, j0, avail, jr0, jr1, tiny);
        if (kUnpack) loose_columns(recv_k, unpack_out, p, q, x, last, j0, avail, jr0, jr1, tiny);
    }
}

}  // namespace
}  // namespace bcs

using namespace bcs;

extern "C" {

bcs_status bcs_allgather_tables(uint32_t p, uint32_t n, uint32_t r, const int8_t *recv,
                                const int8_t *send, int32_t *pack_out, int32_t *unpack_out,
                                void *cuda_stream)
{
    PTable tab;
    bcs_status st = make_table(p, &tab);
    if (st != BCS_OK) return st;
    if (r >= p) return BCS_ERR_RANGE;
    if (n == 0) return BCS_ERR_ARG;
    if (n > 0x7fffff00u) return BCS_ERR_UNSUPPORTED;
    if (tab.q == 0) return BCS_OK;
    if (recv == nullptr || send == nullptr || (pack_out == nullptr && unpack_out == nullptr))
        return BCS_ERR_ARG;
    if ((reinterpret_cast<uintptr_t>(pack_out) & 3u) || (reinterpret_cast<uintptr_t>(unpack_out) & 3u) ||
        !aligned16(recv) || !aligned16(send))
        return BCS_ERR_ALIGN;
    // A CTA stages the schedule rows of its buffers once and then streams rows of the output: the
    // rounds are cut into as many chunks (a multiple of four rounds each) as it takes to have
    // about kAgCtas CTAs (measured best on p = 100 003, n = 1000: 5.9 TB/s; a quarter or four times
    // as many CTAs 5.1 resp. 4.5 TB/s).
    const uint32_t rounds = n - 1u + (uint32_t)tab.q;
    const uint32_t col_blocks = (p + kAgThreads - 1) / kAgThreads;
    uint32_t chunks = (kAgCtas + col_blocks - 1) / col_blocks;
    uint32_t per_cta = ((rounds + chunks - 1) / chunks + 3u) & ~3u;
    chunks = (rounds + per_cta - 1) / per_cta;
    dim3 grid(col_blocks, chunks);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (pack_out && unpack_out)
        allgather_kernel<true, true><<<grid, kAgThreads, 0, stream>>>(tab, n, r, per_cta, recv, send, pack_out, unpack_out);
    else if (pack_out)
        allgather_kernel<true, false><<<grid, kAgThreads, 0, stream>>>(tab, n, r, per_cta, recv, send, pack_out, nullptr);
    else
        allgather_kernel<false, true><<<grid, kAgThreads, 0, stream>>>(tab, n, r, per_cta, recv, send, nullptr, unpack_out);
    return launch_status();
}

}  // extern "C"
