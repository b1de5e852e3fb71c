// Index tables of the irregular allgather (arXiv 2205.10072, Algorithm 9 without the data
// movement): for one processor r, which block of buffer[j] is packed and which is unpacked in
// every round.  Processor r treats buffer j as virtual processor (r-j) mod p of a broadcast
// rooted at j, so entry [round][j] is the send resp. receive block of that virtual processor's
// round (Algorithm 6's closed form).  A pure store stream: 8 bytes per (round, buffer).
#include "bcs_common.cuh"

namespace bcs {
namespace {

constexpr int kAgThreads = 256;   // buffers per CTA (one per thread)
constexpr int kAgRounds = 64;     // rounds per CTA

// Rows of `table` ([p][q] int8, 16-byte aligned) for the ranks hi, hi-1, ..., hi-n+1 (mod p), brought into shared
// memory with 16-byte loads (the rows are one contiguous run, or two when the ranks pass 0) and
// spread round-major and made non-negative: out[k][c] = table[(hi - c) mod p][k] + 2q (< 128).
__device__ __forceinline__ void stage_rows_descending(const int8_t *__restrict__ table, uint32_t p,
                                                      int q, uint32_t hi, uint32_t n,
                                                      uint8_t *rows /* (n * q + 32) bytes */,
                                                      int8_t (*out)[kAgThreads])
{
    const uint32_t first = n <= hi + 1u ? n : hi + 1u;     // columns served by ranks hi-first+1..hi
    const uint32_t lo = hi + 1u - first;
    const uint64_t byte_a = (uint64_t)lo * q;
    const uint32_t shift_a = (uint32_t)(byte_a & 15u);
    load_span(rows, shift_a, first * (uint32_t)q, table, byte_a);
    __syncthreads();
    if (threadIdx.x < first) {
        const uint8_t *row = rows + shift_a + (first - 1u - threadIdx.x) * q;
        for (int k = 0; k < q; ++k) out[k][threadIdx.x] = (int8_t)((int8_t)row[k] + 2 * q);
    }
    __syncthreads();
    if (first < n) {                                       // the rest: ranks p-1, p-2, ...
        const uint32_t rest = n - first;
        const uint64_t byte_b = (uint64_t)(p - rest) * q;
        const uint32_t shift_b = (uint32_t)(byte_b & 15u);
        load_span(rows, shift_b, rest * (uint32_t)q, table, byte_b);
        __syncthreads();
        if (threadIdx.x >= first && threadIdx.x < n) {
            const uint8_t *row = rows + shift_b + (n - 1u - threadIdx.x) * q;
            for (int k = 0; k < q; ++k) out[k][threadIdx.x] = (int8_t)((int8_t)row[k] + 2 * q);
        }
        __syncthreads();
    }
}

__global__ void __launch_bounds__(kAgThreads)
allgather_kernel(PTable tab, uint32_t n, uint32_t r, const int8_t *__restrict__ recv,
                 const int8_t *__restrict__ send, int32_t *__restrict__ pack_out,
                 int32_t *__restrict__ unpack_out)
{
    // schedule entries of this CTA's 256 virtual processors, round-major so that the threads of a
    // warp read consecutive bytes
    __shared__ __align__(16) int8_t send_k[BCS_MAX_Q][kAgThreads];
    __shared__ __align__(16) int8_t recv_k[BCS_MAX_Q][kAgThreads];
    __shared__ __align__(16) uint8_t rows[kAgThreads * BCS_MAX_Q + 32];
    const uint32_t p = tab.p;
    const int q = tab.q;
    const uint32_t rounds = n - 1u + (uint32_t)q;
    const int x = (int)(((uint32_t)q - rounds % (uint32_t)q) % (uint32_t)q);
    const uint32_t j0 = blockIdx.x * kAgThreads;                   // first buffer of the CTA
    const uint32_t cols = p - j0 < (uint32_t)kAgThreads ? p - j0 : (uint32_t)kAgThreads;
    uint32_t hi = r + p - j0;                                      // (r - j0) mod p: virtual rank of column 0
    if (hi >= p) hi -= p;
    if (pack_out) stage_rows_descending(send, p, q, hi, cols, rows, send_k);
    if (unpack_out) stage_rows_descending(recv, p, q, hi, cols, rows, recv_k);
    // Four rows at a time: thread t works on rows jr0 + t / 64, +4, +8, ... and on four consecutive
    // buffers, chosen so that its 16 bytes are 16-byte aligned in the output.  Rows are p * 4 bytes
    // long, so the alignment of a row's start differs from row to row -- but four rows on it is
    // the same again (16 p bytes), so each thread finds its alignment once per table.  The up to
    // three buffers before the first and after the last aligned group of the CTA's 256 are
    // written one by one.
    const uint32_t jr0 = blockIdx.y * kAgRounds;
    const uint32_t jr1 = jr0 + kAgRounds < rounds ? jr0 + kAgRounds : rounds;
    const int last = (int)n - 1;
    const uint32_t sub = threadIdx.x >> 6, grp = threadIdx.x & 63u;
    uint32_t jr = jr0 + sub;
    if (jr >= jr1) return;
    const uint32_t i0 = jr + (uint32_t)x;
    uint32_t k = i0 % (uint32_t)q;
    int base = (int)(i0 / (uint32_t)q) * q - x - 2 * q;            // q * floor(i / q) - x, minus the staging offset
    uint64_t at = (uint64_t)jr * p + j0;                           // element index of the CTA's first buffer
    uint32_t head[2] = {0, 0};                                     // buffers before the first 16-byte boundary
    int32_t *const outs[2] = {pack_out, unpack_out};
#pragma unroll
    for (int which = 0; which < 2; ++which) {
        if (outs[which] == nullptr) continue;
        uint32_t hd = (uint32_t)((16u - (uint32_t)(reinterpret_cast<uintptr_t>(outs[which] + at) & 15u)) & 15u) >> 2;
        head[which] = hd > cols ? cols : hd;
    }
    for (; jr < jr1; jr += 4) {
#pragma unroll
        for (int which = 0; which < 2; ++which) {
            int32_t *out = outs[which];
            if (out == nullptr) continue;
            const int8_t *src = which == 0 ? send_k[k] : recv_k[k];
            const uint32_t c = head[which] + 4u * grp;             // first of this thread's four buffers
            if (c + 4u <= cols) {
                // four consecutive bytes from two aligned words
                const uint32_t *words = reinterpret_cast<const uint32_t *>(src) + (c >> 2);
                const uint32_t lo = words[0], hi = (c & 3u) ? words[1] : 0u;
                const uint32_t four = __funnelshift_r(lo, hi, (c & 3u) * 8u);
                // the staged bytes are entries + 2q (unsigned); below 0 -> -1, above n-1 -> n-1
                int4 v;
                v.x = max(min((int)__byte_perm(four, 0u, 0x4440u) + base, last), -1);
                v.y = max(min((int)__byte_perm(four, 0u, 0x4441u) + base, last), -1);
                v.z = max(min((int)__byte_perm(four, 0u, 0x4442u) + base, last), -1);
                v.w = max(min((int)__byte_perm(four, 0u, 0x4443u) + base, last), -1);
                __stcs(reinterpret_cast<int4 *>(out + at + c), v);
            } else {
                for (uint32_t e = c; e < cols; ++e) {              // ragged end of the CTA's columns
                    const int b = (int)(uint8_t)src[e] + base;
                    out[at + e] = b < 0 ? -1 : (b > last ? last : b);
                }
            }
            if (grp < head[which]) {                               // ragged start
                const int b = (int)(uint8_t)src[grp] + base;
                out[at + grp] = b < 0 ? -1 : (b > last ? last : b);
            }
        }
        at += 4ull * p;
        k += 4;
        while (k >= (uint32_t)q) {
            k -= (uint32_t)q;
            base += q;
        }
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
    const uint32_t rounds = n - 1u + (uint32_t)tab.q;
    const uint64_t chunks = ((uint64_t)rounds + kAgRounds - 1) / kAgRounds;
    if (chunks > 65535u) return BCS_ERR_UNSUPPORTED;              // grid.y limit: n up to ~4.19 million
    dim3 grid((unsigned)((p + kAgThreads - 1) / kAgThreads), (unsigned)chunks);
    allgather_kernel<<<grid, kAgThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        tab, n, r, recv, send, pack_out, unpack_out);
    return launch_status();
}

}  // extern "C"
