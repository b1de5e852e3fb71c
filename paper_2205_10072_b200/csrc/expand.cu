// Round tables of the n-block broadcast (arXiv 2205.10072, Algorithm 6 without the
// Send||Recv): a pure store stream, one 16-byte record per (rank, round).
#include "bcs_common.cuh"
#include "paper_path.cuh"

namespace bcs {
namespace {

// ---------------------------------------------------------------- Algorithm 6: round tables
constexpr int kExpandThreads = 256;
constexpr uint32_t kExpandRecords = 8192;      // records (128 KB of output) that a CTA aims for
constexpr uint32_t kExpandSharedBytes = 48 * 1024;

// A CTA takes `ranks_per_cta` consecutive ranks.  Their records are one contiguous stretch of
// the output, which the threads walk as a flat stream, thread t at the records t - shift,
// t - shift + 256, ...: `shift` (0..7) is chosen so that a warp's 32 x 16 bytes are four whole
// 128-byte lines of memory wherever the stretch starts (stores that cut lines or 32-byte sectors
// cost up to a fifth of the write bandwidth), and short rows (few rounds) fill the threads as
// well as long ones.  Rank, round, entry and phase of a thread's record are kept incrementally.
// kBuildRows: the caller gave no schedule tables, so the CTA computes the rows of its ranks as
// Algorithm 6 itself does: the receive entry of round k by running Algorithm 4 up to round k,
// the send entry as the receive entry of the to-processor (Algorithm 5) -- one (rank, round)
// pair per thread, the paper's own per-rank construction, no table and no scratch memory.
template <bool kBuildRows>
__global__ void __launch_bounds__(kExpandThreads)
expand_kernel(PTable tab, uint32_t n, uint64_t r_begin, uint64_t r_end, uint32_t ranks_per_cta,
              const int8_t *__restrict__ recv, const int8_t *__restrict__ send,
              int4 *__restrict__ table_out)
{
    // per rank of the CTA and per round k of a phase: {send entry - x, recv entry - x, to, from}.
    // Algorithm 6 adds q to an entry after each use and starts entries k < x at +q because
    // their first use is in the second phase; both are covered by adding q * floor(i / q).
    extern __shared__ int4 base[];             // [ranks_per_cta][q], then (kBuildRows) the skips
    uint32_t *skips_sh = reinterpret_cast<uint32_t *>(base + (size_t)ranks_per_cta * tab.q);
    if (kBuildRows) {
        if (threadIdx.x < kRow) skips_sh[threadIdx.x] = tab.s[threadIdx.x];
        __syncthreads();
    }
    const uint32_t q = (uint32_t)tab.q;
    const uint32_t p = tab.p;
    const uint32_t rounds = n - 1u + q;
    const uint32_t x = (q - rounds % q) % q;
    const uint64_t j0 = (uint64_t)blockIdx.x * ranks_per_cta;
    const uint64_t count = r_end - r_begin;
    const uint32_t ranks = (uint32_t)(count - j0 < (uint64_t)ranks_per_cta ? count - j0 : (uint64_t)ranks_per_cta);
    {
        const int8_t *srow = kBuildRows ? nullptr : send + j0 * q;     // the CTA's rows are contiguous
        const int8_t *rrow = kBuildRows ? nullptr : recv + j0 * q;
        for (uint32_t e = threadIdx.x; e < ranks * q; e += kExpandThreads) {
            const uint32_t g = e / q, k = e - g * q;
            const uint32_t r = (uint32_t)(r_begin + j0 + g);
            const uint32_t sk = tab.s[k];
            uint32_t to = r + sk;
            if (to >= p) to -= p;
            const uint32_t from = r >= sk ? r - sk : r + p - sk;
            int sent, received;
            if (kBuildRows) {
                received = (int8_t)recv_rounds(skips_sh, p, (int)q, r, (int)k, nullptr);
                sent = (int8_t)recv_rounds(skips_sh, p, (int)q, to, (int)k, nullptr);
            } else {
                sent = srow[e];
                received = rrow[e];
            }
            base[e] = make_int4(sent - (int)x, received - (int)x, (int)to, (int)from);
        }
    }
    __syncthreads();
    const uint32_t total = ranks * rounds;                           // records of the CTA (ranks > 1 only when rounds < kExpandRecords)
    const uint64_t first = j0 * rounds;                              // index of its first record
    int4 *out = table_out + first;
    const uint32_t shift = (uint32_t)((reinterpret_cast<uintptr_t>(table_out) >> 4) + first) & 7u;
    uint32_t e = threadIdx.x >= shift ? threadIdx.x - shift : threadIdx.x + kExpandThreads - shift;
    if (e >= total) return;
    // record e is round j of the CTA's rank number gq / q; round j uses i = j + x: entry
    // k = i mod q of phase floor(i / q), whose block numbers are the entries plus add = q * floor(i / q)
    uint32_t j = e % rounds, gq = e / rounds * q;
    int k = (int)((j + x) % q), add = (int)((j + x) / q * q);
    const int step_k = kExpandThreads % q, step_add = kExpandThreads / q * q;
    const int row_k = (int)(rounds % q), row_add = (int)(rounds / q * q);   // what a whole row adds to k and add
    const int last = (int)n - 1;
    for (;;) {
        const int4 rec = base[gq + (uint32_t)k];
        int sb = rec.x + add, rb = rec.y + add;
        sb = sb < 0 ? -1 : (sb > last ? last : sb);
        rb = rb < 0 ? -1 : (rb > last ? last : rb);
        __stcs(out + e, make_int4(sb, rb, rec.z, rec.w));
        e += kExpandThreads;
        if (e >= total) break;
        j += kExpandThreads;
        k += step_k;
        add += step_add;
        if (k >= (int)q) { k -= (int)q; add += (int)q; }
        while (j >= rounds) {                                        // on to the next rank: i falls by `rounds`
            j -= rounds;
            gq += q;
            k -= row_k;
            add -= row_add;
            if (k < 0) { k += (int)q; add -= (int)q; }
        }
    }
}

// ---------------------------------------------------------------- Algorithms 7 and 8: round tables
// One 16-byte record per (rank, round k), q records per rank.  Regular allgather (Algorithm 7):
// {to = r - skips[k], from = r + skips[k] (mod p), blocks exchanged skips[k+1] - skips[k],
// receive offset skips[k]}.  Census (Algorithm 8): when 2 skips[k] > skips[k+1] the edges are one
// shorter and only the partial sum S is sent: {to, from, 1 if x_r is added to what is sent, 0}.
__global__ void __launch_bounds__(256)
circulant_rounds_kernel(PTable tab, uint64_t r_begin, uint64_t n_records, int census,
                        int4 *__restrict__ out)
{
    const uint64_t e = (uint64_t)blockIdx.x * 256 + threadIdx.x;
    if (e >= n_records) return;
    const uint32_t q = (uint32_t)tab.q, p = tab.p;
    const uint64_t j = e / q;
    const uint32_t k = (uint32_t)(e - j * q);
    const uint32_t r = (uint32_t)(r_begin + j);
    const uint32_t lo = tab.s[k], hi = tab.s[k + 1];
    uint32_t step = lo;
    int c = (int)(hi - lo), d = (int)lo;
    if (census) {
        const bool shorter = 2ull * lo > hi;
        step = shorter ? lo - 1u : lo;
        c = shorter ? 0 : 1;
        d = 0;
    }
    const uint32_t to = r >= step ? r - step : r + p - step;
    uint32_t from = r + step;
    if (from >= p) from -= p;
    __stcs(out + e, make_int4((int)to, (int)from, c, d));
}

}  // namespace
}  // namespace bcs

using namespace bcs;

extern "C" {

bcs_status bcs_expand(uint32_t p, uint32_t n, uint64_t r_begin, uint64_t r_end,
                      const int8_t *recv, const int8_t *send, int32_t *table_out,
                      void *cuda_stream)
{
    bcs_status st = check_range(p, r_begin, r_end);
    if (st != BCS_OK) return st;
    if (n == 0) return BCS_ERR_ARG;
    if (n > 0x7fffff00u) return BCS_ERR_UNSUPPORTED;   // block numbers and n-1+q stay in int32
    PTable tab;
    make_table(p, &tab);
    const uint64_t count = r_end - r_begin;
    if (count == 0 || tab.q == 0) return BCS_OK;
    if (table_out == nullptr || (recv == nullptr) != (send == nullptr)) return BCS_ERR_ARG;
    if (!aligned16(table_out)) return BCS_ERR_ALIGN;
    // ranks per CTA: about kExpandRecords records, as far as the per-rank constants fit in shared memory
    const uint32_t rounds = n - 1u + (uint32_t)tab.q;
    uint32_t per_cta = (kExpandRecords + rounds - 1) / rounds;
    const uint32_t extra = recv == nullptr ? kRow * 4u : 0u;     // room for the skips when the rows are built here
    const uint32_t fit = (kExpandSharedBytes - extra) / (16u * (uint32_t)tab.q);
    if (per_cta > fit) per_cta = fit;
    const uint64_t blocks = (count + per_cta - 1) / per_cta;
    if (blocks > 0x7fffffffull) return BCS_ERR_UNSUPPORTED;
    if (recv == nullptr)                               // no tables: the kernel builds the rows it needs
        expand_kernel<true><<<(unsigned)blocks, kExpandThreads, (size_t)per_cta * tab.q * 16u + kRow * 4u,
                              static_cast<cudaStream_t>(cuda_stream)>>>(
            tab, n, r_begin, r_end, per_cta, nullptr, nullptr, reinterpret_cast<int4 *>(table_out));
    else
        expand_kernel<false><<<(unsigned)blocks, kExpandThreads, (size_t)per_cta * tab.q * 16u,
                               static_cast<cudaStream_t>(cuda_stream)>>>(
            tab, n, r_begin, r_end, per_cta, recv, send, reinterpret_cast<int4 *>(table_out));
    return launch_status();
}

bcs_status bcs_circulant_rounds(uint32_t p, uint64_t r_begin, uint64_t r_end, int census,
                                int32_t *table_out, void *cuda_stream)
{
    bcs_status st = check_range(p, r_begin, r_end);
    if (st != BCS_OK) return st;
    PTable tab;
    make_table(p, &tab);
    const uint64_t records = (r_end - r_begin) * (uint64_t)tab.q;
    if (records == 0) return BCS_OK;
    if (table_out == nullptr) return BCS_ERR_ARG;
    if (!aligned16(table_out)) return BCS_ERR_ALIGN;
    const uint64_t blocks = (records + 255) / 256;
    if (blocks > 0x7fffffffull) return BCS_ERR_UNSUPPORTED;
    circulant_rounds_kernel<<<(unsigned)blocks, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        tab, r_begin, records, census != 0, reinterpret_cast<int4 *>(table_out));
    return launch_status();
}

}  // extern "C"
