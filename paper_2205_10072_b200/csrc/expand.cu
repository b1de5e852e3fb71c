// Round tables of the n-block broadcast (arXiv 2205.10072, Algorithm 6 without the
// Send||Recv): a pure store stream, one 16-byte record per (rank, round).
#include "bcs_common.cuh"

namespace bcs {
namespace {

// ---------------------------------------------------------------- Algorithm 6: round tables
constexpr int kExpandThreads = 256;
constexpr int kExpandRanks = 8;   // ranks per CTA

__global__ void __launch_bounds__(kExpandThreads)
expand_kernel(PTable tab, uint32_t n, uint64_t r_begin, uint64_t r_end,
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
    if (recv == nullptr || send == nullptr || table_out == nullptr) return BCS_ERR_ARG;
    if (!aligned16(table_out)) return BCS_ERR_ALIGN;
    const unsigned blocks = (unsigned)((count + kExpandRanks - 1) / kExpandRanks);
    expand_kernel<<<blocks, kExpandThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        tab, n, r_begin, r_end, recv, send, reinterpret_cast<int4 *>(table_out));
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
