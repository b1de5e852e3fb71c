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

__global__ void __launch_bounds__(kAgThreads)
allgather_kernel(PTable tab, uint32_t n, uint32_t r, const int8_t *__restrict__ recv,
                 const int8_t *__restrict__ send, int32_t *__restrict__ pack_out,
                 int32_t *__restrict__ unpack_out)
{
    // schedule entries of this CTA's 256 virtual processors, round-major so that the threads of a
    // warp read consecutive bytes
    __shared__ int8_t send_k[BCS_MAX_Q][kAgThreads];
    __shared__ int8_t recv_k[BCS_MAX_Q][kAgThreads];
    const uint32_t p = tab.p;
    const int q = tab.q;
    const uint32_t rounds = n - 1u + (uint32_t)q;
    const int x = (int)(((uint32_t)q - rounds % (uint32_t)q) % (uint32_t)q);
    const uint32_t j = blockIdx.x * kAgThreads + threadIdx.x;      // buffer
    const bool valid = j < p;
    if (valid) {
        uint32_t v = r + p - j;                                    // (r - j) mod p, j <= p - 1
        if (v >= p) v -= p;
        const int8_t *srow = send + (uint64_t)v * q, *rrow = recv + (uint64_t)v * q;
        for (int k = 0; k < q; ++k) {
            send_k[k][threadIdx.x] = srow[k];
            recv_k[k][threadIdx.x] = rrow[k];
        }
    }
    // each thread reads back only what it wrote: no barrier needed
    if (!valid) return;
    const uint32_t jr0 = blockIdx.y * kAgRounds;
    const uint32_t jr1 = jr0 + kAgRounds < rounds ? jr0 + kAgRounds : rounds;
    const int last = (int)n - 1;
    uint32_t i = jr0 + (uint32_t)x;
    uint32_t k = i % (uint32_t)q;
    int base = (int)(i / (uint32_t)q) * q - x;                     // q * floor(i / q) - x
    int32_t *pk = pack_out ? pack_out + (uint64_t)jr0 * p + j : nullptr;
    int32_t *up = unpack_out ? unpack_out + (uint64_t)jr0 * p + j : nullptr;
    for (uint32_t jr = jr0; jr < jr1; ++jr) {
        if (pk) {
            int b = (int)send_k[k][threadIdx.x] + base;
            b = b < 0 ? -1 : (b > last ? last : b);
            __stcs(pk, b);
            pk += p;
        }
        if (up) {
            int b = (int)recv_k[k][threadIdx.x] + base;
            b = b < 0 ? -1 : (b > last ? last : b);
            __stcs(up, b);
            up += p;
        }
        if (++k == (uint32_t)q) {
            k = 0;
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
    if ((reinterpret_cast<uintptr_t>(pack_out) & 3u) || (reinterpret_cast<uintptr_t>(unpack_out) & 3u))
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
