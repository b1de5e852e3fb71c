// Checker of the properties that every schedule of the construction has (arXiv 2205.10072,
// text after Theorem 1 and Algorithm 5), run over tables already on the device.  It uses
// Algorithm 2 (homerange descent) for the baseblocks, not the skip codes of the fast
// construction, so that it does not share its arithmetic with what it checks.
#include "bcs_common.cuh"

namespace bcs {
namespace {

// Algorithm 2: peel off the head of the homerange until r is a skip itself.
__device__ __forceinline__ int base_block_of(const uint32_t *s, uint32_t r)
{
    for (;;) {
        const int k = home_of(s, r);
        const uint32_t v = s[k];
        if (r == v) return k;
        r -= v;
    }
}

__global__ void __launch_bounds__(kTile)
validate_kernel(PTable tab, uint64_t r_begin, uint64_t r_end, const int8_t *__restrict__ recv,
                const int8_t *__restrict__ send, unsigned long long *violations)
{
    __shared__ uint32_t s[kRow];
    __shared__ __align__(16) uint8_t recv_rows[kTile * 32];
    __shared__ __align__(16) uint8_t send_rows[kTile * 32];
    const int q = tab.q;
    const uint32_t p = tab.p;
    if (threadIdx.x < kRow) s[threadIdx.x] = tab.s[threadIdx.x];
    const uint64_t count = r_end - r_begin;
    const uint64_t g0 = (uint64_t)blockIdx.x * kTile;
    const uint32_t n = (uint32_t)(count - g0 < (uint64_t)kTile ? count - g0 : (uint64_t)kTile);
    if (recv) load_span(recv_rows, 0, n * (uint32_t)q, recv, g0 * (uint64_t)q);
    if (send) load_span(send_rows, 0, n * (uint32_t)q, send, g0 * (uint64_t)q);
    __syncthreads();
    unsigned bad_recv = 0, bad_send = 0, bad_pair = 0;
    if (threadIdx.x < n) {
        const uint32_t r = (uint32_t)(r_begin + g0 + threadIdx.x);
        const int8_t *rrow = reinterpret_cast<const int8_t *>(recv_rows) + threadIdx.x * q;
        const int8_t *srow = reinterpret_cast<const int8_t *>(send_rows) + threadIdx.x * q;
        int h = -1, bb = -1;
        if (r > 0) {
            h = home_of(s, r);
            bb = base_block_of(s, r);
        }
        if (recv) {
            // the baseblock once, in the home round; q-1 different blocks of the previous phase
            uint32_t seen = bb >= 0 ? 1u << bb : 0u;
            for (int i = 0; i < q; ++i) {
                const int v = rrow[i];
                if (i == h) {
                    if (v != bb) bad_recv = 1;
                } else {
                    const int b = v + q;
                    if (v >= 0 || b < 0 || ((seen >> b) & 1u)) bad_recv = 1;
                    else seen |= 1u << b;
                }
            }
        }
        if (send) {
            // the root sends block k in round k; everybody else sends a previous-phase block that it
            // received in an earlier round of the row, or its baseblock of the previous phase,
            // or -- after the home round -- its baseblock of the current phase
            uint32_t have = bb >= 0 ? 1u << bb : 0u;     // previous-phase blocks that may be sent
            for (int k = 0; k < q; ++k) {
                const int v = srow[k];
                if (r == 0) {
                    if (v != k) bad_send = 1;
                } else if (!(k > h && v == bb)) {
                    const int b = v + q;
                    if (v >= 0 || b < 0 || (recv && !((have >> b) & 1u))) bad_send = 1;
                }
                if (recv && k != h) {
                    const int b = rrow[k] + q;
                    if (b >= 0 && b < q) have |= 1u << b;
                }
            }
        }
        if (recv && send) {
            // Algorithm 5 / Algorithm 9: what r sends in round k is what r + skips[k] receives
            for (int k = 0; k < q; ++k) {
                uint32_t t = r + s[k];
                if (t >= p) t -= p;
                if (t >= r_begin && t < r_end &&
                    recv[(t - r_begin) * (uint64_t)q + k] != srow[k])
                    bad_pair = 1;
            }
        }
    }
    const unsigned n_recv = __syncthreads_count(bad_recv);
    const unsigned n_send = __syncthreads_count(bad_send);
    const unsigned n_pair = __syncthreads_count(bad_pair);
    if (threadIdx.x == 0) {
        if (n_recv) atomicAdd(violations + 0, (unsigned long long)n_recv);
        if (n_send) atomicAdd(violations + 1, (unsigned long long)n_send);
        if (n_pair) atomicAdd(violations + 2, (unsigned long long)n_pair);
    }
}

// ---------------------------------------------------------------- broadcast simulation
// One round of the n-block broadcast for every rank at once (Algorithm 6 with the blocks taken
// from the int8 tables by the closed form block = entry - x + q * floor(i / q), i = j + x).
// held[r]: bit b set iff rank r holds block b before the round; next[r]: after it.
__global__ void __launch_bounds__(kTile)
simulate_round_kernel(PTable tab, uint32_t n, uint32_t i, const int8_t *__restrict__ recv,
                      const int8_t *__restrict__ send, const unsigned long long *__restrict__ held,
                      unsigned long long *__restrict__ next, unsigned long long *counts,
                      int last_round)
{
    const uint32_t p = tab.p;
    const int q = tab.q;
    const uint32_t k = i % (uint32_t)q;
    const int shift = (int)(i / (uint32_t)q) * q;          // q * floor(i / q)
    const int x = (int)(((uint32_t)q - (n - 1u + (uint32_t)q) % (uint32_t)q) % (uint32_t)q);
    const int top = (int)n - 1;
    const uint64_t r64 = (uint64_t)blockIdx.x * kTile + threadIdx.x;
    unsigned unheld = 0, unpaired = 0, twice = 0, early = 0;
    if (r64 < p) {
        const uint32_t r = (uint32_t)r64;
        const unsigned long long all = n >= 64u ? ~0ull : (1ull << n) - 1ull;
        const unsigned long long mine = held[r];
        int sb = (int)send[(uint64_t)r * q + k] - x + shift;
        int rb = (int)recv[(uint64_t)r * q + k] - x + shift;
        sb = sb < 0 ? -1 : (sb > top ? top : sb);
        rb = rb < 0 ? -1 : (rb > top ? top : rb);
        uint32_t to = r + tab.s[k];
        if (to >= p) to -= p;
        int rb_to = (int)recv[(uint64_t)to * q + k] - x + shift;   // what the to-processor receives
        rb_to = rb_to < 0 ? -1 : (rb_to > top ? top : rb_to);
        if (sb >= 0 && !((mine >> sb) & 1ull)) unheld = 1;         // condition a): sends only held blocks
        if (rb_to != sb) unpaired = 1;
        unsigned long long after = mine;
        if (rb >= 0) {
            if (r != 0 && ((mine >> rb) & 1ull)) twice = 1;        // condition b): every receipt is new
            after |= 1ull << rb;
        }
        next[r] = after;
        if (last_round && mine == all) early = 1;                  // complete before the last round
    }
    const unsigned c0 = __syncthreads_count(unheld);
    const unsigned c1 = __syncthreads_count(unpaired);
    const unsigned c2 = __syncthreads_count(twice);
    const unsigned c3 = __syncthreads_count(early);
    if (threadIdx.x == 0) {
        if (c0) atomicAdd(counts + 0, (unsigned long long)c0);
        if (c1) atomicAdd(counts + 1, (unsigned long long)c1);
        if (c2) atomicAdd(counts + 2, (unsigned long long)c2);
        if (c3) atomicAdd(counts + 4, (unsigned long long)c3);
    }
}

__global__ void __launch_bounds__(kTile)
simulate_init_kernel(uint32_t p, uint32_t n, unsigned long long *held)
{
    const uint64_t r = (uint64_t)blockIdx.x * kTile + threadIdx.x;
    if (r < p) held[r] = r == 0 ? (n >= 64u ? ~0ull : (1ull << n) - 1ull) : 0ull;
}

__global__ void __launch_bounds__(kTile)
simulate_final_kernel(uint32_t p, uint32_t n, const unsigned long long *__restrict__ held,
                      unsigned long long *counts)
{
    const uint64_t r = (uint64_t)blockIdx.x * kTile + threadIdx.x;
    const unsigned long long all = n >= 64u ? ~0ull : (1ull << n) - 1ull;
    const unsigned c = __syncthreads_count(r < p && held[r] != all);
    if (threadIdx.x == 0 && c) atomicAdd(counts + 3, (unsigned long long)c);
}

}  // namespace
}  // namespace bcs

using namespace bcs;

extern "C" {

bcs_status bcs_validate(uint32_t p, uint64_t r_begin, uint64_t r_end, const int8_t *recv,
                        const int8_t *send, uint64_t *violations_dev, void *cuda_stream)
{
    bcs_status st = check_range(p, r_begin, r_end);
    if (st != BCS_OK) return st;
    if (violations_dev == nullptr) return BCS_ERR_ARG;
    if (recv == nullptr && send == nullptr) return BCS_ERR_ARG;
    if (!aligned16(recv) || !aligned16(send)) return BCS_ERR_ALIGN;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemsetAsync(violations_dev, 0, 3 * sizeof(uint64_t), stream) != cudaSuccess)
        return BCS_ERR_CUDA;
    PTable tab;
    make_table(p, &tab);
    const uint64_t count = r_end - r_begin;
    if (count == 0 || tab.q == 0) return BCS_OK;
    const unsigned blocks = (unsigned)((count + kTile - 1) / kTile);
    validate_kernel<<<blocks, kTile, 0, stream>>>(
        tab, r_begin, r_end, recv, send, reinterpret_cast<unsigned long long *>(violations_dev));
    return launch_status();
}

bcs_status bcs_simulate(uint32_t p, uint32_t n, const int8_t *recv, const int8_t *send,
                        uint64_t *state_dev, uint64_t *counts_dev, void *cuda_stream)
{
    PTable tab;
    bcs_status st = make_table(p, &tab);
    if (st != BCS_OK) return st;
    if (n == 0 || counts_dev == nullptr) return BCS_ERR_ARG;
    if (n > 64) return BCS_ERR_UNSUPPORTED;           // the held blocks of a rank are one 64-bit set
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemsetAsync(counts_dev, 0, 5 * sizeof(uint64_t), stream) != cudaSuccess)
        return BCS_ERR_CUDA;
    if (tab.q == 0) return BCS_OK;
    if (recv == nullptr || send == nullptr || state_dev == nullptr) return BCS_ERR_ARG;
    if ((reinterpret_cast<uintptr_t>(state_dev) & 7u) != 0) return BCS_ERR_ALIGN;
    unsigned long long *held = reinterpret_cast<unsigned long long *>(state_dev);
    unsigned long long *next = held + p;
    unsigned long long *counts = reinterpret_cast<unsigned long long *>(counts_dev);
    const unsigned blocks = (unsigned)((p + kTile - 1) / kTile);
    const uint32_t rounds = n - 1u + (uint32_t)tab.q;
    const uint32_t x = ((uint32_t)tab.q - rounds % (uint32_t)tab.q) % (uint32_t)tab.q;
    simulate_init_kernel<<<blocks, kTile, 0, stream>>>(p, n, held);
    if ((st = launch_status()) != BCS_OK) return st;
    for (uint32_t j = 0; j < rounds; ++j) {
        simulate_round_kernel<<<blocks, kTile, 0, stream>>>(tab, n, j + x, recv, send, held, next,
                                                            counts, j + 1 == rounds);
        if ((st = launch_status()) != BCS_OK) return st;
        unsigned long long *t = held;
        held = next;
        next = t;
    }
    simulate_final_kernel<<<blocks, kTile, 0, stream>>>(p, n, held, counts);
    return launch_status();
}

}  // extern "C"
