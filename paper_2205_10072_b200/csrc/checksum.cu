// Position-weighted checksum of schedule entries (no counterpart in the paper): a read-only
// stream over the table, reduced per warp, per CTA and with one atomic per CTA.
#include "bcs_common.cuh"

namespace bcs {
namespace {

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
// Largest grid: 64 CTAs per SM.  Measured on a 1.6 GB buffer: 8 CTAs per SM (one resident wave
// that strides over the buffer) 5.8 TB/s, 64 and 128 per SM 6.4 TB/s, 512 per SM 5.6 TB/s.
constexpr uint64_t kSumMaxCtas = 148u * 64u;

// Weighted sum of one 16-byte vector whose first word has index g.  kSameHigh: all word indices
// of the call share their high half, whose term of the weight (hi_term) is then the same for the
// whole call, and the indices are 32-bit additions.
template <bool kSameHigh>
__device__ __forceinline__ unsigned long long vector_sum(const uint4 w, uint64_t g, uint32_t hi_term)
{
    unsigned long long t;
    if (kSameHigh) {
        const uint32_t lo = (uint32_t)g;
        t = (unsigned long long)w.x * (fmix32(lo ^ hi_term) | 1u);
        t += (unsigned long long)w.y * (fmix32((lo + 1u) ^ hi_term) | 1u);
        t += (unsigned long long)w.z * (fmix32((lo + 2u) ^ hi_term) | 1u);
        t += (unsigned long long)w.w * (fmix32((lo + 3u) ^ hi_term) | 1u);
    } else {
        t = (unsigned long long)w.x * word_weight(g);
        t += (unsigned long long)w.y * word_weight(g + 1);
        t += (unsigned long long)w.z * word_weight(g + 2);
        t += (unsigned long long)w.w * word_weight(g + 3);
    }
    return t;
}

// n_words full 32-bit words, then tail_bytes (0..3) bytes of one more, zero-padded.  The bulk is
// read as 16-byte vectors, four loads in flight per thread (the few words before the first
// 16-byte boundary and after the last full vector are taken one by one by the first CTA).
template <bool kSameHigh>
__global__ void __launch_bounds__(kSumThreads)
checksum_kernel(const uint32_t *__restrict__ words, uint64_t n_words, uint32_t tail_bytes,
                uint64_t first_word, unsigned long long *sum)
{
    unsigned long long acc = 0;
    uint64_t head = ((16u - (uint32_t)(reinterpret_cast<uintptr_t>(words) & 15u)) & 15u) >> 2;
    if (head > n_words) head = n_words;
    const uint4 *vec = reinterpret_cast<const uint4 *>(words + head);
    const uint64_t n_vec = (n_words - head) >> 2;
    const uint64_t stride = (uint64_t)gridDim.x * kSumThreads;
    const uint64_t g0 = first_word + head;
    const uint32_t hi_term = 0x9E3779B9u * (uint32_t)(first_word >> 32);
    uint64_t v = (uint64_t)blockIdx.x * kSumThreads + threadIdx.x;
    for (; v + 3 * stride < n_vec; v += 4 * stride) {
        const uint4 w0 = __ldcs(vec + v);
        const uint4 w1 = __ldcs(vec + v + stride);
        const uint4 w2 = __ldcs(vec + v + 2 * stride);
        const uint4 w3 = __ldcs(vec + v + 3 * stride);
        acc += vector_sum<kSameHigh>(w0, g0 + 4 * v, hi_term);
        acc += vector_sum<kSameHigh>(w1, g0 + 4 * (v + stride), hi_term);
        acc += vector_sum<kSameHigh>(w2, g0 + 4 * (v + 2 * stride), hi_term);
        acc += vector_sum<kSameHigh>(w3, g0 + 4 * (v + 3 * stride), hi_term);
    }
    for (; v < n_vec; v += stride) acc += vector_sum<kSameHigh>(__ldcs(vec + v), g0 + 4 * v, hi_term);
    if (blockIdx.x == 0) {
        const uint64_t done = head + 4 * n_vec;            // words [done, n_words) are left over
        const uint64_t loose = head + (n_words - done);    // <= 6
        if (threadIdx.x < loose) {
            const uint64_t w = threadIdx.x < head ? threadIdx.x : done + (threadIdx.x - head);
            acc += (unsigned long long)words[w] * word_weight(first_word + w);
        }
        if (tail_bytes && threadIdx.x == 32) {
            const uint8_t *b = reinterpret_cast<const uint8_t *>(words + n_words);
            uint32_t v = 0;
            for (uint32_t t = 0; t < tail_bytes; ++t) v |= (uint32_t)b[t] << (8 * t);
            acc += (unsigned long long)v * word_weight(first_word + n_words);
        }
    }
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, o);
    __shared__ unsigned long long part[kSumThreads / 32];
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long t = 0;
        for (int w = 0; w < kSumThreads / 32; ++w) t += part[w];
        if (t) atomicAdd(sum, t);
    }
}

}  // namespace
}  // namespace bcs

using namespace bcs;

extern "C" {

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
    uint64_t blocks = (n_words / 16 + kSumThreads - 1) / kSumThreads;   // >= 4 vectors per thread
    if (blocks < 1) blocks = 1;
    if (blocks > kSumMaxCtas) blocks = kSumMaxCtas;
    const uint64_t first_word = first_entry_index / 4;
    // do all word indices of the call (first_word .. first_word + n_words) share their high half?
    const bool same_high = (first_word >> 32) == ((first_word + n_words) >> 32);
    auto kernel = same_high ? checksum_kernel<true> : checksum_kernel<false>;
    kernel<<<(unsigned)blocks, kSumThreads, 0, stream>>>(
        reinterpret_cast<const uint32_t *>(buf_dev), n_words, (uint32_t)(n_entries & 3u),
        first_word, reinterpret_cast<unsigned long long *>(sum_dev));
    return launch_status();
}

}  // extern "C"
