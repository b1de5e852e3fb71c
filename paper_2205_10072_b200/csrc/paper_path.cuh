// The paper's own per-rank construction (arXiv 2205.10072, Algorithms 2-4) as device functions:
// one thread runs Algorithm 4 for one rank with the range search done by descending the
// homeranges.  Used by the self-contained kernels of the schedule translation unit and by the
// round-table kernel when it has to build the rows of its ranks itself.
#pragma once
#include "bcs_common.cuh"

namespace bcs {

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
static __device__ __noinline__ uint32_t cyclic_mask(const uint32_t *s, uint32_t p, int q,
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

}  // namespace bcs
