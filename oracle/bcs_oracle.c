/*
 * bcs_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, single-purpose CPU restatement of the schedule construction of
 * J. L. Traff, "(Poly)Logarithmic Time Construction of Round-optimal n-Block
 * Broadcast Schedules for Broadcast and irregular Allgather in MPI"
 * (arXiv 2205.10072), Section 2.  It exists so that the CUDA library can be
 * compared with something written straight from the paper.  It shares no code,
 * header, table or helper with the CUDA path and must never be called from it:
 * only the tests, the smoke check and the CPU-baseline leg of the benchmark
 * link or load this file.
 *
 * Two independent forms are provided and the tests demand that they agree:
 *
 *   per-rank form  (O(log p) space, any p < 2^31): Algorithm 1 (skips),
 *       Algorithm 2 (baseblock), the range search that Algorithm 3 stands for,
 *       Algorithm 4 (receive schedule, with the paper's two special rounds
 *       written out) and Algorithm 5 (send schedule by re-running Algorithm 4
 *       for the to-neighbour).
 *
 *   array form  (O(p log p) space): the linear-time baseblock list of
 *       Section 2 ("root sends block i to skips[i], everybody below forwards"),
 *       per-block prefix counts over that list so that "which baseblocks lie in
 *       a window" is a subtraction, the uniform window rule of Algorithm 4 for
 *       every round, and the send table by the lookup of Algorithm 9
 *       (sendsched[j][k] = recvsched[(j+skips[k]) mod p][k]).
 *
 * Readings of places where the paper is silent or garbled (each is also listed
 * in the design notes of the repository):
 *   - Algorithm 4 starts with B = {} but the text after Theorem 1 says a receive
 *     row holds the baseblock once and q-1 different other blocks; so for r > 0
 *     the own baseblock is put into B before the first round.
 *   - "for i = 0..k" in Algorithm 4 together with "recvsched(r+skips[i], i)[i]"
 *     in Algorithm 5 means: entries 0..i inclusive are computed when entry i is
 *     wanted.
 *   - r + skips[i] in Algorithm 5 is taken mod p (as Algorithm 9 does).
 *   - The printed body of Algorithm 3 does not match its own description; the
 *     function is defined here by what the text says it returns: the set of
 *     baseblocks of the processors in a (possibly cyclic) range.  The root
 *     (rank 0) has no baseblock and contributes nothing.
 *   - max(U \ B): the largest block, as the text says.
 *   - An empty second window yields the empty set; an empty U \ B after the
 *     second window is reported as an error (never seen).
 *   - Expansion (Algorithm 6): a block < 0 is reported as -1 ("neither sent nor
 *     received"); to/from are still the circulant neighbours.
 *
 * Parity pins (see tests/): the paper's Tables 1-5, a brute-force broadcast
 * simulation, the power-of-two closed form, Lemma 1 and Lemma 2, agreement of
 * the two forms, and a definitional scan for the range search.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define BCSO_MAXQ 32

/* q = ceil(log2 p) (Section 2, first paragraph).  p >= 1. */
int bcso_q(uint32_t p)
{
    int q = 0;
    uint64_t v = 1;
    while (v < p) { v *= 2; q++; }
    return q;
}

/* Algorithm 1: skips[q] = p, then successive ceil-halving down to skips[0] = 1.
 * Writes q+1 words; returns q. */
int bcso_skips(uint32_t p, uint32_t *skips)
{
    int q = bcso_q(p);
    int k = q;
    uint32_t v = p;
    while (v > 1) {
        skips[k] = v;
        v = v / 2 + v % 2;
        k = k - 1;
    }
    skips[k] = v;
    return q;
}

/* Algorithm 2: baseblock of processor r, 0 < r < p, searching the skips
 * downwards from skips[q].  Returns -1 for the root (it has none). */
int bcso_baseblock(uint32_t p, uint32_t r)
{
    uint32_t s[BCSO_MAXQ + 1];
    int k;
    if (r == 0 || r >= p) return -1;
    k = bcso_skips(p, s);
    while (r != s[k]) {
        k = k - 1;
        if (s[k] < r) r = r - s[k];
    }
    return k;
}

/* Section 2, paragraph after Algorithm 2: the list of baseblocks in linear
 * time by doing what the first q rounds do.  In round i the root sends block i
 * to processor skips[i]; every processor 1 <= r < skips[i] forwards its
 * baseblock to r + skips[i] when that is below skips[i+1].  bb[0] = -1. */
void bcso_baseblock_list(uint32_t p, int8_t *bb)
{
    uint32_t s[BCSO_MAXQ + 1];
    int q = bcso_skips(p, s);
    int i;
    uint32_t r;
    bb[0] = -1;
    for (i = 0; i < q; i++) {
        bb[s[i]] = (int8_t)i;
        for (r = 1; r < s[i]; r++)
            if (r + s[i] < s[i + 1]) bb[r + s[i]] = bb[r];
    }
}

/* Largest k with skips[k] <= x, for 1 <= x < p ("homerange" of x). */
static int home_of(const uint32_t *s, int q, uint32_t x)
{
    int k = q - 1;
    while (s[k] > x) k--;
    return k;
}

/* Set of baseblocks (bit k = block k) of the processors a..b, 1 <= a <= b < p.
 * This is what Algorithm 3 is described to return.  Walk down the homeranges:
 * the homerange [skips[k], skips[k+1]-1] without its first processor repeats
 * the baseblocks of [1, skips[k+1]-skips[k]-1]; a range [1, y] holds exactly
 * the blocks 0..home(y). */
static uint32_t range_set_linear(const uint32_t *s, int q, uint32_t a, uint32_t b)
{
    uint32_t set = 0;
    while (a <= b) {
        int k = home_of(s, q, b);
        if (a > s[k]) {            /* whole range inside homerange k, past its head */
            a -= s[k];
            b -= s[k];
        } else {                   /* a <= skips[k] <= b */
            uint32_t y = b - s[k]; /* part after the head is a copy of [1, y] */
            set |= 1u << k;
            if (y >= 1) {
                int j = home_of(s, q, y);
                set |= (2u << j) - 1u;
            }
            b = s[k] - 1;          /* continue with the part before the head */
        }
    }
    return set;
}

/* What the root adds to a range that contains it.  0 (the reading used):
 * nothing.  1: block 0, 2: every block -- only for the self-test that shows the
 * choice cannot change a schedule (the tables print 0 or -1 in that cell). */
static int g_root_mode = 0;
void bcso_set_root_mode(int mode) { g_root_mode = mode; }

/* Range search for a cyclic range given by signed end points lo <= hi + 1
 * (processor numbers are taken mod p; rank 0 contributes nothing). */
static uint32_t range_set_cyclic(const uint32_t *s, int q, uint32_t p,
                                 int64_t lo, int64_t hi)
{
    int64_t len = hi - lo + 1;
    uint32_t all = q >= 32 ? 0xffffffffu : ((1u << q) - 1u);
    uint32_t set = 0;
    int64_t a, b;
    if (len <= 0) return 0;
    if (len >= (int64_t)p) return all;
    a = lo % (int64_t)p; if (a < 0) a += p;
    b = a + len - 1;
    if (a == 0 || b >= (int64_t)p)            /* the root lies in the range */
        set = g_root_mode == 1 ? 1u : g_root_mode == 2 ? all : 0u;
    if (b < (int64_t)p) {                     /* no wrap */
        if (a == 0) a = 1;
        if (a <= b) set |= range_set_linear(s, q, (uint32_t)a, (uint32_t)b);
    } else {                                  /* [a, p-1] then [0, b-p] */
        if (a == 0) a = 1;
        set |= range_set_linear(s, q, (uint32_t)a, p - 1);
        b -= p;
        if (b >= 1) set |= range_set_linear(s, q, 1, (uint32_t)b);
    }
    return set;
}

/* Exported for tests: the range search, per-rank form. */
uint32_t bcso_rangeblocks(uint32_t p, int64_t lo, int64_t hi)
{
    uint32_t s[BCSO_MAXQ + 1];
    int q = bcso_skips(p, s);
    return range_set_cyclic(s, q, p, lo, hi);
}

/* Exported for tests: the same set by its definition -- visit every processor
 * of the cyclic range and ask Algorithm 2 for its baseblock. */
uint32_t bcso_rangeblocks_scan(uint32_t p, int64_t lo, int64_t hi)
{
    uint32_t set = 0;
    int64_t x, cnt = 0;
    for (x = lo; x <= hi && cnt < (int64_t)p; x++, cnt++) {
        int64_t m = x % (int64_t)p;
        if (m < 0) m += p;
        if (m != 0) set |= 1u << bcso_baseblock(p, (uint32_t)m);
    }
    return set;
}

static int top_bit(uint32_t v)
{
    int k = -1;
    while (v) { v >>= 1; k++; }
    return k;
}

/* Algorithm 4: receive blocks of rounds 0..last for processor r (last <= q-1).
 * special != 0: rounds 0 and q-1 as the paper writes them (baseblock of r-1;
 * the one block that is left); special == 0: the two-window rule in every
 * round.  Returns 0, or -1 if no new block was found (internal error). */
static int recv_rounds(const uint32_t *s, int q, uint32_t p, uint32_t r,
                       int last, int special, int8_t *out)
{
    uint32_t B = 0;
    uint32_t all = q >= 32 ? 0xffffffffu : ((1u << q) - 1u);
    int64_t sum = 0;                 /* sum_{j<=i} skips[j] */
    int i;
    if (r > 0) B = 1u << bcso_baseblock(p, r);
    for (i = 0; i <= last; i++) {
        sum += s[i];
        if (s[i] <= r && r < s[i + 1]) {
            out[i] = (int8_t)bcso_baseblock(p, r);
        } else {
            int b;
            if (special && i == 0) {
                b = bcso_baseblock(p, (r + p - 1) % p);
            } else if (!special || i < q - 1) {
                uint32_t U = range_set_cyclic(s, q, p, (int64_t)r - s[i + 1] + 1,
                                              (int64_t)r - s[i]) & ~B;
                if (U == 0)
                    U = range_set_cyclic(s, q, p, (int64_t)r - sum,
                                         (int64_t)r - s[i + 1]) & ~B;
                if (U == 0) return -1;
                b = top_bit(U);
            } else {
                uint32_t U = all & ~B;
                if (U == 0 || (U & (U - 1)) != 0) return -1;   /* exactly one left */
                b = top_bit(U);
            }
            B |= 1u << b;
            out[i] = (int8_t)(b - q);
        }
    }
    return 0;
}

/* Algorithm 4, exported: first last+1 receive blocks of processor r. */
int bcso_recvsched(uint32_t p, uint32_t r, int last, int special, int8_t *out)
{
    uint32_t s[BCSO_MAXQ + 1];
    int q = bcso_skips(p, s);
    if (r >= p || last >= q) return -2;
    if (last < 0) return 0;
    return recv_rounds(s, q, p, r, last, special, out);
}

/* Algorithm 5 (the straightforward variant): send block of round i is receive
 * block i of the to-processor (r + skips[i]) mod p. */
int bcso_sendsched(uint32_t p, uint32_t r, int special, int8_t *out)
{
    uint32_t s[BCSO_MAXQ + 1];
    int8_t tmp[BCSO_MAXQ];
    int q = bcso_skips(p, s);
    int i;
    if (r >= p) return -2;
    for (i = 0; i < q; i++) {
        uint32_t t = (uint32_t)(((uint64_t)r + s[i]) % p);
        int rc = recv_rounds(s, q, p, t, i, special, tmp);
        if (rc) return rc;
        out[i] = tmp[i];
    }
    return 0;
}

/* Per-rank form over a rank range: recv and send rows, rank-major, q bytes per
 * rank.  Either output may be NULL.  Parallel over ranks when built with
 * OpenMP (the construction is communication-free). */
int bcso_build_range(uint32_t p, uint64_t r_begin, uint64_t r_end, int special,
                     int8_t *recv, int8_t *send)
{
    int q = bcso_q(p);
    int err = 0;
    int64_t n = (int64_t)(r_end - r_begin), j;
    if (r_begin > r_end || r_end > p) return -2;
#pragma omp parallel for schedule(dynamic, 256)
    for (j = 0; j < n; j++) {
        uint32_t r = (uint32_t)(r_begin + j);
        if (recv && bcso_recvsched(p, r, q - 1, special, recv + (size_t)j * q)) err = -1;
        if (send && bcso_sendsched(p, r, special, send + (size_t)j * q)) err = -1;
    }
    return err;
}

/* Per-rank form on a list of ranks (spot checks at very large p). */
int bcso_build_ranks(uint32_t p, const uint64_t *ranks, uint64_t n_ranks,
                     int8_t *recv, int8_t *send)
{
    int q = bcso_q(p);
    int err = 0;
    int64_t j;
#pragma omp parallel for schedule(dynamic, 64)
    for (j = 0; j < (int64_t)n_ranks; j++) {
        uint32_t r = (uint32_t)ranks[j];
        if (recv && bcso_recvsched(p, r, q - 1, 1, recv + (size_t)j * q)) err = -1;
        if (send && bcso_sendsched(p, r, 1, send + (size_t)j * q)) err = -1;
    }
    return err;
}

/* Array form.  cnt[k][x] = number of processors 1..x whose baseblock is k, so
 * block k lies in [a, b] (1 <= a <= b < p) iff cnt[k][b] - cnt[k][a-1] > 0. */
static uint32_t window_by_counts(const uint32_t *cnt, int q, uint32_t p,
                                 int64_t lo, int64_t hi)
{
    int64_t len = hi - lo + 1, a, b;
    uint32_t set = 0;
    int k;
    if (len <= 0) return 0;
    if (len >= (int64_t)p) return q >= 32 ? 0xffffffffu : ((1u << q) - 1u);
    a = lo % (int64_t)p; if (a < 0) a += p;
    b = a + len - 1;
    for (k = 0; k < q; k++) {
        const uint32_t *c = cnt + (size_t)k * p;
        uint32_t n;
        if (b < (int64_t)p) {
            n = c[b] - (a >= 1 ? c[a - 1] : 0);
        } else {
            n = (c[p - 1] - (a >= 1 ? c[a - 1] : 0)) + c[b - p];
        }
        if (n) set |= 1u << k;
    }
    return set;
}

/* Full schedule of all p processors, array form: recv[r*q + i], send[r*q + i].
 * Returns 0, -1 (no new block found), -3 (out of memory). */
int bcso_full_table(uint32_t p, int8_t *recv, int8_t *send)
{
    uint32_t s[BCSO_MAXQ + 1];
    int q = bcso_skips(p, s);
    int8_t *bb;
    uint32_t *cnt;
    int err = 0, k;
    int64_t r;
    if (q == 0) return 0;
    bb = (int8_t *)malloc(p);
    cnt = (uint32_t *)malloc((size_t)q * p * sizeof(uint32_t));
    if (!bb || !cnt) { free(bb); free(cnt); return -3; }
    bcso_baseblock_list(p, bb);
    for (k = 0; k < q; k++) {
        uint32_t *c = cnt + (size_t)k * p;
        uint32_t x;
        c[0] = 0;
        for (x = 1; x < p; x++) c[x] = c[x - 1] + (bb[x] == k ? 1u : 0u);
    }
#pragma omp parallel for schedule(static)
    for (r = 0; r < (int64_t)p; r++) {
        uint32_t B = r > 0 ? 1u << bb[r] : 0;
        int64_t sum = 0;
        int i;
        for (i = 0; i < q; i++) {
            sum += s[i];
            if (s[i] <= (uint32_t)r && (uint32_t)r < s[i + 1]) {
                recv[(size_t)r * q + i] = bb[r];
            } else {
                uint32_t U = window_by_counts(cnt, q, p, r - s[i + 1] + 1, r - s[i]) & ~B;
                int b;
                if (U == 0)
                    U = window_by_counts(cnt, q, p, r - sum, r - s[i + 1]) & ~B;
                if (U == 0) { err = -1; b = 0; } else b = top_bit(U);
                B |= 1u << b;
                recv[(size_t)r * q + i] = (int8_t)(b - q);
            }
        }
    }
    if (send) {
        /* Algorithm 9, second loop: a lookup in the receive table. */
#pragma omp parallel for schedule(static)
        for (r = 0; r < (int64_t)p; r++) {
            int i;
            for (i = 0; i < q; i++) {
                uint64_t t = ((uint64_t)r + s[i]) % p;
                send[(size_t)r * q + i] = recv[(size_t)t * q + i];
            }
        }
    }
    free(bb);
    free(cnt);
    return err;
}

/* Algorithm 6 without the Send||Recv: the n-1+q rounds of processor r, written
 * as the paper's loop (adjust the two arrays by -x, or -x+q for the x virtual
 * rounds already done; per round use entry k = i mod q, then add q to it).
 * out[4*j + {0,1,2,3}] = send block, receive block, to-processor,
 * from-processor of round j = i - x.  Blocks above n-1 become n-1, blocks below
 * 0 become -1. */
void bcso_expand_rank(uint32_t p, uint32_t n, uint32_t r, const int8_t *recv_row,
                      const int8_t *send_row, int32_t *out)
{
    uint32_t s[BCSO_MAXQ + 1];
    int64_t rs[BCSO_MAXQ], ss[BCSO_MAXQ];
    int q = bcso_skips(p, s);
    int64_t x, i;
    if (q == 0) return;
    x = (q - ((int64_t)n - 1 + q) % q) % q;
    for (i = 0; i < q; i++) {
        if (i < x) {
            rs[i] = recv_row[i] - x + q;
            ss[i] = send_row[i] - x + q;
        } else {
            rs[i] = recv_row[i] - x;
            ss[i] = send_row[i] - x;
        }
    }
    i = x;
    while (i < (int64_t)n + q - 1 + x) {
        int k = (int)(i % q);
        int64_t t = ((int64_t)r + s[k]) % p;
        int64_t f = ((int64_t)r - s[k] + p) % p;
        int64_t sb = ss[k], rb = rs[k];
        int32_t *o = out + 4 * (i - x);
        if (sb > (int64_t)n - 1) sb = n - 1;
        if (rb > (int64_t)n - 1) rb = n - 1;
        if (sb < 0) sb = -1;
        if (rb < 0) rb = -1;
        o[0] = (int32_t)sb; o[1] = (int32_t)rb; o[2] = (int32_t)t; o[3] = (int32_t)f;
        ss[k] += q;
        rs[k] += q;
        i = i + 1;
    }
}

/* Algorithm 6 for the ranks r_begin..r_end-1; recv/send are the FULL [p][q]
 * tables; out holds (r_end-r_begin) * (n-1+q) * 4 words. */
void bcso_expand_range(uint32_t p, uint32_t n, uint64_t r_begin, uint64_t r_end,
                       const int8_t *recv, const int8_t *send, int32_t *out)
{
    int q = bcso_q(p);
    size_t rounds = (size_t)n - 1 + q;
    int64_t j, cnt = (int64_t)(r_end - r_begin);
#pragma omp parallel for schedule(static)
    for (j = 0; j < cnt; j++) {
        uint64_t r = r_begin + j;
        bcso_expand_rank(p, n, (uint32_t)r, recv + r * q, send + r * q,
                         out + (size_t)j * rounds * 4);
    }
}

/* Algorithm 7 (regular allgather) without the data: for processor r and round k
 * out[4k..4k+3] = to-processor (r - skips[k] + p) mod p, from-processor
 * (r + skips[k]) mod p, number of blocks exchanged skips[k+1] - skips[k] (blocks
 * 0..count-1 of the buffer are sent), offset skips[k] at which the received
 * blocks are stored.  The edges run opposite to the broadcast's. */
void bcso_allgather_rounds(uint32_t p, uint32_t r, int32_t *out)
{
    uint32_t s[BCSO_MAXQ + 1];
    int q = bcso_skips(p, s), k;
    for (k = 0; k < q; k++) {
        out[4 * k + 0] = (int32_t)(((int64_t)r - s[k] + p) % p);
        out[4 * k + 1] = (int32_t)(((int64_t)r + s[k]) % p);
        out[4 * k + 2] = (int32_t)(s[k + 1] - s[k]);
        out[4 * k + 3] = (int32_t)s[k];
    }
}

/* Algorithm 8 (census / allreduce) without the data: for processor r and round
 * k out[4k..4k+3] = to-processor, from-processor, 1 if the value sent is
 * x_r (+) S and 0 if it is S alone, 0.  When skips[k] + skips[k] > skips[k+1]
 * the edges are shortened by one and S alone is sent (the listing tests
 * skips[i]; the round index k is meant). */
void bcso_census_rounds(uint32_t p, uint32_t r, int32_t *out)
{
    uint32_t s[BCSO_MAXQ + 1];
    int q = bcso_skips(p, s), k;
    for (k = 0; k < q; k++) {
        if ((uint64_t)s[k] + s[k] > s[k + 1]) {
            out[4 * k + 0] = (int32_t)(((int64_t)r - s[k] + 1 + p) % p);
            out[4 * k + 1] = (int32_t)(((int64_t)r + s[k] - 1) % p);
            out[4 * k + 2] = 0;
        } else {
            out[4 * k + 0] = (int32_t)(((int64_t)r - s[k] + p) % p);
            out[4 * k + 1] = (int32_t)(((int64_t)r + s[k]) % p);
            out[4 * k + 2] = 1;
        }
        out[4 * k + 3] = 0;
    }
}

/* Algorithm 9 without the data movement, for processor r: which block of
 * buffer[j] is packed (sent) and which is unpacked (received) in every round.
 * The full schedule is given (recv / send are the [p][q] tables of a root-0
 * broadcast); working copies are adjusted as Algorithm 6 does (-x, and +q for
 * the x entries whose first use falls into the second phase) -- Algorithm 9
 * as printed leaves this adjustment out, without it the first real round
 * would use block x instead of block 0 -- and then every use of an entry adds
 * q to it, exactly as the pack and unpack loops are written.
 * pack[jr * p + j], unpack[jr * p + j] for round jr = i - x and buffer j:
 * block numbers after the rule "below 0: nothing (-1), above n-1: n-1".
 * Returns -3 if out of memory. */
int bcso_allgather_rank(uint32_t p, uint32_t n, uint32_t r, const int8_t *recv,
                        const int8_t *send, int adjust, int32_t *pack, int32_t *unpack)
{
    uint32_t s[BCSO_MAXQ + 1];
    int q = bcso_skips(p, s);
    int64_t *rs, *ss, x, i, j, k;
    if (q == 0) return 0;
    rs = (int64_t *)malloc((size_t)p * q * sizeof(int64_t));
    ss = (int64_t *)malloc((size_t)p * q * sizeof(int64_t));
    if (!rs || !ss) { free(rs); free(ss); return -3; }
    x = (q - ((int64_t)n - 1 + q) % q) % q;
    for (j = 0; j < (int64_t)p; j++)
        for (k = 0; k < q; k++) {
            int64_t adj = !adjust ? 0 : k < x ? -x + q : -x;   /* adjust == 0: as printed (self-test) */
            rs[j * q + k] = recv[j * q + k] + adj;
            ss[j * q + k] = send[j * q + k] + adj;
        }
    i = x;
    while (i < (int64_t)n + q - 1 + x) {
        int64_t jr = i - x;
        k = i % q;
        for (j = 0; j < (int64_t)p; j++) {            /* pack */
            int64_t rr = ((int64_t)r - j + p) % p, b = ss[rr * q + k];
            if (b > (int64_t)n - 1) b = n - 1;
            if (b < 0) b = -1;
            pack[jr * p + j] = (int32_t)b;
            ss[rr * q + k] += q;
        }
        for (j = 0; j < (int64_t)p; j++) {            /* unpack */
            int64_t rr = ((int64_t)r - j + p) % p, b = rs[rr * q + k];
            if (b > (int64_t)n - 1) b = n - 1;
            if (b < 0) b = -1;
            unpack[jr * p + j] = (int32_t)b;
            rs[rr * q + k] += q;
        }
        i = i + 1;
    }
    free(rs); free(ss);
    return 0;
}

/* Position-weighted 64-bit checksum of a stretch of schedule entries (not from
 * the paper: a tool for comparing outputs too large to copy).  Entry number e
 * of the whole stream is byte e mod 4 of the little-endian 32-bit word
 * g = floor(e / 4); the sum is  sum_e (byte_e << 8 (e mod 4)) * weight(g)  mod
 * 2^64 with weight(g) = fmix32(low32(g) ^ 0x9E3779B9 * high32(g)) | 1, fmix32
 * being the finaliser of MurmurHash3 (Appleby, public domain). */
static uint32_t murmur3_fmix32(uint32_t h)
{
    h ^= h >> 16;
    h *= 0x85ebca6bu;
    h ^= h >> 13;
    h *= 0xc2b2ae35u;
    h ^= h >> 16;
    return h;
}

uint64_t bcso_checksum(const int8_t *buf, uint64_t n_entries, uint64_t first_index)
{
    uint64_t sum = 0, e;
    for (e = 0; e < n_entries; e++) {
        uint64_t pos = first_index + e;
        uint64_t g = pos / 4;
        uint32_t w = murmur3_fmix32((uint32_t)g ^ (0x9E3779B9u * (uint32_t)(g >> 32))) | 1u;
        sum += ((uint64_t)(uint8_t)buf[e] << (8 * (pos % 4))) * (uint64_t)w;
    }
    return sum;
}

/* Counts the ranks r_begin..r_end-1 whose rows break what the text after
 * Theorem 1 and Algorithms 5 / 9 promise (the same three counts the library's
 * checker reports; recv / send hold the rows of the range, either may be NULL):
 *   counts[0] receive row: baseblock (Algorithm 2) exactly in the home round,
 *             all other entries negative, their blocks b = entry + q different
 *             from each other and from the baseblock;
 *   counts[1] send row: root sends k in round k; others send a previous-phase
 *             block received in an earlier round of the row, or the own
 *             baseblock of the previous phase, or -- after the home round -- the
 *             baseblock of the current phase;
 *   counts[2] send[r][k] != recv[(r + skips[k]) mod p][k] for a to-processor
 *             inside the range. */
void bcso_validate(uint32_t p, uint64_t r_begin, uint64_t r_end, const int8_t *recv,
                   const int8_t *send, uint64_t *counts)
{
    uint32_t s[BCSO_MAXQ + 1];
    int q = bcso_skips(p, s);
    uint64_t j, n = r_end - r_begin;
    counts[0] = counts[1] = counts[2] = 0;
    for (j = 0; j < n; j++) {
        uint32_t r = (uint32_t)(r_begin + j);
        const int8_t *rr = recv ? recv + j * q : NULL, *sr = send ? send + j * q : NULL;
        int bb = bcso_baseblock(p, r), h = -1, k, bad;
        for (k = 0; k < q; k++)
            if (s[k] <= r && r < s[k + 1]) h = k;
        if (rr) {
            int used[BCSO_MAXQ + 1] = {0};
            bad = 0;
            if (bb >= 0) used[bb] = 1;
            for (k = 0; k < q; k++) {
                if (k == h) {
                    if (rr[k] != bb) bad = 1;
                } else {
                    int b = rr[k] + q;
                    if (rr[k] >= 0 || b < 0 || used[b]) bad = 1;
                    else used[b] = 1;
                }
            }
            counts[0] += bad;
        }
        if (sr) {
            int have[BCSO_MAXQ + 1] = {0};
            bad = 0;
            if (bb >= 0) have[bb] = 1;
            for (k = 0; k < q; k++) {
                if (r == 0) {
                    if (sr[k] != k) bad = 1;
                } else if (!(k > h && sr[k] == bb)) {
                    int b = sr[k] + q;
                    if (sr[k] >= 0 || b < 0 || (rr && !have[b])) bad = 1;
                }
                if (rr && k != h && rr[k] < 0 && rr[k] + q >= 0) have[rr[k] + q] = 1;
            }
            counts[1] += bad;
        }
        if (rr && sr) {
            bad = 0;
            for (k = 0; k < q; k++) {
                uint64_t t = ((uint64_t)r + s[k]) % p;
                if (t >= r_begin && t < r_end && recv[(t - r_begin) * q + k] != sr[k]) bad = 1;
            }
            counts[2] += bad;
        }
    }
}

/* Brute-force run of Algorithm 6 for all p ranks at once (rank 0 holds the n
 * blocks, n <= 64): every rank's rounds come from the literal loop of
 * bcso_expand_rank; counts as the library's simulator reports them:
 *   [0] sends of a block the sender does not hold, [1] rounds in which what r
 *   sends is not what its to-processor receives, [2] receipts by a non-root
 *   rank of a block it already has, [3] ranks incomplete after the last round,
 *   [4] ranks already complete before the last round.  Returns -3 if out of
 *   memory, -2 for n > 64. */
int bcso_simulate(uint32_t p, uint32_t n, const int8_t *recv, const int8_t *send,
                  uint64_t *counts)
{
    int q = bcso_q(p);
    size_t rounds = (size_t)n - 1 + q, j;
    uint64_t all = n >= 64 ? ~(uint64_t)0 : (((uint64_t)1 << n) - 1);
    uint64_t *held, *next, r;
    int32_t *tab;
    counts[0] = counts[1] = counts[2] = counts[3] = counts[4] = 0;
    if (n > 64) return -2;
    if (q == 0) return 0;
    held = (uint64_t *)calloc(p, sizeof(uint64_t));
    next = (uint64_t *)calloc(p, sizeof(uint64_t));
    tab = (int32_t *)malloc((size_t)p * rounds * 4 * sizeof(int32_t));
    if (!held || !next || !tab) { free(held); free(next); free(tab); return -3; }
    for (r = 0; r < p; r++)
        bcso_expand_rank(p, n, (uint32_t)r, recv + r * q, send + r * q, tab + r * rounds * 4);
    held[0] = all;
    for (j = 0; j < rounds; j++) {
        for (r = 0; r < p; r++) {
            const int32_t *o = tab + (r * rounds + j) * 4;
            int32_t sb = o[0], rb = o[1], to = o[2];
            if (sb >= 0 && !((held[r] >> sb) & 1)) counts[0]++;
            if (tab[((size_t)to * rounds + j) * 4 + 1] != sb) counts[1]++;
            next[r] = held[r];
            if (rb >= 0) {
                if (r != 0 && ((held[r] >> rb) & 1)) counts[2]++;
                next[r] |= (uint64_t)1 << rb;
            }
            if (j + 1 == rounds && held[r] == all) counts[4]++;
        }
        { uint64_t *t = held; held = next; next = t; }
    }
    for (r = 0; r < p; r++)
        if (held[r] != all) counts[3]++;
    free(held); free(next); free(tab);
    return 0;
}

int bcso_num_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
