/*
 * skipcode_mirror.c -- CPU restatement, with operation counters, of the construction that the
 * fast CUDA kernels run (TEST INFRASTRUCTURE; shares no code with the kernels or the oracle).
 *
 * The kernels do not descend the homeranges as Algorithm 3 of arXiv 2205.10072 does.  They give
 * every rank x a "skip code": x is written as a sum of distinct skips, largest first (the sums
 * that Algorithm 2 walks down), and bit k of code(x) says whether skips[k] is a term.  The
 * lowest set bit is the baseblock of x, the highest its homerange, and codes order like ranks.
 * The largest baseblock among the ranks x+1..y is then the highest bit in which code(x) and
 * code(y) differ; everything Algorithm 4 needs per round (the largest block of a window that is
 * not in B yet) follows from the two codes that bound the window.
 *
 * This file computes receive and send rows that way, one rank at a time, in plain C, and counts
 * the integer operations an ideal translation of each step needs (no address arithmetic beyond
 * what the step itself requires, no loop overhead).  The tests compare its rows with the
 * oracle's; the benchmark takes its operation counts as the model numerator of the integer
 * roofline.  Operations shared by the four consecutive ranks that a GPU thread handles are
 * counted as a quarter each: all counters are in QUARTER operations.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define SKM_MAX_Q 31
#define Q4(n) ((uint64_t)(4 * (n)))     /* n whole operations, in quarter operations */

enum {
    SKM_RANKS = 0,          /* ranks whose receive row was built                                */
    SKM_CODE_OPS,           /* skip codes (one scan per block of 32 ranks); homerange, baseblock, B */
    SKM_TABLE_OPS,          /* rounds decided from the window's exact block set (short windows)  */
    SKM_HEAD_OPS,           /* rounds decided by the first head                                  */
    SKM_STEP2_OPS,          /* extra work when the first head was taken and the second step decides */
    SKM_REST_OPS,           /* extra work of the full search and of the second window            */
    SKM_HOME_OPS,           /* the home round                                                    */
    SKM_STORE_OPS,          /* row byte and the share of the packed column word, per entry       */
    SKM_SEND_OPS,           /* send row by lookup in the round-major receive table               */
    SKM_ROUNDS_TABLE, SKM_ROUNDS_HEAD, SKM_ROUNDS_STEP2, SKM_ROUNDS_REST, SKM_ROUNDS_SECOND,
    SKM_ROUNDS_HOME,
    SKM_NCOUNT
};

typedef struct {
    uint32_t p;
    int q;
    uint32_t s[SKM_MAX_Q + 2];       /* skips[0..q] */
    uint32_t full[SKM_MAX_Q + 2];    /* full[d] = code(skips[d] - 1) */
    uint32_t len2[SKM_MAX_Q + 1];    /* ranks in the second window of round i */
    int table_rounds;                /* rounds 0..table_rounds-1 have windows within 41 ranks */
    const uint32_t *codes;           /* codes of all ranks when the caller has them, else NULL */
} skm_ctx;

/* Which rounds are decided from exact window sets: 0 = as the GPU kernels do (the rounds with
 * skips[i+1] <= 33 when p >= 64), 1 = none (every round by the code search), 2 = those rounds
 * for every p.  All three must give the same rows. */
static int g_table_mode = 0;
void skm_set_table_mode(int mode) { g_table_mode = mode; }

static int top_bit(uint32_t v) { return v ? 31 - __builtin_clz(v) : -1; }

/* Greedy decomposition of x into skips, largest first. */
static uint32_t code_of(const skm_ctx *c, uint32_t x)
{
    if (c->codes) return c->codes[x];
    uint32_t code = 0;
    for (int k = c->q - 1; k >= 0; --k)
        if (x >= c->s[k]) { x -= c->s[k]; code |= 1u << k; }
    return code;
}

static void ctx_init(skm_ctx *c, uint32_t p)
{
    memset(c, 0, sizeof *c);
    c->p = p;
    int q = 0;
    while (((uint64_t)1 << q) < p) ++q;
    c->q = q;
    uint32_t v = p;
    for (int k = q; k >= 0; --k) { c->s[k] = v; v = (v + 1) / 2; }
    for (int d = 0; d <= q; ++d) c->full[d] = code_of(c, c->s[d] - 1);
    uint64_t sum = 0;
    for (int i = 0; i < q; ++i) {
        sum += c->s[i];
        c->len2[i] = sum >= c->s[i + 1] ? (uint32_t)(sum - c->s[i + 1] + 1) : 0;
    }
    if (g_table_mode == 2 || (g_table_mode == 0 && p >= 64))
        while (c->table_rounds < q && c->table_rounds < 6 && c->s[c->table_rounds + 1] <= 33)
            ++c->table_rounds;
}

/* Largest block not in B among the baseblocks of the ranks x+1..y, given X = code(x) and
 * F = code(y), x <= y; -1 if there is none.  *ops is charged with the operations of every
 * step taken. */
static int search_codes(const skm_ctx *c, uint32_t X, uint32_t F, uint32_t B, uint64_t *ops)
{
    uint32_t low = 0;                       /* blocks 0..m known to be in the range, as a mask */
    for (;;) {
        uint32_t diff = X ^ F;              *ops += Q4(2);   /* xor, test */
        if (diff == 0) break;
        int d = top_bit(diff);
        uint32_t bit = 1u << d;             *ops += Q4(3);   /* leading bit, shift, compare with low */
        if (bit <= low) break;              /* this head and all later ones are already in `low` */
        *ops += Q4(2);                      /* and, test */
        if (!(B & bit)) return d;
        /* behind the head: a copy of the ranks 1..rest(y), which hold the blocks 0..top(rest) */
        uint32_t rest = F & (bit - 1);      *ops += Q4(2);
        if (rest) { low |= (2u << top_bit(rest)) - 1; *ops += Q4(4); }
        /* before the head: rest(x)+1 .. skips[d]-1 inside a copy of 1..skips[d]-1 */
        X &= bit - 1;
        F = c->full[d];                     *ops += Q4(2);
    }
    uint32_t U = low & ~B;                  *ops += Q4(3);
    return top_bit(U);
}

/* The same for the `len` ranks that end at rank e (mod p); the root holds no block. */
static int search_cyclic(const skm_ctx *c, uint32_t e, uint32_t len, uint32_t B, uint64_t *ops)
{
    const uint32_t p = c->p;
    *ops += Q4(2);
    if (len == 0) return -1;
    if (len >= p) return top_bit(((c->q >= 32) ? 0xffffffffu : ((1u << c->q) - 1)) & ~B);
    if (e >= len) {                          /* ranks e-len+1 .. e, all at least 1 */
        *ops += Q4(2);                       /* one more code: the rank just before the window */
        return search_codes(c, code_of(c, e - len), code_of(c, e), B, ops);
    }
    /* the window reaches the root: ranks p-(len-e)+1 .. p-1 (if any), then 1 .. e (if any) */
    uint32_t over = len - e;                 /* ranks at or before the root, root included */
    int b1 = -1, b2 = -1;
    *ops += Q4(4);
    if (over >= 2) b1 = search_codes(c, code_of(c, p - over), c->full[c->q], B, ops);
    if (e >= 1) b2 = search_codes(c, 0, code_of(c, e), B, ops);
    return b1 > b2 ? b1 : b2;
}

/* Exact set of the baseblocks of the `len` ranks ending `back` ranks below r (mod p), root
 * excluded: what the tile's table of OR-ed baseblock bits delivers for a short window. */
static uint32_t window_set(const skm_ctx *c, uint32_t r, uint32_t back, uint32_t len)
{
    uint32_t set = 0;
    for (uint32_t j = 0; j < len; ++j) {
        uint64_t x = ((uint64_t)r + c->p - (back + j) % c->p) % c->p;
        uint32_t cx = code_of(c, (uint32_t)x);
        set |= cx & (0u - cx);               /* lowest set bit; 0 for the root */
    }
    return set;
}

/* Receive entries of rounds 0..last of rank r (Algorithm 4 on skip codes). */
static void recv_row(const skm_ctx *c, uint32_t r, int last, int8_t *row, uint64_t *cnt)
{
    const uint32_t p = c->p;
    const int q = c->q;
    uint32_t own = code_of(c, r);
    int h = top_bit(own);                     /* homerange; -1 for the root */
    int bb = own ? __builtin_ctz(own) : 0;    /* baseblock */
    uint32_t B = own ? 1u << bb : 0;
    if (cnt) {
        cnt[SKM_RANKS] += 1;
        cnt[SKM_CODE_OPS] += Q4(3);           /* h, bb, B from the rank's code; the code itself is
                                                 charged by the caller, per block of 32 ranks */
    }
    uint64_t dummy[SKM_NCOUNT];
    if (!cnt) { memset(dummy, 0, sizeof dummy); cnt = dummy; }
    for (int i = 0; i <= last; ++i) {
        const uint32_t lo = c->s[i], hi = c->s[i + 1];
        int entry;
        if (i == h) {
            entry = bb;                                            /* the baseblock itself */
            cnt[SKM_HOME_OPS] += Q4(1);
            cnt[SKM_ROUNDS_HOME] += 1;
        } else if (i < c->table_rounds) {
            /* Short windows: both windows as exact block sets (on the GPU four words of the
             * tile's run table: 4 loads, 2 or, 2 and-not), first window unless it is empty of
             * new blocks (1 select), then leading bit, its mask, entry, set update. */
            uint32_t U = window_set(c, r, lo, hi - lo) & ~B;
            if (U == 0 && c->len2[i]) U = window_set(c, r, hi, c->len2[i]) & ~B;
            cnt[SKM_TABLE_OPS] += Q4(4 + 2 + 2 + 1 + 4);
            cnt[SKM_ROUNDS_TABLE] += 1;
            int blk = top_bit(U);
            if (blk >= 0) B |= 1u << blk;
            entry = blk >= 0 ? blk - q : 127;
        } else {
            /* window of round i: the ranks below+1 .. above with below = r - skips[i+1],
             * above = r - skips[i] (both mod p; both wrapped past the home round, neither before) */
            const uint32_t below = (uint32_t)(((uint64_t)r + p - hi) % p);
            const uint32_t above = (uint32_t)(((uint64_t)r + p - lo) % p);
            const uint32_t lower = code_of(c, below), upper = code_of(c, above);
            /* address of the lower code: shared by the four ranks of a thread (1/4); its load;
             * the upper code is last round's lower one */
            cnt[SKM_HEAD_OPS] += 1 + Q4(1);
            const uint32_t diff = lower ^ upper;
            const int d = top_bit(diff);
            const uint32_t bit = d >= 0 ? 1u << d : 0;
            const uint32_t fresh = bit & ~B;
            cnt[SKM_HEAD_OPS] += Q4(5 + 2);      /* xor, leading bit, shift, and-not, test; or into B, entry */
            int blk;
            if (fresh) {
                blk = d;
                cnt[SKM_ROUNDS_HEAD] += 1;
            } else {
                /* second step of the search, decided without a loop when it ends there: the
                 * head is taken, the run of low blocks behind it has a new block, and the next
                 * head (before the first one) is not above that run */
                blk = -1;
                int decided = 0;
                if (diff != 0) {
                    const uint32_t below_head = bit - 1;
                    const uint32_t rest = upper & below_head;
                    const uint32_t low = rest ? (2u << top_bit(rest)) - 1 : 0;
                    const uint32_t diff2 = (lower & below_head) ^ c->full[d];
                    const uint32_t news = low & ~B;
                    cnt[SKM_STEP2_OPS] += Q4(12);
                    if (news != 0 && (diff2 == 0 || (1u << top_bit(diff2)) <= low)) {
                        blk = top_bit(news);
                        decided = 1;
                        cnt[SKM_ROUNDS_STEP2] += 1;
                    }
                }
                if (!decided) {
                    cnt[SKM_ROUNDS_REST] += 1;
                    blk = diff ? search_codes(c, lower, upper, B, &cnt[SKM_REST_OPS]) : -1;
                    if (blk < 0) {
                        cnt[SKM_ROUNDS_SECOND] += 1;
                        blk = search_cyclic(c, below, c->len2[i], B, &cnt[SKM_REST_OPS]);
                    }
                }
            }
            if (blk >= 0) B |= 1u << blk;
            entry = blk >= 0 ? blk - q : 127;
        }
        /* the entry's byte in the rank-major row, and its share of the round's packed word of
         * four ranks in the round-major copy (3 byte merges and 1 store per four entries) */
        cnt[SKM_STORE_OPS] += Q4(1) + 4;
        if (row) row[i] = (int8_t)entry;
    }
}

/* ------------------------------------------------------------------ codes, 32 ranks per scan
 * The codes of 32 consecutive ranks g .. g+31 (16 for q <= 22) from one greedy scan.  Rank g+e decides like g
 * at every level until the one where the remainder R of g has R < skips[k] <= R + e: there g+e
 * takes skips[k] and keeps R + e - skips[k] < 31, and g does not take it.  The levels below LOW
 * come from a table, low[v] = code of v over those levels (v < skips[LOW]), which also serves
 * the small remainders of the ranks that left.  One such level per block is recorded; a second
 * one sends the block to the plain scan (none has been seen for any p tried).
 * Operations charged (whole operations, to ops[0]): per level of the scan 5 (subtract, the two
 * tests, select, or), 3 more at a splitting level; per four ranks 3 for the side of the split and
 * the table address, 4 table loads, 4 or, 1 vector store, and 8 more where the split falls
 * inside the four; the table's 3 per level and entry once per 256 blocks; a plain scan 3 per
 * level and rank.  ops[1] = blocks, ops[2] = blocks with a splitting level, ops[3] = plain. */
#define SKM_LOW 8
#define SKM_BLOCK 32          /* ranks per scan for q > 22; 16 for a smaller p */
static int g_batch = 0;       /* the batch kernel scans 32 ranks at a time for every q */
void skm_set_batch(int on) { g_batch = on; }
static uint32_t block_of(int q) { return (q <= 22 && !g_batch) ? 16u : SKM_BLOCK; }
#define SKM_BLOCKS_FROM 8192   /* smaller p are charged the plain scan, 3 per level and rank (the
                                  GPU scans them rank by rank: most blocks would cross p) */

static void codes_block(const skm_ctx *c, const uint16_t *low, int low_levels, uint32_t g,
                        uint32_t *out /* 32, or NULL */, uint64_t *ops)
{
    const uint32_t p = c->p;
    const uint32_t block = block_of(c->q);
    uint32_t rem = g, code = 0, stay = block, left = 0;
    int plain = 0;
    for (int k = c->q - 1; k >= low_levels; --k) {
        const uint32_t skip = c->s[k];
        ops[0] += 5;
        if (rem < skip && skip <= rem + (block - 1)) {
            ops[0] += 3;
            if (stay == block) { stay = skip - rem; left = code | (1u << k); }
            else plain = 1;
        }
        if (rem >= skip) { rem -= skip; code |= 1u << k; }
    }
    ops[1] += 1;
    if (stay != block) ops[2] += 1;
    if (plain) ops[3] += 1;
    for (uint32_t e0 = 0; e0 < block && g + e0 < p; e0 += 4) {
        if (plain) ops[0] += 4ull * 3 * (uint64_t)c->q;
        else ops[0] += 12 + ((stay > e0 && stay < e0 + 4) ? 8 : 0);
        for (uint32_t e = e0; e < e0 + 4 && g + e < p; ++e) {
            uint32_t v;
            if (plain) {
                uint32_t x = g + e;
                v = 0;
                for (int k = c->q - 1; k >= 0; --k)
                    if (x >= c->s[k]) { x -= c->s[k]; v |= 1u << k; }
            } else if (e < stay) {
                v = code | low[rem + e];
            } else {
                v = left | low[e - stay];
            }
            if (out) out[e] = v;
        }
    }
}

static int build_low(const skm_ctx *c, uint16_t *low /* 1 << SKM_LOW */)
{
    const int levels = c->q < SKM_LOW ? c->q : SKM_LOW;
    for (uint32_t v = 0; v < (1u << levels); ++v) {
        uint32_t x = v, code = 0;
        for (int k = levels - 1; k >= 0; --k)
            if (x >= c->s[k]) { x -= c->s[k]; code |= 1u << k; }
        low[v] = (uint16_t)code;
    }
    return levels;
}

/* Codes of the ranks g_begin .. g_end-1 (g_begin a multiple of 32); codes may be NULL (count
 * only); ops[4] accumulated as described above. */
int skm_codes_blocks(uint32_t p, uint64_t g_begin, uint64_t g_end, uint32_t *codes, uint64_t *ops)
{
    if (p == 0 || p > 0x7fffffffu || g_begin % SKM_BLOCK || g_begin > g_end || g_end > p || ops == NULL)
        return -1;
    skm_ctx c;
    ctx_init(&c, p);
    uint16_t low[1 << SKM_LOW];
    const int levels = build_low(&c, low);
    uint32_t tmp[SKM_BLOCK];
    const uint32_t block = block_of(c.q);
    for (uint64_t g = g_begin; g < g_end; g += block) {
        if ((g - g_begin) % (256u * block) == 0) ops[0] += (3ull * levels) << levels;
        codes_block(&c, low, levels, (uint32_t)g, tmp, ops);
        if (codes)
            for (uint32_t e = 0; e < block && g + e < g_end; ++e) codes[g - g_begin + e] = tmp[e];
    }
    return 0;
}

/* The same codes by the plain scan, rank by rank (what skm_codes_blocks must reproduce). */
int skm_codes_plain(uint32_t p, uint64_t g_begin, uint64_t g_end, uint32_t *codes)
{
    if (p == 0 || p > 0x7fffffffu || g_begin > g_end || g_end > p || codes == NULL) return -1;
    skm_ctx c;
    ctx_init(&c, p);
    for (uint64_t g = g_begin; g < g_end; ++g) codes[g - g_begin] = code_of(&c, (uint32_t)g);
    return 0;
}

/* ------------------------------------------------------------ small p, everything in one block
 * What the batch kernel for p <= 1024 does: the baseblock bits of all ranks as level 0 of a table
 * run[l][x] = bits of the 2^l ranks that end at x (cyclically; the root has no bit), one level
 * from the one below; a window of L ranks that ends at rank e is run[l][e] | run[l][e - (L - 2^l)]
 * with l = floor(log2 L); every round of every rank looks its first window up, and the second one
 * when the first holds nothing new.  Operations charged (whole operations): the code of a rank 3
 * per level; a table entry 4 (index, wrap, two loads counted as one, or); a round 6 for what the
 * round shares among the ranks of a thread (a quarter each), then 3 for the window's end, 3 for
 * the other run's index, 2 loads, 2 for or / and-not, 1 test, 3 for leading bit, bit and B, 2 for
 * the entry, 1 store; a second window 10 more; the home round 2; a send entry 5 (to-processor,
 * wrap, index, load, store). */
#define SKM_SMALL_MAX 1024

int skm_small(uint32_t p, int8_t *recv, int8_t *send, uint64_t *counters)
{
    if (p == 0 || p > SKM_SMALL_MAX || recv == NULL) return -1;
    skm_ctx c;
    ctx_init(&c, p);
    const int q = c.q;
    if (q == 0) return 0;
    static uint16_t run[10][SKM_SMALL_MAX];
    uint32_t code[SKM_SMALL_MAX];
    uint64_t ops = 0;
    for (uint32_t x = 0; x < p; ++x) {
        uint32_t v = x, cd = 0;
        for (int k = q - 1; k >= 0; --k)
            if (v >= c.s[k]) { v -= c.s[k]; cd |= 1u << k; }
        code[x] = cd;
        run[0][x] = (uint16_t)(cd & (0u - cd));
        ops += 3ull * q + 2;
    }
    const int top = top_bit(p - 1);
    for (int l = 1; l <= top; ++l) {
        const uint32_t half = 1u << (l - 1);
        for (uint32_t x = 0; x < p; ++x) {
            run[l][x] = run[l - 1][x] | run[l - 1][(x + p - half) % p];
            ops += 4;
        }
    }
    uint64_t rounds_first = 0, rounds_second = 0, rounds_home = 0;
    for (uint32_t r = 0; r < p; ++r) {
        const uint32_t cd = code[r];
        const int h = top_bit(cd);
        uint32_t B = cd & (0u - cd);
        ops += 3;
        for (int i = 0; i < q; ++i) {
            const uint32_t lo = c.s[i], hi = c.s[i + 1];
            int entry;
            if (i == h) {
                entry = cd ? __builtin_ctz(cd) : 0;
                ops += 2;
                rounds_home += 1;
            } else {
                const uint32_t len1 = hi - lo;
                const int l1 = top_bit(len1);
                const uint32_t e = (r + p - lo) % p;
                uint32_t U = (run[l1][e] | run[l1][(e + p - (len1 - (1u << l1))) % p]) & ~B;
                ops += 2 + 17;                       /* 6/4 rounded up for the shared part */
                rounds_first += 1;
                if (U == 0) {
                    const uint32_t len = c.len2[i];
                    if (len >= p) U = ((1u << q) - 1u) & ~B;
                    else if (len) {
                        const int l2 = top_bit(len);
                        const uint32_t e2 = (r + p - hi % p) % p;
                        U = (run[l2][e2] | run[l2][(e2 + p - (len - (1u << l2))) % p]) & ~B;
                    }
                    ops += 10;
                    rounds_second += 1;
                }
                const int blk = top_bit(U);
                if (blk >= 0) B |= 1u << blk;
                entry = blk >= 0 ? blk - q : 127;
            }
            recv[(uint64_t)r * q + i] = (int8_t)entry;
        }
    }
    if (send) {
        for (uint32_t r = 0; r < p; ++r)
            for (int k = 0; k < q; ++k)
                send[(uint64_t)r * q + k] = recv[(uint64_t)((r + c.s[k]) % p) * q + k];
    }
    if (counters) {
        counters[SKM_RANKS] += p;
        counters[SKM_TABLE_OPS] += Q4(ops);
        counters[SKM_SEND_OPS] += Q4(5ull * p * q);
        counters[SKM_ROUNDS_TABLE] += rounds_first;
        counters[SKM_ROUNDS_SECOND] += rounds_second;
        counters[SKM_ROUNDS_HOME] += rounds_home;
    }
    return 0;
}

/* ------------------------------------------------------------------------------------ API */
int skm_q(uint32_t p)
{
    skm_ctx c;
    ctx_init(&c, p);
    return c.q;
}

/* Receive and send rows of the listed ranks.  recv, send: n * q bytes, rank-major; either may
 * be NULL.  A send entry is the receive entry of the to-processor in that round; the counters
 * charge it as the GPU obtains it -- a lookup in the round-major receive table (per four
 * entries two word loads, a funnel shift, three byte merges and a store: 7/4 per entry). */
int skm_rows(uint32_t p, const uint64_t *ranks, uint64_t n, int8_t *recv, int8_t *send,
             uint64_t *counters /* SKM_NCOUNT, accumulated */)
{
    if (p == 0 || p > 0x7fffffffu) return -1;
    skm_ctx c;
    ctx_init(&c, p);
    const int q = c.q;
    int8_t tmp[SKM_MAX_Q + 1];
    uint16_t low[1 << SKM_LOW];
    const int levels = build_low(&c, low);
    uint64_t block_ops[4] = {0, 0, 0, 0};
    for (uint64_t m = 0; m < n; ++m) {
        const uint32_t r = (uint32_t)ranks[m];
        if (r >= p) return -2;
        if (p >= SKM_BLOCKS_FROM) codes_block(&c, low, levels, r & ~(block_of(q) - 1u), NULL, block_ops);
        if (recv) recv_row(&c, r, q - 1, recv + m * (uint64_t)q, counters);
        else recv_row(&c, r, q - 1, tmp, counters);
        if (send) {
            for (int k = 0; k < q; ++k) {
                const uint32_t to = (uint32_t)(((uint64_t)r + c.s[k]) % p);
                recv_row(&c, to, k, tmp, NULL);
                send[m * (uint64_t)q + k] = tmp[k];
                if (counters) counters[SKM_SEND_OPS] += 7;
            }
        }
    }
    /* every listed rank pays 1/32 of its block's scan and of the table's share of 32 ranks */
    if (counters && p >= SKM_BLOCKS_FROM)
        counters[SKM_CODE_OPS] += Q4(block_ops[0]) / block_of(q) + Q4(n * ((3ull * levels) << levels)) / (256u * block_of(q));
    else if (counters)
        counters[SKM_CODE_OPS] += Q4(n * 3ull * (uint64_t)q);
    return 0;
}

/* All ranks of p: recv and send are p * q bytes each (send may be NULL). */
int skm_full(uint32_t p, int8_t *recv, int8_t *send, uint64_t *counters)
{
    if (p == 0 || p > 0x7fffffffu || recv == NULL) return -1;
    skm_ctx c;
    ctx_init(&c, p);
    const int q = c.q;
    uint32_t *codes = (uint32_t *)malloc((size_t)p * sizeof(uint32_t));
    if (codes == NULL) return -3;
    uint64_t block_ops[4] = {0, 0, 0, 0};
    if (skm_codes_blocks(p, 0, p, codes, block_ops) != 0) { free(codes); return -4; }
    if (counters) counters[SKM_CODE_OPS] += p >= SKM_BLOCKS_FROM ? Q4(block_ops[0]) : Q4(3ull * p * (uint64_t)q);
    c.codes = codes;
    for (uint32_t r = 0; r < p; ++r) recv_row(&c, r, q - 1, recv + (uint64_t)r * q, counters);
    free(codes);
    if (send) {
        for (uint32_t r = 0; r < p; ++r)
            for (int k = 0; k < q; ++k) {
                const uint32_t to = (uint32_t)(((uint64_t)r + c.s[k]) % p);
                send[(uint64_t)r * q + k] = recv[(uint64_t)to * q + k];
            }
        if (counters) counters[SKM_SEND_OPS] += 7ull * p * q;
    }
    return 0;
}

int skm_ncount(void) { return SKM_NCOUNT; }
