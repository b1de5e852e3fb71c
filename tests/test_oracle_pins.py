"""Pins for the CPU oracle: everything here compares the oracle with something that is NOT the
oracle -- the schedules printed in the paper, a brute-force broadcast simulation, closed forms,
the paper's lemmas, and brute-force definitions on tiny inputs."""
import numpy as np
import pytest

import oracle
from tests import bcast_sim
from tests.golden_tables import SECOND_P9, TABLES, load


# ---------------------------------------------------------------- printed worked examples
@pytest.mark.parametrize("name", TABLES)
def test_printed_tables_match_both_forms(name):
    g = load(name)
    p, q = g["p"], g["q"]
    assert oracle.q_of(p) == q
    assert list(oracle.skips(p)) == g["skips"]                      # captions of Tables 1-4
    bb = oracle.baseblock_list(p)
    assert list(bb[1:]) == g["baseblock"][1:]                       # root cell ignored
    assert [oracle.baseblock(p, r) for r in range(1, p)] == g["baseblock"][1:]   # Algorithm 2
    recv_a, send_a = oracle.full_table(p)                           # array form
    recv_r, send_r = oracle.build_range(p, 0, p)                    # per-rank form, Alg. 4/5
    recv_u, send_u = oracle.build_range(p, 0, p, special=False)     # two-window rule everywhere
    for recv, send in ((recv_a, send_a), (recv_r, send_r), (recv_u, send_u)):
        assert np.array_equal(recv, g["recv"])
        assert np.array_equal(send, g["send"])


def test_second_p9_schedule_is_valid_but_not_ours():
    """Table 5, right: also a correct schedule, differing in the four bold cells.  The simulation
    accepts it, so the simulation alone does not pin the construction; the printed tables do."""
    left, right = load(TABLES[-1]), load(SECOND_P9)
    p, q = 9, 4
    recv, send = oracle.full_table(p)
    assert np.array_equal(recv, left["recv"]) and np.array_equal(send, left["send"])
    diff = [(int(r), int(k)) for r, k in zip(*np.nonzero(recv != right["recv"]))]
    assert diff == [(8, 1), (8, 2)]                                  # bold receive cells
    diff = [(int(r), int(k)) for r, k in zip(*np.nonzero(send != right["send"]))]
    assert sorted(diff) == [(5, 2), (6, 1)]                          # bold send cells
    for n in (1, 2, 5, q + 3):
        assert bcast_sim.simulate(p, n, oracle.expand(p, n, right["recv"], right["send"])) is None
        assert bcast_sim.simulate(p, n, oracle.expand(p, n, left["recv"], left["send"])) is None


# ---------------------------------------------------------------- Algorithm 1 and Lemma 1
def test_skips_closed_form_and_lemma1():
    for p in list(range(1, 3000)) + [2**20 + 1, 2**30 - 1, 2**31 - 1, 100003, 2**16, 2**16 + 1]:
        s = [int(v) for v in oracle.skips(p)]
        q = oracle.q_of(p)
        assert q == bcast_sim.ceil_log2(p) and len(s) == q + 1
        assert s == bcast_sim.closed_form_skips(p)                  # nested ceil-halving
        assert s[0] == 1 and s[q] == p
        if q >= 1:
            assert s[1] == 2 or p < 2 or q == 1 and s[1] == p
        for k in range(q):
            assert s[k] < s[k + 1]
            assert 2 * s[k] >= s[k + 1]                             # Lemma 1, first claim
            assert sum(s[: k + 1]) >= s[k + 1] - 1                  # Lemma 1, second claim
        assert sum(s[k + 1] - s[k] for k in range(q)) == p - 1      # Lemma 1, third claim
        if p & (p - 1) == 0:
            assert s == [1 << k for k in range(q + 1)]              # powers of two


# ---------------------------------------------------------------- Algorithm 2
def test_baseblock_two_ways_and_structure():
    for p in list(range(2, 700)) + [1000, 1024, 1025, 4097]:
        s = [int(v) for v in oracle.skips(p)]
        bb = oracle.baseblock_list(p)
        assert bb[0] == -1 and oracle.baseblock(p, 0) == -1
        assert [oracle.baseblock(p, r) for r in range(1, p)] == list(bb[1:])
        for k in range(oracle.q_of(p)):
            assert bb[s[k]] == k                                     # "baseblock of skips[k] is k"
            lo, hi = s[k], s[k + 1] - 1                              # homerange repeats [1, ...]
            assert list(bb[lo + 1: hi + 1]) == list(bb[1: hi - lo + 1])
        assert (bb[1:-1] != bb[2:]).all()                            # successive baseblocks differ


def test_baseblock_power_of_two_is_ctz():
    for q in range(1, 13):
        p = 1 << q
        bb = oracle.baseblock_list(p)
        assert all(bb[r] == (r & -r).bit_length() - 1 for r in range(1, p))


# ---------------------------------------------------------------- the range search
def test_rangeblocks_equals_definition():
    rng = np.random.default_rng(1)
    for p in list(range(2, 80)) + [127, 128, 129, 255, 300, 513]:
        bb = oracle.baseblock_list(p)
        pairs = [(a, b) for a in range(-p - 2, p + 2) for b in range(a - 1, a + p + 1)]
        if len(pairs) > 4000:
            pairs = [pairs[i] for i in rng.choice(len(pairs), 4000, replace=False)]
        for a, b in pairs:
            want = 0
            if b - a + 1 >= p:
                want = (1 << oracle.q_of(p)) - 1
            else:
                for x in range(a, b + 1):
                    if x % p:
                        want |= 1 << int(bb[x % p])
            assert oracle.rangeblocks(p, a, b) == want, (p, a, b)
            assert oracle.rangeblocks_scan(p, a, b) == want, (p, a, b)


def test_lemma2_window_counts():
    """Lemma 2: a range of skips[k] processors holds >= k different baseblocks, a range of
    1 + sum_{i<k} skips[i] processors holds >= k+1 (ranges of non-root processors)."""
    for p in list(range(2, 260)) + [511, 512, 513, 1000]:
        s = [int(v) for v in oracle.skips(p)]
        q = oracle.q_of(p)
        bb = oracle.baseblock_list(p).astype(np.int64)
        onehot = np.zeros((p, q), dtype=np.int64)
        onehot[np.arange(1, p), bb[1:]] = 1
        pre = np.vstack([np.zeros((1, q), dtype=np.int64), np.cumsum(onehot, axis=0)])  # pre[x+1]
        for k in range(q + 1):
            for size, least in ((s[k], k), (1 + sum(s[:k]), k + 1)):
                if size > p - 1:
                    continue
                a = np.arange(1, p - size + 1)
                distinct = ((pre[a + size] - pre[a]) > 0).sum(axis=1)
                assert (distinct >= min(least, q)).all(), (p, k, size)


# ---------------------------------------------------------------- schedule invariants
def _check_rows(p, recv, send):
    q = oracle.q_of(p)
    s = [int(v) for v in oracle.skips(p)]
    bb = oracle.baseblock_list(p)
    assert list(send[0]) == list(range(q))                           # root sends block k in round k
    assert sorted(recv[0]) == list(range(-q, 0))                     # root row: all previous-phase
    for r in range(1, p):
        h = max(k for k in range(q) if s[k] <= r)
        row = [int(v) for v in recv[r]]
        assert row[h] == bb[r]                                       # baseblock in the home round
        others = sorted(row[:h] + row[h + 1:])
        assert others == sorted(b - q for b in range(q) if b != bb[r])   # q-1 different others
        allowed = {bb[r] - q}
        for i in range(q):                                           # a sent block was received before
            v = int(send[r][i])
            assert v in allowed or v == bb[r] and i > h, (p, r, i)
            allowed.add(row[i])
    t = (np.arange(p)[:, None] + np.array(s[:q])[None, :]) % p       # Algorithm 5 / Algorithm 9
    assert np.array_equal(send, recv[t, np.arange(q)[None, :]])


def test_row_invariants_small_p():
    for p in list(range(2, 400)) + [1023, 1024, 1025]:
        recv, send = oracle.full_table(p)
        _check_rows(p, recv, send)


def test_power_of_two_closed_form():
    """For p = 2^q the schedule is the classical one: baseblock ctz(r); in a non-home round i the
    window (r-2^(i+1), r-2^i] holds exactly one multiple of 2^i and its block i+ctz(.) is new."""
    for q in range(1, 13):
        p = 1 << q
        recv, _ = oracle.full_table(p)
        for r in range(p):
            for i in range(q):
                if r >> i == 1:
                    want = (r & -r).bit_length() - 1
                else:
                    m = ((r >> i) - 1) % (1 << (q - i))
                    ctz = (m & -m).bit_length() - 1 if m else q - i
                    want = i + ctz - q
                assert recv[r][i] == want, (p, r, i)


def test_two_forms_agree_exhaustive_small_and_sampled_large():
    for p in range(1, 1400):
        if p == 1:
            assert oracle.full_table(1)[0].shape == (1, 0)
            continue
        a, b = oracle.full_table(p), oracle.build_range(p, 0, p)
        assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1]), p
    rng = np.random.default_rng(7)
    for p in (4097, 65535, 65537, 100003, 2**20 + 1):
        ranks = np.unique(np.concatenate([rng.integers(0, p, 300), [0, 1, 2, p - 2, p - 1]]))
        a = oracle.full_table(p)
        b = oracle.build_ranks(p, ranks)
        assert np.array_equal(a[0][ranks], b[0]) and np.array_equal(a[1][ranks], b[1]), p


def test_special_rounds_equal_uniform_rule():
    """Rounds 0 and q-1 as Algorithm 4 writes them (baseblock of r-1; the last missing block)
    give what the two-window rule gives."""
    for p in range(2, 500):
        a = oracle.build_range(p, 0, p, special=True)
        b = oracle.build_range(p, 0, p, special=False)
        assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1]), p


def test_root_cell_reading_is_immaterial():
    """Whether the root adds nothing, block 0 or every block to a range containing it does not
    change any schedule (the printed tables show 0 in four tables and -1 in one)."""
    try:
        for p in list(range(2, 300)) + [1000, 1024, 1025, 4099]:
            oracle.set_root_mode(0)
            base = oracle.build_range(p, 0, p)
            for mode in (1, 2):
                oracle.set_root_mode(mode)
                alt = oracle.build_range(p, 0, p)
                assert np.array_equal(base[0], alt[0]) and np.array_equal(base[1], alt[1]), (p, mode)
    finally:
        oracle.set_root_mode(0)


def test_degenerate_p():
    assert oracle.q_of(1) == 0 and list(oracle.skips(1)) == [1]
    recv, send = oracle.full_table(2)
    assert recv.tolist() == [[-1], [0]] and send.tolist() == [[0], [-1]]
    recv, send = oracle.build_range(2, 0, 2)
    assert recv.tolist() == [[-1], [0]] and send.tolist() == [[0], [-1]]
    recv, send = oracle.full_table(3)
    assert bcast_sim.simulate(3, 4, oracle.expand(3, 4, recv, send)) is None


# ---------------------------------------------------------------- Algorithm 6 + brute force
def test_expansion_closed_form():
    """Round j uses entry k=(j+x) mod q and block sched[k] - x + q*floor((j+x)/q), x the number of
    virtual rounds; below 0 -> -1, above n-1 -> n-1."""
    for p in (2, 3, 9, 20, 33, 64, 100):
        q = oracle.q_of(p)
        s = [int(v) for v in oracle.skips(p)]
        recv, send = oracle.full_table(p)
        for n in (1, 2, 3, q, q + 1, 2 * q + 3, 40):
            tab = oracle.expand(p, n, recv, send)
            x = (q - (n - 1 + q) % q) % q
            assert (x + n - 1 + q) % q == 0
            for r in range(p):
                for j in range(n - 1 + q):
                    i = j + x
                    k = i % q
                    want = []
                    for row in (send, recv):
                        blk = int(row[r][k]) - x + q * (i // q)
                        want.append(-1 if blk < 0 else min(blk, n - 1))
                    want += [(r + s[k]) % p, (r - s[k]) % p]
                    assert tab[r, j].tolist() == want, (p, n, r, j)


def test_broadcast_simulation_every_p_up_to_1024():
    for p in range(2, 1025):
        q = oracle.q_of(p)
        recv, send = oracle.full_table(p)
        for n in (1, 2, 5, q + 3):
            err = bcast_sim.simulate(p, n, oracle.expand(p, n, recv, send))
            assert err is None, (p, n, err)


def test_broadcast_simulation_rerooted():
    rng = np.random.default_rng(3)
    for p in (2, 3, 9, 20, 31, 32, 33, 100, 257, 1000):
        q = oracle.q_of(p)
        recv, send = oracle.full_table(p)
        for n in (1, 5, q + 3):
            tab = oracle.expand(p, n, recv, send)
            for root in {0, 1, p - 1, int(rng.integers(0, p))}:
                err = bcast_sim.simulate(p, n, bcast_sim.reroot(tab, root), root=root)
                assert err is None, (p, n, root, err)


def test_simulation_rejects_planted_mistakes():
    """The simulation is only a pin if it fails for wrong schedules: plant typical mistakes in a
    copy of the oracle's tables (on the CPU) and expect a violation."""
    p, n = 33, 9
    q = oracle.q_of(p)
    recv, send = oracle.full_table(p)
    assert bcast_sim.simulate(p, n, oracle.expand(p, n, recv, send)) is None
    bad = recv.copy(); bad[7, 1], bad[7, 2] = recv[7, 2], recv[7, 1]         # swapped rounds
    assert bcast_sim.simulate(p, n, oracle.expand(p, n, bad, send)) is not None
    bad = send.copy(); bad[5, 0] = send[5, 0] + 1                             # wrong send block
    assert bcast_sim.simulate(p, n, oracle.expand(p, n, recv, bad)) is not None
    bad_r, bad_s = recv.copy(), send.copy()                                   # min instead of max
    bad_r[:, :] = np.where(recv < 0, -q - 1 - recv, recv)
    bad_s[:, :] = np.where(send < 0, -q - 1 - send, send)
    assert bcast_sim.simulate(p, n, oracle.expand(p, n, bad_r, bad_s)) is not None
    tab = oracle.expand(p, n, recv, send)                                     # wrong neighbour
    tab2 = tab.copy(); tab2[:, 3, 2] = (tab[:, 3, 2] + 1) % p
    assert bcast_sim.simulate(p, n, tab2) is not None
    tab2 = tab.copy(); tab2[:, -1, :2] = -1                                   # one round short
    assert bcast_sim.simulate(p, n, tab2) is not None


# ---------------------------------------------------------------- Algorithm 9 index tables
def test_allgather_tables_are_rerooted_broadcast_rounds():
    """Processor r handles buffer j as virtual processor (r-j) mod p of a broadcast rooted at j
    (Section 2.4): its pack / unpack blocks are the send / receive blocks of that virtual
    processor's broadcast rounds (the expansion, pinned above)."""
    for p in (2, 3, 9, 20, 33, 100):
        q = oracle.q_of(p)
        recv, send = oracle.full_table(p)
        for n in (1, 2, 5, q + 3, 40):
            E = oracle.expand(p, n, recv, send)                 # [virtual rank][round][4]
            for r in {0, 1, p // 2, p - 1}:
                pack, unpack = oracle.allgather_rank(p, n, r, recv, send)
                virt = (r - np.arange(p)) % p
                assert np.array_equal(pack, E[virt, :, 0].T), (p, n, r)
                assert np.array_equal(unpack, E[virt, :, 1].T), (p, n, r)


def test_allgather_simulation_and_the_need_for_the_adjustment():
    """All p processors run Algorithm 9 on block numbers (tests/bcast_sim.py): every block of
    every buffer arrives everywhere exactly once in n-1+q rounds.  Leaving out Algorithm 6's
    adjustment of the schedules, as the printed Algorithm 9 does, breaks it whenever there are
    virtual rounds (x != 0)."""
    for p in (2, 3, 5, 9, 16, 20, 33):
        q = oracle.q_of(p)
        recv, send = oracle.full_table(p)
        for n in (1, 2, 5, q + 3):
            tabs = [oracle.allgather_rank(p, n, r, recv, send) for r in range(p)]
            err = bcast_sim.simulate_allgather(p, n, [t[0] for t in tabs], [t[1] for t in tabs])
            assert err is None, (p, n, err)
            x = (q - (n - 1 + q) % q) % q
            raw = [oracle.allgather_rank(p, n, r, recv, send, adjust=False) for r in range(p)]
            err = bcast_sim.simulate_allgather(p, n, [t[0] for t in raw], [t[1] for t in raw])
            assert (err is None) == (x == 0), (p, n, x, err)
    p, n = 9, 5                                               # a planted mistake must be caught
    recv, send = oracle.full_table(p)
    tabs = [list(oracle.allgather_rank(p, n, r, recv, send)) for r in range(p)]
    tabs[4][0][2, 3] = (tabs[4][0][2, 3] + 1) % n
    assert bcast_sim.simulate_allgather(p, n, [t[0] for t in tabs], [t[1] for t in tabs]) is not None


# ---------------------------------------------------------------- Algorithms 7 and 8
def test_regular_allgather_rounds_gather_everything():
    """Algorithm 7 run on block identities: processor r starts with its own block in buffer[0];
    after q rounds buffer[i] holds the block of processor (r+i) mod p for every i."""
    for p in list(range(1, 70)) + [100, 127, 128, 129, 1000]:
        q = oracle.q_of(p)
        tab = oracle.circulant_rounds(p, 0, p, census=False)
        buf = np.full((p, p), -1, dtype=np.int64)
        buf[:, 0] = np.arange(p)
        filled = 1
        for k in range(q):
            to, fr, cnt, off = (tab[:, k, c].astype(np.int64) for c in range(4))
            assert (cnt == cnt[0]).all() and (off == off[0]).all() and off[0] == filled
            assert np.array_equal(fr[to], np.arange(p))          # to/from are mutually consistent
            c, o = int(cnt[0]), int(off[0])
            assert c <= filled                                    # only blocks it already has
            sent = buf[:, :c].copy()                              # everybody sends buffer[0..c-1]
            buf[:, o:o + c] = sent[fr]                            # and stores what arrives at skips[k]
            filled += c
        assert filled == p
        assert np.array_equal(buf, (np.arange(p)[:, None] + np.arange(p)[None, :]) % p), p


def test_census_rounds_sum_every_input_once():
    """Algorithm 8 with + on random integers: every processor ends with the total, i.e. every
    input is counted exactly once (the invariant S = sum of the next skips[k+1]-1 inputs)."""
    rng = np.random.default_rng(8)
    for p in list(range(1, 70)) + [100, 127, 128, 129, 1000]:
        q = oracle.q_of(p)
        s = [int(v) for v in oracle.skips(p)]
        tab = oracle.circulant_rounds(p, 0, p, census=True)
        x = rng.integers(1, 10**6, p)
        S = np.zeros(p, dtype=np.int64)
        for k in range(q):
            to, fr, own = (tab[:, k, c].astype(np.int64) for c in range(3))
            assert np.array_equal(fr[to], np.arange(p))
            assert (own == (0 if 2 * s[k] > s[k + 1] else 1)).all()
            O = np.where(own == 1, x + S, S)
            S = S + O[fr]
            want = sum(np.roll(x, -i) for i in range(1, s[k + 1]))   # x_{r+1} .. x_{r+skips[k+1]-1}
            assert np.array_equal(S, want if s[k + 1] > 1 else np.zeros(p, dtype=np.int64)), (p, k)
        assert np.array_equal(S + x, np.full(p, x.sum())), p


# ---------------------------------------------------------------- property checker
def test_validator_accepts_valid_and_counts_planted_mistakes():
    """oracle.validate counts ranks whose rows break the promised properties.  Valid schedules
    (every small p; both printed p = 9 schedules) give zero; mistakes planted by hand give the
    counts that follow from where they were planted."""
    for p in list(range(2, 300)) + [1000, 1024, 1025]:
        recv, send = oracle.full_table(p)
        assert oracle.validate(p, 0, p, recv, send) == (0, 0, 0), p
        assert oracle.validate(p, p // 3, p, recv[p // 3:], send[p // 3:]) == (0, 0, 0), p
        assert oracle.validate(p, 0, p, recv, None) == (0, 0, 0)
        assert oracle.validate(p, 0, p, None, send) == (0, 0, 0)
    right = load(SECOND_P9)
    assert oracle.validate(9, 0, 9, right["recv"], right["send"]) == (0, 0, 0)
    p = 33                                   # skips 1 2 3 5 9 17 33 (Table 2)
    recv, send = oracle.full_table(p)
    bad = recv.copy(); bad[5, 3] = -1        # rank 5 = skips[3]: home round 3 must hold block 3;
    assert oracle.validate(p, 0, p, bad, send) == (1, 0, 1)      # its sender there is the root
    bad = recv.copy(); bad[10, 0] = bad[10, 1]                   # a block twice in a receive row
    c = oracle.validate(p, 0, p, bad, send)
    assert c[0] == 1 and c[2] == 1           # rank 10's row; rank 9 sends it something else
    bad = send.copy(); bad[0, 3] = 2         # the root must send block 3 in round 3
    assert oracle.validate(p, 0, p, recv, bad) == (0, 1, 1)
    bad = send.copy(); bad[20, 5] = 4        # rank 20 (home round 5, baseblock 2) sends a block
    assert oracle.validate(p, 0, p, recv, bad) == (0, 1, 1)      # of the current phase it lacks
    assert oracle.validate(p, 0, 20, recv[:20], bad[:20]) == (0, 0, 0)   # outside the range
    assert oracle.validate(p, 20, 21, recv[20:21], bad[20:21]) == (0, 1, 0)  # to-processor outside


def test_validator_agrees_with_the_independent_set_based_checker():
    """oracle.validate (C, bit masks) against tests/schedule_props.py (Python sets, written from
    the sentences after Theorem 1, own skips and baseblock list): identical counts on valid tables
    and on several hundred randomly corrupted ones, whole tables and sub-ranges, with both
    tables or one."""
    from tests import schedule_props
    rng = np.random.default_rng(31)
    right = load(SECOND_P9)
    assert schedule_props.count_violations(9, 0, 9, right["recv"], right["send"]) == (0, 0, 0)
    compared = 0
    for p, r0, r1 in ((2, 0, 2), (3, 0, 3), (9, 0, 9), (20, 0, 20), (31, 0, 31), (32, 0, 32),
                      (33, 0, 33), (100, 0, 100), (257, 0, 257), (1000, 0, 1000),
                      (1000, 100, 900), (4097, 4000, 4097), (4097, 0, 300)):
        q = oracle.q_of(p)
        full_recv, full_send = oracle.full_table(p)
        assert schedule_props.count_violations(p, 0, p, full_recv, full_send) == (0, 0, 0), p
        for _ in range(24):
            recv, send = full_recv[r0:r1].copy(), full_send[r0:r1].copy()
            for _ in range(rng.integers(1, 12)):
                tbl = recv if rng.integers(2) else send
                tbl[rng.integers(r1 - r0), rng.integers(q)] = rng.integers(-q - 1, q + 1)
            for a, b in ((recv, send), (recv, None), (None, send)):
                assert oracle.validate(p, r0, r1, a, b) == \
                    schedule_props.count_violations(p, r0, r1, a, b), (p, r0, r1)
                compared += 1
    assert compared > 900


def test_oracle_simulator_agrees_with_the_numpy_simulation():
    """oracle.simulate (C, counts) against tests/bcast_sim.py (numpy, independent skips and round
    semantics): zero counts exactly when the numpy simulation accepts, on valid and on corrupted
    tables; hand-planted mistakes give the counts that follow from them."""
    rng = np.random.default_rng(23)
    for p in (2, 3, 9, 20, 31, 32, 33, 100, 257):
        q = oracle.q_of(p)
        recv, send = oracle.full_table(p)
        for n in (1, 2, 5, q + 3, 64):
            c = oracle.simulate(p, n, recv, send)
            assert c[:4] == (0, 0, 0, 0) and 1 <= c[4] < p, (p, n, c)
            assert bcast_sim.simulate(p, n, oracle.expand(p, n, recv, send)) is None
        for _ in range(12):
            br, bs = recv.copy(), send.copy()
            tbl = br if rng.integers(2) else bs
            j, k = rng.integers(p), rng.integers(q)
            new = rng.integers(-q, q)
            if new == tbl[j, k]:
                continue
            tbl[j, k] = new
            n = int(rng.choice([2, 5, q + 3]))
            c = oracle.simulate(p, n, br, bs)
            ok_numpy = bcast_sim.simulate(p, n, oracle.expand(p, n, br, bs)) is None
            assert (c[:4] == (0, 0, 0, 0) and c[4] < p) == ok_numpy, (p, n, j, k, new, c)
    right = load(SECOND_P9)
    assert oracle.simulate(9, 5, right["recv"], right["send"])[:4] == (0, 0, 0, 0)
    # p = 9, n = 5 (q = 4, eight rounds, no virtual round): in round 0 the root sends block 0 to
    # rank 1; a table in which rank 1 expects block 1 there is unpaired in that round, and rank 1
    # then holds a block nobody sent while block 0 is missing when it has to forward it
    recv, send = oracle.full_table(9)
    bad = recv.copy(); bad[1, 0] = 1
    c = oracle.simulate(9, 5, bad, send)
    assert c[1] == 1 and c[0] >= 1, c


# ---------------------------------------------------------------- checksum helper
def test_checksum_definition_and_additivity():
    rng = np.random.default_rng(5)
    buf = rng.integers(-30, 30, 1003).astype(np.int8)
    m64, m32 = (1 << 64) - 1, (1 << 32) - 1

    def fmix32(h):
        h ^= h >> 16
        h = (h * 0x85EBCA6B) & m32
        h ^= h >> 13
        h = (h * 0xC2B2AE35) & m32
        return h ^ (h >> 16)

    # MurmurHash3 x86_32 of the empty key with seed 1 is fmix32(1) = 0x514E28B7 (reference vector)
    assert fmix32(1) == 0x514E28B7

    def weight(g):
        return fmix32((g & m32) ^ ((0x9E3779B9 * (g >> 32)) & m32)) | 1

    def by_words(b, first):
        assert first % 4 == 0
        pad = np.concatenate([b.view(np.uint8), np.zeros((-len(b)) % 4, dtype=np.uint8)])
        words = pad.view("<u4")
        return sum(int(w) * weight(first // 4 + i) for i, w in enumerate(words)) & m64

    want = by_words(buf, 16)
    assert oracle.checksum(buf, 16) == want
    assert (oracle.checksum(buf[:400], 16) + oracle.checksum(buf[400:], 416)) & m64 == want
    big = (1 << 34) + 8                                   # word index above 2^32
    assert oracle.checksum(buf, big) == by_words(buf, big)
    swapped = buf.copy(); swapped[[3, 700]] = swapped[[700, 3]]
    assert buf[3] != buf[700] and oracle.checksum(swapped, 16) != want


# ---------------------------------------------------------------- independent tripwire digests
def _witness_lines():
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "witness_digests.txt")
    with open(path) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def test_table_digests_of_an_independent_implementation():
    """Digests and one printed row computed by an independent implementation of the same reading
    (see the fixture's header): not the paper's, so a tripwire beside the printed tables."""
    import hashlib
    for f in _witness_lines():
        if f[0] == "row":
            p, r = int(f[1]), int(f[2])
            want = [int(v) for v in f[4].split(",")]
            assert list(oracle.skips(p)) == [1, 2, 4, 7, 13, 25, 49, 98, 196, 391, 782, 1563, 3126,
                                              6251, 12501, 25001, 50002, 100003]
            got = oracle.recvsched(p, r) if f[3] == "recv" else oracle.sendsched(p, r)
            assert list(got) == want, f
            continue
        p = int(f[0])
        recv, send = oracle.full_table(p)
        assert hashlib.sha256(recv.astype(np.int8).tobytes()).hexdigest()[:16] == f[1], p
        assert hashlib.sha256(send.astype(np.int8).tobytes()).hexdigest()[:16] == f[2], p
        assert int(recv.astype(np.int64).sum()) == int(f[3]) == int(send.astype(np.int64).sum()), p
