"""The skip-code construction that the fast CUDA kernels run, restated on the CPU
(tests/skipcode_mirror.c), must give the oracle's rows: the paper's greedy construction
(Algorithm 4's two windows and max(U \\ B), the range search that Algorithm 3 stands for) and
the construction on skip codes are the same function.  Also keeps the committed table of model
operation counts, which the benchmark reads, honest."""
import json

import numpy as np
import pytest

import oracle
from paper_2205_10072_b200 import workloads
from tests import skipcode_mirror as mirror


@pytest.fixture(autouse=True)
def _gpu_mode():
    mirror.set_table_mode(0)
    yield
    mirror.set_table_mode(0)


@pytest.mark.parametrize("mode", [0, 1, 2])
def test_mirror_equals_oracle_for_every_small_p(mode):
    """Every rank of every p < 700, with the short windows taken from exact block sets (as the
    kernels do for p >= 64), never, and for every p."""
    mirror.set_table_mode(mode)
    seen = {"rounds_step2": 0, "rounds_rest": 0, "rounds_second": 0, "rounds_table": 0}
    for p in range(2, 700):
        recv, send, cnt = mirror.full(p)
        want_recv, want_send = oracle.full_table(p)
        assert np.array_equal(recv, want_recv), p
        assert np.array_equal(send, want_send), p
        for k in seen:
            seen[k] += cnt[k]
    # the rare paths were really taken
    if mode == 1:
        assert seen["rounds_table"] == 0
        assert seen["rounds_step2"] > 0 and seen["rounds_rest"] > 0 and seen["rounds_second"] > 0
    else:
        assert seen["rounds_table"] > 0


@pytest.mark.parametrize("p", [workloads.P_EXPAND, workloads.P_SINGLE])
def test_mirror_equals_oracle_on_the_benchmark_tables(p):
    recv, send, _ = mirror.full(p)
    want_recv, want_send = oracle.full_table(p)
    assert np.array_equal(recv, want_recv)
    assert np.array_equal(send, want_send)


@pytest.mark.parametrize("p", [workloads.P_LARGE, 2**31 - 1, 2**29 + 12345])
def test_mirror_equals_oracle_on_sampled_ranks_of_large_p(p):
    q = oracle.q_of(p)
    sk = oracle.skips(p).tolist()
    ranks = workloads.spot_ranks(p, 3000)
    for k in range(q + 1):                          # around every skip, the root and the end
        ranks += [(sk[k] + d) % p for d in (-2, -1, 0, 1, 2)]
    ranks += [0, 1, 2, p - 2, p - 1]
    for mode in (0, 1):
        mirror.set_table_mode(mode)
        recv, send, _ = mirror.rows(p, ranks)
        want_recv, want_send = oracle.build_ranks(p, ranks)
        assert np.array_equal(recv, want_recv), (p, mode)
        assert np.array_equal(send, want_send), (p, mode)


def test_committed_model_table_is_what_the_mirror_counts():
    """tests/skipcode_model_ops.json is written by `python -m tests.skipcode_mirror --write`;
    the q = 17 entry is recomputed here (the others take longer and follow the same code)."""
    table = mirror.load_table()
    assert {"q17_p100003", "q21_p1048577", "q30_p1073741823", "batch_4096p",
            "small_sweep_2_1024"} <= set(table)
    _, _, cnt = mirror.full(workloads.P_EXPAND, want_send=False)
    fresh = mirror.per_rank(cnt)
    assert table["q17_p100003"]["recv_int_ops_per_rank"] == pytest.approx(fresh["recv_int_ops_per_rank"], rel=1e-12)
    for entry in table.values():
        assert 50 < entry["recv_int_ops_per_rank"] < 1000
        json.dumps(entry)


def test_block_codes_equal_the_plain_scan():
    """One greedy scan per block of 32 consecutive ranks (plus the table of the low levels) gives
    the code of every rank that its own scan gives; the second splitting level that would send
    a block to the plain scan does not occur."""
    import numpy as np
    from tests import skipcode_mirror as skm
    split = 0
    for p in list(range(1, 400)) + [1000, 4097, 65535, 65537, 100003, 300007, 2**20 + 1]:
        got, st = skm.codes_blocks(p, 0, p)
        assert np.array_equal(got, skm.codes_plain(p, 0, p)), p
        assert st["plain"] == 0, (p, st)
        split += st["split"]
    assert split > 1000                      # the splitting levels are exercised
    rng = np.random.default_rng(11)
    for p in (2**24 - 3, 2**29 + 12345, 2**30 - 1, 2**30 - 12345, 2**31 - 1):
        starts = [0, (p - 5000) // 32 * 32] + [int(v) // 32 * 32 for v in rng.integers(0, p - 70000, 12)]
        q = skm.skm_q(p)
        v = p
        for _ in range(q - 8):               # just below the larger skips, where blocks split
            v = (v + 1) // 2
            starts.append(max(0, v - 3000) // 32 * 32)
        for g in starts:
            end = min(p, g + 65536)
            got, st = skm.codes_blocks(p, g, end)
            assert np.array_equal(got, skm.codes_plain(p, g, end)), (p, g)
            assert st["plain"] == 0, (p, g, st)


def test_small_p_run_table_construction_equals_the_oracle():
    """The construction of the batch kernel for p <= 1024 (baseblock bits of all ranks, runs of
    2^l ranks, every window looked up as an exact set) gives the oracle's tables for every such p."""
    import numpy as np
    import oracle
    from tests import skipcode_mirror as skm
    for p in range(2, 1025):
        recv, send, _ = skm.small(p)
        want_r, want_s = oracle.full_table(p)
        assert np.array_equal(recv, want_r), p
        assert np.array_equal(send, want_s), p
