"""Parity of the CUDA library (through its C ABI) with the CPU oracle, element by element.
All schedule entries are integers: the bar is bit-exactness."""
import numpy as np
import pytest
import torch

import oracle
from paper_2205_10072_b200 import workloads
from tests import bcast_sim

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bcs():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2205_10072_b200 as lib
    lib.lib()                      # raises if the CUDA library has not been built
    torch.cuda.set_device(0)
    return lib


GUARD = 256


def _guarded(nbytes, fill=0x5A):
    """int8 CUDA buffer of nbytes framed by guard bytes (start stays 16-byte aligned)."""
    raw = torch.full((nbytes + 2 * GUARD,), fill, dtype=torch.int8, device="cuda")
    return raw, raw[GUARD:GUARD + nbytes]


def _guards_intact(raw, nbytes, fill=0x5A):
    return bool((raw[:GUARD] == fill).all()) and bool((raw[GUARD + nbytes:] == fill).all())


def _build(bcs, p, r0, r1, want_recv=True, want_send=True, fast=True):
    """fast=True: with a workspace (skip-code construction); False: self-contained construction."""
    q = bcs.bcs_q(p)
    nb = (r1 - r0) * q
    raw_r, recv = _guarded(nb) if want_recv else (None, None)
    raw_s, send = _guarded(nb) if want_send else (None, None)
    ws = raw_w = None
    if fast:
        need = bcs.bcs_build_workspace_bytes(p, r0, r1)
        raw_w, ws = _guarded(need)
    bcs.bcs_build(p, r0, r1, recv, send, ws)
    torch.cuda.synchronize()
    assert bcs.bcs_wait_expired() == 0      # no CTA gave up waiting for its copies
    if raw_w is not None:
        assert _guards_intact(raw_w, ws.numel())
    out = []
    for raw, t in ((raw_r, recv), (raw_s, send)):
        if t is None:
            out.append(None)
        else:
            assert _guards_intact(raw, nb)
            out.append(t.cpu().numpy().reshape(r1 - r0, q))
    return out


# ---------------------------------------------------------------- printed tables, small p
def test_printed_tables_through_the_gpu(bcs):
    from tests.golden_tables import TABLES, load
    for name in TABLES:
        g = load(name)
        recv, send = _build(bcs, g["p"], 0, g["p"])
        assert np.array_equal(recv, g["recv"]) and np.array_equal(send, g["send"]), name


@pytest.mark.parametrize("fast", [True, False])
def test_every_p_up_to_1024_single_calls(bcs, fast):
    for p in workloads.small_sweep():
        want_r, want_s = oracle.full_table(p)
        recv, send = _build(bcs, p, 0, p, fast=fast)
        assert np.array_equal(recv, want_r), p
        assert np.array_equal(send, want_s), p


def _batch_ws(bcs, plan, fast):
    if not fast:
        return None, None
    return _guarded(plan.workspace_bytes())


@pytest.mark.parametrize("fast", [True, False])
def test_every_p_up_to_1024_batched_and_simulated(bcs, fast):
    plist = workloads.small_sweep()
    plan = bcs.bcs_batch_plan(plist)
    assert plan.total_ranks == 524799 and plan.total_entries == 5072726
    dev = plan.to("cuda")
    raw_r, recv = _guarded(plan.total_entries)
    raw_s, send = _guarded(plan.total_entries)
    raw_w, ws = _batch_ws(bcs, plan, fast)
    bcs.bcs_build_batch(dev, recv, send, ws)
    torch.cuda.synchronize()
    assert raw_w is None or _guards_intact(raw_w, ws.numel())
    assert _guards_intact(raw_r, plan.total_entries) and _guards_intact(raw_s, plan.total_entries)
    recv, send = recv.cpu().numpy(), send.cpu().numpy()
    eo = plan.entry_off.tolist()
    for j, p in enumerate(plist):
        q = oracle.q_of(p)
        want_r, want_s = oracle.full_table(p)
        got_r = recv[eo[j]:eo[j + 1]].reshape(p, q)
        got_s = send[eo[j]:eo[j + 1]].reshape(p, q)
        assert np.array_equal(got_r, want_r), p
        assert np.array_equal(got_s, want_s), p
        if p % 7 == 0 or p < 70:            # broadcast simulation on the GPU's own output
            for n in (1, 2, 5, q + 3):
                tab = torch.empty((p, n - 1 + q, 4), dtype=torch.int32, device="cuda")
                bcs.bcs_expand(p, n, 0, p, torch.from_numpy(got_r.copy()).cuda(),
                               torch.from_numpy(got_s.copy()).cuda(), tab)
                assert bcast_sim.simulate(p, n, tab.cpu().numpy()) is None, (p, n)


@pytest.mark.parametrize("fast", [True, False])
def test_batch_with_trivial_and_duplicate_p(bcs, fast):
    plist = [1, 2, 1, 300, 300, 1, 17, 4096, 1]
    plan = bcs.bcs_batch_plan(plist)
    dev = plan.to("cuda")
    raw_r, recv = _guarded(plan.total_entries)
    raw_s, send = _guarded(plan.total_entries)
    raw_w, ws = _batch_ws(bcs, plan, fast)
    bcs.bcs_build_batch(dev, recv, send, ws)
    torch.cuda.synchronize()
    assert raw_w is None or _guards_intact(raw_w, ws.numel())
    assert _guards_intact(raw_r, plan.total_entries) and _guards_intact(raw_s, plan.total_entries)
    eo = plan.entry_off.tolist()
    for j, p in enumerate(plist):
        if p == 1:
            assert eo[j] == eo[j + 1]
            continue
        want_r, want_s = oracle.full_table(p)
        assert np.array_equal(recv[eo[j]:eo[j + 1]].cpu().numpy().reshape(p, -1), want_r)
        assert np.array_equal(send[eo[j]:eo[j + 1]].cpu().numpy().reshape(p, -1), want_s)
    # receive table alone
    raw_r, recv = _guarded(plan.total_entries)
    bcs.bcs_build_batch(dev, recv, None, ws)
    torch.cuda.synchronize()
    assert np.array_equal(recv[eo[3]:eo[4]].cpu().numpy().reshape(300, -1), oracle.full_table(300)[0])


def test_batch_of_large_and_tiny_p_mixed(bcs):
    """A list whose p average more than 8192 ranks (the batch takes the codes kernel that scans
    blocks of 32 flattened ranks at once) with p = 1, tiny p and p next to multiples of 8192 in
    between: blocks that cross from one p to the next, whole p inside one block, CTAs that touch
    three and more p, a last block cut off by the end of the list."""
    plist = [70001, 1, 2, 3, 65536, 1, 8191, 8193, 31, 32, 33, 16384, 5, 100003, 1, 7, 8192, 40961,
             64, 63, 65, 262147, 1000, 24576, 9, 131071]
    assert sum(plist) // len(plist) >= 8192
    plan = bcs.bcs_batch_plan(plist)
    dev = plan.to("cuda")
    raw_r, recv = _guarded(plan.total_entries)
    raw_s, send = _guarded(plan.total_entries)
    raw_w, ws = _batch_ws(bcs, plan, True)
    bcs.bcs_build_batch(dev, recv, send, ws)
    torch.cuda.synchronize()
    assert _guards_intact(raw_w, ws.numel())
    assert _guards_intact(raw_r, plan.total_entries) and _guards_intact(raw_s, plan.total_entries)
    assert bcs.bcs_wait_expired() == 0
    eo = plan.entry_off.tolist()
    for j, p in enumerate(plist):
        if p == 1:
            assert eo[j] == eo[j + 1]
            continue
        want_r, want_s = oracle.full_table(p)
        assert np.array_equal(recv[eo[j]:eo[j + 1]].cpu().numpy().reshape(p, -1), want_r), (j, p)
        assert np.array_equal(send[eo[j]:eo[j + 1]].cpu().numpy().reshape(p, -1), want_s), (j, p)


def test_batch_output_is_complete_for_the_next_operation_on_the_stream(bcs):
    """The kernels of a batch are launched as dependents of one another and the last one (the
    CTAs of the small p) does not wait for the tiled kernels of the large p before it starts.
    Whatever follows on the stream must still see both tables complete: a copy enqueued right
    after the call, without a synchronisation in between, is compared with the oracle."""
    plist = [5, 2**20 + 1, 300, 1000, 77]
    plan = bcs.bcs_batch_plan(plist)
    dev = plan.to("cuda")
    want = {p: oracle.full_table(p) for p in set(plist)}
    ws = torch.empty(plan.workspace_bytes(), dtype=torch.int8, device="cuda")
    side = torch.cuda.Stream()
    for stream in (None, side):
        for _ in range(3):
            recv = torch.full((plan.total_entries,), 99, dtype=torch.int8, device="cuda")
            send = torch.full((plan.total_entries,), 99, dtype=torch.int8, device="cuda")
            torch.cuda.synchronize()
            with torch.cuda.stream(stream if stream is not None else torch.cuda.current_stream()):
                bcs.bcs_build_batch(dev, recv, send, ws)
                snap_r, snap_s = recv.clone(), send.clone()      # same stream, no synchronisation
            torch.cuda.synchronize()
            eo = plan.entry_off.tolist()
            for j, p in enumerate(plist):
                q = oracle.q_of(p)
                assert np.array_equal(snap_r[eo[j]:eo[j + 1]].cpu().numpy().reshape(p, q), want[p][0]), (j, p)
                assert np.array_equal(snap_s[eo[j]:eo[j + 1]].cpu().numpy().reshape(p, q), want[p][1]), (j, p)


# ---------------------------------------------------------------- ranges, tails, degenerate
@pytest.mark.parametrize("fast", [True, False])
def test_sub_ranges_ragged_tails_and_single_outputs(bcs, fast):
    p = 100003
    q = oracle.q_of(p)
    want_r, want_s = oracle.full_table(p)
    for r0, r1 in ((0, 1), (0, 255), (0, 257), (1, 258), (777, 1300), (p - 300, p), (p - 1, p),
                   (50000, 50000 + 16 * 3 + 5), (99000, 100003),
                   # several 512-rank tiles of the four-ranks-per-thread kernel, odd starts and ends
                   (12345, 14002), (3, 70003), (25001 - 700, 25001 + 700)):
        recv, send = _build(bcs, p, r0, r1, fast=fast)
        assert np.array_equal(recv, want_r[r0:r1]), (r0, r1)
        assert np.array_equal(send, want_s[r0:r1]), (r0, r1)      # partly looked up, partly recomputed
    recv, _ = _build(bcs, p, 123, 999, want_send=False, fast=fast)
    assert np.array_equal(recv, want_r[123:999])
    _, send = _build(bcs, p, 123, 999, want_recv=False, fast=fast)
    assert np.array_equal(send, want_s[123:999])
    assert q == 17


def test_seeded_p_sweep_full_tables_sub_ranges_and_one_batch(bcs):
    """About 170 values of p between 64 and 300 000 -- the neighbours of the powers of two, values
    whose skips contain 33 (six instead of five rounds read from the run table), and 150 seeded
    log-uniform draws: the full tables, one seeded sub-range each, and all of them in one batch."""
    rng = np.random.default_rng(20240)
    edge = [64, 65, 127, 128, 129, 511, 512, 513, 1023, 1025, 2047, 2049, 4095, 4097, 33 * 64, 33 * 64 - 1,
            33 * 128, 33 * 2048, 33 * 2048 - 5, 65535, 65536, 65537, 131071, 131073, 262143, 262145]
    draws = np.exp(rng.uniform(np.log(64), np.log(300000), 150)).astype(np.int64)
    ps = sorted(set(edge + [int(x) for x in draws]))
    tables = {}
    for p in ps:
        want_r, want_s = tables[p] = oracle.full_table(p)
        recv, send = _build(bcs, p, 0, p)
        assert np.array_equal(recv, want_r) and np.array_equal(send, want_s), p
        a = int(rng.integers(0, p - 1))
        b = int(rng.integers(a + 1, p + 1))
        recv, send = _build(bcs, p, a, b)
        assert np.array_equal(recv, want_r[a:b]) and np.array_equal(send, want_s[a:b]), (p, a, b)
    plan = bcs.bcs_batch_plan(ps)
    dplan = plan.to("cuda")
    raw_r, recv = _guarded(plan.total_entries)
    raw_s, send = _guarded(plan.total_entries)
    raw_w, ws = _guarded(plan.workspace_bytes())
    bcs.bcs_build_batch(dplan, recv, send, ws)
    torch.cuda.synchronize()
    assert bcs.bcs_wait_expired() == 0
    assert _guards_intact(raw_r, plan.total_entries) and _guards_intact(raw_s, plan.total_entries)
    assert _guards_intact(raw_w, ws.numel())
    got_r, got_s = recv.cpu().numpy(), send.cpu().numpy()
    eo = plan.entry_off.tolist()
    for j, p in enumerate(ps):
        want_r, want_s = tables[p]
        assert np.array_equal(got_r[eo[j]:eo[j + 1]].reshape(p, -1), want_r), p
        assert np.array_equal(got_s[eo[j]:eo[j + 1]].reshape(p, -1), want_s), p


def test_receive_kernel_instantiations(bcs):
    """The quad receive kernel has four instantiations picked per launch: window bounds loaded as
    16-byte words where a p's skips are multiples of 4 (p just below a power of two), rows stored
    word by word where q is a multiple of 4.  Values of p that take each combination, all ranks
    and a sub-range that starts off a multiple of 4, with and without rows / round-major copy."""
    for p in (4095, 4097, 65535, 65537, 1048575, 1000003, 262143, 300007, 16383, 16385):
        q = oracle.q_of(p)
        want_r, want_s = oracle.full_table(p)
        recv, send = _build(bcs, p, 0, p)
        assert np.array_equal(recv, want_r) and np.array_equal(send, want_s), p
        (recv,) = _build(bcs, p, 0, p, want_send=False)[:1]
        assert np.array_equal(recv, want_r), p
        r0, r1 = 1001, p - 77                                   # rows of the range only, start not on a quad
        recv, send = _build(bcs, p, r0, r1)
        assert np.array_equal(recv, want_r[r0:r1]) and np.array_equal(send, want_s[r0:r1]), p
        raw_w, ws = _guarded(bcs.bcs_prepare_workspace_bytes(p))
        bcs.bcs_prepare(p, ws)                                  # round-major copy only
        raw_s, out = _guarded(p * q)
        bcs.bcs_build_prepared(p, 0, p, None, out, ws)
        torch.cuda.synchronize()
        assert _guards_intact(raw_w, ws.numel()) and _guards_intact(raw_s, p * q)
        assert np.array_equal(out.cpu().numpy().reshape(p, q), want_s), p


def test_prepare_then_build_ranges(bcs):
    """bcs_prepare once, then receive and send rows of arbitrary ranges by bcs_build_prepared."""
    for p in (2, 3, 33, 63, 64, 1000, 4097, 100003):
        q = oracle.q_of(p)
        want_r, want_s = oracle.full_table(p)
        raw_w, ws = _guarded(bcs.bcs_prepare_workspace_bytes(p))
        bcs.bcs_prepare(p, ws)
        ranges = [(0, p), (0, 1), (p - 1, p), (p // 3, p // 3 + min(p - p // 3, 700)),
                  (max(0, p - 300), p), (1, min(p, 258))]
        for r0, r1 in ranges:
            nb = (r1 - r0) * q
            raw_r, recv = _guarded(nb)
            raw_s, send = _guarded(nb)
            bcs.bcs_build_prepared(p, r0, r1, recv, send, ws)
            torch.cuda.synchronize()
            assert _guards_intact(raw_r, nb) and _guards_intact(raw_s, nb) and _guards_intact(raw_w, ws.numel())
            assert np.array_equal(recv.cpu().numpy().reshape(-1, q), want_r[r0:r1]), (p, r0, r1)
            assert np.array_equal(send.cpu().numpy().reshape(-1, q), want_s[r0:r1]), (p, r0, r1)
        raw_s, send = _guarded(p * q)
        bcs.bcs_build_prepared(p, 0, p, None, send, ws)          # one table only
        torch.cuda.synchronize()
        assert np.array_equal(send.cpu().numpy().reshape(p, q), want_s)
    L = bcs.lib()
    small = torch.zeros(64, dtype=torch.int8, device="cuda")
    assert L.bcs_prepare(1000, small.data_ptr(), 64, None) == 1                # too small
    assert L.bcs_build_prepared(1000, 0, 10, small.data_ptr(), None, small.data_ptr(), 64, None) == 1
    assert L.bcs_prepare(1, None, 0, None) == 0 and bcs.bcs_prepare_workspace_bytes(1) == 0
    assert bcs.bcs_prepare_workspace_bytes(20) == 256 + 5 * 32


def test_prepare_in_two_steps_chunk_by_chunk(bcs):
    """bcs_prepare_codes, then bcs_prepare_rows chunk by chunk (in a shuffled order, chunk
    boundaries at multiples of 16 that are not multiples of the kernels' tiles), each chunk's
    receive rows taken straight from the construction; then the send rows of every chunk by
    bcs_build_prepared, and the receive rows once more by transposition: all equal the oracle's."""
    rng = np.random.default_rng(5)
    for p, step in ((33, 16), (63, 32), (64, 16), (1000, 304), (4097, 1008), (100003, 30000),
                    (workloads.P_SINGLE, 333328)):
        q = oracle.q_of(p)
        want_r, want_s = oracle.full_table(p)
        raw_w, ws = _guarded(bcs.bcs_prepare_workspace_bytes(p))
        bcs.bcs_prepare_codes(p, ws)
        chunks = [(a, min(p, a + step)) for a in range(0, p, step)]
        for c in rng.permutation(len(chunks)):
            r0, r1 = chunks[c]
            raw_r, recv = _guarded((r1 - r0) * q)
            if c % 3 == 2:
                bcs.bcs_prepare_rows(p, r0, r1, None, ws)        # round-major copy only
            else:
                bcs.bcs_prepare_rows(p, r0, r1, recv, ws)
                torch.cuda.synchronize()
                assert _guards_intact(raw_r, (r1 - r0) * q)
                assert np.array_equal(recv.cpu().numpy().reshape(-1, q), want_r[r0:r1]), (p, r0, r1)
        for r0, r1 in chunks:
            raw_s, send = _guarded((r1 - r0) * q)
            raw_r, recv = _guarded((r1 - r0) * q)
            bcs.bcs_build_prepared(p, r0, r1, recv, send, ws)
            torch.cuda.synchronize()
            assert _guards_intact(raw_s, (r1 - r0) * q) and _guards_intact(raw_w, ws.numel())
            assert np.array_equal(send.cpu().numpy().reshape(-1, q), want_s[r0:r1]), (p, r0, r1)
            assert np.array_equal(recv.cpu().numpy().reshape(-1, q), want_r[r0:r1]), (p, r0, r1)
    assert bcs.bcs_wait_expired() == 0
    L = bcs.lib()
    small = torch.zeros(4096, dtype=torch.int8, device="cuda")
    assert L.bcs_prepare_rows(1000, 8, 100, small.data_ptr(), ws.data_ptr(), ws.numel(), None) == 3   # r_begin % 16
    assert L.bcs_prepare_rows(1000, 16, 1001, small.data_ptr(), ws.data_ptr(), ws.numel(), None) == 2
    assert L.bcs_prepare_rows(1000, 16, 100, small.data_ptr(), small.data_ptr(), 64, None) == 1        # too small
    assert L.bcs_prepare_codes(1000, small.data_ptr(), 64, None) == 1
    assert L.bcs_prepare_codes(1, None, 0, None) == 0


def test_rooted_builds_are_the_renumbered_schedule(bcs):
    """Section 2: a broadcast from root rho uses the rank-0-rooted rows of virtual rank
    (r - rho) mod p.  Full and partial ranges, runs that pass virtual rank p-1 on and off a
    16-byte boundary, with and without a workspace; and the rooted tables drive a correct
    n-block broadcast from rho in the brute-force simulation."""
    L = bcs.lib()
    for p, roots in ((2, (0, 1)), (20, (0, 7, 19)), (33, (5, 32)), (64, (63,)), (1000, (1, 16, 999)),
                     (4097, (4000,)), (100003, (54607,))):
        q = oracle.q_of(p)
        want_r, want_s = oracle.full_table(p)
        for root in roots:
            virt = (np.arange(p) - root) % p
            for r0, r1 in ((0, p), (root, min(p, root + 1)), (0, min(p, root + 3)),
                           (max(0, root - 5), min(p, root + 300)), (p // 2, p)):
                if r0 >= r1:
                    continue
                nb = (r1 - r0) * q
                for fast in (True, False):
                    raw_r, recv = _guarded(nb)
                    raw_s, send = _guarded(nb)
                    need = bcs.bcs_build_rooted_workspace_bytes(p, root, r0, r1)
                    raw_w, ws = _guarded(need) if fast else (None, None)
                    code = L.bcs_build_rooted(p, root, r0, r1, recv.data_ptr(), send.data_ptr(),
                                              ws.data_ptr() if fast else None, need if fast else 0, None)
                    torch.cuda.synchronize()
                    v0 = (r0 - root) % p
                    len_a = min(r1 - r0, p - v0)
                    staged = (r1 - r0) > len_a and (len_a * q) % 16 != 0
                    if not fast and staged:
                        assert code == 1, (p, root, r0, r1)      # needs the workspace for the copy
                        continue
                    assert code == 0, (p, root, r0, r1, fast)
                    assert _guards_intact(raw_r, nb) and _guards_intact(raw_s, nb)
                    if fast:
                        assert _guards_intact(raw_w, need)
                    assert np.array_equal(recv.cpu().numpy().reshape(-1, q), want_r[virt[r0:r1]]), (p, root, r0, r1)
                    assert np.array_equal(send.cpu().numpy().reshape(-1, q), want_s[virt[r0:r1]]), (p, root, r0, r1)
    # the rooted tables, expanded, broadcast correctly from the root
    p, root, n = 1000, 321, 7
    q = oracle.q_of(p)
    recv = torch.empty(p * q, dtype=torch.int8, device="cuda")
    send = torch.empty(p * q, dtype=torch.int8, device="cuda")
    ws = torch.empty(bcs.bcs_build_rooted_workspace_bytes(p, root, 0, p), dtype=torch.int8, device="cuda")
    bcs.bcs_build_rooted(p, root, 0, p, recv, send, ws)
    table = torch.empty((p, n - 1 + q, 4), dtype=torch.int32, device="cuda")
    bcs.bcs_expand(p, n, 0, p, recv, send, table)
    assert bcast_sim.simulate(p, n, table.cpu().numpy(), root=root) is None
    assert L.bcs_build_rooted(20, 20, 0, 20, recv.data_ptr(), None, None, 0, None) == 2   # root out of range
    assert bcs.bcs_build_rooted_workspace_bytes(20, 20, 0, 20) == 0
    assert bcs.bcs_wait_expired() == 0


def test_degenerate_sizes_and_errors(bcs):
    L = bcs.lib()
    buf = torch.zeros(64, dtype=torch.int8, device="cuda")
    bcs.bcs_build(1, 0, 1, buf, buf, buf)               # q == 0
    bcs.bcs_build(20, 7, 7, buf, buf, buf)              # empty range
    torch.cuda.synchronize()
    assert int(buf.abs().sum()) == 0
    assert bcs.bcs_build_workspace_bytes(1, 0, 1) == 0 and bcs.bcs_build_workspace_bytes(20, 7, 7) == 0
    assert bcs.bcs_build_workspace_bytes(20, 0, 20) == 256 + 5 * 32
    for fast in (True, False):
        recv, send = _build(bcs, 2, 0, 2, fast=fast)
        assert recv.tolist() == [[-1], [0]] and send.tolist() == [[0], [-1]]
        recv, send = _build(bcs, 3, 0, 3, fast=fast)
        want = oracle.full_table(3)
        assert np.array_equal(recv, want[0]) and np.array_equal(send, want[1])
    small = torch.zeros(64, dtype=torch.int8, device="cuda")         # too small a workspace:
    out = torch.zeros(100003 * 17, dtype=torch.int8, device="cuda")  # the slow path must run
    bcs.bcs_build(100003, 0, 100003, out, None, small)
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy().reshape(100003, 17), oracle.full_table(100003)[0])
    assert int(small.abs().sum()) == 0
    assert L.bcs_build(20, 0, 20, buf.data_ptr() + 1, None, None, 0, None) == 3
    assert L.bcs_build(20, 0, 20, buf.data_ptr(), None, buf.data_ptr() + 4, 64, None) == 3
    assert L.bcs_build(20, 0, 21, buf.data_ptr(), None, None, 0, None) == 2
    assert L.bcs_build(0, 0, 0, buf.data_ptr(), None, None, 0, None) == 2
    torch.cuda.synchronize()
    assert int(buf.abs().sum()) == 0                    # an error writes nothing


def test_p_at_the_upper_limit(bcs):
    """p = 2^31 - 1 (q = 31): rank arithmetic near 2^32; a few ranges vs the per-rank oracle.
    Both constructions."""
    p = 2**31 - 1
    for r0, r1 in ((0, 300), (2**30 - 100, 2**30 + 200), (p - 300, p)):
        want_r, want_s = oracle.build_range(p, r0, r1)
        recv, send = _build(bcs, p, r0, r1, fast=False)
        assert np.array_equal(recv, want_r), (r0, r1)
        assert np.array_equal(send, want_s), (r0, r1)
    # the skip-code construction at the same p: 8.6 GB of codes in the workspace
    for r0, r1 in ((0, 300), (2**30 - 100, 2**30 + 200), (p - 300, p)):
        want_r, want_s = oracle.build_range(p, r0, r1)
        q = 31
        recv = torch.empty((r1 - r0) * q, dtype=torch.int8, device="cuda")
        send = torch.empty((r1 - r0) * q, dtype=torch.int8, device="cuda")
        ws = torch.empty(bcs.bcs_build_workspace_bytes(p, r0, r1), dtype=torch.int8, device="cuda")
        bcs.bcs_build(p, r0, r1, recv, send, ws)
        torch.cuda.synchronize()
        assert np.array_equal(recv.cpu().numpy().reshape(-1, q), want_r), (r0, r1)
        assert np.array_equal(send.cpu().numpy().reshape(-1, q), want_s), (r0, r1)
        del ws


# ---------------------------------------------------------------- full-size workloads
@pytest.mark.parametrize("fast", [True, False])
def test_single_p_2pow20_plus_1_full_table(bcs, fast):
    p = workloads.P_SINGLE
    want_r, want_s = oracle.full_table(p)
    recv, send = _build(bcs, p, 0, p, fast=fast)
    assert recv.shape == (p, 21)
    assert np.array_equal(recv, want_r)
    assert np.array_equal(send, want_s)


def test_build_to_host_matches(bcs):
    p = 65537
    q = bcs.bcs_q(p)
    want_r, want_s = oracle.full_table(p)
    nb = p * q
    stage = torch.empty(2 * ((nb + 255) // 256 * 256) + bcs.bcs_build_workspace_bytes(p, 0, p),
                        dtype=torch.int8, device="cuda")
    hr = torch.zeros(nb, dtype=torch.int8).pin_memory()
    hs = torch.zeros(nb, dtype=torch.int8).pin_memory()
    bcs.bcs_build_to_host(p, 0, p, hr, hs, stage)
    torch.cuda.synchronize()
    assert np.array_equal(hr.numpy().reshape(p, q), want_r)
    assert np.array_equal(hs.numpy().reshape(p, q), want_s)
    hs.zero_()
    bcs.bcs_build_to_host(p, 100, 5000, None, hs, stage)
    torch.cuda.synchronize()
    assert np.array_equal(hs.numpy()[: 4900 * q].reshape(4900, q), want_s[100:5000])
    hs.zero_()
    bcs.bcs_build_to_host(p, 100, 5000, None, hs, stage[: 2 * ((4900 * q + 255) // 256 * 256)])
    torch.cuda.synchronize()                                  # no room for a workspace: slow path
    assert np.array_equal(hs.numpy()[: 4900 * q].reshape(4900, q), want_s[100:5000])


def test_batched_irregular_sweep_full_size(bcs):
    """4096 octave-uniform p in [2^10, 2^20): the launch the benchmark uses, 639 M ranks and
    24 GB of tables.  EVERY table is compared byte for byte with the oracle's array form (about
    a minute and a half of host time); for every p >= 2^16, 10^4 seeded ranks plus the ranks
    skips[k]-2 .. skips[k]+2 of every k (where the receive kernel switches to its general tile
    code), the root's neighbours and the last ranks are compared with the oracle's per-rank form
    as well, which shares nothing with the array form but Algorithms 1 and 2; and the library's
    property checker runs over every rank of every p."""
    plist = workloads.batch_p_list()
    plan = bcs.bcs_batch_plan(plist)
    assert plan.total_ranks == 639466253
    dev = plan.to("cuda")
    recv = torch.empty(plan.total_entries, dtype=torch.int8, device="cuda")
    send = torch.empty(plan.total_entries, dtype=torch.int8, device="cuda")
    ws = torch.empty(plan.workspace_bytes(),
                     dtype=torch.int8, device="cuda")
    bcs.bcs_build_batch(dev, recv, send, ws)
    torch.cuda.synchronize()
    assert bcs.bcs_wait_expired() == 0
    del ws
    eo = plan.entry_off.tolist()
    viol = torch.zeros(3, dtype=torch.int64, device="cuda")
    total_viol = torch.zeros(3, dtype=torch.int64, device="cuda")
    rng = np.random.default_rng(220510072)
    cache = {}
    for j, p in enumerate(plist):
        q = oracle.q_of(p)
        got_r, got_s = recv[eo[j]:eo[j + 1]], send[eo[j]:eo[j + 1]]
        if p not in cache:                       # duplicates of p are allowed in the list
            want_r, want_s = oracle.full_table(p)
            cache[p] = (torch.from_numpy(want_r).cuda().view(-1), torch.from_numpy(want_s).cuda().view(-1))
        assert torch.equal(got_r, cache[p][0]), (j, p)
        assert torch.equal(got_s, cache[p][1]), (j, p)
        if p < 2**16:
            del cache[p]                         # keep only what a duplicate could ask for again
        else:
            sk = oracle.skips(p)
            near = np.concatenate([sk[k] + np.arange(-2, 3) for k in range(q + 1)] + [[0, 1, 2]]) % p
            ranks = np.unique(np.concatenate([rng.integers(0, p, 10000), near]))
            want_r, want_s = oracle.build_ranks(p, ranks)
            idx = (torch.from_numpy(ranks)[:, None] * q + torch.arange(q)[None, :]).cuda()
            assert np.array_equal(got_r[idx].cpu().numpy(), want_r), p
            assert np.array_equal(got_s[idx].cpu().numpy(), want_s), p
            if len(cache) > 64:
                cache.clear()
        # bcs_validate wants 16-byte aligned tables; a table of the batch starts at any byte
        if eo[j] % 16 != 0:
            got_r, got_s = got_r.clone(), got_s.clone()
        bcs.bcs_validate(p, 0, p, got_r, got_s, viol)
        total_viol += viol
    assert total_viol.cpu().tolist() == [0, 0, 0]


def test_expansion_full_size(bcs):
    """p = 100003, n = 1000: 1016 rounds, 16 bytes per record, compared record by record."""
    p, n = workloads.P_EXPAND, workloads.N_EXPAND
    q = oracle.q_of(p)
    want_r, want_s = oracle.full_table(p)
    recv = torch.from_numpy(want_r).cuda()
    send = torch.from_numpy(want_s).cuda()
    rounds = n - 1 + q
    assert rounds == 1016 and p * rounds * 16 == 1625648768
    tab = torch.empty((p, rounds, 4), dtype=torch.int32, device="cuda")
    bcs.bcs_expand(p, n, 0, p, recv, send, tab)
    torch.cuda.synchronize()
    step = 20000
    for r0 in range(0, p, step):
        r1 = min(p, r0 + step)
        want = oracle.expand(p, n, want_r, want_s, r0, r1)
        assert np.array_equal(tab[r0:r1].cpu().numpy(), want), r0
    # a sub-range with rows of that range only, ragged against the 8-rank CTA tile
    sub = torch.empty((1003, rounds, 4), dtype=torch.int32, device="cuda")
    bcs.bcs_expand(p, n, 4321, 5324, recv[4321:5324].contiguous(), send[4321:5324].contiguous(), sub)
    torch.cuda.synchronize()
    assert torch.equal(sub, tab[4321:5324])


def test_expansion_small_cases_and_simulation(bcs):
    for p in (2, 3, 9, 20, 33, 257, 1000):
        q = oracle.q_of(p)
        want_r, want_s = oracle.full_table(p)
        recv, send = torch.from_numpy(want_r).cuda(), torch.from_numpy(want_s).cuda()
        for n in (1, 2, 5, q, q + 1, q + 3, 3 * q + 2, 700):
            raw = torch.full((p * (n - 1 + q) * 4 + 128,), -77, dtype=torch.int32, device="cuda")
            tab = raw[64:64 + p * (n - 1 + q) * 4].view(p, n - 1 + q, 4)
            bcs.bcs_expand(p, n, 0, p, recv, send, tab)
            torch.cuda.synchronize()
            assert bool((raw[:64] == -77).all()) and bool((raw[-64:] == -77).all())
            got = tab.cpu().numpy()
            assert np.array_equal(got, oracle.expand(p, n, want_r, want_s)), (p, n)
            if n <= 40:
                assert bcast_sim.simulate(p, n, got) is None


def test_expansion_builds_its_rows_when_given_no_tables(bcs):
    """bcs_expand with both tables NULL computes the rows of its ranks itself (Algorithm 6 calls
    recvsched and sendsched): same records as the oracle's literal loop, for whole small p, for
    sub-ranges around the root and the skips of larger p, and for the expansion workload's p."""
    for p in (2, 3, 9, 20, 33, 257, 1000):
        q = oracle.q_of(p)
        want_r, want_s = oracle.full_table(p)
        for n in (1, 5, q + 3, 3 * q + 2):
            raw = torch.full((p * (n - 1 + q) * 4 + 128,), -77, dtype=torch.int32, device="cuda")
            tab = raw[64:64 + p * (n - 1 + q) * 4].view(p, n - 1 + q, 4)
            bcs.bcs_expand(p, n, 0, p, None, None, tab)
            torch.cuda.synchronize()
            assert bool((raw[:64] == -77).all()) and bool((raw[-64:] == -77).all())
            assert np.array_equal(tab.cpu().numpy(), oracle.expand(p, n, want_r, want_s)), (p, n)
    for p, n, r0, r1 in ((workloads.P_EXPAND, workloads.N_EXPAND, 50000, 50100),
                         (workloads.P_EXPAND, 7, 0, 3000), (workloads.P_EXPAND, 40, 99000, 100003),
                         (workloads.P_SINGLE, 30, 2**19 - 50, 2**19 + 200),
                         (workloads.P_LARGE, 12, 2**29 - 20, 2**29 + 20), (2**31 - 1, 3, 0, 40)):
        q = oracle.q_of(p)
        want_r, want_s = oracle.build_range(p, r0, r1)
        tab = torch.empty((r1 - r0, n - 1 + q, 4), dtype=torch.int32, device="cuda")
        bcs.bcs_expand(p, n, r0, r1, None, None, tab)
        torch.cuda.synchronize()
        assert np.array_equal(tab.cpu().numpy(), oracle.expand_rows(p, n, r0, want_r, want_s)), (p, n, r0)
    L = bcs.lib()
    assert L.bcs_expand(10, 4, 0, 10, None, tab.data_ptr(), tab.data_ptr(), None) == 1   # one table only


def test_allgather_tables_match_oracle(bcs):
    """Algorithm 9's pack / unpack block numbers: every entry against the oracle's literal loops
    for small p, the library's own tables simulated (all p processors) for tiny p, and the
    expansion workload's size (p = 100003, n = 1000: 2 x 406 MB per processor) on sampled columns."""
    for p in (2, 3, 9, 33, 257, 1000):
        q = oracle.q_of(p)
        want_r, want_s = oracle.full_table(p)
        recv, send = torch.from_numpy(want_r).cuda(), torch.from_numpy(want_s).cuda()
        for n in (1, 2, 5, q + 3, 70, 300):
            rounds = n - 1 + q
            tabs = []
            for r in sorted({0, 1, p // 2, p - 1}) if p > 9 or n > 12 else range(p):
                raw = torch.full((2 * rounds * p + 64,), -77, dtype=torch.int32, device="cuda")
                pack = raw[32:32 + rounds * p].view(rounds, p)
                unpack = raw[32 + rounds * p:32 + 2 * rounds * p].view(rounds, p)
                bcs.bcs_allgather_tables(p, n, r, recv, send, pack, unpack)
                torch.cuda.synchronize()
                assert bool((raw[:32] == -77).all()) and bool((raw[-32:] == -77).all())
                o_pack, o_unpack = oracle.allgather_rank(p, n, r, want_r, want_s)
                assert np.array_equal(pack.cpu().numpy(), o_pack), (p, n, r)
                assert np.array_equal(unpack.cpu().numpy(), o_unpack), (p, n, r)
                tabs.append((pack.cpu().numpy(), unpack.cpu().numpy()))
            if len(tabs) == p:
                assert bcast_sim.simulate_allgather(p, n, [t[0] for t in tabs],
                                                    [t[1] for t in tabs]) is None, (p, n)
    p, n = workloads.P_EXPAND, workloads.N_EXPAND
    q = oracle.q_of(p)
    want_r, want_s = oracle.full_table(p)
    recv, send = torch.from_numpy(want_r).cuda(), torch.from_numpy(want_s).cuda()
    rounds = n - 1 + q
    pack = torch.empty((rounds, p), dtype=torch.int32, device="cuda")
    unpack = torch.empty((rounds, p), dtype=torch.int32, device="cuda")
    r = 54607
    bcs.bcs_allgather_tables(p, n, r, recv, send, pack, unpack)
    E = oracle.expand(p, n, want_r, want_s)          # identity pinned on the CPU: virtual ranks
    virt = (r - np.arange(p)) % p
    assert np.array_equal(pack.cpu().numpy(), E[virt, :, 0].T)
    assert np.array_equal(unpack.cpu().numpy(), E[virt, :, 1].T)
    only = torch.full((rounds, p), -5, dtype=torch.int32, device="cuda")
    bcs.bcs_allgather_tables(p, n, r, recv, send, None, only)
    assert torch.equal(only, unpack)
    L = bcs.lib()
    assert L.bcs_allgather_tables(p, n, p, recv.data_ptr(), send.data_ptr(), pack.data_ptr(), None, None) == 2
    assert L.bcs_allgather_tables(p, 0, 0, recv.data_ptr(), send.data_ptr(), pack.data_ptr(), None, None) == 1
    assert L.bcs_allgather_tables(p, n, 0, recv.data_ptr(), send.data_ptr(), None, None, None) == 1


def test_circulant_round_tables_match_oracle(bcs):
    """Algorithms 7 and 8: neighbour / range records for every rank and round."""
    for p, r0, r1 in ((1, 0, 1), (2, 0, 2), (33, 0, 33), (1000, 0, 1000), (100003, 0, 100003),
                      (100003, 4321, 5000), (2**31 - 1, 2**31 - 300, 2**31 - 1)):
        q = oracle.q_of(p)
        for census in (False, True):
            raw = torch.full(((r1 - r0) * q * 4 + 128,), -9, dtype=torch.int32, device="cuda")
            tab = raw[64:64 + (r1 - r0) * q * 4].view(r1 - r0, q, 4)
            bcs.bcs_circulant_rounds(p, r0, r1, census, tab if q else raw[64:])
            torch.cuda.synchronize()
            assert bool((raw[:64] == -9).all()) and bool((raw[-64:] == -9).all())
            assert np.array_equal(tab.cpu().numpy(), oracle.circulant_rounds(p, r0, r1, census)), (p, census)


def test_checksum_matches_oracle(bcs):
    rng = np.random.default_rng(11)
    out = torch.zeros(1, dtype=torch.int64, device="cuda")
    # (the word index passes 2^32, where the weights' high half changes, in the 2^34 - 40 case)
    for nbytes, first in ((0, 0), (1, 0), (3, 4), (4, 8), (1000, 16), (1003, 2**34 + 8),
                          (200003, 2**34 - 40), (5 * 2**20 + 1, 2**36)):
        host = rng.integers(-31, 31, nbytes).astype(np.int8)
        dev = torch.from_numpy(host).cuda() if nbytes else torch.zeros(4, dtype=torch.int8,
                                                                       device="cuda")
        bcs.bcs_checksum(dev, first, out, n_entries=nbytes)
        got = int(out.cpu()[0]) & (2**64 - 1)
        assert got == oracle.checksum(host, first), (nbytes, first)


def test_validate_counts_match_oracle(bcs):
    """bcs_validate on valid and on deliberately corrupted tables (corrupted on the CPU, in a copy
    of the oracle's tables): the three violation counts equal the oracle's."""
    rng = np.random.default_rng(17)
    out = torch.zeros(3, dtype=torch.int64, device="cuda")
    for p, r0, r1 in ((2, 0, 2), (33, 0, 33), (1000, 0, 1000), (100003, 0, 100003),
                      (100003, 777, 60001), (65537, 65000, 65537)):
        q = oracle.q_of(p)
        recv, send = oracle.full_table(p)
        recv, send = recv[r0:r1].copy(), send[r0:r1].copy()
        for corrupt in (0, 1, 40):
            for _ in range(corrupt):
                tbl = recv if rng.integers(2) else send
                j, k = rng.integers(r1 - r0), rng.integers(q)
                tbl[j, k] = rng.integers(-q, q)
            want = oracle.validate(p, r0, r1, recv, send)
            d_recv, d_send = torch.from_numpy(recv).cuda(), torch.from_numpy(send).cuda()
            bcs.bcs_validate(p, r0, r1, d_recv, d_send, out)
            assert tuple(out.cpu().tolist()) == want, (p, r0, r1, corrupt)
            if corrupt == 0:
                assert want == (0, 0, 0)
            bcs.bcs_validate(p, r0, r1, d_recv, None, out)
            assert tuple(out.cpu().tolist()) == oracle.validate(p, r0, r1, recv, None)
            bcs.bcs_validate(p, r0, r1, None, d_send, out)
            assert tuple(out.cpu().tolist()) == oracle.validate(p, r0, r1, None, send)
    L = bcs.lib()
    assert L.bcs_validate(10, 0, 10, None, None, out.data_ptr(), None) == 1
    assert L.bcs_validate(10, 0, 10, out.data_ptr(), None, None, None) == 1
    assert L.bcs_validate(10, 0, 11, out.data_ptr(), None, out.data_ptr(), None) == 2


def test_simulate_counts_match_oracle(bcs):
    """bcs_simulate against the oracle's brute-force run (and, for validity, the numpy simulation)
    on valid and corrupted tables, then on the benchmark's p = 2^20+1 built by the library."""
    rng = np.random.default_rng(29)
    counts = torch.zeros(5, dtype=torch.int64, device="cuda")
    for p in (2, 3, 9, 33, 100, 1000, 4097):
        q = oracle.q_of(p)
        recv, send = oracle.full_table(p)
        state = torch.empty(2 * p, dtype=torch.int64, device="cuda")
        for corrupt in (0, 1, 6):
            br, bs = recv.copy(), send.copy()
            for _ in range(corrupt):
                tbl = br if rng.integers(2) else bs
                tbl[rng.integers(p), rng.integers(q)] = rng.integers(-q, q)
            for n in (1, 2, 5, q + 3, 64):
                bcs.bcs_simulate(p, n, torch.from_numpy(br).cuda(), torch.from_numpy(bs).cuda(),
                                 state, counts)
                got = tuple(counts.cpu().tolist())
                assert got == oracle.simulate(p, n, br, bs), (p, n, corrupt)
                if corrupt == 0:
                    assert got[:4] == (0, 0, 0, 0) and got[4] < p
                    if n <= 13:
                        assert bcast_sim.simulate(p, n, oracle.expand(p, n, br, bs)) is None
    p = workloads.P_SINGLE
    q = bcs.bcs_q(p)
    recv = torch.empty(p * q, dtype=torch.int8, device="cuda")
    send = torch.empty(p * q, dtype=torch.int8, device="cuda")
    ws = torch.empty(bcs.bcs_build_workspace_bytes(p, 0, p), dtype=torch.int8, device="cuda")
    bcs.bcs_build(p, 0, p, recv, send, ws)
    state = torch.empty(2 * p, dtype=torch.int64, device="cuda")
    for n in (1, 5, q + 3):
        bcs.bcs_simulate(p, n, recv, send, state, counts)
        got = counts.cpu().tolist()
        assert got[:4] == [0, 0, 0, 0] and 1 <= got[4] < p, (n, got)
    L = bcs.lib()
    assert L.bcs_simulate(p, 65, recv.data_ptr(), send.data_ptr(), state.data_ptr(),
                          counts.data_ptr(), None) == 4
    assert L.bcs_simulate(p, 0, recv.data_ptr(), send.data_ptr(), state.data_ptr(),
                          counts.data_ptr(), None) == 1


def test_large_p_full_broadcast_simulation(bcs):
    """Every rank of p = 2^30 - 1: both complete tables (64 GB) built from one bcs_prepare, then
    the five-block broadcast simulated on the device -- 34 rounds, every rank receives every
    block exactly once from a rank that holds it."""
    torch.cuda.empty_cache()
    p, q, n = workloads.P_LARGE, 30, 5
    ws = torch.empty(bcs.bcs_prepare_workspace_bytes(p), dtype=torch.int8, device="cuda")
    bcs.bcs_prepare(p, ws)
    recv = torch.empty(p * q, dtype=torch.int8, device="cuda")
    send = torch.empty(p * q, dtype=torch.int8, device="cuda")
    bcs.bcs_build_prepared(p, 0, p, recv, send, ws)
    torch.cuda.synchronize()
    del ws
    torch.cuda.empty_cache()
    state = torch.empty(2 * p, dtype=torch.int64, device="cuda")
    counts = torch.zeros(5, dtype=torch.int64, device="cuda")
    bcs.bcs_simulate(p, n, recv, send, state, counts)
    got = counts.cpu().tolist()
    assert got[:4] == [0, 0, 0, 0] and 1 <= got[4] < p, got
    assert bcs.bcs_wait_expired() == 0
    del recv, send, state
    torch.cuda.empty_cache()


def test_large_p_chunked_spot_checked(bcs):
    """p = 2^30 - 1 (q = 30) in 8 rank chunks through one reused buffer: per chunk a checksum
    (two runs must agree; additive pieces must add up), the property checker over every rank of
    the chunk, and seeded sample ranks against the
    per-rank oracle (10^6 ranks for the receive rows, a tenth of them for the send rows, which
    the oracle recomputes with Algorithm 5 at cubic cost)."""
    p = workloads.P_LARGE
    q = 30
    chunks = workloads.large_chunks()
    assert len(chunks) == 8 and chunks[-1][1] == p
    ranks = np.array(workloads.spot_ranks(p, 1000000), dtype=np.int64)
    want_r, _ = oracle.build_ranks(p, ranks, want_send=False)
    send_ranks = ranks[:100000]
    _, want_s = oracle.build_ranks(p, send_ranks, want_recv=False)
    cap = (1 << 27) * q
    recv = torch.empty(cap, dtype=torch.int8, device="cuda")
    send = torch.empty(cap, dtype=torch.int8, device="cuda")
    ws = torch.empty(bcs.bcs_prepare_workspace_bytes(p), dtype=torch.int8, device="cuda")   # 36.5 GB
    bcs.bcs_prepare(p, ws)
    sums = torch.zeros(4, dtype=torch.int64, device="cuda")
    viol = torch.zeros(3, dtype=torch.int64, device="cuda")
    m64 = 2**64 - 1
    SEND_BASE = 1 << 36                 # entry index at which the send table is taken to start
    checked = 0
    for c, (r0, r1) in enumerate(chunks):
        nb = (r1 - r0) * q
        bcs.bcs_build_prepared(p, r0, r1, recv, send, ws)
        bcs.bcs_checksum(recv, r0 * q, sums[0:1], n_entries=nb)
        bcs.bcs_checksum(send, SEND_BASE + r0 * q, sums[1:2], n_entries=nb)
        bcs.bcs_validate(p, r0, r1, recv, send, viol)     # every rank of the chunk: row properties
        assert viol.cpu().tolist() == [0, 0, 0], c        # and pairing inside the chunk
        half = (nb // 2) // 4 * 4
        bcs.bcs_checksum(recv[:half], r0 * q, sums[2:3], n_entries=half)
        bcs.bcs_checksum(recv[half:], r0 * q + half, sums[3:4], n_entries=nb - half)
        first = [int(v) & m64 for v in sums.cpu()]
        assert (first[2] + first[3]) & m64 == first[0]
        sel = (ranks >= r0) & (ranks < r1)
        idx = (torch.from_numpy(ranks[sel] - r0)[:, None] * q + torch.arange(q)[None, :]).cuda()
        assert np.array_equal(recv[idx].cpu().numpy(), want_r[sel]), c
        sel_s = (send_ranks >= r0) & (send_ranks < r1)
        idx = (torch.from_numpy(send_ranks[sel_s] - r0)[:, None] * q
               + torch.arange(q)[None, :]).cuda()
        assert np.array_equal(send[idx].cpu().numpy(), want_s[sel_s]), c
        checked += int(sel.sum())
        # head of the chunk against the oracle's own checksum of its own rows
        head = 3000
        o_r, _ = oracle.build_range(p, r0, r0 + head, want_send=False)
        bcs.bcs_checksum(recv, r0 * q, sums[2:3], n_entries=head * q)
        assert int(sums.cpu()[2]) & m64 == oracle.checksum(o_r, r0 * q)
        if c in (0, 7):     # rebuilt by bcs_build (self-contained construction; at the last chunk
            recv.fill_(0)   # with its own workspace): same sums
            send.fill_(0)
            own = None
            if c == 7:
                own = torch.empty(bcs.bcs_build_workspace_bytes(p, r0, r1), dtype=torch.int8,
                                  device="cuda")
            bcs.bcs_build(p, r0, r1, recv, send, own)
            del own
            bcs.bcs_checksum(recv, r0 * q, sums[0:1], n_entries=nb)
            bcs.bcs_checksum(send, SEND_BASE + r0 * q, sums[1:2], n_entries=nb)
            again = [int(v) & m64 for v in sums.cpu()]
            assert again[:2] == first[:2]
    assert checked == len(ranks)
