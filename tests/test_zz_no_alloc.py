"""bcs_build_static: the entry point for callers that can neither allocate device memory nor
pass a workspace (it uses an 8 MiB scratch array that is part of the library).  Its tables must
be byte-identical to those of bcs_build and to the CPU oracle's, call after call, although every
call reuses the same scratch and finds the previous call's leftovers in it.

This file sorts last on purpose: a run that stops at the first failure has then already gone
through every other test.  It does not depend on them: it also passes alone in a fresh process.
"""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bcs():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2205_10072_b200 as lib
    lib.lib()
    torch.cuda.set_device(0)
    return lib


def _reference(bcs, p, r0, r1):
    q = bcs.bcs_q(p)
    recv = torch.empty((r1 - r0) * q, dtype=torch.int8, device="cuda")
    send = torch.empty((r1 - r0) * q, dtype=torch.int8, device="cuda")
    ws = torch.empty(bcs.bcs_build_workspace_bytes(p, r0, r1), dtype=torch.int8, device="cuda")
    bcs.bcs_build(p, r0, r1, recv, send, ws)
    torch.cuda.synchronize()
    return recv, send


_oracle_tables = {}


def _oracle_rows(p, r0, r1):
    """Rows r0..r1-1 of the oracle's tables (array form), as flat int8 CUDA tensors."""
    if p not in _oracle_tables:
        _oracle_tables[p] = oracle.full_table(p)
    recv, send = _oracle_tables[p]
    return (torch.from_numpy(np.ascontiguousarray(recv[r0:r1])).cuda().view(-1),
            torch.from_numpy(np.ascontiguousarray(send[r0:r1])).cuda().view(-1))


def test_static_scratch_matches_bcs_build_on_consecutive_calls(bcs):
    L = bcs.lib()
    limit = 8 << 20
    # two calls in a row, then more with other p and sub-ranges, all through the same scratch
    cases = [(100003, 0, 100003), (100003, 0, 100003), (65537, 1000, 60001), (300007, 0, 300007),
             (1000, 0, 1000), (2**20 + 1, 2**19, 2**19 + 150000), (100003, 99000, 100003)]
    for p, r0, r1 in cases:
        assert bcs.bcs_build_workspace_bytes(p, r0, r1) <= limit
        want_recv, want_send = _reference(bcs, p, r0, r1)
        q = bcs.bcs_q(p)
        recv = torch.full(((r1 - r0) * q,), 99, dtype=torch.int8, device="cuda")
        send = torch.full(((r1 - r0) * q,), 99, dtype=torch.int8, device="cuda")
        st = L.bcs_build_static(p, r0, r1, recv.data_ptr(), send.data_ptr(),
                                torch.cuda.current_stream().cuda_stream or None)
        assert st == 0, bcs.bcs_status_str(st)
        torch.cuda.synchronize()
        assert torch.equal(recv, want_recv), (p, r0, r1)     # integer tables: bit-exact
        assert torch.equal(send, want_send), (p, r0, r1)
        oracle_recv, oracle_send = _oracle_rows(p, r0, r1)   # and against the CPU oracle
        assert torch.equal(recv, oracle_recv), (p, r0, r1)
        assert torch.equal(send, oracle_send), (p, r0, r1)
    # one output only
    want_recv, want_send = _reference(bcs, 100003, 5, 7000)
    send = torch.empty_like(want_send)
    bcs.bcs_build_static(100003, 5, 7000, None, send)
    torch.cuda.synchronize()
    assert torch.equal(send, want_send)
    assert torch.equal(send, _oracle_rows(100003, 5, 7000)[1])
    _oracle_tables.clear()


def test_static_scratch_rejects_what_does_not_fit(bcs):
    L = bcs.lib()
    p = 2**20 + 1                                   # all ranks would need 26 MB of scratch
    assert bcs.bcs_build_workspace_bytes(p, 0, p) > (8 << 20)
    out = torch.full((4096,), 77, dtype=torch.int8, device="cuda")
    assert L.bcs_build_static(p, 0, p, out.data_ptr(), None, None) == 4     # BCS_ERR_UNSUPPORTED
    with pytest.raises(bcs.BcsError) as e:
        bcs.bcs_build_static(2**30 - 1, 0, 16, out, None)                   # 4*p alone is too much
    assert e.value.status == 4
    assert L.bcs_build_static(0, 0, 0, out.data_ptr(), None, None) == 2
    assert L.bcs_build_static(100, 0, 100, None, None, None) == 1
    assert L.bcs_build_static(1, 0, 1, None, None, None) == 0               # q == 0
    torch.cuda.synchronize()
    assert bool((out == 77).all())                   # a refused call writes nothing
