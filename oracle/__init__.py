"""CPU oracle for the circulant-graph broadcast schedules -- TEST INFRASTRUCTURE.

Thin ctypes access to ``bcs_oracle.c`` (plain C, built with gcc on first use).
Nothing in the product package may import this module; only the tests, the
smoke check and the CPU-baseline leg of the benchmark do.  It imports nothing
from the product package either.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bcs_oracle.c")
_LIB = os.path.join(_HERE, "libbcs_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP for the rank-parallel loops)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-Wall", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        c = ctypes
        i8p = c.POINTER(c.c_int8)
        lib.bcso_q.argtypes = [c.c_uint32]
        lib.bcso_q.restype = c.c_int
        lib.bcso_skips.argtypes = [c.c_uint32, c.POINTER(c.c_uint32)]
        lib.bcso_skips.restype = c.c_int
        lib.bcso_baseblock.argtypes = [c.c_uint32, c.c_uint32]
        lib.bcso_baseblock.restype = c.c_int
        lib.bcso_baseblock_list.argtypes = [c.c_uint32, i8p]
        lib.bcso_baseblock_list.restype = None
        lib.bcso_rangeblocks.argtypes = [c.c_uint32, c.c_int64, c.c_int64]
        lib.bcso_rangeblocks.restype = c.c_uint32
        lib.bcso_rangeblocks_scan.argtypes = [c.c_uint32, c.c_int64, c.c_int64]
        lib.bcso_rangeblocks_scan.restype = c.c_uint32
        lib.bcso_recvsched.argtypes = [c.c_uint32, c.c_uint32, c.c_int, c.c_int, i8p]
        lib.bcso_recvsched.restype = c.c_int
        lib.bcso_sendsched.argtypes = [c.c_uint32, c.c_uint32, c.c_int, i8p]
        lib.bcso_sendsched.restype = c.c_int
        lib.bcso_build_range.argtypes = [c.c_uint32, c.c_uint64, c.c_uint64, c.c_int, i8p, i8p]
        lib.bcso_build_range.restype = c.c_int
        lib.bcso_build_ranks.argtypes = [c.c_uint32, c.POINTER(c.c_uint64), c.c_uint64, i8p, i8p]
        lib.bcso_build_ranks.restype = c.c_int
        lib.bcso_full_table.argtypes = [c.c_uint32, i8p, i8p]
        lib.bcso_full_table.restype = c.c_int
        lib.bcso_expand_rank.argtypes = [c.c_uint32, c.c_uint32, c.c_uint32, i8p, i8p,
                                         c.POINTER(c.c_int32)]
        lib.bcso_expand_rank.restype = None
        lib.bcso_expand_range.argtypes = [c.c_uint32, c.c_uint32, c.c_uint64, c.c_uint64, i8p, i8p,
                                          c.POINTER(c.c_int32)]
        lib.bcso_expand_range.restype = None
        lib.bcso_checksum.argtypes = [i8p, c.c_uint64, c.c_uint64]
        lib.bcso_checksum.restype = c.c_uint64
        lib.bcso_validate.argtypes = [c.c_uint32, c.c_uint64, c.c_uint64, i8p, i8p,
                                      c.POINTER(c.c_uint64)]
        lib.bcso_validate.restype = None
        lib.bcso_simulate.argtypes = [c.c_uint32, c.c_uint32, i8p, i8p, c.POINTER(c.c_uint64)]
        lib.bcso_simulate.restype = c.c_int
        lib.bcso_allgather_rank.argtypes = [c.c_uint32, c.c_uint32, c.c_uint32, i8p, i8p, c.c_int,
                                            c.POINTER(c.c_int32), c.POINTER(c.c_int32)]
        lib.bcso_allgather_rank.restype = c.c_int
        lib.bcso_allgather_rounds.argtypes = [c.c_uint32, c.c_uint32, c.POINTER(c.c_int32)]
        lib.bcso_allgather_rounds.restype = None
        lib.bcso_census_rounds.argtypes = [c.c_uint32, c.c_uint32, c.POINTER(c.c_int32)]
        lib.bcso_census_rounds.restype = None
        lib.bcso_set_root_mode.argtypes = [c.c_int]
        lib.bcso_set_root_mode.restype = None
        lib.bcso_num_threads.argtypes = []
        lib.bcso_num_threads.restype = c.c_int
        _lib = lib
    return _lib


def _i8(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int8)) if a is not None else None


def q_of(p: int) -> int:
    """q = ceil(log2 p) (Section 2)."""
    return _load().bcso_q(p)


def skips(p: int) -> np.ndarray:
    """Algorithm 1: the q+1 skips of the circulant graph."""
    buf = (ctypes.c_uint32 * 33)()
    q = _load().bcso_skips(p, buf)
    return np.array(buf[: q + 1], dtype=np.int64)


def baseblock(p: int, r: int) -> int:
    """Algorithm 2 (returns -1 for the root)."""
    return _load().bcso_baseblock(p, r)


def baseblock_list(p: int) -> np.ndarray:
    """Linear-time baseblock list (Section 2, text after Algorithm 2); entry 0 is -1."""
    out = np.empty(p, dtype=np.int8)
    _load().bcso_baseblock_list(p, _i8(out))
    return out


def rangeblocks(p: int, lo: int, hi: int) -> int:
    """Baseblocks of the cyclic processor range lo..hi as a bit set (what Algorithm 3 returns)."""
    return _load().bcso_rangeblocks(p, lo, hi)


def rangeblocks_scan(p: int, lo: int, hi: int) -> int:
    """Same set by visiting every processor of the range (the definition)."""
    return _load().bcso_rangeblocks_scan(p, lo, hi)


def recvsched(p: int, r: int, last: int | None = None, special: bool = True) -> np.ndarray:
    """Algorithm 4: receive blocks of rounds 0..last (default q-1) of processor r."""
    q = q_of(p)
    if last is None:
        last = q - 1
    out = np.zeros(max(last + 1, 0), dtype=np.int8)
    rc = _load().bcso_recvsched(p, r, last, int(special), _i8(out))
    if rc:
        raise RuntimeError("oracle recvsched failed: %d" % rc)
    return out


def sendsched(p: int, r: int, special: bool = True) -> np.ndarray:
    """Algorithm 5: send blocks of processor r by re-running Algorithm 4 for each to-neighbour."""
    q = q_of(p)
    out = np.zeros(q, dtype=np.int8)
    rc = _load().bcso_sendsched(p, r, int(special), _i8(out))
    if rc:
        raise RuntimeError("oracle sendsched failed: %d" % rc)
    return out


def build_range(p: int, r_begin: int, r_end: int, special: bool = True,
                want_recv: bool = True, want_send: bool = True):
    """Per-rank form (Algorithms 4 and 5) for ranks r_begin..r_end-1 -> (recv, send) int8 [n][q]."""
    q = q_of(p)
    n = r_end - r_begin
    recv = np.zeros((n, q), dtype=np.int8) if want_recv else None
    send = np.zeros((n, q), dtype=np.int8) if want_send else None
    rc = _load().bcso_build_range(p, r_begin, r_end, int(special), _i8(recv), _i8(send))
    if rc:
        raise RuntimeError("oracle build_range failed: %d" % rc)
    return recv, send


def build_ranks(p: int, ranks, want_recv: bool = True, want_send: bool = True):
    """Per-rank form on a list of ranks -> (recv, send) int8 [len(ranks)][q]."""
    q = q_of(p)
    ranks = np.ascontiguousarray(ranks, dtype=np.uint64)
    n = ranks.shape[0]
    recv = np.zeros((n, q), dtype=np.int8) if want_recv else None
    send = np.zeros((n, q), dtype=np.int8) if want_send else None
    rc = _load().bcso_build_ranks(p, ranks.ctypes.data_as(ctypes.POINTER(ctypes.c_uint64)), n,
                                  _i8(recv), _i8(send))
    if rc:
        raise RuntimeError("oracle build_ranks failed: %d" % rc)
    return recv, send


def full_table(p: int, want_send: bool = True):
    """Array form: all p receive rows by prefix counts over the baseblock list, send rows by the
    lookup of Algorithm 9 -> (recv, send) int8 [p][q]."""
    q = q_of(p)
    recv = np.zeros((p, q), dtype=np.int8)
    send = np.zeros((p, q), dtype=np.int8) if want_send else None
    rc = _load().bcso_full_table(p, _i8(recv), _i8(send))
    if rc:
        raise RuntimeError("oracle full_table failed: %d" % rc)
    return recv, send


def expand(p: int, n: int, recv: np.ndarray, send: np.ndarray, r_begin: int = 0,
           r_end: int | None = None) -> np.ndarray:
    """Algorithm 6 (without the communication): int32 [ranks][n-1+q][4] =
    (send block, receive block, to, from); recv/send are the full [p][q] tables."""
    q = q_of(p)
    if r_end is None:
        r_end = p
    recv = np.ascontiguousarray(recv, dtype=np.int8)
    send = np.ascontiguousarray(send, dtype=np.int8)
    assert recv.shape == (p, q) and send.shape == (p, q)
    out = np.zeros((r_end - r_begin, n - 1 + q, 4), dtype=np.int32)
    _load().bcso_expand_range(p, n, r_begin, r_end, _i8(recv), _i8(send),
                              out.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)))
    return out


def expand_rows(p: int, n: int, r_begin: int, recv_rows: np.ndarray, send_rows: np.ndarray) -> np.ndarray:
    """Algorithm 6 for the processors r_begin, r_begin+1, ... given only THEIR schedule rows
    ([count][q] each): int32 [count][n-1+q][4], one call of the literal per-processor loop each."""
    q = q_of(p)
    recv_rows = np.ascontiguousarray(recv_rows, dtype=np.int8)
    send_rows = np.ascontiguousarray(send_rows, dtype=np.int8)
    count = recv_rows.shape[0]
    assert recv_rows.shape == (count, q) and send_rows.shape == (count, q)
    out = np.zeros((count, n - 1 + q, 4), dtype=np.int32)
    fn = _load().bcso_expand_rank
    for j in range(count):
        fn(p, n, r_begin + j, _i8(recv_rows[j]), _i8(send_rows[j]),
           out[j].ctypes.data_as(ctypes.POINTER(ctypes.c_int32)))
    return out


def checksum(buf: np.ndarray, first_index: int = 0) -> int:
    """Order-independent 64-bit checksum of int8 entries (not from the paper)."""
    buf = np.ascontiguousarray(buf, dtype=np.int8).reshape(-1)
    return int(_load().bcso_checksum(_i8(buf), buf.shape[0], first_index))


def validate(p: int, r_begin: int, r_end: int, recv, send):
    """Ranks of the range whose rows break the promised properties -> (bad receive rows,
    bad send rows, send/receive mismatches); recv/send are [r_end-r_begin][q] or None."""
    q = q_of(p)
    n = r_end - r_begin
    if recv is not None:
        recv = np.ascontiguousarray(recv, dtype=np.int8).reshape(n, q)
    if send is not None:
        send = np.ascontiguousarray(send, dtype=np.int8).reshape(n, q)
    out = (ctypes.c_uint64 * 3)()
    _load().bcso_validate(p, r_begin, r_end, _i8(recv), _i8(send), out)
    return tuple(int(v) for v in out)


def simulate(p: int, n: int, recv, send):
    """Brute-force broadcast of n <= 64 blocks over the full tables -> (unheld sends, unpaired
    rounds, repeated receipts, ranks incomplete at the end, ranks complete before the last round)."""
    q = q_of(p)
    recv = np.ascontiguousarray(recv, dtype=np.int8).reshape(p, q)
    send = np.ascontiguousarray(send, dtype=np.int8).reshape(p, q)
    out = (ctypes.c_uint64 * 5)()
    rc = _load().bcso_simulate(p, n, _i8(recv), _i8(send), out)
    if rc:
        raise RuntimeError("oracle simulate failed: %d" % rc)
    return tuple(int(v) for v in out)


def allgather_rank(p: int, n: int, r: int, recv, send, adjust: bool = True):
    """Algorithm 9's pack and unpack block numbers of processor r -> (pack, unpack), int32
    [n-1+q][p]: entry [round][j] is the block of buffer[j] sent resp. received in that round.
    adjust=False leaves out the schedule adjustment of Algorithm 6 (Algorithm 9 as printed; only
    for the self-test that shows it is needed)."""
    q = q_of(p)
    recv = np.ascontiguousarray(recv, dtype=np.int8).reshape(p, q)
    send = np.ascontiguousarray(send, dtype=np.int8).reshape(p, q)
    pack = np.zeros((n - 1 + q, p), dtype=np.int32)
    unpack = np.zeros((n - 1 + q, p), dtype=np.int32)
    i32 = ctypes.POINTER(ctypes.c_int32)
    rc = _load().bcso_allgather_rank(p, n, r, _i8(recv), _i8(send), int(adjust),
                                     pack.ctypes.data_as(i32), unpack.ctypes.data_as(i32))
    if rc:
        raise RuntimeError("oracle allgather_rank failed: %d" % rc)
    return pack, unpack


def circulant_rounds(p: int, r_begin: int, r_end: int, census: bool) -> np.ndarray:
    """Round tables of Algorithm 7 (census=False: to, from, block count, receive offset) or
    Algorithm 8 (census=True: to, from, 1 if x_r is added to what is sent, 0) -> int32 [ranks][q][4]."""
    q = q_of(p)
    out = np.zeros((r_end - r_begin, q, 4), dtype=np.int32)
    fn = _load().bcso_census_rounds if census else _load().bcso_allgather_rounds
    i32 = ctypes.POINTER(ctypes.c_int32)
    for j, r in enumerate(range(r_begin, r_end)):
        fn(p, r, out[j].ctypes.data_as(i32))
    return out


def set_root_mode(mode: int) -> None:
    """Self-test switch: what the root adds to a range containing it (0 nothing, 1 block 0, 2 all)."""
    _load().bcso_set_root_mode(mode)


def num_threads() -> int:
    return _load().bcso_num_threads()
