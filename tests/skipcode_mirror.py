"""Python access to skipcode_mirror.c: the CPU restatement, with operation counters, of the
skip-code construction that the fast CUDA kernels run (test infrastructure).

    python -m tests.skipcode_mirror --write     rewrites tests/skipcode_model_ops.json

The JSON table holds the model's integer operations per rank for the benchmark's workloads
(q = 17, 21, 30 and the batched mix); bench.py reads it as the model numerator of the integer
roofline.  Nothing here touches the CUDA library or the oracle.
"""
from __future__ import annotations

import ctypes
import json
import os
import subprocess
import sys

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "skipcode_mirror.c")
_LIB = os.path.join(_HERE, "libskipcode_mirror.so")
TABLE = os.path.join(_HERE, "skipcode_model_ops.json")
_lib = None

COUNTERS = ["ranks", "code_ops", "table_ops", "head_ops", "step2_ops", "rest_ops", "home_ops",
            "store_ops", "send_ops", "rounds_table", "rounds_head", "rounds_step2", "rounds_rest",
            "rounds_second", "rounds_home"]
_QUARTERS = {"code_ops", "table_ops", "head_ops", "step2_ops", "rest_ops", "home_ops", "store_ops",
             "send_ops"}


def _load():
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
            tmp = _LIB + ".%d.tmp" % os.getpid()
            subprocess.check_call(["gcc", "-O2", "-std=c99", "-Wall", "-shared", "-fPIC", "-o", tmp, _SRC])
            os.replace(tmp, _LIB)
        L = ctypes.CDLL(_LIB)
        c = ctypes
        L.skm_q.argtypes = [c.c_uint32]
        L.skm_rows.argtypes = [c.c_uint32, c.c_void_p, c.c_uint64, c.c_void_p, c.c_void_p, c.c_void_p]
        L.skm_full.argtypes = [c.c_uint32, c.c_void_p, c.c_void_p, c.c_void_p]
        L.skm_codes_blocks.argtypes = [c.c_uint32, c.c_uint64, c.c_uint64, c.c_void_p, c.c_void_p]
        L.skm_codes_plain.argtypes = [c.c_uint32, c.c_uint64, c.c_uint64, c.c_void_p]
        L.skm_small.argtypes = [c.c_uint32, c.c_void_p, c.c_void_p, c.c_void_p]
        L.skm_set_table_mode.argtypes = [c.c_int]
        L.skm_set_table_mode.restype = None
        L.skm_set_batch.argtypes = [c.c_int]
        L.skm_set_batch.restype = None
        assert L.skm_ncount() == len(COUNTERS)
        _lib = L
    return _lib


def set_table_mode(mode: int) -> None:
    """0: short windows from exact sets when p >= 64 (as the GPU); 1: never; 2: for every p."""
    _load().skm_set_table_mode(mode)


def set_batch(on: bool) -> None:
    """Codes as the batch kernel scans them (32 ranks per scan for every q) or as the kernel of
    one p does (16 for q <= 22)."""
    _load().skm_set_batch(1 if on else 0)


def _counts(raw) -> dict:
    out = {}
    for name, v in zip(COUNTERS, raw.tolist()):
        out[name] = v / 4.0 if name in _QUARTERS else v
    return out


def full(p: int, want_send: bool = True):
    """(recv [p][q], send [p][q] or None, counters) for all ranks of p."""
    L = _load()
    q = L.skm_q(p)
    recv = np.zeros((p, q), dtype=np.int8)
    send = np.zeros((p, q), dtype=np.int8) if want_send else None
    cnt = np.zeros(len(COUNTERS), dtype=np.uint64)
    rc = L.skm_full(p, recv.ctypes.data, send.ctypes.data if want_send else None, cnt.ctypes.data)
    if rc:
        raise RuntimeError("skm_full: %d" % rc)
    return recv, send, _counts(cnt)


def rows(p: int, ranks, want_send: bool = True):
    """(recv [n][q], send [n][q] or None, counters) for the listed ranks of p."""
    L = _load()
    q = L.skm_q(p)
    rk = np.ascontiguousarray(np.asarray(ranks, dtype=np.uint64))
    recv = np.zeros((rk.size, q), dtype=np.int8)
    send = np.zeros((rk.size, q), dtype=np.int8) if want_send else None
    cnt = np.zeros(len(COUNTERS), dtype=np.uint64)
    rc = L.skm_rows(p, rk.ctypes.data, rk.size, recv.ctypes.data,
                    send.ctypes.data if want_send else None, cnt.ctypes.data)
    if rc:
        raise RuntimeError("skm_rows: %d" % rc)
    return recv, send, _counts(cnt)


def small(p: int, want_send: bool = True):
    """(recv [p][q], send [p][q] or None, counters) for all ranks of a p <= 1024 by the run table
    over all ranks (what the batch kernel for small p does)."""
    L = _load()
    q = L.skm_q(p)
    recv = np.zeros((p, q), dtype=np.int8)
    send = np.zeros((p, q), dtype=np.int8) if want_send else None
    cnt = np.zeros(len(COUNTERS), dtype=np.uint64)
    rc = L.skm_small(p, recv.ctypes.data, send.ctypes.data if want_send else None, cnt.ctypes.data)
    if rc:
        raise RuntimeError("skm_small: %d" % rc)
    return recv, send, _counts(cnt)


def codes_blocks(p: int, g_begin: int, g_end: int, want_codes: bool = True):
    """(codes of the ranks g_begin..g_end-1 or None, {"ops", "blocks", "split", "plain"}) by one
    scan per block of 32 ranks; g_begin a multiple of 32."""
    L = _load()
    codes = np.zeros(g_end - g_begin, dtype=np.uint32) if want_codes else None
    ops = np.zeros(4, dtype=np.uint64)
    rc = L.skm_codes_blocks(p, g_begin, g_end, codes.ctypes.data if want_codes else None, ops.ctypes.data)
    if rc:
        raise RuntimeError("skm_codes_blocks: %d" % rc)
    return codes, dict(zip(("ops", "blocks", "split", "plain"), (int(v) for v in ops)))


def codes_plain(p: int, g_begin: int, g_end: int):
    """The same codes by the greedy scan of every rank."""
    L = _load()
    codes = np.zeros(g_end - g_begin, dtype=np.uint32)
    rc = L.skm_codes_plain(p, g_begin, g_end, codes.ctypes.data)
    if rc:
        raise RuntimeError("skm_codes_plain: %d" % rc)
    return codes


def per_rank(counts: dict) -> dict:
    """Model operations per rank: receive construction (skip code + rounds + stores), send lookup."""
    n = counts["ranks"]
    recv = sum(counts[k] for k in ("code_ops", "table_ops", "head_ops", "step2_ops", "rest_ops",
                                   "home_ops", "store_ops")) / n
    out = {"recv_int_ops_per_rank": recv, "send_int_ops_per_rank": counts["send_ops"] / n,
           "code_ops_per_rank": counts["code_ops"] / n, "ranks_counted": n}
    rounds = sum(counts[k] for k in ("rounds_table", "rounds_head", "rounds_step2", "rounds_rest",
                                     "rounds_home"))
    for k in ("rounds_table", "rounds_head", "rounds_step2", "rounds_rest", "rounds_second", "rounds_home"):
        out["share_" + k] = counts[k] / rounds
    return out


def model_table() -> dict:
    """The benchmark's workloads (seeded; the list generators live with the product's input
    recipes, which hold no schedule arithmetic)."""
    sys.path.insert(0, os.path.dirname(_HERE))
    from paper_2205_10072_b200 import workloads
    set_table_mode(0)
    table = {}
    for name, p in (("q17_p100003", workloads.P_EXPAND), ("q21_p1048577", workloads.P_SINGLE)):
        _, _, c = full(p, want_send=False)
        c["send_ops"] = 7 / 4 * skm_q(p) * c["ranks"]
        table[name] = dict(per_rank(c), p=p, q=skm_q(p), sample="all ranks")
    p = workloads.P_LARGE
    ranks = workloads.spot_ranks(p, 200000)
    _, _, c = rows(p, ranks, want_send=False)
    c["send_ops"] = 7 / 4 * skm_q(p) * c["ranks"]
    table["q30_p1073741823"] = dict(per_rank(c), p=p, q=skm_q(p),
                                    sample="200000 ranks next() %% p, splitmix64 seed %d" % workloads.SEED_SPOT)
    # batched mix: 512 seeded ranks of each of the 4096 p, weighted by p
    set_batch(True)
    g = workloads.SplitMix64(workloads.SEED_SPOT)
    tot = {}
    weight = 0
    for pj in workloads.batch_p_list():
        rk = [g.next() % pj for _ in range(512)]
        _, _, c = rows(pj, rk, want_send=False)
        c["send_ops"] = 7 / 4 * skm_q(pj) * c["ranks"]
        for k, v in c.items():
            tot[k] = tot.get(k, 0.0) + v * (pj / c["ranks"])
        weight += pj
    set_batch(False)
    table["batch_4096p"] = dict(per_rank(tot), sample="512 seeded ranks of each p, weighted by p",
                                total_ranks=weight)
    # every p in 2..1024, as one batch: each p by the run table over all its ranks
    tot = {}
    for pj in workloads.small_sweep():
        _, _, c = small(pj, want_send=True)
        for k, v in c.items():
            tot[k] = tot.get(k, 0.0) + v
    table["small_sweep_2_1024"] = dict(per_rank(tot), sample="all ranks of every p")
    return table


def skm_q(p: int) -> int:
    return _load().skm_q(p)


def load_table() -> dict:
    with open(TABLE) as f:
        return json.load(f)


if __name__ == "__main__":
    t = model_table()
    text = json.dumps(t, indent=1, sort_keys=True)
    if "--write" in sys.argv:
        with open(TABLE, "w") as f:
            f.write(text + "\n")
    print(text)
