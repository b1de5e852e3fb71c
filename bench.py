#!/usr/bin/env python
"""Benchmark of the schedule construction on one B200 (or N independent replicas).

Headline workload: the large single p = 2^30 - 1 (q = 30), all ranks, receive and send schedule
(64.4 GB of int8 tables), built in 8 rank chunks through one reused chunk buffer.  A step =
bcs_prepare_codes + 8 x bcs_prepare_rows + 8 x bcs_build_prepared.  The metric is schedule ranks
built per second.  The other workloads (single p = 2^20+1, the two batched sweeps, the round-table
expansion) are timed beside it, each with its roofline block and the oracle's time on the host.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--only PART]

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle on the host cores.
`--only PART` runs one small part alone (the profiler-friendly runs that profiles/ cites).
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "schedule ranks built/sec (int8 recv+send, q entries)"
UNIT = "ranks/s"
SM_COUNT = 148
ISSUE_PER_SM = 4 * 32          # thread instructions per clock: 4 schedulers x 32 lanes
ALU_LANES_PER_SM = 64          # INT32 lanes per SM per clock (one pipe)


# ------------------------------------------------------------------------------------ inputs
def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), float(d.get("sm_max_mhz", 1965.0)), "measured"
    return 6650.0, 1965.0, "fallback"


def _executed_counts():
    """profiles/executed_instructions.txt: thread instructions per rank that each kernel executes
    (smsp__thread_inst_executed.sum / ranks of an ncu capture) and the DRAM bytes of that launch."""
    out = {}
    path = os.path.join(ROOT, "profiles", "executed_instructions.txt")
    with open(path) as f:
        for ln in f:
            ln = ln.split("#")[0].split()
            if len(ln) >= 4:
                out[ln[0]] = {"thread_inst_per_rank": float(ln[1]),
                              "dram_bytes": None if ln[2] == "-" else float(ln[2]),
                              "ranks_captured": float(ln[3])}
    return out


def _model_ops():
    """tests/skipcode_model_ops.json, written by `python -m tests.skipcode_mirror --write`: integer
    operations per rank that the counted CPU restatement of the construction needs."""
    with open(os.path.join(ROOT, "tests", "skipcode_model_ops.json")) as f:
        return json.load(f)


class ClockSampler:
    """Polls SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nv = None

    def _run(self):
        nv = self._nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self._h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.005)

    def __enter__(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


class Probe:
    """libbcs_probe.so: the integer instruction rate of this GPU (benchmark helper, not product)."""

    def __init__(self, torch):
        from paper_2205_10072_b200 import build_ext
        self.torch = torch
        self.lib = ctypes.CDLL(build_ext.build_probe())
        self.lib.bcs_probe_int_rate.argtypes = [ctypes.c_int, ctypes.c_uint32, ctypes.c_void_p,
                                                ctypes.POINTER(ctypes.c_double),
                                                ctypes.POINTER(ctypes.c_float), ctypes.c_void_p]
        self.sink = torch.zeros(1, dtype=torch.int32, device="cuda")

    def rate(self, mix: int, iters: int = 4096) -> float:
        ops, ms = ctypes.c_double(0), ctypes.c_float(0)
        st = self.lib.bcs_probe_int_rate(mix, iters, self.sink.data_ptr(), ctypes.byref(ops),
                                         ctypes.byref(ms), self.torch.cuda.current_stream().cuda_stream or None)
        if st != 0:
            raise RuntimeError("bcs_probe_int_rate: status %d" % st)
        return ops.value / (ms.value * 1e-3)

    def all(self):
        names = ("logic_only", "logic_imad_mix", "logic_add_mix")
        out = {nm: max(self.rate(mix) for _ in range(3)) / 1e12 for mix, nm in enumerate(names)}
        out["unit"] = "Tint-op/s"
        return out


# ------------------------------------------------------------------------------------ reference arm
def run_reference(args) -> None:
    """CPU oracle (per-rank form: Algorithms 4 and 5 for every rank) on the host cores, on a bounded
    sample of the headline workload per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2205_10072_b200 import workloads
    p = workloads.P_LARGE
    sample = 16384                       # ranks per step: seeded spot ranks of the same p
    ranks = workloads.spot_ranks(p, sample)
    for _ in range(args.warmup):
        oracle.build_ranks(p, ranks)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.build_ranks(p, ranks)
    dt = time.perf_counter() - t0
    value = args.steps * sample / dt
    cores = oracle.num_threads()
    sample_txt = ("%d seeded ranks (next() %% p, splitmix64 seed %d) of p=2^30-1 per step, per-rank "
                  "form (Algorithms 4+5)" % (sample, workloads.SEED_SPOT))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8/int32",
        "data": "synthetic",
        "config": {"workload": WORKLOAD_LARGE, "p": p, "sample": sample_txt},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample_txt},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------------------------ timing helpers
def _event_ms(torch, fn, flush, steps, warmup):
    """Device time of `steps` calls of fn, each preceded by an (untimed) L2 flush."""
    for _ in range(warmup):
        flush()
        fn()
    torch.cuda.synchronize()
    pairs = []
    for _ in range(steps):
        flush()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        pairs.append((a, b))
    torch.cuda.synchronize()
    return [a.elapsed_time(b) for a, b in pairs]


def _no_flush():
    pass


def _alu_roofline(kernels, ranks, ms, out_bytes, hbm_gbs, sm_max_mhz, counts, model, measured):
    """Roofline block of a construction step (integer-issue bound).
    kernels: keys of profiles/executed_instructions.txt whose kernels ran in the `ms` that were timed;
    model: integer operations per rank of the counted CPU restatement, or None."""
    issue_peak = SM_COUNT * ISSUE_PER_SM * sm_max_mhz * 1e6 / 1e12           # T thread-inst/s
    one_pipe = SM_COUNT * ALU_LANES_PER_SM * sm_max_mhz * 1e6 / 1e12
    per_rank = sum(counts[k]["thread_inst_per_rank"] for k in kernels)
    achieved = per_rank * ranks / (ms * 1e-3) / 1e12
    t_int_ms = per_rank * ranks / (issue_peak * 1e12) * 1e3
    t_hbm_ms = out_bytes / (hbm_gbs * 1e9) * 1e3
    roof = {"bound": "alu", "kernel": "+".join(kernels), "achieved": achieved, "peak": issue_peak,
            "unit": "Tthread-inst/s", "frac": achieved / issue_peak, "ms": ms,
            "executed_thread_inst_per_rank": per_rank,
            "executed_source": "profiles/executed_instructions.txt (ncu smsp__thread_inst_executed.sum / ranks)",
            "peak_source": "issue limit: 148 SMs x 4 schedulers x 32 lanes x %.0f MHz (max SM clock)" % sm_max_mhz,
            "t_int_ms": t_int_ms, "t_hbm_ms": t_hbm_ms, "roofline_ms": max(t_int_ms, t_hbm_ms),
            "frac_of_max_t_int_t_hbm": max(t_int_ms, t_hbm_ms) / ms,
            "hbm_peak_gbs": hbm_gbs}
    if measured:
        two_pipe = max(measured["logic_imad_mix"], measured["logic_add_mix"])
        roof["peak_measured"] = measured
        roof["frac_of_measured_two_pipe_mix"] = achieved / two_pipe
    if model is not None:
        m_ach = model * ranks / (ms * 1e-3) / 1e12
        roof["model"] = {"int_ops_per_rank": model, "achieved": m_ach, "unit": "Tint-op/s",
                         "source": "tests/skipcode_model_ops.json (tests/skipcode_mirror.py --write)",
                         "frac_of_issue_limit": m_ach / issue_peak,
                         "frac_of_one_pipe_%.1fT" % one_pipe: m_ach / one_pipe}
        if measured:
            roof["model"]["frac_of_measured_two_pipe_mix"] = m_ach / max(measured["logic_imad_mix"],
                                                                         measured["logic_add_mix"])
    return roof


WORKLOAD_LARGE = ("large single p=2^30-1 (q=30), all ranks, recv+send int8 (64.4 GB), 8 rank chunks "
                  "through one reused chunk buffer")


class LargeP:
    """p = 2^30 - 1 in 8 rank chunks through one buffer pair (never all 64 GB resident)."""

    def __init__(self, torch, bcs, workloads):
        self.torch, self.bcs = torch, bcs
        self.p = workloads.P_LARGE
        self.q = bcs.bcs_q(self.p)
        self.chunks = workloads.large_chunks()
        cap = max(r1 - r0 for r0, r1 in self.chunks)
        self.recv = torch.empty(cap * self.q, dtype=torch.int8, device="cuda")
        self.send = torch.empty(cap * self.q, dtype=torch.int8, device="cuda")
        self.ws = torch.empty(bcs.bcs_prepare_workspace_bytes(self.p), dtype=torch.int8, device="cuda")
        self.launches_per_step = 1 + 2 * len(self.chunks)

    def step(self):
        bcs, p, ws = self.bcs, self.p, self.ws
        bcs.bcs_prepare_codes(p, ws)
        for r0, r1 in self.chunks:                   # receive rows of the chunk, round-major copy
            bcs.bcs_prepare_rows(p, r0, r1, self.recv, ws)
        for r0, r1 in self.chunks:                   # send rows of the chunk (Algorithm 9's lookup)
            bcs.bcs_build_prepared(p, r0, r1, None, self.send, ws)

    def parts_ms(self, reps=3):
        """codes / receive rows / send rows of a step, by CUDA events."""
        torch, bcs, p, ws = self.torch, self.bcs, self.p, self.ws
        acc = [0.0, 0.0, 0.0]
        for _ in range(reps):
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            ev[0].record()
            bcs.bcs_prepare_codes(p, ws)
            ev[1].record()
            for r0, r1 in self.chunks:
                bcs.bcs_prepare_rows(p, r0, r1, self.recv, ws)
            ev[2].record()
            for r0, r1 in self.chunks:
                bcs.bcs_build_prepared(p, r0, r1, None, self.send, ws)
            ev[3].record()
            torch.cuda.synchronize()
            for i in range(3):
                acc[i] += ev[i].elapsed_time(ev[i + 1]) / reps
        return acc

    def checked_step(self):
        """The step with a checksum of every chunk and the property check of its rows."""
        torch, bcs, p, q, ws = self.torch, self.bcs, self.p, self.q, self.ws
        sums = torch.zeros(2, dtype=torch.int64, device="cuda")
        viol = torch.zeros(3, dtype=torch.int64, device="cuda")
        total = torch.zeros(3, dtype=torch.int64, device="cuda")
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        bcs.bcs_prepare_codes(p, ws)
        for r0, r1 in self.chunks:
            bcs.bcs_prepare_rows(p, r0, r1, self.recv, ws)
            bcs.bcs_checksum(self.recv, r0 * q, sums[0:1], n_entries=(r1 - r0) * q)
            bcs.bcs_validate(p, r0, r1, self.recv, None, viol)
            total += viol
        for r0, r1 in self.chunks:
            bcs.bcs_build_prepared(p, r0, r1, None, self.send, ws)
            bcs.bcs_checksum(self.send, (1 << 36) + r0 * q, sums[1:2], n_entries=(r1 - r0) * q)
            bcs.bcs_validate(p, r0, r1, None, self.send, viol)
            total += viol
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b), total.cpu().tolist()

    def e2e(self, steps):
        """The step with every chunk copied to pinned HOST buffers inside the timed region: the
        kernels on one stream, the copies on a second one, two chunk buffers per table in turn, so
        that a chunk is built while the one before it crosses the link."""
        torch, bcs, p, ws, q = self.torch, self.bcs, self.p, self.ws, self.q
        dev = [[self.recv, torch.empty_like(self.recv)], [self.send, torch.empty_like(self.send)]]
        host = [[torch.empty(self.recv.numel(), dtype=torch.int8).pin_memory() for _ in range(2)]
                for _ in range(2)]
        main = torch.cuda.current_stream()
        copier = torch.cuda.Stream()
        free = [[torch.cuda.Event() for _ in range(2)] for _ in range(2)]   # buffer copied out

        def one():
            bcs.bcs_prepare_codes(p, ws)
            for table in (0, 1):                     # receive rows of all chunks, then send rows
                for i, (r0, r1) in enumerate(self.chunks):
                    n = (r1 - r0) * q
                    buf = dev[table][i & 1]
                    main.wait_event(free[table][i & 1])
                    if table == 0:
                        bcs.bcs_prepare_rows(p, r0, r1, buf, ws)
                    else:
                        bcs.bcs_build_prepared(p, r0, r1, None, buf, ws)
                    built = torch.cuda.Event()
                    built.record(main)
                    copier.wait_event(built)
                    with torch.cuda.stream(copier):
                        host[table][i & 1][:n].copy_(buf[:n], non_blocking=True)
                        free[table][i & 1].record(copier)
            torch.cuda.synchronize()

        one()
        t0 = time.perf_counter()
        for _ in range(steps):
            one()
        dt = (time.perf_counter() - t0) / steps
        return {"value": p / dt, "unit": UNIT, "h2d_bytes_per_step": 0,
                "d2h_bytes_per_step": 2 * p * self.q, "ms_per_step": dt * 1e3, "steps": steps,
                "how": "bcs_prepare_codes / bcs_prepare_rows / bcs_build_prepared through the C ABI, every "
                       "chunk copied to pinned host memory on a second stream while the next chunk is "
                       "built (two chunk buffers per table; inputs are scalars: no H2D)"}


def _bench_single(torch, bcs, workloads, flush, steps, hbm_gbs, sm_max_mhz, counts, model, measured):
    """Single p = 2^20+1: one bcs_build per step, L2 flushed before every step."""
    p = workloads.P_SINGLE
    q = bcs.bcs_q(p)
    nb = p * q
    recv = torch.empty(nb, dtype=torch.int8, device="cuda")
    send = torch.empty(nb, dtype=torch.int8, device="cuda")
    ws = torch.empty(bcs.bcs_build_workspace_bytes(p, 0, p), dtype=torch.int8, device="cuda")
    ms = _event_ms(torch, lambda: bcs.bcs_build(p, 0, p, recv, send, ws), flush, steps, 5)
    step_ms = statistics.mean(ms)
    # codes + receive kernel as the step runs them (rows and round-major copy), by bcs_prepare_rows
    pws = torch.empty(bcs.bcs_prepare_workspace_bytes(p), dtype=torch.int8, device="cuda")

    def recv_part():
        bcs.bcs_prepare_codes(p, pws)
        bcs.bcs_prepare_rows(p, 0, p, recv, pws)
    recv_ms = statistics.mean(_event_ms(torch, recv_part, flush, max(20, steps // 4), 3))
    slow_ms = statistics.mean(_event_ms(torch, lambda: bcs.bcs_build(p, 0, p, recv, send, None), flush, 10, 2))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(2000):
        bcs.bcs_build(p, 0, p, recv, send, ws)
    e1.record()
    torch.cuda.synchronize()
    res = {"workload": "single p=2^20+1 (q=21), all ranks, recv+send int8 (44 MB), one bcs_build per step",
           "ranks": p, "ms": step_ms, "median_ms": statistics.median(ms), "min_ms": min(ms),
           "ranks_per_s": p / step_ms * 1e3, "out_gbs": 2 * nb / step_ms / 1e6,
           "l2": "flushed before every timed step (256 MiB write)",
           "back_to_back_ms": e0.elapsed_time(e1) / 2000,
           "kernel_ms": {"codes+recv (bcs_prepare_codes + bcs_prepare_rows)": recv_ms,
                         "send transposition (difference)": max(step_ms - recv_ms, 0.0),
                         "self_contained_construction_step": slow_ms},
           "roofline": _alu_roofline(["codes_single_kernel@q21", "recv_codes_quad_kernel<true,true>@q21"], p,
                                     recv_ms, nb + nb, hbm_gbs, sm_max_mhz, counts,
                                     model["q21_p1048577"]["recv_int_ops_per_rank"], measured),
           "step_roofline": _alu_roofline(["codes_single_kernel@q21", "recv_codes_quad_kernel<true,true>@q21",
                                           "send_transpose_kernel@q21"], p, step_ms, 2 * nb, hbm_gbs,
                                          sm_max_mhz, counts,
                                          model["q21_p1048577"]["recv_int_ops_per_rank"]
                                          + model["q21_p1048577"]["send_int_ops_per_rank"], measured)}
    res["roofline"]["traffic"] = counts["recv_codes_quad_kernel<true,true>@q21"]["dram_bytes"]
    # property check and brute-force broadcast of the tables just built
    viol = torch.zeros(3, dtype=torch.int64, device="cuda")
    v_ms = statistics.mean(_event_ms(torch, lambda: bcs.bcs_validate(p, 0, p, recv, send, viol), flush, 10, 2))
    res["validate"] = {"ms": v_ms, "violations": viol.cpu().tolist()}
    state = torch.empty(2 * p, dtype=torch.int64, device="cuda")
    cnt = torch.zeros(5, dtype=torch.int64, device="cuda")
    s_ms = statistics.mean(_event_ms(torch, lambda: bcs.bcs_simulate(p, 5, recv, send, state, cnt), flush, 5, 1))
    res["simulate_5_blocks_25_rounds"] = {"ms": s_ms, "counts": cnt.cpu().tolist()}
    return res


def _bench_expand(torch, bcs, workloads, flush, hbm_gbs, peak_src, steps, counts):
    pe, ne = workloads.P_EXPAND, workloads.N_EXPAND
    qe = bcs.bcs_q(pe)
    er = torch.empty(pe * qe, dtype=torch.int8, device="cuda")
    es = torch.empty(pe * qe, dtype=torch.int8, device="cuda")
    ews = torch.empty(bcs.bcs_build_workspace_bytes(pe, 0, pe), dtype=torch.int8, device="cuda")
    bcs.bcs_build(pe, 0, pe, er, es, ews)
    rounds = ne - 1 + qe
    table = torch.empty((pe, rounds, 4), dtype=torch.int32, device="cuda")
    ms = statistics.mean(_event_ms(
        torch, lambda: bcs.bcs_expand(pe, ne, 0, pe, er, es, table), flush, steps, 3))
    nbytes = pe * rounds * 16
    gbs = nbytes / ms / 1e6
    res = {"workload": "round-table expansion p=100003, n=1000, all ranks, 1016 rounds, 16 B records", "ms": ms,
           "bytes": nbytes, "gbs": gbs, "ranks_per_s": pe / ms * 1e3,
           "roofline": {"bound": "hbm", "kernel": "expand_kernel", "achieved": gbs, "peak": hbm_gbs,
                        "unit": "GB/s", "frac": gbs / hbm_gbs,
                        "traffic": counts["expand_kernel@p100003_n1000"]["dram_bytes"],
                        "peak_source": peak_src}}
    # context: a plain store-only stream over the same buffer (cudaMemset through torch) and the
    # nominal HBM3e figure -- the measured copy peak mixes reads and writes
    st_ms = statistics.mean(_event_ms(torch, lambda: table.zero_(), flush, 5, 2))
    bcs.bcs_expand(pe, ne, 0, pe, er, es, table)
    res["roofline"]["store_only_fill_gbs"] = nbytes / st_ms / 1e6
    res["roofline"]["frac_of_store_only_fill"] = gbs / (nbytes / st_ms / 1e6)
    res["roofline"]["frac_of_nominal_8000"] = gbs / 8000.0
    return res, table


def _bench_allgather(torch, bcs, workloads, flush, hbm_gbs, peak_src, steps, counts):
    p, n = workloads.P_EXPAND, workloads.N_EXPAND
    q = bcs.bcs_q(p)
    er = torch.empty(p * q, dtype=torch.int8, device="cuda")
    es = torch.empty(p * q, dtype=torch.int8, device="cuda")
    ews = torch.empty(bcs.bcs_build_workspace_bytes(p, 0, p), dtype=torch.int8, device="cuda")
    bcs.bcs_build(p, 0, p, er, es, ews)
    rounds = n - 1 + q
    pack = torch.empty((rounds, p), dtype=torch.int32, device="cuda")
    unpack = torch.empty((rounds, p), dtype=torch.int32, device="cuda")
    ms = statistics.mean(_event_ms(
        torch, lambda: bcs.bcs_allgather_tables(p, n, 54607, er, es, pack, unpack), flush, steps, 3))
    nbytes = 2 * rounds * p * 4
    gbs = nbytes / ms / 1e6
    return {"workload": "p=100003, n=1000, processor 54607: pack+unpack int32 [1016][100003]",
            "ms": ms, "bytes": nbytes, "gbs": gbs,
            "roofline": {"bound": "hbm", "kernel": "allgather_kernel", "achieved": gbs,
                         "peak": hbm_gbs, "unit": "GB/s", "frac": gbs / hbm_gbs,
                         "traffic": counts["allgather_kernel@p100003_n1000"]["dram_bytes"],
                         "peak_source": peak_src}}


def _bench_checksum(torch, bcs, flush, hbm_gbs, peak_src, table, steps, counts):
    sums = torch.zeros(1, dtype=torch.int64, device="cuda")
    tb = table.view(torch.int8).view(-1)
    ms = statistics.mean(_event_ms(torch, lambda: bcs.bcs_checksum(tb, 0, sums), flush, steps, 3))
    gbs = tb.numel() / ms / 1e6
    return {"workload": "%.2f GB buffer" % (tb.numel() / 1e9), "ms": ms, "gbs": gbs,
            "roofline": {"bound": "hbm", "kernel": "checksum_kernel", "achieved": gbs,
                         "peak": hbm_gbs, "unit": "GB/s", "frac": gbs / hbm_gbs,
                         "traffic": counts["checksum_kernel@1625648768B"]["dram_bytes"]
                         if tb.numel() == 1625648768 else None,
                         "peak_source": peak_src}}


def _bench_batch(torch, bcs, workloads, flush, full, hbm_gbs, sm_max_mhz, counts, model, measured):
    out = {}
    plan = bcs.bcs_batch_plan(workloads.small_sweep())
    dplan = plan.to("cuda")
    br = torch.empty(plan.total_entries, dtype=torch.int8, device="cuda")
    bs = torch.empty(plan.total_entries, dtype=torch.int8, device="cuda")
    bw = torch.empty(plan.workspace_bytes(),
                     dtype=torch.int8, device="cuda")
    ms = statistics.mean(_event_ms(
        torch, lambda: bcs.bcs_build_batch(dplan, br, bs, bw),
        flush, 20, 3))
    batch_kernels = ["codes_batch_kernel", "recv_quad_batch_kernel<true>", "send_batch_kernel"]
    small_kernels = ["fused_small_batch_kernel<true>"]
    out["batch_small_sweep"] = {
        "workload": "every p in 2..1024, all ranks, one bcs_build_batch (one launch: a CTA per p)",
        "ranks": plan.total_ranks, "ms": ms, "ranks_per_s": plan.total_ranks / ms * 1e3,
        "out_gbs": 2 * plan.total_entries / ms / 1e6,
        "l2": "flushed before every timed step",
        "roofline": _alu_roofline([k + "@small_sweep" for k in small_kernels], plan.total_ranks, ms,
                                  2 * plan.total_entries, hbm_gbs, sm_max_mhz, counts,
                                  model["small_sweep_2_1024"]["recv_int_ops_per_rank"]
                                  + model["small_sweep_2_1024"]["send_int_ops_per_rank"], measured)}
    plist = workloads.batch_p_list() if full else workloads.batch_p_list(count=256)
    plan = bcs.bcs_batch_plan(plist)
    dplan = plan.to("cuda")
    del br, bs, bw
    br = torch.empty(plan.total_entries, dtype=torch.int8, device="cuda")
    bs = torch.empty(plan.total_entries, dtype=torch.int8, device="cuda")
    bw = torch.empty(plan.workspace_bytes(),
                     dtype=torch.int8, device="cuda")
    ms = statistics.mean(_event_ms(
        torch, lambda: bcs.bcs_build_batch(dplan, br, bs, bw),
        _no_flush, 3, 1))                          # the outputs exceed L2 by themselves
    out["batch_irregular_sweep"] = {
        "workload": "%d octave-uniform p in [2^10,2^20), seed %d, one bcs_build_batch"
                    % (len(plist), workloads.SEED_BATCH),
        "ranks": plan.total_ranks, "ms": ms, "ranks_per_s": plan.total_ranks / ms * 1e3,
        "out_gbs": 2 * plan.total_entries / ms / 1e6,
        "l2": "outputs (%.1f GB) exceed L2" % (2 * plan.total_entries / 1e9),
        "roofline": _alu_roofline([k + "@256p_sample" for k in batch_kernels], plan.total_ranks, ms,
                                  2 * plan.total_entries, hbm_gbs, sm_max_mhz, counts,
                                  model["batch_4096p"]["recv_int_ops_per_rank"]
                                  + model["batch_4096p"]["send_int_ops_per_rank"], measured)}
    return out


def _cpu_baselines(oracle, workloads):
    """The oracle as it stands on the host cores: a bounded sample of every workload."""
    res = {}
    cores = oracle.num_threads()
    # headline: seeded ranks of p = 2^30-1, per-rank form, about 10 s
    p = workloads.P_LARGE
    ranks = workloads.spot_ranks(p, 1 << 16)
    n, dt = 0, 0.0
    while dt < 10.0:
        t0 = time.perf_counter()
        oracle.build_ranks(p, ranks)
        dt += time.perf_counter() - t0
        n += len(ranks)
    head = {"value": n / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "%d x 65536 seeded ranks (next() %% p, splitmix64 seed %d) of p=2^30-1, per-rank form "
                      "(Algorithms 4+5), %.1f s; the whole workload at this rate would take %.0f s "
                      "(extrapolated)" % (n // 65536, workloads.SEED_SPOT, dt, p / (n / dt))}
    t0 = time.perf_counter()
    oracle.build_ranks(p, ranks, want_send=False)
    head["recv_only_value"] = len(ranks) / (time.perf_counter() - t0)
    # every p <= 1024 (array form, all of it)
    t0 = time.perf_counter()
    total = 0
    for pj in workloads.small_sweep():
        oracle.full_table(pj)
        total += pj
    res["batch_small_sweep"] = {"value": total / (time.perf_counter() - t0), "unit": UNIT, "cores": cores,
                                "sample": "all of it, array form"}
    # single p = 2^20+1: array form (all of it) and per-rank form (2^18 ranks)
    p2 = workloads.P_SINGLE
    t0 = time.perf_counter()
    want_r, want_s = oracle.full_table(p2)
    res["single_p"] = {"array_form_value": p2 / (time.perf_counter() - t0), "unit": UNIT, "cores": cores}
    t0 = time.perf_counter()
    oracle.build_range(p2, 0, 1 << 18)
    res["single_p"]["value"] = (1 << 18) / (time.perf_counter() - t0)
    res["single_p"]["sample"] = "ranks 0..262143, per-rank form; array form: all ranks"
    # batched irregular sweep: the first 64 p of the list, array form
    t0 = time.perf_counter()
    total = 0
    for pj in workloads.batch_p_list(count=64):
        oracle.full_table(pj)
        total += pj
    res["batch_irregular_sweep"] = {"value": total / (time.perf_counter() - t0), "unit": UNIT, "cores": cores,
                                    "sample": "the first 64 p of the list (%d ranks), array form" % total}
    # expansion: Algorithm 6's literal loop for 4096 ranks of p = 100003, n = 1000
    pe, ne = workloads.P_EXPAND, workloads.N_EXPAND
    er, es = oracle.full_table(pe)
    t0 = time.perf_counter()
    oracle.expand(pe, ne, er, es, 0, 4096)
    dt = time.perf_counter() - t0
    res["expand"] = {"value": 4096 / dt, "unit": UNIT, "gbs": 4096 * (ne - 1 + oracle.q_of(pe)) * 16 / dt / 1e9,
                     "cores": cores, "sample": "ranks 0..4095 of p=100003, n=1000 (schedules given)"}
    return head, res


# ------------------------------------------------------------------------------------ our arm
def run_ours(args) -> None:
    import torch
    import torch.distributed as dist

    import paper_2205_10072_b200 as bcs
    from paper_2205_10072_b200 import workloads

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    bcs.lib()

    hbm_gbs, sm_max_mhz, peak_src = _peaks()
    counts = _executed_counts()
    model = _model_ops()
    flush_buf = torch.empty(256 << 20, dtype=torch.int8, device="cuda")   # > 126 MB L2

    def flush():
        flush_buf.fill_(1)

    if args.only != "all":                         # small single-part runs (what profiles/ cites)
        if rank == 0:
            print(json.dumps({"only": args.only, "steps": args.steps,
                              "aux": _run_part(args, torch, bcs, workloads, flush, hbm_gbs, sm_max_mhz,
                                               peak_src, counts, model)}))
        return

    large = LargeP(torch, bcs, workloads)
    p, q = large.p, large.q

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- the timed region: K steps, device time per step by CUDA events (a step writes 64 GB
    # through 8 GB chunk buffers: far more than the L2 holds, so no flush between steps)
    for _ in range(args.warmup):
        large.step()
    barrier()
    with ClockSampler(local) as clk:
        t_wall0 = time.perf_counter()
        ms = _event_ms(torch, large.step, _no_flush, args.steps, 0)
        barrier()
        t_wall = time.perf_counter() - t_wall0
    total_ms = sum(ms)
    if world > 1:
        t = torch.tensor([total_ms], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    ms_per_step = total_ms / args.steps
    value = world * p / (ms_per_step * 1e-3)

    out = None
    if rank == 0:
        measured = Probe(torch).all()
        codes_ms, rows_ms, send_ms = large.parts_ms()
        m30 = model["q30_p1073741823"]
        roof = _alu_roofline(["recv_codes_quad_kernel<true,true>@q30"], p, rows_ms, 2 * p * q, hbm_gbs,
                             sm_max_mhz, counts, m30["recv_int_ops_per_rank"] - m30["code_ops_per_rank"],
                             measured)
        roof["kernel"] = "recv_codes_quad_kernel<true,true> (8 launches of bcs_prepare_rows: %.1f%% of the step)" \
                         % (100 * rows_ms / (codes_ms + rows_ms + send_ms))
        roof["traffic"] = None
        roof["traffic_note"] = ("not captured at this size (8 GB per launch); the DRAM bytes of a 2^22-rank "
                                "range of the same p are in profiles/, they do not scale in proportion "
                                "(re-reads of the skip codes depend on what the L2 still holds)")
        step_roof = _alu_roofline(["codes_single_kernel@q30", "recv_codes_quad_kernel<true,true>@q30",
                                   "send_transpose_kernel@q30"], p, ms_per_step, 2 * p * q, hbm_gbs,
                                  sm_max_mhz, counts,
                                  m30["recv_int_ops_per_rank"] + m30["send_int_ops_per_rank"], measured)
        checked_ms, violations = large.checked_step()
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u32", "data": "synthetic",
            "config": {"workload": WORKLOAD_LARGE, "p": p, "q": q, "chunks": len(large.chunks),
                       "send_variant": "lookup (rotated transposition of the round-major receive copy)",
                       "l2": "no flush: every step streams 64 GB of outputs through 8 GB chunk buffers, "
                             "far beyond the 126 MB L2",
                       "workspace_bytes": large.ws.numel(),
                       "parallelism": "replicas" if world > 1 else "1 GPU",
                       "timed_wall_s": t_wall},
            "out_gbs": 2 * p * q / ms_per_step / 1e6,
            "timing": {"median_ms": statistics.median(ms), "min_ms": min(ms), "max_ms": max(ms)},
            "kernel_ms": {"codes (bcs_prepare_codes)": codes_ms, "receive rows (8 x bcs_prepare_rows)": rows_ms,
                          "send rows (8 x bcs_build_prepared)": send_ms},
            "roofline": roof, "step_roofline": step_roof,
            "gpu_launches": large.launches_per_step * args.steps, "clocks": clk.summary(),
            "checked_step": {"what": "the step plus a checksum and the property check of every chunk",
                             "ms": checked_ms, "violations": violations},
            "wait_expired": bcs.bcs_wait_expired(),
        }
        out["e2e"] = large.e2e(2)
        del large
        torch.cuda.empty_cache()
        # ---- the other workloads (each with its own roofline block)
        cfg = {}
        cfg["single_p"] = _bench_single(torch, bcs, workloads, flush, 300, hbm_gbs, sm_max_mhz, counts,
                                        model, measured)
        cfg.update(_bench_batch(torch, bcs, workloads, flush, True, hbm_gbs, sm_max_mhz, counts, model,
                                measured))
        cfg["expand"], table = _bench_expand(torch, bcs, workloads, flush, hbm_gbs, peak_src, 20, counts)
        cfg["checksum"] = _bench_checksum(torch, bcs, flush, hbm_gbs, peak_src, table, 20, counts)
        del table
        cfg["allgather_tables"] = _bench_allgather(torch, bcs, workloads, flush, hbm_gbs, peak_src, 20,
                                                   counts)
        out["configs"] = cfg
        # ---- CPU baseline: the oracle as it stands, bounded samples
        import oracle
        out["cpu_baseline"], per_cfg = _cpu_baselines(oracle, workloads)
        for name, base in per_cfg.items():
            cfg[name]["cpu_baseline"] = base
    else:
        del large
    barrier()
    if world > 1:
        dist.destroy_process_group()
    if out is not None:
        print(json.dumps(out))


def _run_part(args, torch, bcs, workloads, flush, hbm_gbs, sm_max_mhz, peak_src, counts, model):
    """One part alone, small enough for a profiler (see profiles/ for the commands)."""
    res = {}
    if args.only == "probe":
        probe = Probe(torch)
        res["int_rate_probe"] = {nm: [probe.rate(mix, 1024) / 1e12 for _ in range(2)]
                                 for mix, nm in enumerate(("logic_only", "logic_imad_mix", "logic_add_mix"))}
        res["int_rate_probe"]["unit"] = "Tint-op/s"
    elif args.only == "build":
        res["single_p"] = _bench_single(torch, bcs, workloads, flush, args.steps, hbm_gbs, sm_max_mhz, counts,
                                        model, None)
    elif args.only == "large-sample":
        # 2^22 ranks in the middle of p = 2^30-1 through bcs_build with its workspace: the same codes and
        # receive kernels as the headline's step on 4.4 GB of device memory (the send rows of a
        # sub-range come from the gather kernel, which the headline does not use)
        p = workloads.P_LARGE
        q = bcs.bcs_q(p)
        r0, r1 = 1 << 29, (1 << 29) + (1 << 22)
        recv = torch.empty((r1 - r0) * q, dtype=torch.int8, device="cuda")
        send = torch.empty((r1 - r0) * q, dtype=torch.int8, device="cuda")
        ws = torch.empty(bcs.bcs_build_workspace_bytes(p, r0, r1), dtype=torch.int8, device="cuda")
        ms = _event_ms(torch, lambda: bcs.bcs_build(p, r0, r1, recv, send, ws), _no_flush, args.steps, 1)
        res["large_sample"] = {"p": p, "ranks": r1 - r0, "ms": statistics.mean(ms)}
    elif args.only == "large-transpose":
        # the send transposition of the headline on a p with the same q = 30 that fits in 20 GB
        p = (1 << 29) + 1
        q = bcs.bcs_q(p)
        ws = torch.empty(bcs.bcs_prepare_workspace_bytes(p), dtype=torch.int8, device="cuda")
        bcs.bcs_prepare(p, ws)
        r0, r1 = 1 << 28, (1 << 28) + (1 << 24)
        send = torch.empty((r1 - r0) * q, dtype=torch.int8, device="cuda")
        ms = _event_ms(torch, lambda: bcs.bcs_build_prepared(p, r0, r1, None, send, ws), _no_flush, args.steps, 1)
        res["large_transpose"] = {"p": p, "ranks": r1 - r0, "ms": statistics.mean(ms)}
    elif args.only == "allgather":
        res["allgather_tables"] = _bench_allgather(torch, bcs, workloads, flush, hbm_gbs, peak_src, args.steps,
                                                   counts)
    elif args.only in ("expand", "checksum"):
        ex, table = _bench_expand(torch, bcs, workloads, flush, hbm_gbs, peak_src, args.steps, counts)
        res["expand"] = ex
        if args.only == "checksum":
            res["checksum"] = _bench_checksum(torch, bcs, flush, hbm_gbs, peak_src, table, args.steps, counts)
    elif args.only == "batch":
        res = _bench_batch(torch, bcs, workloads, flush, False, hbm_gbs, sm_max_mhz, counts, model, None)
    return res


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--only", default="all",
                    choices=["all", "build", "large-sample", "large-transpose", "expand", "checksum", "batch",
                             "allgather", "probe"],
                    help="run one part only (small, profiler-friendly runs); 'all' is the benchmark")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
