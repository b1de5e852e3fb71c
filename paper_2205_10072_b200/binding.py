"""ctypes binding of libbcs.so: argument marshalling only (include/bcs.h has the contracts)."""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

from . import build_ext

BCS_SKIPS_STRIDE = 32
BCS_BAD_ENTRY = 127

_c = ctypes
_lib = None


class BcsError(RuntimeError):
    """A bcs_* call returned a status other than BCS_OK."""

    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s" % (where, bcs_status_str(status)))


def lib_path() -> str:
    return build_ext.LIB_PATH


def lib():
    """Loads libbcs.so (must have been built: python -m paper_2205_10072_b200.build_ext)."""
    global _lib
    if _lib is None:
        if not os.path.exists(build_ext.LIB_PATH):
            raise ImportError(
                "libbcs.so is missing: build it with paper_2205_10072_b200.build_ext.build(); "
                "there is no CPU fallback")
        L = _c.CDLL(build_ext.LIB_PATH)
        vp, u32, u64, i32 = _c.c_void_p, _c.c_uint32, _c.c_uint64, _c.c_int
        L.bcs_status_str.argtypes = [i32]
        L.bcs_status_str.restype = _c.c_char_p
        L.bcs_q.argtypes = [u32]
        L.bcs_q.restype = i32
        L.bcs_skips.argtypes = [u32, vp]
        L.bcs_skips.restype = i32
        L.bcs_build_workspace_bytes.argtypes = [u32, u64, u64]
        L.bcs_build_workspace_bytes.restype = _c.c_size_t
        L.bcs_build.argtypes = [u32, u64, u64, vp, vp, vp, _c.c_size_t, vp]
        L.bcs_build.restype = i32
        L.bcs_prepare_workspace_bytes.argtypes = [u32]
        L.bcs_prepare_workspace_bytes.restype = _c.c_size_t
        L.bcs_prepare.argtypes = [u32, vp, _c.c_size_t, vp]
        L.bcs_prepare.restype = i32
        L.bcs_prepare_codes.argtypes = [u32, vp, _c.c_size_t, vp]
        L.bcs_prepare_codes.restype = i32
        L.bcs_prepare_rows.argtypes = [u32, u64, u64, vp, vp, _c.c_size_t, vp]
        L.bcs_prepare_rows.restype = i32
        L.bcs_build_prepared.argtypes = [u32, u64, u64, vp, vp, vp, _c.c_size_t, vp]
        L.bcs_build_prepared.restype = i32
        L.bcs_build_static.argtypes = [u32, u64, u64, vp, vp, vp]
        L.bcs_build_static.restype = i32
        L.bcs_build_to_host.argtypes = [u32, u64, u64, vp, vp, vp, _c.c_size_t, vp]
        L.bcs_build_to_host.restype = i32
        L.bcs_batch_plan.argtypes = [vp, u32, vp, vp, vp, vp, vp, vp]
        L.bcs_batch_plan.restype = i32
        L.bcs_build_batch_workspace_bytes.argtypes = [u64, u64]
        L.bcs_build_batch_workspace_bytes.restype = _c.c_size_t
        L.bcs_build_batch.argtypes = [vp, vp, vp, vp, vp, vp, vp, u32, u64, u64, u64, u64, vp, vp, vp,
                                      _c.c_size_t, vp]
        L.bcs_build_batch.restype = i32
        L.bcs_expand.argtypes = [u32, u32, u64, u64, vp, vp, vp, vp]
        L.bcs_expand.restype = i32
        L.bcs_validate.argtypes = [u32, u64, u64, vp, vp, vp, vp]
        L.bcs_validate.restype = i32
        L.bcs_circulant_rounds.argtypes = [u32, u64, u64, i32, vp, vp]
        L.bcs_circulant_rounds.restype = i32
        L.bcs_allgather_tables.argtypes = [u32, u32, u32, vp, vp, vp, vp, vp]
        L.bcs_allgather_tables.restype = i32
        L.bcs_simulate.argtypes = [u32, u32, vp, vp, vp, vp, vp]
        L.bcs_simulate.restype = i32
        L.bcs_build_rooted_workspace_bytes.argtypes = [u32, u32, u64, u64]
        L.bcs_build_rooted_workspace_bytes.restype = _c.c_size_t
        L.bcs_build_rooted.argtypes = [u32, u32, u64, u64, vp, vp, vp, _c.c_size_t, vp]
        L.bcs_build_rooted.restype = i32
        L.bcs_wait_expired.argtypes = [_c.POINTER(u64)]
        L.bcs_wait_expired.restype = i32
        L.bcs_checksum.argtypes = [vp, u64, u64, vp, vp]
        L.bcs_checksum.restype = i32
        _lib = L
    return _lib


def _check(status: int, where: str) -> None:
    if status != 0:
        raise BcsError(status, where)


def _ptr(t) -> int | None:
    return None if t is None else t.data_ptr()


def _stream(stream) -> int | None:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream or None


def bcs_status_str(status: int) -> str:
    return lib().bcs_status_str(int(status)).decode()


def bcs_q(p: int) -> int:
    return lib().bcs_q(p)


def bcs_skips(p: int) -> list[int]:
    buf = (_c.c_uint32 * (BCS_SKIPS_STRIDE + 1))()
    _check(lib().bcs_skips(p, buf), "bcs_skips")
    return list(buf[: bcs_q(p) + 1])


def _nbytes(t) -> int:
    return 0 if t is None else t.numel() * t.element_size()


def bcs_build_workspace_bytes(p: int, r_begin: int, r_end: int) -> int:
    return lib().bcs_build_workspace_bytes(p, r_begin, r_end)


def bcs_build(p: int, r_begin: int, r_end: int, recv_out, send_out, workspace=None,
              stream=None) -> None:
    """recv_out / send_out: CUDA int8 tensors of (r_end-r_begin)*q elements, or None;
    workspace: CUDA tensor of bcs_build_workspace_bytes(...) bytes (fast path) or None."""
    _check(lib().bcs_build(p, r_begin, r_end, _ptr(recv_out), _ptr(send_out), _ptr(workspace),
                           _nbytes(workspace), _stream(stream)), "bcs_build")


def bcs_build_rooted_workspace_bytes(p: int, root: int, r_begin: int, r_end: int) -> int:
    return lib().bcs_build_rooted_workspace_bytes(p, root, r_begin, r_end)


def bcs_build_rooted(p: int, root: int, r_begin: int, r_end: int, recv_out, send_out,
                     workspace=None, stream=None) -> None:
    """As bcs_build for a broadcast rooted at `root`: row r is the rank-0-rooted row of virtual
    rank (r - root) mod p."""
    _check(lib().bcs_build_rooted(p, root, r_begin, r_end, _ptr(recv_out), _ptr(send_out),
                                  _ptr(workspace), _nbytes(workspace), _stream(stream)),
           "bcs_build_rooted")


def bcs_prepare_workspace_bytes(p: int) -> int:
    return lib().bcs_prepare_workspace_bytes(p)


def bcs_prepare(p: int, workspace, stream=None) -> None:
    """Runs the construction once for all ranks of p into `workspace` (CUDA tensor of
    bcs_prepare_workspace_bytes(p) bytes) for later bcs_build_prepared calls."""
    _check(lib().bcs_prepare(p, _ptr(workspace), _nbytes(workspace), _stream(stream)), "bcs_prepare")


def bcs_prepare_codes(p: int, workspace, stream=None) -> None:
    """First half of bcs_prepare: the skip codes of all ranks of p into `workspace`."""
    _check(lib().bcs_prepare_codes(p, _ptr(workspace), _nbytes(workspace), _stream(stream)),
           "bcs_prepare_codes")


def bcs_prepare_rows(p: int, r_begin: int, r_end: int, recv_out, workspace, stream=None) -> None:
    """Second half, for one range (r_begin a multiple of 16): its entries into the round-major copy
    in `workspace` and, if recv_out is not None, its rank-major receive rows into recv_out."""
    _check(lib().bcs_prepare_rows(p, r_begin, r_end, _ptr(recv_out), _ptr(workspace),
                                  _nbytes(workspace), _stream(stream)), "bcs_prepare_rows")


def bcs_build_prepared(p: int, r_begin: int, r_end: int, recv_out, send_out, workspace,
                       stream=None) -> None:
    """Rank-major receive / send rows of a range from a workspace filled by bcs_prepare."""
    _check(lib().bcs_build_prepared(p, r_begin, r_end, _ptr(recv_out), _ptr(send_out),
                                    _ptr(workspace), _nbytes(workspace), _stream(stream)),
           "bcs_build_prepared")


def bcs_build_static(p: int, r_begin: int, r_end: int, recv_out, send_out, stream=None) -> None:
    """bcs_build with the library's built-in 8 MiB scratch: for callers that cannot allocate or
    pass a workspace.  Raises BcsError (BCS_ERR_UNSUPPORTED) when the range needs more."""
    _check(lib().bcs_build_static(p, r_begin, r_end, _ptr(recv_out), _ptr(send_out),
                                  _stream(stream)), "bcs_build_static")


def bcs_build_to_host(p: int, r_begin: int, r_end: int, recv_host, send_host, stage_dev,
                      stream=None) -> None:
    """recv_host / send_host: CPU int8 tensors (pinned for asynchronous copies) or None;
    stage_dev: CUDA uint8/int8 tensor used as staging."""
    _check(lib().bcs_build_to_host(p, r_begin, r_end, _ptr(recv_host), _ptr(send_host),
                                   _ptr(stage_dev), stage_dev.numel() * stage_dev.element_size(),
                                   _stream(stream)), "bcs_build_to_host")


@dataclass
class BatchPlan:
    """Host-side result of bcs_batch_plan (int64/int32 tensors hold the uint64/uint32 bit patterns)."""
    p_list: torch.Tensor      # int32 [num_p]
    rank_off: torch.Tensor    # int64 [num_p+1]
    entry_off: torch.Tensor   # int64 [num_p+1]
    tile_off: torch.Tensor    # int64 [num_p+1]
    copy_off: torch.Tensor    # int64 [num_p+1]
    skips_tab: torch.Tensor   # int32 [num_p, 32]
    full_tab: torch.Tensor    # int32 [num_p, 32]
    totals: tuple = ()        # (ranks, entries, tiles, copy bytes), kept on the host

    @property
    def num_p(self) -> int:
        return self.p_list.numel()

    @property
    def total_ranks(self) -> int:
        return self.totals[0]

    @property
    def total_entries(self) -> int:
        return self.totals[1]

    @property
    def total_tiles(self) -> int:
        return self.totals[2]

    @property
    def total_copy(self) -> int:
        return self.totals[3]

    def workspace_bytes(self) -> int:
        """bcs_build_batch_workspace_bytes for this plan."""
        return bcs_build_batch_workspace_bytes(self.total_ranks, self.total_copy)

    def to(self, device, non_blocking: bool = False) -> "BatchPlan":
        return BatchPlan(*(t.to(device, non_blocking=non_blocking)
                           for t in (self.p_list, self.rank_off, self.entry_off, self.tile_off,
                                     self.copy_off, self.skips_tab, self.full_tab)), totals=self.totals)


def bcs_batch_plan(p_list, pin: bool = False) -> BatchPlan:
    pl = torch.as_tensor(list(p_list) if not torch.is_tensor(p_list) else p_list,
                         dtype=torch.int64)
    if pl.numel() and (int(pl.min()) < 0 or int(pl.max()) > 0xFFFFFFFF):
        raise BcsError(2, "bcs_batch_plan")
    n = pl.numel()
    # uint32 bit patterns in an int32 tensor
    p32 = torch.where(pl >= 2**31, pl - 2**32, pl).to(torch.int32).contiguous()
    offs = [torch.zeros(n + 1, dtype=torch.int64) for _ in range(4)]
    skips_tab = torch.zeros((n, BCS_SKIPS_STRIDE), dtype=torch.int32)
    full_tab = torch.zeros((n, BCS_SKIPS_STRIDE), dtype=torch.int32)
    if pin:
        p32, skips_tab, full_tab = (t.pin_memory() for t in (p32, skips_tab, full_tab))
        offs = [t.pin_memory() for t in offs]
    _check(lib().bcs_batch_plan(p32.data_ptr(), n, offs[0].data_ptr(), offs[1].data_ptr(),
                                offs[2].data_ptr(), offs[3].data_ptr(), skips_tab.data_ptr(),
                                full_tab.data_ptr()), "bcs_batch_plan")
    return BatchPlan(p32, offs[0], offs[1], offs[2], offs[3], skips_tab, full_tab,
                     totals=tuple(int(t[-1]) for t in offs))


def bcs_build_batch_workspace_bytes(total_ranks: int, total_copy: int) -> int:
    return lib().bcs_build_batch_workspace_bytes(total_ranks, total_copy)


def bcs_build_batch(plan_dev: BatchPlan, recv_out, send_out, workspace=None, stream=None) -> None:
    """plan_dev: a BatchPlan whose tensors live on the CUDA device; workspace: CUDA tensor of
    plan.workspace_bytes() bytes (fast construction) or None."""
    _check(lib().bcs_build_batch(plan_dev.p_list.data_ptr(), plan_dev.rank_off.data_ptr(),
                                 plan_dev.entry_off.data_ptr(), plan_dev.tile_off.data_ptr(),
                                 plan_dev.copy_off.data_ptr(), plan_dev.skips_tab.data_ptr(),
                                 plan_dev.full_tab.data_ptr(), plan_dev.num_p, plan_dev.total_ranks,
                                 plan_dev.total_entries, plan_dev.total_tiles, plan_dev.total_copy,
                                 _ptr(recv_out), _ptr(send_out), _ptr(workspace),
                                 _nbytes(workspace), _stream(stream)), "bcs_build_batch")


def bcs_expand(p: int, n: int, r_begin: int, r_end: int, recv, send, table_out, stream=None) -> None:
    """recv/send: CUDA int8 rows of ranks r_begin..r_end-1; table_out: CUDA int32
    [(r_end-r_begin), n-1+q, 4]."""
    _check(lib().bcs_expand(p, n, r_begin, r_end, _ptr(recv), _ptr(send), _ptr(table_out),
                            _stream(stream)), "bcs_expand")


def bcs_validate(p: int, r_begin: int, r_end: int, recv, send, violations_out, stream=None) -> None:
    """recv/send: CUDA int8 rows of the range (or None); violations_out: CUDA int64 tensor with
    three elements: ranks with a bad receive row, a bad send row, a send/receive mismatch."""
    _check(lib().bcs_validate(p, r_begin, r_end, _ptr(recv), _ptr(send), _ptr(violations_out),
                              _stream(stream)), "bcs_validate")


def bcs_circulant_rounds(p: int, r_begin: int, r_end: int, census: bool, table_out,
                         stream=None) -> None:
    """table_out: CUDA int32 [(r_end-r_begin), q, 4]: rounds of Algorithm 7 (census=False) or
    Algorithm 8 (census=True)."""
    _check(lib().bcs_circulant_rounds(p, r_begin, r_end, int(census), _ptr(table_out),
                                      _stream(stream)), "bcs_circulant_rounds")


def bcs_allgather_tables(p: int, n: int, r: int, recv, send, pack_out, unpack_out,
                         stream=None) -> None:
    """recv/send: full [p][q] CUDA int8 tables; pack_out/unpack_out: CUDA int32 [n-1+q, p]
    (or None): blocks of buffer[j] processor r packs / unpacks per round (Algorithm 9)."""
    _check(lib().bcs_allgather_tables(p, n, r, _ptr(recv), _ptr(send), _ptr(pack_out),
                                      _ptr(unpack_out), _stream(stream)), "bcs_allgather_tables")


def bcs_simulate(p: int, n: int, recv, send, state, counts_out, stream=None) -> None:
    """recv/send: full [p][q] CUDA int8 tables; state: CUDA int64 tensor of 2*p elements (scratch);
    counts_out: CUDA int64 tensor of five elements (see include/bcs.h)."""
    _check(lib().bcs_simulate(p, n, _ptr(recv), _ptr(send), _ptr(state), _ptr(counts_out),
                              _stream(stream)), "bcs_simulate")


def bcs_wait_expired() -> int:
    """CTAs of the transposition kernel that gave up waiting for their copies (0 = none)."""
    v = _c.c_uint64(0)
    _check(lib().bcs_wait_expired(_c.byref(v)), "bcs_wait_expired")
    return v.value


def bcs_checksum(buf, first_entry_index: int, sum_out, stream=None, n_entries: int | None = None) -> None:
    """buf: CUDA int8 tensor; sum_out: CUDA int64 tensor with one element (uint64 bit pattern)."""
    n = buf.numel() if n_entries is None else n_entries
    _check(lib().bcs_checksum(_ptr(buf), n, first_entry_index, _ptr(sum_out), _stream(stream)),
           "bcs_checksum")
