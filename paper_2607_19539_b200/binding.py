"""Thin ctypes binding of the moe_ovl C ABI (include/moe_ovl.h).

Argument marshalling only: every step of the path runs in the CUDA library.
PyTorch is used for device memory and streams.  There is no fallback: if the
library cannot be built or loaded this module raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Dict, Optional

import numpy as np

from . import build as _build

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_CUDA, ERR_WORKSPACE, ERR_TIMEOUT, ERR_BAD_ROUTING = -1, -2, -3, -4, -5, -6
MODE_OVERLAP, MODE_NON_OVERLAP, MODE_IN_KERNEL, MODE_AUTO = 0, 1, 2, 3
FLAG_HOST_STAGING = 1
FLAG_TEST_NO_FLAGS = 2
FLAG_TRACE = 4
FLAG_TEST_SKIP_GATHER = 8
FLAG_NO_SMALL_GROUP_TILES = 16
FLAG_TEST_ALL_SMALL_GROUP_TILES = 32
FLAG_NO_STACKED_BANDS = 64
FLAG_NO_LOCAL_RIDERS = 128
FLAG_TEST_ZERO_ROWS_EARLY = 256
TRACE_ITEM, TRACE_UNIT = 0, 1
BUF_XA, BUF_H, BUF_Y = 0, 1, 2
TB_M, TB_N, H_TILE = 128, 256, 128

EXPORTS = [
    "moe_ovl_workspace_bytes", "moe_ovl_limits", "moe_ovl_create", "moe_ovl_expert_return",
    "moe_ovl_expert_return_host", "moe_ovl_host_join", "moe_ovl_query_status", "moe_ovl_get_report", "moe_ovl_get_plan",
    "moe_ovl_get_sm_map", "moe_ovl_get_gemm_time", "moe_ovl_read_buffer", "moe_ovl_destroy", "moe_ovl_strerror", "moe_ovl_last_cuda_error",
    "moe_ovl_return_slots_static", "moe_ovl_get_trace",
]


class Config(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("device", C.c_int32), ("num_src_ranks", C.c_int32),
                ("self_rank", C.c_int32), ("tokens_per_rank", C.c_int32), ("num_local_experts", C.c_int32),
                ("top_k", C.c_int32), ("d_model", C.c_int32), ("d_ffn", C.c_int32), ("max_rows", C.c_int32),
                ("mid_seg_bands", C.c_int32), ("group_bands", C.c_int32), ("wait_timeout_us", C.c_int32),
                ("producer_sm_limit", C.c_int32), ("single_gemm_out", C.c_int32), ("flags", C.c_uint32)]


class Args(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("num_rows", C.c_int32), ("x", C.c_void_p),
                ("expert_counts", C.c_void_p), ("src_rank", C.c_void_p), ("src_token", C.c_void_p),
                ("gate", C.c_void_p), ("w1", C.c_void_p), ("w2", C.c_void_p), ("consumer_sm_count", C.c_int32),
                ("mode", C.c_int32), ("ret", C.c_void_p), ("ret_rows_per_rank", C.c_int64), ("out", C.c_void_p),
                ("slot_out", C.c_void_p), ("rows_per_rank_out", C.c_void_p), ("segs_per_rank_out", C.c_void_p),
                ("stream", C.c_void_p)]


class HostArgs(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("num_rows", C.c_int32), ("x", C.c_void_p),
                ("expert_counts", C.c_void_p), ("src_rank", C.c_void_p), ("src_token", C.c_void_p),
                ("gate", C.c_void_p), ("w1", C.c_void_p), ("w2", C.c_void_p), ("consumer_sm_count", C.c_int32),
                ("mode", C.c_int32), ("out", C.c_void_p), ("stream", C.c_void_p)]


class Report(C.Structure):
    _fields_ = [("padded_rows", C.c_int32), ("num_bands", C.c_int32), ("num_items", C.c_int32),
                ("num_segments", C.c_int32), ("producer_ctas", C.c_int32), ("consumer_ctas", C.c_int32),
                ("kernel_launches", C.c_int32), ("segments_by_gemm_ctas", C.c_int32), ("return_units", C.c_int32),
                ("mode_used", C.c_int32),
                ("timing_valid", C.c_int32), ("ms_total", C.c_float),
                ("ms_prep", C.c_float), ("ms_expert_return", C.c_float), ("ms_producer", C.c_float),
                ("ms_mover", C.c_float), ("ms_combine", C.c_float), ("us_first_flag", C.c_float),
                ("us_gemm_done", C.c_float), ("us_return_done", C.c_float), ("copy_gbs_per_cta", C.c_float),
                ("overlap_ratio", C.c_float)]


class TraceRecord(C.Structure):
    _fields_ = [("kind", C.c_int32), ("index", C.c_int32), ("cta", C.c_int32), ("who", C.c_int32),
                ("rows", C.c_int32), ("chunks", C.c_int32), ("ns_claim", C.c_int64), ("ns_ready", C.c_int64),
                ("ns_done0", C.c_int64), ("ns_done1", C.c_int64), ("ns_operand_wait", C.c_int64),
                ("ns_epilogue_start", C.c_int64), ("ns_first_operand_wait", C.c_int64),
                ("ns_accumulator_wait", C.c_int64), ("ns_inputs_ready", C.c_int64)]


TRACE_DTYPE = np.dtype([("kind", np.int32), ("index", np.int32), ("cta", np.int32), ("who", np.int32),
                        ("rows", np.int32), ("chunks", np.int32), ("ns_claim", np.int64), ("ns_ready", np.int64),
                        ("ns_done0", np.int64), ("ns_done1", np.int64), ("ns_operand_wait", np.int64),
                        ("ns_epilogue_start", np.int64), ("ns_first_operand_wait", np.int64),
                        ("ns_accumulator_wait", np.int64), ("ns_inputs_ready", np.int64)])


class PlanView(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("group_rows", "pos", "band_expert", "band_dest", "band_valid",
                                          "band_slot0", "sched_band", "item", "seg", "tok_slot", "tok_gate")]


class MoeOvlError(RuntimeError):
    def __init__(self, code: int, what: str, cuda_error: int = 0):
        self.code = code
        self.cuda_error = cuda_error
        msg = f"{what}: {strerror(code)} ({code})"
        if cuda_error:
            msg += f", cudaError={cuda_error}"
        super().__init__(msg)


_lib: Optional[C.CDLL] = None


def library_path() -> str:
    return _build.LIB


def load(rebuild_if_stale: bool = True) -> C.CDLL:
    """Loads the CUDA library (building it with nvcc first when it is missing or stale)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_build.LIB) or (rebuild_if_stale and _build.is_stale()):
        _build.build()
    lib = C.CDLL(_build.LIB)
    for name in EXPORTS:
        getattr(lib, name)      # raises AttributeError if a declared symbol is missing
    lib.moe_ovl_strerror.restype = C.c_char_p
    lib.moe_ovl_strerror.argtypes = [C.c_int]
    lib.moe_ovl_workspace_bytes.argtypes = [C.POINTER(Config), C.POINTER(C.c_size_t)]
    lib.moe_ovl_limits.argtypes = [C.POINTER(Config), C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    lib.moe_ovl_create.argtypes = [C.POINTER(C.c_void_p), C.POINTER(Config), C.c_void_p, C.c_size_t]
    lib.moe_ovl_expert_return.argtypes = [C.c_void_p, C.POINTER(Args)]
    lib.moe_ovl_expert_return_host.argtypes = [C.c_void_p, C.POINTER(HostArgs)]
    lib.moe_ovl_host_join.argtypes = [C.c_void_p, C.c_void_p]
    lib.moe_ovl_query_status.argtypes = [C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_int64)]
    lib.moe_ovl_get_report.argtypes = [C.c_void_p, C.POINTER(Report)]
    lib.moe_ovl_get_plan.argtypes = [C.c_void_p, C.POINTER(PlanView)]
    lib.moe_ovl_get_gemm_time.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_float), C.POINTER(C.c_int32)]
    lib.moe_ovl_get_sm_map.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
    lib.moe_ovl_read_buffer.argtypes = [C.c_void_p, C.c_int32, C.c_size_t, C.c_size_t, C.c_void_p]
    lib.moe_ovl_get_trace.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t, C.POINTER(C.c_size_t)]
    lib.moe_ovl_destroy.argtypes = [C.c_void_p]
    lib.moe_ovl_last_cuda_error.argtypes = [C.c_void_p]
    lib.moe_ovl_return_slots_static.argtypes = [C.c_int32] * 5 + [C.c_void_p] * 6
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load().moe_ovl_strerror(int(code)).decode()


def make_config(*, device: int, num_src_ranks: int, self_rank: int, tokens_per_rank: int, num_local_experts: int,
                top_k: int, d_model: int, d_ffn: int, max_rows: int, mid_seg_bands: int = 1, group_bands: int = 0,
                wait_timeout_us: int = 0, producer_sm_limit: int = 0, single_gemm_out: int = 0,
                flags: int = 0) -> Config:
    return Config(C.sizeof(Config), device, num_src_ranks, self_rank, tokens_per_rank, num_local_experts, top_k,
                  d_model, d_ffn, max_rows, mid_seg_bands, group_bands, wait_timeout_us, producer_sm_limit,
                  single_gemm_out, flags)


def moe_ovl_workspace_bytes(cfg: Config) -> int:
    n = C.c_size_t(0)
    rc = load().moe_ovl_workspace_bytes(C.byref(cfg), C.byref(n))
    if rc != OK:
        raise MoeOvlError(rc, "moe_ovl_workspace_bytes")
    return int(n.value)


def moe_ovl_limits(cfg: Config):
    b, i = C.c_int32(0), C.c_int32(0)
    rc = load().moe_ovl_limits(C.byref(cfg), C.byref(b), C.byref(i))
    if rc != OK:
        raise MoeOvlError(rc, "moe_ovl_limits")
    return int(b.value), int(i.value)


def moe_ovl_return_slots_static(*, device: int, num_src_ranks: int, tokens_per_rank: int, num_local_experts: int,
                                expert_counts, src_rank, src_token, slot_out, rows_per_rank_out=None,
                                stream=None) -> None:
    """Return slots computed with the library's built-in scratch array: for callers that cannot allocate
    device memory (their application owns all of it, or cudaMalloc's synchronisation is unaffordable) and
    have no workspace to give.  Nothing is allocated here either: outputs are the caller's tensors."""
    import torch
    st = torch.cuda.current_stream(device) if stream is None else stream
    rc = load().moe_ovl_return_slots_static(device, num_src_ranks, tokens_per_rank, num_local_experts,
                                            int(src_rank.shape[0]), _ptr(expert_counts), _ptr(src_rank),
                                            _ptr(src_token), _ptr(slot_out), _ptr(rows_per_rank_out), st.cuda_stream)
    if rc != OK:
        raise MoeOvlError(rc, "moe_ovl_return_slots_static")


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return int(t.data_ptr())


@dataclass
class ReportView:
    padded_rows: int
    num_bands: int
    num_items: int
    num_segments: int
    producer_ctas: int
    consumer_ctas: int
    kernel_launches: int
    ms_total: float
    ms_prep: float
    ms_expert_return: float
    ms_producer: float
    ms_mover: float
    ms_combine: float
    segments_by_gemm_ctas: int = 0
    us_first_flag: float = 0.0
    us_gemm_done: float = 0.0
    us_return_done: float = 0.0
    overlap_ratio: float = 0.0
    copy_gbs_per_cta: float = 0.0
    mode_used: int = 0
    timing_valid: int = 1
    return_units: int = 0


class MoeOvl:
    """One context (moe_ovl_create .. moe_ovl_destroy) with a torch-owned workspace."""

    def __init__(self, cfg: Config):
        import torch
        self._torch = torch
        self.lib = load()
        self.cfg = cfg
        self.kmax = min(cfg.top_k, cfg.num_local_experts)
        nbytes = moe_ovl_workspace_bytes(cfg)
        self.max_bands, self.max_items = moe_ovl_limits(cfg)
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=f"cuda:{cfg.device}")
        self.ctx = C.c_void_p(None)
        rc = self.lib.moe_ovl_create(C.byref(self.ctx), C.byref(cfg), self.workspace.data_ptr(), nbytes)
        if rc != OK:
            raise MoeOvlError(rc, "moe_ovl_create")
        self.last_rows = 0

    def _check(self, rc: int, what: str):
        if rc != OK:
            raise MoeOvlError(rc, what, int(self.lib.moe_ovl_last_cuda_error(self.ctx)))

    def moe_ovl_expert_return(self, *, x, expert_counts, src_rank, src_token, gate, w1, w2, ret, out,
                              consumer_sm_count: int = 8, mode: int = MODE_OVERLAP, slot_out=None,
                              rows_per_rank_out=None, segs_per_rank_out=None, num_rows: Optional[int] = None,
                              stream=None) -> None:
        torch = self._torch
        M = int(src_rank.shape[0]) if num_rows is None else int(num_rows)
        st = torch.cuda.current_stream(self.cfg.device) if stream is None else stream
        a = Args(C.sizeof(Args), M, _ptr(x), _ptr(expert_counts), _ptr(src_rank), _ptr(src_token), _ptr(gate),
                 _ptr(w1), _ptr(w2), int(consumer_sm_count), int(mode), _ptr(ret),
                 int(ret.shape[1]) if ret.dim() == 3 else int(ret.shape[0]) // self.cfg.num_src_ranks,
                 _ptr(out), _ptr(slot_out), _ptr(rows_per_rank_out), _ptr(segs_per_rank_out), st.cuda_stream)
        self.last_rows = M
        self._check(self.lib.moe_ovl_expert_return(self.ctx, C.byref(a)), "moe_ovl_expert_return")

    def moe_ovl_expert_return_host(self, *, x, expert_counts, src_rank, src_token, gate, w1, w2, out,
                                   consumer_sm_count: int = 8, mode: int = MODE_OVERLAP, stream=None) -> None:
        torch = self._torch
        M = int(src_rank.shape[0])
        st = torch.cuda.current_stream(self.cfg.device) if stream is None else stream
        h = HostArgs(C.sizeof(HostArgs), M, _ptr(x), _ptr(expert_counts), _ptr(src_rank), _ptr(src_token),
                     _ptr(gate), _ptr(w1), _ptr(w2), int(consumer_sm_count), int(mode), _ptr(out), st.cuda_stream)
        self.last_rows = M
        self._check(self.lib.moe_ovl_expert_return_host(self.ctx, C.byref(h)), "moe_ovl_expert_return_host")

    def moe_ovl_host_join(self, stream=None) -> None:
        st = self._torch.cuda.current_stream(self.cfg.device) if stream is None else stream
        self._check(self.lib.moe_ovl_host_join(self.ctx, st.cuda_stream), "moe_ovl_host_join")

    def moe_ovl_query_status(self):
        code, detail = C.c_int32(0), C.c_int64(0)
        self._check(self.lib.moe_ovl_query_status(self.ctx, C.byref(code), C.byref(detail)), "moe_ovl_query_status")
        return int(code.value), int(detail.value)

    def moe_ovl_get_report(self) -> ReportView:
        r = Report()
        self._check(self.lib.moe_ovl_get_report(self.ctx, C.byref(r)), "moe_ovl_get_report")
        return ReportView(r.padded_rows, r.num_bands, r.num_items, r.num_segments, r.producer_ctas, r.consumer_ctas,
                          r.kernel_launches, r.ms_total, r.ms_prep, r.ms_expert_return, r.ms_producer, r.ms_mover,
                          r.ms_combine, r.segments_by_gemm_ctas, r.us_first_flag, r.us_gemm_done, r.us_return_done,
                          r.overlap_ratio, r.copy_gbs_per_cta, r.mode_used, r.timing_valid, r.return_units)

    def moe_ovl_get_plan(self) -> Dict[str, np.ndarray]:
        rep = self.moe_ovl_get_report()
        G = self.cfg.num_local_experts * self.cfg.num_src_ranks
        ntokk = self.cfg.num_src_ranks * self.cfg.tokens_per_rank * self.kmax
        B, M = rep.num_bands, self.last_rows
        arrs = {
            "group_rows": np.zeros(G, np.int32), "pos": np.zeros(M, np.int32),
            "band_expert": np.zeros(B, np.int32), "band_dest": np.zeros(B, np.int32),
            "band_valid": np.zeros(B, np.int32), "band_slot0": np.zeros(B, np.int32),
            "sched_band": np.zeros(B, np.int32), "item": np.zeros((rep.num_items, 4), np.int32),
            "seg": np.zeros((rep.num_segments, 4), np.int32), "tok_slot": np.zeros(ntokk, np.int32),
            "tok_gate": np.zeros(ntokk, np.float32),
        }
        v = PlanView(*[arrs[n].ctypes.data for n, _ in PlanView._fields_])
        self._check(self.lib.moe_ovl_get_plan(self.ctx, C.byref(v)), "moe_ovl_get_plan")
        arrs["tok_slot"] = arrs["tok_slot"].reshape(-1, self.kmax)
        arrs["tok_gate"] = arrs["tok_gate"].reshape(-1, self.kmax)
        return arrs

    def moe_ovl_get_trace(self) -> np.ndarray:
        """Trace records of the last call as a structured array (fields of moe_ovl_trace_record)."""
        need = C.c_size_t(0)
        self._check(self.lib.moe_ovl_get_trace(self.ctx, None, 0, C.byref(need)), "moe_ovl_get_trace")
        assert need.value % C.sizeof(TraceRecord) == 0 and TRACE_DTYPE.itemsize == C.sizeof(TraceRecord)
        out = np.zeros(need.value // TRACE_DTYPE.itemsize, TRACE_DTYPE)
        if need.value:
            self._check(self.lib.moe_ovl_get_trace(self.ctx, out.ctypes.data, need.value, C.byref(need)),
                        "moe_ovl_get_trace")
        return out

    def moe_ovl_get_gemm_time(self, last_n: int):
        """(mean GEMM kernel duration in ms over the last calls, number of calls averaged)."""
        ms, n = C.c_float(0), C.c_int32(0)
        self._check(self.lib.moe_ovl_get_gemm_time(self.ctx, int(last_n), C.byref(ms), C.byref(n)),
                    "moe_ovl_get_gemm_time")
        return float(ms.value), int(n.value)

    def moe_ovl_get_sm_map(self):
        rep = self.moe_ovl_get_report()
        prod = np.full(max(rep.producer_ctas, 1), -1, np.int32)
        cons = np.full(max(rep.consumer_ctas, 1), -1, np.int32)
        self._check(self.lib.moe_ovl_get_sm_map(self.ctx, prod.ctypes.data, cons.ctypes.data), "moe_ovl_get_sm_map")
        return prod[:rep.producer_ctas], cons[:rep.consumer_ctas]

    def moe_ovl_read_buffer(self, which: int, row0: int, rows: int) -> np.ndarray:
        """Rows [row0, row0+rows) of the aligned input (BUF_XA), hidden (BUF_H) or output (BUF_Y) buffer, bf16 bits."""
        cols = self.cfg.d_model
        if which == BUF_H:
            cols = self.cfg.d_ffn
        elif which == BUF_Y and self.cfg.single_gemm_out:
            cols = self.cfg.single_gemm_out
        out = np.zeros((rows, cols), np.uint16)
        self._check(self.lib.moe_ovl_read_buffer(self.ctx, which, row0 * cols * 2, rows * cols * 2, out.ctypes.data),
                    "moe_ovl_read_buffer")
        return out

    def moe_ovl_destroy(self) -> None:
        if self.ctx:
            self.lib.moe_ovl_destroy(self.ctx)
            self.ctx = C.c_void_p(None)

    def __del__(self):
        try:
            self.moe_ovl_destroy()
        except Exception:
            pass
