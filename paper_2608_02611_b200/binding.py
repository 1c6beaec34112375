"""ctypes binding of the kb C ABI (include/kb.h): argument marshalling only.

Every step of the path runs in the CUDA library; torch is used here for device
memory and the current stream.  There is no CPU fallback: loading fails loudly
when ``libkb.so`` is missing, and the entry points need CUDA tensors.
"""
from __future__ import annotations

import ctypes
import os
import sys
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libkb.so")

KB_OK = 0
STATUS_NAMES = {
    0: "KB_OK", 1: "KB_ERR_INVALID_ARG", 2: "KB_ERR_ALIGNMENT", 3: "KB_ERR_UNSUPPORTED",
    4: "KB_ERR_WORKSPACE", 5: "KB_ERR_CUDA", 6: "KB_ERR_NONFINITE", 7: "KB_ERR_DEVICE_TIMEOUT",
}
KB_F32, KB_F16, KB_BF16, KB_F8E4M3, KB_F8E5M2 = 0, 1, 2, 3, 4
KB_SELECT_ERR_THEN_TIME, KB_SELECT_TIME = 0, 1
KB_TIMER_SCREEN_STREAM, KB_TIMER_WINS = 0, 1
DTYPE_CODE = {torch.float32: KB_F32, torch.float16: KB_F16, torch.bfloat16: KB_BF16,
              torch.float8_e4m3fn: KB_F8E4M3, torch.float8_e5m2: KB_F8E5M2}

# kb_screen_result as a numpy record (48 bytes)
RESULT_DTYPE = np.dtype([
    ("mismatch_count", "<u8"), ("nan_count", "<u8"), ("inf_count", "<u8"), ("argmax_idx", "<i8"),
    ("max_abs_err", "<f4"), ("max_rel_err", "<f4"), ("pass", "<u4"), ("reserved", "<u4"),
])
RESULT_BYTES = 48
# kb_screen_result_f64 (56 bytes)
RESULT_F64_DTYPE = np.dtype([
    ("mismatch_count", "<u8"), ("nan_count", "<u8"), ("inf_count", "<u8"), ("argmax_idx", "<i8"),
    ("max_abs_err", "<f8"), ("max_rel_err", "<f8"), ("pass", "<u4"), ("reserved", "<u4"),
])
RESULT_F64_BYTES = 56

EXPORTS = [
    "kb_ctx_create", "kb_ctx_destroy", "kb_last_error", "kb_ctx_poll", "kb_ctx_set_grid",
    "kb_ctx_enable_timing", "kb_ctx_read_timer", "kb_alu_probe", "kb_ctx_launch_count", "kb_ctx_set_wins_algo", "kb_ctx_set_small_path", "kb_ctx_set_dependent_launch",
    "kb_mask_create_strided", "kb_mask_create_bitmap", "kb_mask_count", "kb_mask_destroy",
    "kb_screen", "kb_screen_f64", "kb_screen_host", "kb_screen_static", "kb_screen_indexed", "kb_screen_multi", "kb_merge_ranges", "kb_adjudicate", "kb_adjudicate_ragged", "kb_select",
    "kb_select_by_score", "kb_tail_ratios", "kb_copeland", "kb_confirm",
    "kb_ctx_fail_next_allocs", "kb_ctx_selftest_wait", "kb_ctx_check_guards", "kb_static_scratch_read", "kb_ctx_set_filter", "kb_ctx_last_filter",
]


class KbError(RuntimeError):
    def __init__(self, status: int, where: str, text: str = ""):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} {text}".strip())


_lib = None


def load() -> ctypes.CDLL:
    """Load libkb.so (built by ``python -m paper_2608_02611_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build the CUDA library first "
            "(python -m paper_2608_02611_b200.build); there is no CPU fallback")
    L = ctypes.CDLL(LIB_PATH)
    vp, u32, u64, i32, f32 = (ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint64, ctypes.c_int,
                              ctypes.c_float)
    pvp = ctypes.POINTER(ctypes.c_void_p)
    L.kb_ctx_create.argtypes = [i32, pvp]
    L.kb_ctx_destroy.argtypes = [vp]
    L.kb_last_error.argtypes = [vp]
    L.kb_last_error.restype = ctypes.c_char_p
    L.kb_ctx_poll.argtypes = [vp, vp, ctypes.POINTER(i32)]
    L.kb_ctx_set_grid.argtypes = [vp, u32]
    L.kb_ctx_enable_timing.argtypes = [vp, i32]
    L.kb_ctx_read_timer.argtypes = [vp, i32, vp, u32, ctypes.POINTER(u32)]
    L.kb_alu_probe.argtypes = [vp, u32, ctypes.POINTER(ctypes.c_double), vp]
    L.kb_ctx_launch_count.argtypes = [vp, ctypes.POINTER(u64)]
    L.kb_ctx_set_wins_algo.argtypes = [vp, i32]
    L.kb_ctx_set_small_path.argtypes = [vp, i32]
    L.kb_ctx_set_dependent_launch.argtypes = [vp, i32]
    L.kb_ctx_set_filter.argtypes = [vp, i32]
    L.kb_ctx_last_filter.argtypes = [vp, ctypes.POINTER(i32)]
    L.kb_ctx_fail_next_allocs.argtypes = [vp, u32, u32]
    L.kb_ctx_check_guards.argtypes = [vp, vp, ctypes.POINTER(u32), ctypes.POINTER(u32)]
    L.kb_static_scratch_read.argtypes = [vp, u32]
    L.kb_ctx_selftest_wait.argtypes = [vp, u64, vp]
    L.kb_mask_create_strided.argtypes = [vp, u64, u32, u32, u32, pvp]
    L.kb_mask_create_bitmap.argtypes = [vp, u64, u32, vp, pvp]
    L.kb_mask_count.argtypes = [vp, ctypes.POINTER(u64)]
    L.kb_mask_destroy.argtypes = [vp]
    L.kb_screen.argtypes = [vp, vp, vp, u32, u64, i32, f32, f32, vp, vp, vp]
    L.kb_screen_f64.argtypes = [vp, vp, vp, u32, u64, ctypes.c_double, ctypes.c_double, vp, vp, vp]
    L.kb_screen_host.argtypes = [vp, vp, vp, u32, u64, i32, f32, f32, vp, vp, vp]
    L.kb_screen_indexed.argtypes = [vp, vp, vp, u32, vp, vp, u32, u64, i32, f32, f32, vp, vp, vp]
    L.kb_screen_multi.argtypes = [vp, u32, vp, vp, vp, vp, i32, f32, f32, vp, vp]
    L.kb_merge_ranges.argtypes = [vp, vp, u32, u32, vp, vp, vp]
    L.kb_screen_static.argtypes = [vp, vp, u32, u64, i32, f32, f32, vp, vp]
    L.kb_adjudicate.argtypes = [vp, vp, u32, u32, vp, vp, vp, vp]
    L.kb_adjudicate_ragged.argtypes = [vp, vp, vp, u32, u32, u64, vp, vp, vp, vp]
    L.kb_select.argtypes = [vp, vp, vp, u32, i32, u32, vp, vp, vp]
    L.kb_select_by_score.argtypes = [vp, vp, vp, u32, u32, u32, f32, f32, u32, vp, vp, vp, vp]
    L.kb_tail_ratios.argtypes = [vp, vp, u32, u32, vp, vp]
    L.kb_copeland.argtypes = [vp, vp, u32, u32, vp, vp, vp]
    L.kb_confirm.argtypes = [vp, vp, vp, vp, u32, f32, vp, vp, vp]
    for name in EXPORTS:
        if name != "kb_last_error":
            getattr(L, name).restype = i32
    _lib = L
    return L


def _stream_ptr(device) -> int:
    return int(torch.cuda.current_stream(device).cuda_stream)


class Mask:
    """A fidelity mask over tiles of 2**log2_tile elements (owned by a Context)."""

    def __init__(self, ctx: "Context", handle: int, spec: tuple):
        self._ctx, self._h, self.spec = ctx, handle, spec

    @property
    def n_selected(self) -> int:
        n = ctypes.c_uint64(0)
        rc = load().kb_mask_count(self._h, ctypes.byref(n))
        if rc != KB_OK:
            raise KbError(rc, "kb_mask_count")
        return int(n.value)

    def close(self):
        if self._h:
            load().kb_mask_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            if not sys.is_finalizing():
                self.close()
        except Exception:
            pass


class Candidates:
    """K candidate tensors checked once, with their device pointers already laid out as the
    ``const void* const*`` array the screening calls take.  Building the array costs about
    0.4 us per tensor in Python, which at K = 1024 is longer than the kernels run; a caller
    that screens the same tensors again (another tolerance, another tier's mask) passes this
    object instead of the list.  Holds references to the tensors so the pointers stay valid."""

    def __init__(self, tensors: Sequence[torch.Tensor]):
        self.tensors = list(tensors)
        K = len(self.tensors)
        first = self.tensors[0] if K else None
        self.dtype = first.dtype if K else None
        self.numel = first.numel() if K else 0
        self.device = first.device if K else None
        for c in self.tensors:
            if (c.dtype != self.dtype or c.numel() != self.numel or not c.is_cuda
                    or not c.is_contiguous() or c.device != self.device):
                raise KbError(1, "Candidates", "candidates must be contiguous CUDA tensors of one "
                                               "dtype, element count and device")
        self.ptrs = (ctypes.c_void_p * max(K, 1))(*[c.data_ptr() for c in self.tensors])

    def __len__(self) -> int:
        return len(self.tensors)


def _marshal_cands(cands, ref: torch.Tensor, where: str):
    """(K, pointer array) of a list of tensors or of a Candidates object, checked against ref."""
    if isinstance(cands, Candidates):
        if len(cands) and (cands.dtype != ref.dtype or cands.numel != ref.numel()
                           or cands.device != ref.device):
            raise KbError(1, where, "candidates must have the reference's dtype, element count "
                                    "and device")
        return len(cands), cands.ptrs
    N = ref.numel()
    for c in cands:
        if c.dtype != ref.dtype or c.numel() != N or not c.is_cuda or not c.is_contiguous():
            raise KbError(1, where, "candidates must be contiguous CUDA tensors with the "
                                    "reference's dtype and element count")
    K = len(cands)
    return K, (ctypes.c_void_p * max(K, 1))(*[c.data_ptr() for c in cands])


class Context:
    """kb_ctx bound to one CUDA device."""

    def __init__(self, device: int = 0):
        L = load()
        h = ctypes.c_void_p()
        rc = L.kb_ctx_create(int(device), ctypes.byref(h))
        if rc != KB_OK:
            raise KbError(rc, "kb_ctx_create", (L.kb_last_error(None) or b"").decode())
        self._h = h.value
        self.device = torch.device("cuda", int(device))

    # -- plumbing -----------------------------------------------------------
    def _check(self, rc: int, where: str):
        if rc != KB_OK:
            raise KbError(rc, where, (load().kb_last_error(self._h) or b"").decode())

    def close(self):
        if getattr(self, "_h", None):
            load().kb_ctx_destroy(self._h)
            self._h = None

    def __del__(self):
        # never call into CUDA while the interpreter is shutting down (the runtime may be
        # half torn down by then); the process is about to release everything anyway
        try:
            if not sys.is_finalizing():
                self.close()
        except Exception:
            pass

    def poll(self) -> int:
        """Synchronise the current stream and return (and clear) the device status."""
        st = ctypes.c_int(0)
        self._check(load().kb_ctx_poll(self._h, _stream_ptr(self.device), ctypes.byref(st)),
                    "kb_ctx_poll")
        return int(st.value)

    def set_grid(self, blocks: int):
        self._check(load().kb_ctx_set_grid(self._h, int(blocks)), "kb_ctx_set_grid")

    def set_small_path(self, on: bool):
        """Enable/disable the single-launch kernel for small problems (a test hook)."""
        self._check(load().kb_ctx_set_small_path(self._h, 1 if on else 0), "kb_ctx_set_small_path")

    def set_dependent_launch(self, on: bool):
        """Launch the streaming kernel as a programmatic dependent of the lead kernel (default)
        or in plain stream order (a test hook)."""
        self._check(load().kb_ctx_set_dependent_launch(self._h, 1 if on else 0), "kb_ctx_set_dependent_launch")

    def set_filter(self, mode: int):
        """0 automatic, 1 always the plain streaming kernel, 2 always the sharp one, 3 always the
        one that tests by the definition beyond the lean bound (a tuning hook)."""
        self._check(load().kb_ctx_set_filter(self._h, int(mode)), "kb_ctx_set_filter")

    @property
    def last_filter_sharp(self) -> bool:
        """Whether the last streaming launch used another instantiation than the plain one."""
        return self.last_filter_mode != 0

    @property
    def last_filter_mode(self) -> int:
        """Instantiation of the last streaming launch: 0 plain, 1 sharp, 3 by definition."""
        v = ctypes.c_int(0)
        self._check(load().kb_ctx_last_filter(self._h, ctypes.byref(v)), "kb_ctx_last_filter")
        return int(v.value)

    def set_wins_algo(self, algo: int):
        """0 automatic, 1 direct comparison of all sample pairs, 2 binary search on sorted rows,
        3 lane-per-row merge of sorted rows."""
        self._check(load().kb_ctx_set_wins_algo(self._h, int(algo)), "kb_ctx_set_wins_algo")

    def fail_next_allocs(self, n: int, skip: int = 0):
        """Test hook: after `skip` more device allocations of this context, the next n fail."""
        self._check(load().kb_ctx_fail_next_allocs(self._h, int(skip), int(n)), "kb_ctx_fail_next_allocs")

    def check_guards(self):
        """Test hook: (buffers checked, guard-band bytes overwritten) over the context's buffers."""
        nb, bad = ctypes.c_uint32(0), ctypes.c_uint32(0)
        self._check(load().kb_ctx_check_guards(self._h, _stream_ptr(self.device), ctypes.byref(nb),
                                               ctypes.byref(bad)), "kb_ctx_check_guards")
        return int(nb.value), int(bad.value)

    def selftest_wait(self, limit_ns: int):
        """Test hook: one warp waits `limit_ns` on a barrier nothing completes, then gives up;
        poll() afterwards reports KB_ERR_DEVICE_TIMEOUT once."""
        self._check(load().kb_ctx_selftest_wait(self._h, int(limit_ns), _stream_ptr(self.device)),
                    "kb_ctx_selftest_wait")

    def enable_timing(self, on: bool = True, keep: bool = False):
        """Event pairs around the instrumented kernels: on starts a new record (or, with
        ``keep``, goes on with the one there is); off stops recording and keeps the record."""
        self._check(load().kb_ctx_enable_timing(self._h, (2 if keep else 1) if on else 0), "kb_ctx_enable_timing")

    def read_timer(self, which: int, cap: int = 256) -> np.ndarray:
        """Durations (ms) of the instrumented kernel's launches since the last read."""
        buf = np.zeros(cap, dtype=np.float32)
        n = ctypes.c_uint32(0)
        self._check(load().kb_ctx_read_timer(self._h, int(which), buf.ctypes.data, cap,
                                             ctypes.byref(n)), "kb_ctx_read_timer")
        return buf[: n.value].copy()

    @property
    def launch_count(self) -> int:
        n = ctypes.c_uint64(0)
        self._check(load().kb_ctx_launch_count(self._h, ctypes.byref(n)), "kb_ctx_launch_count")
        return int(n.value)

    def alu_probe(self, iters: int = 20000) -> float:
        """kb_alu_probe: measured sample pairs per second of the direct win count's inner loop."""
        v = ctypes.c_double(0.0)
        self._check(load().kb_alu_probe(self._h, iters, ctypes.byref(v), _stream_ptr(self.device)),
                    "kb_alu_probe")
        return float(v.value)

    # -- masks --------------------------------------------------------------
    def mask_strided(self, N: int, log2_tile: int, stride: int, phase: int) -> Mask:
        h = ctypes.c_void_p()
        self._check(load().kb_mask_create_strided(self._h, N, log2_tile, stride, phase,
                                                  ctypes.byref(h)), "kb_mask_create_strided")
        return Mask(self, h.value, ("strided", log2_tile, stride, phase))

    def mask_bitmap(self, N: int, log2_tile: int, words: np.ndarray) -> Mask:
        words = np.ascontiguousarray(words, dtype=np.uint64)
        h = ctypes.c_void_p()
        self._check(load().kb_mask_create_bitmap(self._h, N, log2_tile, words.ctypes.data,
                                                 ctypes.byref(h)), "kb_mask_create_bitmap")
        return Mask(self, h.value, ("bitmap", log2_tile, words.copy()))

    # -- the three calls ----------------------------------------------------
    def screen(self, ref: torch.Tensor, cands: Sequence[torch.Tensor], atol: float, rtol: float,
               mask: Optional[Mask] = None, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """kb_screen.  ``cands`` is a sequence of tensors or a ``Candidates`` object.  Returns a
        uint8 CUDA tensor [K, 48] of kb_screen_result records (see ``records``); asynchronous on
        the current stream."""
        N = ref.numel()
        code = DTYPE_CODE.get(ref.dtype, -1)
        if not ref.is_cuda or not ref.is_contiguous():
            raise KbError(1, "kb_screen", "reference must be a contiguous CUDA tensor")
        K, ptrs = _marshal_cands(cands, ref, "kb_screen")
        if out is None:
            out = torch.empty((K, RESULT_BYTES), dtype=torch.uint8, device=ref.device)
        rc = load().kb_screen(self._h, ref.data_ptr(), ptrs, K, N, code, float(atol), float(rtol),
                              mask._h if mask is not None else None, out.data_ptr(),
                              _stream_ptr(ref.device))
        self._check(rc, "kb_screen")
        return out

    def screen_f64(self, ref: torch.Tensor, cands: Sequence[torch.Tensor], atol: float, rtol: float,
                   mask: Optional[Mask] = None, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """kb_screen_f64 on float64 CUDA tensors.  Returns a uint8 CUDA tensor [K, 56] of
        kb_screen_result_f64 records (see ``records_f64``); asynchronous on the current stream."""
        K = len(cands)
        N = ref.numel()
        for c in list(cands) + [ref]:
            if c.dtype != torch.float64 or c.numel() != N or not c.is_cuda or not c.is_contiguous():
                raise KbError(1, "kb_screen_f64", "tensors must be contiguous CUDA float64 tensors of "
                                                  "one element count")
        if out is None:
            out = torch.empty((K, RESULT_F64_BYTES), dtype=torch.uint8, device=ref.device)
        ptrs = (ctypes.c_void_p * max(K, 1))(*[c.data_ptr() for c in cands])
        rc = load().kb_screen_f64(self._h, ref.data_ptr(), ptrs, K, N, float(atol), float(rtol),
                                  mask._h if mask is not None else None, out.data_ptr(),
                                  _stream_ptr(ref.device))
        self._check(rc, "kb_screen_f64")
        return out

    def screen_host(self, ref: torch.Tensor, cands: Sequence[torch.Tensor], atol: float,
                    rtol: float, mask: Optional[Mask] = None) -> np.ndarray:
        """kb_screen_host: all tensors in host memory; returns K records (synchronous)."""
        K = len(cands)
        N = ref.numel()
        code = DTYPE_CODE.get(ref.dtype, -1)
        for c in list(cands) + [ref]:
            if c.is_cuda or not c.is_contiguous() or c.dtype != ref.dtype or c.numel() != N:
                raise KbError(1, "kb_screen_host", "tensors must be contiguous host tensors of one "
                                                   "dtype and element count")
        out = np.zeros(K, dtype=RESULT_DTYPE)
        ptrs = (ctypes.c_void_p * max(K, 1))(*[c.data_ptr() for c in cands])
        rc = load().kb_screen_host(self._h, ref.data_ptr(), ptrs, K, N, code, float(atol),
                                   float(rtol), mask._h if mask is not None else None,
                                   out.ctypes.data, _stream_ptr(self.device))
        self._check(rc, "kb_screen_host")
        return out

    def adjudicate(self, timings: torch.Tensor, want_wins: bool = True, out=None):
        """kb_adjudicate on a CUDA float32 tensor [K, S] -> (median[K], iqr[K], wins[K,K] or None).
        wins is int32 storage holding uint32 counts (values < 2^31 for S < 32768).
        `out` = (median, iqr, wins) gives pre-allocated outputs."""
        if timings.dtype != torch.float32 or timings.dim() != 2 or not timings.is_cuda \
                or not timings.is_contiguous():
            raise KbError(1, "kb_adjudicate", "timings must be a contiguous CUDA float32 [K, S] tensor")
        K, S = timings.shape
        if out is not None:
            med, iqr, wins = out
        else:
            med = torch.empty(K, dtype=torch.float32, device=timings.device)
            iqr = torch.empty(K, dtype=torch.float32, device=timings.device)
            wins = torch.empty((K, K), dtype=torch.int32, device=timings.device) if want_wins else None
        rc = load().kb_adjudicate(self._h, timings.data_ptr(), K, S, med.data_ptr(), iqr.data_ptr(),
                                  wins.data_ptr() if want_wins else None,
                                  _stream_ptr(timings.device))
        self._check(rc, "kb_adjudicate")
        return med, iqr, wins

    def select(self, screen_out: torch.Tensor, median: torch.Tensor, policy: int, budget: int, out=None):
        """kb_select -> (survivors int32 [budget] in rank order, n int32 [1]) on the device.
        `out` = (survivors, n) gives pre-allocated outputs."""
        K = median.numel()
        if out is not None:
            surv, n = out
        else:
            surv = torch.empty(budget, dtype=torch.int32, device=median.device)
            n = torch.empty(1, dtype=torch.int32, device=median.device)
        rc = load().kb_select(self._h, screen_out.data_ptr(), median.data_ptr(), K, int(policy),
                              int(budget), surv.data_ptr(), n.data_ptr(), _stream_ptr(median.device))
        self._check(rc, "kb_select")
        return surv, n


KB_STATIC_MAX_K = 1024


def screen_static(ref: torch.Tensor, cands: Sequence[torch.Tensor], atol: float, rtol: float,
                  out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """kb_screen_static: the gate for hosts that forbid allocation by third parties.

    Needs no Context and makes the library allocate nothing; its scratch is a fixed array
    inside the library (at most KB_STATIC_MAX_K candidates, no mask).  Pass ``out`` (a uint8
    CUDA tensor [K, 48]) to keep torch from allocating as well.  Calls share the array: do
    not let two of them overlap on the GPU.  Works on the current device and stream.
    """
    K = len(cands)
    N = ref.numel()
    code = DTYPE_CODE.get(ref.dtype, -1)
    if out is None:
        out = torch.empty((K, RESULT_BYTES), dtype=torch.uint8, device=ref.device)
    ptrs = (ctypes.c_void_p * max(K, 1))(*[c.data_ptr() for c in cands])
    with torch.cuda.device(ref.device):
        rc = load().kb_screen_static(ref.data_ptr(), ptrs, K, N, code, float(atol), float(rtol),
                                     out.data_ptr(), _stream_ptr(ref.device))
    if rc != KB_OK:
        raise KbError(rc, "kb_screen_static", (load().kb_last_error(None) or b"").decode())
    return out


KB_STATIC_SCRATCH_BYTES = 256 + 2 * 1024 * 48 + 1024 * 8


def static_scratch_read(nbytes: int = KB_STATIC_SCRATCH_BYTES) -> np.ndarray:
    """Test hook: the scratch array of kb_screen_static on the current device, as bytes."""
    buf = np.zeros(nbytes, dtype=np.uint8)
    rc = load().kb_static_scratch_read(buf.ctypes.data, nbytes)
    if rc != KB_OK:
        raise KbError(rc, "kb_static_scratch_read")
    return buf


def _ctx_method(fn):
    setattr(Context, fn.__name__, fn)
    return fn


@_ctx_method
def select_by_score(self, screen_out: torch.Tensor, median: torch.Tensor, rung: int, rung_budget: int,
                    alpha: float, beta: float, budget: int):
    """kb_select_by_score -> (score float32 [K], survivors int32 [budget], n int32 [1])."""
    K = median.numel()
    score = torch.empty(K, dtype=torch.float32, device=median.device)
    surv = torch.empty(budget, dtype=torch.int32, device=median.device)
    n = torch.empty(1, dtype=torch.int32, device=median.device)
    rc = load().kb_select_by_score(self._h, screen_out.data_ptr(), median.data_ptr(), K, int(rung),
                                   int(rung_budget), float(alpha), float(beta), int(budget),
                                   score.data_ptr(), surv.data_ptr(), n.data_ptr(),
                                   _stream_ptr(median.device))
    self._check(rc, "kb_select_by_score")
    return score, surv, n


@_ctx_method
def tail_ratios(self, timings: torch.Tensor) -> torch.Tensor:
    """kb_tail_ratios -> float32 [K, 3] = p90/p50, p95/p50, p99/p50."""
    K, S = timings.shape
    out = torch.empty((K, 3), dtype=torch.float32, device=timings.device)
    rc = load().kb_tail_ratios(self._h, timings.data_ptr(), K, S, out.data_ptr(),
                               _stream_ptr(timings.device))
    self._check(rc, "kb_tail_ratios")
    return out


@_ctx_method
def copeland(self, wins: torch.Tensor, S: int):
    """kb_copeland -> (beats int32 [K], ties int32 [K])."""
    K = wins.shape[0]
    beats = torch.empty(K, dtype=torch.int32, device=wins.device)
    ties = torch.empty(K, dtype=torch.int32, device=wins.device)
    rc = load().kb_copeland(self._h, wins.data_ptr(), K, int(S), beats.data_ptr(), ties.data_ptr(),
                            _stream_ptr(wins.device))
    self._check(rc, "kb_copeland")
    return beats, ties


@_ctx_method
def pointer_table(self, cands: Sequence[torch.Tensor]) -> torch.Tensor:
    """A device array holding the candidates' addresses (for screen_indexed)."""
    return torch.tensor([c.data_ptr() for c in cands], dtype=torch.int64, device=self.device)


@_ctx_method
def screen_indexed(self, ref: torch.Tensor, table: torch.Tensor, index: torch.Tensor,
                   count: torch.Tensor, atol: float, rtol: float, mask=None,
                   out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """kb_screen_indexed: slot j is candidate table[index[j]] for j < count; everything stays
    on the device (no host synchronisation).  Returns a uint8 CUDA tensor [len(index), 48]."""
    Kmax = index.numel()
    if out is None:
        out = torch.empty((Kmax, RESULT_BYTES), dtype=torch.uint8, device=ref.device)
    rc = load().kb_screen_indexed(self._h, ref.data_ptr(), table.data_ptr(), table.numel(),
                                  index.data_ptr(), count.data_ptr(), Kmax, ref.numel(),
                                  DTYPE_CODE.get(ref.dtype, -1), float(atol), float(rtol),
                                  mask._h if mask is not None else None, out.data_ptr(),
                                  _stream_ptr(ref.device))
    self._check(rc, "kb_screen_indexed")
    return out


@_ctx_method
def adjudicate_ragged(self, flat: torch.Tensor, offsets: torch.Tensor, S_max: int):
    """kb_adjudicate_ragged: flat float32 timings, int32 offsets [K+1] (both CUDA) ->
    (median[K], iqr[K], wins[K,K])."""
    K = offsets.numel() - 1
    med = torch.empty(K, dtype=torch.float32, device=flat.device)
    iqr = torch.empty(K, dtype=torch.float32, device=flat.device)
    wins = torch.empty((K, K), dtype=torch.int32, device=flat.device)
    rc = load().kb_adjudicate_ragged(self._h, flat.data_ptr(), offsets.data_ptr(), K, int(S_max),
                                     flat.numel(), med.data_ptr(), iqr.data_ptr(), wins.data_ptr(),
                                     _stream_ptr(flat.device))
    self._check(rc, "kb_adjudicate_ragged")
    return med, iqr, wins


@_ctx_method
def screen_multi(self, groups, atol: float, rtol: float, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """kb_screen_multi: groups = [(ref, [cands...]), ...] of different sizes, one launch.
    Returns a uint8 CUDA tensor [sum K, 48] in group order."""
    G = len(groups)
    refs = (ctypes.c_void_p * G)(*[r.data_ptr() for r, _ in groups])
    Ks = (ctypes.c_uint32 * G)(*[len(c) for _, c in groups])
    Ns = (ctypes.c_uint64 * G)(*[r.numel() for r, _ in groups])
    flat = [c for _, cs in groups for c in cs]
    for r, cs in groups:
        for c in cs:
            if c.dtype != groups[0][0].dtype or c.numel() != r.numel() or not c.is_contiguous():
                raise KbError(1, "kb_screen_multi", "every tensor of a group must have the group's size "
                                                    "and the call's dtype")
    ptrs = (ctypes.c_void_p * max(len(flat), 1))(*[c.data_ptr() for c in flat])
    dev = groups[0][0].device
    if out is None:
        out = torch.empty((len(flat), RESULT_BYTES), dtype=torch.uint8, device=dev)
    rc = load().kb_screen_multi(self._h, G, refs, ptrs, Ks, Ns, DTYPE_CODE.get(groups[0][0].dtype, -1),
                                float(atol), float(rtol), out.data_ptr(), _stream_ptr(dev))
    self._check(rc, "kb_screen_multi")
    return out


@_ctx_method
def merge_ranges(self, parts: torch.Tensor, first, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """kb_merge_ranges: ``parts`` is a uint8 CUDA tensor [R, K, 48] of the records of R
    consecutive parts of an element range, ``first`` the global index of each part's first
    element.  Returns the [K, 48] records of the whole range."""
    R, K = int(parts.shape[0]), int(parts.shape[1])
    if parts.dtype != torch.uint8 or parts.dim() != 3 or parts.shape[2] != RESULT_BYTES or not parts.is_contiguous():
        raise KbError(1, "kb_merge_ranges", "parts must be a contiguous uint8 tensor [R, K, 48]")
    firsts = (ctypes.c_uint64 * max(R, 1))(*[int(x) for x in first])
    if len(first) != R:
        raise KbError(1, "kb_merge_ranges", "one first index per part")
    if out is None:
        out = torch.empty((K, RESULT_BYTES), dtype=torch.uint8, device=parts.device)
    rc = load().kb_merge_ranges(self._h, parts.data_ptr(), R, K, firsts, out.data_ptr(), _stream_ptr(parts.device))
    self._check(rc, "kb_merge_ranges")
    return out


@_ctx_method
def confirm(self, first: torch.Tensor, second: torch.Tensor, prev: torch.Tensor, threshold: float):
    """kb_confirm -> (status int32 [K], score float32 [K])."""
    K = first.numel()
    status = torch.empty(K, dtype=torch.int32, device=first.device)
    score = torch.empty(K, dtype=torch.float32, device=first.device)
    rc = load().kb_confirm(self._h, first.data_ptr(), second.data_ptr(), prev.data_ptr(), K,
                           float(threshold), status.data_ptr(), score.data_ptr(),
                           _stream_ptr(first.device))
    self._check(rc, "kb_confirm")
    return status, score


def records_f64(screen_out: torch.Tensor) -> np.ndarray:
    """Copy a [K, 56] uint8 result tensor of kb_screen_f64 to the host as K numpy records."""
    return screen_out.cpu().numpy().view(RESULT_F64_DTYPE).reshape(-1)


def records(screen_out: torch.Tensor) -> np.ndarray:
    """Copy a [K, 48] uint8 result tensor to the host as K numpy records (synchronises)."""
    return screen_out.cpu().numpy().view(RESULT_DTYPE).reshape(-1)
