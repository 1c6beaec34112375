"""CPU oracle for the screen / adjudicate / select path -- TEST INFRASTRUCTURE.

A thin ctypes wrapper over ``kb_oracle.c`` (plain C, binary32 arithmetic, no
fused multiply-add).  Only tests, the smoke check and the CPU-baseline leg of
the benchmark may import this package; the product never does, and this
package never imports the product.

Inputs are numpy arrays: ``float32`` for fp32 tensors and timings, ``uint16``
holding the raw bit patterns for fp16 / bf16 tensors, ``uint8`` for the two
8-bit float formats.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kb_oracle.c")
_LIB = os.path.join(_HERE, "libkb_oracle.so")

F32, F16, BF16, F8E4M3, F8E5M2 = 0, 1, 2, 3, 4
MASK_NONE, MASK_STRIDED, MASK_BITMAP = 0, 1, 2

RESULT_DTYPE = np.dtype(
    [
        ("mismatch_count", "<u8"),
        ("nan_count", "<u8"),
        ("inf_count", "<u8"),
        ("argmax_idx", "<i8"),
        ("max_abs_err", "<f4"),
        ("max_rel_err", "<f4"),
        ("pass", "<u4"),
        ("reserved", "<u4"),
    ]
)
assert RESULT_DTYPE.itemsize == 48

RESULT_F64_DTYPE = np.dtype(
    [
        ("mismatch_count", "<u8"),
        ("nan_count", "<u8"),
        ("inf_count", "<u8"),
        ("argmax_idx", "<i8"),
        ("max_abs_err", "<f8"),
        ("max_rel_err", "<f8"),
        ("pass", "<u4"),
        ("reserved", "<u4"),
    ]
)
assert RESULT_F64_DTYPE.itemsize == 56


class NonFiniteTiming(ValueError):
    """A timing was NaN or +-Inf; the adjudication is undefined."""


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = [
            "gcc", "-O2", "-std=c99", "-ffp-contract=off", "-fno-fast-math",
            "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm",
        ]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        u64, u32, i32, f32 = ctypes.c_uint64, ctypes.c_uint32, ctypes.c_int, ctypes.c_float
        vp = ctypes.c_void_p
        L.kbo_screen.argtypes = [vp, vp, u64, i32, f32, f32, i32, u32, u32, u32, vp, vp]
        L.kbo_screen.restype = i32
        f64 = ctypes.c_double
        L.kbo_screen_f64.argtypes = [vp, vp, u64, f64, f64, i32, u32, u32, u32, vp, vp]
        L.kbo_screen_f64.restype = i32
        L.kbo_quantiles.argtypes = [vp, u32, vp, vp]
        L.kbo_quantiles.restype = i32
        L.kbo_wins_pair.argtypes = [vp, vp, u32]
        L.kbo_wins_pair.restype = u64
        L.kbo_adjudicate.argtypes = [vp, u32, u32, vp, vp, vp]
        L.kbo_adjudicate.restype = i32
        L.kbo_wins_rows.argtypes = [vp, u32, u32, u32, u32, vp]
        L.kbo_wins_rows.restype = i32
        L.kbo_select.argtypes = [vp, vp, u32, i32, u32, vp, vp]
        L.kbo_select.restype = i32
        L.kbo_score.argtypes = [f32, u32, u32, f32, f32]
        L.kbo_score.restype = f32
        L.kbo_select_by_score.argtypes = [vp, vp, u32, u32, u32, f32, f32, u32, vp, vp, vp]
        L.kbo_select_by_score.restype = i32
        L.kbo_tail_ratios.argtypes = [vp, u32, vp]
        L.kbo_tail_ratios.restype = i32
        L.kbo_copeland.argtypes = [vp, u32, u32, vp, vp]
        L.kbo_copeland.restype = i32
        L.kbo_confirm.argtypes = [vp, vp, vp, u32, f32, vp, vp]
        L.kbo_confirm.restype = i32
        L.kbo_adjudicate_ragged.argtypes = [vp, vp, u32, vp, vp, vp]
        L.kbo_adjudicate_ragged.restype = i32
        L.kbo_merge_ranges.argtypes = [vp, u32, u32, vp, vp]
        L.kbo_merge_ranges.restype = i32
        L.kbo_decode_f16.argtypes = [ctypes.c_uint16]
        L.kbo_decode_f16.restype = f32
        L.kbo_decode_bf16.argtypes = [ctypes.c_uint16]
        L.kbo_decode_bf16.restype = f32
        L.kbo_decode_f8e4m3.argtypes = [ctypes.c_uint8]
        L.kbo_decode_f8e4m3.restype = f32
        L.kbo_decode_f8e5m2.argtypes = [ctypes.c_uint8]
        L.kbo_decode_f8e5m2.restype = f32
        _lib = L
    return _lib


def _tensor(a: np.ndarray, dtype: int) -> np.ndarray:
    want = np.float32 if dtype == F32 else (np.uint8 if dtype in (F8E4M3, F8E5M2) else np.uint16)
    a = np.ascontiguousarray(a)
    if a.dtype != want:
        raise TypeError(f"dtype code {dtype} needs a {want.__name__} array, got {a.dtype}")
    return a.reshape(-1)


def _mask_args(mask):
    """mask: None | ("strided", log2_tile, stride, phase) | ("bitmap", log2_tile, uint64 words)."""
    if mask is None:
        return MASK_NONE, 0, 1, 0, None, None
    if mask[0] == "strided":
        _, log2_tile, stride, phase = mask
        return MASK_STRIDED, int(log2_tile), int(stride), int(phase), None, None
    if mask[0] == "bitmap":
        _, log2_tile, words = mask
        words = np.ascontiguousarray(words, dtype=np.uint64)
        return MASK_BITMAP, int(log2_tile), 1, 0, words.ctypes.data, words
    raise ValueError(f"unknown mask {mask!r}")


def screen_one(ref: np.ndarray, cand: np.ndarray, dtype: int, atol: float, rtol: float,
               mask=None) -> np.ndarray:
    """Gate one candidate against the reference; returns one RESULT_DTYPE record."""
    r = _tensor(ref, dtype)
    c = _tensor(cand, dtype)
    if r.size != c.size:
        raise ValueError("reference and candidate differ in size")
    kind, log2_tile, stride, phase, bits_ptr, keep = _mask_args(mask)
    out = np.zeros(1, dtype=RESULT_DTYPE)
    rc = lib().kbo_screen(r.ctypes.data, c.ctypes.data, r.size, dtype,
                          float(np.float32(atol)), float(np.float32(rtol)), kind, log2_tile, stride, phase,
                          bits_ptr, out.ctypes.data)
    del keep
    if rc != 0:
        raise ValueError(f"kbo_screen rejected its arguments (rc={rc})")
    return out[0]


def screen(ref: np.ndarray, cands, dtype: int, atol: float, rtol: float, mask=None,
           threads: int = 1) -> np.ndarray:
    """Gate every candidate in ``cands`` (a sequence of arrays); returns K records."""
    K = len(cands)
    out = np.zeros(K, dtype=RESULT_DTYPE)

    def work(k):
        out[k] = screen_one(ref, cands[k], dtype, atol, rtol, mask)

    if threads <= 1:
        for k in range(K):
            work(k)
    else:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(work, range(K)))
    return out


def screen_f64(ref: np.ndarray, cands, atol: float, rtol: float, mask=None, threads: int = 1) -> np.ndarray:
    """Gate every float64 candidate in ``cands`` in binary64; returns K RESULT_F64_DTYPE records."""
    r = np.ascontiguousarray(ref).reshape(-1)
    if r.dtype != np.float64:
        raise TypeError("the double-precision gate needs float64 arrays")
    K = len(cands)
    out = np.zeros(K, dtype=RESULT_F64_DTYPE)
    kind, log2_tile, stride, phase, bits_ptr, keep = _mask_args(mask)

    def work(k):
        c = np.ascontiguousarray(cands[k]).reshape(-1)
        if c.dtype != np.float64 or c.size != r.size:
            raise TypeError("candidates must be float64 arrays of the reference's size")
        one = np.zeros(1, dtype=RESULT_F64_DTYPE)
        rc = lib().kbo_screen_f64(r.ctypes.data, c.ctypes.data, r.size, float(atol), float(rtol),
                                  kind, log2_tile, stride, phase, bits_ptr, one.ctypes.data)
        if rc != 0:
            raise ValueError(f"kbo_screen_f64 rejected its arguments (rc={rc})")
        out[k] = one[0]

    if threads <= 1:
        for k in range(K):
            work(k)
    else:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(work, range(K)))
    del keep
    return out


def quantiles(row: np.ndarray):
    """(Q1, median, Q3, iqr) of one row, and the sorted row."""
    row = np.ascontiguousarray(row, dtype=np.float32).reshape(-1)
    out4 = np.zeros(4, dtype=np.float32)
    srt = np.zeros(row.size, dtype=np.float32)
    rc = lib().kbo_quantiles(row.ctypes.data, row.size, out4.ctypes.data, srt.ctypes.data)
    if rc == -2:
        raise NonFiniteTiming("non-finite timing")
    if rc != 0:
        raise ValueError(f"kbo_quantiles rejected its arguments (rc={rc})")
    return out4, srt


def wins_pair(a: np.ndarray, b: np.ndarray) -> int:
    a = np.ascontiguousarray(a, dtype=np.float32).reshape(-1)
    b = np.ascontiguousarray(b, dtype=np.float32).reshape(-1)
    if a.size != b.size:
        raise ValueError("rows differ in length")
    return int(lib().kbo_wins_pair(a.ctypes.data, b.ctypes.data, a.size))


def adjudicate(timings: np.ndarray, want_wins: bool = True, threads: int = 1):
    """median[K], iqr[K], wins[K][K] (or None) of timings[K][S]."""
    t = np.ascontiguousarray(timings, dtype=np.float32)
    if t.ndim != 2:
        raise ValueError("timings must be [K][S]")
    K, S = t.shape
    med = np.zeros(K, dtype=np.float32)
    iqr = np.zeros(K, dtype=np.float32)
    rc = lib().kbo_adjudicate(t.ctypes.data, K, S, med.ctypes.data, iqr.ctypes.data, None)
    if rc == -2:
        raise NonFiniteTiming("non-finite timing")
    if rc != 0:
        raise ValueError(f"kbo_adjudicate rejected its arguments (rc={rc})")
    wins = None
    if want_wins:
        wins = np.zeros((K, K), dtype=np.uint32)
        if threads <= 1:
            rc = lib().kbo_adjudicate(t.ctypes.data, K, S, None, None, wins.ctypes.data)
            assert rc == 0
        else:
            step = max(1, (K + 4 * threads - 1) // (4 * threads))

            def work(a0):
                a1 = min(K, a0 + step)
                rc_ = lib().kbo_wins_rows(t.ctypes.data, K, S, a0, a1, wins[a0:a1].ctypes.data)
                assert rc_ == 0

            with ThreadPoolExecutor(max_workers=threads) as ex:
                list(ex.map(work, range(0, K, step)))
    return med, iqr, wins


def wins_rows(timings: np.ndarray, a0: int, a1: int) -> np.ndarray:
    """Rows [a0, a1) of the win matrix."""
    t = np.ascontiguousarray(timings, dtype=np.float32)
    K, S = t.shape
    out = np.zeros((a1 - a0, K), dtype=np.uint32)
    rc = lib().kbo_wins_rows(t.ctypes.data, K, S, a0, a1, out.ctypes.data)
    if rc != 0:
        raise ValueError(f"kbo_wins_rows rejected its arguments (rc={rc})")
    return out


def select(screen_records: np.ndarray, median: np.ndarray, policy: int, budget: int):
    """Survivor indices in rank order (length n) for the next fidelity tier."""
    rec = np.ascontiguousarray(screen_records, dtype=RESULT_DTYPE)
    med = np.ascontiguousarray(median, dtype=np.float32)
    K = rec.size
    surv = np.zeros(budget, dtype=np.int32)
    n = np.zeros(1, dtype=np.uint32)
    rc = lib().kbo_select(rec.ctypes.data, med.ctypes.data, K, policy, budget,
                          surv.ctypes.data, n.ctypes.data)
    if rc != 0:
        raise ValueError(f"kbo_select rejected its arguments (rc={rc})")
    return surv, int(n[0])


def decode_f16(h: int) -> float:
    return float(lib().kbo_decode_f16(int(h)))


def decode_bf16(b: int) -> float:
    return float(lib().kbo_decode_bf16(int(b)))


def score(median_ms: float, rung: int, rung_budget: int, alpha: float, beta: float) -> np.float32:
    """Runtime score S(p, r) of Eq. 2 for one adjudicated latency in milliseconds."""
    return np.float32(lib().kbo_score(float(np.float32(median_ms)), int(rung), int(rung_budget),
                                      float(np.float32(alpha)), float(np.float32(beta))))


def select_by_score(screen_records: np.ndarray, median: np.ndarray, rung: int, rung_budget: int,
                    alpha: float, beta: float, budget: int):
    """(scores[K], survivors[budget], n): promotion by runtime score, ties to the lower index."""
    rec = np.ascontiguousarray(screen_records, dtype=RESULT_DTYPE)
    med = np.ascontiguousarray(median, dtype=np.float32)
    K = rec.size
    sc = np.zeros(K, dtype=np.float32)
    surv = np.zeros(budget, dtype=np.int32)
    n = np.zeros(1, dtype=np.uint32)
    rc = lib().kbo_select_by_score(rec.ctypes.data, med.ctypes.data, K, int(rung), int(rung_budget),
                                   float(np.float32(alpha)), float(np.float32(beta)), int(budget),
                                   sc.ctypes.data, surv.ctypes.data, n.ctypes.data)
    if rc != 0:
        raise ValueError(f"kbo_select_by_score rejected its arguments (rc={rc})")
    return sc, surv, int(n[0])


def tail_ratios(timings: np.ndarray) -> np.ndarray:
    """[K][3] = p90/p50, p95/p50, p99/p50 of each row."""
    t = np.ascontiguousarray(timings, dtype=np.float32)
    if t.ndim == 1:
        t = t[None, :]
    K, S = t.shape
    out = np.zeros((K, 3), dtype=np.float32)
    for k in range(K):
        rc = lib().kbo_tail_ratios(t[k].ctypes.data, S, out[k].ctypes.data)
        if rc == -2:
            raise NonFiniteTiming("non-finite timing")
        if rc != 0:
            raise ValueError(f"kbo_tail_ratios rejected its arguments (rc={rc})")
    return out


def copeland(wins: np.ndarray, S: int):
    """(beats[K], ties[K]) from a win matrix."""
    w = np.ascontiguousarray(wins, dtype=np.uint32)
    K = w.shape[0]
    beats = np.zeros(K, dtype=np.uint32)
    ties = np.zeros(K, dtype=np.uint32)
    rc = lib().kbo_copeland(w.ctypes.data, K, int(S), beats.ctypes.data, ties.ctypes.data)
    if rc != 0:
        raise ValueError(f"kbo_copeland rejected its arguments (rc={rc})")
    return beats, ties


def confirm(s1, s2, prev, threshold: float):
    """(status uint32 [K], score float32 [K]) of the re-measure-and-confirm rule."""
    a = np.ascontiguousarray(s1, dtype=np.float32)
    b = np.ascontiguousarray(s2, dtype=np.float32)
    c = np.ascontiguousarray(prev, dtype=np.float32)
    K = a.size
    st = np.zeros(K, dtype=np.uint32)
    sc = np.zeros(K, dtype=np.float32)
    rc = lib().kbo_confirm(a.ctypes.data, b.ctypes.data, c.ctypes.data, K, float(np.float32(threshold)),
                           st.ctypes.data, sc.ctypes.data)
    if rc != 0:
        raise ValueError(f"kbo_confirm rejected its arguments (rc={rc})")
    return st, sc


def adjudicate_ragged(rows):
    """median[K], iqr[K], wins[K][K] for rows of different lengths (a list of 1-D arrays)."""
    rows = [np.ascontiguousarray(r, dtype=np.float32).reshape(-1) for r in rows]
    K = len(rows)
    off = np.zeros(K + 1, dtype=np.uint32)
    off[1:] = np.cumsum([r.size for r in rows])
    flat = np.concatenate(rows) if K else np.zeros(0, np.float32)
    med = np.zeros(K, dtype=np.float32)
    iqr = np.zeros(K, dtype=np.float32)
    wins = np.zeros((K, K), dtype=np.uint32)
    rc = lib().kbo_adjudicate_ragged(flat.ctypes.data, off.ctypes.data, K, med.ctypes.data,
                                     iqr.ctypes.data, wins.ctypes.data)
    if rc == -2:
        raise NonFiniteTiming("non-finite timing")
    if rc != 0:
        raise ValueError(f"kbo_adjudicate_ragged rejected its arguments (rc={rc})")
    return med, iqr, wins


def merge_ranges(parts, first) -> np.ndarray:
    """Records of a whole element range from the records of R consecutive parts of it:
    ``parts`` is a sequence of R record arrays (K each), ``first`` the global index of each
    part's first element."""
    R = len(parts)
    K = len(parts[0])
    flat = np.ascontiguousarray(np.concatenate([np.asarray(p, dtype=RESULT_DTYPE).reshape(-1) for p in parts]))
    if flat.size != R * K:
        raise ValueError("every part must hold K records")
    first = np.ascontiguousarray(first, dtype=np.uint64)
    out = np.zeros(K, dtype=RESULT_DTYPE)
    rc = lib().kbo_merge_ranges(flat.ctypes.data, R, K, first.ctypes.data, out.ctypes.data)
    if rc != 0:
        raise ValueError(f"kbo_merge_ranges rejected its arguments (rc={rc})")
    return out
