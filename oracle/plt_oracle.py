"""ctypes front end of the fp64 C oracle (``plt_oracle.c``).

TEST INFRASTRUCTURE ONLY: the product package never imports this module.  It takes a
problem object with the attributes of the synthetic-input container (plain numpy arrays
and integers) and returns float64 numpy arrays.  It compiles the C file with gcc on first
use; no CUDA, no torch.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "plt_oracle.c"
_LIB = _HERE / "_build" / "libplt_oracle.so"
_lib = None


class _Problem(ctypes.Structure):
    _fields_ = [
        ("dtype", ctypes.c_int32), ("B", ctypes.c_int32), ("L", ctypes.c_int32), ("Hq", ctypes.c_int32),
        ("Hkv", ctypes.c_int32), ("d", ctypes.c_int32), ("w", ctypes.c_int32), ("page_size", ctypes.c_int32),
        ("max_pages", ctypes.c_int32), ("kv_dtype", ctypes.c_int32),
        ("kv_stride_b", ctypes.c_int64), ("kv_stride_n", ctypes.c_int64), ("kv_stride_h", ctypes.c_int64),
        ("kv_stride_page", ctypes.c_int64), ("sm_scale", ctypes.c_double),
        ("q", ctypes.c_void_p), ("k_cache", ctypes.c_void_p), ("v_cache", ctypes.c_void_p),
        ("seq_lens", ctypes.c_void_p), ("page_table", ctypes.c_void_p), ("k_win", ctypes.c_void_p),
        ("v_win", ctypes.c_void_p), ("win_lens", ctypes.c_void_p), ("gate_logits", ctypes.c_void_p),
        ("loop_offset", ctypes.c_void_p), ("k_scale", ctypes.c_void_p), ("v_scale", ctypes.c_void_p),
    ]


def build(force: bool = False) -> Path:
    """Compile the C oracle into oracle/_build/ (gcc, -O2, OpenMP over output rows only)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        _LIB.parent.mkdir(exist_ok=True)
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.run(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-o", str(tmp), str(_SRC), "-lm"],
                       check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(str(build()))
        _lib.plt_oracle_decode_attn.argtypes = [ctypes.POINTER(_Problem), ctypes.c_void_p]
        _lib.plt_oracle_decode_attn.restype = ctypes.c_int
        _lib.plt_oracle_decode_attn_rows.argtypes = [ctypes.POINTER(_Problem), ctypes.c_void_p, ctypes.c_int64,
                                                     ctypes.c_void_p]
        _lib.plt_oracle_decode_attn_rows.restype = ctypes.c_int
        _lib.plt_oracle_threads.restype = ctypes.c_int
        _lib.plt_oracle_set_threads.argtypes = [ctypes.c_int]
    return _lib


def threads() -> int:
    return int(_load().plt_oracle_threads())


def set_threads(n: int) -> None:
    _load().plt_oracle_set_threads(int(n))


def _marshal(p):
    """Returns (struct, keepalive list). Arrays must be C-contiguous numpy arrays of the stored type."""
    keep = []

    def ptr(a, dt):
        if a is None:
            return None
        a = np.ascontiguousarray(a, dtype=dt)
        keep.append(a)
        return a.ctypes.data

    st = np.uint16 if p.dtype == "bf16" else np.float32
    e4m3 = getattr(p, "kv_dtype", "") == "e4m3"
    kst = np.uint8 if e4m3 else st     # storage type of the caches and windows
    s = _Problem()
    s.dtype = 1 if p.dtype == "bf16" else 0
    s.B, s.L, s.Hq, s.Hkv, s.d, s.w = p.B, p.L, p.Hq, p.Hkv, p.d, p.w
    s.page_size = int(p.page_size)
    s.max_pages = 0 if p.page_table is None else int(p.page_table.shape[1])
    s.kv_dtype = 3 if e4m3 else 0
    kc = np.ascontiguousarray(p.k_cache, dtype=kst)
    # dense [B, N, Hkv, d] or pool [P, page, Hkv, d]
    s.kv_stride_h = p.d
    s.kv_stride_n = p.Hkv * p.d
    s.kv_stride_b = int(kc.shape[1]) * p.Hkv * p.d
    s.kv_stride_page = s.kv_stride_b
    s.sm_scale = float(p.sm_scale) if p.sm_scale > 0 else 1.0 / float(np.sqrt(np.float64(p.d)))
    s.q = ptr(p.q, st)
    s.k_cache = ptr(kc, kst)
    s.v_cache = ptr(p.v_cache, kst)
    s.seq_lens = ptr(p.seq_lens, np.int32)
    s.page_table = ptr(p.page_table, np.int32)
    s.k_win = ptr(p.k_win, kst)
    s.v_win = ptr(p.v_win, kst)
    s.k_scale = ptr(getattr(p, "k_scale", None), np.float32) if e4m3 else None
    s.v_scale = ptr(getattr(p, "v_scale", None), np.float32) if e4m3 else None
    s.win_lens = ptr(p.win_lens, np.int32)
    s.gate_logits = ptr(p.gate_logits, np.float32)
    s.loop_offset = ptr(p.loop_offset, np.int32)
    return s, keep


def decode_attn(p) -> np.ndarray:
    """All outputs O[B, L, Hq, d] in float64."""
    lib = _load()
    s, keep = _marshal(p)
    out = np.empty((p.B, p.L, p.Hq, p.d), dtype=np.float64)
    rc = lib.plt_oracle_decode_attn(ctypes.byref(s), out.ctypes.data)
    if rc != 0:
        raise RuntimeError(f"plt_oracle_decode_attn failed with code {rc}")
    del keep
    return out


def decode_attn_rows(p, rows) -> np.ndarray:
    """Outputs for the listed (b, l0, h) triples (l0 zero-indexed loop): float64 [n, d]."""
    lib = _load()
    s, keep = _marshal(p)
    rows = np.ascontiguousarray(rows, dtype=np.int32).reshape(-1, 3)
    out = np.empty((rows.shape[0], p.d), dtype=np.float64)
    rc = lib.plt_oracle_decode_attn_rows(ctypes.byref(s), rows.ctypes.data, rows.shape[0], out.ctypes.data)
    if rc != 0:
        raise RuntimeError(f"plt_oracle_decode_attn_rows failed with code {rc}")
    del keep
    return out


def decode_attn_multi(p, q, gate_logits, q_len: int) -> np.ndarray:
    """Multi-token decode step: O[B, L, q_len, Hq, d] in float64.

    q: [B, L, q_len, Hq, d] stored values, gate_logits: [B, L-1, q_len, Hq]; p carries the caches, windows (in age
    order, oldest entry in slot 0) and seq_lens AFTER all q_len tokens of the step were appended. The loops are
    displaced by whole tokens (Sec. 2.2.1), so token j (oldest first) of every loop is served exactly as a single-token
    step would have served it q_len-1-j tokens earlier: it sees that many fewer entries of the shared cache and that
    many fewer (the newest) slots of its loop's window. Written as q_len calls of the single-token definition above,
    each on the shortened lengths."""
    from dataclasses import replace
    B, L = p.B, p.L
    delta = list(range(L)) if p.loop_offset is None else [int(x) for x in p.loop_offset]
    out = np.zeros((B, L, q_len, p.Hq, p.d), dtype=np.float64)
    for j in range(q_len):
        newer = q_len - 1 - j
        lens = np.maximum(p.seq_lens.astype(np.int64) - newer, 0).astype(np.int32)
        win = None
        if L > 1:
            win = np.zeros((B, L - 1), dtype=np.int32)
            for b in range(B):
                for l in range(1, L):
                    cut_loop = max(0, int(p.seq_lens[b]) - delta[l])          # keys the loop's newest token sees
                    wl_loop = min(p.w, cut_loop) if p.win_lens is None else int(np.clip(p.win_lens[b, l - 1], 0, p.w))
                    win[b, l - 1] = max(0, wl_loop - newer)
        pj = replace(p, q=np.ascontiguousarray(q[:, :, j]), seq_lens=lens, win_lens=win,
                     gate_logits=np.ascontiguousarray(gate_logits[:, :, j]) if L > 1 else p.gate_logits)
        out[:, :, j] = decode_attn(pj)
    return out
