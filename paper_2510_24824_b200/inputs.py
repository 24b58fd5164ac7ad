"""Seeded synthetic inputs for the CLP decode-attention path.

This module only draws random numbers, lays them out and converts storage
types.  It contains none of the attention arithmetic and is the one piece of
code that both the tests' CPU oracle and the CUDA binding are fed from.
The two length helpers of the container (``cuts``, ``window_lengths``) serve the
byte model (``algorithmic_bytes``) and the generator's tail fill only: neither the
kernels nor the oracle nor the oracle's pins take their cutoffs from here.

Recipe: numpy ``default_rng(seed)``, draw order fixed: ``Q, lens, page permutation,
Kwin, Vwin, gate``; the shared cache of sequence ``b`` comes from its own stream
``default_rng([seed, 2, b])`` (K, then V, then the positions of its sharp peaks), and the
peak positions of the windows from ``default_rng([seed, 1])``.
All values are drawn in float32 and, for bf16 problems, rounded to bfloat16
(round-to-nearest-even) and kept as uint16 bit patterns, so that every consumer
sees exactly the same stored values.
"""
from __future__ import annotations

import math
import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field, replace
from typing import Optional

import numpy as np

__all__ = [
    "ClpProblem",
    "WORKLOADS",
    "workload",
    "shrunk_workload",
    "make_problem",
    "f32_to_bf16_bits",
    "bf16_bits_to_f32",
    "algorithmic_bytes",
    "SeqProblem",
    "make_seq_problem",
    "seq_attn_flops",
]


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round-to-nearest-even. Finite inputs only."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (((u >> 16) & 1) + np.uint32(0x7FFF))
    return (rounded >> 16).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32)


@dataclass
class ClpProblem:
    """One decode step's inputs, host side. Arrays are float32, or uint16 bf16 bit patterns."""

    name: str
    dtype: str  # "f32" | "bf16"
    B: int
    L: int
    Hq: int
    Hkv: int
    d: int
    w: int
    max_seq_len: int  # capacity of the shared cache per sequence
    page_size: int  # 0 = contiguous [B, max_seq_len, Hkv, d]; else pool [P, page_size, Hkv, d]
    q: np.ndarray  # [B, L, Hq, d]
    k_cache: np.ndarray
    v_cache: np.ndarray
    seq_lens: np.ndarray  # [B] int32, current token included
    k_win: np.ndarray  # [B, max(L-1,1), w, Hkv, d]
    v_win: np.ndarray
    gate_logits: np.ndarray  # [B, max(L-1,1), Hq] float32, pre-sigmoid
    page_table: Optional[np.ndarray] = None  # [B, max_pages] int32
    win_lens: Optional[np.ndarray] = None  # [B, L-1] int32 or None (= min(w, cut))
    loop_offset: Optional[np.ndarray] = None  # [L] int32 or None (= l-1)
    sm_scale: float = 0.0  # <= 0: 1/sqrt(d)
    kv_dtype: str = ""  # "": caches and windows stored like q; "e4m3": uint8 E4M3 codes with per-KV-head scales
    k_scale: Optional[np.ndarray] = None  # [Hkv] float32 (e4m3 only): value = code value * scale
    v_scale: Optional[np.ndarray] = None
    meta: dict = field(default_factory=dict)

    @property
    def elem_size(self) -> int:
        return 2 if self.dtype == "bf16" else 4

    @property
    def kv_elem_size(self) -> int:
        return 1 if self.kv_dtype == "e4m3" else self.elem_size

    @property
    def max_pages(self) -> int:
        return 0 if self.page_table is None else int(self.page_table.shape[1])

    @property
    def num_pool_pages(self) -> int:
        return int(self.k_cache.shape[0]) if self.page_size else 0

    def scale(self) -> float:
        return self.sm_scale if self.sm_scale > 0 else 1.0 / math.sqrt(self.d)

    def offsets(self) -> np.ndarray:
        if self.loop_offset is not None:
            return np.asarray(self.loop_offset, dtype=np.int64)
        return np.arange(self.L, dtype=np.int64)

    def cuts(self) -> np.ndarray:
        """[B, L] number of shared-cache keys each loop's query may see."""
        return np.maximum(0, self.seq_lens.astype(np.int64)[:, None] - self.offsets()[None, :])

    def window_lengths(self) -> np.ndarray:
        """[B, L-1] valid window slots per non-first loop."""
        if self.L == 1:
            return np.zeros((self.B, 0), dtype=np.int64)
        if self.win_lens is not None:
            return np.clip(self.win_lens.astype(np.int64), 0, self.w)
        return np.minimum(self.w, self.cuts()[:, 1:])

    def with_(self, **kw) -> "ClpProblem":
        return replace(self, **kw)


def algorithmic_bytes(p: ClpProblem) -> dict:
    """Bytes one decode step must move, each tensor counted once (no partials, padding or re-reads)."""
    s = p.elem_size
    row = p.Hkv * p.d * 2 * p.kv_elem_size  # K and V of one token, all KV heads
    shared = int(np.max(p.cuts(), axis=1).sum()) * row if p.B else 0
    window = int(p.window_lengths().sum()) * row
    qo = 2 * p.B * p.L * p.Hq * p.d * s
    gates = 4 * p.B * (p.L - 1) * p.Hq
    index = 4 * p.B + (4 * int(np.ceil(p.seq_lens / p.page_size).sum()) if p.page_size else 0)
    return {
        "shared_kv": shared,
        "window_kv": window,
        "q_o": qo,
        "gates": gates,
        "index": index,
        "total": shared + window + qo + gates + index,
    }


# The five workloads (index 0..4 = config 1..5). "lens": ("fixed", N) | ("uniform", lo, hi)
# | ("loguniform", lo, hi, overrides). Seeds: config index.
WORKLOADS = [
    dict(name="tiny_fp32", dtype="f32", B=1, L=2, Hq=4, Hkv=1, d=64, w=16, lens=("fixed", 256),
         gate_std=1.0, peaks=0.0, page_size=0, seed=0),
    dict(name="bf16_decode_batch", dtype="bf16", B=64, L=2, Hq=32, Hkv=8, d=128, w=64, lens=("fixed", 4096),
         gate_std=1.0, peaks=0.0, page_size=0, seed=1),
    dict(name="bf16_deeper_loops", dtype="bf16", B=128, L=3, Hq=32, Hkv=8, d=128, w=128,
         lens=("uniform", 1024, 8192), gate_std=1.0, peaks=0.01, page_size=0, seed=2),
    dict(name="bf16_long_context", dtype="bf16", B=16, L=4, Hq=64, Hkv=8, d=128, w=512, lens=("fixed", 32768),
         gate_std=2.0, peaks=0.0, page_size=0, seed=3),
    dict(name="bf16_paged_serving_mix", dtype="bf16", B=256, L=3, Hq=32, Hkv=4, d=128, w=256,
         lens=("loguniform", 128, 16384, (1, 2, 3, 63, 64, 255)), gate_std=1.0, peaks=0.0, page_size=64, seed=4),
]


def workload(index: int) -> dict:
    return dict(WORKLOADS[index])


def shrunk_workload(index: int, **override) -> dict:
    """Same structure as WORKLOADS[index], sized so the CPU oracle finishes in seconds."""
    spec = workload(index)
    small = {
        0: {},
        1: dict(B=3, lens=("fixed", 600)),
        2: dict(B=5, lens=("uniform", 100, 900)),
        3: dict(B=2, lens=("fixed", 2100), w=160),
        4: dict(B=12, lens=("loguniform", 20, 1500, (1, 2, 3, 63, 64, 255))),
    }[index]
    spec.update(small)
    spec.update(override)
    spec["name"] = spec["name"] + "_small"
    return spec


def _draw_lens(rng: np.random.Generator, spec, B: int) -> np.ndarray:
    kind = spec[0]
    if kind == "fixed":
        return np.full(B, spec[1], dtype=np.int32)
    if kind == "uniform":
        return rng.integers(spec[1], spec[2] + 1, size=B).astype(np.int32)
    if kind == "loguniform":
        lens = np.rint(np.exp(rng.uniform(math.log(spec[1]), math.log(spec[2]), size=B))).astype(np.int32)
        for i, n in enumerate(spec[3][:B]):
            lens[i] = n
        return lens
    if kind == "list":
        return np.asarray(spec[1], dtype=np.int32)
    raise ValueError(f"unknown length recipe {kind}")


def _store(x: np.ndarray, dtype: str) -> np.ndarray:
    return f32_to_bf16_bits(x) if dtype == "bf16" else np.ascontiguousarray(x, dtype=np.float32)


def make_problem(spec: dict, seed: Optional[int] = None, tail_fill: Optional[float] = None) -> ClpProblem:
    """Materialise a workload.

    tail_fill: value written to cache rows at or beyond N_b and window slots at or
    beyond wl (default 0). Tests pass NaN here to show that nothing outside the
    valid ranges can reach the output.
    """
    spec = dict(spec)
    seed = spec.get("seed", 0) if seed is None else seed
    rng = np.random.default_rng(seed)
    dtype, B, L, Hq, Hkv, d, w = (spec[k] for k in ("dtype", "B", "L", "Hq", "Hkv", "d", "w"))
    page = int(spec.get("page_size", 0))
    peaks = float(spec.get("peaks", 0.0))
    Lm = max(L - 1, 1)
    st = np.uint16 if dtype == "bf16" else np.float32
    fill = _store(np.full(1, 0.0 if tail_fill is None else tail_fill, dtype=np.float32), dtype)[0]
    if dtype == "bf16" and tail_fill is not None and math.isnan(tail_fill):
        fill = np.uint16(0x7FC0)

    q = _store(rng.standard_normal((B, L, Hq, d), dtype=np.float32), dtype)
    lens = _draw_lens(rng, spec["lens"], B)
    cap = int(spec.get("max_seq_len", max(int(lens.max()) if B else 1, 1)))
    if page:
        cap = -(-cap // page) * page

    # Shared first-loop cache, filled per sequence so that peak memory stays near the final size.
    rng_peaks = np.random.default_rng([seed, 1])  # second stream: positions of the sharp peaks
    page_table = None
    if page:
        pages_per_seq = -(-lens.astype(np.int64) // page)
        P = int(pages_per_seq.sum()) + int(spec.get("spare_pages", 3))
        perm = rng.permutation(P).astype(np.int32)
        page_table = np.zeros((B, cap // page), dtype=np.int32)
        shape = (P, page, Hkv, d)
    else:
        shape = (B, cap, Hkv, d)
    if fill == 0:
        k_cache, v_cache = np.zeros(shape, dtype=st), np.zeros(shape, dtype=st)
    else:
        k_cache, v_cache = np.full(shape, fill, dtype=st), np.full(shape, fill, dtype=st)
    starts = np.concatenate([[0], np.cumsum(pages_per_seq)]) if page else None

    def fill_sequence(b: int) -> None:
        # Sequence b draws from its own stream (seed, 2, b), so sequences can be generated concurrently.
        n = int(lens[b])
        rb = np.random.default_rng([seed, 2, b])
        kb = rb.standard_normal((n, Hkv, d), dtype=np.float32)
        vb = rb.standard_normal((n, Hkv, d), dtype=np.float32)
        if peaks:
            # Sharp softmax peaks: a Bernoulli(peaks) set of token positions has its K and V rows (all heads) tripled.
            hot = rb.random(n) < peaks
            kb[hot] *= 3.0
            vb[hot] *= 3.0
        kb, vb = _store(kb, dtype), _store(vb, dtype)
        if page:
            ids = perm[int(starts[b]):int(starts[b + 1])]
            page_table[b, :len(ids)] = ids
            for i, pid in enumerate(ids):
                lo, hi = i * page, min((i + 1) * page, n)
                k_cache[pid, : hi - lo] = kb[lo:hi]
                v_cache[pid, : hi - lo] = vb[lo:hi]
        else:
            k_cache[b, :n] = kb
            v_cache[b, :n] = vb

    workers = min(B, os.cpu_count() or 1, 16)
    if workers > 1:
        with ThreadPoolExecutor(max_workers=workers) as ex:
            list(ex.map(fill_sequence, range(B)))
    else:
        for b in range(B):
            fill_sequence(b)

    k_win_f = rng.standard_normal((B, Lm, w, Hkv, d), dtype=np.float32)
    v_win_f = rng.standard_normal((B, Lm, w, Hkv, d), dtype=np.float32)
    gate = (rng.standard_normal((B, Lm, Hq), dtype=np.float32) * np.float32(spec.get("gate_std", 1.0))).astype(np.float32)
    if peaks:
        hotw = rng_peaks.random((B, Lm, w)) < peaks
        k_win_f[hotw] *= 3.0
        v_win_f[hotw] *= 3.0

    prob = ClpProblem(
        name=spec["name"], dtype=dtype, B=B, L=L, Hq=Hq, Hkv=Hkv, d=d, w=w, max_seq_len=cap, page_size=page,
        q=q, k_cache=k_cache, v_cache=v_cache, seq_lens=lens,
        k_win=_store(k_win_f, dtype), v_win=_store(v_win_f, dtype), gate_logits=gate, page_table=page_table,
        loop_offset=None if spec.get("loop_offset") is None else np.asarray(spec["loop_offset"], dtype=np.int32),
        sm_scale=float(spec.get("sm_scale", 0.0)), meta={"seed": seed, "spec": spec},
    )
    if tail_fill is not None and L > 1:
        wl = prob.window_lengths()
        for b in range(B):
            for l in range(L - 1):
                prob.k_win[b, l, int(wl[b, l]):] = fill
                prob.v_win[b, l, int(wl[b, l]):] = fill
    if spec.get("kv_dtype") == "e4m3":
        prob = quantize_kv_e4m3(prob)
    return prob


def quantize_kv_e4m3(p: ClpProblem) -> ClpProblem:
    """The same problem with the shared cache and the windows stored as E4M3 codes (uint8) and one scale per KV head
    for K and one for V (largest magnitude of that head over cache and windows / 448). Input preparation only: the
    rounding is torch's float32 -> float8_e4m3fn cast (round to nearest even)."""
    import torch

    def f32(a):
        return bf16_bits_to_f32(a) if a.dtype == np.uint16 else a.astype(np.float32, copy=False)

    def amax(a, b):  # per KV head (axis -2) over everything else, NaN-free inputs
        m = np.zeros(p.Hkv, dtype=np.float32)
        for x in (a, b):
            for i in range(x.shape[0]):     # chunked over the leading axis to bound the float32 temporaries
                v = np.abs(f32(x[i])).reshape(-1, p.Hkv, p.d)
                if v.size:
                    m = np.maximum(m, v.max(axis=(0, 2)))
        return m

    def codes(a, scale):
        out = np.empty(a.shape, dtype=np.uint8)
        inv = (1.0 / scale).astype(np.float32).reshape(1, p.Hkv, 1)
        for i in range(a.shape[0]):
            x = torch.from_numpy(np.ascontiguousarray(f32(a[i]).reshape(-1, p.Hkv, p.d) * inv))
            x = torch.clamp(x, -448.0, 448.0)
            out[i] = x.to(torch.float8_e4m3fn).view(torch.uint8).numpy().reshape(a[i].shape)
        return out

    k_scale = np.maximum(amax(p.k_cache, p.k_win), 1e-12).astype(np.float32) / np.float32(448.0)
    v_scale = np.maximum(amax(p.v_cache, p.v_win), 1e-12).astype(np.float32) / np.float32(448.0)
    return replace(p, kv_dtype="e4m3", k_scale=k_scale.astype(np.float32), v_scale=v_scale.astype(np.float32),
                   k_cache=codes(p.k_cache, k_scale), v_cache=codes(p.v_cache, v_scale),
                   k_win=codes(p.k_win, k_scale), v_win=codes(p.v_win, v_scale))


# ---- sequence-shaped problems (prefill / training-forward attention) --------------------------------------------
@dataclass
class SeqProblem:
    """Inputs of the sequence-shaped PLT attention, host side: every decode step of a sequence at once. Arrays hold
    bf16 bit patterns (uint16); T is the padded length, seq_lens the true ones."""

    name: str
    B: int
    L: int
    T: int
    Hq: int
    Hkv: int
    d: int
    w: int
    q: np.ndarray            # [B, L, T, Hq, d]
    k_share: np.ndarray      # [B, T, Hkv, d]  first-loop keys (shared by every loop)
    v_share: np.ndarray
    k_loc: np.ndarray        # [B, max(L-1,1), T, Hkv, d]  own keys of loops 2..L
    v_loc: np.ndarray
    gate_logits: np.ndarray  # [B, max(L-1,1), T, Hq] float32, pre-sigmoid
    seq_lens: np.ndarray     # [B] int32
    loop_offset: Optional[np.ndarray] = None
    sm_scale: float = 0.0
    dtype: str = "bf16"

    def with_(self, **kw) -> "SeqProblem":
        return replace(self, **kw)


def make_seq_problem(B: int, L: int, T: int, Hq: int, Hkv: int, d: int, w: int, lens=None, seed: int = 0,
                     gate_std: float = 1.0, loop_offset=None, name: str = "seq", sm_scale: float = 0.0) -> SeqProblem:
    """Seeded N(0,1) values rounded to bf16; draw order q, k_share, v_share, k_loc, v_loc, gate. The shapes follow the
    paper's serving recipe (prefill 5000, batch 4-64, GQA 32/8, d = 128, w = 64, L in {2, 3})."""
    rng = np.random.default_rng([seed, 7])
    Lm = max(L - 1, 1)
    draw = lambda *shape: f32_to_bf16_bits(rng.standard_normal(shape, dtype=np.float32))
    q = draw(B, L, T, Hq, d)
    k_share, v_share = draw(B, T, Hkv, d), draw(B, T, Hkv, d)
    k_loc, v_loc = draw(B, Lm, T, Hkv, d), draw(B, Lm, T, Hkv, d)
    gate = (rng.standard_normal((B, Lm, T, Hq), dtype=np.float32) * np.float32(gate_std)).astype(np.float32)
    seq_lens = np.full(B, T, dtype=np.int32) if lens is None else np.asarray(lens, dtype=np.int32)
    assert seq_lens.shape == (B,) and int(seq_lens.max(initial=0)) <= T
    return SeqProblem(name=name, B=B, L=L, T=T, Hq=Hq, Hkv=Hkv, d=d, w=w, q=q, k_share=k_share, v_share=v_share,
                      k_loc=k_loc, v_loc=v_loc, gate_logits=gate, seq_lens=seq_lens,
                      loop_offset=None if loop_offset is None else np.asarray(loop_offset, dtype=np.int32),
                      sm_scale=sm_scale)


def seq_attn_flops(p: SeqProblem) -> int:
    """Multiply-adds x 2 of the two products over the key sets the definition names (masked-out keys not counted)."""
    delta = np.arange(p.L) if p.loop_offset is None else np.asarray(p.loop_offset, dtype=np.int64)
    total = 0
    for n in p.seq_lens.astype(np.int64):
        t = np.arange(int(n), dtype=np.int64)
        for l in range(p.L):
            cut = np.maximum(0, t + 1 - delta[l])
            keys = int(cut.sum())
            if l > 0:
                keys += int(np.where(cut > 0, np.minimum(cut, p.w), 0).sum())
            total += keys * p.Hq * p.d * 4
    return int(total)
