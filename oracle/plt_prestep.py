"""fp64 / byte-exact CPU oracle of the step that precedes the CLP decode attention (test infrastructure only).

One decode step runs L loops side by side (Algorithm 1: first loop on token i, second loop on token i-1, ...).
Before the two attentions of Algorithm 3 can run, the K and V that its f_qkv produced for this step have
to be where the attention reads them, and its gate needs the logits of f_gate:

  * the first loop's K, V row is appended to the shared cache (the decode step of Algorithm 1 returns the updated cache);
  * every later loop keeps only its w newest K/V entries (Sec. 2.2.2): its row replaces the oldest entry of its
    window, i.e. goes to slot (index of its token in its own stream) mod w;
  * f_gate maps each head's query to a single number for that head (Sec. 2.2.2): logit[h] = <w_gate[h], Q[h]> + b_gate[h].

With the convention of the attention oracle (seq_lens counts the current token, loop l sees
cut_l = max(0, N - delta_l) keys) the token loop l handles in this step has index cut_l - 1 in its stream.
With caches of E4M3 codes (one fp32 scale per KV head) the new rows arrive in the type of the queries and are
quantised on the way in: code = round-to-nearest-even of (x / scale) in float32, clamped to the largest finite
magnitude 448 (the rounding itself is a library cast).
The paper fixes WHICH entries a window keeps, not where they sit: the slot rule and the E4M3 scaling are conventions of
this library (parity unpinned by the paper for them; pinned against the replay over plain token lists, which does not
depend on the slot order, and against the format's facts).
Plain numpy and Python loops, copies of the inputs, nothing shared with the CUDA path.
"""
from __future__ import annotations

from dataclasses import replace

import numpy as np


def _to_f64(a: np.ndarray) -> np.ndarray:
    """Stored values (float32, or bfloat16 bit patterns in uint16) as float64."""
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return a.astype(np.float64)


def quantise_e4m3(x: np.ndarray, scale: np.ndarray) -> np.ndarray:
    """E4M3 codes (uint8) of rows x[..., Hkv, d] (stored values) for per-KV-head scales: float32 division by the
    scale, clamp to [-448, 448], round to nearest even (torch's float32 -> float8_e4m3fn cast)."""
    import torch

    xf = _to_f64(x).astype(np.float32)                       # stored values are exact in float32
    y = xf / scale.astype(np.float32).reshape((1,) * (xf.ndim - 2) + (-1, 1))
    y = np.clip(y, np.float32(-448.0), np.float32(448.0))
    t = torch.from_numpy(np.ascontiguousarray(y)).to(torch.float8_e4m3fn)
    return t.view(torch.uint8).numpy()


def gate_logits(q: np.ndarray, w_gate: np.ndarray, b_gate: np.ndarray) -> np.ndarray:
    """[B, L-1, Hq] float64: the head-wise gate linear f_gate of Algorithm 3 (before the sigmoid) for loops 2..L."""
    qf = _to_f64(q)                                    # [B, L, Hq, d]
    B, L, Hq, d = qf.shape
    out = np.zeros((B, max(L - 1, 0), Hq), dtype=np.float64)
    for b in range(B):
        for l in range(1, L):
            for h in range(Hq):
                acc = 0.0
                for j in range(d):
                    acc += float(w_gate[h, j]) * qf[b, l, h, j]
                out[b, l - 1, h] = acc + float(b_gate[h])
    return out


def prestep(p, k_new: np.ndarray, v_new: np.ndarray, w_gate: np.ndarray, b_gate: np.ndarray):
    """Returns (problem after the step's cache updates with the new gate logits stored as float32, logits in float64).

    p: the synthetic-input container with the caches as they were BEFORE this step and seq_lens already counting the
    current token. k_new, v_new: [B, L, Hkv, d] in the storage type of the queries (row l = what loop l+1 produced).
    """
    if getattr(p, "kv_dtype", "") == "e4m3":               # rows are quantised with the head's scale on the way in
        k_new, v_new = quantise_e4m3(k_new, p.k_scale), quantise_e4m3(v_new, p.v_scale)
    kc, vc = p.k_cache.copy(), p.v_cache.copy()
    kw, vw = p.k_win.copy(), p.v_win.copy()
    # Loop l (1-indexed) serves token i - l + 1 (Sec. 2.2.1, Algorithm 1): it sees cut_l = max(0, N_b - delta_l) keys,
    # delta_l = l - 1 unless the problem carries other offsets.
    delta = np.arange(p.L) if p.loop_offset is None else np.asarray(p.loop_offset, dtype=np.int64)
    cuts = np.zeros((p.B, p.L), dtype=np.int64)
    for b in range(p.B):
        for l in range(p.L):
            cuts[b, l] = max(0, int(p.seq_lens[b]) - int(delta[l]))
    for b in range(p.B):
        c0 = int(cuts[b, 0])
        if c0 > 0:                                     # first loop: append at position c0 - 1 of the shared cache
            pos = c0 - 1
            if p.page_size:
                page = int(p.page_table[b, pos // p.page_size])
                kc[page, pos % p.page_size] = k_new[b, 0]
                vc[page, pos % p.page_size] = v_new[b, 0]
            else:
                kc[b, pos] = k_new[b, 0]
                vc[b, pos] = v_new[b, 0]
        for l in range(1, p.L):                        # later loops: overwrite the oldest window entry
            c = int(cuts[b, l])
            if c > 0:
                slot = (c - 1) % p.w
                kw[b, l - 1, slot] = k_new[b, l]
                vw[b, l - 1, slot] = v_new[b, l]
    g = gate_logits(p.q, w_gate, b_gate)
    g32 = g.astype(np.float32) if p.L > 1 else p.gate_logits
    return replace(p, k_cache=kc, v_cache=vc, k_win=kw, v_win=vw, gate_logits=g32), g
