"""fp64 CPU oracle of the sequence-shaped PLT attention (test infrastructure only; the product never imports it).

What the decode-step oracle computes for ONE step, for every step of a sequence at once: the attention of a
prefill or training-forward pass (Algorithm 2 "Training for PLT" with the attention of Algorithm 3 in the non-first
loops; the prefill line of Algorithm 1). Row t of loop l (1-indexed l, 0-indexed t) is the query that loop l holds at
decode step t, i.e. the l-th loop of token t - delta_l with delta_l = l - 1 (Sec. 2.2.1 "Inference"); delta = 0 gives
the reading of Algorithm 2, where the shifted hidden states sit at their own positions. Per (b, l, t, h), with
kvh = h // (Hq / Hkv) and n_b the length of sequence b:

    cut      = max(0, t + 1 - delta_l)                       keys of the shared first-loop K/V the row may see
    y_global = softmax(sm_scale * q K_share[0:cut]^T) V_share[0:cut]                       Algorithm 3, global
    y_local  = softmax(sm_scale * q K_l[lo:t+1]^T) V_l[lo:t+1],  lo = max(delta_l, t + 1 - w)  Algorithm 3, SWA
    g        = sigmoid(gate_logit[b, l, t, h])
    O        = g * y_local + (1 - g) * y_global   (l >= 2),   O = y_global   (l = 1)        Eq. 2

K_l, V_l are loop l's own keys and values (row t' = what that loop produced at step t'; rows t' < delta_l do not
exist); the window of a row is the loop's w newest entries including its own (Sec. 2.2.2). Rows with cut = 0 and
rows t >= n_b are zero.

The definition written out: one score matrix per (b, loop, head) by a library matmul, masks, softmax by max / exp /
sum / divide, a second matmul. No tiling, no online rescaling. Inputs are the stored values widened to float64.
"""
from __future__ import annotations

import numpy as np


def _f64(a: np.ndarray) -> np.ndarray:
    if a.dtype == np.uint16:   # bfloat16 bit patterns
        return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return a.astype(np.float64)


def _masked_softmax_times_v(s: np.ndarray, allowed: np.ndarray, v: np.ndarray) -> np.ndarray:
    """softmax over the allowed keys of each row of s [T, T] times v [T, d]; rows without an allowed key give 0."""
    s = np.where(allowed, s, -np.inf)
    m = s.max(axis=1, keepdims=True)
    m = np.where(np.isfinite(m), m, 0.0)
    e = np.exp(s - m)                      # exp(-inf) = 0 for masked keys
    den = e.sum(axis=1, keepdims=True)
    y = e @ v
    return np.where(den > 0, y / np.where(den > 0, den, 1.0), 0.0)


def seq_attn(p, rows=None) -> np.ndarray:
    """O[B, L, T, Hq, d] in float64 for a sequence problem p (attributes: B, L, T, Hq, Hkv, d, w, q [B,L,T,Hq,d],
    k_share / v_share [B,T,Hkv,d], k_loc / v_loc [B,L-1,T,Hkv,d], gate_logits [B,L-1,T,Hq] float32, seq_lens [B],
    loop_offset or None, sm_scale (<= 0: 1/sqrt(d))).

    rows: optional list of (b, l0, h) triples (l0 zero-indexed loop); then only those (sequence, loop, head) planes are
    computed and the rest of the result stays zero (used to sample large problems)."""
    B, L, T, Hq, Hkv, d, w = p.B, p.L, p.T, p.Hq, p.Hkv, p.d, p.w
    G = Hq // Hkv
    scale = float(p.sm_scale) if p.sm_scale > 0 else 1.0 / float(np.sqrt(np.float64(d)))
    delta = list(range(L)) if p.loop_offset is None else [int(x) for x in p.loop_offset]
    out = np.zeros((B, L, T, Hq, d), dtype=np.float64)
    planes = [(b, l, h) for b in range(B) for l in range(L) for h in range(Hq)] if rows is None else [tuple(map(int, r)) for r in rows]
    t_idx = np.arange(T)[:, None]          # query step
    j_idx = np.arange(T)[None, :]          # key index
    for b, l, h in planes:
        n = int(p.seq_lens[b])
        if n <= 0:
            continue
        kvh = h // G
        q = _f64(p.q[b, l, :, h])                                    # [T, d]
        live = t_idx < n
        cut = np.maximum(0, t_idx + 1 - delta[l])                    # [T, 1]
        s = scale * (q @ _f64(p.k_share[b, :, kvh]).T)
        yg = _masked_softmax_times_v(s, live & (j_idx < cut), _f64(p.v_share[b, :, kvh]))
        if l == 0:
            out[b, l, :, h] = yg
            continue
        lo = np.maximum(delta[l], t_idx + 1 - w)
        s = scale * (q @ _f64(p.k_loc[b, l - 1, :, kvh]).T)
        yl = _masked_softmax_times_v(s, live & (cut > 0) & (j_idx >= lo) & (j_idx <= t_idx), _f64(p.v_loc[b, l - 1, :, kvh]))
        g = 1.0 / (1.0 + np.exp(-p.gate_logits[b, l - 1, :, h].astype(np.float64)))[:, None]
        o = g * yl + (1.0 - g) * yg
        # a gate of exactly 0 or 1 (logit -inf / +inf) must not turn an unused 0 * finite into anything else: it is 0
        out[b, l, :, h] = np.where(live & (cut > 0), o, 0.0)
    return out
