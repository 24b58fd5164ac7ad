"""Pins of the multi-token decode step of the oracle (q_len query tokens per loop in one step; CPU only).

The loops are displaced by whole tokens (Sec. 2.2.1), so the tokens of one step differ only in how far back their
causal cutoff lies. Two things hold the definition: the sequence-shaped oracle (independent numpy code), whose rows
N - q_len .. N - 1 are exactly these tokens as long as no window has evicted anything, and a brute force with explicit
slices for the case of full windows.
"""
import math

import numpy as np
import pytest

import oracle
from paper_2510_24824_b200.inputs import bf16_bits_to_f32, make_problem, make_seq_problem


def f64(a):
    return bf16_bits_to_f32(a).astype(np.float64) if a.dtype == np.uint16 else a.astype(np.float64)


def decode_problem_from_sequence(sp, q_len, w_cap):
    """The decode-step problem after all N tokens of a sequence problem: shared cache = its shared K/V, every non-first
    loop's window = its newest min(w_cap, cut) own rows, oldest first; plus the queries and gates of the last q_len rows."""
    N = sp.T
    delta = list(range(sp.L)) if sp.loop_offset is None else [int(x) for x in sp.loop_offset]
    spec = dict(name="mt", dtype="bf16", B=sp.B, L=sp.L, Hq=sp.Hq, Hkv=sp.Hkv, d=sp.d, w=w_cap, lens=("fixed", N),
                gate_std=1.0, peaks=0.0, page_size=0, seed=0, loop_offset=sp.loop_offset)
    p = make_problem(spec)
    kw, vw = np.zeros_like(p.k_win), np.zeros_like(p.v_win)
    for l in range(1, sp.L):
        wl = min(w_cap, max(0, N - delta[l]))
        kw[:, l - 1, :wl] = sp.k_loc[:, l - 1, N - wl:N]
        vw[:, l - 1, :wl] = sp.v_loc[:, l - 1, N - wl:N]
    p = p.with_(k_cache=sp.k_share.copy(), v_cache=sp.v_share.copy(), k_win=kw, v_win=vw, max_seq_len=N)
    q = np.ascontiguousarray(sp.q[:, :, N - q_len:N])                        # [B, L, q_len, Hq, d]
    gate = np.ascontiguousarray(sp.gate_logits[:, :, N - q_len:N])           # [B, L-1, q_len, Hq]
    return p, q, gate


@pytest.mark.parametrize("offsets", [None, [0, 0, 0], [0, 2, 5]])
@pytest.mark.parametrize("q_len", [1, 2, 4])
def test_tokens_of_a_step_are_rows_of_the_sequence_shaped_attention(q_len, offsets):
    """With windows that have evicted nothing (capacity >= N), token j of the step is row N - q_len + j of the sequence."""
    sp = make_seq_problem(B=2, L=3, T=21, Hq=4, Hkv=2, d=8, w=64, seed=11, loop_offset=offsets)
    p, q, gate = decode_problem_from_sequence(sp, q_len, w_cap=32)
    got = oracle.decode_attn_multi(p, q, gate, q_len)
    want = oracle.seq_attn(sp)[:, :, sp.T - q_len:sp.T]
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)


def test_full_windows_lose_their_newest_slots_per_older_token():
    """Capacity 5 < N: token j sees the first cut - (q_len-1-j) shared keys and the first wl - (q_len-1-j) window slots;
    softmaxes and the gate mix written out by hand."""
    q_len, w_cap = 3, 5
    sp = make_seq_problem(B=1, L=2, T=17, Hq=2, Hkv=1, d=4, w=64, seed=4)
    p, q, gate = decode_problem_from_sequence(sp, q_len, w_cap)
    got = oracle.decode_attn_multi(p, q, gate, q_len)
    K, V, Kw, Vw, Q = f64(p.k_cache), f64(p.v_cache), f64(p.k_win), f64(p.v_win), f64(q)
    scale = 1.0 / math.sqrt(p.d)

    def attend(qv, keys, vals):
        e = np.exp(scale * (keys @ qv) - np.max(scale * (keys @ qv)))
        return (e / e.sum()) @ vals

    for l in range(p.L):
        for j in range(q_len):
            newer = q_len - 1 - j
            cut = 17 - l - newer
            for h in range(p.Hq):
                yg = attend(Q[0, l, j, h], K[0, :cut, 0], V[0, :cut, 0])
                if l == 0:
                    want = yg
                else:
                    wl = min(w_cap, 17 - l) - newer
                    yl = attend(Q[0, l, j, h], Kw[0, l - 1, :wl, 0], Vw[0, l - 1, :wl, 0])
                    g = 1.0 / (1.0 + math.exp(-float(gate[0, l - 1, j, h])))
                    want = g * yl + (1 - g) * yg
                np.testing.assert_allclose(got[0, l, j, h], want, rtol=1e-12, atol=1e-13)


def test_one_token_per_loop_is_the_plain_step():
    sp = make_seq_problem(B=2, L=2, T=9, Hq=2, Hkv=1, d=4, w=64, seed=6)
    p, q, gate = decode_problem_from_sequence(sp, 1, w_cap=4)
    plain = oracle.decode_attn(p.with_(q=np.ascontiguousarray(q[:, :, 0]), gate_logits=np.ascontiguousarray(gate[:, :, 0])))
    np.testing.assert_array_equal(oracle.decode_attn_multi(p, q, gate, 1)[:, :, 0], plain)
