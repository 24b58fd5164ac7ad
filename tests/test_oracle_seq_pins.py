"""Pins of the sequence-shaped attention oracle (CPU only): what the paper and the mathematics fix about it.

The oracle is the definition with library matmuls; these tests hold it to things it does not compute itself: the
decode-step oracle on re-arranged tensors (every step of a sequence is a decode step), a library attention routine,
closed forms, the closed cases of the gate, and a brute force written with Python loops.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2510_24824_b200.inputs import bf16_bits_to_f32, make_problem, make_seq_problem


def f64(a):
    return bf16_bits_to_f32(a).astype(np.float64) if a.dtype == np.uint16 else a.astype(np.float64)


def small(**kw):
    base = dict(B=2, L=3, T=24, Hq=4, Hkv=2, d=8, w=5, lens=[24, 9], seed=3)
    base.update(kw)
    return make_seq_problem(**base)


def brute_force(p):
    """Python loops over every (b, l, t, h) and every allowed key; exponentials and sums by hand."""
    delta = list(range(p.L)) if p.loop_offset is None else [int(x) for x in p.loop_offset]
    scale = p.sm_scale if p.sm_scale > 0 else 1.0 / math.sqrt(p.d)
    q, ks, vs, kl, vl = f64(p.q), f64(p.k_share), f64(p.v_share), f64(p.k_loc), f64(p.v_loc)
    G = p.Hq // p.Hkv
    out = np.zeros((p.B, p.L, p.T, p.Hq, p.d))

    def attend(qv, keys, vals):
        sc = [scale * sum(qv[c] * k[c] for c in range(p.d)) for k in keys]
        m = max(sc)
        e = [math.exp(x - m) for x in sc]
        z = sum(e)
        return np.array([sum(e[i] * vals[i][c] for i in range(len(e))) / z for c in range(p.d)])

    for b in range(p.B):
        for l in range(p.L):
            for t in range(int(p.seq_lens[b])):
                cut = max(0, t + 1 - delta[l])
                if cut == 0:
                    continue
                for h in range(p.Hq):
                    kv = h // G
                    yg = attend(q[b, l, t, h], ks[b, :cut, kv], vs[b, :cut, kv])
                    if l == 0:
                        out[b, l, t, h] = yg
                        continue
                    lo = max(delta[l], t + 1 - p.w)
                    yl = attend(q[b, l, t, h], kl[b, l - 1, lo:t + 1, kv], vl[b, l - 1, lo:t + 1, kv])
                    g = 1.0 / (1.0 + math.exp(-float(p.gate_logits[b, l - 1, t, h])))
                    out[b, l, t, h] = g * yl + (1 - g) * yg
    return out


@pytest.mark.parametrize("kw", [dict(), dict(L=1, w=0), dict(L=2, w=1), dict(loop_offset=[0, 0, 0]), dict(loop_offset=[0, 3, 7]),
                                dict(w=40), dict(T=6, lens=[6, 0], B=2)])
def test_bruteforce_tiny(kw):
    p = small(**kw)
    np.testing.assert_allclose(oracle.seq_attn(p), brute_force(p), rtol=1e-12, atol=1e-13)


def decode_problem_at_step(p, t):
    """The decode-step problem of step t: queries of row t, the shared cache up to and including token t, every
    non-first loop's window = its newest min(w, cut) own rows (stored oldest first), seq_lens = t + 1."""
    delta = list(range(p.L)) if p.loop_offset is None else [int(x) for x in p.loop_offset]
    spec = dict(name="step", dtype="bf16", B=p.B, L=p.L, Hq=p.Hq, Hkv=p.Hkv, d=p.d, w=max(p.w, 1), lens=("fixed", t + 1),
                gate_std=1.0, peaks=0.0, page_size=0, seed=0, loop_offset=p.loop_offset)
    dp = make_problem(spec)
    kw, vw = np.zeros_like(dp.k_win), np.zeros_like(dp.v_win)
    for l in range(1, p.L):
        cut = max(0, t + 1 - delta[l])
        wl = min(p.w, cut)
        kw[:, l - 1, :wl] = p.k_loc[:, l - 1, t + 1 - wl:t + 1]
        vw[:, l - 1, :wl] = p.v_loc[:, l - 1, t + 1 - wl:t + 1]
    gate = p.gate_logits[:, :, t] if p.L > 1 else dp.gate_logits
    return dp.with_(q=np.ascontiguousarray(p.q[:, :, t]), k_cache=np.ascontiguousarray(p.k_share[:, :t + 1]),
                    v_cache=np.ascontiguousarray(p.v_share[:, :t + 1]), k_win=kw, v_win=vw,
                    gate_logits=np.ascontiguousarray(gate), max_seq_len=t + 1)


@pytest.mark.parametrize("kw", [dict(), dict(loop_offset=[0, 0, 0]), dict(L=2, w=64, T=40, lens=[40, 40]), dict(loop_offset=[0, 2, 9])])
def test_every_step_is_a_decode_step(kw):
    """Row t of the sequence-shaped result equals the decode-step oracle at step t (cache length t + 1): the last
    position and every one before it."""
    p = small(lens=None, **{k: v for k, v in kw.items() if k != "lens"}) if "lens" not in kw else small(**kw)
    p = p.with_(seq_lens=np.full(p.B, p.T, dtype=np.int32))
    got = oracle.seq_attn(p)
    for t in range(p.T):
        want = oracle.decode_attn(decode_problem_at_step(p, t))      # [B, L, Hq, d]
        np.testing.assert_allclose(got[:, :, t], want, rtol=1e-12, atol=1e-13, err_msg=f"step {t}")


def test_single_loop_is_library_causal_attention():
    p = small(L=1, w=0, B=2, T=33, Hq=6, Hkv=2, d=16, lens=[33, 17])
    got = oracle.seq_attn(p)
    G = p.Hq // p.Hkv
    for b in range(p.B):
        n = int(p.seq_lens[b])
        q = torch.from_numpy(f64(p.q[b, 0, :n])).permute(1, 0, 2)[None]                               # [1, Hq, n, d]
        k = torch.from_numpy(f64(p.k_share[b, :n])).permute(1, 0, 2).repeat_interleave(G, 0)[None]
        v = torch.from_numpy(f64(p.v_share[b, :n])).permute(1, 0, 2).repeat_interleave(G, 0)[None]
        ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True)[0].permute(1, 0, 2).numpy()
        np.testing.assert_allclose(got[b, 0, :n], ref, rtol=1e-12, atol=1e-13)
        assert np.all(got[b, 0, n:] == 0.0)


def test_gate_closed_cases():
    """Gate logit -inf: every loop is causal attention over the shared K/V alone (the "KV share" row of Table 1);
    +inf: non-first loops are pure sliding-window attention over their own K/V."""
    p = small(loop_offset=[0, 0, 0])
    with np.errstate(over="ignore"):
        closed = oracle.seq_attn(p.with_(gate_logits=np.full_like(p.gate_logits, -np.inf)))
        opened = oracle.seq_attn(p.with_(gate_logits=np.full_like(p.gate_logits, np.inf)))
    for l in range(1, p.L):
        as_first = p.with_(L=1, q=np.ascontiguousarray(p.q[:, l:l + 1]))
        np.testing.assert_allclose(closed[:, l], oracle.seq_attn(as_first)[:, 0], rtol=1e-13, atol=1e-14)
    # pure SWA, against a banded mask handed to the library routine
    G = p.Hq // p.Hkv
    for b in range(p.B):
        n = int(p.seq_lens[b])
        t, j = np.arange(n)[:, None], np.arange(n)[None, :]
        band = torch.from_numpy((j <= t) & (j > t - p.w))
        for l in range(1, p.L):
            q = torch.from_numpy(f64(p.q[b, l, :n])).permute(1, 0, 2)[None]
            k = torch.from_numpy(f64(p.k_loc[b, l - 1, :n])).permute(1, 0, 2).repeat_interleave(G, 0)[None]
            v = torch.from_numpy(f64(p.v_loc[b, l - 1, :n])).permute(1, 0, 2).repeat_interleave(G, 0)[None]
            ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, attn_mask=band)[0].permute(1, 0, 2).numpy()
            np.testing.assert_allclose(opened[b, l, :n], ref, rtol=1e-12, atol=1e-13)


def test_window_covering_the_sequence_makes_the_gate_irrelevant():
    """w >= n with the loop's own K/V equal to the shared ones: SWA is full causal attention, so y_local = y_global."""
    p = small(w=64, loop_offset=[0, 0, 0])
    p = p.with_(k_loc=np.stack([p.k_share] * (p.L - 1), axis=1), v_loc=np.stack([p.v_share] * (p.L - 1), axis=1))
    with np.errstate(over="ignore"):
        ref = oracle.seq_attn(p.with_(gate_logits=np.full_like(p.gate_logits, -np.inf)))
    for shift in (-2.0, 0.0, 3.0):
        np.testing.assert_allclose(oracle.seq_attn(p.with_(gate_logits=p.gate_logits + np.float32(shift))), ref,
                                   rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("offsets", [None, [0, 0, 0], [0, 2, 5]])
def test_zero_queries_give_the_mean_of_the_visible_keys(offsets):
    """Q = 0: uniform weights. With V[j] = j the global part is the mean index of the visible keys, (cut - 1) / 2, and
    the local part the mean index of the band [max(delta, t + 1 - w), t]: pins cutoffs, offsets and the band's ends."""
    p = small(B=1, lens=[24], loop_offset=offsets)
    ramp = np.broadcast_to(np.arange(p.T, dtype=np.float32)[None, :, None, None], p.v_share.shape)
    from paper_2510_24824_b200.inputs import f32_to_bf16_bits
    vs = f32_to_bf16_bits(np.ascontiguousarray(ramp))
    vl = np.stack([f32_to_bf16_bits(np.ascontiguousarray(ramp + 100.0))] * (p.L - 1), axis=1)
    delta = list(range(p.L)) if offsets is None else offsets
    for gate, pick in ((-np.inf, "global"), (np.inf, "local")):
        with np.errstate(over="ignore"):
            got = oracle.seq_attn(p.with_(q=np.zeros_like(p.q), v_share=vs, v_loc=vl,
                                          gate_logits=np.full_like(p.gate_logits, gate)))
        for l in range(p.L):
            for t in range(p.T):
                cut = max(0, t + 1 - delta[l])
                if cut == 0:
                    want = 0.0
                elif l == 0 or pick == "global":
                    want = (cut - 1) / 2
                else:
                    lo = max(delta[l], t + 1 - p.w)
                    want = 100.0 + (lo + t) / 2
                np.testing.assert_allclose(got[0, l, t], want, rtol=1e-12, atol=1e-12, err_msg=f"l={l} t={t} {pick}")


def test_rows_beyond_the_length_and_rows_without_a_token_are_zero():
    p = small(lens=[24, 9])
    got = oracle.seq_attn(p)
    assert np.all(got[1, :, 9:] == 0.0)
    assert np.all(got[:, 1, 0] == 0.0) and np.all(got[:, 2, :2] == 0.0)      # delta = (0, 1, 2)
    assert np.abs(got[0, 2, 2]).max() > 0


def test_sampled_planes_match_the_full_result():
    p = small()
    full = oracle.seq_attn(p)
    rows = [(0, 2, 1), (1, 0, 3)]
    part = oracle.seq_attn(p, rows)
    for b, l, h in rows:
        np.testing.assert_array_equal(part[b, l, :, h], full[b, l, :, h])
