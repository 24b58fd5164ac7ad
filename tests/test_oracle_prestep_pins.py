"""CPU-only pins of the pre-step oracle (cache append, window ring, head-wise gate linear).

The decisive pin replays a whole decode of a tiny model-free stream: T steps of pre-step + attention must equal,
at every step, attention computed directly from the lists of everything each loop has produced so far
(all first-loop K/V rows, and the w newest K/V rows of the loop itself, Sec. 2.2.2), with no cache and no ring at all.
"""
import math

import numpy as np
import pytest

import oracle
from paper_2510_24824_b200.inputs import ClpProblem, bf16_bits_to_f32, f32_to_bf16_bits, make_problem


def empty_problem(B, L, Hq, Hkv, d, w, cap, dtype="f32", page_size=0, seed=0):
    rng = np.random.default_rng(seed)
    st = np.uint16 if dtype == "bf16" else np.float32
    junk = (lambda shape: f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))) if dtype == "bf16" else \
           (lambda shape: rng.standard_normal(shape).astype(np.float32))
    table = None
    if page_size:
        pages = B * (cap // page_size)
        kc, vc = junk((pages, page_size, Hkv, d)), junk((pages, page_size, Hkv, d))
        table = rng.permutation(pages).astype(np.int32).reshape(B, cap // page_size)
    else:
        kc, vc = junk((B, cap, Hkv, d)), junk((B, cap, Hkv, d))
    return ClpProblem(name="stream", dtype=dtype, B=B, L=L, Hq=Hq, Hkv=Hkv, d=d, w=w, max_seq_len=cap, page_size=page_size,
                      q=np.zeros((B, L, Hq, d), dtype=st), k_cache=kc, v_cache=vc, seq_lens=np.zeros(B, dtype=np.int32),
                      k_win=junk((B, max(L - 1, 1), w, Hkv, d)), v_win=junk((B, max(L - 1, 1), w, Hkv, d)),
                      gate_logits=np.zeros((B, max(L - 1, 1), Hq), dtype=np.float32), page_table=table)


def f64(a):
    return (bf16_bits_to_f32(a) if a.dtype == np.uint16 else a).astype(np.float64)


def softmax_attend(q, K, V, scale):
    e = np.exp((K @ q) * scale)
    return (e / e.sum()) @ V


@pytest.mark.parametrize("dtype,page_size", [("f32", 0), ("bf16", 0), ("f32", 4)])
def test_replayed_decode_equals_attention_over_plain_token_lists(dtype, page_size):
    B, L, Hq, Hkv, d, w, T = 2, 3, 4, 2, 4, 3, 9
    rng = np.random.default_rng(5)
    p = empty_problem(B, L, Hq, Hkv, d, w, cap=12, dtype=dtype, page_size=page_size)
    store = (lambda x: f32_to_bf16_bits(x.astype(np.float32))) if dtype == "bf16" else (lambda x: x.astype(np.float32))
    w_gate, b_gate = rng.standard_normal((Hq, d)), rng.standard_normal(Hq)
    hist_k = [[[] for _ in range(L)] for _ in range(B)]   # per sequence and loop: every K row produced so far
    hist_v = [[[] for _ in range(L)] for _ in range(B)]
    G = Hq // Hkv
    for step in range(T):
        q = store(rng.standard_normal((B, L, Hq, d)))
        k_new, v_new = store(rng.standard_normal((B, L, Hkv, d))), store(rng.standard_normal((B, L, Hkv, d)))
        p = p.with_(q=q, seq_lens=np.full(B, step + 1, dtype=np.int32))
        p, logits = oracle.prestep(p, k_new, v_new, w_gate, b_gate)
        got = oracle.decode_attn(p)
        for b in range(B):
            for l in range(L):
                if step - l < 0:                       # loop l+1 has no token yet (Algorithm 1: it lags l tokens)
                    assert np.all(got[b, l] == 0.0)
                    continue
                hist_k[b][l].append(f64(k_new[b, l]))
                hist_v[b][l].append(f64(v_new[b, l]))
                for h in range(Hq):
                    kv, qv = h // G, f64(q[b, l, h])
                    # shared cache: the first loop's rows of tokens 0 .. step - l
                    Ks = np.array([r[kv] for r in hist_k[b][0][:step - l + 1]])
                    Vs = np.array([r[kv] for r in hist_v[b][0][:step - l + 1]])
                    yg = softmax_attend(qv, Ks, Vs, p.scale())
                    if l == 0:
                        want = yg
                    else:
                        Kl = np.array([r[kv] for r in hist_k[b][l][-w:]])   # the w newest rows of this loop
                        Vl = np.array([r[kv] for r in hist_v[b][l][-w:]])
                        yl = softmax_attend(qv, Kl, Vl, p.scale())
                        x = float(np.float32(float(np.dot(w_gate[h], qv)) + b_gate[h]))
                        g = 1.0 / (1.0 + math.exp(-x))
                        want = g * yl + (1 - g) * yg
                    np.testing.assert_allclose(got[b, l, h], want, rtol=1e-9, atol=1e-11)


def test_ring_slot_holds_the_token_with_that_residue():
    """After n tokens of a loop, slot s holds the newest token whose index is s mod w, older ones are gone."""
    B, L, Hq, Hkv, d, w = 1, 2, 1, 1, 2, 4
    p = empty_problem(B, L, Hq, Hkv, d, w, cap=16)
    for step in range(11):
        k_new = np.full((B, L, Hkv, d), 0.0, dtype=np.float32)
        k_new[0, 1] = 100.0 + (step - 1)               # second loop handles token step - 1; tag the row with its index
        p = p.with_(seq_lens=np.array([step + 1], dtype=np.int32))
        p, _ = oracle.prestep(p, k_new, k_new.copy(), np.zeros((Hq, d)), np.zeros(Hq))
        n = step                                       # tokens the second loop has seen (its stream lags one token)
        for s in range(w):
            if n > s:
                newest = max(i for i in range(n) if i % w == s)
                assert p.k_win[0, 0, s, 0, 0] == 100.0 + newest


def test_loops_without_a_token_and_empty_sequences_write_nothing():
    p = make_problem(dict(name="e", dtype="f32", B=3, L=3, Hq=2, Hkv=1, d=4, w=3, lens=("list", [0, 1, 2]), gate_std=1.0,
                          peaks=0.0, page_size=0, seed=3))
    k_new = np.full((3, 3, 1, 4), 7.0, dtype=np.float32)
    after, _ = oracle.prestep(p, k_new, k_new, np.zeros((2, 4)), np.zeros(2))
    assert np.array_equal(after.k_cache[0], p.k_cache[0]) and np.array_equal(after.k_win[0], p.k_win[0])  # N = 0
    assert np.all(after.k_cache[1, 0] == 7.0) and np.array_equal(after.k_win[1], p.k_win[1])            # N = 1: loop 1 only
    assert np.all(after.k_cache[2, 1] == 7.0) and np.array_equal(after.k_cache[2, 0], p.k_cache[2, 0])
    assert np.all(after.k_win[2, 0, 0] == 7.0) and np.array_equal(after.k_win[2, 1], p.k_win[2, 1])      # loop 3 lags 2


def test_gate_linear_closed_forms():
    rng = np.random.default_rng(1)
    q = rng.standard_normal((2, 3, 4, 8)).astype(np.float32)
    b = rng.standard_normal(4)
    eye = np.zeros((4, 8)); eye[np.arange(4), [0, 3, 5, 7]] = 1.0      # unit vectors pick one coordinate of each head
    g = oracle.gate_logits(q, eye, b)
    for h, j in enumerate([0, 3, 5, 7]):
        np.testing.assert_allclose(g[:, :, h], q[:, 1:, h, j].astype(np.float64) + b[h], rtol=0, atol=1e-15)
    assert np.allclose(oracle.gate_logits(np.zeros_like(q), rng.standard_normal((4, 8)), b), b[None, None, :])
    w = rng.standard_normal((4, 8))
    np.testing.assert_allclose(oracle.gate_logits(q, w, b), np.einsum("blhd,hd->blh", q.astype(np.float64), w)[:, 1:] + b,
                               rtol=1e-12, atol=1e-12)
    # head-wise: head h's logit ignores every other head's query
    q2 = q.copy(); q2[:, :, 1] += 5.0
    g2 = oracle.gate_logits(q2, w, b)
    assert np.array_equal(g2[:, :, [0, 2, 3]], oracle.gate_logits(q, w, b)[:, :, [0, 2, 3]])


def test_paged_append_lands_where_the_page_table_points():
    p = empty_problem(2, 2, 2, 1, 4, 3, cap=8, page_size=4, seed=9)
    k_new = np.arange(2 * 2 * 1 * 4, dtype=np.float32).reshape(2, 2, 1, 4) + 1000.0
    p = p.with_(seq_lens=np.array([6, 1], dtype=np.int32))
    after, _ = oracle.prestep(p, k_new, -k_new, np.zeros((2, 4)), np.zeros(2))
    assert np.array_equal(after.k_cache[p.page_table[0, 1], 1], k_new[0, 0])      # position 5 = page slot 1, offset 1
    assert np.array_equal(after.v_cache[p.page_table[1, 0], 0], -k_new[1, 0])     # position 0
    changed = np.argwhere(after.k_cache != p.k_cache)
    assert len({(int(a), int(b_)) for a, b_, _, _ in changed}) == 2               # exactly two rows were written
