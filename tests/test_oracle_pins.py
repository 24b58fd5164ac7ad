"""CPU-only checks that pin the fp64 oracle to facts fixed by the paper and by mathematics.

Each test names the statement it relies on. None of them calls the CUDA path.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2510_24824_b200.inputs import (ClpProblem, algorithmic_bytes, bf16_bits_to_f32, f32_to_bf16_bits,
                                          make_problem, shrunk_workload)


def spec(**kw):
    base = dict(name="pin", dtype="f32", B=2, L=3, Hq=4, Hkv=2, d=8, w=5, lens=("list", [9, 4]), gate_std=1.0,
                peaks=0.0, page_size=0, seed=11)
    base.update(kw)
    if "B" in kw and "lens" not in kw:
        base["lens"] = ("list", [9 + 3 * i for i in range(kw["B"])])
    return base


def as_f64(p: ClpProblem, name: str) -> np.ndarray:
    a = getattr(p, name)
    return (bf16_bits_to_f32(a) if p.dtype == "bf16" else a).astype(np.float64)


def cutoffs(p: ClpProblem) -> np.ndarray:
    """[B, L]: loop l (1-indexed) serves token i - l + 1 (Sec. 2.2.1), so it may see max(0, N_b - delta_l) keys of the
    shared cache, delta_l = l - 1 unless the problem carries other offsets. Written here, not taken from the package."""
    delta = list(range(p.L)) if p.loop_offset is None else [int(x) for x in p.loop_offset]
    return np.array([[max(0, int(n) - delta[l]) for l in range(p.L)] for n in p.seq_lens], dtype=np.int64).reshape(p.B, p.L)


def window_lens(p: ClpProblem) -> np.ndarray:
    """[B, L-1]: a non-first loop keeps its w newest entries (Sec. 2.2.2): min(w, tokens it has seen) unless given."""
    if p.win_lens is not None:
        return np.clip(np.asarray(p.win_lens, dtype=np.int64), 0, p.w)
    return np.minimum(p.w, cutoffs(p)[:, 1:])


def independent_reference(p: ClpProblem) -> np.ndarray:
    """Written from the definition with numpy primitives only (np.exp, sums); dense contiguous caches."""
    q, K, V = as_f64(p, "q"), as_f64(p, "k_cache"), as_f64(p, "v_cache")
    Kw, Vw = as_f64(p, "k_win"), as_f64(p, "v_win")
    G = p.Hq // p.Hkv
    out = np.zeros((p.B, p.L, p.Hq, p.d))
    cuts, wls = cutoffs(p), window_lens(p)
    for b in range(p.B):
        for l in range(p.L):
            for h in range(p.Hq):
                n = int(cuts[b, l])
                if n == 0:
                    continue
                kv = h // G
                e = np.exp((K[b, :n, kv] @ q[b, l, h]) * p.scale())
                yg = (e / e.sum()) @ V[b, :n, kv]
                if l == 0:
                    out[b, l, h] = yg
                    continue
                m = int(wls[b, l - 1])
                yl = np.zeros(p.d)
                if m:
                    e = np.exp((Kw[b, l - 1, :m, kv] @ q[b, l, h]) * p.scale())
                    yl = (e / e.sum()) @ Vw[b, l - 1, :m, kv]
                g = 1.0 / (1.0 + math.exp(-float(p.gate_logits[b, l - 1, h])))
                out[b, l, h] = g * yl + (1 - g) * yg
    return out


# ---- P4: brute force on tiny inputs -------------------------------------------------------------
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("L,Hq,Hkv,d,w,lens", [(1, 2, 1, 4, 3, [6]), (2, 2, 2, 4, 3, [6, 1]), (3, 2, 1, 2, 2, [5, 2, 3]),
                                               (3, 4, 2, 8, 5, [9, 4, 1, 2])])
def test_bruteforce_tiny(dtype, L, Hq, Hkv, d, w, lens):
    p = make_problem(spec(dtype=dtype, B=len(lens), L=L, Hq=Hq, Hkv=Hkv, d=d, w=w, lens=("list", lens)))
    np.testing.assert_allclose(oracle.decode_attn(p), independent_reference(p), rtol=1e-12, atol=1e-13)


# ---- P1: L = 1 is standard causal decode attention (first loop = vanilla transformer) -----------
def test_single_loop_equals_library_attention():
    p = make_problem(spec(B=3, L=1, Hq=6, Hkv=2, d=16, w=0, lens=("list", [17, 1, 40])))
    got = oracle.decode_attn(p)
    G = p.Hq // p.Hkv
    for b in range(p.B):
        n = int(p.seq_lens[b])
        q = torch.from_numpy(p.q[b, 0].astype(np.float64))[None, :, None, :]  # [1, Hq, 1, d]
        k = torch.from_numpy(p.k_cache[b, :n].astype(np.float64)).permute(1, 0, 2).repeat_interleave(G, 0)[None]
        v = torch.from_numpy(p.v_cache[b, :n].astype(np.float64)).permute(1, 0, 2).repeat_interleave(G, 0)[None]
        ref = torch.nn.functional.scaled_dot_product_attention(q, k, v)[0, :, 0].numpy()
        np.testing.assert_allclose(got[b, 0], ref, rtol=1e-12, atol=1e-13)


# ---- P2: gate closed cases. g = 0 is the paper's "KV share" variant, g = 1 is pure SWA ----------
def test_gate_closed_is_shared_kv_attention_and_open_is_pure_swa():
    p = make_problem(spec())
    base = p.with_(L=1, q=None)
    closed = oracle.decode_attn(p.with_(gate_logits=np.full_like(p.gate_logits, -np.inf)))
    opened = oracle.decode_attn(p.with_(gate_logits=np.full_like(p.gate_logits, np.inf)))
    cuts, wls = cutoffs(p), window_lens(p)
    for l in range(1, p.L):
        # g = 0: loop l equals a single-loop problem with that loop's queries and the cache cut at `cut`.
        single = base.with_(q=np.ascontiguousarray(p.q[:, l:l + 1]), seq_lens=cuts[:, l].astype(np.int32))
        np.testing.assert_allclose(closed[:, l], oracle.decode_attn(single)[:, 0], rtol=1e-13, atol=1e-14)
        # g = 1: loop l equals a single-loop problem whose cache is that loop's window.
        kw, vw = np.ascontiguousarray(p.k_win[:, l - 1]), np.ascontiguousarray(p.v_win[:, l - 1])
        lens = np.where(cuts[:, l] > 0, wls[:, l - 1], 0).astype(np.int32)
        local = base.with_(q=np.ascontiguousarray(p.q[:, l:l + 1]), k_cache=kw, v_cache=vw, seq_lens=lens,
                           max_seq_len=p.w)
        np.testing.assert_allclose(opened[:, l], oracle.decode_attn(local)[:, 0], rtol=1e-13, atol=1e-14)
    assert np.isfinite(closed).all() and np.isfinite(opened).all()


# ---- P3: a window that holds the whole visible context makes SWA equal full attention -----------
def test_window_covering_context_makes_gate_irrelevant():
    lens = [9, 4]
    p = make_problem(spec(w=12, lens=("list", lens)))
    cuts = cutoffs(p)
    kw, vw = p.k_win.copy(), p.v_win.copy()
    for b in range(p.B):
        for l in range(1, p.L):
            n = int(cuts[b, l])
            kw[b, l - 1, :n] = p.k_cache[b, :n]
            vw[b, l - 1, :n] = p.v_cache[b, :n]
    p = p.with_(k_win=kw, v_win=vw)
    ref = oracle.decode_attn(p.with_(gate_logits=np.full_like(p.gate_logits, -np.inf)))
    for shift in (-3.0, 0.0, 2.5):
        np.testing.assert_allclose(oracle.decode_attn(p.with_(gate_logits=p.gate_logits + np.float32(shift))), ref,
                                   rtol=1e-12, atol=1e-13)


# ---- P5: Q = 0 gives uniform weights: closed form that pins cutoffs, delta_l and wl --------------
@pytest.mark.parametrize("offsets", [None, [0, 0, 0], [0, 2, 5]])
def test_zero_query_closed_form_pins_cutoffs(offsets):
    lens = [9, 4, 1, 2, 3]
    p = make_problem(spec(B=5, lens=("list", lens), loop_offset=offsets))
    K, V = p.k_cache, p.v_cache.copy()
    V[...] = 0
    V[:, :, :, 0] = np.arange(V.shape[1], dtype=np.float32)[None, :, None]  # V[b, j, h, 0] = j
    Vw = p.v_win.copy()
    Vw[...] = 0
    Vw[:, :, :, :, 0] = 1000.0 + np.arange(p.w, dtype=np.float32)[None, None, :, None]
    p = p.with_(q=np.zeros_like(p.q), v_cache=V, v_win=Vw)
    got = oracle.decode_attn(p)
    delta = offsets if offsets is not None else [0, 1, 2]
    for b, n in enumerate(lens):
        for l in range(p.L):
            cut = max(0, n - delta[l])
            for h in range(p.Hq):
                if cut == 0:
                    want = 0.0
                else:
                    yg = (cut - 1) / 2.0
                    if l == 0:
                        want = yg
                    else:
                        wl = min(p.w, cut)
                        yl = 1000.0 + (wl - 1) / 2.0
                        g = 1.0 / (1.0 + math.exp(-float(p.gate_logits[b, l - 1, h])))
                        want = g * yl + (1 - g) * yg
                assert got[b, l, h, 0] == pytest.approx(want, rel=1e-13, abs=1e-13)
                assert np.all(got[b, l, h, 1:] == 0.0)


def test_explicit_window_lengths_and_empty_window():
    lens = [9, 6]
    p = make_problem(spec(lens=("list", lens)))
    Vw = np.zeros_like(p.v_win)
    Vw[..., 0] = 7.0
    V = np.zeros_like(p.v_cache)
    V[..., 0] = 3.0
    wl = np.array([[2, 0], [5, 1]], dtype=np.int32)
    got = oracle.decode_attn(p.with_(v_cache=V, v_win=Vw, win_lens=wl))
    for b in range(2):
        for l in range(1, 3):
            for h in range(p.Hq):
                g = 1.0 / (1.0 + math.exp(-float(p.gate_logits[b, l - 1, h])))
                yl = 7.0 if wl[b, l - 1] > 0 else 0.0  # empty window with a visible context: y_local = 0
                assert got[b, l, h, 0] == pytest.approx(g * yl + (1 - g) * 3.0, rel=1e-13)


# ---- P6: convexity ------------------------------------------------------------------------------
def test_constant_values_give_constant_output_and_outputs_are_bounded():
    p = make_problem(spec(B=3, dtype="bf16"))
    c = f32_to_bf16_bits(np.full(1, 1.75, dtype=np.float32))[0]
    got = oracle.decode_attn(p.with_(v_cache=np.full_like(p.v_cache, c), v_win=np.full_like(p.v_win, c)))
    active = cutoffs(p) > 0
    np.testing.assert_allclose(got[active], 1.75, rtol=1e-13)
    assert np.all(got[~active] == 0.0)
    plain = oracle.decode_attn(p)
    vmax = max(np.abs(as_f64(p, "v_cache")).max(), np.abs(as_f64(p, "v_win")).max())
    assert np.abs(plain).max() <= vmax


# ---- P7: the newest key is visible to loop 1 only (direction of the per-loop cutoff) ------------
def test_dominant_last_key_is_seen_by_first_loop_only():
    n = 12
    p = make_problem(spec(B=1, L=3, Hq=2, Hkv=1, d=8, w=4, lens=("list", [n])))
    K = p.k_cache.copy()
    qsum = p.q[0].reshape(-1, p.d)
    # Key n-1 lines up with every query (sum of sign patterns would cancel, so use a per-query test below).
    got = []
    for l in range(p.L):
        for h in range(p.Hq):
            Kl = K.copy()
            Kl[0, n - 1, 0] = 50.0 * p.q[0, l, h] / np.linalg.norm(p.q[0, l, h])
            o = oracle.decode_attn(p.with_(k_cache=Kl, gate_logits=np.full_like(p.gate_logits, -np.inf)))[0, l, h]
            got.append((l, np.abs(o - p.v_cache[0, n - 1, 0]).max()))
    for l, err in got:
        if l == 0:
            assert err < 1e-9  # softmax collapses onto key n-1
        else:
            assert err > 1e-2  # loops >= 2 serve older tokens and must not see it
    # With delta = 0 for every loop (the training-shift reading), all loops see it.
    for l in range(p.L):
        Kl = K.copy()
        Kl[0, n - 1, 0] = 50.0 * p.q[0, l, 0] / np.linalg.norm(p.q[0, l, 0])
        o = oracle.decode_attn(p.with_(k_cache=Kl, gate_logits=np.full_like(p.gate_logits, -np.inf),
                                       loop_offset=np.zeros(3, np.int32)))[0, l, 0]
        assert np.abs(o - p.v_cache[0, n - 1, 0]).max() < 1e-9


# ---- P8: order of keys is irrelevant; paging is only an address map -----------------------------
def test_key_permutation_invariance_and_window_rotation():
    p = make_problem(spec(B=2, lens=("list", [9, 7])))
    ref = oracle.decode_attn(p)
    rng = np.random.default_rng(5)
    K, V = p.k_cache.copy(), p.v_cache.copy()
    for b in range(p.B):
        m = int(cutoffs(p)[b].min())  # keys every loop sees
        perm = rng.permutation(m)
        K[b, :m] = K[b, perm]
        V[b, :m] = V[b, perm]
    np.testing.assert_allclose(oracle.decode_attn(p.with_(k_cache=K, v_cache=V)), ref, rtol=1e-12, atol=1e-14)
    # A full ring buffer may sit in any rotation.
    full = window_lens(p).min() == p.w
    assert full
    np.testing.assert_allclose(
        oracle.decode_attn(p.with_(k_win=np.roll(p.k_win, 2, axis=2), v_win=np.roll(p.v_win, 2, axis=2))), ref,
        rtol=1e-12, atol=1e-14)


def test_paged_equals_contiguous():
    sp = shrunk_workload(4, B=7, lens=("list", [1, 2, 3, 63, 64, 255, 130]), page_size=16, Hq=8, Hkv=2, d=16, w=20)
    paged = make_problem(sp)
    assert paged.page_table is not None
    # Undo the paging by hand.
    cap = paged.max_seq_len
    K = np.zeros((paged.B, cap, paged.Hkv, paged.d), dtype=paged.k_cache.dtype)
    V = np.zeros_like(K)
    for b in range(paged.B):
        for j in range(int(paged.seq_lens[b])):
            pid = paged.page_table[b, j // 16]
            K[b, j] = paged.k_cache[pid, j % 16]
            V[b, j] = paged.v_cache[pid, j % 16]
    flat = paged.with_(k_cache=K, v_cache=V, page_table=None, page_size=0)
    np.testing.assert_array_equal(oracle.decode_attn(paged), oracle.decode_attn(flat))
    np.testing.assert_allclose(oracle.decode_attn(flat), independent_reference(flat), rtol=1e-12, atol=1e-13)


# ---- P9: softmax shift invariance, no overflow ---------------------------------------------------
def test_score_shift_invariance_and_large_scores():
    p = make_problem(spec(B=1, L=2, Hq=1, Hkv=1, d=8, w=4, lens=("list", [10])))
    ref = oracle.decode_attn(p)
    # Adding c*q/|q|^2 to every key adds the same constant to every score of that query (one head, one loop).
    for l in range(2):
        qv = p.q[0, l, 0].astype(np.float64)
        bump = (40.0 / p.scale()) * qv / (qv @ qv)
        K = (p.k_cache.astype(np.float64) + bump).astype(np.float32)
        Kw = (p.k_win.astype(np.float64) + bump).astype(np.float32)
        got = oracle.decode_attn(p.with_(k_cache=K, k_win=Kw))
        np.testing.assert_allclose(got[0, l], ref[0, l], rtol=1e-4, atol=1e-5)
    big = oracle.decode_attn(p.with_(q=(p.q * 1e3).astype(np.float32)))
    assert np.isfinite(big).all()


# ---- P10: GQA map (contiguous groups) -------------------------------------------------------------
def test_gqa_head_mapping():
    p = make_problem(spec(B=1, L=2, Hq=6, Hkv=3, d=4, w=3, lens=("list", [8])))
    V = np.zeros_like(p.v_cache)
    Vw = np.zeros_like(p.v_win)
    for kv in range(p.Hkv):
        V[:, :, kv, :] = 10.0 * (kv + 1)
        Vw[:, :, :, kv, :] = 10.0 * (kv + 1)
    got = oracle.decode_attn(p.with_(v_cache=V, v_win=Vw))
    for h in range(p.Hq):
        np.testing.assert_allclose(got[0, :, h], 10.0 * (h // 2 + 1), rtol=1e-13)


# ---- Eq. 2 mixes two separately normalised softmaxes ---------------------------------------------
def test_mix_is_not_a_joint_softmax():
    p = make_problem(spec(B=1, L=2, Hq=1, Hkv=1, d=4, w=2, lens=("list", [9])))
    V = np.zeros_like(p.v_cache)
    Vw = np.ones_like(p.v_win)
    gate = np.zeros_like(p.gate_logits)  # g = 1/2
    got = oracle.decode_attn(p.with_(q=np.zeros_like(p.q), v_cache=V, v_win=Vw, gate_logits=gate))
    # separate softmaxes: 0.5 * 1 + 0.5 * 0; a joint softmax over 8 + 2 keys would give 0.2
    np.testing.assert_allclose(got[0, 1, 0], 0.5, rtol=1e-14)


# ---- sampled rows agree with the full run; stored types ------------------------------------------
def test_row_sampling_matches_full_output():
    p = make_problem(shrunk_workload(2))
    full = oracle.decode_attn(p)
    rows = np.array([[0, 0, 0], [4, 2, 31], [2, 1, 7], [3, 2, 16]], dtype=np.int32)
    part = oracle.decode_attn_rows(p, rows)
    for i, (b, l, h) in enumerate(rows):
        np.testing.assert_array_equal(part[i], full[b, l, h])


def test_bf16_storage_roundtrip():
    x = np.array([1.0, -2.5, 3.140625, 1e-3, 65504.0, 1.00390625, 1.01171875], dtype=np.float32)
    bits = f32_to_bf16_bits(x)
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(bf16_bits_to_f32(bits), want)
    r = np.random.default_rng(0).standard_normal(10000).astype(np.float32)
    np.testing.assert_array_equal(bf16_bits_to_f32(f32_to_bf16_bits(r)),
                                  torch.from_numpy(r).to(torch.bfloat16).to(torch.float32).numpy())


# ---- byte model against the paper's printed KV-cache sizes ---------------------------------------
def test_byte_model_reproduces_printed_kv_overhead():
    from pathlib import Path
    rows = [l.split() for l in (Path(__file__).parent / "golden" / "kv_cache_overhead.txt").read_text().splitlines()
            if l and not l.startswith("#")]
    printed = {int(a): int(b) for a, b in rows}
    for L, size in printed.items():
        p = make_problem(dict(name="kv", dtype="bf16", B=4, L=L, Hq=4, Hkv=2, d=8, w=64, lens=("fixed", 5000),
                              page_size=0, seed=0))
        by = algorithmic_bytes(p)
        # Window tokens served: loops 2..L hold min(w, cut) = 64 entries each.
        ratio = (by["shared_kv"] + by["window_kv"]) / by["shared_kv"]
        assert round(printed[1] * ratio) == size
