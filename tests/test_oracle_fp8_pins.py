"""CPU-only pins of the E4M3-cache variant of the oracle: the code table against the format's definition and a
library cast, and the attention on codes against the ordinary oracle fed the dequantised values."""
import ctypes
import math

import numpy as np
import pytest
import torch

import oracle
from oracle import plt_oracle
from paper_2510_24824_b200.inputs import bf16_bits_to_f32, make_problem, quantize_kv_e4m3


def e4m3_value(code: int) -> float:
    lib = plt_oracle._load()
    lib.plt_oracle_e4m3_value.restype = ctypes.c_double
    lib.plt_oracle_e4m3_value.argtypes = [ctypes.c_uint8]
    return float(lib.plt_oracle_e4m3_value(code))


def test_code_table_matches_the_library_cast_and_the_format_facts():
    lib_vals = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    for c in range(256):
        v = e4m3_value(c)
        if c & 0x7F == 0x7F:
            assert math.isnan(v) and math.isnan(lib_vals[c])
        else:
            assert v == lib_vals[c], c
    # facts of the format: largest finite 448, smallest subnormal 2^-9, smallest normal 2^-6, 1.0 = 0x38, signed zero
    assert e4m3_value(0x7E) == 448.0 and e4m3_value(0xFE) == -448.0
    assert e4m3_value(0x01) == 2.0 ** -9 and e4m3_value(0x08) == 2.0 ** -6 and e4m3_value(0x38) == 1.0
    assert e4m3_value(0x00) == 0.0 and e4m3_value(0x80) == 0.0


def spec(**kw):
    base = dict(name="fp8", dtype="bf16", B=3, L=3, Hq=4, Hkv=2, d=8, w=5, lens=("list", [9, 4, 1]), gate_std=1.0,
                peaks=0.0, page_size=0, seed=13, kv_dtype="e4m3")
    base.update(kw)
    return base


@pytest.mark.parametrize("page_size", [0, 4])
def test_attention_on_codes_equals_the_plain_oracle_on_dequantised_values(page_size):
    """With scales that are powers of two the dequantised values are exact in float32, so the ordinary float32 path of
    the oracle can be fed them directly: both routes must agree to rounding."""
    p = make_problem(spec(page_size=page_size))
    p = p.with_(k_scale=np.array([0.25, 2.0], dtype=np.float32), v_scale=np.array([0.5, 0.125], dtype=np.float32))
    got = oracle.decode_attn(p)

    def deq(codes, scale):
        vals = torch.from_numpy(codes).view(torch.float8_e4m3fn).to(torch.float32).numpy()
        shape = [1] * (codes.ndim - 2) + [p.Hkv, 1]      # [.., Hkv, d] layouts of the cache and of the windows
        return vals * scale.reshape(shape).astype(np.float32)

    plain = p.with_(dtype="f32", kv_dtype="", k_scale=None, v_scale=None, q=bf16_bits_to_f32(p.q),
                    k_cache=deq(p.k_cache, p.k_scale), v_cache=deq(p.v_cache, p.v_scale),
                    k_win=deq(p.k_win, p.k_scale), v_win=deq(p.v_win, p.v_scale))
    np.testing.assert_allclose(got, oracle.decode_attn(plain), rtol=1e-12, atol=1e-14)


def test_scales_act_per_kv_head_and_linearly():
    p = make_problem(spec())
    base = oracle.decode_attn(p)
    G = p.Hq // p.Hkv
    # doubling the V scale of KV head 1 doubles the outputs of its query heads and leaves the others alone
    twice = oracle.decode_attn(p.with_(v_scale=p.v_scale * np.array([1.0, 2.0], dtype=np.float32)))
    np.testing.assert_allclose(twice[:, :, G:], 2.0 * base[:, :, G:], rtol=1e-12)
    assert np.array_equal(twice[:, :, :G], base[:, :, :G])
    # a K scale is a per-head score scale: scaling it by c equals scaling sm_scale by c when all heads share it
    c = np.float32(0.5)
    a = oracle.decode_attn(p.with_(k_scale=p.k_scale * c))
    b = oracle.decode_attn(p.with_(sm_scale=p.scale() * float(c)))
    np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-14)


def test_quantised_problem_stays_close_to_the_unquantised_one():
    """E4M3 keeps 3 mantissa bits (relative step 2^-3, error <= 2^-4): the attention on codes must stay within a few
    percent of the attention on the values it was quantised from, and the generator's scales must cover the range."""
    raw = make_problem(spec(kv_dtype="", d=64, lens=("list", [200, 50, 7])))
    q8 = quantize_kv_e4m3(raw)
    assert q8.k_cache.dtype == np.uint8 and q8.k_scale.shape == (raw.Hkv,)
    kmax = np.abs(bf16_bits_to_f32(raw.k_cache)).max(axis=(0, 1, 3))
    assert np.all(q8.k_scale * 448.0 >= kmax * 0.999) and np.all((q8.k_cache & 0x7F) != 0x7F)
    a, b = oracle.decode_attn(raw), oracle.decode_attn(q8)
    assert np.abs(a - b).max() < 0.15 and np.abs(a - b).mean() < 0.02


def test_quantisation_of_appended_rows():
    """Facts of round-to-nearest-even onto the E4M3 grid, with power-of-two scales so that everything is exact."""
    scale = np.array([0.5, 2.0], dtype=np.float32)

    def q(vals):   # vals: per head a list -> [1, Hkv, d]
        x = np.array(vals, dtype=np.float32)[None]
        return oracle.quantise_e4m3(x, scale)[0]

    # representable values come back as their own codes (head 0: x / 0.5; head 1: x / 2)
    codes = q([[0.5, -0.5, 224.0, 0.0], [2.0, 3.5, -896.0, 2.0 ** -8]])
    assert list(codes[0]) == [0x38, 0xB8, 0x7E, 0x00] and list(codes[1]) == [0x38, 0x3E, 0xFE, 0x01]
    # ties go to the even mantissa: 1.0625 -> 1.0 (0x38), 1.1875 -> 1.25 (0x3A); halfway to the smallest subnormal -> 0
    codes = q([[0.53125, 0.59375, 2.0 ** -11, 3 * 2.0 ** -11], [0, 0, 0, 0]])
    assert list(codes[0]) == [0x38, 0x3A, 0x00, 0x02]
    # beyond the largest finite value: clamped, never NaN
    codes = q([[1e6, -1e6, 225.0, 240.0], [0, 0, 0, 0]])
    assert list(codes[0]) == [0x7E, 0xFE, 0x7E, 0x7E]
    # every code value, times the scale, maps back to its own code (negative zero keeps its sign bit)
    vals = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float32).numpy()
    ok = np.isfinite(vals)
    back = oracle.quantise_e4m3((vals[ok] * 0.5).reshape(1, 1, -1).repeat(2, axis=1), scale)[0, 0]
    assert np.array_equal(back, np.arange(256, dtype=np.uint8)[ok])


def test_prestep_on_e4m3_caches_appends_quantised_rows():
    p = make_problem(spec(lens=("list", [9, 4, 1])))
    rng = np.random.default_rng(2)
    from paper_2510_24824_b200.inputs import f32_to_bf16_bits
    k_new = f32_to_bf16_bits(rng.standard_normal((p.B, p.L, p.Hkv, p.d)).astype(np.float32))
    v_new = f32_to_bf16_bits(rng.standard_normal((p.B, p.L, p.Hkv, p.d)).astype(np.float32))
    after, _ = oracle.prestep(p, k_new, v_new, np.zeros((p.Hq, p.d)), np.zeros(p.Hq))
    want = oracle.quantise_e4m3(k_new, p.k_scale)
    assert np.array_equal(after.k_cache[0, 8], want[0, 0]) and np.array_equal(after.k_win[0, 0, (9 - 1 - 1) % p.w], want[0, 1])
    # the stored code is the nearest grid point: dequantised error at most half a grid step of that magnitude
    deq = torch.from_numpy(after.k_cache[0, 8]).view(torch.float8_e4m3fn).to(torch.float32).numpy() * p.k_scale[:, None]
    x = bf16_bits_to_f32(k_new[0, 0])
    assert np.all(np.abs(deq - x) <= np.maximum(np.abs(x) * 2.0 ** -4, p.k_scale[:, None] * 2.0 ** -10) * 1.0001)
