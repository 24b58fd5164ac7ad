"""GPU parity of the sequence-shaped attention (plt_seq_attn_run through the C ABI) against the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_24824_b200 import binding as B
from paper_2510_24824_b200.inputs import make_seq_problem
from paper_2510_24824_b200.runner import SeqAttn

from gpu_util import assert_parity

pytestmark = pytest.mark.gpu


def run_seq(p):
    with SeqAttn(p) as op:
        op.out.fill_(float("nan"))
        op.run()
        bits = op.check()
        assert bits == 0, f"device status 0x{bits:x}"
        first = op.out.clone()
        op.run()
        assert op.check() == 0
        assert torch.equal(first, op.out), "two runs on the same inputs differ"
    return first.float().cpu().numpy().astype(np.float64)


def oracle_seq(p):
    with np.errstate(over="ignore"):
        return oracle.seq_attn(p)


def oracle_seq_planes(p, planes):
    with np.errstate(over="ignore"):
        return oracle.seq_attn(p, planes)


def oracle_f32(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32)


# lengths around the tile sizes (128-key tiles, 256 rows per block), loop counts of the paper, window 64
@pytest.mark.parametrize("L", [2, 3])
@pytest.mark.parametrize("n", [1, 127, 128, 129, 255, 256, 257, 700])
def test_lengths_around_the_tiles(n, L):
    p = make_seq_problem(B=2, L=L, T=n, Hq=4, Hkv=2, d=128, w=64, lens=[n, max(1, n // 2)], seed=n + L)
    assert_parity(run_seq(p), oracle_seq(p), "bf16", f"n={n} L={L}")


@pytest.mark.parametrize("L", [2, 3])
def test_prefill_length_of_the_serving_recipe(L):
    """n = 5000 (the paper's prefill length), one sequence, GQA 2:1."""
    p = make_seq_problem(B=1, L=L, T=5000, Hq=2, Hkv=1, d=128, w=64, seed=50 + L)
    got = run_seq(p)
    ref = oracle_seq(p)
    assert_parity(got, ref, "bf16", f"n=5000 L={L}")


def test_single_loop_is_plain_causal_attention():
    p = make_seq_problem(B=2, L=1, T=300, Hq=4, Hkv=4, d=128, w=0, lens=[300, 77], seed=5)
    got = run_seq(p)
    assert_parity(got, oracle_seq(p), "bf16", "L=1")
    q = torch.from_numpy(np.ascontiguousarray(p.q)).view(torch.bfloat16).float()[:, 0].permute(0, 2, 1, 3)
    k = torch.from_numpy(np.ascontiguousarray(p.k_share)).view(torch.bfloat16).float().permute(0, 2, 1, 3)
    v = torch.from_numpy(np.ascontiguousarray(p.v_share)).view(torch.bfloat16).float().permute(0, 2, 1, 3)
    lib = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True).permute(0, 2, 1, 3).numpy()
    assert np.abs(got[0, 0] - lib[0]).max() < 2e-2


@pytest.mark.parametrize("offsets", [[0, 0, 0], [0, 1, 2], [0, 5, 130], [0, 300, 3]])
def test_loop_offsets(offsets):
    p = make_seq_problem(B=1, L=3, T=400, Hq=2, Hkv=1, d=128, w=64, loop_offset=offsets, seed=9)
    got = run_seq(p)
    assert_parity(got, oracle_seq(p), "bf16", f"delta={offsets}")
    for l, dl in enumerate(offsets):
        assert np.all(got[0, l, :dl] == 0.0), "rows of a loop that has no token yet must be exactly zero"


@pytest.mark.parametrize("w", [1, 7, 64, 128, 129, 300, 1000])
def test_window_sizes(w):
    p = make_seq_problem(B=1, L=2, T=520, Hq=2, Hkv=2, d=128, w=w, seed=w)
    assert_parity(run_seq(p), oracle_seq(p), "bf16", f"w={w}")


def test_gate_extremes():
    p = make_seq_problem(B=1, L=2, T=300, Hq=2, Hkv=1, d=128, w=64, seed=4)
    for val in (-np.inf, np.inf, -30.0, 30.0):
        q = p.with_(gate_logits=np.full_like(p.gate_logits, val))
        assert_parity(run_seq(q), oracle_seq(q), "bf16", f"gate={val}")


def test_ragged_batch_and_garbage_beyond_the_lengths():
    """Rows of K, V and Q at or beyond a sequence's length hold NaN: they must not reach any output, and the output
    rows beyond the length are zero."""
    lens = [513, 1, 300, 0, 256]
    p = make_seq_problem(B=5, L=3, T=513, Hq=4, Hkv=2, d=128, w=64, lens=lens, seed=8)
    clean = run_seq(p)
    dirty = p.with_(q=p.q.copy(), k_share=p.k_share.copy(), v_share=p.v_share.copy(), k_loc=p.k_loc.copy(), v_loc=p.v_loc.copy())
    for b, n in enumerate(lens):
        dirty.q[b, :, n:] = 0x7FC0
        dirty.k_share[b, n:] = 0x7FC0
        dirty.v_share[b, n:] = 0x7FC0
        dirty.k_loc[b, :, n:] = 0x7FC0
        dirty.v_loc[b, :, n:] = 0x7FC0
    got = run_seq(dirty)
    assert np.isfinite(got).all()
    np.testing.assert_array_equal(got, clean)
    for b, n in enumerate(lens):
        assert np.all(got[b, :, n:] == 0.0)
    assert_parity(got, oracle_seq(p), "bf16", "ragged")


def test_large_scores_and_peaks():
    p = make_seq_problem(B=1, L=2, T=600, Hq=2, Hkv=1, d=128, w=64, seed=12, sm_scale=1.0)   # scores of std ~11
    assert_parity(run_seq(p), oracle_seq(p), "bf16", "large scores")


def test_argument_errors_and_clamped_lengths():
    p = make_seq_problem(B=2, L=2, T=200, Hq=2, Hkv=1, d=128, w=64, seed=2)
    with SeqAttn(p) as op:
        stream = torch.cuda.current_stream().cuda_stream
        a = B.make_seq_args(3, op.q, op.k_share, op.v_share, op.seq_lens, op.out, op.k_loc, op.v_loc, op.gate_logits)
        with pytest.raises(B.PltError) as e:
            B.plt_seq_attn_run(op.handle, a, stream)
        assert e.value.status == B.PLT_ERR_CAPACITY
        a = B.make_seq_args(2, None, op.k_share, op.v_share, op.seq_lens, op.out, op.k_loc, op.v_loc, op.gate_logits)
        with pytest.raises(B.PltError) as e:
            B.plt_seq_attn_run(op.handle, a, stream)
        assert e.value.status == B.PLT_ERR_INVALID_ARG
        op.seq_lens.copy_(torch.tensor([9999, -3], dtype=torch.int32))
        op.run()
        assert op.check() == B.PLT_DEV_SEQ_LEN_CLAMPED
        clamped = p.with_(seq_lens=np.array([200, 0], dtype=np.int32))
        assert_parity(op.out.float().cpu().numpy().astype(np.float64), oracle_seq(clamped), "bf16", "clamped")


def test_bench_shape_sampled_planes():
    """The shape bench.py times (B=4, L=2, n=5000, GQA 32/8, w=64), checked on sampled (sequence, loop, head) planes the
    oracle computes one by one, plus properties that hold for every row."""
    p = make_seq_problem(B=4, L=2, T=5000, Hq=32, Hkv=8, d=128, w=64, seed=0, name="seq_B4_L2_n5000")
    got = run_seq(p)
    assert np.isfinite(got).all()
    vmax = float(max(np.abs(oracle_f32(p.v_share)).max(), np.abs(oracle_f32(p.v_loc)).max()))
    assert np.abs(got).max() <= vmax * (1 + 2 ** -7)              # convex mixes of V rows
    assert np.all(got[:, 1, 0] == 0.0)                            # loop 2 has no token at step 0 (delta = 1)
    planes = [(0, 0, 0), (1, 1, 5), (2, 0, 31), (3, 1, 16), (0, 1, 30), (2, 1, 9)]
    ref = oracle_seq_planes(p, planes)
    for b, l, h in planes:
        assert_parity(got[b, l, :, h], ref[b, l, :, h], "bf16", f"plane {(b, l, h)}")
