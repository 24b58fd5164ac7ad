"""GPU parity of the multi-token decode step (config.q_len > 1: several query tokens per loop in one step) against the
oracle, through the C ABI. Served by the warp-level bf16 kernel (also on E4M3 caches); other paths must refuse it."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_24824_b200 import binding as B
from paper_2510_24824_b200.inputs import f32_to_bf16_bits, make_problem, quantize_kv_e4m3
from paper_2510_24824_b200.runner import DeviceProblem, to_torch

from gpu_util import assert_parity

pytestmark = pytest.mark.gpu


def run_multi(p, q, gate, q_len, **tuning):
    dp = DeviceProblem(p, "cuda:0")
    dq = to_torch(q, "bf16", "cuda:0")
    dg = to_torch(gate, "", "cuda:0") if p.L > 1 else None
    out = torch.full(q.shape, float("nan"), dtype=torch.bfloat16, device="cuda:0")
    cfg = B.make_config("bf16", p.B, p.L, p.Hq, p.Hkv, p.d, p.max_seq_len, p.w, page_size=p.page_size, device=0,
                        loop_offset=None if p.loop_offset is None else [int(x) for x in p.loop_offset],
                        kv_dtype=p.kv_dtype, q_len=q_len, **tuning)
    h = B.plt_decode_attn_create(cfg)
    try:
        a = dp.args(out)
        a.q = dq.data_ptr()
        a.gate_logits = dg.data_ptr() if dg is not None else None
        stream = torch.cuda.current_stream().cuda_stream
        B.plt_decode_attn_run(h, a, stream)
        assert B.plt_decode_attn_check(h, stream) == 0
    finally:
        B.plt_decode_attn_destroy(h)
    return out.float().cpu().numpy().astype(np.float64)


def case(q_len, B_=3, L=2, Hq=8, Hkv=2, w=40, lens=(300, 77, 2), page_size=0, seed=31, kv="", offsets=None):
    spec = dict(name="mt", dtype="bf16", B=B_, L=L, Hq=Hq, Hkv=Hkv, d=128, w=w, lens=("list", list(lens)), gate_std=1.0,
                peaks=0.0, page_size=page_size, seed=seed, loop_offset=offsets)
    p = make_problem(spec)
    if kv:
        p = quantize_kv_e4m3(p)
    rng = np.random.default_rng(seed + 1)
    q = f32_to_bf16_bits(rng.standard_normal((B_, L, q_len, Hq, 128)).astype(np.float32))
    gate = rng.standard_normal((B_, max(L - 1, 1), q_len, Hq)).astype(np.float32)
    return p, q, gate


@pytest.mark.parametrize("q_len,L,Hq,Hkv", [(2, 2, 8, 2), (4, 2, 8, 2), (3, 3, 8, 2), (4, 2, 16, 2), (8, 2, 8, 2), (2, 4, 32, 4), (5, 1, 8, 2)])
def test_multi_token_step_matches_the_oracle(q_len, L, Hq, Hkv):
    p, q, gate = case(q_len, L=L, Hq=Hq, Hkv=Hkv, lens=(300, 77, q_len + 1))
    got = run_multi(p, q, gate, q_len)
    assert_parity(got, oracle.decode_attn_multi(p, q, gate, q_len), "bf16", f"q_len={q_len} L={L}")


def test_lengths_shorter_than_the_step_and_the_loop_offsets():
    """Sequences with fewer tokens than the step carries: the oldest tokens of a loop have nothing to see and are zero."""
    p, q, gate = case(4, B_=6, L=3, Hq=4, Hkv=2, w=8, lens=(0, 1, 2, 3, 5, 40))
    got = run_multi(p, q, gate, 4)
    ref = oracle.decode_attn_multi(p, q, gate, 4)
    assert_parity(got, ref, "bf16", "short")
    assert np.all(got[ref == 0.0] == 0.0)
    assert np.all(got[0] == 0.0) and np.all(got[1, 0, :3] == 0.0) and np.abs(got[1, 0, 3]).max() > 0


@pytest.mark.parametrize("kv,page_size", [("", 64), ("e4m3", 0), ("e4m3", 64)])
def test_paged_and_e4m3_caches(kv, page_size):
    p, q, gate = case(3, B_=4, L=3, Hq=8, Hkv=2, w=100, lens=(700, 129, 64, 5), page_size=page_size, kv=kv)
    got = run_multi(p, q, gate, 3)
    assert_parity(got, oracle.decode_attn_multi(p, q, gate, 3), "bf16", f"{kv} page={page_size}")


@pytest.mark.parametrize("hpc,kw,ks,rw", [(1, 1, 1, 1), (2, 2, 1, 1), (1, 4, 1, 1), (2, 1, 2, 2), (1, 2, 2, 1)])
def test_launch_variants(hpc, kw, ks, rw):
    p, q, gate = case(3, L=2, Hq=8, Hkv=2, lens=(513, 64, 9))        # 24 packed rows
    got = run_multi(p, q, gate, 3, heads_per_cta=hpc, key_slices=kw, slices_per_warp=ks, row_warps=rw)
    assert_parity(got, oracle.decode_attn_multi(p, q, gate, 3), "bf16", f"hpc={hpc} kw={kw} ks={ks} rw={rw}")


def test_one_token_is_the_plain_step_bit_for_bit():
    p, q, gate = case(1)
    got = run_multi(p, q, gate, 1)
    plain = p.with_(q=np.ascontiguousarray(q[:, :, 0]), gate_logits=np.ascontiguousarray(gate[:, :, 0]))
    dp = DeviceProblem(plain, "cuda:0")
    from paper_2510_24824_b200.runner import DecodeAttn
    with DecodeAttn(plain) as op:
        want = op.run(dp).float().cpu().numpy().astype(np.float64)
    np.testing.assert_array_equal(got[:, :, 0], want)


def test_paths_that_do_not_serve_it_refuse():
    for kw in (dict(dtype="f32"), dict(dtype="bf16", kernel_path=B.PLT_PATH_TCGEN05), dict(dtype="bf16", L=4, Hq=32, Hkv=2)):
        base = dict(dtype="bf16", max_batch=2, L=2, Hq=8, Hkv=2, d=128, max_seq_len=512, w=64, q_len=4)
        base.update(kw)
        with pytest.raises(B.PltError) as e:
            B.plt_decode_attn_workspace_bytes(B.make_config(**base))
        assert e.value.status == B.PLT_ERR_UNSUPPORTED
