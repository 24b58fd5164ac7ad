"""GPU parity of the E4M3-cache variant (config.kv_dtype = PLT_KV_E4M3) through the C ABI against the oracle, which
applies the same definition to the dequantised values. Same tolerance as the bf16 path: q and out are bf16."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_24824_b200 import binding as B
from paper_2510_24824_b200.inputs import make_problem, shrunk_workload
from paper_2510_24824_b200.runner import DecodeAttn, DeviceProblem

from gpu_util import inactive_rows, assert_parity, run_gpu

pytestmark = pytest.mark.gpu


def custom(**kw):
    base = dict(name="fp8", dtype="bf16", kv_dtype="e4m3", B=3, L=2, Hq=8, Hkv=2, d=128, w=40, lens=("list", [300, 77, 1]),
                gate_std=1.0, peaks=0.0, page_size=0, seed=41)
    base.update(kw)
    return base


@pytest.mark.parametrize("index", [1, 2, 3, 4])
def test_shrunk_workloads(index):
    p = make_problem(shrunk_workload(index, kv_dtype="e4m3"))
    assert p.k_cache.dtype == np.uint8
    assert_parity(run_gpu(p), oracle.decode_attn(p), "bf16", p.name)


@pytest.mark.parametrize("spec", [
    custom(B=3, L=1, w=0, lens=("list", [129, 1, 64])),                                      # single loop
    custom(B=4, L=3, Hq=32, Hkv=8, w=70, lens=("list", [513, 64, 2, 1000])),                 # 12 packed rows
    custom(B=3, L=3, Hq=32, Hkv=4, w=50, lens=("list", [700, 65, 3])),                       # 24 packed rows
    custom(B=3, L=4, Hq=32, Hkv=4, w=90, lens=("list", [900, 130, 2])),                      # 32 packed rows
    custom(B=2, L=4, Hq=32, Hkv=2, w=33, lens=("list", [400, 5])),                           # 64 packed rows
    custom(B=8, L=4, Hq=8, Hkv=2, w=32, lens=("list", [0, 1, 2, 3, 4, 31, 32, 33])),         # fewer tokens than loops
    custom(B=2, L=3, Hq=8, Hkv=2, w=300, lens=("list", [2000, 290])),                        # windows of several tiles
    custom(B=3, L=3, Hq=12, Hkv=2, loop_offset=[0, 70, 200]),                                # other causal offsets
], ids=["L1", "R12", "R24", "R32", "R64", "short", "wide-window", "offsets"])
def test_shapes_and_edges(spec):
    p = make_problem(spec)
    got = run_gpu(p)
    assert_parity(got, oracle.decode_attn(p), "bf16", spec.get("name", ""))
    assert np.all(got[inactive_rows(p)] == 0.0), "rows of loops without a token must be exactly zero"


@pytest.mark.parametrize("hpc,kw,rw", [(1, 1, 1), (2, 1, 1), (4, 1, 1), (1, 2, 1), (2, 2, 1), (1, 1, 2), (2, 1, 2), (1, 2, 2)])
def test_launch_variants(hpc, kw, rw):
    p = make_problem(custom(B=3, L=3, Hq=24, Hkv=4, w=50, lens=("list", [700, 65, 3])))      # 18 packed rows
    got = run_gpu(p, heads_per_cta=hpc, key_slices=kw, row_warps=rw)
    assert_parity(got, oracle.decode_attn(p), "bf16", f"hpc={hpc} kw={kw} rw={rw}")


def test_scales_reach_the_kernel_per_head():
    p = make_problem(custom(B=2, L=2, Hq=8, Hkv=2, lens=("list", [200, 31])))
    q = p.with_(k_scale=(p.k_scale * np.array([0.5, 3.0])).astype(np.float32),
                v_scale=(p.v_scale * np.array([2.0, 0.25])).astype(np.float32))
    assert_parity(run_gpu(q), oracle.decode_attn(q), "bf16", "rescaled")


@pytest.mark.parametrize("page_size", [64, 128])
def test_paged_cache(page_size):
    p = make_problem(shrunk_workload(4, kv_dtype="e4m3", B=9, lens=("list", [1, 2, 3, 63, 64, 255, 700, 129, 16]),
                                     page_size=page_size, w=100))
    assert_parity(run_gpu(p), oracle.decode_attn(p), "bf16", f"paged {page_size}")


def test_garbage_codes_outside_valid_ranges_cannot_reach_the_output():
    p = make_problem(custom(B=4, L=3, Hq=12, Hkv=2, w=40, lens=("list", [300, 77, 5, 0]), max_seq_len=384))
    dirty_k, dirty_v = p.k_cache.copy(), p.v_cache.copy()
    kw_, vw_ = p.k_win.copy(), p.v_win.copy()
    wl = p.window_lengths()
    for b in range(p.B):
        dirty_k[b, int(p.seq_lens[b]):] = 0x7F            # NaN codes beyond the valid keys
        dirty_v[b, int(p.seq_lens[b]):] = 0xFF
        for l in range(p.L - 1):
            kw_[b, l, int(wl[b, l]):] = 0x7F
            vw_[b, l, int(wl[b, l]):] = 0x7F
    a = run_gpu(p)
    b_ = run_gpu(p.with_(k_cache=dirty_k, v_cache=dirty_v, k_win=kw_, v_win=vw_))
    assert np.isfinite(b_).all()
    np.testing.assert_array_equal(a, b_)


def test_unsupported_combinations_are_refused():
    for bad in (custom(d=64), custom(dtype="f32"), custom(page_size=16)):
        with pytest.raises((B.PltError, Exception)):
            DecodeAttn(make_problem(bad))
    p = make_problem(custom(B=2, L=4, Hq=32, Hkv=2, w=33, lens=("list", [400, 5])))   # 64 packed rows
    with pytest.raises(B.PltError):
        DecodeAttn(p, kernel_path=B.PLT_PATH_TCGEN05)
    p = make_problem(custom())
    dp = DeviceProblem(p, "cuda:0")
    with DecodeAttn(p) as op:
        a = dp.args()
        a.k_scale = None
        with pytest.raises(B.PltError):
            B.plt_decode_attn_run(op.handle, a, torch.cuda.current_stream().cuda_stream)
