"""GPU parity of the tcgen05 / tensor-memory main kernel (config.kernel_path = PLT_PATH_TCGEN05), called through the
C ABI, against the fp64 oracle on the same seeded inputs. Same bar as the default path."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_24824_b200 import binding as B
from paper_2510_24824_b200.inputs import make_problem, shrunk_workload
from paper_2510_24824_b200.runner import DecodeAttn, DeviceProblem

from gpu_util import inactive_rows, BF16_MEAN_ABS, assert_parity, bf16_bound, run_gpu

pytestmark = pytest.mark.gpu
TC = dict(kernel_path=B.PLT_PATH_TCGEN05)


def custom(**kw):
    base = dict(name="case", dtype="bf16", B=3, L=2, Hq=8, Hkv=2, d=128, w=40, lens=("list", [300, 77, 1]),
                gate_std=1.0, peaks=0.0, page_size=0, seed=21)
    base.update(kw)
    return base


def test_path_is_reported_and_unsupported_shapes_are_refused():
    p = make_problem(custom())
    with DecodeAttn(p, **TC) as op:
        assert op.info["kernel_path"] == B.PLT_PATH_TCGEN05 and op.info["grid"] >= 1 and op.info["stages"] in (4, 6)
    with DecodeAttn(p) as op:
        assert op.info["kernel_path"] == B.PLT_PATH_WARP_MMA
    # automatic choice: tcgen05 only above 48 packed rows on long-context configurations
    wide = custom(B=1, L=4, Hq=32, Hkv=2, w=33, lens=("list", [400]))
    with DecodeAttn(make_problem(dict(wide, max_seq_len=16384))) as op:
        assert op.info["kernel_path"] == B.PLT_PATH_TCGEN05
    with DecodeAttn(make_problem(dict(wide, max_seq_len=4096))) as op:
        assert op.info["kernel_path"] == B.PLT_PATH_WARP_MMA
    for bad in (custom(d=64), custom(dtype="f32"), custom(page_size=48, lens=("list", [300, 77, 1]))):
        with pytest.raises(B.PltError) as e:
            DecodeAttn(make_problem(bad), **TC)
        assert e.value.status in (B.PLT_ERR_UNSUPPORTED, B.PLT_ERR_INVALID_ARG)
    with pytest.raises(B.PltError):
        DecodeAttn(p, stages=5, **TC)


@pytest.mark.parametrize("index", [1, 2, 3, 4])
def test_shrunk_workloads(index):
    p = make_problem(shrunk_workload(index))
    assert_parity(run_gpu(p, **TC), oracle.decode_attn(p), p.dtype, p.name)


@pytest.mark.parametrize("stages,inflight", [(4, 0), (4, 1), (6, 1), (6, 3)])
def test_ring_sizes_give_the_same_answer(stages, inflight):
    p = make_problem(custom(B=4, L=3, Hq=32, Hkv=8, w=70, lens=("list", [513, 64, 2, 1000])))
    assert_parity(run_gpu(p, stages=stages, loads_in_flight=inflight, **TC), oracle.decode_attn(p), "bf16", f"stages={stages}")


@pytest.mark.parametrize("spec", [
    custom(B=3, L=1, w=0, lens=("list", [129, 1, 64])),                                      # single loop
    custom(B=3, L=3, Hq=32, Hkv=4, w=50, lens=("list", [700, 65, 3])),                       # 24 packed rows
    custom(B=2, L=4, Hq=32, Hkv=2, w=33, lens=("list", [400, 5])),                           # 64 packed rows
    custom(B=8, L=4, Hq=8, Hkv=2, w=32, lens=("list", [0, 1, 2, 3, 4, 31, 32, 33])),         # fewer tokens than loops
    custom(B=2, L=3, Hq=8, Hkv=2, w=300, lens=("list", [2000, 290])),                        # windows of several tiles
    custom(B=3, L=3, Hq=12, Hkv=2, loop_offset=[0, 70, 200]),                                # other causal offsets
], ids=["L1", "R24", "R64", "short", "wide-window", "offsets"])
def test_shapes_and_edges(spec):
    p = make_problem(spec)
    ref = oracle.decode_attn(p)
    got = run_gpu(p, **TC)
    assert_parity(got, ref, "bf16", spec.get("name", ""))
    inactive = inactive_rows(p)
    assert np.all(got[inactive] == 0.0), "rows of loops without a token must be exactly zero"


def test_many_pieces_per_block_and_long_pieces():
    """Enough tiles that every block streams several tiles, wraps its rings and crosses several piece boundaries
    (short and long sequences mixed, two windows of two tiles each); sampled rows against the oracle."""
    lens = [5000, 3000, 7000, 100, 20000, 9000, 64, 12000, 300, 4000, 8000, 15000, 2, 6000, 1000, 11000]
    p = make_problem(custom(B=16, L=3, w=200, Hq=16, Hkv=2, lens=("list", lens)))
    dp = DeviceProblem(p, "cuda:0")
    dp.out.fill_(float("nan"))
    with DecodeAttn(p, **TC) as op:
        for _ in range(3):
            op.run(dp)
            assert op.check() == 0
        first = dp.out.clone()
        op.run(dp)
        assert op.check() == 0
    assert torch.equal(first, dp.out), "two runs on the same inputs differ"
    got = dp.out.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    rows = np.array([(b, l, h) for b in range(p.B) for l in range(p.L) for h in (0, 7, p.Hq - 1)], dtype=np.int32)
    ref = oracle.decode_attn_rows(p, rows)
    err = np.abs(got[rows[:, 0], rows[:, 1], rows[:, 2]] - ref)
    assert (err / bf16_bound(ref)).max() <= 1.0 and err.mean() <= BF16_MEAN_ABS


def test_gate_extremes_and_window_lengths():
    p = make_problem(custom(B=4, L=3, Hq=12, Hkv=2, w=40, lens=("list", [300, 77, 5, 50])))
    for val in (-np.inf, np.inf):
        q = p.with_(gate_logits=np.full_like(p.gate_logits, val))
        assert_parity(run_gpu(q, **TC), oracle.decode_attn(q), "bf16", f"gate={val}")
    q = p.with_(win_lens=np.array([[40, 0], [1, 17], [3, 0], [16, 33]], dtype=np.int32))
    assert_parity(run_gpu(q, **TC), oracle.decode_attn(q), "bf16", "win_lens")


def test_garbage_outside_valid_ranges_cannot_reach_the_output():
    spec = custom(B=4, L=3, Hq=12, Hkv=2, w=40, lens=("list", [300, 77, 5, 0]), max_seq_len=384)
    clean, dirty = make_problem(spec), make_problem(spec, tail_fill=float("nan"))
    a, b = run_gpu(clean, **TC), run_gpu(dirty, **TC)
    assert np.isfinite(b).all()
    np.testing.assert_array_equal(a, b)


def test_peaked_softmax_and_large_scores():
    p = make_problem(custom(B=2, L=2, lens=("list", [2000, 300]), peaks=0.02))
    assert_parity(run_gpu(p, **TC), oracle.decode_attn(p), "bf16", "peaks")
    big = p.with_(sm_scale=4.0)  # scores of magnitude ~50: the lazily updated maxima must keep up
    assert_parity(run_gpu(big, **TC), oracle.decode_attn(big), "bf16", "large scores")


@pytest.mark.parametrize("page_size", [16, 64, 128, 256])
def test_paged_cache(page_size):
    sp = shrunk_workload(4, B=9, lens=("list", [1, 2, 3, 63, 64, 255, 700, 129, 16]), page_size=page_size, w=100)
    p = make_problem(sp)
    assert_parity(run_gpu(p, **TC), oracle.decode_attn(p), "bf16", f"paged {page_size}")


def test_strided_head_major_cache():
    p = make_problem(custom(B=3, L=2, Hq=8, Hkv=2, lens=("list", [300, 77, 1]), max_seq_len=320))
    ref = oracle.decode_attn(p)
    dp = DeviceProblem(p, "cuda:0")
    dp.k_cache = dp.k_cache.permute(0, 2, 1, 3).contiguous()   # [B, Hkv, N, d] storage viewed through strides
    dp.v_cache = dp.v_cache.permute(0, 2, 1, 3).contiguous()
    args = dp.args()
    args.kv_stride_b, args.kv_stride_h, args.kv_stride_n = p.Hkv * 320 * p.d, 320 * p.d, p.d
    with DecodeAttn(p, **TC) as op:
        B.plt_decode_attn_run(op.handle, args, torch.cuda.current_stream().cuda_stream)
        assert op.check() == 0
    assert_parity(dp.out.float().cpu().numpy().astype(np.float64), ref, "bf16", "HND strides")


def test_workspace_reuse_and_clamped_device_values():
    big = make_problem(custom(B=6, L=3, Hq=12, Hkv=2, w=40, lens=("list", [3000, 2500, 4000, 3500, 2000, 3900]), max_seq_len=4096))
    tiny = make_problem(custom(B=1, L=3, Hq=12, Hkv=2, w=40, lens=("list", [70]), max_seq_len=4096, seed=5))
    dbig, dtiny = DeviceProblem(big, "cuda:0"), DeviceProblem(tiny, "cuda:0")
    with DecodeAttn(big, **TC) as op:
        for _ in range(2):
            op.run(dbig)
            torch.cuda.synchronize()
            assert_parity(dbig.out.float().cpu().numpy().astype(np.float64), oracle.decode_attn(big), "bf16", "big")
            op.run(dtiny)
            torch.cuda.synchronize()
            assert_parity(dtiny.out.float().cpu().numpy().astype(np.float64), oracle.decode_attn(tiny), "bf16", "tiny")
        assert op.check() == 0
    p = make_problem(custom(B=3, lens=("list", [300, 77, 1]), max_seq_len=320))
    bad = p.with_(seq_lens=np.array([300, 100000, -5], dtype=np.int32))
    dp = DeviceProblem(bad, "cuda:0")
    with DecodeAttn(bad, **TC) as op:
        op.run(dp)
        assert op.check() & B.PLT_DEV_SEQ_LEN_CLAMPED
    clamped = p.with_(seq_lens=np.array([300, 320, 0], dtype=np.int32))
    assert_parity(dp.out.float().cpu().numpy().astype(np.float64), oracle.decode_attn(clamped), "bf16", "clamped")
