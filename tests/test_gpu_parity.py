"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_24824_b200 import binding as B
from paper_2510_24824_b200.inputs import make_problem, shrunk_workload, workload
from paper_2510_24824_b200.runner import DecodeAttn, DeviceProblem

from gpu_util import assert_parity, inactive_rows, parity_report, run_gpu

pytestmark = pytest.mark.gpu


def custom(**kw):
    base = dict(name="case", dtype="bf16", B=3, L=2, Hq=8, Hkv=2, d=128, w=40, lens=("list", [300, 77, 1]),
                gate_std=1.0, peaks=0.0, page_size=0, seed=21)
    base.update(kw)
    return base


# ---- the five workloads, shrunk so the oracle finishes in seconds but several tiles and ragged tails remain ----
@pytest.mark.parametrize("index", [0, 1, 2, 3, 4])
def test_shrunk_workloads(index):
    p = make_problem(shrunk_workload(index))
    assert_parity(run_gpu(p), oracle.decode_attn(p), p.dtype, p.name)


def test_tiny_fp32_config_exact_shape():
    p = make_problem(workload(0))
    assert (p.B, p.L, p.Hq, p.Hkv, p.d, p.w, int(p.seq_lens[0])) == (1, 2, 4, 1, 64, 16, 256)
    assert_parity(run_gpu(p), oracle.decode_attn(p), "f32", "config 1")


# ---- every launch variant must give the same answer (split invariance) --------------------------------------
# heads_per_cta x key_slices (warps along the keys) x slices_per_warp x row_warps; R = packed rows per KV head.
@pytest.mark.parametrize("hpc,kw", [(1, 1), (1, 2), (1, 4), (2, 1), (2, 2), (2, 4), (4, 1), (4, 2), (8, 1), (1, 8)])
def test_bf16_variants_12_rows(hpc, kw):
    p = make_problem(custom(B=4, L=3, Hq=32, Hkv=8, w=70, lens=("list", [513, 64, 2, 1000])))
    ref = oracle.decode_attn(p)
    for cps, stages in ((1, 2), (2, 0)):
        assert_parity(run_gpu(p, heads_per_cta=hpc, key_slices=kw, ctas_per_sm=cps, stages=stages), ref, "bf16",
                      f"hpc={hpc} kw={kw} cps={cps}")


@pytest.mark.parametrize("hpc,kw,ks,rw", [(1, 1, 1, 1), (1, 2, 1, 1), (1, 4, 1, 1), (2, 1, 1, 1), (2, 2, 1, 1), (4, 1, 1, 1),
                                          (1, 1, 2, 1), (2, 2, 2, 1), (4, 1, 2, 1), (1, 1, 1, 2), (2, 2, 1, 2), (2, 1, 2, 2),
                                          (1, 4, 2, 2)])
def test_bf16_variants_24_rows(hpc, kw, ks, rw):
    """24 packed rows: one warp with three 8-row groups, or two warps with two groups each (the second half empty)."""
    p = make_problem(custom(B=3, L=3, Hq=32, Hkv=4, w=50, lens=("list", [700, 65, 3])))
    got = run_gpu(p, heads_per_cta=hpc, key_slices=kw, slices_per_warp=ks, row_warps=rw)
    assert_parity(got, oracle.decode_attn(p), "bf16", f"hpc={hpc} kw={kw} ks={ks} rw={rw}")


@pytest.mark.parametrize("hpc,kw,ks,rw", [(1, 1, 1, 1), (2, 2, 1, 1), (1, 2, 2, 1), (2, 1, 2, 2), (1, 2, 1, 2), (4, 1, 1, 2)])
def test_bf16_variants_32_rows(hpc, kw, ks, rw):
    """32 packed rows: four 8-row groups in one warp, or two in each of two warps (the automatic choice)."""
    p = make_problem(custom(B=3, L=4, Hq=32, Hkv=4, w=90, lens=("list", [900, 130, 2])))
    got = run_gpu(p, heads_per_cta=hpc, key_slices=kw, slices_per_warp=ks, row_warps=rw)
    assert_parity(got, oracle.decode_attn(p), "bf16", f"hpc={hpc} kw={kw} ks={ks} rw={rw}")


@pytest.mark.parametrize("hpc,kw,ks", [(1, 1, 1), (1, 2, 1), (2, 1, 1), (1, 1, 2), (1, 2, 2)])
def test_bf16_variants_64_rows(hpc, kw, ks):
    p = make_problem(custom(B=2, L=4, Hq=32, Hkv=2, w=33, lens=("list", [400, 5])))  # two warps of 32 rows
    got = run_gpu(p, heads_per_cta=hpc, key_slices=kw, slices_per_warp=ks)
    assert_parity(got, oracle.decode_attn(p), "bf16", f"hpc={hpc} kw={kw} ks={ks}")


def test_variant_arguments_are_checked():
    p = make_problem(custom(B=2, L=4, Hq=32, Hkv=2, w=33, lens=("list", [400, 5])))   # 64 packed rows
    for bad in (dict(row_warps=3), dict(slices_per_warp=3), dict(row_warps=1, heads_per_cta=1),   # 64 rows need 2 warps
                dict(heads_per_cta=3), dict(heads_per_cta=1, key_slices=3)):
        with pytest.raises(B.PltError):
            DecodeAttn(p, **bad)


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_head_dims(d, dtype):
    p = make_problem(custom(dtype=dtype, d=d, B=3, L=2, Hq=8, Hkv=2, lens=("list", [300, 77, 1])))
    assert_parity(run_gpu(p), oracle.decode_attn(p), dtype, f"d={d} {dtype}")


def test_fp32_many_rows_and_long_context():
    p = make_problem(custom(dtype="f32", B=2, L=4, Hq=16, Hkv=1, d=64, w=20, lens=("list", [3000, 31])))  # 64 rows
    assert_parity(run_gpu(p), oracle.decode_attn(p), "f32", "fp32 R=64")


# ---- degenerate and edge cases -------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_single_loop_is_plain_decode_attention(dtype):
    p = make_problem(custom(dtype=dtype, L=1, w=0, lens=("list", [129, 1, 64])))
    assert_parity(run_gpu(p), oracle.decode_attn(p), dtype, "L=1")


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_lengths_below_loop_count_and_window(dtype):
    p = make_problem(custom(dtype=dtype, B=8, L=4, Hq=8, Hkv=2, w=32, lens=("list", [0, 1, 2, 3, 4, 31, 32, 33])))
    ref = oracle.decode_attn(p)
    got = run_gpu(p)
    assert_parity(got, ref, dtype, "short sequences")
    inactive = inactive_rows(p)
    assert inactive.any()
    assert np.all(got[inactive] == 0.0), "rows of loops without a token must be exactly zero"


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_gate_extremes(dtype):
    p = make_problem(custom(dtype=dtype))
    for val in (-np.inf, np.inf, -30.0, 30.0):
        q = p.with_(gate_logits=np.full_like(p.gate_logits, val))
        assert_parity(run_gpu(q), oracle.decode_attn(q), dtype, f"gate={val}")


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_loop_offsets_of_the_training_shift_reading(dtype):
    p = make_problem(custom(dtype=dtype, L=3, Hq=12, Hkv=2, loop_offset=[0, 0, 0]))
    assert_parity(run_gpu(p), oracle.decode_attn(p), dtype, "delta=0")
    p = make_problem(custom(dtype=dtype, L=3, Hq=12, Hkv=2, loop_offset=[0, 70, 200]))
    assert_parity(run_gpu(p), oracle.decode_attn(p), dtype, "delta=(0,70,200)")


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_explicit_window_lengths(dtype):
    p = make_problem(custom(dtype=dtype, B=4, L=3, Hq=12, Hkv=2, w=40, lens=("list", [300, 77, 5, 50])))
    wl = np.array([[40, 0], [1, 17], [3, 0], [16, 33]], dtype=np.int32)
    q = p.with_(win_lens=wl)
    assert_parity(run_gpu(q), oracle.decode_attn(q), dtype, "win_lens")


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_garbage_outside_valid_ranges_cannot_reach_the_output(dtype):
    spec = custom(dtype=dtype, B=4, L=3, Hq=12, Hkv=2, w=40, lens=("list", [300, 77, 5, 0]), max_seq_len=384)
    clean, dirty = make_problem(spec), make_problem(spec, tail_fill=float("nan"))
    a, b = run_gpu(clean), run_gpu(dirty)
    assert np.isfinite(b).all()
    np.testing.assert_array_equal(a, b)


def test_peaked_softmax_and_large_scores():
    p = make_problem(custom(B=2, L=2, lens=("list", [2000, 300]), peaks=0.02))
    assert_parity(run_gpu(p), oracle.decode_attn(p), "bf16", "peaks")
    big = p.with_(sm_scale=4.0)  # scores of magnitude ~50: softmax collapses onto a few keys
    assert_parity(run_gpu(big), oracle.decode_attn(big), "bf16", "large scores")


# ---- layouts ---------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("page_size", [16, 64, 128])
def test_paged_matches_oracle_and_contiguous(page_size):
    sp = shrunk_workload(4, B=9, lens=("list", [1, 2, 3, 63, 64, 255, 700, 129, 16]), page_size=page_size, w=100)
    p = make_problem(sp)
    ref = oracle.decode_attn(p)
    got = run_gpu(p)
    assert_parity(got, ref, "bf16", f"paged {page_size}")
    # the same tokens in a contiguous cache give bit-identical results when the tiling is the same
    cap = p.max_seq_len
    K = np.zeros((p.B, cap, p.Hkv, p.d), dtype=np.uint16)
    V = np.zeros_like(K)
    for b in range(p.B):
        for j0 in range(0, int(p.seq_lens[b]), page_size):
            n = min(page_size, int(p.seq_lens[b]) - j0)
            pid = p.page_table[b, j0 // page_size]
            K[b, j0:j0 + n] = p.k_cache[pid, :n]
            V[b, j0:j0 + n] = p.v_cache[pid, :n]
    flat = p.with_(k_cache=K, v_cache=V, page_table=None, page_size=0)
    got_flat = run_gpu(flat, key_slices=1, heads_per_cta=2)
    got_paged = run_gpu(p, key_slices=1, heads_per_cta=2)
    np.testing.assert_array_equal(got_flat, got_paged)


def test_strided_head_major_cache():
    p = make_problem(custom(B=3, L=2, Hq=8, Hkv=2, lens=("list", [300, 77, 1]), max_seq_len=320))
    ref = oracle.decode_attn(p)
    dp = DeviceProblem(p, "cuda:0")
    # [B, Hkv, N, d] storage viewed through strides
    k_hnd = dp.k_cache.permute(0, 2, 1, 3).contiguous()
    v_hnd = dp.v_cache.permute(0, 2, 1, 3).contiguous()
    dp.k_cache, dp.v_cache = k_hnd, v_hnd
    args = dp.args()
    args.kv_stride_b, args.kv_stride_h, args.kv_stride_n = p.Hkv * 320 * p.d, 320 * p.d, p.d
    from paper_2510_24824_b200 import binding as B
    with DecodeAttn(p) as op:
        B.plt_decode_attn_run(op.handle, args, torch.cuda.current_stream().cuda_stream)
        assert op.check() == 0
    assert_parity(dp.out.float().cpu().numpy().astype(np.float64), ref, "bf16", "HND strides")


# ---- boundary behaviour on a device --------------------------------------------------------------------------
def test_batch_smaller_than_capacity_and_guard_bands():
    p = make_problem(custom(B=3))
    ref = oracle.decode_attn(p)
    dp = DeviceProblem(p, "cuda:0")
    n = dp.out.numel()
    guard = torch.full((n + 2048,), 7.0, dtype=dp.out.dtype, device="cuda:0")
    out = guard[1024:1024 + n].view_as(dp.out)
    with DecodeAttn(p, max_batch=17) as op:
        op.run(dp, out=out)
        assert op.check() == 0
    assert_parity(out.float().cpu().numpy().astype(np.float64), ref, "bf16", "max_batch=17")
    assert torch.all(guard[:1024] == 7.0) and torch.all(guard[1024 + n:] == 7.0)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_workspace_reuse_across_different_batches(dtype):
    """One handle, a long batch and then a tiny one: partials left by the first run must not leak into the second
    (with fewer tiles than thread blocks some blocks own nothing and write nothing)."""
    big = make_problem(custom(dtype=dtype, B=6, L=3, Hq=12, Hkv=2, w=40, lens=("list", [3000, 2500, 4000, 3500, 2000, 3900]),
                              max_seq_len=4096))
    tiny = make_problem(custom(dtype=dtype, B=1, L=3, Hq=12, Hkv=2, w=40, lens=("list", [70]), max_seq_len=4096, seed=5))
    dbig, dtiny = DeviceProblem(big, "cuda:0"), DeviceProblem(tiny, "cuda:0")
    with DecodeAttn(big) as op:
        for _ in range(2):
            op.run(dbig)
            torch.cuda.synchronize()
            assert_parity(dbig.out.float().cpu().numpy().astype(np.float64), oracle.decode_attn(big), dtype, "big")
            op.run(dtiny)
            torch.cuda.synchronize()
            assert_parity(dtiny.out.float().cpu().numpy().astype(np.float64), oracle.decode_attn(tiny), dtype, "tiny")
        assert op.check() == 0


def test_repeated_runs_are_bitwise_identical():
    p = make_problem(shrunk_workload(2))
    dp = DeviceProblem(p, "cuda:0")
    with DecodeAttn(p) as op:
        a = op.run(dp).clone()
        for _ in range(3):
            b = op.run(dp)
            torch.cuda.synchronize()
            assert torch.equal(a, b)
        assert op.check() == 0


def test_out_of_range_device_values_are_clamped_and_flagged():
    from paper_2510_24824_b200 import binding as B
    p = make_problem(custom(B=3, lens=("list", [300, 77, 1]), max_seq_len=320))
    bad = p.with_(seq_lens=np.array([300, 100000, -5], dtype=np.int32))
    dp = DeviceProblem(bad, "cuda:0")
    with DecodeAttn(bad) as op:
        op.run(dp)
        bits = op.check()
        assert bits & B.PLT_DEV_SEQ_LEN_CLAMPED
        assert op.check() == 0  # cleared
    clamped = p.with_(seq_lens=np.array([300, 320, 0], dtype=np.int32))
    assert_parity(dp.out.float().cpu().numpy().astype(np.float64), oracle.decode_attn(clamped), "bf16", "clamped")


def test_run_argument_errors():
    from paper_2510_24824_b200 import binding as B
    p = make_problem(custom(B=3))
    dp = DeviceProblem(p, "cuda:0")
    with DecodeAttn(p) as op:
        stream = torch.cuda.current_stream().cuda_stream
        a = dp.args(); a.batch = 4
        with pytest.raises(B.PltError) as e:
            B.plt_decode_attn_run(op.handle, a, stream)
        assert e.value.status == B.PLT_ERR_CAPACITY
        a = dp.args(); a.q = None
        with pytest.raises(B.PltError) as e:
            B.plt_decode_attn_run(op.handle, a, stream)
        assert e.value.status == B.PLT_ERR_INVALID_ARG
        a = dp.args(); a.k_cache = dp.k_cache.data_ptr() + 2
        with pytest.raises(B.PltError) as e:
            B.plt_decode_attn_run(op.handle, a, stream)
        assert e.value.status == B.PLT_ERR_INVALID_ARG
        a = dp.args(); a.kv_stride_b, a.kv_stride_n, a.kv_stride_h = 1000, 3, 128
        with pytest.raises(B.PltError) as e:
            B.plt_decode_attn_run(op.handle, a, stream)
        assert e.value.status == B.PLT_ERR_INVALID_ARG
        a = dp.args(); a.batch = 0
        B.plt_decode_attn_run(op.handle, a, stream)  # empty batch: nothing to do
        op.run(dp)
        assert op.check() == 0
    assert_parity(dp.out.float().cpu().numpy().astype(np.float64), oracle.decode_attn(p), "bf16", "after errors")


@pytest.mark.parametrize("index,kv", [(0, ""), (1, ""), (4, ""), (1, "e4m3"), (4, "e4m3")])
def test_host_buffer_entry_point(index, kv):
    p = make_problem(shrunk_workload(index, kv_dtype=kv))
    hp = DeviceProblem(p, device=None, pin=True)
    with DecodeAttn(p) as op:
        out = op.run_host(hp)
        out2 = op.run_host(hp).clone()
        assert op.check() == 0
    assert torch.equal(out, out2)
    assert_parity(out.float().numpy().astype(np.float64), oracle.decode_attn(p), p.dtype, "run_host")


def test_back_to_back_steps_on_one_handle_do_not_disturb_each_other():
    """Consecutive launches overlap at their edges (the merge kernel's and the next main kernel's set-up start early):
    two different batches alternated on one handle, 40 runs with no host synchronisation in between, must each
    give exactly what they give alone."""
    big = make_problem(custom(B=6, L=3, Hq=12, Hkv=2, w=40, lens=("list", [3000, 2500, 4000, 3500, 2000, 3900]), max_seq_len=4096))
    small = make_problem(custom(B=2, L=3, Hq=12, Hkv=2, w=40, lens=("list", [70, 5]), max_seq_len=4096, seed=5))
    dbig, dsmall = DeviceProblem(big, "cuda:0"), DeviceProblem(small, "cuda:0")
    with DecodeAttn(big) as op:
        op.run(dbig)
        op.run(dsmall)
        torch.cuda.synchronize()
        alone_big, alone_small = dbig.out.clone(), dsmall.out.clone()
        outs = []
        for i in range(40):
            dp = dbig if i % 2 == 0 else dsmall
            o = torch.full_like(dp.out, float("nan"))
            op.run(dp, out=o)
            outs.append(o)
        torch.cuda.synchronize()
        assert op.check() == 0
    for i, o in enumerate(outs):
        assert torch.equal(o, alone_big if i % 2 == 0 else alone_small), f"run {i} differs"
    assert_parity(alone_big.float().cpu().numpy().astype(np.float64), oracle.decode_attn(big), "bf16", "big")


@pytest.mark.parametrize("kv", ["", "e4m3"])
def test_maximum_batch_of_short_sequences(kv):
    """4096 sequences (the largest batch a handle takes) of 0..70 tokens: thousands of items, most blocks hold dozens."""
    p = make_problem(custom(B=4096, L=3, Hq=8, Hkv=2, w=24, lens=("uniform", 0, 70), kv_dtype=kv, seed=3))
    assert_parity(run_gpu(p), oracle.decode_attn(p), "bf16", f"B=4096 {kv}")


def test_runs_can_be_captured_in_a_cuda_graph():
    """plt_decode_attn_run allocates nothing and never synchronises: a stream capture records its two launches (with
    their programmatic dependencies) and replays give the same bits."""
    p = make_problem(custom(B=6, L=3, Hq=12, Hkv=2, w=40, lens=("list", [3000, 2500, 4000, 3500, 2000, 3900]), max_seq_len=4096))
    dp = DeviceProblem(p, "cuda:0")
    with DecodeAttn(p) as op:
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            op.run(dp, stream=side.cuda_stream)       # first call encodes the tensor maps (host work, not captured)
        torch.cuda.synchronize()
        want = dp.out.clone()
        dp.out.zero_()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for _ in range(3):
                op.run(dp, stream=torch.cuda.current_stream().cuda_stream)
        for _ in range(4):
            graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(dp.out, want)
        assert op.check() == 0
    assert_parity(want.float().cpu().numpy().astype(np.float64), oracle.decode_attn(p), "bf16", "graph")


@pytest.mark.parametrize("kv", ["", "e4m3"])
def test_one_very_long_sequence(kv):
    """A single sequence of 131069 tokens: one item split over every block of the grid, merged from hundreds of pieces."""
    p = make_problem(custom(B=1, L=2, Hq=8, Hkv=2, w=64, lens=("list", [131069]), kv_dtype=kv, seed=9))
    assert_parity(run_gpu(p), oracle.decode_attn(p), "bf16", f"N=131069 {kv}")


# ---- the workload with tripled K/V rows under every launch variant ----------------------------------------------
# Sharp softmax peaks on large values are where the rounding of the probabilities shows most (outputs of magnitude
# 4-8 next to the 2e-2 bound); every accepted variant has to stay inside the bound there, three seeds each.
@pytest.mark.parametrize("hpc,kw,ks", [(0, 0, 0), (1, 1, 1), (1, 2, 1), (1, 4, 1), (2, 1, 1), (2, 2, 1), (2, 4, 1), (4, 1, 1),
                                       (4, 2, 1), (8, 1, 1), (1, 8, 1), (1, 1, 2), (2, 2, 2), (4, 1, 2), (1, 4, 2)])
def test_peaked_workload_under_every_variant(hpc, kw, ks):
    worst = 0.0
    for seed in (2, 12, 22):
        p = make_problem(shrunk_workload(2), seed=seed)
        ref = oracle.decode_attn(p)
        got = run_gpu(p, heads_per_cta=hpc, key_slices=kw, slices_per_warp=ks)
        assert_parity(got, ref, "bf16", f"peaks hpc={hpc} kw={kw} ks={ks} seed={seed}")
        worst = max(worst, parity_report(got, ref, "bf16")["worst_of_bound"])
    print(f"peaked workload hpc={hpc} kw={kw} ks={ks}: worst error / bound {worst:.2f}")


# ---- several handles that share one kernel instance ---------------------------------------------------------------
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_two_handles_of_one_variant_with_different_shared_memory(dtype):
    """The shared-memory limit of a kernel belongs to the function, not to a handle: a second, smaller handle of the
    same variant must not lower it under the first (its shared memory grows with max_batch)."""
    p = make_problem(custom(dtype=dtype, B=3))
    ref = oracle.decode_attn(p)
    dp = DeviceProblem(p, "cuda:0")
    with DecodeAttn(p, max_batch=4096) as big, DecodeAttn(p, max_batch=8) as small:
        for op in (big, small, big, small, big):
            dp.out.fill_(float("nan"))
            op.run(dp)
            assert op.check() == 0
            assert_parity(dp.out.float().cpu().numpy().astype(np.float64), ref, dtype, "two handles")
