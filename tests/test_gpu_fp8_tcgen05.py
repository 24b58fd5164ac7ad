"""GPU parity of the tcgen05 main kernel for E4M3 caches (config.kv_dtype = PLT_KV_E4M3 with kernel_path =
PLT_PATH_TCGEN05: products on the codes themselves, queries as two and probabilities as three E4M3 terms) through the
C ABI against the oracle. Same tolerance as every bf16-query path."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_24824_b200 import binding as B
from paper_2510_24824_b200.inputs import bf16_bits_to_f32, f32_to_bf16_bits, make_problem, shrunk_workload
from paper_2510_24824_b200.runner import DecodeAttn, DeviceProblem

from gpu_util import inactive_rows, assert_parity, parity_report, run_gpu

pytestmark = pytest.mark.gpu

T5 = dict(kernel_path=B.PLT_PATH_TCGEN05)


def custom(**kw):
    base = dict(name="fp8-t5", dtype="bf16", kv_dtype="e4m3", B=3, L=2, Hq=8, Hkv=2, d=128, w=40, lens=("list", [300, 77, 1]),
                gate_std=1.0, peaks=0.0, page_size=0, seed=41)
    base.update(kw)
    return base


def test_path_is_reported():
    p = make_problem(custom())
    with DecodeAttn(p, **T5) as op:
        assert op.info["kernel_path"] == B.PLT_PATH_TCGEN05
        assert op.info["kernels_per_run"] == 3


def test_automatic_choice_for_long_unpaged_caches_at_32_rows():
    """E4M3 caches at 25 to 32 packed rows that can reach 8192 keys (contiguous, in pages that hold whole tiles or in
    pages of 64 tokens), or at 17 to 24 rows that can reach 32768 (pages of 64 left out): the library picks this kernel
    by itself."""
    spec = custom(B=2, L=4, Hq=16, Hkv=2, w=90, lens=("list", [900, 130]), max_seq_len=32768)
    p = make_problem(spec)
    with DecodeAttn(p) as op:
        assert op.info["kernel_path"] == B.PLT_PATH_TCGEN05 and op.info["heads_per_cta"] == 2
    assert_parity(run_gpu(p), oracle.decode_attn(p), "bf16", "automatic")
    for page_size in (256, 64):
        paged = make_problem(dict(spec, page_size=page_size))
        with DecodeAttn(paged) as op:
            assert op.info["kernel_path"] == B.PLT_PATH_TCGEN05
        assert_parity(run_gpu(paged), oracle.decode_attn(paged), "bf16", f"automatic, pages of {page_size}")
    rows24 = make_problem(custom(B=2, L=3, Hq=16, Hkv=2, w=90, lens=("list", [900, 130]), max_seq_len=32768))
    with DecodeAttn(rows24) as op:
        assert op.info["kernel_path"] == B.PLT_PATH_TCGEN05
    assert_parity(run_gpu(rows24), oracle.decode_attn(rows24), "bf16", "automatic, 24 rows")
    # a length the caller expects most sequences to reach decides instead of the capacity
    hinted = make_problem(custom(B=2, L=4, Hq=16, Hkv=2, w=90, lens=("list", [2100, 2050]), max_seq_len=4096))
    with DecodeAttn(hinted, typical_seq_len=2048) as op:
        assert op.info["kernel_path"] == B.PLT_PATH_TCGEN05
    with DecodeAttn(hinted) as op:
        assert op.info["kernel_path"] == B.PLT_PATH_WARP_MMA
    assert_parity(run_gpu(hinted, typical_seq_len=2048), oracle.decode_attn(hinted), "bf16", "automatic with a typical length")
    with DecodeAttn(make_problem(spec), typical_seq_len=512) as op:
        assert op.info["kernel_path"] == B.PLT_PATH_WARP_MMA
    for other in (custom(B=2, L=3, Hq=16, Hkv=2, w=90, lens=("list", [900, 130]), max_seq_len=16384),     # 24 rows, shorter caches
                  custom(B=2, L=2, Hq=16, Hkv=2, w=90, lens=("list", [900, 130]), max_seq_len=32768),     # 16 rows
                  custom(B=2, L=4, Hq=16, Hkv=2, w=90, lens=("list", [900, 130]), max_seq_len=4096),      # 32 rows, short caches
                  custom(B=2, L=3, Hq=16, Hkv=2, w=90, lens=("list", [900, 130]), max_seq_len=32768, page_size=64),   # 24 rows
                  custom(B=2, L=4, Hq=16, Hkv=2, w=90, lens=("list", [900, 130]), max_seq_len=32768, page_size=32)):
        with DecodeAttn(make_problem(other)) as op:
            assert op.info["kernel_path"] == B.PLT_PATH_WARP_MMA


@pytest.mark.parametrize("index", [1, 2, 3, 4])
def test_shrunk_workloads(index):
    p = make_problem(shrunk_workload(index, kv_dtype="e4m3"))
    assert_parity(run_gpu(p, **T5), oracle.decode_attn(p), "bf16", p.name)


@pytest.mark.parametrize("spec", [
    custom(B=3, L=1, w=0, lens=("list", [129, 1, 64])),                                      # single loop
    custom(B=4, L=3, Hq=32, Hkv=8, w=70, lens=("list", [513, 64, 2, 1000])),                 # 12 packed rows
    custom(B=3, L=3, Hq=32, Hkv=4, w=50, lens=("list", [700, 65, 3])),                       # 24 packed rows
    custom(B=3, L=4, Hq=32, Hkv=4, w=90, lens=("list", [900, 130, 2])),                      # 32 packed rows
    custom(B=3, L=2, Hq=34, Hkv=2, w=90, lens=("list", [900, 130, 2])),                      # 34 rows: refused
    custom(B=8, L=4, Hq=8, Hkv=2, w=32, lens=("list", [0, 1, 2, 3, 4, 31, 32, 33])),         # fewer tokens than loops
    custom(B=2, L=3, Hq=8, Hkv=2, w=300, lens=("list", [2000, 290])),                        # windows of several tiles
    custom(B=3, L=3, Hq=12, Hkv=2, loop_offset=[0, 70, 200]),                                # other causal offsets
    custom(B=5, L=2, Hq=16, Hkv=8, w=64, lens=("list", [5000, 4097, 128, 127, 129])),        # tile edges, many tiles
], ids=["L1", "R12", "R24", "R32", "R34", "short", "wide-window", "offsets", "edges"])
def test_shapes_and_edges(spec):
    p = make_problem(spec)
    if p.L * (p.Hq // p.Hkv) > 32:
        with pytest.raises(B.PltError):
            DecodeAttn(p, **T5)
        return
    got = run_gpu(p, **T5)
    assert_parity(got, oracle.decode_attn(p), "bf16", spec.get("name", ""))
    assert np.all(got[inactive_rows(p)] == 0.0), "rows of loops without a token must be exactly zero"


@pytest.mark.parametrize("hpc", [1, 2])
@pytest.mark.parametrize("spec", [
    custom(B=3, L=3, Hq=32, Hkv=4, w=50, lens=("list", [700, 65, 3])),                       # 24 packed rows
    custom(B=2, L=3, Hq=8, Hkv=2, w=300, lens=("list", [2000, 290])),                        # windows of several tiles
    custom(B=9, L=4, Hq=32, Hkv=4, w=100, page_size=64, lens=("list", [1, 2, 3, 63, 64, 255, 700, 129, 16])),
], ids=["R24", "wide-window", "paged"])
def test_heads_per_item(spec, hpc):
    """One or two KV heads per work item (two: their tiles of the same keys take turns in one block)."""
    p = make_problem(spec)
    with DecodeAttn(p, heads_per_cta=hpc, **T5) as op:
        assert op.info["heads_per_cta"] == hpc
    assert_parity(run_gpu(p, heads_per_cta=hpc, **T5), oracle.decode_attn(p), "bf16", f"hpc={hpc}")


def test_odd_number_of_kv_heads_takes_one_head_per_item():
    p = make_problem(custom(B=3, L=2, Hq=12, Hkv=3, lens=("list", [700, 65, 3])))
    with DecodeAttn(p, **T5) as op:
        assert op.info["heads_per_cta"] == 1
    with pytest.raises(B.PltError):
        DecodeAttn(p, heads_per_cta=2, **T5)
    assert_parity(run_gpu(p, **T5), oracle.decode_attn(p), "bf16", "Hkv=3")


@pytest.mark.parametrize("stages,inflight", [(7, 1), (8, 2), (8, 4)])
def test_ring_depths(stages, inflight):
    p = make_problem(custom(B=3, L=3, Hq=24, Hkv=4, w=50, lens=("list", [1700, 65, 3])))
    got = run_gpu(p, stages=stages, loads_in_flight=inflight, **T5)
    assert_parity(got, oracle.decode_attn(p), "bf16", f"stages={stages}")


def test_scales_reach_the_kernel_per_head():
    p = make_problem(custom(B=2, L=2, Hq=8, Hkv=2, lens=("list", [200, 31])))
    q = p.with_(k_scale=(p.k_scale * np.array([0.5, 3.0])).astype(np.float32),
                v_scale=(p.v_scale * np.array([2.0, 0.25])).astype(np.float32))
    assert_parity(run_gpu(q, **T5), oracle.decode_attn(q), "bf16", "rescaled")


@pytest.mark.parametrize("qscale", [2.0 ** -12, 1.0, 37.0, 2.0 ** 10])
def test_query_magnitudes(qscale):
    """The queries are rescaled by a power of two per (sequence, KV head) before they are split into two E4M3 terms:
    the result must not depend on their magnitude (the softmax scale is divided by the same factor here)."""
    p = make_problem(custom(B=2, L=3, Hq=12, Hkv=2, lens=("list", [700, 131])))
    q2 = f32_to_bf16_bits((bf16_bits_to_f32(p.q) * np.float32(qscale)).astype(np.float32))
    big = p.with_(q=q2, sm_scale=p.scale() / qscale)
    assert_parity(run_gpu(big, **T5), oracle.decode_attn(big), "bf16", f"q x {qscale}")


def test_rows_of_very_different_magnitude_share_one_scale():
    p = make_problem(custom(B=2, L=2, Hq=16, Hkv=2, lens=("list", [600, 90])))
    q = bf16_bits_to_f32(p.q).copy()
    q[:, :, 0::2] *= np.float32(2.0 ** -7)   # every other head 128 times smaller: its low term reaches the subnormal codes
    small = p.with_(q=f32_to_bf16_bits(q))
    assert_parity(run_gpu(small, **T5), oracle.decode_attn(small), "bf16", "mixed magnitudes")


def test_pages_of_half_a_tile_with_every_kind_of_last_tile():
    """Pages of 64 tokens are two loads per tile, the second only when that page holds data: lengths that end in the
    first half of a tile, exactly at its middle, in the second half and at its end, on one and on several tiles."""
    lens = [1, 63, 64, 65, 127, 128, 129, 191, 192, 193, 1000, 1024, 1087, 1088, 1089]
    for L, Hq in ((4, 16), (3, 6), (1, 4)):
        p = make_problem(custom(B=len(lens), L=L, Hq=Hq, Hkv=2, w=70, lens=("list", lens), page_size=64, max_seq_len=1152))
        assert_parity(run_gpu(p, **T5), oracle.decode_attn(p), "bf16", f"pages of 64, L={L}")


@pytest.mark.parametrize("page_size", [64, 128, 256])
def test_paged_cache(page_size):
    p = make_problem(shrunk_workload(4, kv_dtype="e4m3", B=9, lens=("list", [1, 2, 3, 63, 64, 255, 700, 129, 16]),
                                     page_size=page_size, w=100))
    assert_parity(run_gpu(p, **T5), oracle.decode_attn(p), "bf16", f"paged {page_size}")


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
    a = run_gpu(p, **T5)
    b_ = run_gpu(p.with_(k_cache=dirty_k, v_cache=dirty_v, k_win=kw_, v_win=vw_), **T5)
    assert np.isfinite(b_).all()
    np.testing.assert_array_equal(a, b_)


def test_peaked_softmax_and_large_scores():
    worst = 0.0
    for seed in (2, 12, 22):
        p = make_problem(shrunk_workload(2, kv_dtype="e4m3"), seed=seed)   # tripled K/V rows: sharp peaks on large values
        ref = oracle.decode_attn(p)
        got = run_gpu(p, **T5)
        assert_parity(got, ref, "bf16", f"peaks seed={seed}")
        worst = max(worst, parity_report(got, ref, "bf16")["worst_of_bound"])
    print(f"peaked workload, tcgen05 E4M3: worst error / bound {worst:.2f}")
    # Scores of magnitude ~50: the softmax collapses onto a few keys and the reference maximum moves often. The outputs
    # are then single V rows of magnitude 1-4, whose rounding to bf16 alone has a mean of 2.2e-3: the element-wise
    # bound applies as always, the mean is held to that rounding plus 1e-4.
    p = make_problem(custom(B=2, L=2, lens=("list", [2000, 300]), peaks=0.02))
    big = p.with_(sm_scale=4.0)
    ref = oracle.decode_attn(big)
    got = run_gpu(big, **T5)
    rep = parity_report(got, ref, "bf16")
    assert np.isfinite(got).all() and rep["worst_of_bound"] <= 1.0, rep
    rounding = np.abs(torch.tensor(ref).to(torch.bfloat16).double().numpy() - ref).mean()
    assert rep["mean_abs"] <= rounding + 1e-4, (rep["mean_abs"], rounding)


def test_repeated_runs_are_bitwise_identical_and_match_the_warp_level_kernel_closely():
    p = make_problem(shrunk_workload(3, kv_dtype="e4m3"))
    dp = DeviceProblem(p, "cuda:0")
    with DecodeAttn(p, **T5) as op:
        a = op.run(dp).clone()
        for _ in range(3):
            b = op.run(dp)
            torch.cuda.synchronize()
            assert torch.equal(a, b)
        assert op.check() == 0
    warp = run_gpu(p)
    assert np.abs(a.float().cpu().numpy() - warp).max() < 2e-2


def test_batch_smaller_than_capacity_and_reuse():
    big = make_problem(custom(B=6, L=3, Hq=12, Hkv=2, w=40, lens=("list", [3000, 2500, 4000, 3500, 2000, 3900]), max_seq_len=4096))
    tiny = make_problem(custom(B=1, L=3, Hq=12, Hkv=2, w=40, lens=("list", [70]), max_seq_len=4096, seed=5))
    with DecodeAttn(big, **T5) as op:
        for prob in (big, tiny, big):
            dp = DeviceProblem(prob, "cuda:0")
            got = op.run(dp).float().cpu().numpy().astype(np.float64)
            assert_parity(got, oracle.decode_attn(prob), "bf16", f"B={prob.B}")
        assert op.check() == 0


def test_allocation_free_entry_point_with_this_kernel():
    """plt_decode_attn_run_no_alloc places the query images and their scale factors in the built-in scratch array too."""
    torch.cuda.set_device(0)
    p = make_problem(custom(B=3, L=3, Hq=24, Hkv=4, w=50, lens=("list", [1700, 65, 3])))
    dp = DeviceProblem(p, "cuda:0")
    stream = torch.cuda.current_stream().cuda_stream
    with DecodeAttn(p, **T5) as op:
        want = op.run(dp).clone()
        assert op.check() == 0
    cfg = B.make_config(p.dtype, p.B, p.L, p.Hq, p.Hkv, p.d, p.max_seq_len, p.w, page_size=p.page_size, sm_scale=p.sm_scale,
                        device=0, kv_dtype=p.kv_dtype, **T5)
    assert B.plt_decode_attn_workspace_bytes(cfg) <= B.PLT_NO_ALLOC_SCRATCH_BYTES
    out = torch.empty_like(dp.out)
    for call in range(2):
        out.fill_(float("nan"))
        B.plt_decode_attn_run_no_alloc(cfg, dp.args(out), stream)
        torch.cuda.synchronize()
        assert B.plt_decode_attn_check(None, stream) == 0
        assert torch.equal(out, want), f"call {call}: differs from the handle path"
    assert_parity(out.float().cpu().numpy().astype(np.float64), oracle.decode_attn(p), "bf16", "no-alloc")


def test_explicit_window_lengths():
    p = make_problem(custom(B=4, L=3, Hq=12, Hkv=2, w=40, lens=("list", [300, 77, 5, 50])))
    wl = np.array([[40, 0], [1, 17], [3, 0], [16, 33]], dtype=np.int32)
    q = p.with_(win_lens=wl)
    assert_parity(run_gpu(q, **T5), oracle.decode_attn(q), "bf16", "win_lens")


def test_out_of_range_device_values_are_clamped_and_flagged():
    p = make_problem(custom(B=3, lens=("list", [300, 77, 1]), max_seq_len=320))
    bad = p.with_(seq_lens=np.array([300, 100000, -5], dtype=np.int32))
    dp = DeviceProblem(bad, "cuda:0")
    with DecodeAttn(bad, **T5) as op:
        op.run(dp)
        bits = op.check()
        assert bits & B.PLT_DEV_SEQ_LEN_CLAMPED and not bits & B.PLT_DEV_WAIT_TIMEOUT
        assert op.check() == 0  # cleared
    clamped = p.with_(seq_lens=np.array([300, 320, 0], dtype=np.int32))
    assert_parity(dp.out.float().cpu().numpy().astype(np.float64), oracle.decode_attn(clamped), "bf16", "clamped")
    # page ids outside the pool: clamped and flagged, on pages that hold whole tiles and on smaller ones
    for page_size in (128, 64):
        pp = make_problem(custom(B=2, L=2, Hq=8, Hkv=2, lens=("list", [700, 130]), page_size=page_size))
        table = pp.page_table.copy()
        table[0, 1] = 10 ** 6
        table[1, 0] = -3
        dq = DeviceProblem(pp.with_(page_table=table), "cuda:0")
        with DecodeAttn(pp, **T5) as op:
            op.run(dq)
            bits = op.check()
            assert bits & B.PLT_DEV_PAGE_ID_CLAMPED and not bits & B.PLT_DEV_WAIT_TIMEOUT
        as_clamped = pp.with_(page_table=np.clip(table, 0, pp.num_pool_pages - 1).astype(np.int32))
        assert_parity(dq.out.float().cpu().numpy().astype(np.float64), oracle.decode_attn(as_clamped), "bf16",
                      f"clamped page ids, pages of {page_size}")


def test_runs_can_be_captured_in_a_cuda_graph():
    """Three launches per run on this path (query pack, main with its programmatic dependency, merge): a stream
    capture records them and replays give the same bits."""
    p = make_problem(custom(B=6, L=4, Hq=16, Hkv=2, w=40, lens=("list", [3000, 2500, 4000, 3500, 2000, 3900]), max_seq_len=4096))
    dp = DeviceProblem(p, "cuda:0")
    with DecodeAttn(p, **T5) as op:
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


def test_decode_step_with_pre_step_on_this_path():
    """plt_decode_attn_step (cache append with quantisation, window ring update, gate linear) ahead of this kernel: the
    main kernel's loads may start while the query pack kernel runs, but never before the pre-step has finished."""
    import test_gpu_prestep as TP
    for spec in (custom(B=3, L=3, Hq=24, Hkv=4, w=50, lens=("list", [1700, 65, 3])),
                 custom(B=4, L=4, Hq=16, Hkv=4, w=16, lens=("list", [16, 17, 33, 500]))):
        p = make_problem(spec)
        rows = TP.new_rows(p, 9)
        dp = DeviceProblem(p, "cuda:0")
        with DecodeAttn(p, **T5) as op:
            got = TP.run_step(p, op, dp, *rows)
        TP.check_against_oracle(p, dp, got, *rows, what="step on the tcgen05 path")
