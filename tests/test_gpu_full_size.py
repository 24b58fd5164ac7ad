"""Parity at the full sizes of the bf16 workloads, in the launch configuration bench.py times (automatic variant),
on sampled output rows the oracle computes one by one, plus properties that hold at any size."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_24824_b200 import binding as B
from paper_2510_24824_b200.inputs import make_problem, workload
from paper_2510_24824_b200.runner import DecodeAttn, DeviceProblem

from gpu_util import inactive_rows, BF16_MEAN_ABS, bf16_bound

pytestmark = pytest.mark.gpu


def sample_rows(p, n, rng, forced=()):
    rows = {tuple(r) for r in forced}
    while len(rows) < n:
        rows.add((int(rng.integers(p.B)), int(rng.integers(p.L)), int(rng.integers(p.Hq))))
    return np.array(sorted(rows), dtype=np.int32)


# (workload index, cache type, page size or None for the workload's own): the E4M3 form of the long-context workload
# runs on the tcgen05 kernel for E4M3, contiguous and in pages of 64 tokens (its two-boxes-per-tile variant)
@pytest.mark.parametrize("index,kv,page_size", [(1, "", None), (2, "", None), (3, "", None), (4, "", None), (1, "e4m3", None),
                                                (4, "e4m3", None), (3, "e4m3", None), (3, "e4m3", 64)])
def test_full_size_sampled_rows(index, kv, page_size):
    spec = dict(workload(index), kv_dtype=kv)
    if page_size is not None:
        spec["page_size"] = page_size
    p = make_problem(spec)
    dp = DeviceProblem(p, "cuda:0")
    dp.out.fill_(float("nan"))
    with DecodeAttn(p) as op:
        if index == 3 and kv:
            assert op.info["kernel_path"] == B.PLT_PATH_TCGEN05
        op.run(dp)
        assert op.check() == 0
        first = dp.out.clone()
        op.run(dp)
        assert op.check() == 0
    assert torch.equal(first, dp.out), "two runs on the same inputs differ"
    got = dp.out.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    # convexity: every output lies within the range of the values it can mix
    if kv:   # E4M3 codes: the largest finite code value is 448, times the largest V scale
        vmax = 448.0 * float(p.v_scale.max())
    else:
        vmax = float(max(dp.v_cache.float().abs().max().item(), dp.v_win.float().abs().max().item()))
    assert np.abs(got).max() <= vmax * (1 + 2 ** -7)
    inactive = inactive_rows(p)
    assert np.all(got[inactive] == 0.0)

    rng = np.random.default_rng(100 + index)
    forced = []
    if index == 4:  # the short sequences (N < L, N < w, page boundary) in every loop
        forced = [(b, l, h) for b in range(6) for l in range(p.L) for h in (0, p.Hq - 1)]
        forced += [(int(np.argmax(p.seq_lens)), l, 5) for l in range(p.L)]
    if index == 2:
        forced = [(int(np.argmax(p.seq_lens)), l, 3) for l in range(p.L)] + [(int(np.argmin(p.seq_lens)), l, 9) for l in range(p.L)]
    rows = sample_rows(p, 96, rng, forced)
    ref = oracle.decode_attn_rows(p, rows)
    sel = got[rows[:, 0], rows[:, 1], rows[:, 2]]
    err = np.abs(sel - ref)
    assert (err / bf16_bound(ref)).max() <= 1.0, f"{p.name}: max abs err {err.max():.3e}"
    assert err.mean() <= BF16_MEAN_ABS, f"{p.name}: mean abs err {err.mean():.3e}"
