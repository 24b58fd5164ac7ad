"""The ablation legs of Table 1 at kernel level give the same numbers as the fused step with its gate closed.

Sequential single-loop calls over the shared cache (the loop order of the vanilla loop transformer) and one
cross-loop-parallel call over L private caches ("Loop+CLP" before KV sharing) both compute, per loop, the global
attention of Algorithm 3 on that loop's visible keys; with gate logits of -inf the library's step computes the
same thing in one launch over one cache. All three are held to the oracle.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_24824_b200.inputs import make_problem, shrunk_workload
from paper_2510_24824_b200.runner import DecodeAttn, DeviceProblem, LoopOrderAblation

from gpu_util import assert_parity

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("index,kv", [(1, ""), (2, ""), (3, ""), (4, ""), (2, "e4m3"), (4, "e4m3")])
def test_sequential_and_private_cache_legs_match_the_closed_gate_step(index, kv):
    p = make_problem(shrunk_workload(index, kv_dtype=kv))
    closed = p.with_(gate_logits=np.full_like(p.gate_logits, -np.inf))
    ref = oracle.decode_attn(closed)                       # [B, L, Hq, d]: the global part of every loop
    dp = DeviceProblem(closed, "cuda:0")
    with DecodeAttn(closed) as op:
        fused = op.run(dp).float().cpu().numpy().astype(np.float64)
        assert op.check() == 0
    assert_parity(fused, ref, "bf16", "fused step, gate closed")
    abl = LoopOrderAblation(closed, dp)
    try:
        seq = torch.cat(abl.run_sequential(), dim=1).float().cpu().numpy().astype(np.float64)
        priv = abl.run_private().reshape(p.B, p.L, p.Hq, p.d).float().cpu().numpy().astype(np.float64)
        assert abl.check() == 0
    finally:
        abl.close()
    assert_parity(seq, ref, "bf16", "L sequential single-loop calls")
    assert_parity(priv, ref, "bf16", "one call over L private caches")
    # the three agree with each other to rounding (different packings of the rows, same products)
    assert np.abs(seq - fused).max() <= 2e-2 and np.abs(priv - fused).max() <= 2e-2
