"""The allocation-free entry point against the handle-based one.

Some users of the library cannot allocate device memory when they need the attention (a serving process whose
HBM is fully committed to the KV cache, a plug-in that only receives tensors). plt_decode_attn_run_no_alloc
serves them from a scratch array built into the library. This test calls it through the C ABI twice in a row
(the array keeps the first call's contents, so the second call shows that nothing stale is read) and compares
both results with plt_decode_attn_run on the same inputs (same kernels, same plan: bit for bit) and with the fp64
oracle. A second test alternates two configurations on the shared array, so that partials and block tables left by a
different layout are what each call finds. It is collected last so that a run stopping at the first failure has
already exercised everything else.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_24824_b200 import binding as B
from paper_2510_24824_b200.inputs import make_problem, shrunk_workload
from paper_2510_24824_b200.runner import DecodeAttn, DeviceProblem

from gpu_util import assert_parity

pytestmark = pytest.mark.gpu


def config_for(p):
    return B.make_config(p.dtype, p.B, p.L, p.Hq, p.Hkv, p.d, p.max_seq_len, p.w, page_size=p.page_size,
                         sm_scale=p.sm_scale, device=0)


@pytest.mark.parametrize("index", [1, 0, 4])
def test_no_alloc_matches_handle_path_twice(index):
    torch.cuda.set_device(0)
    p = make_problem(shrunk_workload(index))
    dp = DeviceProblem(p, "cuda:0")
    stream = torch.cuda.current_stream().cuda_stream
    with DecodeAttn(p) as op:
        op.run(dp)
        assert op.check() == 0
    want_bits = dp.out.clone()
    ref = oracle.decode_attn(p)

    cfg = config_for(p)
    assert B.plt_decode_attn_workspace_bytes(cfg) <= B.PLT_NO_ALLOC_SCRATCH_BYTES
    out = torch.empty_like(dp.out)
    for call in range(2):
        out.fill_(float("nan"))
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated()
        B.plt_decode_attn_run_no_alloc(cfg, dp.args(out), stream)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        assert B.plt_decode_attn_check(None, stream) == 0     # the status word of the built-in array
        assert torch.equal(out, want_bits), f"{p.name} call {call}: differs from the handle path"
        assert_parity(out.float().cpu().numpy().astype(np.float64), ref, p.dtype, f"{p.name} call {call}")


def test_no_alloc_alternating_configurations_share_the_array():
    """bf16, fp32, paged bf16 and back: every call finds the previous layout's partials, prefix and block table."""
    torch.cuda.set_device(0)
    stream = torch.cuda.current_stream().cuda_stream
    cases = []
    for index in (1, 0, 4):
        p = make_problem(shrunk_workload(index))
        cases.append((p, DeviceProblem(p, "cuda:0"), config_for(p), oracle.decode_attn(p)))
    for round_ in range(2):
        for p, dp, cfg, ref in cases:
            dp.out.fill_(float("nan"))
            B.plt_decode_attn_run_no_alloc(cfg, dp.args(), stream)
            assert B.plt_decode_attn_check(None, stream) == 0
            assert_parity(dp.out.float().cpu().numpy().astype(np.float64), ref, p.dtype, f"{p.name} round {round_}")


def test_no_alloc_status_word_is_readable_without_a_handle():
    torch.cuda.set_device(0)
    stream = torch.cuda.current_stream().cuda_stream
    p = make_problem(shrunk_workload(1))
    bad = p.with_(seq_lens=np.array([p.max_seq_len + 5] * p.B, dtype=np.int32))   # clamped to the capacity, flagged
    dp = DeviceProblem(bad, "cuda:0")
    B.plt_decode_attn_run_no_alloc(config_for(p), dp.args(), stream)
    assert B.plt_decode_attn_check(None, stream) == B.PLT_DEV_SEQ_LEN_CLAMPED
    assert B.plt_decode_attn_check(None, stream) == 0     # reading clears it


def test_no_alloc_rejects_what_does_not_fit():
    torch.cuda.set_device(0)
    big = B.make_config("bf16", 4096, 4, 64, 8, 128, 32768, 512, device=0)
    assert B.plt_decode_attn_workspace_bytes(big) > B.PLT_NO_ALLOC_SCRATCH_BYTES
    p = make_problem(shrunk_workload(1))
    dp = DeviceProblem(p, "cuda:0")
    with pytest.raises(B.PltError) as e:
        B.plt_decode_attn_run_no_alloc(big, dp.args(), torch.cuda.current_stream().cuda_stream)
    assert e.value.status == B.PLT_ERR_CAPACITY
    assert str(B.PLT_NO_ALLOC_SCRATCH_BYTES) in e.value.message
