"""GPU parity of plt_decode_attn_step (pre-step + attention) through the C ABI against the oracle: the caches and
windows after the call bit for bit, the gate logits within fp32 dot-product rounding, the attention output within
the usual tolerance."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_24824_b200 import binding as B
from paper_2510_24824_b200.inputs import f32_to_bf16_bits, make_problem, shrunk_workload
from paper_2510_24824_b200.runner import DecodeAttn, DeviceProblem, to_torch

from gpu_util import assert_parity

pytestmark = pytest.mark.gpu


def custom(**kw):
    base = dict(name="case", dtype="bf16", B=3, L=3, Hq=8, Hkv=2, d=128, w=40, lens=("list", [300, 77, 1]),
                gate_std=1.0, peaks=0.0, page_size=0, seed=31)
    base.update(kw)
    return base


def new_rows(p, seed):
    rng = np.random.default_rng(seed)
    store = (lambda x: f32_to_bf16_bits(x.astype(np.float32))) if p.dtype == "bf16" else (lambda x: x.astype(np.float32))
    k_new, v_new = store(rng.standard_normal((p.B, p.L, p.Hkv, p.d))), store(rng.standard_normal((p.B, p.L, p.Hkv, p.d)))
    w_gate = (rng.standard_normal((p.Hq, p.d)) / np.sqrt(p.d)).astype(np.float32)
    b_gate = rng.standard_normal(p.Hq).astype(np.float32)
    return k_new, v_new, w_gate, b_gate


def bits(t):
    t = t.cpu()
    return (t.view(torch.int16).numpy().view(np.uint16) if t.dtype == torch.bfloat16 else t.numpy())


def run_step(p, op, dp, k_new, v_new, w_gate, b_gate):
    dev = dp.q.device
    op.step(dp, to_torch(k_new, p.dtype, dev), to_torch(v_new, p.dtype, dev), to_torch(w_gate, "", dev),
            to_torch(b_gate, "", dev))
    assert op.check() == 0
    return dp.out.float().cpu().numpy().astype(np.float64)


def check_against_oracle(p, dp, got, k_new, v_new, w_gate, b_gate, what):
    after, logits = oracle.prestep(p, k_new, v_new, w_gate.astype(np.float64), b_gate.astype(np.float64))
    for name in ("k_cache", "v_cache", "k_win", "v_win"):
        assert np.array_equal(bits(getattr(dp, name)), getattr(after, name)), f"{what}: {name} differs"
    if p.L > 1:
        from oracle.plt_prestep import _to_f64
        mag = np.einsum("blhd,hd->blh", np.abs(_to_f64(p.q)), np.abs(w_gate.astype(np.float64)))[:, 1:] + np.abs(b_gate)
        err = np.abs(dp.gate_logits.cpu().numpy().astype(np.float64) - logits)
        assert np.all(err <= 1e-5 * mag + 1e-7), f"{what}: gate logits off by {err.max():.3e}"
    assert_parity(got, oracle.decode_attn(after), p.dtype, what)
    return after


@pytest.mark.parametrize("spec", [
    custom(),
    custom(dtype="f32", d=64, Hq=4, Hkv=2, B=2, lens=("list", [130, 3])),
    custom(B=6, lens=("list", [0, 1, 2, 3, 41, 80])),                           # loops without a token, ring wrap
    custom(L=1, w=0, lens=("list", [129, 1, 64])),                              # plain decode: append only
    custom(B=4, L=4, Hq=16, Hkv=4, w=16, lens=("list", [16, 17, 33, 500])),     # slots at the ring boundary
    custom(loop_offset=[0, 2, 5], lens=("list", [300, 4, 6])),
], ids=["bf16", "f32", "short", "L1", "ring-edge", "offsets"])
def test_one_step(spec):
    p = make_problem(spec)
    rows = new_rows(p, 7)
    dp = DeviceProblem(p, "cuda:0")
    with DecodeAttn(p) as op:
        got = run_step(p, op, dp, *rows)
    check_against_oracle(p, dp, got, *rows, what=spec.get("name", ""))


@pytest.mark.parametrize("spec", [
    custom(kv_dtype="e4m3"),
    custom(kv_dtype="e4m3", B=6, lens=("list", [0, 1, 2, 3, 41, 80])),
    custom(kv_dtype="e4m3", B=4, L=4, Hq=16, Hkv=4, w=16, lens=("list", [16, 17, 33, 500])),
    custom(kv_dtype="e4m3", B=3, page_size=64, lens=("list", [63, 64, 300])),
], ids=["plain", "short", "ring-edge", "paged"])
def test_one_step_on_e4m3_caches(spec):
    """The appended rows are quantised with the head's scale: the codes in the caches must match the oracle's bit for
    bit (including values beyond the range the scales were made for, which saturate)."""
    p = make_problem(spec)
    k_new, v_new, w_gate, b_gate = new_rows(p, 9)
    from paper_2510_24824_b200.inputs import bf16_bits_to_f32
    big = bf16_bits_to_f32(k_new)
    big[0, 0, 0, :4] = [1e4, -1e4, 0.0, 3e-6]          # saturation, zero, a value in the subnormal range of the grid
    k_new = f32_to_bf16_bits(big)
    dp = DeviceProblem(p, "cuda:0")
    with DecodeAttn(p) as op:
        got = run_step(p, op, dp, k_new, v_new, w_gate, b_gate)
    check_against_oracle(p, dp, got, k_new, v_new, w_gate, b_gate, what=spec.get("name", ""))


@pytest.mark.parametrize("page_size", [16, 64])
def test_one_step_paged(page_size):
    p = make_problem(shrunk_workload(4, B=9, lens=("list", [1, 2, 3, 63, 64, 255, 700, 129, 16]), page_size=page_size, w=100))
    rows = new_rows(p, 8)
    dp = DeviceProblem(p, "cuda:0")
    with DecodeAttn(p) as op:
        got = run_step(p, op, dp, *rows)
    check_against_oracle(p, dp, got, *rows, what=f"paged {page_size}")


def test_several_steps_carry_the_state_on_the_device():
    """Five consecutive decode steps on one handle: the device state after each must equal the oracle's replay."""
    p = make_problem(custom(B=3, L=3, w=8, lens=("list", [20, 5, 1]), max_seq_len=64))
    dp = DeviceProblem(p, "cuda:0")
    with DecodeAttn(p) as op:
        for step in range(5):
            rows = new_rows(p, 100 + step)
            rng = np.random.default_rng(300 + step)
            qh = f32_to_bf16_bits(rng.standard_normal((p.B, p.L, p.Hq, p.d)).astype(np.float32))
            p = p.with_(q=qh, seq_lens=(p.seq_lens + (1 if step else 0)).astype(np.int32))
            dp.q.copy_(to_torch(qh, "bf16", "cuda:0"))
            dp.seq_lens.copy_(to_torch(p.seq_lens, "", "cuda:0"))
            dp.problem = p
            got = run_step(p, op, dp, *rows)
            p = check_against_oracle(p, dp, got, *rows, what=f"step {step}")


def test_argument_errors():
    p = make_problem(custom())
    dp = DeviceProblem(p, "cuda:0")
    k_new, v_new, w_gate, b_gate = (to_torch(x, p.dtype if i < 2 else "", "cuda:0") for i, x in enumerate(new_rows(p, 1)))
    with DecodeAttn(p) as op:
        stream = torch.cuda.current_stream().cuda_stream
        with pytest.raises(B.PltError) as e:
            B.plt_decode_attn_step(op.handle, dp.args(), B.make_step_args(None, v_new, w_gate, b_gate, dp.gate_logits), stream)
        assert e.value.status == B.PLT_ERR_INVALID_ARG
        with pytest.raises(B.PltError):
            B.plt_decode_attn_step(op.handle, dp.args(), B.make_step_args(k_new, v_new, None, b_gate, dp.gate_logits), stream)
        a = dp.args()
        wl = torch.zeros((p.B, p.L - 1), dtype=torch.int32, device="cuda:0")
        a.win_lens = wl.data_ptr()
        with pytest.raises(B.PltError):
            B.plt_decode_attn_step(op.handle, a, B.make_step_args(k_new, v_new, w_gate, b_gate, dp.gate_logits), stream)
        bad = B.make_step_args(k_new, v_new, w_gate, b_gate, dp.gate_logits)
        bad.struct_size = 8
        with pytest.raises(B.PltError):
            B.plt_decode_attn_step(op.handle, dp.args(), bad, stream)
