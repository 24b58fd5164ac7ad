"""Helpers shared by the GPU parity tests: run the CUDA path through the C ABI, compare with the oracle."""
import numpy as np
import torch

from paper_2510_24824_b200.runner import DecodeAttn, DeviceProblem

from parity_bounds import (BF16_MAX_ABS, BF16_MEAN_ABS, F32_REL, assert_parity, bf16_bound,  # noqa: F401
                           inactive_rows, parity_report)


def run_gpu(p, check_status=True, **tuning) -> np.ndarray:
    dp = DeviceProblem(p, "cuda:0")
    dp.out.fill_(float("nan"))
    with DecodeAttn(p, **tuning) as op:
        op.run(dp)
        bits = op.check()
    if check_status:
        assert bits == 0, f"device status 0x{bits:x}"
    return dp.out.float().cpu().numpy().astype(np.float64)
