"""Tolerances of the parity bar, in one place for the GPU tests and the smoke check (numpy only).

bf16 inputs: max-abs error 2e-2 and mean-abs error 2e-3; fp32 inputs: 1e-5 relative.
The output is stored in bf16 (8 significant bits), so storing it costs up to half a unit in the last place of the
reference value: 2^(e-8) for |ref| in [2^e, 2^(e+1)). Below |ref| = 8 that is at most 2^-6 = 0.0156 and the plain 2e-2
holds. From 8 up the store alone can exceed 2e-2 (0.031 in [8, 16)), so there the bound is that half unit plus the
budget the plain bound leaves the arithmetic in the binade just below: 2e-2 - 2^-6 = 0.0044.
"""
import numpy as np

BF16_MAX_ABS, BF16_MEAN_ABS = 2e-2, 2e-3
BF16_KERNEL_BUDGET = BF16_MAX_ABS - 2.0 ** -6
F32_REL = 1e-5


def bf16_half_ulp(ref: np.ndarray) -> np.ndarray:
    """Half a unit in the last place of bf16 at the magnitude of ref (for |ref| >= 1)."""
    a = np.maximum(np.abs(ref), 1.0)
    return 2.0 ** (np.floor(np.log2(a)) - 8.0)


def bf16_bound(ref: np.ndarray) -> np.ndarray:
    return np.where(np.abs(ref) < 8.0, BF16_MAX_ABS, bf16_half_ulp(ref) + BF16_KERNEL_BUDGET)


def inactive_rows(p) -> np.ndarray:
    """[B, L] mask of loops that have no token yet (N_b <= delta_l, delta_l = l - 1 by default): their output rows must be 0."""
    delta = np.arange(p.L) if p.loop_offset is None else np.asarray(p.loop_offset, dtype=np.int64)
    return (np.asarray(p.seq_lens, dtype=np.int64)[:, None] - delta[None, :]) <= 0


def parity_report(got: np.ndarray, ref: np.ndarray, dtype: str) -> dict:
    """Numbers of one comparison: worst error, mean error, worst error as a fraction of its bound, and (bf16) how many
    elements lie beyond the plain 2e-2 with the range of |ref| they have (all of them must be >= 8)."""
    err = np.abs(got - ref)
    out = {"max_abs": float(err.max()) if err.size else 0.0, "mean_abs": float(err.mean()) if err.size else 0.0}
    if dtype == "bf16":
        frac = err / bf16_bound(ref)
        over = err > BF16_MAX_ABS
        out["worst_of_bound"] = float(frac.max()) if err.size else 0.0
        out["over_plain"] = int(over.sum())
        out["over_plain_ref_min"] = float(np.abs(ref)[over].min()) if over.any() else None
    else:
        out["worst_of_bound"] = float(err.max() / (F32_REL * max(np.abs(ref).max(), 1e-30))) if err.size else 0.0
    return out


def assert_parity(got: np.ndarray, ref: np.ndarray, dtype: str, what: str = ""):
    assert got.shape == ref.shape
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    err = np.abs(got - ref)
    rep = parity_report(got, ref, dtype)
    if dtype == "bf16":
        assert rep["worst_of_bound"] <= 1.0, (
            f"{what}: max abs err {rep['max_abs']:.3e} ({rep['worst_of_bound']:.2f} of the bound); "
            f"{rep['over_plain']} elements beyond 2e-2, smallest |ref| among them {rep['over_plain_ref_min']}")
        assert rep["mean_abs"] <= BF16_MEAN_ABS, f"{what}: mean abs err {rep['mean_abs']:.3e}"
    else:
        scale = np.abs(ref).max() if ref.size else 0.0
        assert err.max(initial=0.0) <= F32_REL * max(scale, 1e-30), f"{what}: max err {err.max():.3e} vs max|ref| {scale:.3e}"
        bad = err > F32_REL * np.abs(ref) + 1e-6
        assert not bad.any(), f"{what}: {bad.sum()} elements beyond 1e-5 relative + 1e-6"
    return rep["max_abs"], rep["mean_abs"]
