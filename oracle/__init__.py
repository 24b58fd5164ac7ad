"""fp64 CPU oracle for the CLP decode-step attention (test infrastructure, not part of the product).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this package.
"""
from .plt_oracle import build, decode_attn, decode_attn_multi, decode_attn_rows, threads, set_threads  # noqa: F401
from .plt_prestep import gate_logits, prestep, quantise_e4m3  # noqa: F401
from .plt_seq_attn import seq_attn  # noqa: F401
