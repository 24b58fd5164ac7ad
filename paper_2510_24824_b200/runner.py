"""Device plumbing around the C ABI: moves a host problem into torch device tensors and calls the library.

torch is used for device memory and streams only; the attention itself runs in libplt_decode_attn.so.
"""
from __future__ import annotations

from typing import Optional

import numpy as np
import torch

from . import binding as B


def to_torch(a: Optional[np.ndarray], dtype: str, device, pin: bool = False):
    """Host array (float32 / int32, or bf16 bit patterns when dtype == 'bf16') as a torch tensor on `device`."""
    if a is None:
        return None
    t = torch.from_numpy(np.ascontiguousarray(a))
    if a.dtype == np.uint16 and dtype == "bf16":
        t = t.view(torch.bfloat16)
    if device is None:
        return t.pin_memory() if pin else t
    return t.to(device, non_blocking=False)


class DeviceProblem:
    """Tensors of one decode step on a device (or, with device=None, in pinned host memory)."""

    FIELDS = ("q", "k_cache", "v_cache", "seq_lens", "k_win", "v_win", "gate_logits", "page_table", "win_lens",
              "k_scale", "v_scale")

    def __init__(self, p, device="cuda:0", pin: bool = False):
        self.problem = p
        self.device = device
        for f in self.FIELDS:
            a = getattr(p, f)
            is_data = f == "q" or (f in ("k_cache", "v_cache", "k_win", "v_win") and p.kv_dtype != "e4m3")
            setattr(self, f, to_torch(a, p.dtype if is_data else "", device, pin))   # E4M3 codes stay uint8
        tdt = torch.bfloat16 if p.dtype == "bf16" else torch.float32
        if device is None:
            self.out = torch.empty((p.B, p.L, p.Hq, p.d), dtype=tdt)
            if pin:
                self.out = self.out.pin_memory()
        else:
            self.out = torch.empty((p.B, p.L, p.Hq, p.d), dtype=tdt, device=device)

    def args(self, out=None) -> B.Args:
        p = self.problem
        return B.make_args(
            p.B, self.q, self.k_cache, self.v_cache, self.seq_lens, self.out if out is None else out,
            k_win=self.k_win if p.L > 1 else None, v_win=self.v_win if p.L > 1 else None,
            gate_logits=self.gate_logits if p.L > 1 else None, page_table=self.page_table,
            max_pages=p.max_pages, num_pool_pages=p.num_pool_pages, win_lens=self.win_lens,
            k_scale=self.k_scale, v_scale=self.v_scale)

    def h2d_bytes(self) -> int:
        n = 0
        for f in self.FIELDS:
            t = getattr(self, f)
            if t is not None and not (self.problem.L == 1 and f in ("k_win", "v_win", "gate_logits", "win_lens")):
                n += t.numel() * t.element_size()
        return n

    def d2h_bytes(self) -> int:
        return self.out.numel() * self.out.element_size()


class DecodeAttn:
    """Owns one plt_decode_attn handle sized for a problem (or for explicit limits)."""

    def __init__(self, p, device_index: int = 0, max_batch: Optional[int] = None, **tuning):
        self.config = B.make_config(
            p.dtype, max_batch or max(p.B, 1), p.L, p.Hq, p.Hkv, p.d, p.max_seq_len, p.w, page_size=p.page_size,
            sm_scale=p.sm_scale, device=device_index,
            loop_offset=None if p.loop_offset is None else [int(x) for x in p.loop_offset], kv_dtype=p.kv_dtype,
            **tuning)
        self.handle = B.plt_decode_attn_create(self.config)
        self.info = B.plt_decode_attn_launch_info(self.handle)

    def run(self, dp: DeviceProblem, stream: Optional[int] = None, out=None):
        if stream is None:
            stream = torch.cuda.current_stream().cuda_stream
        B.plt_decode_attn_run(self.handle, dp.args(out), stream)
        return dp.out if out is None else out

    def step(self, dp: DeviceProblem, k_new, v_new, w_gate, b_gate, stream: Optional[int] = None):
        """Pre-step (cache append, window ring update, gate linear into dp.gate_logits) and attention in one call.
        k_new, v_new, w_gate, b_gate: device tensors."""
        if stream is None:
            stream = torch.cuda.current_stream().cuda_stream
        st = B.make_step_args(k_new, v_new, w_gate, b_gate, dp.gate_logits if dp.problem.L > 1 else None)
        B.plt_decode_attn_step(self.handle, dp.args(), st, stream)
        return dp.out

    def run_host(self, hp: DeviceProblem, stream: Optional[int] = None):
        if stream is None:
            stream = torch.cuda.current_stream().cuda_stream
        B.plt_decode_attn_run_host(self.handle, hp.args(), stream)
        return hp.out

    def check(self, stream: Optional[int] = None) -> int:
        if stream is None:
            stream = torch.cuda.current_stream().cuda_stream
        return B.plt_decode_attn_check(self.handle, stream)

    def close(self):
        if self.handle is not None:
            B.plt_decode_attn_destroy(self.handle)
            self.handle = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class SeqAttn:
    """One plt_seq_attn handle and the device tensors of a sequence problem (torch for memory and streams only)."""

    FIELDS = ("q", "k_share", "v_share", "k_loc", "v_loc")

    def __init__(self, p, device="cuda:0", device_index: int = 0):
        self.problem = p
        for f in self.FIELDS:
            setattr(self, f, to_torch(getattr(p, f), "bf16", device))
        self.gate_logits = to_torch(p.gate_logits, "", device)
        self.seq_lens = to_torch(p.seq_lens, "", device)
        self.out = torch.empty((p.B, p.L, p.T, p.Hq, p.d), dtype=torch.bfloat16, device=device)
        self.config = B.make_seq_config(
            max(p.B, 1), p.L, p.Hq, p.Hkv, p.d, p.T, p.w, sm_scale=p.sm_scale, device=device_index,
            loop_offset=None if p.loop_offset is None else [int(x) for x in p.loop_offset])
        self.handle = B.plt_seq_attn_create(self.config)
        many = p.L > 1
        self.args = B.make_seq_args(p.B, self.q, self.k_share, self.v_share, self.seq_lens, self.out,
                                    k_loc=self.k_loc if many else None, v_loc=self.v_loc if many else None,
                                    gate_logits=self.gate_logits if many else None)

    def run(self, stream: Optional[int] = None):
        if stream is None:
            stream = torch.cuda.current_stream().cuda_stream
        B.plt_seq_attn_run(self.handle, self.args, stream)
        return self.out

    def check(self, stream: Optional[int] = None) -> int:
        if stream is None:
            stream = torch.cuda.current_stream().cuda_stream
        return B.plt_seq_attn_check(self.handle, stream)

    def close(self):
        if self.handle is not None:
            B.plt_seq_attn_destroy(self.handle)
            self.handle = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()
