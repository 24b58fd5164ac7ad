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


class LoopOrderAblation:
    """The ablation rows of Table 1 at kernel level, on the tensors of a device problem: the same loop-queries served

      * as L sequential single-loop calls, each scanning the shared cache again (the loop order of the vanilla loop
        transformer: L launches, L scans), and
      * as ONE cross-loop-parallel call over L private caches, one per loop ("Loop+CLP" before KV sharing: one launch,
        L caches read once each; the private caches are device-side copies of the shared one at other addresses),

    beside the library's own step (one launch, one shared cache). Global attention only (no window, no gate): what
    the three have in common. torch is used for device memory only.
    """

    def __init__(self, p, dp: DeviceProblem, device_index: int = 0, kernel_path: int = 0, private: bool = True):
        self.p, self.dp, self.L = p, dp, p.L
        dev = dp.q.device
        offs = [int(x) for x in p.offsets()]
        lens = dp.seq_lens.to(torch.int64)
        self.loop_lens = [torch.clamp(lens - o, min=0).to(torch.int32) for o in offs]
        p1 = p.with_(L=1, w=0, q=np.ascontiguousarray(p.q[:, :1]), loop_offset=None, win_lens=None)
        # ---- sequential single-loop calls over the shared cache ----
        self.seq_op = DecodeAttn(p1, device_index=device_index, kernel_path=kernel_path)
        self.seq_q = [dp.q[:, l:l + 1].contiguous() for l in range(p.L)]
        self.seq_out = [torch.empty_like(q) for q in self.seq_q]
        self.seq_args = [B.make_args(p.B, q, dp.k_cache, dp.v_cache, n, o, page_table=dp.page_table, max_pages=p.max_pages,
                                     num_pool_pages=p.num_pool_pages, k_scale=dp.k_scale, v_scale=dp.v_scale)
                         for q, n, o in zip(self.seq_q, self.loop_lens, self.seq_out)]
        # ---- one call over L private caches: sequence b * L + l is loop l of sequence b with a cache of its own ----
        self.priv_op = None
        if private:
            self.priv_op = DecodeAttn(p1, device_index=device_index, kernel_path=kernel_path, max_batch=p.B * p.L)
            self.priv_q = dp.q.reshape(p.B * p.L, 1, p.Hq, p.d)
            self.priv_out = torch.empty_like(self.priv_q)
            self.priv_lens = torch.stack(self.loop_lens, dim=1).reshape(-1).contiguous()
            if p.page_size:
                P = p.num_pool_pages
                self.priv_k = dp.k_cache.repeat(p.L, 1, 1, 1)
                self.priv_v = dp.v_cache.repeat(p.L, 1, 1, 1)
                shift = (torch.arange(p.L, device=dev, dtype=torch.int32) * P).view(1, p.L, 1)
                self.priv_table = (dp.page_table.view(p.B, 1, -1) + shift).reshape(p.B * p.L, -1).contiguous()
                pool = P * p.L
            else:
                self.priv_k = dp.k_cache.repeat_interleave(p.L, dim=0)
                self.priv_v = dp.v_cache.repeat_interleave(p.L, dim=0)
                self.priv_table, pool = None, 0
            self.priv_args = B.make_args(p.B * p.L, self.priv_q, self.priv_k, self.priv_v, self.priv_lens, self.priv_out,
                                         page_table=self.priv_table, max_pages=p.max_pages, num_pool_pages=pool,
                                         k_scale=dp.k_scale, v_scale=dp.v_scale)

    def run_sequential(self, stream: Optional[int] = None):
        """L launches of the single-loop attention; returns the outputs stacked as [B, L, Hq, d]."""
        if stream is None:
            stream = torch.cuda.current_stream().cuda_stream
        for a in self.seq_args:
            B.plt_decode_attn_run(self.seq_op.handle, a, stream)
        return self.seq_out

    def run_private(self, stream: Optional[int] = None):
        """One launch over the L private caches; returns [B * L, 1, Hq, d] (row b * L + l)."""
        if stream is None:
            stream = torch.cuda.current_stream().cuda_stream
        B.plt_decode_attn_run(self.priv_op.handle, self.priv_args, stream)
        return self.priv_out

    def check(self, stream: Optional[int] = None) -> int:
        bits = self.seq_op.check(stream)
        if self.priv_op is not None:
            bits |= self.priv_op.check(stream)
        return bits

    def close(self):
        self.seq_op.close()
        if self.priv_op is not None:
            self.priv_op.close()
