"""ctypes binding of libplt_decode_attn.so: argument marshalling only.

The functions carry the names of the C entry points they call. Every step of the attention runs in
the CUDA kernels of the library; there is no Python or CPU implementation behind these calls, and
loading fails loudly when the library has not been built.
"""
from __future__ import annotations

import ctypes
from pathlib import Path
from typing import Optional, Sequence

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libplt_decode_attn.so"

PLT_OK, PLT_ERR_INVALID_ARG, PLT_ERR_UNSUPPORTED, PLT_ERR_OUT_OF_MEMORY, PLT_ERR_CUDA, PLT_ERR_CAPACITY, \
    PLT_ERR_DEVICE_CHECK = range(7)
PLT_F32, PLT_BF16 = 0, 1
PLT_PATH_AUTO, PLT_PATH_WARP_MMA, PLT_PATH_TCGEN05 = 0, 1, 2
PLT_KV_SAME, PLT_KV_E4M3 = 0, 1
PLT_DEV_SEQ_LEN_CLAMPED, PLT_DEV_PAGE_ID_CLAMPED, PLT_DEV_WAIT_TIMEOUT, PLT_DEV_WIN_LEN_CLAMPED = 1, 2, 4, 8

EXPORTS = (
    "plt_decode_attn_create", "plt_decode_attn_run", "plt_decode_attn_run_host", "plt_decode_attn_check",
    "plt_decode_attn_destroy", "plt_decode_attn_last_error", "plt_decode_attn_workspace_bytes",
    "plt_decode_attn_launch_info", "plt_decode_attn_set_profile_events", "plt_decode_attn_run_no_alloc",
    "plt_decode_attn_step",
    "plt_seq_attn_create", "plt_seq_attn_run", "plt_seq_attn_check", "plt_seq_attn_destroy", "plt_seq_attn_last_error",
)
PLT_NO_ALLOC_SCRATCH_BYTES = 16 << 20


class PltError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"plt status {status}: {message}")
        self.status = status
        self.message = message


class Config(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32), ("dtype", ctypes.c_int32), ("max_batch", ctypes.c_int32),
        ("L", ctypes.c_int32), ("Hq", ctypes.c_int32), ("Hkv", ctypes.c_int32), ("d", ctypes.c_int32),
        ("max_seq_len", ctypes.c_int32), ("w", ctypes.c_int32), ("page_size", ctypes.c_int32),
        ("sm_scale", ctypes.c_float), ("device", ctypes.c_int32), ("loop_offset", ctypes.POINTER(ctypes.c_int32)),
        ("heads_per_cta", ctypes.c_int32), ("key_slices", ctypes.c_int32), ("stages", ctypes.c_int32),
        ("ctas_per_sm", ctypes.c_int32), ("kernel_path", ctypes.c_int32),
        ("loads_in_flight", ctypes.c_int32), ("slices_per_warp", ctypes.c_int32), ("row_warps", ctypes.c_int32),
        ("kv_dtype", ctypes.c_int32), ("q_len", ctypes.c_int32), ("typical_seq_len", ctypes.c_int32),
    ]


class Args(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32), ("batch", ctypes.c_int32),
        ("q", ctypes.c_void_p), ("k_cache", ctypes.c_void_p), ("v_cache", ctypes.c_void_p),
        ("kv_stride_b", ctypes.c_int64), ("kv_stride_n", ctypes.c_int64), ("kv_stride_h", ctypes.c_int64),
        ("seq_lens", ctypes.c_void_p), ("page_table", ctypes.c_void_p),
        ("max_pages", ctypes.c_int32), ("num_pool_pages", ctypes.c_int32),
        ("k_win", ctypes.c_void_p), ("v_win", ctypes.c_void_p), ("win_lens", ctypes.c_void_p),
        ("gate_logits", ctypes.c_void_p), ("out", ctypes.c_void_p),
        ("k_scale", ctypes.c_void_p), ("v_scale", ctypes.c_void_p),
    ]


class StepArgs(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32), ("k_new", ctypes.c_void_p), ("v_new", ctypes.c_void_p),
        ("w_gate", ctypes.c_void_p), ("b_gate", ctypes.c_void_p), ("gate_logits", ctypes.c_void_p),
    ]


class SeqConfig(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32), ("max_batch", ctypes.c_int32), ("L", ctypes.c_int32), ("Hq", ctypes.c_int32),
        ("Hkv", ctypes.c_int32), ("d", ctypes.c_int32), ("max_seq_len", ctypes.c_int32), ("w", ctypes.c_int32),
        ("sm_scale", ctypes.c_float), ("device", ctypes.c_int32), ("loop_offset", ctypes.POINTER(ctypes.c_int32)),
    ]


class SeqArgs(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32), ("batch", ctypes.c_int32), ("q", ctypes.c_void_p),
        ("k_share", ctypes.c_void_p), ("v_share", ctypes.c_void_p), ("k_loc", ctypes.c_void_p),
        ("v_loc", ctypes.c_void_p), ("gate_logits", ctypes.c_void_p), ("seq_lens", ctypes.c_void_p),
        ("out", ctypes.c_void_p),
    ]


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads the shared library; raises if it is missing (there is no other implementation to fall back to)."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2510_24824_b200.build`")
        lib = ctypes.CDLL(str(LIB_PATH))
        h = ctypes.c_void_p
        lib.plt_decode_attn_create.argtypes = [ctypes.POINTER(Config), ctypes.POINTER(h)]
        lib.plt_decode_attn_run.argtypes = [h, ctypes.POINTER(Args), ctypes.c_void_p]
        lib.plt_decode_attn_run_host.argtypes = [h, ctypes.POINTER(Args), ctypes.c_void_p]
        lib.plt_decode_attn_step.argtypes = [h, ctypes.POINTER(Args), ctypes.POINTER(StepArgs), ctypes.c_void_p]
        lib.plt_decode_attn_check.argtypes = [h, ctypes.c_void_p, ctypes.POINTER(ctypes.c_uint32)]
        lib.plt_decode_attn_destroy.argtypes = [h]
        lib.plt_decode_attn_last_error.argtypes = [h]
        lib.plt_decode_attn_last_error.restype = ctypes.c_char_p
        lib.plt_decode_attn_workspace_bytes.argtypes = [ctypes.POINTER(Config), ctypes.POINTER(ctypes.c_size_t)]
        i32p = ctypes.POINTER(ctypes.c_int32)
        lib.plt_decode_attn_launch_info.argtypes = [h, i32p, i32p, i32p, i32p, i32p, i32p, i32p]
        lib.plt_decode_attn_set_profile_events.argtypes = [h, ctypes.c_void_p, ctypes.c_void_p]
        lib.plt_decode_attn_run_no_alloc.argtypes = [ctypes.POINTER(Config), ctypes.POINTER(Args), ctypes.c_void_p]
        lib.plt_seq_attn_create.argtypes = [ctypes.POINTER(SeqConfig), ctypes.POINTER(h)]
        lib.plt_seq_attn_run.argtypes = [h, ctypes.POINTER(SeqArgs), ctypes.c_void_p]
        lib.plt_seq_attn_check.argtypes = [h, ctypes.c_void_p, ctypes.POINTER(ctypes.c_uint32)]
        lib.plt_seq_attn_destroy.argtypes = [h]
        lib.plt_seq_attn_last_error.argtypes = [h]
        lib.plt_seq_attn_last_error.restype = ctypes.c_char_p
        for name in EXPORTS:
            if not name.endswith("_last_error"):
                getattr(lib, name).restype = ctypes.c_int
        _lib = lib
    return _lib


def _raise(status: int, handle) -> None:
    msg = load_library().plt_decode_attn_last_error(handle)
    raise PltError(status, msg.decode() if msg else "")


def make_config(dtype, max_batch: int, L: int, Hq: int, Hkv: int, d: int, max_seq_len: int, w: int,
                page_size: int = 0, sm_scale: float = 0.0, device: int = 0,
                loop_offset: Optional[Sequence[int]] = None, heads_per_cta: int = 0, key_slices: int = 0,
                stages: int = 0, ctas_per_sm: int = 0, kernel_path: int = 0, loads_in_flight: int = 0,
                row_warps: int = 0, slices_per_warp: int = 0, kv_dtype: int = 0, q_len: int = 0,
                typical_seq_len: int = 0) -> Config:
    c = Config()
    c.struct_size = ctypes.sizeof(Config)
    c.dtype = {"f32": PLT_F32, "bf16": PLT_BF16}.get(dtype, dtype)
    c.max_batch, c.L, c.Hq, c.Hkv, c.d = max_batch, L, Hq, Hkv, d
    c.max_seq_len, c.w, c.page_size = max_seq_len, w, page_size
    c.sm_scale, c.device = sm_scale, device
    if loop_offset is not None:
        arr = (ctypes.c_int32 * len(loop_offset))(*[int(x) for x in loop_offset])
        c._keep = arr
        c.loop_offset = ctypes.cast(arr, ctypes.POINTER(ctypes.c_int32))
    c.heads_per_cta, c.key_slices, c.stages, c.ctas_per_sm = heads_per_cta, key_slices, stages, ctas_per_sm
    c.kernel_path = kernel_path
    c.loads_in_flight = loads_in_flight
    c.row_warps = row_warps
    c.slices_per_warp = slices_per_warp
    c.kv_dtype = {"": PLT_KV_SAME, "e4m3": PLT_KV_E4M3}.get(kv_dtype, kv_dtype)
    c.q_len = q_len
    c.typical_seq_len = typical_seq_len
    return c


def plt_decode_attn_create(config: Config) -> ctypes.c_void_p:
    lib = load_library()
    handle = ctypes.c_void_p()
    st = lib.plt_decode_attn_create(ctypes.byref(config), ctypes.byref(handle))
    if st != PLT_OK:
        _raise(st, None)
    return handle


def plt_decode_attn_workspace_bytes(config: Config) -> int:
    out = ctypes.c_size_t()
    st = load_library().plt_decode_attn_workspace_bytes(ctypes.byref(config), ctypes.byref(out))
    if st != PLT_OK:
        _raise(st, None)
    return int(out.value)


def _ptr(x) -> Optional[int]:
    """Address of a torch tensor (device or pinned host), a numpy array, or a raw integer; None stays NULL."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return int(x.data_ptr())
    if hasattr(x, "ctypes"):
        return int(x.ctypes.data)
    raise TypeError(f"cannot take the address of {type(x)}")


def make_args(batch: int, q, k_cache, v_cache, seq_lens, out, k_win=None, v_win=None, gate_logits=None,
              page_table=None, max_pages: int = 0, num_pool_pages: int = 0, win_lens=None,
              kv_strides=(0, 0, 0), k_scale=None, v_scale=None) -> Args:
    a = Args()
    a.struct_size = ctypes.sizeof(Args)
    a.batch = batch
    a.q, a.k_cache, a.v_cache = _ptr(q), _ptr(k_cache), _ptr(v_cache)
    a.kv_stride_b, a.kv_stride_n, a.kv_stride_h = (int(s) for s in kv_strides)
    a.seq_lens, a.page_table = _ptr(seq_lens), _ptr(page_table)
    a.max_pages, a.num_pool_pages = max_pages, num_pool_pages
    a.k_win, a.v_win, a.win_lens = _ptr(k_win), _ptr(v_win), _ptr(win_lens)
    a.gate_logits, a.out = _ptr(gate_logits), _ptr(out)
    a.k_scale, a.v_scale = _ptr(k_scale), _ptr(v_scale)
    return a


def plt_decode_attn_run(handle, args: Args, stream: int = 0) -> None:
    st = load_library().plt_decode_attn_run(handle, ctypes.byref(args), ctypes.c_void_p(stream))
    if st != PLT_OK:
        _raise(st, handle)


def make_step_args(k_new, v_new, w_gate=None, b_gate=None, gate_logits=None) -> StepArgs:
    s = StepArgs()
    s.struct_size = ctypes.sizeof(StepArgs)
    s.k_new, s.v_new = _ptr(k_new), _ptr(v_new)
    s.w_gate, s.b_gate, s.gate_logits = _ptr(w_gate), _ptr(b_gate), _ptr(gate_logits)
    return s


def plt_decode_attn_step(handle, args: Args, step: StepArgs, stream: int = 0) -> None:
    st = load_library().plt_decode_attn_step(handle, ctypes.byref(args), ctypes.byref(step), ctypes.c_void_p(stream))
    if st != PLT_OK:
        _raise(st, handle)


def plt_decode_attn_run_host(handle, args: Args, stream: int = 0) -> None:
    st = load_library().plt_decode_attn_run_host(handle, ctypes.byref(args), ctypes.c_void_p(stream))
    if st != PLT_OK:
        _raise(st, handle)


def plt_decode_attn_check(handle, stream: int = 0) -> int:
    """Synchronises the stream; returns the device status bits (0 = clean) and clears them."""
    bits = ctypes.c_uint32()
    st = load_library().plt_decode_attn_check(handle, ctypes.c_void_p(stream), ctypes.byref(bits))
    if st not in (PLT_OK, PLT_ERR_DEVICE_CHECK):
        _raise(st, handle)
    return int(bits.value)


def plt_decode_attn_destroy(handle) -> None:
    load_library().plt_decode_attn_destroy(handle)


def plt_decode_attn_launch_info(handle) -> dict:
    vals = [ctypes.c_int32() for _ in range(7)]
    st = load_library().plt_decode_attn_launch_info(handle, *[ctypes.byref(v) for v in vals])
    if st != PLT_OK:
        _raise(st, handle)
    keys = ("kernels_per_run", "heads_per_cta", "key_slices", "stages", "ctas_per_sm", "grid", "kernel_path")
    return {k: int(v.value) for k, v in zip(keys, vals)}


def plt_decode_attn_set_profile_events(handle, ev_main_begin: Optional[int], ev_main_end: Optional[int]) -> None:
    st = load_library().plt_decode_attn_set_profile_events(handle, ev_main_begin, ev_main_end)
    if st != PLT_OK:
        _raise(st, handle)


def plt_decode_attn_run_no_alloc(config: Config, args: Args, stream: int = 0) -> None:
    """The decode-step attention without a handle and without any device allocation (scratch is built into the
    library). For callers that may not allocate; config.device must be the current device."""
    st = load_library().plt_decode_attn_run_no_alloc(ctypes.byref(config), ctypes.byref(args), ctypes.c_void_p(stream))
    if st != PLT_OK:
        _raise(st, None)


# ---- sequence-shaped attention (plt_seq_attn.h) -------------------------------------------------------------------
def _raise_seq(status: int, handle) -> None:
    msg = load_library().plt_seq_attn_last_error(handle)
    raise PltError(status, msg.decode() if msg else "")


def make_seq_config(max_batch: int, L: int, Hq: int, Hkv: int, d: int, max_seq_len: int, w: int, sm_scale: float = 0.0,
                    device: int = 0, loop_offset: Optional[Sequence[int]] = None) -> SeqConfig:
    c = SeqConfig()
    c.struct_size = ctypes.sizeof(SeqConfig)
    c.max_batch, c.L, c.Hq, c.Hkv, c.d, c.max_seq_len, c.w = max_batch, L, Hq, Hkv, d, max_seq_len, w
    c.sm_scale, c.device = sm_scale, device
    if loop_offset is not None:
        arr = (ctypes.c_int32 * len(loop_offset))(*[int(x) for x in loop_offset])
        c._keep = arr
        c.loop_offset = ctypes.cast(arr, ctypes.POINTER(ctypes.c_int32))
    return c


def make_seq_args(batch: int, q, k_share, v_share, seq_lens, out, k_loc=None, v_loc=None, gate_logits=None) -> SeqArgs:
    """Tensors are anything with data_ptr() (device memory); None becomes NULL."""
    a = SeqArgs()
    a.struct_size = ctypes.sizeof(SeqArgs)
    a.batch = batch
    ptr = lambda t: None if t is None else t.data_ptr()
    a.q, a.k_share, a.v_share, a.k_loc, a.v_loc = ptr(q), ptr(k_share), ptr(v_share), ptr(k_loc), ptr(v_loc)
    a.gate_logits, a.seq_lens, a.out = ptr(gate_logits), ptr(seq_lens), ptr(out)
    a._keep = (q, k_share, v_share, k_loc, v_loc, gate_logits, seq_lens, out)
    return a


def plt_seq_attn_create(config: SeqConfig):
    handle = ctypes.c_void_p()
    st = load_library().plt_seq_attn_create(ctypes.byref(config), ctypes.byref(handle))
    if st != PLT_OK:
        _raise_seq(st, None)
    return handle


def plt_seq_attn_run(handle, args: SeqArgs, stream: int = 0) -> None:
    st = load_library().plt_seq_attn_run(handle, ctypes.byref(args), ctypes.c_void_p(stream))
    if st != PLT_OK:
        _raise_seq(st, handle)


def plt_seq_attn_check(handle, stream: int = 0) -> int:
    bits = ctypes.c_uint32()
    st = load_library().plt_seq_attn_check(handle, ctypes.c_void_p(stream), ctypes.byref(bits))
    if st not in (PLT_OK, PLT_ERR_DEVICE_CHECK):
        _raise_seq(st, handle)
    return int(bits.value)


def plt_seq_attn_destroy(handle) -> None:
    load_library().plt_seq_attn_destroy(handle)
