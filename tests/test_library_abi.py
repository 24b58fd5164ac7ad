"""CPU-only checks of the boundary: the library loads, exports what the header declares, and the
binding's structs match the C layout. No compute call is made here."""
import ctypes
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parents[1]


@pytest.fixture(scope="module")
def lib():
    from paper_2510_24824_b200 import build
    build.build()
    from paper_2510_24824_b200 import binding
    return binding.load_library()


def header_functions():
    names = set()
    for header in sorted((ROOT / "include").glob("*.h")):
        text = re.sub(r"/\*.*?\*/", "", header.read_text(), flags=re.S)
        names |= set(re.findall(r"\b(plt_(?:decode|seq)_attn_\w+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported(lib):
    names = header_functions()
    assert "plt_decode_attn_create" in names and "plt_decode_attn_run" in names and "plt_decode_attn_destroy" in names
    assert "plt_seq_attn_create" in names and "plt_seq_attn_run" in names and "plt_seq_attn_destroy" in names
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in the header but not exported"
    from paper_2510_24824_b200 import binding
    assert sorted(binding.EXPORTS) == names


def test_struct_layout_matches_c(tmp_path):
    """Compile a tiny C program against the header and compare sizeof/offsetof with the ctypes structs."""
    import subprocess
    from paper_2510_24824_b200 import binding
    structs = [("plt_decode_attn_config", binding.Config), ("plt_decode_attn_args", binding.Args),
               ("plt_decode_attn_step_args", binding.StepArgs), ("plt_seq_attn_config", binding.SeqConfig),
               ("plt_seq_attn_args", binding.SeqArgs)]
    src = tmp_path / "layout.c"
    lines = ['#include <stdio.h>', '#include <stddef.h>', f'#include "{ROOT}/include/plt_seq_attn.h"', 'int main(void){']
    for cname, st in structs:
        lines += [f'printf("%zu\\n", sizeof({cname}));']
        lines += [f'printf("%zu\\n", offsetof({cname}, {f}));' for f, _ in st._fields_]
    lines += ['return 0;}']
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-std=c11", "-o", str(exe), str(src)], check=True)
    vals = [int(x) for x in subprocess.run([str(exe)], capture_output=True, text=True, check=True).stdout.split()]
    want = []
    for _, st in structs:
        want += [ctypes.sizeof(st)] + [getattr(st, f).offset for f, _ in st._fields_]
    assert vals == want


def test_host_side_validation_needs_no_gpu(lib):
    """Argument checks that run before any CUDA call return their codes on a machine without a GPU."""
    from paper_2510_24824_b200 import binding as B
    ok = dict(dtype="bf16", max_batch=4, L=2, Hq=8, Hkv=2, d=128, max_seq_len=512, w=64)
    bad = [
        (dict(ok, d=96), B.PLT_ERR_UNSUPPORTED),
        (dict(ok, Hq=7), B.PLT_ERR_INVALID_ARG),
        (dict(ok, L=9), B.PLT_ERR_UNSUPPORTED),
        (dict(ok, L=4, Hq=64, Hkv=2), B.PLT_ERR_UNSUPPORTED),  # 128 packed rows
        (dict(ok, w=0), B.PLT_ERR_INVALID_ARG),
        (dict(ok, page_size=24), B.PLT_ERR_UNSUPPORTED),
        (dict(ok, max_batch=0), B.PLT_ERR_INVALID_ARG),
        (dict(ok, max_batch=5000), B.PLT_ERR_UNSUPPORTED),
        (dict(ok, loop_offset=[0, -1]), B.PLT_ERR_INVALID_ARG),
        (dict(ok, heads_per_cta=3), B.PLT_ERR_INVALID_ARG),
    ]
    for kw, code in bad:
        with pytest.raises(B.PltError) as e:
            B.plt_decode_attn_workspace_bytes(B.make_config(**kw))
        assert e.value.status == code, (kw, e.value)
        assert e.value.message
    cfg = B.make_config(**ok)
    cfg.struct_size = 8
    with pytest.raises(B.PltError) as e:
        B.plt_decode_attn_workspace_bytes(cfg)
    assert e.value.status == B.PLT_ERR_INVALID_ARG
    assert B.plt_decode_attn_workspace_bytes(B.make_config(**ok)) > 0
    # E4M3 caches on the tcgen05 path: at most 32 packed rows; its workspace (one block per SM, two heads per item, a
    # query image and a scale factor per (sequence, KV head)) differs from the warp-level path's, and the automatic
    # choice is that path at 25-32 rows on caches (contiguous, pages of whole tiles or of 64 tokens) that can reach 8192
    # keys and at 17-24 rows on caches (contiguous or pages of whole tiles) that can reach 32768
    fp8 = dict(ok, L=4, Hq=16, kv_dtype="e4m3")                                  # 32 packed rows
    size = lambda **kw: B.plt_decode_attn_workspace_bytes(B.make_config(**dict(fp8, **kw)))
    assert size(kernel_path=B.PLT_PATH_TCGEN05) > 4 * 2 * 8192
    assert size() == size(kernel_path=B.PLT_PATH_WARP_MMA) != size(kernel_path=B.PLT_PATH_TCGEN05)
    assert size(max_seq_len=32768) == size(max_seq_len=32768, kernel_path=B.PLT_PATH_TCGEN05)
    assert size(max_seq_len=32768, page_size=128) == size(max_seq_len=32768, page_size=128, kernel_path=B.PLT_PATH_TCGEN05)
    assert size(max_seq_len=32768, page_size=64) == size(max_seq_len=32768, page_size=64, kernel_path=B.PLT_PATH_TCGEN05)
    assert size(max_seq_len=32768, page_size=32) == size(max_seq_len=32768, page_size=32, kernel_path=B.PLT_PATH_WARP_MMA)
    assert size(max_seq_len=32768, page_size=64, L=3) == size(max_seq_len=32768, page_size=64, L=3, kernel_path=B.PLT_PATH_WARP_MMA)
    assert size(max_seq_len=8192) == size(max_seq_len=8192, kernel_path=B.PLT_PATH_TCGEN05)
    assert size(max_seq_len=8191) == size(max_seq_len=8191, kernel_path=B.PLT_PATH_WARP_MMA)
    # a length the caller expects most sequences to reach replaces the cautious judgement by max_seq_len
    assert size(max_seq_len=4096, typical_seq_len=2048) == size(max_seq_len=4096, kernel_path=B.PLT_PATH_TCGEN05, typical_seq_len=2048)
    assert size(max_seq_len=32768, typical_seq_len=1024) == size(max_seq_len=32768, kernel_path=B.PLT_PATH_WARP_MMA, typical_seq_len=1024)
    assert size(max_seq_len=16384, L=3, typical_seq_len=8192) == size(max_seq_len=16384, L=3, kernel_path=B.PLT_PATH_TCGEN05, typical_seq_len=8192)
    assert size(max_seq_len=4096, typical_seq_len=10 ** 6) == size(max_seq_len=4096, kernel_path=B.PLT_PATH_TCGEN05, typical_seq_len=10 ** 6)
    with pytest.raises(B.PltError) as e:
        size(typical_seq_len=-1)
    assert e.value.status == B.PLT_ERR_INVALID_ARG
    for rows_24_or_16, longest, path in ((3, 32768, B.PLT_PATH_TCGEN05), (3, 32767, B.PLT_PATH_WARP_MMA), (2, 65536, B.PLT_PATH_WARP_MMA)):
        assert size(max_seq_len=longest, L=rows_24_or_16) == size(max_seq_len=longest, L=rows_24_or_16, kernel_path=path)
        assert size(max_seq_len=longest, L=rows_24_or_16) != size(max_seq_len=longest, L=rows_24_or_16, kernel_path=3 - path)
    with pytest.raises(B.PltError) as e:
        size(Hq=32, kernel_path=B.PLT_PATH_TCGEN05)   # 64 rows
    assert e.value.status == B.PLT_ERR_UNSUPPORTED
    B.plt_decode_attn_destroy(None)  # NULL is accepted
    # the sequence-shaped entry points validate before they touch a device too
    for kw, code in [(dict(d=64), B.PLT_ERR_UNSUPPORTED), (dict(Hq=7), B.PLT_ERR_INVALID_ARG), (dict(L=9), B.PLT_ERR_UNSUPPORTED),
                     (dict(w=0), B.PLT_ERR_INVALID_ARG), (dict(loop_offset=[0, -2]), B.PLT_ERR_INVALID_ARG)]:
        base = dict(max_batch=2, L=2, Hq=8, Hkv=2, d=128, max_seq_len=512, w=64)
        base.update(kw)
        with pytest.raises(B.PltError) as e:
            B.plt_seq_attn_create(B.make_seq_config(**base))
        assert e.value.status == code, (kw, e.value)
    B.plt_seq_attn_destroy(None)


def test_create_without_a_device_fails_loudly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    from paper_2510_24824_b200 import binding as B
    with pytest.raises(B.PltError) as e:
        B.plt_decode_attn_create(B.make_config("bf16", 4, 2, 8, 2, 128, 512, 64))
    assert e.value.status == B.PLT_ERR_CUDA
