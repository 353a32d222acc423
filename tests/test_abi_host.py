"""CPU-side checks of the C-ABI library: it builds, loads, exports every declared symbol, and its
host-side validation rejects bad calls before anything touches a GPU."""
import ctypes
import os
import re

import pytest

from paper_2511_09323_b200 import binding as B
from paper_2511_09323_b200 import build as moc_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    moc_build.build()
    return B.load()


def _declared_symbols():
    names = []
    inc = os.path.join(ROOT, "include")
    for fn in sorted(os.listdir(inc)):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            names += re.findall(r"MOC_API\s+[\w\s\*]+?\b(moc_\w+)\s*\(", text)
    return names


def test_library_exports_every_declared_symbol(lib):
    names = _declared_symbols()
    assert len(names) >= 8
    for n in names:
        assert hasattr(lib, n), n
    assert set(B.EXPORTED) <= set(names)


def test_status_strings(lib):
    seen = set()
    for code in range(0, -7, -1):
        s = B.status_string(code)
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 7
    assert B.status_string(-99) == "unknown status"


def test_descriptor_validation_is_host_side(lib):
    ok = B.make_desc(256, 128, 512, 64, B.MOC_F32)
    assert B.moc_ffn_workspace_bytes(ok, B.MOC_OP_FORWARD) > 0
    assert B.moc_ffn_workspace_bytes(ok, B.MOC_OP_BACKWARD) > 0
    assert B.moc_ffn_workspace_bytes(ok, B.MOC_OP_DECODE) > 0   # 256 tokens: the largest decode batch
    assert B.moc_ffn_workspace_bytes(B.make_desc(257, 128, 512, 64, B.MOC_F32), B.MOC_OP_DECODE) == 0
    assert B.moc_ffn_saved_bytes_per_token(ok) == 64 * (2 + 2 * 4)
    assert B.moc_ffn_saved_bytes_per_token(B.make_desc(1, 2048, 5504, 688, B.MOC_BF16)) == 4128
    bad = [
        B.make_desc(256, 128, 512, 0, B.MOC_F32),       # k < 1
        B.make_desc(256, 128, 512, 513, B.MOC_F32),     # k > d_ff
        B.make_desc(-1, 128, 512, 64, B.MOC_F32),       # negative tokens
        B.make_desc(256, 128, 512, 64, B.MOC_F32, d_ff_ld=500),
        B.make_desc(256, 128, 512, 64, B.MOC_F32, flags=8),
    ]
    for d in bad:
        assert B.moc_ffn_workspace_bytes(d, B.MOC_OP_FORWARD) == 0
        rc = lib.moc_ffn_forward(ctypes.byref(d), *([None] * 9), 0, None)
        assert rc == B.MOC_ERR_INVALID_ARG
    unsupported = [
        B.make_desc(256, 128, 40000, 64, B.MOC_F32),    # int16 indices
        B.make_desc(256, 100, 512, 64, B.MOC_F32),      # d_model % 8
        B.make_desc(256, 128, 512, 64, 7),              # dtype
        B.make_desc(2 ** 31, 128, 512, 64, B.MOC_F32),  # tokens * k >= 2^32
    ]
    for d in unsupported:
        rc = lib.moc_ffn_backward(ctypes.byref(d), *([None] * 13), 0, None)
        assert rc == B.MOC_ERR_UNSUPPORTED
    assert lib.moc_ffn_forward(None, *([None] * 9), 0, None) == B.MOC_ERR_INVALID_ARG


def test_null_pointers_and_small_workspace_are_rejected_before_launch(lib):
    d = B.make_desc(4, 16, 32, 4, B.MOC_BF16)
    # NULL data pointers
    assert lib.moc_ffn_forward(ctypes.byref(d), *([None] * 9), 0, None) == B.MOC_ERR_INVALID_ARG
    # misaligned pointer (fake addresses are never dereferenced: validation fails first)
    fake = ctypes.c_void_p(0x1000)
    odd = ctypes.c_void_p(0x1004)
    assert lib.moc_ffn_forward(ctypes.byref(d), odd, fake, fake, fake, fake, None, None, None, None, 0,
                               None) == B.MOC_ERR_INVALID_ARG
    # some but not all of the saved outputs
    assert lib.moc_ffn_forward(ctypes.byref(d), fake, fake, fake, fake, fake, fake, None, None, None, 0,
                               None) == B.MOC_ERR_INVALID_ARG
    # workspace missing / too small
    assert lib.moc_ffn_forward(ctypes.byref(d), fake, fake, fake, fake, fake, None, None, None, None, 0,
                               None) == B.MOC_ERR_WORKSPACE
    assert lib.moc_ffn_forward(ctypes.byref(d), fake, fake, fake, fake, fake, None, None, None, fake, 8,
                               None) == B.MOC_ERR_WORKSPACE
    assert lib.moc_ffn_backward(ctypes.byref(d), *([fake] * 12), None, 0, None) == B.MOC_ERR_WORKSPACE
    # decode batch limit
    big = B.make_desc(257, 16, 32, 4, B.MOC_BF16)
    assert lib.moc_ffn_decode(ctypes.byref(big), fake, fake, fake, fake, fake, None, 0, None) == B.MOC_ERR_UNSUPPORTED
    # zero tokens is a no-op that needs no buffers
    zero = B.make_desc(0, 16, 32, 4, B.MOC_BF16)
    assert lib.moc_ffn_forward(ctypes.byref(zero), *([None] * 9), 0, None) == B.MOC_OK
    assert B.moc_ffn_workspace_bytes(zero, B.MOC_OP_FORWARD) == 0
    # selector argument checks
    assert lib.moc_topk_select(4, 8, 8, 9, fake, fake, None) == B.MOC_ERR_INVALID_ARG
    assert lib.moc_topk_select(4, 40000, 40000, 9, fake, fake, None) == B.MOC_ERR_UNSUPPORTED
    assert lib.moc_topk_select(0, 8, 8, 2, None, None, None) == B.MOC_OK


def test_block_form_and_selection_flags_are_validated_on_the_host(lib):
    fake = ctypes.c_void_p(0x1000)
    eps = ctypes.c_float(1e-6)
    block = lambda d, *ptrs, ws=None, n=0, e=eps: lib.moc_ffn_decode_block(ctypes.byref(d), ptrs[0], ptrs[1], e, *ptrs[2:],
                                                                         ws, n, None)
    zero = B.make_desc(0, 16, 32, 8, B.MOC_BF16)
    assert block(zero, *([None] * 6)) == B.MOC_OK                       # no tokens: a no-op that needs no buffers
    f32 = B.make_desc(4, 16, 32, 8, B.MOC_F32)
    assert B.moc_ffn_workspace_bytes(f32, B.MOC_OP_DECODE_BLOCK) == 0   # bf16 only
    assert block(f32, *([fake] * 6)) == B.MOC_ERR_UNSUPPORTED
    big = B.make_desc(257, 16, 32, 8, B.MOC_BF16)
    assert block(big, *([fake] * 6)) == B.MOC_ERR_UNSUPPORTED           # at most 256 tokens
    d = B.make_desc(4, 16, 32, 8, B.MOC_BF16)
    need = B.moc_ffn_workspace_bytes(d, B.MOC_OP_DECODE_BLOCK)
    assert need > B.moc_ffn_workspace_bytes(d, B.MOC_OP_DECODE) > 0     # the normalised rows live behind the decode workspace
    assert block(d, *([None] * 6)) == B.MOC_ERR_INVALID_ARG
    assert block(d, *([fake] * 6), e=ctypes.c_float(-1.0)) == B.MOC_ERR_INVALID_ARG
    assert block(d, *([fake] * 6)) == B.MOC_ERR_WORKSPACE
    assert block(d, *([fake] * 6), ws=fake, n=need - 1) == B.MOC_ERR_WORKSPACE
    # selection flags: the two rules exclude each other; the post-SiLU variant has no block form
    both = B.make_desc(4, 16, 32, 8, B.MOC_BF16, flags=B.MOC_FLAG_SELECT_2_OF_8 | B.MOC_FLAG_SELECT_POST_SILU)
    assert lib.moc_ffn_forward(ctypes.byref(both), *([None] * 9), 0, None) == B.MOC_ERR_INVALID_ARG
    post = B.make_desc(4, 16, 32, 8, B.MOC_BF16, flags=B.MOC_FLAG_SELECT_POST_SILU)
    assert B.moc_ffn_workspace_bytes(post, B.MOC_OP_FORWARD) > 0
    assert B.moc_ffn_workspace_bytes(post, B.MOC_OP_DECODE) > 0
    assert B.moc_ffn_workspace_bytes(post, B.MOC_OP_DECODE_BLOCK) == 0
    assert block(post, *([fake] * 6)) == B.MOC_ERR_UNSUPPORTED


def test_binding_fails_loudly_without_library(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(RuntimeError):
        B.load()
