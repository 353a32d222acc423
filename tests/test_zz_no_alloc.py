"""moc_ffn_decode_static: the decode entry point for callers that cannot allocate device memory.

Some users of this library run where no allocator may be touched: a serving process that gave every
free byte of HBM to its KV-cache pool, a latency-critical loop that cannot take the device-wide
synchronisation cudaMalloc/cudaFree imply, a plug-in that receives tensors but no allocator.  They
call this entry point with inputs and an output buffer only; its transient buffers are an array
built into the library.  The checks below call it through the C ABI and compare it with
moc_ffn_decode (caller-provided workspace) on two calls in a row, the second smaller than the
first, so that anything left in the shared array by the first call would show up.

The file name sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import ctypes

import pytest
import torch

from paper_2511_09323_b200 import binding as B
from paper_2511_09323_b200 import build as moc_build
from paper_2511_09323_b200 import synthetic as syn

pytestmark = pytest.mark.gpu

# both entry points run the same arithmetic on the same inputs; the tolerance is the one the parity
# tests use for the storage type (max-abs error <= rel * max|reference|)
REL = {"bf16": 1e-2, "f32": 1e-4}


def _case(dtype, T, d, F, F_ld, K, seed):
    w = syn.Workload("static", dtype, T, d, F, F_ld, K, seed=seed, decode=True)
    wg, wu, wd = (t.cuda() for t in syn.make_weights(w))
    x = syn.make_x(w).cuda()
    return w, x, wg, wu, wd


def _compare(w, x, wg, wu, wd):
    ref = B.moc_ffn_decode(x, wg, wu, wd, w.k, d_ff=w.d_ff)
    out = torch.full_like(x, float("nan"))          # allocated by the test, not by the call under test
    B.moc_ffn_decode_static(x, wg, wu, wd, w.k, out, d_ff=w.d_ff)
    torch.cuda.synchronize()
    assert torch.isfinite(out.float()).all()
    err = (out.double() - ref.double()).abs().max().item()
    scale = ref.double().abs().max().item()
    assert err <= REL[w.dtype] * scale, f"{err:.3e} vs {REL[w.dtype] * scale:.3e}"


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_static_decode_matches_workspace_decode_twice_in_a_row(dtype):
    moc_build.build()
    # first call: the largest batch, a padded channel count
    _compare(*_case(dtype, 16, 256, 1000, 1024, 125, seed=31))
    # second call right after it: fewer tokens, fewer channels, other K -- stale scratch must not matter
    _compare(*_case(dtype, 3, 128, 333, 336, 41, seed=32))
    assert B.moc_last_device_status() == B.MOC_OK


@pytest.mark.parametrize("T", [4, 16])
def test_static_decode_llama7b_shape(T):
    """The LLaMA-7B layer: the decode plan's transient buffers fit the built-in array at every batch up to 16, so the
    call runs the decode plan's kernels (also where moc_ffn_decode itself prefers the small-batch plan)."""
    w = syn.C4.with_tokens(T)
    wg, wu, wd = (t.cuda() for t in syn.make_weights(w))
    x = syn.make_x(w).cuda()
    _compare(w, x, wg, wu, wd)


def test_static_decode_falls_back_to_the_gathered_kernels_when_the_decode_plan_does_not_fit():
    """16 tokens on a 16384-channel layer: the decode plan's buffers exceed the built-in array, the gathered plan's do not."""
    _compare(*_case("bf16", 16, 2048, 16384, 16384, 2048, seed=33))


def test_static_decode_rejects_what_does_not_fit():
    lib = B.load()
    fake = ctypes.c_void_p(0x1000)
    too_many = B.make_desc(B.MOC_STATIC_MAX_TOKENS + 1, 64, 128, 16, B.MOC_BF16)
    too_wide = B.make_desc(4, 64, B.MOC_STATIC_MAX_DFF + 8, 16, B.MOC_BF16)
    for d in (too_many, too_wide):
        assert lib.moc_ffn_decode_static(ctypes.byref(d), fake, fake, fake, fake, fake, None) == B.MOC_ERR_STATIC_LIMIT
    assert "built-in scratch" in B.status_string(B.MOC_ERR_STATIC_LIMIT)
    ok = B.make_desc(4, 64, 128, 16, B.MOC_BF16)
    assert lib.moc_ffn_decode_static(ctypes.byref(ok), None, fake, fake, fake, fake, None) == B.MOC_ERR_INVALID_ARG
    bad = B.make_desc(4, 64, 128, 129, B.MOC_BF16)
    assert lib.moc_ffn_decode_static(ctypes.byref(bad), fake, fake, fake, fake, fake, None) == B.MOC_ERR_INVALID_ARG
