"""moc_ffn_decode_static: the decode entry point for callers that cannot allocate device memory.

Some users of this library run where no allocator may be touched: a serving process that gave every
free byte of HBM to its KV-cache pool, a latency-critical loop that cannot take the device-wide
synchronisation cudaMalloc/cudaFree imply, a plug-in that receives tensors but no allocator.  They
call this entry point with inputs and an output buffer only; its transient buffers are an array
built into the library.  The checks below call it through the C ABI and compare it with
moc_ffn_decode (caller-provided workspace) and with the CPU oracle on two calls in a row, the
second smaller than the first, so that anything left in the shared array by the first call would
show up; one more check watches the device's free memory across a series of calls.

The file name sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import moc_oracle as orc
from oracle import parity
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
    # and against the definition itself: the two entry points may share kernels, the oracle shares nothing with them
    F = w.d_ff
    x64, wg64, wu64, wd64 = (syn.to_f64(t) for t in (x, wg[:F], wu[:F], wd[:F]))
    parity.check_decode(syn.to_f64(out), x64, wg64, wu64, wd64, w.k, w.dtype, "static decode")


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


@pytest.mark.parametrize("dtype,T,d,F,F_ld,K", [("bf16", 12, 128, 1000, 1024, 125), ("f32", 5, 72, 333, 336, 41)])
def test_static_decode_honours_the_post_silu_key(dtype, T, d, F, F_ld, K):
    """MOC_FLAG_SELECT_POST_SILU (the Top-K placed after the activation) on inputs with fewer positive gate values than
    K, where the two selection rules keep different channels: the entry point must give the post-SiLU result of the
    oracle, as moc_ffn_decode does, whichever of its kernel plans the problem size would otherwise pick."""
    w = syn.Workload("static-ps", dtype, T, d, F, F_ld, K, seed=35)
    wg, wu, wd = syn.make_weights(w)
    x = (syn.make_x(w).float() + 1.0).to(wg.dtype)
    wg = (wg.float() - 0.05 / np.sqrt(d / 128)).to(wg.dtype)
    wg[F:] = 0
    xd, wgd, wud, wdd = (t.cuda() for t in (x, wg, wu, wd))
    out = torch.full_like(xd, float("nan"))
    B.moc_ffn_decode_static(xd, wgd, wud, wdd, K, out, d_ff=F, post_silu=True)
    ref_dev = B.moc_ffn_decode(xd, wgd, wud, wdd, K, d_ff=F, post_silu=True)
    torch.cuda.synchronize()
    x64, wg64, wu64, wd64 = (syn.to_f64(t) for t in (x, wg[:F], wu[:F], wd[:F]))
    ref = orc.forward_post_silu(x64, wg64, wu64, wd64, K)
    assert np.median((ref["g"] > 0).sum(axis=1)) < K, "the inputs must make the two rules differ"
    pre = orc.forward(x64, wg64, wu64, wd64, K)
    assert not np.array_equal(ref["idx"], pre["idx"])
    got = syn.to_f64(out)
    scale = np.abs(ref["out"]).max()
    # With every gate value negative the post-SiLU rule keeps the channels whose SiLU is closest to zero; the channels
    # at its threshold carry SiLU values of a few 1e-3, so a near-tie there decided the other way moves the output by
    # far less than the tolerance: every token must match the oracle's post-SiLU output, and none the default rule's.
    err = np.abs(got - ref["out"]).max(axis=1)
    assert np.all(err <= REL[dtype] * scale), f"{err.max():.3e} vs {REL[dtype] * scale:.3e}"
    differs = np.abs(pre["out"] - ref["out"]).max(axis=1) > 10 * REL[dtype] * scale
    assert differs.sum() >= T // 2
    assert np.all(np.abs(got - pre["out"]).max(axis=1)[differs] > REL[dtype] * scale)
    assert (out.double() - ref_dev.double()).abs().max().item() <= REL[dtype] * scale


def test_static_decode_leaves_device_memory_alone():
    """What the entry point is for: after the first call on the device (which looks up the built-in array's address),
    further calls change neither the device's free memory nor what torch's allocator holds -- on the decode plan's
    kernels and on the gathered kernels alike."""
    cases = [_case("bf16", 16, 256, 1000, 1024, 125, seed=36), _case("f32", 3, 128, 333, 336, 41, seed=37)]
    outs = [torch.empty_like(c[1]) for c in cases]
    for (w, x, wg, wu, wd), out in zip(cases, outs):     # first calls: one-time set-up happens here
        B.moc_ffn_decode_static(x, wg, wu, wd, w.k, out, d_ff=w.d_ff)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    held0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for _ in range(5):
        for (w, x, wg, wu, wd), out in zip(cases, outs):
            B.moc_ffn_decode_static(x, wg, wu, wd, w.k, out, d_ff=w.d_ff)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == (held0, reserved0)
    assert free1 == free0, f"free device memory changed by {free0 - free1} bytes"
    assert B.moc_last_device_status() == B.MOC_OK


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
