"""`moc_ffn_decode_block`: out = h + MoC_FFN(RMSNorm(h)) on the three small-batch plans, against the oracle."""
import numpy as np
import pytest
import torch

from oracle import moc_oracle as orc
from oracle import parity
from paper_2511_09323_b200 import binding as B
from paper_2511_09323_b200 import build as moc_build
from paper_2511_09323_b200 import synthetic as syn

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    moc_build.build()
    B.load()
    assert B.moc_last_device_status() == B.MOC_OK
    yield
    assert B.moc_last_device_status() == B.MOC_OK


def _bf16(a):
    """What storing float64 values as bf16 does to them (round to nearest even)."""
    return torch.from_numpy(np.ascontiguousarray(a)).to(torch.bfloat16).double().numpy()


def _inputs(w, scale=2.5):
    wg, wu, wd = syn.make_weights(w)
    gen = torch.Generator().manual_seed(w.seed + 1000)
    h = (torch.randn(w.tokens, w.d_model, generator=gen) * scale).to(torch.bfloat16)
    gamma = (0.5 + torch.rand(w.d_model, generator=gen)).to(torch.bfloat16)
    return h, gamma, wg, wu, wd


def _check(out_dev, h, gamma, eps, wg, wu, wd, K, what):
    h64, g64, wg64, wu64, wd64 = map(syn.to_f64, (h, gamma, wg, wu, wd))
    ref, x, full = orc.decode_block(h64, g64, eps, wg64, wu64, wd64, K, store=_bf16)
    out64 = syn.to_f64(out_dev)
    F = wg64.shape[0]
    tol = parity.REL_TOL["bf16"] * np.abs(ref).max()
    for t in range(h64.shape[0]):
        err = np.abs(out64[t] - ref[t]).max()
        if err <= tol:
            continue
        # a token whose K-th and (K+1)-th gate values nearly tie may have taken the swapped pick (the device
        # normalises in fp32: a rare element of its input differs from the oracle's by one bf16 step)
        g = full["g"][t]
        order = np.lexsort((np.arange(F), -g))
        assert K < F and g[order[K - 1]] - g[order[K]] <= 1e-3, f"{what}: token {t} error {err:.3e} > {tol:.3e}"
        alt = np.sort(np.concatenate([order[: K - 1], order[K: K + 1]])).astype(np.int32)[None]
        alt_out = h64[t] + orc.forward_given_idx(x[t: t + 1], wg64, wu64, wd64, alt)["out"][0]
        assert np.abs(out64[t] - alt_out).max() <= tol, f"{what}: token {t} matches neither pick"


@pytest.mark.parametrize("T,d,F,F_ld,K", [
    (1, 264, 333, 336, 41),        # cooperative kernel, ragged everything
    (2, 520, 776, 776, 97),        # cooperative kernel, two tokens
    (3, 264, 333, 336, 41),        # four-kernel plan
    (5, 520, 776, 776, 97),
    (16, 128, 1000, 1024, 125),    # small-batch plan from here on (half of the channels in use)
    (40, 768, 2048, 2048, 256),
    (256, 256, 520, 520, 65),
])
def test_block_against_oracle(T, d, F, F_ld, K):
    w = syn.Workload(f"blk-{T}-{d}-{F}", "bf16", T, d, F, F_ld, K, seed=4100 + T)
    h, gamma, wg, wu, wd = _inputs(w)
    out = B.moc_ffn_decode_block(h.cuda(), gamma.cuda(), 1e-5, wg.cuda(), wu.cuda(), wd.cuda(), K, d_ff=F)
    torch.cuda.synchronize()
    _check(out, h, gamma, 1e-5, wg[:F], wu[:F], wd[:F], K, f"block T={T}")


@pytest.mark.parametrize("T", [1, 4, 17])
def test_block_llama7b_shape(T):
    w = syn.C4.with_tokens(T)
    h, gamma, wg, wu, wd = _inputs(w, scale=1.0)
    out = B.moc_ffn_decode_block(h.cuda(), gamma.cuda(), 1e-6, wg.cuda(), wu.cuda(), wd.cuda(), w.k)
    torch.cuda.synchronize()
    _check(out, h, gamma, 1e-6, wg, wu, wd, w.k, f"7B block T={T}")


@pytest.mark.parametrize("T", [2, 6, 48])
def test_block_in_place_and_against_the_unfused_steps(T):
    """`out` may be `h`; and the call agrees with RMSNorm (torch, fp32) -> moc_ffn_decode -> add, up to the one
    rounding of D that the unfused chain has on top."""
    w = syn.Workload(f"blk-ip-{T}", "bf16", T, 256, 1024, 1024, 128, seed=4200 + T)
    h, gamma, wg, wu, wd = _inputs(w)
    hd, gd, wgd, wud, wdd = (t.cuda() for t in (h, gamma, wg, wu, wd))
    out = B.moc_ffn_decode_block(hd, gd, 1e-5, wgd, wud, wdd, w.k)
    inplace = hd.clone()
    B.moc_ffn_decode_block(inplace, gd, 1e-5, wgd, wud, wdd, w.k, out=inplace)
    torch.cuda.synchronize()
    torch.testing.assert_close(inplace.float(), out.float(), rtol=1e-2, atol=1e-2)
    hf = hd.float()
    xn = (hf * torch.rsqrt(hf.pow(2).mean(dim=1, keepdim=True) + 1e-5) * gd.float()).to(torch.bfloat16)
    D = B.moc_ffn_decode(xn, wgd, wud, wdd, w.k)
    torch.testing.assert_close(out.float(), hf + D.float(), rtol=2e-2, atol=2e-2)


def test_block_two_of_eight_mask():
    w = syn.Workload("blk-g28", "bf16", 3, 256, 1024, 1024, 256, seed=4300)
    h, gamma, wg, wu, wd = _inputs(w)
    hd, gd, wgd, wud, wdd = (t.cuda() for t in (h, gamma, wg, wu, wd))
    for T in (1, 3):
        out = B.moc_ffn_decode_block(hd[:T], gd, 1e-5, wgd, wud, wdd, None, grouped=True)
        torch.cuda.synchronize()
        h64, g64, wg64, wu64, wd64 = map(syn.to_f64, (h[:T], gamma, wg, wu, wd))
        x = _bf16(orc.rmsnorm(h64, g64, 1e-5))
        ref = orc.residual(h64, orc.forward_grouped(x, wg64, wu64, wd64)["out"])
        parity.assert_close(syn.to_f64(out), ref, "bf16", f"2:8 block T={T}")


def test_block_argument_errors():
    w = syn.Workload("blk-err", "bf16", 4, 64, 96, 96, 12, seed=4400)
    h, gamma, wg, wu, wd = _inputs(w)
    hd, gd, wgd, wud, wdd = (t.cuda() for t in (h, gamma, wg, wu, wd))
    with pytest.raises(B.MocError):   # fp32 storage has no block form
        B.moc_ffn_decode_block(hd.float(), gd.float(), 1e-5, wgd.float(), wud.float(), wdd.float(), w.k)
    with pytest.raises(B.MocError):   # a workspace that is too small
        B.moc_ffn_decode_block(hd, gd, 1e-5, wgd, wud, wdd, w.k, workspace=torch.empty(64, dtype=torch.uint8, device="cuda"))
    with pytest.raises(B.MocError):   # negative eps
        B.moc_ffn_decode_block(hd, gd, -1.0, wgd, wud, wdd, w.k)
    assert B.moc_last_device_status() == B.MOC_OK


@pytest.mark.parametrize("T,d,F,F_ld,K", [
    (6, 264, 333, 336, 41),        # ragged everything, one stage per matrix
    (16, 2048, 5461, 5464, 683),   # the LLaMA-1B layer
    (32, 1024, 2048, 2048, 256),   # the largest batch of the one-kernel form
])
def test_block_in_one_kernel_for_a_few_dozen_tokens(T, d, F, F_ld, K):
    """5 to 32 tokens (at K = d_ff / 8): one cooperative kernel, no normalisation kernel in front (its selector CTAs normalise the
    tokens); `out` may be `h`; a second call on the same workspace gives the same."""
    w = syn.Workload(f"blk1-{T}-{d}-{F}", "bf16", T, d, F, F_ld, K, seed=4300 + T)
    h, gamma, wg, wu, wd = _inputs(w)
    hd, gd, wgd, wud, wdd = (t.cuda() for t in (h, gamma, wg, wu, wd))
    B.moc_profile_enable(True)
    out = B.moc_ffn_decode_block(hd, gd, 1e-5, wgd, wud, wdd, K, d_ff=F)
    prof = B.moc_profile_collect()
    B.moc_profile_enable(False)
    names = {k for k, (n, _) in prof.items() if n}
    assert names == {"sb_fused"}, names
    torch.cuda.synchronize()
    _check(out, h, gamma, 1e-5, wg, wu, wd, K, f"one-kernel block T={T}")
    inplace = hd.clone()
    B.moc_ffn_decode_block(inplace, gd, 1e-5, wgd, wud, wdd, K, d_ff=F, out=inplace)
    torch.cuda.synchronize()
    torch.testing.assert_close(inplace.float(), out.float(), rtol=2e-2, atol=1e-3 * float(out.float().abs().max()))
    assert B.moc_last_device_status() == B.MOC_OK
