"""A few hundred tokens on the tensor-core plan: the down projection's contraction is split in two (two problems of one
GEMM launch into fp32 partial outputs, added by a small kernel) because its output has too few tiles for the GPU.
Forward against the oracle on shapes inside that range, with ragged and padded channel counts."""
import numpy as np
import pytest
import torch

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


@pytest.mark.parametrize("T,d,F,F_ld,K", [
    (400, 1024, 2048, 2048, 256),    # two halves of 1024 channels
    (257, 512, 2000, 2048, 250),     # the smallest batch of the plan; halves of 1024 and 976 channels, padding rows
    (512, 768, 2047 + 9, 2056, 257), # second half ends inside a 64-channel block
    (300, 264, 1000, 1000, 125),     # output 264 columns wide: two column tiles, the second 8 wide
])
def test_forward_with_split_down_projection(T, d, F, F_ld, K):
    w = syn.Workload(f"split-{T}-{d}-{F}", "bf16", T, d, F, F_ld, K, seed=7000 + T)
    wg, wu, wd = syn.make_weights(w)
    if F_ld > F:
        for m in (wg, wu, wd):
            m[F:] = 3.0
    x = syn.make_x(w)
    xd, wgd, wud, wdd = (t.cuda() for t in (x, wg, wu, wd))
    B.moc_profile_enable(True)
    out, idx, tg, tu = B.moc_ffn_forward(xd, wgd, wud, wdd, K, d_ff=F)
    prof = B.moc_profile_collect()
    B.moc_profile_enable(False)
    names = {k for k, (n, _) in prof.items() if n}
    assert "tc_split_sum" in names and "tc_down_gemm" in names, names
    x64, wg64, wu64, wd64 = map(syn.to_f64, (x, wg[:F], wu[:F], wd[:F]))
    dev = dict(out=syn.to_f64(out), idx=idx.cpu().numpy(), gval=syn.to_f64(tg), uval=syn.to_f64(tu))
    parity.check_forward(dev, x64, wg64, wu64, wd64, K, F, w.dtype)
    # the unsplit GEMM of a batch just above the range gives the same rows
    big = torch.cat([xd, xd, xd, xd, xd, xd, xd, xd, xd])[: max(2400, 5 * T)]
    out_big = B.moc_ffn_forward(big, wgd, wud, wdd, K, d_ff=F, save=False)[0]
    torch.cuda.synchronize()
    torch.testing.assert_close(out.float(), out_big[:T].float(), rtol=2e-2, atol=2e-3 * float(out.float().abs().max()))


@pytest.mark.parametrize("T,d,F,F_ld,K", [
    (400, 1024, 2048, 2048, 256),
    (257, 520, 2000, 2048, 250),     # output 520 columns wide: three column tiles, the last 8 wide; padding rows
])
def test_backward_with_split_grad_x(T, d, F, F_ld, K):
    """The grad_x GEMM of the same range: its two contraction segments (dG' Wg and dU' Wu, Eq. (bp-5)) run as two
    problems of one launch into fp32 partial outputs, which the same small kernel adds."""
    w = syn.Workload(f"splitb-{T}-{d}-{F}", "bf16", T, d, F, F_ld, K, seed=7100 + T)
    wg, wu, wd = syn.make_weights(w)
    x, dD = syn.make_x(w), syn.make_grad_out(w)
    xd, wgd, wud, wdd, dDd = (t.cuda() for t in (x, wg, wu, wd, dD))
    out, idx, tg, tu = B.moc_ffn_forward(xd, wgd, wud, wdd, K, d_ff=F)
    B.moc_profile_enable(True)
    grads = B.moc_ffn_backward(xd, wgd, wud, wdd, idx, tg, tu, dDd, d_ff=F)
    prof = B.moc_profile_collect()
    B.moc_profile_enable(False)
    assert prof.get("tc_split_sum", (0, 0))[0] == 1 and prof.get("tc_dx_gemm", (0, 0))[0] == 1, prof
    torch.cuda.synchronize()
    x64, wg64, wu64, wd64, dD64 = map(syn.to_f64, (x, wg[:F], wu[:F], wd[:F], dD))
    gdev = {k: syn.to_f64(v) for k, v in grads.items()}
    parity.check_backward(gdev, x64, wg64, wu64, wd64, idx.cpu().numpy(), syn.to_f64(tg), syn.to_f64(tu), dD64, F, w.dtype)
    # only grad_x asked for: the same path, the same bits (the halves are added in a fixed order)
    gx = B.moc_ffn_backward(xd, wgd, wud, wdd, idx, tg, tu, dDd, d_ff=F, want=("x",))["grad_x"]
    torch.cuda.synchronize()
    assert torch.equal(gx, grads["grad_x"])
