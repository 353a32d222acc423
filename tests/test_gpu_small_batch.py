"""The small-batch plan (bf16, up to 256 tokens: three weight-streaming tensor-core kernels) against the oracle, through
`moc_ffn_forward` (with and without the saved triple) and `moc_ffn_decode`."""
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


def _problem(w):
    wg, wu, wd = syn.make_weights(w)
    return syn.make_x(w), wg, wu, wd, syn.make_grad_out(w)


def _forward_backward(w, junk_padding=False):
    x, wg, wu, wd, dD = _problem(w)
    if junk_padding:
        for m in (wg, wu, wd):
            m[w.d_ff:] = 3.0      # larger than any real gate value: must never be selected or read as channels
    xd, wgd, wud, wdd, dDd = (t.cuda() for t in (x, wg, wu, wd, dD))
    out, idx, tg, tu = B.moc_ffn_forward(xd, wgd, wud, wdd, w.k, d_ff=w.d_ff)
    torch.cuda.synchronize()
    x64, wg64, wu64, wd64, dD64 = map(syn.to_f64, (x, wg[:w.d_ff], wu[:w.d_ff], wd[:w.d_ff], dD))
    dev = dict(out=syn.to_f64(out), idx=idx.cpu().numpy(), gval=syn.to_f64(tg), uval=syn.to_f64(tu))
    rep = parity.check_forward(dev, x64, wg64, wu64, wd64, w.k, w.d_ff, w.dtype)
    grads = B.moc_ffn_backward(xd, wgd, wud, wdd, idx, tg, tu, dDd, d_ff=w.d_ff)
    torch.cuda.synchronize()
    gdev = {k: syn.to_f64(v) for k, v in grads.items()}
    parity.check_backward(gdev, x64, wg64, wu64, wd64, dev["idx"], dev["gval"], dev["uval"], dD64, w.d_ff, w.dtype)
    return rep, (xd, wgd, wud, wdd), (out, idx, tg, tu)


def _check_against_oracle_picks(out64, x64, wg64, wu64, wd64, K, what):
    """No indices come back, so the comparison is with the oracle's own picks; a token whose K-th and (K+1)-th gate
    values are closer than 1e-4 (inside the 1e-3 exclusion band) may have taken the swapped pick."""
    full = orc.forward(x64, wg64, wu64, wd64, K, want_g=True)
    F = wg64.shape[0]
    tol = parity.REL_TOL["bf16"] * np.abs(full["out"]).max()
    for t in range(x64.shape[0]):
        err = np.abs(out64[t] - full["out"][t]).max()
        if err <= tol:
            continue
        g = full["g"][t]
        order = np.lexsort((np.arange(F), -g))
        assert K < F and g[order[K - 1]] - g[order[K]] <= 1e-4, f"{what}: token {t} error {err:.3e} > {tol:.3e}"
        alt = np.sort(np.concatenate([order[: K - 1], order[K: K + 1]])).astype(np.int32)[None]
        ref = orc.forward_given_idx(x64[t: t + 1], wg64, wu64, wd64, alt)["out"][0]
        assert np.abs(out64[t] - ref).max() <= tol, f"{what}: token {t} matches neither pick"


@pytest.mark.parametrize("T,d,F,F_ld,K", [
    (17, 64, 96, 96, 12),          # the smallest batch of the plan, a single tile of everything
    (32, 264, 333, 336, 41),       # contraction 4 blocks + 8 elements; channels 2 tiles + ragged tail
    (33, 128, 1000, 1024, 125),    # 64-token MMA with 31 empty columns
    (64, 768, 2048, 2048, 256),    # the 130M layer
    (100, 520, 777, 784, 97),      # 128-token MMA, five column blocks in the down projection, the last 8 wide
    (128, 256, 520, 520, 1),       # a single kept channel
    (128, 136, 264, 264, 264),     # K = F: dense SwiGLU
    (40, 64, 200, 200, 199),       # all but one channel kept
    (24, 64, 16000, 16000, 1200),  # rows longer than the selector keeps in registers
    (20, 64, 24000, 24000, 1500),  # rows so long that the up row stays in global memory
    (6, 64, 96, 96, 12),           # below 17 tokens the plan runs where at least half of the channels are in use
    (20, 8, 8, 8, 1),              # the smallest width of everything
    (200, 264, 333, 336, 41),      # 224-token MMA
    (256, 768, 2048, 2048, 256),   # the largest batch: 256-token MMA, all of the tensor memory
    (256, 64, 20000, 20000, 300),  # 256 tokens x 256-channel tiles: the gate+up tile does not fit the ring (direct stores)
])
def test_small_batch_forward_backward(T, d, F, F_ld, K):
    w = syn.Workload(f"sb-{T}-{d}-{F}-{K}", "bf16", T, d, F, F_ld, K, seed=900 + T)
    _forward_backward(w)


def test_small_batch_llama1b_padded_shape_with_junk_in_the_padding_rows():
    _forward_backward(syn.C3.with_tokens(48), junk_padding=True)


@pytest.mark.parametrize("T", [17, 64, 128, 256])
def test_small_batch_decode_llama7b_shape(T):
    w = syn.C4.with_tokens(T)
    wg, wu, wd = syn.make_weights(w)
    x = syn.make_x(w)
    out = B.moc_ffn_decode(x.cuda(), wg.cuda(), wu.cuda(), wd.cuda(), w.k)
    torch.cuda.synchronize()
    x64, wg64, wu64, wd64 = map(syn.to_f64, (x, wg, wu, wd))
    _check_against_oracle_picks(syn.to_f64(out), x64, wg64, wu64, wd64, w.k, f"decode T={T}")


def test_small_batch_decode_forward_without_saves_and_workspace_reuse():
    """decode == forward(save=False) up to the summation order of the down projection's partial sums; one workspace
    serves calls of different batch sizes back to back (its counters and accumulator are left ready)."""
    w = syn.Workload("sb-reuse", "bf16", 128, 256, 1000, 1000, 125, seed=41)
    x, wg, wu, wd, _ = _problem(w)
    xd, wgd, wud, wdd = (t.cuda() for t in (x, wg, wu, wd))
    desc = B.make_desc(128, w.d_model, w.d_ff, w.k, xd.dtype)
    ws = B.alloc_workspace(desc, B.MOC_OP_DECODE, xd.device)
    ws.fill_(0xff)   # nothing may depend on what the workspace held
    x64, wg64, wu64, wd64 = map(syn.to_f64, (x, wg, wu, wd))
    for T in (128, 20, 77, 128):
        out = B.moc_ffn_decode(xd[:T], wgd, wud, wdd, w.k, workspace=ws)
        out_f, *_ = B.moc_ffn_forward(xd[:T], wgd, wud, wdd, w.k, save=False, workspace=ws)
        torch.cuda.synchronize()
        torch.testing.assert_close(out.float(), out_f.float(), rtol=2e-2, atol=1e-3)
        _check_against_oracle_picks(syn.to_f64(out), x64[:T], wg64, wu64, wd64, w.k, f"decode T={T}")
    assert B.moc_last_device_status() == B.MOC_OK


def test_small_batch_ties_and_degenerate_tokens():
    """Duplicated gate rows (bit-identical gate values: the lower channel of a pair wins), an all-zero token (every
    value ties: channels 0..K-1), and a token scaled by 1e4."""
    w = syn.Workload("sb-ties", "bf16", 64, 128, 512, 512, 65, seed=77)
    wg, wu, wd = syn.make_weights(w)
    wg[1::2] = wg[0::2]
    x = syn.make_x(w)
    x[5] = 0
    x[9] *= 1e4
    out, idx, tg, tu = B.moc_ffn_forward(x.cuda(), wg.cuda(), wu.cuda(), wd.cuda(), w.k)
    idx = idx.cpu().numpy().astype(np.int64)
    np.testing.assert_array_equal(idx[5], np.arange(w.k))
    assert torch.all(out[5] == 0)
    for t in range(w.tokens):
        sel = set(idx[t].tolist())
        for j in idx[t]:
            if j % 2 == 1:
                assert j - 1 in sel, f"token {t}: channel {j} kept without its equal lower twin {j - 1}"
    x64, wg64, wu64, wd64 = map(syn.to_f64, (x, wg, wu, wd))
    dev = dict(out=syn.to_f64(out), idx=idx, gval=syn.to_f64(tg), uval=syn.to_f64(tu))
    parity.check_forward(dev, x64, wg64, wu64, wd64, w.k, w.d_ff, w.dtype)


@pytest.mark.parametrize("T", [24, 128])
def test_small_batch_grouped_mask(T):
    """MoC 2:8 through the small-batch plan: picks per group, values on the device's picks, decode == forward."""
    w = syn.Workload(f"sb-g28-{T}", "bf16", T, 256, 1024, 1024, 256, seed=2800 + T)
    x, wg, wu, wd, dD = _problem(w)
    xd, wgd, wud, wdd, dDd = (t.cuda() for t in (x, wg, wu, wd, dD))
    out, idx, tg, tu = B.moc_ffn_forward(xd, wgd, wud, wdd, None, grouped=True)
    out_d = B.moc_ffn_decode(xd, wgd, wud, wdd, None, grouped=True)
    grads = B.moc_ffn_backward(xd, wgd, wud, wdd, idx, tg, tu, dDd)
    torch.cuda.synchronize()
    x64, wg64, wu64, wd64, dD64 = map(syn.to_f64, (x, wg, wu, wd, dD))
    idx_np = idx.cpu().numpy()
    parity.check_picks_grouped(idx_np, orc.gate_projection(x64, wg64))
    ref = orc.forward_given_idx(x64, wg64, wu64, wd64, idx_np.astype(np.int32))
    parity.assert_close(syn.to_f64(out), ref["out"], "bf16", "out")
    parity.assert_close(syn.to_f64(out_d), ref["out"], "bf16", "decode out")
    parity.assert_close(syn.to_f64(tg), ref["gval"], "bf16", "topk_gate")
    parity.assert_close(syn.to_f64(tu), ref["uval"], "bf16", "topk_up")
    gdev = {k: syn.to_f64(v) for k, v in grads.items()}
    parity.check_backward(gdev, x64, wg64, wu64, wd64, idx_np, syn.to_f64(tg), syn.to_f64(tu), dD64, w.d_ff, "bf16")
