"""MOC_FLAG_SELECT_POST_SILU: the Top-K on SiLU(g) (the ablation variant), against the oracle."""
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


def _mostly_negative(w, share):
    """Weights and inputs whose gate values are positive for about `share` of the channels: x gets a common positive
    component and the gate weights a negative one, which shifts every gate value down."""
    wg, wu, wd = syn.make_weights(w)
    x = syn.make_x(w)
    if share < 0.5:
        x = (x.float() + 1.0).to(x.dtype)
        wg = (wg.float() - 0.02 * (1.2 if share > 0.1 else 2.5) / np.sqrt(w.d_model / 128)).to(wg.dtype)
    return x, wg, wu, wd


def _check_picks(idx_dev, s, K, band=1e-3):
    """Device picks against the oracle's keys s [T, F]: all channels clearly above the threshold are kept, none
    clearly below it, K distinct ascending channels per token."""
    T, F = s.shape
    idx_dev = idx_dev.astype(np.int64)
    for t in range(T):
        row = idx_dev[t]
        assert np.all(np.diff(row) > 0) and row[0] >= 0 and row[-1] < F
        order = np.sort(s[t])[::-1]
        tau = order[K - 1]
        margin = band * max(1.0, np.abs(s[t]).max())
        kept = np.zeros(F, bool)
        kept[row] = True
        assert np.all(kept[s[t] > tau + margin]), f"token {t}: a channel clearly above the threshold is missing"
        assert not np.any(kept[s[t] < tau - margin]), f"token {t}: a channel clearly below the threshold was kept"


@pytest.mark.parametrize("dtype,T,d,F,F_ld,K,share", [
    ("f32", 64, 128, 512, 512, 64, 0.5),      # enough positive gate values: the same picks as the default rule
    ("f32", 64, 128, 512, 512, 64, 0.05),     # fewer positive values than K: SiLU reorders the negative ones
    ("f32", 33, 72, 333, 336, 41, 0.05),      # ragged sizes, padded weight rows
    ("bf16", 40, 128, 1000, 1024, 125, 0.05),  # bf16 storage: small batch
    ("bf16", 300, 256, 512, 512, 96, 0.2),    # bf16 storage: a batch the tensor-core plan would take otherwise
])
def test_post_silu_forward_backward(dtype, T, d, F, F_ld, K, share):
    w = syn.Workload(f"ps-{dtype}-{T}-{F}", dtype, T, d, F, F_ld, K, seed=5100 + T)
    x, wg, wu, wd = _mostly_negative(w, share)
    dD = syn.make_grad_out(w)
    xd, wgd, wud, wdd, dDd = (t.cuda() for t in (x, wg, wu, wd, dD))
    out, idx, tg, tu = B.moc_ffn_forward(xd, wgd, wud, wdd, K, d_ff=F, post_silu=True)
    out_d = B.moc_ffn_decode(xd[:16], wgd, wud, wdd, K, d_ff=F, post_silu=True)
    torch.cuda.synchronize()
    x64, wg64, wu64, wd64, dD64 = map(syn.to_f64, (x, wg[:F], wu[:F], wd[:F], dD))
    ref = orc.forward_post_silu(x64, wg64, wu64, wd64, K)
    n_pos = (ref["g"] > 0).sum(axis=1)
    if share < 0.5:
        assert np.median(n_pos) < K, "the inputs must make the two rules differ"
        assert not np.array_equal(ref["idx"], orc.forward(x64, wg64, wu64, wd64, K)["idx"])
    idx_np = idx.cpu().numpy()
    _check_picks(idx_np, ref["s"], K)
    # values on the device's own picks
    on_dev = orc.forward_given_idx(x64, wg64, wu64, wd64, idx_np.astype(np.int32))
    parity.assert_close(syn.to_f64(out), on_dev["out"], dtype, "out")
    parity.assert_close(syn.to_f64(tg), on_dev["gval"], dtype, "topk_gate")
    parity.assert_close(syn.to_f64(tu), on_dev["uval"], dtype, "topk_up")
    parity.assert_close(syn.to_f64(out_d), on_dev["out"][:16], dtype, "decode out")
    # most tokens take exactly the oracle's picks
    same = (idx_np == ref["idx"]).all(axis=1).mean()
    assert same >= 0.9, f"only {same:.2f} of the tokens agree with the oracle's picks"
    # the backward pass takes the mask as saved
    grads = B.moc_ffn_backward(xd, wgd, wud, wdd, idx, tg, tu, dDd, d_ff=F)
    torch.cuda.synchronize()
    gdev = {k: syn.to_f64(v) for k, v in grads.items()}
    parity.check_backward(gdev, x64, wg64, wu64, wd64, idx_np, syn.to_f64(tg), syn.to_f64(tu), dD64, F, dtype)


def test_post_silu_equals_default_rule_with_enough_positive_gates():
    w = syn.Workload("ps-same", "f32", 48, 64, 256, 256, 32, seed=5200)
    x, wg, wu, wd = _mostly_negative(w, 0.5)
    xd, wgd, wud, wdd = (t.cuda() for t in (x, wg, wu, wd))
    a = B.moc_ffn_forward(xd, wgd, wud, wdd, w.k, post_silu=True)
    b = B.moc_ffn_forward(xd, wgd, wud, wdd, w.k)
    torch.cuda.synchronize()
    assert torch.equal(a[1], b[1]) and torch.equal(a[0], b[0])


def test_post_silu_flag_rules():
    w = syn.Workload("ps-err", "bf16", 4, 64, 96, 96, 24, seed=5300)
    x, wg, wu, wd = (t.cuda() for t in (syn.make_x(w), *syn.make_weights(w)))
    with pytest.raises(B.MocError):   # not combinable with the 2-of-8 mask
        B.moc_ffn_forward(x, wg, wu, wd, None, grouped=True, post_silu=True)
    desc = B.make_desc(4, 64, 96, 24, x.dtype, flags=B.MOC_FLAG_SELECT_POST_SILU)
    assert B.moc_ffn_workspace_bytes(desc, B.MOC_OP_DECODE_BLOCK) == 0   # no block form for the ablation variant
