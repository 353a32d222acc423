"""The torch.autograd front end: same kernels as the C-ABI calls, gradients checked against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import parity
from paper_2511_09323_b200 import binding as B
from paper_2511_09323_b200 import build as moc_build
from paper_2511_09323_b200 import synthetic as syn
from paper_2511_09323_b200.autograd import MoCFFN, moc_ffn

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    moc_build.build()
    B.load()
    yield
    assert B.moc_last_device_status() == B.MOC_OK


@pytest.mark.parametrize("dtype,batch,seq,d,F,K", [
    ("bf16", 5, 64, 256, 1024, 128),   # 320 tokens: tensor-core plan
    ("f32", 2, 24, 64, 160, 20),       # gathered plan
])
def test_function_matches_direct_calls_and_oracle(dtype, batch, seq, d, F, K):
    w = syn.Workload(f"autograd-{dtype}", dtype, batch * seq, d, F, F, K, seed=901)
    wg, wu, wd = syn.make_weights(w)
    x, dD = syn.make_x(w), syn.make_grad_out(w)
    leaves = [t.cuda().requires_grad_(True) for t in (x.reshape(batch, seq, d), wg, wu, wd)]
    out = moc_ffn(*leaves, K)
    assert out.shape == (batch, seq, d)
    (out * dD.cuda().reshape(batch, seq, d)).sum().backward()
    torch.cuda.synchronize()
    # the same numbers as the two C-ABI calls made by hand (both paths are deterministic here)
    xd, wgd, wud, wdd = (t.detach().reshape(-1, t.shape[-1]) if i == 0 else t.detach() for i, t in enumerate(leaves))
    o2, idx, tg, tu = B.moc_ffn_forward(xd, wgd, wud, wdd, K)
    g2 = B.moc_ffn_backward(xd, wgd, wud, wdd, idx, tg, tu, dD.cuda())
    assert torch.equal(out.detach().reshape(-1, d), o2)
    assert torch.equal(leaves[0].grad.reshape(-1, d), g2["grad_x"])
    for leaf, name in zip(leaves[1:], ("grad_w_gate", "grad_w_up", "grad_w_down")):
        assert torch.equal(leaf.grad, g2[name]), name
    # and against the oracle, given the saved tensors the device used
    x64, wg64, wu64, wd64, dD64 = map(syn.to_f64, (x, wg, wu, wd, dD))
    dev = dict(out=syn.to_f64(o2), idx=idx.cpu().numpy(), gval=syn.to_f64(tg), uval=syn.to_f64(tu))
    parity.check_forward(dev, x64, wg64, wu64, wd64, K, F, dtype)
    gdev = dict(grad_x=syn.to_f64(leaves[0].grad.reshape(-1, d)), grad_w_gate=syn.to_f64(leaves[1].grad),
                grad_w_up=syn.to_f64(leaves[2].grad), grad_w_down=syn.to_f64(leaves[3].grad))
    parity.check_backward(gdev, x64, wg64, wu64, wd64, dev["idx"], dev["gval"], dev["uval"], dD64, F, dtype)


def test_module_trains_a_step_and_skips_unneeded_gradients():
    torch.manual_seed(3)
    m = MoCFFN(128, 512, 64, dtype=torch.bfloat16)
    assert m.saved_bytes_per_token() == 64 * 6
    x = torch.randn(4, 80, 128, device="cuda", dtype=torch.bfloat16)
    # inference: nothing requires grad -> nothing is saved
    with torch.no_grad():
        y0 = m(x)
    # frozen gate: its gradient is not computed, the others are
    m.w_gate.requires_grad_(False)
    y = m(x)
    assert torch.equal(y, y0)
    y.float().pow(2).mean().backward()
    assert m.w_gate.grad is None and m.w_up.grad is not None and m.w_down.grad is not None
    assert np.isfinite(m.w_up.grad.float().abs().sum().item()) and m.w_up.grad.float().abs().sum().item() > 0
    # rows of channels no token selected get exactly zero gradient (Eqs. (bp-1), (bp-4))
    _, idx, _, _ = B.moc_ffn_forward(x.reshape(-1, 128), m.w_gate.detach(), m.w_up.detach(), m.w_down.detach(), 64)
    unused = torch.ones(512, dtype=torch.bool, device="cuda")
    unused[idx.long().unique()] = False
    assert torch.all(m.w_down.grad[unused] == 0) and torch.all(m.w_up.grad[unused] == 0)


@pytest.mark.parametrize("dtype,T,d,F,F_ld,K", [
    ("bf16", 320, 256, 1000, 1024, 125),   # tensor-core plan: dense U with the forward's GEMM, then a gather
    ("bf16", 40, 128, 520, 520, 65),       # a small batch: forward on the small-batch plan, up values again on the tensor cores
    ("bf16", 5, 64, 32768, 32768, 11008),  # rows too long for the tensor-core selector: gathered plan
    ("f32", 33, 64, 160, 160, 20),         # fp32: gathered plan
])
def test_recompute_up_reproduces_the_saved_up_values(dtype, T, d, F, F_ld, K):
    """topk_up formed again from x, w_up and the saved indices: against the oracle's u on the same indices, against what
    the forward pass saved (the same contraction on the same inputs: at most one rounding step apart), and as the
    input of a backward pass whose gradients are checked with the recomputed values as the saved ones."""
    w = syn.Workload(f"reup-{dtype}-{T}", dtype, T, d, F, F_ld, K, seed=4300 + T)
    wg, wu, wd = syn.make_weights(w)
    x, dD = syn.make_x(w), syn.make_grad_out(w)
    xd, wgd, wud, wdd, dDd = (t.cuda() for t in (x, wg, wu, wd, dD))
    out, idx, tg, tu = B.moc_ffn_forward(xd, wgd, wud, wdd, K, d_ff=F)
    tu2 = B.moc_ffn_recompute_up(xd, wud, idx, d_ff=F)
    torch.cuda.synchronize()
    x64, wg64, wu64, wd64, dD64 = map(syn.to_f64, (x, wg[:F], wu[:F], wd[:F], dD))
    idx_np = idx.cpu().numpy()
    u_ref = np.einsum("td,tkd->tk", x64, wu64[idx_np.astype(np.int64)])
    parity.assert_close(syn.to_f64(tu2), u_ref, dtype, "recomputed topk_up")
    ulp = 2.0 ** -7 if dtype == "bf16" else 2.0 ** -20
    a, b = syn.to_f64(tu2), syn.to_f64(tu)
    assert np.all(np.abs(a - b) <= ulp * np.maximum(np.abs(b), 1e-3)), "recomputed and saved up values differ by more than a rounding step"
    grads = B.moc_ffn_backward(xd, wgd, wud, wdd, idx, tg, tu2, dDd, d_ff=F)
    gdev = {k: syn.to_f64(v) for k, v in grads.items()}
    parity.check_backward(gdev, x64, wg64, wu64, wd64, idx_np, syn.to_f64(tg), syn.to_f64(tu2), dD64, F, dtype)


def test_recompute_up_option_of_the_module_and_bad_indices():
    torch.manual_seed(5)
    m = MoCFFN(128, 512, 64, dtype=torch.bfloat16, recompute_up=True)
    ref = MoCFFN(128, 512, 64, dtype=torch.bfloat16)
    ref.load_state_dict(m.state_dict())
    assert m.saved_bytes_per_token() == 64 * 4 and ref.saved_bytes_per_token() == 64 * 6
    x = torch.randn(3, 100, 128, device="cuda", dtype=torch.bfloat16)
    xa, xb = x.clone().requires_grad_(True), x.clone().requires_grad_(True)
    ya, yb = m(xa), ref(xb)
    assert torch.equal(ya, yb)
    ya.float().pow(2).mean().backward()
    yb.float().pow(2).mean().backward()
    torch.testing.assert_close(xa.grad.float(), xb.grad.float(), rtol=2e-2, atol=1e-5)
    for pa, pb in zip(m.parameters(), ref.parameters()):
        torch.testing.assert_close(pa.grad.float(), pb.grad.float(), rtol=2e-2, atol=1e-5)
    # an index outside [0, d_ff) yields 0 and raises the device status; the others are unaffected
    w = syn.Workload("reup-bad", "bf16", 300, 64, 96, 96, 8, seed=12)
    wg, wu, wd = (t.cuda() for t in syn.make_weights(w))
    xd = syn.make_x(w).cuda()
    _, idx, _, tu = B.moc_ffn_forward(xd, wg, wu, wd, w.k)
    good = B.moc_ffn_recompute_up(xd, wu, idx)
    bad = idx.clone()
    bad[3, 2] = 96
    bad[7, 0] = -5
    assert B.moc_last_device_status() == B.MOC_OK
    got = B.moc_ffn_recompute_up(xd, wu, bad)
    assert B.moc_last_device_status() == B.MOC_ERR_BAD_INDEX
    assert got[3, 2] == 0 and got[7, 0] == 0
    mask = torch.ones_like(got, dtype=torch.bool)
    mask[3, 2] = mask[7, 0] = False
    assert torch.equal(got[mask], good[mask])


def test_module_post_silu_option_matches_direct_calls():
    """post_silu=True reaches the library (MOC_FLAG_SELECT_POST_SILU) through the module, forward and backward."""
    torch.manual_seed(7)
    m = MoCFFN(64, 256, 32, dtype=torch.float32, post_silu=True)
    with torch.no_grad():
        m.w_gate -= 0.05   # with x > 0 below most gate values are negative: the two rules differ
    x = (torch.rand(24, 64, device="cuda") + 0.5).requires_grad_(True)
    y = m(x)
    y.sum().backward()
    out, idx, tg, tu = B.moc_ffn_forward(x.detach(), m.w_gate.detach(), m.w_up.detach(), m.w_down.detach(), 32, post_silu=True)
    default = B.moc_ffn_forward(x.detach(), m.w_gate.detach(), m.w_up.detach(), m.w_down.detach(), 32)
    assert torch.equal(y.detach(), out)
    assert not torch.equal(idx, default[1])
    g = B.moc_ffn_backward(x.detach(), m.w_gate.detach(), m.w_up.detach(), m.w_down.detach(), idx, tg, tu, torch.ones_like(out))
    assert torch.equal(x.grad, g["grad_x"]) and torch.equal(m.w_down.grad, g["grad_w_down"])
