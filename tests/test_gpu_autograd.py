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
