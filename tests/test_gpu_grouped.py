"""MoC 2:8 (the grouped mask of Section 4: the 2 largest of every 8 consecutive channels) through the C ABI, against
the oracle's grouped selection; everything after the mask is the operator the other GPU tests cover."""
import numpy as np
import pytest
import torch

from oracle import moc_oracle as orc
from oracle import parity
from paper_2511_09323_b200 import binding as B
from paper_2511_09323_b200 import build as moc_build
from paper_2511_09323_b200 import synthetic as syn
from paper_2511_09323_b200.autograd import MoCFFN

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    moc_build.build()
    B.load()
    yield
    assert B.moc_last_device_status() == B.MOC_OK


def _forward_backward(w: syn.Workload, grouped_backward: bool = True):
    wg, wu, wd = syn.make_weights(w)
    x, dD = syn.make_x(w), syn.make_grad_out(w)
    xd, wgd, wud, wdd, dDd = (t.cuda() for t in (x, wg, wu, wd, dD))
    out, idx, tg, tu = B.moc_ffn_forward(xd, wgd, wud, wdd, None, grouped=True)
    grads = B.moc_ffn_backward(xd, wgd, wud, wdd, idx, tg, tu, dDd, grouped=grouped_backward)
    torch.cuda.synchronize()
    assert B.moc_last_device_status() == B.MOC_OK
    x64, wg64, wu64, wd64, dD64 = map(syn.to_f64, (x, wg, wu, wd, dD))
    idx_np = idx.cpu().numpy()
    assert idx_np.shape == (w.tokens, w.d_ff // 4)
    parity.check_picks_grouped(idx_np, orc.gate_projection(x64, wg64))
    ref = orc.forward_given_idx(x64, wg64, wu64, wd64, idx_np.astype(np.int32))
    parity.assert_close(syn.to_f64(out), ref["out"], w.dtype, "out")
    parity.assert_close(syn.to_f64(tg), ref["gval"], w.dtype, "topk_gate")
    parity.assert_close(syn.to_f64(tu), ref["uval"], w.dtype, "topk_up")
    gdev = {k: syn.to_f64(v) for k, v in grads.items()}
    parity.check_backward(gdev, x64, wg64, wu64, wd64, idx_np, syn.to_f64(tg), syn.to_f64(tu), dD64, w.d_ff, w.dtype)
    return (xd, wgd, wud, wdd), out


@pytest.mark.parametrize("dtype,T,d,F", [
    ("bf16", 300, 128, 1024),    # tensor-core plan: the mask fused into the gate+up GEMM's epilogue
    ("bf16", 700, 264, 1000),    # the same with ragged tiles: 125 groups, the last channel tile 104 wide, K = 250
    ("bf16", 5, 64, 256),        # a handful of tokens: small-batch forward, tensor-core backward
    ("f32", 40, 64, 256),        # gathered plan
])
def test_grouped_forward_backward(dtype, T, d, F):
    _forward_backward(syn.Workload(f"g28-{dtype}-{T}", dtype, T, d, F, F, F // 4, seed=2800 + T))


@pytest.mark.parametrize("T,d,F,grouped_backward", [
    (300, 1024, 1024, True),     # d_model >= 1024: down projection and grad_x on the 2:4-sparse MMA; one ragged tile pair
    (300, 1024, 1024, False),    # the same saved tensors through the dense grad_x (no promise about the indices)
    (700, 1288, 1280, True),     # ragged in every direction: 700 tokens, 1288 columns (5 tiles + 8), 10 blocks of 128 channels
    (520, 1024, 1000, True),     # d_ff not a multiple of 128: compressed forward, dense grad_x
])
def test_grouped_forward_backward_on_the_sparse_mma(T, d, F, grouped_backward):
    _forward_backward(syn.Workload(f"g28sp-{T}-{d}-{F}", "bf16", T, d, F, F, F // 4, seed=2900 + T), grouped_backward)


def _run_isolated(code, env_extra):
    """Runs `code` in a fresh interpreter (the library reads its environment switches once per process); the code saves a
    dictionary of tensors to the path it gets as its argument."""
    import os
    import subprocess
    import sys
    import tempfile
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    with tempfile.NamedTemporaryFile(suffix=".pt") as fh:
        subprocess.run([sys.executable, "-c", code, fh.name], check=True, cwd=root, env=dict(os.environ, **env_extra),
                       timeout=600)
        return torch.load(fh.name)


_SPARSE_CASE = (
    "import torch, sys; sys.path.insert(0, '.');"
    "from paper_2511_09323_b200 import binding as B, synthetic as syn;"
    "w = syn.Workload('g28cmp', 'bf16', 600, 1024, 2048, 2048, 512, seed=77);"
    "wg, wu, wd = (t.cuda() for t in syn.make_weights(w)); x = syn.make_x(w).cuda(); dD = syn.make_grad_out(w).cuda();"
    "out, idx, tg, tu = B.moc_ffn_forward(x, wg, wu, wd, None, grouped=True);"
    "g = B.moc_ffn_backward(x, wg, wu, wd, idx, tg, tu, dD, grouped=True); torch.cuda.synchronize();"
    "st = B.moc_last_device_status();"
    "torch.save({'out': out.cpu(), 'idx': idx.cpu(), 'gx': g['grad_x'].cpu(), 'status': st}, sys.argv[1])")


def test_grouped_sparse_paths_agree_with_the_dense_ones():
    """The same layer with the sparse MMA switched off is a different set of kernels for the same arithmetic: down
    projection and grad_x (the latter on the sparse MMA only when asked for) must agree within the bf16 tolerance, and the
    sparse grad_x must match the oracle."""
    sparse = _run_isolated(_SPARSE_CASE, {"MOC_FFN_SPARSE": "1", "MOC_FFN_SPARSE_DX": "1"})
    dense = _run_isolated(_SPARSE_CASE, {"MOC_FFN_SPARSE": "0"})
    assert sparse["status"] == B.MOC_OK and dense["status"] == B.MOC_OK
    assert torch.equal(sparse["idx"], dense["idx"])
    for key in ("out", "gx"):
        a, b = sparse[key].double(), dense[key].double()
        assert (a - b).abs().max().item() <= 1e-2 * b.abs().max().item(), key
    w = syn.Workload("g28cmp", "bf16", 600, 1024, 2048, 2048, 512, seed=77)
    wg, wu, wd = syn.make_weights(w)
    x, dD = syn.make_x(w), syn.make_grad_out(w)
    toks = np.arange(0, 600, 7)
    x64, dD64 = syn.to_f64(x[toks]), syn.to_f64(dD[toks])
    wg64, wu64, wd64 = map(syn.to_f64, (wg, wu, wd))
    idx_np = sparse["idx"].numpy()[toks].astype(np.int32)
    ref = orc.forward_given_idx(x64, wg64, wu64, wd64, idx_np)
    parity.assert_close(syn.to_f64(sparse["out"][toks]), ref["out"], "bf16", "out (sparse down projection)")
    rb = orc.backward(x64, wg64, wu64, wd64, idx_np, syn.round_to(ref["gval"], "bf16"), syn.round_to(ref["uval"], "bf16"),
                      dD64, F=w.d_ff, want=("x",))
    parity.assert_close(syn.to_f64(sparse["gx"][toks]), rb["grad_x"], "bf16", "grad_x (sparse MMA)")


def test_backward_flag_on_rows_that_are_not_2_of_8_is_reported():
    """Saved indices from the row Top-K (several kept channels in one group of 4) with the 2-of-8 promise set and grad_x
    on the sparse MMA: the surplus channels are left out and the status word says so; nothing faults."""
    code = (
        "import torch, sys; sys.path.insert(0, '.');"
        "from paper_2511_09323_b200 import binding as B, synthetic as syn;"
        "w = syn.Workload('g28-bad', 'bf16', 300, 1024, 1024, 1024, 256, seed=41);"
        "wg, wu, wd = (t.cuda() for t in syn.make_weights(w)); x = syn.make_x(w).cuda(); dD = syn.make_grad_out(w).cuda();"
        "out, idx, tg, tu = B.moc_ffn_forward(x, wg, wu, wd, w.k);"
        "B.moc_ffn_backward(x, wg, wu, wd, idx, tg, tu, dD, grouped=True);"
        "st1 = B.moc_last_device_status(); st2 = B.moc_last_device_status();"
        "ok = B.moc_ffn_backward(x, wg, wu, wd, idx, tg, tu, dD); torch.cuda.synchronize();"
        "torch.save({'st1': st1, 'st2': st2, 'st3': B.moc_last_device_status(),"
        " 'finite': bool(torch.isfinite(ok['grad_x'].float()).all())}, sys.argv[1])")
    res = _run_isolated(code, {"MOC_FFN_SPARSE_DX": "1"})
    assert res["st1"] == B.MOC_ERR_BAD_INDEX and res["st2"] == B.MOC_OK
    assert res["st3"] == B.MOC_OK and res["finite"]


def test_grouped_ties_keep_the_lower_channels_exactly():
    """Channels 8q+1, 8q+3 copy the gate rows of 8q, 8q+2: bit-identical gate values; the kept pair of a group is
    then decided by the tie rule and must equal the oracle's choice on the device's own fp32 gate values."""
    w = syn.Workload("g28-ties", "bf16", 300, 64, 512, 512, 128, seed=31)
    wg, wu, wd = syn.make_weights(w)
    wg[1::8], wg[3::8] = wg[0::8].clone(), wg[2::8].clone()
    x = syn.make_x(w)
    _, idx, tg, _ = B.moc_ffn_forward(x.cuda(), wg.cuda(), wu.cuda(), wd.cuda(), None, grouped=True)
    idx = idx.cpu().numpy().astype(np.int64)
    for t in range(w.tokens):
        sel = set(idx[t].tolist())
        for j in idx[t]:
            if j % 8 in (1, 3):
                assert j - 1 in sel, f"token {t}: channel {j} kept without its equal lower twin"


@pytest.mark.parametrize("T", [1, 2, 3, 16])   # 1, 2: decode plan; 3, 16: small-batch plan (half the channels in use)
def test_grouped_decode_matches_forward_and_oracle(T):
    w = syn.Workload(f"g28-dec-{T}", "bf16", T, 512, 2048, 2048, 512, seed=77 + T)
    wg, wu, wd = syn.make_weights(w)
    x = syn.make_x(w)
    xd, wgd, wud, wdd = (t.cuda() for t in (x, wg, wu, wd))
    out = B.moc_ffn_decode(xd, wgd, wud, wdd, None, grouped=True)
    out_s = torch.empty_like(xd)
    B.moc_ffn_decode_static(xd, wgd, wud, wdd, None, out_s, grouped=True)
    out_f, idx, _, _ = B.moc_ffn_forward(xd, wgd, wud, wdd, None, grouped=True)
    torch.cuda.synchronize()
    x64, wg64, wu64, wd64 = map(syn.to_f64, (x, wg, wu, wd))
    idx_np = idx.cpu().numpy()
    parity.check_picks_grouped(idx_np, orc.gate_projection(x64, wg64))
    ref = orc.forward_given_idx(x64, wg64, wu64, wd64, idx_np.astype(np.int32))["out"]
    for name, o in (("decode", out), ("decode_static", out_s), ("forward", out_f)):
        parity.assert_close(syn.to_f64(o), ref, "bf16", name)


def test_grouped_argument_rules_and_module():
    x = torch.zeros(4, 64, dtype=torch.bfloat16, device="cuda")
    wbad = torch.zeros(100, 64, dtype=torch.bfloat16, device="cuda")     # d_ff not a multiple of 8
    with pytest.raises(ValueError):
        B.moc_ffn_forward(x, wbad, wbad, wbad, None, grouped=True)
    w = torch.zeros(128, 64, dtype=torch.bfloat16, device="cuda")
    desc = B.make_desc(4, 64, 128, 16, torch.bfloat16, flags=B.MOC_FLAG_SELECT_2_OF_8)   # k must be d_ff / 4 = 32
    assert B.moc_ffn_workspace_bytes(desc, B.MOC_OP_FORWARD) == 0
    m = MoCFFN(64, 128, None, grouped=True)
    assert m.k == 32
    y = m(torch.randn(2, 7, 64, device="cuda", dtype=torch.bfloat16))
    y.float().sum().backward()
    assert m.w_down.grad is not None and torch.isfinite(m.w_down.grad.float()).all()


def test_grouped_forward_without_cta_pairs():
    """MOC_FFN_GEMM=single (read once per process): without CTA pairs the 2-of-8 mask is not fused into the gate+up
    GEMM's epilogue; the GEMM writes G and U and a kernel with one thread per group applies the mask.  Run the
    tensor-core cases again in a child process with it set."""
    import os
    import subprocess
    import sys
    env = dict(os.environ, MOC_FFN_GEMM="single")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(root, "tests", "test_gpu_grouped.py"), "-q", "-x",
                        "-m", "gpu", "-k", "grouped_forward_backward or ties_keep"],
                       cwd=root, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]


def test_grouped_full_size_bench_layer_sampled_against_oracle():
    """The 2-of-8 mask on C2's layer at its full 16384 tokens (the configuration bench.py's `moc_2of8` line times): picks of
    sampled tokens per group, their out / saved values / grad_x and sampled rows of the weight gradients against the
    oracle; the slot layout of every token."""
    import dataclasses
    w = dataclasses.replace(syn.C2, k=syn.C2.d_ff // 4, name="C2-2of8")
    wg, wu, wd = syn.make_weights(w)
    x, dD = syn.make_x(w), syn.make_grad_out(w)
    xd, wgd, wud, wdd, dDd = (t.cuda() for t in (x, wg, wu, wd, dD))
    out, idx, tg, tu = B.moc_ffn_forward(xd, wgd, wud, wdd, None, grouped=True)
    grads = B.moc_ffn_backward(xd, wgd, wud, wdd, idx, tg, tu, dDd)
    torch.cuda.synchronize()
    assert B.moc_last_device_status() == B.MOC_OK
    idx_np = idx.cpu().numpy().astype(np.int64)
    slots = np.arange(w.k)
    assert np.all(idx_np // 8 == slots // 2), "slot 2q, 2q+1 must hold channels of group q"
    assert np.all(idx_np[:, 0::2] < idx_np[:, 1::2])
    rng = np.random.default_rng(0)
    toks = np.sort(rng.choice(w.tokens, 96, replace=False))
    wg64, wu64, wd64 = map(syn.to_f64, (wg, wu, wd))
    x64s, dD64s = syn.to_f64(x[toks]), syn.to_f64(dD[toks])
    parity.check_picks_grouped(idx_np[toks], orc.gate_projection(x64s, wg64))
    ref = orc.forward_given_idx(x64s, wg64, wu64, wd64, idx_np[toks].astype(np.int32))
    parity.assert_close(syn.to_f64(out[toks]), ref["out"], "bf16", "out")
    parity.assert_close(syn.to_f64(tg[toks]), ref["gval"], "bf16", "topk_gate")
    parity.assert_close(syn.to_f64(tu[toks]), ref["uval"], "bf16", "topk_up")
    rb = orc.backward(x64s, wg64, wu64, wd64, idx_np[toks].astype(np.int32), syn.to_f64(tg[toks]), syn.to_f64(tu[toks]),
                      dD64s, F=w.d_ff, want=("x",))
    parity.assert_close(syn.to_f64(grads["grad_x"][toks]), rb["grad_x"], "bf16", "grad_x (sampled tokens)")
    rows = np.sort(rng.choice(w.d_ff, 16, replace=False)).astype(np.int32)
    wrows = orc.backward_weight_rows(syn.to_f64(x), wd64, idx_np.astype(np.int32), syn.to_f64(tg), syn.to_f64(tu),
                                     syn.to_f64(dD), rows, w.d_ff)
    for name in ("grad_w_gate", "grad_w_up", "grad_w_down"):
        got = syn.to_f64(grads[name][torch.from_numpy(rows.astype(np.int64)).cuda()])
        parity.assert_close(got, wrows[name], "bf16", name + " (sampled rows)")
