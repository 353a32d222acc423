"""Seeded random shapes through every entry point: forward + backward, decode and the block form against the oracle.
The fixed cases of the other files pin known corners; this sweep walks the plan boundaries (1 ... 300 tokens, ragged
widths, padded weight rows, K from 1 to d_ff) with shapes nobody chose by hand."""
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


def _random_workloads(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        dtype = "bf16" if rng.random() < 0.75 else "f32"
        T = int(rng.choice([1, 2, 3, 5, 6, 16, 17, 31, 64, 100, 129, 256, 257, 300]))
        d = 8 * int(rng.integers(1, 66))
        F = int(rng.integers(8, 1500 if dtype == "f32" else 3000))
        F_ld = F + 8 * int(rng.integers(0, 3)) if rng.random() < 0.4 else F
        F_ld = (F_ld + 7) // 8 * 8 if F_ld > F else F_ld
        K = int(rng.integers(1, F + 1)) if rng.random() < 0.3 else max(1, int(F * rng.uniform(0.03, 0.3)))
        out.append(syn.Workload(f"fuzz-{seed}-{i}", dtype, T, d, F, F_ld, K, seed=7000 + 31 * seed + i))
    return out


def _band_check(out64, full, x64, wg64, wu64, wd64, K, F, dtype, what, base=None):
    """Rows of `out64` against the oracle's; a token whose K-th and (K+1)-th gate values nearly tie may have taken the
    swapped pick.  `base`: what is added to the layer's output (the residual stream of the block form)."""
    ref = full["out"] if base is None else base + full["out"]
    tol = parity.REL_TOL[dtype] * max(np.abs(ref).max(), 1e-30)
    for t in range(out64.shape[0]):
        err = np.abs(out64[t] - ref[t]).max()
        if err <= tol:
            continue
        g = full["g"][t]
        order = np.lexsort((np.arange(F), -g))
        assert K < F and g[order[K - 1]] - g[order[K]] <= 1e-3, f"{what}: token {t} error {err:.3e} > {tol:.3e}"
        alt = np.sort(np.concatenate([order[: K - 1], order[K: K + 1]])).astype(np.int32)[None]
        alt_out = orc.forward_given_idx(x64[t: t + 1], wg64, wu64, wd64, alt)["out"][0]
        if base is not None:
            alt_out = base[t] + alt_out
        assert np.abs(out64[t] - alt_out).max() <= tol, f"{what}: token {t} matches neither pick"


@pytest.mark.parametrize("w", _random_workloads(28, 1), ids=lambda w: f"{w.dtype}-T{w.tokens}-d{w.d_model}-F{w.d_ff}of{w.d_ff_ld}-K{w.k}")
def test_random_shape_forward_backward_decode(w):
    wg, wu, wd = syn.make_weights(w)
    x, dD = syn.make_x(w), syn.make_grad_out(w)
    xd, wgd, wud, wdd, dDd = (t.cuda() for t in (x, wg, wu, wd, dD))
    F, K = w.d_ff, w.k
    out, idx, tg, tu = B.moc_ffn_forward(xd, wgd, wud, wdd, K, d_ff=F)
    grads = B.moc_ffn_backward(xd, wgd, wud, wdd, idx, tg, tu, dDd, d_ff=F)
    torch.cuda.synchronize()
    x64, wg64, wu64, wd64, dD64 = map(syn.to_f64, (x, wg[:F], wu[:F], wd[:F], dD))
    dev = dict(out=syn.to_f64(out), idx=idx.cpu().numpy(), gval=syn.to_f64(tg), uval=syn.to_f64(tu))
    parity.check_forward(dev, x64, wg64, wu64, wd64, K, F, w.dtype)
    gdev = {k: syn.to_f64(v) for k, v in grads.items()}
    parity.check_backward(gdev, x64, wg64, wu64, wd64, dev["idx"], dev["gval"], dev["uval"], dD64, F, w.dtype)
    if w.d_ff_ld > F:
        for name in ("grad_w_gate", "grad_w_up", "grad_w_down"):
            assert torch.all(grads[name][F:] == 0), name
    if w.tokens <= 256:
        full = orc.forward(x64, wg64, wu64, wd64, K, want_g=True)
        out_d = B.moc_ffn_decode(xd, wgd, wud, wdd, K, d_ff=F)
        torch.cuda.synchronize()
        _band_check(syn.to_f64(out_d), full, x64, wg64, wu64, wd64, K, F, w.dtype, "decode")
        desc = B.make_desc(w.tokens, w.d_model, F, K, xd.dtype, d_ff_ld=w.d_ff_ld)
        if B.moc_ffn_workspace_bytes(desc, B.MOC_OP_DECODE_BLOCK) > 0:
            gen = torch.Generator().manual_seed(w.seed + 5)
            h = (torch.randn(w.tokens, w.d_model, generator=gen) * 2.0).to(torch.bfloat16)
            gamma = (0.5 + torch.rand(w.d_model, generator=gen)).to(torch.bfloat16)
            out_b = B.moc_ffn_decode_block(h.cuda(), gamma.cuda(), 1e-5, wgd, wud, wdd, K, d_ff=F)
            torch.cuda.synchronize()
            h64 = syn.to_f64(h)
            store = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(torch.bfloat16).double().numpy()
            _, xn, fb = orc.decode_block(h64, syn.to_f64(gamma), 1e-5, wg64, wu64, wd64, K, store=store)
            _band_check(syn.to_f64(out_b), fb, xn, wg64, wu64, wd64, K, F, "bf16", "block", base=h64)


def test_random_rows_through_the_selector_hook_are_bit_exact():
    """`moc_topk_select` on 48 seeded random problems (row counts either side of the 256-row switch between the two
    selectors, widths up to the int16 limit, duplicates, all-equal rows, tiny values, NaN / +-inf / -0): the indices
    must equal the oracle's on the same fp32 array."""
    rng = np.random.default_rng(11)
    for i in range(48):
        rows = int(rng.choice([1, 3, 17, 200, 256, 257, 700]))
        n = int(rng.integers(1, 12000)) if rng.random() < 0.8 else int(rng.integers(12000, 32768))
        n_ld = n + int(rng.integers(0, 9))
        k = int(rng.integers(1, n + 1)) if rng.random() < 0.3 else max(1, int(n * rng.uniform(0.01, 0.3)))
        mode = int(rng.integers(0, 6))
        g = rng.standard_normal((rows, n_ld)).astype(np.float32)
        if mode == 1:
            g = np.round(g * 4) / 4            # heavy duplicates
        elif mode == 2:
            g = np.round(g * 64) / 64
        elif mode == 3:
            g[:] = g[:, :1]                    # every row a constant
        elif mode == 4:
            g = np.abs(g) * 1e-30              # tiny values
        elif mode == 5:
            g[rng.random(g.shape) < 0.01] = np.nan
            g[rng.random(g.shape) < 0.01] = -np.inf
            g[rng.random(g.shape) < 0.005] = np.inf
            g[rng.random(g.shape) < 0.02] = -0.0
        g = np.ascontiguousarray(g.astype(np.float32))
        ref = orc.topk(g, k, F=n)
        got = B.moc_topk_select(torch.from_numpy(g).cuda(), k, n=n).cpu().numpy().astype(np.int32)
        assert np.array_equal(ref, got), f"problem {i}: rows={rows} n={n} n_ld={n_ld} k={k} mode={mode}"


@pytest.mark.parametrize("dtype,T,d,F,F_ld,K", [
    ("bf16", 1, 8192, 512, 512, 64),        # d_model beyond the cooperative kernel's 4096 columns: four-kernel plan
    ("bf16", 2, 8192, 520, 520, 65),
    ("bf16", 4, 8192, 512, 512, 64),
    ("bf16", 20, 8192, 512, 512, 64),       # small-batch plan, 128 contraction blocks
    ("bf16", 300, 8192, 512, 512, 64),      # tensor-core plan
    ("bf16", 1, 16384, 256, 256, 32),
    ("bf16", 5, 12288, 256, 256, 32),
    ("bf16", 40, 16384, 264, 264, 33),
    ("f32", 3, 8192, 256, 256, 32),
    ("bf16", 1, 8, 8, 8, 1),                # the smallest of everything
    ("bf16", 1, 8, 16, 16, 16),             # K = d_ff on the decode path
    ("bf16", 256, 8, 8, 8, 8),
    ("bf16", 3, 4104, 300, 304, 7),         # one 8-column step past 4096, padded weight rows
    ("bf16", 2, 4096, 32768, 32768, 4096),  # the int16 limit of d_ff on the cooperative kernel
    ("bf16", 1, 64, 32768, 32768, 1),
    ("bf16", 16, 64, 32760, 32768, 4000),
    ("bf16", 200, 64, 30000, 30000, 3000),
])
def test_extreme_shapes(dtype, T, d, F, F_ld, K):
    test_random_shape_forward_backward_decode(
        syn.Workload(f"extreme-{T}-{d}-{F}", dtype, T, d, F, F_ld, K, seed=9500 + T + d + F))


@pytest.mark.parametrize("T,d,F,K", [(1, 520, 776, 97), (2, 520, 776, 97), (4, 264, 333, 41), (16, 768, 2048, 256),
                                     (40, 768, 2048, 256), (300, 768, 2048, 256)])
def test_results_do_not_depend_on_what_the_workspace_held(T, d, F, K):
    """Every operation with a workspace of zeros, of 0xff bytes and of random bytes: the same results (up to the
    order in which partial sums meet); decode twice in a row on the same workspace as well."""
    w = syn.Workload("ws", "bf16", T, d, F, (F + 7) // 8 * 8, K, seed=321 + T)
    wg, wu, wd = (t.cuda() for t in syn.make_weights(w))
    x, dD = syn.make_x(w).cuda(), syn.make_grad_out(w).cuda()
    desc = B.make_desc(T, d, F, K, x.dtype, d_ff_ld=w.d_ff_ld)
    saved = B.moc_ffn_forward(x, wg, wu, wd, K, d_ff=F)
    gamma = torch.ones(d, dtype=x.dtype, device="cuda")

    def run(op, ws):
        if op == B.MOC_OP_FORWARD:
            o = B.moc_ffn_forward(x, wg, wu, wd, K, d_ff=F, workspace=ws)
            return [o[0].clone(), o[1].float(), o[2].clone(), o[3].clone()]
        if op == B.MOC_OP_BACKWARD:
            g = B.moc_ffn_backward(x, wg, wu, wd, saved[1], saved[2], saved[3], dD, d_ff=F, workspace=ws)
            return [g[k].clone() for k in sorted(g)]
        if op == B.MOC_OP_DECODE:
            return [B.moc_ffn_decode(x, wg, wu, wd, K, d_ff=F, workspace=ws).clone(),
                    B.moc_ffn_decode(x, wg, wu, wd, K, d_ff=F, workspace=ws).clone()]
        return [B.moc_ffn_decode_block(x, gamma, 1e-5, wg, wu, wd, K, d_ff=F, workspace=ws).clone()]

    gen = torch.Generator(device="cuda").manual_seed(5)
    for op in (B.MOC_OP_FORWARD, B.MOC_OP_BACKWARD, B.MOC_OP_DECODE, B.MOC_OP_DECODE_BLOCK):
        n = B.moc_ffn_workspace_bytes(desc, op)
        if n == 0:
            continue
        results = []
        for fill in ("zero", "ff", "random"):
            ws = torch.empty(n, dtype=torch.uint8, device="cuda")
            if fill == "zero":
                ws.zero_()
            elif fill == "ff":
                ws.fill_(0xff)
            else:
                ws.copy_(torch.randint(0, 256, (n,), dtype=torch.uint8, device="cuda", generator=gen))
            results.append(run(op, ws))
        torch.cuda.synchronize()
        for other in results[1:]:
            for a, b in zip(other, results[0]):
                torch.testing.assert_close(a.float(), b.float(), rtol=2e-2, atol=2e-3 * max(1.0, b.float().abs().max().item()))
    assert B.moc_last_device_status() == B.MOC_OK
