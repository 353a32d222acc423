"""Parity of the CUDA library (called through its C ABI) with the CPU oracle on the same seeded inputs."""
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


def _dev(t):
    return t.to("cuda")


def _problem(w: syn.Workload):
    wg, wu, wd = syn.make_weights(w)
    x = syn.make_x(w)
    dD = syn.make_grad_out(w)
    return x, wg, wu, wd, dD


def _run_forward_backward(w: syn.Workload, decode=False):
    x, wg, wu, wd, dD = _problem(w)
    xd, wgd, wud, wdd, dDd = map(_dev, (x, wg, wu, wd, dD))
    out, idx, tg, tu = B.moc_ffn_forward(xd, wgd, wud, wdd, w.k, d_ff=w.d_ff)
    torch.cuda.synchronize()
    x64, wg64, wu64, wd64, dD64 = map(syn.to_f64, (x, wg, wu, wd, dD))
    dev = dict(out=syn.to_f64(out), idx=idx.cpu().numpy(), gval=syn.to_f64(tg), uval=syn.to_f64(tu))
    rep = parity.check_forward(dev, x64, wg64, wu64, wd64, w.k, w.d_ff, w.dtype)
    grads = B.moc_ffn_backward(xd, wgd, wud, wdd, idx, tg, tu, dDd, d_ff=w.d_ff)
    torch.cuda.synchronize()
    gdev = {k: syn.to_f64(v) for k, v in grads.items()}
    rep.update(parity.check_backward(gdev, x64, wg64, wu64, wd64, dev["idx"], dev["gval"], dev["uval"], dD64,
                                     w.d_ff, w.dtype))
    return rep, (xd, wgd, wud, wdd, dDd), (out, idx, tg, tu), grads


# ------------------------------------------------------------------ selector alone: bit exact


def _adversarial_rows(n):
    r = np.arange(n, dtype=np.float32)
    rows = [
        np.zeros(n, np.float32),
        r.copy(),
        -r,
        np.where(r % 3 == 0, 1.0, -1.0).astype(np.float32),
        np.where(r % 2 == 0, 0.0, -0.0).astype(np.float32),
        np.concatenate([[np.inf, -np.inf], np.linspace(-1, 1, n - 2)]).astype(np.float32),
        np.full(n, -np.inf, np.float32),
        np.where(r % 5 == 0, np.nan, np.sin(r)).astype(np.float32),
        (np.round(np.random.default_rng(1).standard_normal(n) * 16) / 16).astype(np.float32),  # many duplicates
        np.random.default_rng(2).standard_normal(n).astype(np.float32) * 1e-30,               # tiny magnitudes
        np.float32(1e30) * np.random.default_rng(3).standard_normal(n).astype(np.float32),
        (np.float32(2.0) ** (-(r % 140))).astype(np.float32),                                  # thinning out over 140 octaves
        (np.float32(1.0) + (r % 97) * np.float32(1.2e-7)).astype(np.float32),                  # a few ulps apart
        np.where(r == 0, 1e30, np.where(r == 1, -1e30,                                          # two outliers stretch
                 np.random.default_rng(4).standard_normal(n) * 1e-3)).astype(np.float32),      # the range of a cluster
        (np.random.default_rng(5).standard_normal(n) * 1e-42).astype(np.float32),              # denormals
    ]
    return np.stack(rows)


@pytest.mark.parametrize("repeat", [1, 20])   # 15 rows: a CTA per row; 300 rows: the gathered plan's selector
@pytest.mark.parametrize("n,n_ld", [(1, 4), (37, 40), (37, 37), (256, 256), (257, 264), (2048, 2048), (5461, 5504),
                                    (11008, 11008), (32768, 32768)])
def test_selector_bit_exact_adversarial(n, n_ld, repeat):
    rows = _adversarial_rows(max(n, 3))[:, :n] if n >= 3 else np.zeros((3, n), np.float32)
    rows = np.tile(rows, (repeat, 1))
    g = np.full((rows.shape[0], n_ld), 1e9, np.float32)  # padding columns hold large values: must be ignored
    g[:, :n] = rows
    gd = torch.from_numpy(g).cuda()
    for k in sorted({1, 2, max(1, n // 8), max(1, n - 1), n}):
        if k > n:
            continue
        got = B.moc_topk_select(gd, k, n=n).cpu().numpy().astype(np.int32)
        np.testing.assert_array_equal(got, orc.topk(g, k, F=n), err_msg=f"n={n} k={k}")


@pytest.mark.parametrize("name", ["C1", "C2", "C3", "C4"])
def test_selector_bit_exact_on_oracle_gate_values(name):
    """The selector is fed float32(oracle gate values) of the configuration's shape."""
    w = syn.WORKLOADS[name]
    T = 48 if w.d_ff > 4000 else 96
    wg, _, _ = syn.make_weights(w)
    x = syn.make_x(w, tokens=T)
    g64 = syn.to_f64(x) @ syn.to_f64(wg)[: w.d_ff].T
    g32 = np.zeros((T, w.d_ff_ld), np.float32)
    g32[:, : w.d_ff] = g64.astype(np.float32)
    got = B.moc_topk_select(torch.from_numpy(g32).cuda(), w.k, n=w.d_ff).cpu().numpy().astype(np.int32)
    np.testing.assert_array_equal(got, orc.topk(g32, w.k, F=w.d_ff))


def test_selector_many_rows_grid_stride():
    rng = np.random.default_rng(7)
    g = rng.standard_normal((6000, 96)).astype(np.float32)  # more rows than the selector's grid
    got = B.moc_topk_select(torch.from_numpy(g).cuda(), 12).cpu().numpy().astype(np.int32)
    np.testing.assert_array_equal(got, orc.topk(g, 12))


# ------------------------------------------------------------------ forward + backward


def test_c1_tiny_fp32_forward_backward():
    rep, *_ = _run_forward_backward(syn.C1)
    assert rep["out"][0] <= 1e-4 * rep["out"][1]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("T,d,F,F_ld,K", [
    (1, 8, 8, 8, 1),            # smallest legal shape
    (3, 16, 40, 40, 39),        # K = F - 1
    (5, 24, 33, 40, 33),        # K = F (dense SwiGLU) with a padded tail
    (70, 264, 333, 336, 41),    # nothing a multiple of a tile
    (300, 768, 520, 520, 65),   # several tiles + ragged tails
])
def test_ragged_shapes(dtype, T, d, F, F_ld, K):
    w = syn.Workload(f"rag-{T}-{d}-{F}-{K}", dtype, T, d, F, F_ld, K, seed=100 + T)
    _run_forward_backward(w)


def test_llama130m_shape_bf16_slice():
    """C2's layer shape on a token slice the oracle finishes in seconds."""
    w = syn.C2.with_tokens(640)
    rep, *_ = _run_forward_backward(w)
    assert rep["tokens_with_band_picks"] <= 64


def test_llama1b_shape_bf16_padded_slice():
    """C3's layer shape: d_ff = 5461 in arrays of 5504 rows; the oracle runs the unpadded problem."""
    w = syn.C3.with_tokens(96)
    _run_forward_backward(w)


def test_k_equals_dff_matches_dense_swiglu_formula():
    w = syn.Workload("dense", "f32", 33, 64, 96, 96, 96, seed=5)
    x, wg, wu, wd, _ = _problem(w)
    out, idx, tg, tu = B.moc_ffn_forward(_dev(x), _dev(wg), _dev(wu), _dev(wd), w.k)
    x64, wg64, wu64, wd64 = map(syn.to_f64, (x, wg, wu, wd))
    G, U = x64 @ wg64.T, x64 @ wu64.T
    dense = (G / (1 + np.exp(-G)) * U) @ wd64
    parity.assert_close(syn.to_f64(out), dense, "f32", "dense SwiGLU")
    np.testing.assert_array_equal(idx.cpu().numpy(), np.tile(np.arange(96, dtype=np.int16), (33, 1)))


def test_inference_forward_saves_nothing_and_matches_training_forward():
    w = syn.Workload("inf", "bf16", 300, 128, 256, 256, 32, seed=9)
    x, wg, wu, wd, _ = map(_dev, _problem(w))
    out_a, *_ = B.moc_ffn_forward(x, wg, wu, wd, w.k, save=True)
    out_b, idx, tg, tu = B.moc_ffn_forward(x, wg, wu, wd, w.k, save=False)
    assert idx is None and tg is None and tu is None
    assert torch.equal(out_a, out_b)


def test_forward_and_backward_are_deterministic():
    w = syn.Workload("det", "bf16", 257, 128, 300, 304, 40, seed=3)
    _, (x, wg, wu, wd, dD), (out, idx, tg, tu), g1 = _run_forward_backward(w)
    out2, idx2, tg2, tu2 = B.moc_ffn_forward(x, wg, wu, wd, w.k, d_ff=w.d_ff)
    assert torch.equal(out, out2) and torch.equal(idx, idx2) and torch.equal(tg, tg2) and torch.equal(tu, tu2)
    g2 = B.moc_ffn_backward(x, wg, wu, wd, idx, tg, tu, dD, d_ff=w.d_ff)
    for k in g1:
        assert torch.equal(g1[k], g2[k]), k


def test_backward_partial_outputs_and_accumulate_flag():
    w = syn.Workload("acc", "f32", 64, 64, 128, 128, 16, seed=8)
    _, (x, wg, wu, wd, dD), (out, idx, tg, tu), full = _run_forward_backward(w)
    part = B.moc_ffn_backward(x, wg, wu, wd, idx, tg, tu, dD, want=("w_up",))
    assert part["grad_x"] is None and part["grad_w_down"] is None
    assert torch.equal(part["grad_w_up"], full["grad_w_up"])
    only_x = B.moc_ffn_backward(x, wg, wu, wd, idx, tg, tu, dD, want=("x",))
    assert torch.equal(only_x["grad_x"], full["grad_x"])
    base = {k: torch.full_like(v, 0.5) for k, v in full.items() if k != "grad_x"}
    acc = B.moc_ffn_backward(x, wg, wu, wd, idx, tg, tu, dD, want=("w_gate", "w_up", "w_down"), grads=base,
                             accumulate=True)
    for k in ("grad_w_gate", "grad_w_up", "grad_w_down"):
        torch.testing.assert_close(acc[k], full[k] + 0.5, rtol=1e-6, atol=1e-6)
    # rows of channels no token selected are exactly zero
    used = torch.zeros(w.d_ff, dtype=torch.bool, device="cuda")
    used[idx.long().flatten()] = True
    if (~used).any():
        for k in ("grad_w_gate", "grad_w_up", "grad_w_down"):
            assert torch.all(full[k][~used] == 0)


def test_corrupted_saved_index_is_skipped_and_reported():
    w = syn.Workload("bad", "bf16", 40, 64, 96, 96, 8, seed=12)
    _, (x, wg, wu, wd, dD), (out, idx, tg, tu), full = _run_forward_backward(w)
    bad = idx.clone()
    bad[3, 2] = 96       # == d_ff: out of range
    bad[7, 0] = -5
    assert B.moc_last_device_status() == B.MOC_OK
    g = B.moc_ffn_backward(x, wg, wu, wd, bad, tg, tu, dD)
    assert B.moc_last_device_status() == B.MOC_ERR_BAD_INDEX
    assert B.moc_last_device_status() == B.MOC_OK      # reading clears it
    # the other tokens' grad_x rows are untouched by the corruption
    keep = torch.ones(w.tokens, dtype=torch.bool, device="cuda")
    keep[3] = keep[7] = False
    assert torch.equal(g["grad_x"][keep], full["grad_x"][keep])
    assert torch.isfinite(g["grad_w_down"].float()).all()


def test_host_errors_raise_before_launch():
    w = syn.Workload("err", "bf16", 8, 64, 96, 96, 8, seed=1)
    x, wg, wu, wd, _ = map(_dev, _problem(w))
    with pytest.raises(B.MocError) as e:
        B.moc_ffn_forward(x, wg, wu, wd, 97)
    assert e.value.status == B.MOC_ERR_INVALID_ARG
    with pytest.raises(B.MocError) as e:
        B.moc_ffn_forward(x, wg, wu, wd, 8, workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert e.value.status == B.MOC_ERR_WORKSPACE
    with pytest.raises(B.MocError) as e:
        B.moc_ffn_decode(_dev(syn.make_x(w, tokens=257)), wg, wu, wd, 8)
    assert e.value.status == B.MOC_ERR_UNSUPPORTED
    assert B.moc_last_device_status() == B.MOC_OK


def test_zero_tokens_is_a_noop():
    x = torch.empty((0, 64), dtype=torch.bfloat16, device="cuda")
    wg = torch.zeros((32, 64), dtype=torch.bfloat16, device="cuda")
    out, idx, tg, tu = B.moc_ffn_forward(x, wg, wg, wg, 4)
    assert out.shape == (0, 64) and idx.shape == (0, 4)


# ------------------------------------------------------------------ decode


def _check_decode(out64, x64, wg64, wu64, wd64, K, dtype, what):
    parity.check_decode(out64, x64, wg64, wu64, wd64, K, dtype, what)


@pytest.mark.parametrize("T", [1, 2, 4, 5, 6, 16])   # 1, 2: cooperative kernel; to 5: four-kernel plan; from 6: small-batch plan
def test_decode_llama7b_shape(T):
    w = syn.C4.with_tokens(T)
    wg, wu, wd = syn.make_weights(w)
    x = syn.make_x(w)
    out = B.moc_ffn_decode(_dev(x), _dev(wg), _dev(wu), _dev(wd), w.k)
    torch.cuda.synchronize()
    x64, wg64, wu64, wd64 = map(syn.to_f64, (x, wg, wu, wd))
    _check_decode(syn.to_f64(out), x64, wg64, wu64, wd64, w.k, "bf16", f"decode T={T}")


def test_decode_with_padded_weight_arrays():
    """d_ff = 1000 in arrays of 1024 rows whose tail holds junk: the padding rows must never be selected or read as
    channels by the decode path (bf16 decode plan at few tokens or few kept channels, the small-batch plan where most
    channels are used, and the fp32 gathered plan)."""
    for dtype, T, K in (("bf16", 3, 125), ("bf16", 16, 20), ("bf16", 16, 125), ("f32", 2, 125)):
        w = syn.Workload(f"dec-pad-{dtype}-{T}-{K}", dtype, T, 128, 1000, 1024, K, seed=640 + T)
        wg, wu, wd = syn.make_weights(w)
        for m in (wg, wu, wd):
            m[w.d_ff:] = 3.0      # junk, larger than any real gate value
        x = syn.make_x(w)
        out = B.moc_ffn_decode(_dev(x), _dev(wg), _dev(wu), _dev(wd), w.k, d_ff=w.d_ff)
        torch.cuda.synchronize()
        x64, wg64, wu64, wd64 = map(syn.to_f64, (x, wg[:w.d_ff], wu[:w.d_ff], wd[:w.d_ff]))
        _check_decode(syn.to_f64(out), x64, wg64, wu64, wd64, w.k, dtype, f"padded decode {dtype} T={T} K={K}")


@pytest.mark.parametrize("dtype,T,d,F,K", [
    ("f32", 3, 64, 200, 25),
    ("bf16", 16, 256, 1000, 125),   # most channels used by some token: small-batch plan
    ("bf16", 16, 512, 4096, 64),    # sixteen tokens, few kept channels: decode plan with its full batch
    ("bf16", 5, 520, 777, 97),      # decode plan, ragged everything
    ("bf16", 7, 520, 777, 97),      # small-batch plan below 17 tokens
])
def test_decode_small_shapes(dtype, T, d, F, K):
    w = syn.Workload("dec", dtype, T, d, F, F, K, seed=77, decode=True)
    wg, wu, wd = syn.make_weights(w)
    x = syn.make_x(w)
    out = B.moc_ffn_decode(_dev(x), _dev(wg), _dev(wu), _dev(wd), K)
    out_f, *_ = B.moc_ffn_forward(_dev(x), _dev(wg), _dev(wu), _dev(wd), K, save=False)
    x64, wg64, wu64, wd64 = map(syn.to_f64, (x, wg, wu, wd))
    _check_decode(syn.to_f64(out), x64, wg64, wu64, wd64, K, dtype, "decode")
    _check_decode(syn.to_f64(out_f), x64, wg64, wu64, wd64, K, dtype, "forward(save=False)")


# ------------------------------------------------------------------ tensor-core plan (bf16)


@pytest.mark.parametrize("T,d,F,F_ld,K", [
    (513, 264, 1100, 1104, 137),   # d not a multiple of 64, F not a multiple of 256, ragged token tile
    (320, 128, 96, 96, 96),        # K = F: dense SwiGLU through the tensor-core plan
    (384, 512, 4500, 4504, 563),   # more than 4096 channels: few warps per SM in the warp-per-token selector
    (257, 8, 64, 64, 1),           # smallest contraction, a single kept channel
    (300, 64, 200, 200, 199),      # all but one channel kept
    (270, 64, 2048, 2048, 1500),   # more kept channels than the search scratch can park: gate row freed late
    (300, 128, 9000, 9000, 700),   # long rows: teams of four warps, two tokens in flight per SM
    (260, 64, 16000, 16000, 1200), # rows too long for separate gate and up buffers: both rows share one buffer
    (260, 64, 24000, 24000, 1500), # rows too long for any shared-memory slice: CTA-per-token selector
])
def test_tc_plan_shapes(T, d, F, F_ld, K):
    w = syn.Workload(f"tc-{T}-{d}-{F}-{K}", "bf16", T, d, F, F_ld, K, seed=200 + T)
    _run_forward_backward(w)


def test_bf16_rows_too_long_for_the_tensor_core_selector_take_the_gathered_plan():
    """(d_ff + k) * 4 bytes beyond the selector's shared memory: bf16 falls back to the exact gathered kernels."""
    w = syn.Workload("bf16-gathered", "bf16", 5, 64, 32768, 32768, 11008, seed=77)
    _run_forward_backward(w)


def test_tc_plan_forward_in_several_token_chunks(monkeypatch):
    """A 1 MiB bound on the transient gate array makes the forward run its GEMM + selector over five token chunks
    (the last one ragged); results must not depend on the chunking."""
    monkeypatch.setenv("MOC_FFN_FWD_CHUNK_MIB", "1")
    w = syn.Workload("tc-chunked", "bf16", 513, 264, 1100, 1104, 137, seed=713)
    _run_forward_backward(w)


def test_tc_plan_llama1b_padded_slice():
    """C3's layer (d_ff = 5461 in arrays of 5504 rows) on enough tokens to take the tensor-core plan."""
    _run_forward_backward(syn.C3.with_tokens(384))


def test_tc_plan_sweep_k_fractions():
    """C5's K fractions d_ff/16, d_ff/8, d_ff/4 on a 1B-shaped layer narrowed to keep the oracle fast."""
    for K in (64, 128, 256):
        w = syn.Workload(f"c5-{K}", "bf16", 320, 512, 1024, 1024, K, seed=500 + K)
        _run_forward_backward(w)


def test_ties_go_to_the_lower_channel_on_both_plans():
    """Duplicated gate rows give bit-identical gate values; when only one of a pair fits, it must be the lower."""
    for T in (64, 320):   # gathered plan, tensor-core plan
        w = syn.Workload("ties", "bf16", T, 128, 512, 512, 65, seed=77)
        wg, wu, wd = syn.make_weights(w)
        wg[1::2] = wg[0::2]          # channels 2i and 2i+1 share their gate row
        x = syn.make_x(w)
        out, idx, tg, tu = B.moc_ffn_forward(_dev(x), _dev(wg), _dev(wu), _dev(wd), w.k)
        idx = idx.cpu().numpy().astype(np.int64)
        split = 0
        for t in range(T):
            sel = set(idx[t].tolist())
            for j in idx[t]:
                if j % 2 == 1:
                    assert j - 1 in sel, f"token {t}: channel {j} kept without its equal lower twin {j - 1}"
                elif j + 1 not in sel:
                    split += 1
        assert split > 0   # K is odd: every token splits exactly one pair
        x64, wg64, wu64, wd64 = map(syn.to_f64, (x, wg, wu, wd))
        dev = dict(out=syn.to_f64(out), idx=idx, gval=syn.to_f64(tg), uval=syn.to_f64(tu))
        parity.check_forward(dev, x64, wg64, wu64, wd64, w.k, w.d_ff, w.dtype)


def test_tc_plan_degenerate_and_badly_scaled_tokens():
    """Tokens the selector's bracket cannot anticipate: all-zero rows (every gate value ties: channels 0..K-1 are
    kept), rows scaled by 1e3 and by 1e-3 between ordinary ones (the bracket has to move far and back), and a
    batch whose first launch has no bracket at all (fresh workspace filled with NaN bytes)."""
    w = syn.Workload("odd-tokens", "bf16", 600, 256, 2048, 2048, 256, seed=4242)
    wg, wu, wd = syn.make_weights(w)
    x = syn.make_x(w).float()
    x[5::50] = 0.0
    x[7::50] *= 1.0e3
    x[11::50] *= 1.0e-3
    x = x.to(torch.bfloat16)
    xd, wgd, wud, wdd = map(_dev, (x, wg, wu, wd))
    desc = B.make_desc(w.tokens, w.d_model, w.d_ff, w.k, xd.dtype)
    ws = B.alloc_workspace(desc, B.MOC_OP_FORWARD)
    ws.fill_(0xFF)      # whatever a new workspace holds must not matter
    for attempt in range(2):   # second call: the bracket left by the first one is in the workspace
        out, idx, tg, tu = B.moc_ffn_forward(xd, wgd, wud, wdd, w.k, workspace=ws)
        torch.cuda.synchronize()
        assert B.moc_last_device_status() == B.MOC_OK
        idx_np = idx.cpu().numpy().astype(np.int64)
        for t in range(5, w.tokens, 50):
            assert np.array_equal(idx_np[t], np.arange(w.k)), f"zero token {t}"
        x64, wg64, wu64, wd64 = map(syn.to_f64, (x, wg, wu, wd))
        dev = dict(out=syn.to_f64(out), idx=idx_np, gval=syn.to_f64(tg), uval=syn.to_f64(tu))
        parity.check_forward(dev, x64, wg64, wu64, wd64, w.k, w.d_ff, w.dtype)


def test_tc_plan_backward_options_and_determinism():
    w = syn.Workload("tc-opts", "bf16", 384, 256, 768, 768, 96, seed=41)
    _, (x, wg, wu, wd, dD), (out, idx, tg, tu), full = _run_forward_backward(w)
    out2, idx2, tg2, tu2 = B.moc_ffn_forward(x, wg, wu, wd, w.k)
    assert torch.equal(out, out2) and torch.equal(idx, idx2) and torch.equal(tg, tg2) and torch.equal(tu, tu2)
    again = B.moc_ffn_backward(x, wg, wu, wd, idx, tg, tu, dD)
    for k in full:
        assert torch.equal(full[k], again[k]), k
    part = B.moc_ffn_backward(x, wg, wu, wd, idx, tg, tu, dD, want=("w_down", "x"))
    assert part["grad_w_gate"] is None and part["grad_w_up"] is None
    assert torch.equal(part["grad_w_down"], full["grad_w_down"]) and torch.equal(part["grad_x"], full["grad_x"])
    base = {k: torch.full_like(v, 0.25) for k, v in full.items() if k != "grad_x"}
    acc = B.moc_ffn_backward(x, wg, wu, wd, idx, tg, tu, dD, want=("w_gate", "w_up", "w_down"), grads=base,
                             accumulate=True)
    for k in ("grad_w_gate", "grad_w_up", "grad_w_down"):
        ref = full[k].float() + 0.25
        assert (acc[k].float() - ref).abs().max() <= 1e-2 * ref.abs().max()
    inf_out, *_ = B.moc_ffn_forward(x, wg, wu, wd, w.k, save=False)
    assert torch.equal(inf_out, out)


def test_tc_plan_corrupted_saved_index_is_skipped_and_reported():
    w = syn.Workload("tc-bad", "bf16", 300, 128, 256, 256, 32, seed=13)
    _, (x, wg, wu, wd, dD), (out, idx, tg, tu), full = _run_forward_backward(w)
    bad = idx.clone()
    bad[5, 3] = 256
    bad[9, 0] = -1
    g = B.moc_ffn_backward(x, wg, wu, wd, bad, tg, tu, dD)
    assert B.moc_last_device_status() == B.MOC_ERR_BAD_INDEX
    assert B.moc_last_device_status() == B.MOC_OK
    keep = torch.ones(w.tokens, dtype=torch.bool, device="cuda")
    keep[5] = keep[9] = False
    assert torch.equal(g["grad_x"][keep], full["grad_x"][keep])
    for k in g:
        assert torch.isfinite(g[k].float()).all()


def _full_size_sampled(w, n_tokens, n_rows, graph=False):
    x, wg, wu, wd, dD = _problem(w)
    xd, wgd, wud, wdd, dDd = map(_dev, (x, wg, wu, wd, dD))
    out, idx, tg, tu = B.moc_ffn_forward(xd, wgd, wud, wdd, w.k, d_ff=w.d_ff)
    grads = B.moc_ffn_backward(xd, wgd, wud, wdd, idx, tg, tu, dDd, d_ff=w.d_ff)
    torch.cuda.synchronize()
    if graph:
        # the launch configuration bench.py times: both calls captured once into a CUDA graph (preallocated outputs
        # and workspaces, a side stream) and replayed; the buffers are cleared first so that what is checked below
        # was written by the replays
        names = ("grad_x", "grad_w_gate", "grad_w_up", "grad_w_down")
        desc = B.make_desc(w.tokens, w.d_model, w.d_ff, w.k, xd.dtype, d_ff_ld=w.d_ff_ld)
        ws_f = B.alloc_workspace(desc, B.MOC_OP_FORWARD, xd.device)
        ws_b = B.alloc_workspace(desc, B.MOC_OP_BACKWARD, xd.device)
        stream = torch.cuda.Stream()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            with torch.cuda.graph(g, stream=stream):
                B.moc_ffn_forward(xd, wgd, wud, wdd, w.k, d_ff=w.d_ff, out=out, saved=(idx, tg, tu), workspace=ws_f,
                                  stream=stream)
                B.moc_ffn_backward(xd, wgd, wud, wdd, idx, tg, tu, dDd, d_ff=w.d_ff, grads=grads, workspace=ws_b,
                                   stream=stream)
        torch.cuda.synchronize()
        for t in (out, idx, tg, tu, *(grads[n] for n in names)):
            t.zero_()
        g.replay()
        g.replay()
        torch.cuda.synchronize()
    assert B.moc_last_device_status() == B.MOC_OK
    rng = np.random.default_rng(0)
    toks = np.sort(rng.choice(w.tokens, n_tokens, replace=False))
    wg64, wu64, wd64 = map(syn.to_f64, (wg, wu, wd))
    x64s, dD64s = syn.to_f64(x[toks]), syn.to_f64(dD[toks])
    idx_np = idx.cpu().numpy()
    dev = dict(out=syn.to_f64(out[toks]), idx=idx_np[toks], gval=syn.to_f64(tg[toks]), uval=syn.to_f64(tu[toks]))
    parity.check_forward(dev, x64s, wg64, wu64, wd64, w.k, w.d_ff, w.dtype)
    ref = orc.backward(x64s, wg64, wu64, wd64, idx_np[toks].astype(np.int32), dev["gval"], dev["uval"], dD64s,
                       F=w.d_ff, want=("x",))
    parity.assert_close(syn.to_f64(grads["grad_x"][toks]), ref["grad_x"], w.dtype, "grad_x (sampled tokens)")
    rows = np.sort(rng.choice(w.d_ff, n_rows, replace=False)).astype(np.int32)
    wrows = orc.backward_weight_rows(syn.to_f64(x), wd64, idx_np.astype(np.int32), syn.to_f64(tg), syn.to_f64(tu),
                                     syn.to_f64(dD), rows, w.d_ff)
    for name in ("grad_w_gate", "grad_w_up", "grad_w_down"):
        got = syn.to_f64(grads[name][torch.from_numpy(rows.astype(np.int64)).cuda()])
        parity.assert_close(got, wrows[name], w.dtype, name + " (sampled rows)")
        if w.d_ff_ld > w.d_ff:   # padding rows of the weight gradients stay exactly zero
            assert torch.all(grads[name][w.d_ff:] == 0), name
    # structural properties at full size
    parity.check_index_sets(idx_np, w.d_ff)


def test_full_size_bench_workload_sampled_against_oracle():
    """C2 at its full 16384 tokens, in the configuration bench.py times: sampled tokens of out / saved values /
    grad_x and sampled rows of the weight gradients are recomputed one by one by the oracle."""
    _full_size_sampled(syn.C2, 96, 24)


def test_full_size_bench_workload_replayed_from_a_cuda_graph():
    """The same comparison on the outputs of a CUDA graph replay of forward + backward (how bench.py launches them)."""
    _full_size_sampled(syn.C2, 48, 12, graph=True)


@pytest.mark.parametrize("T", [1, 2, 4, 16, 64])
def test_decode_replayed_from_a_cuda_graph_with_rotating_weights(T):
    """bench.py's decode timing replays a CUDA graph of calls that rotate weight sets: every plan (the cooperative
    kernel, the four-kernel chain, the small-batch kernels) must give under replay what its direct call gives."""
    w = syn.C4.with_tokens(T)
    sets = [tuple(t.cuda() for t in syn.make_weights(w, seed_offset=s)) for s in range(2)]
    x = syn.make_x(w).cuda()
    desc = B.make_desc(T, w.d_model, w.d_ff, w.k, x.dtype)
    ws = B.alloc_workspace(desc, B.MOC_OP_DECODE, x.device)
    direct = [B.moc_ffn_decode(x, *sets[i], w.k, workspace=ws).clone() for i in range(2)]
    torch.cuda.synchronize()
    outs = [torch.zeros_like(x) for _ in range(4)]
    stream = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(g, stream=stream):
            for i in range(4):
                B.moc_ffn_decode(x, *sets[i % 2], w.k, out=outs[i], workspace=ws, stream=stream)
    torch.cuda.synchronize()
    for o in outs:
        o.zero_()
    g.replay()
    g.replay()
    torch.cuda.synchronize()
    assert B.moc_last_device_status() == B.MOC_OK
    for i in range(4):   # the partial sums meet in an order that is not fixed: last-bit differences only
        torch.testing.assert_close(outs[i].float(), direct[i % 2].float(), rtol=2e-2, atol=2e-3)


def test_full_size_llama1b_padded_sampled_against_oracle():
    """C3 at its full 32768 tokens (d_ff = 5461 in arrays of 5504 rows): the same sampled comparison."""
    _full_size_sampled(syn.C3, 64, 16)


@pytest.mark.parametrize("K", [344, 1376])
def test_full_size_sweep_workload_sampled_against_oracle(K):
    """C5 at its full 65536 tokens with the smallest and the largest K of the sweep (d_ff / 16 and d_ff / 4)."""
    import dataclasses
    _full_size_sampled(dataclasses.replace(syn.C5, k=K, name=f"C5-k{K}"), 32, 8)


def test_bounded_wait_runs_out_reports_timeout_and_leaves_the_context_usable():
    """The time-out path all kernels share: a wait on a barrier nothing completes gives up after its limit (here
    50 M cycles, about 25 ms), the kernel returns normally, the status word reads MOC_ERR_TIMEOUT once, and the
    next call works."""
    import time
    assert B.moc_last_device_status() == B.MOC_OK
    t0 = time.perf_counter()
    B.moc_test_bounded_wait(50_000_000)
    assert B.moc_last_device_status() == B.MOC_ERR_TIMEOUT          # synchronises, reports, clears
    assert time.perf_counter() - t0 < 2.0
    assert B.moc_last_device_status() == B.MOC_OK
    with pytest.raises(B.MocError):
        B.moc_test_bounded_wait(0)                                   # limit out of range: nothing launched
    _run_forward_backward(syn.Workload("after-timeout", "bf16", 300, 128, 512, 512, 64, seed=9))
    assert B.moc_last_device_status() == B.MOC_OK


def test_decode_four_kernel_plan_selected_by_environment():
    """MOC_FFN_DECODE=chain (read once per process) keeps one- and two-token batches on the four-kernel decode plan
    instead of the cooperative kernel: run the decode cases again in a child process with it set."""
    import os
    import subprocess
    import sys
    env = dict(os.environ, MOC_FFN_DECODE="chain")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(root, "tests", "test_gpu_parity.py"),
                        os.path.join(root, "tests", "test_gpu_grouped.py"), "-q", "-x", "-m", "gpu", "-k",
                        "decode_llama7b_shape or decode_small_shapes or decode_with_padded or grouped_decode or decode_ties"],
                       cwd=root, env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]


@pytest.mark.parametrize("T", [1, 2, 4, 8])
def test_decode_ties_and_degenerate_tokens(T):
    """Duplicated gate rows (bit-identical gate values; K odd, so exactly one pair is split and the lower channel must
    win), an all-zero token (every value ties: channels 0..K-1) -- through every decode form (cooperative kernel,
    four-kernel plan, small-batch plan)."""
    w = syn.Workload("dec-ties", "bf16", T, 128, 512, 512, 65, seed=77 + T, decode=True)
    wg, wu, wd = syn.make_weights(w)
    wg[1::2] = wg[0::2]
    x = syn.make_x(w)
    x[T - 1] = 0
    out = B.moc_ffn_decode(_dev(x), _dev(wg), _dev(wu), _dev(wd), w.k)
    torch.cuda.synchronize()
    assert torch.all(out[T - 1] == 0)
    x64, wg64, wu64, wd64 = map(syn.to_f64, (x, wg, wu, wd))
    ref = orc.forward(x64, wg64, wu64, wd64, w.k)["out"]     # the oracle's tie rule: the lower channel
    parity.assert_close(syn.to_f64(out), ref, "bf16", f"decode with ties T={T}")
