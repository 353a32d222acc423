"""The one-kernel form of the small-batch plan (up to 32 tokens, nothing saved): streamer CTAs and selector CTAs of one
cooperative launch, two MMA issuers per streamer.  Every case checks that this kernel is the one that ran, compares the
output with the oracle's (the selection of Section 3.2, the gated product of Eq. (MoC-2), the down projection), and
most compare it with the three-kernel form of the same library, which `moc_ffn_forward` takes when it saves the triple.
"""
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


def _kernels_of(call):
    B.moc_profile_enable(True)
    call()
    prof = B.moc_profile_collect()
    B.moc_profile_enable(False)
    return {k for k, (n, _) in prof.items() if n}


def _oracle_check(out, x, wg, wu, wd, F, K, what):
    x64, wg64, wu64, wd64 = map(syn.to_f64, (x, wg[:F], wu[:F], wd[:F]))
    full = orc.forward(x64, wg64, wu64, wd64, K, want_g=True)
    out64 = syn.to_f64(out)
    tol = parity.REL_TOL["bf16"] * max(np.abs(full["out"]).max(), 1e-30)
    for t in range(x64.shape[0]):
        err = np.abs(out64[t] - full["out"][t]).max()
        if err <= tol:
            continue
        # a token whose K-th and (K+1)-th gate values nearly tie may have taken the swapped pick
        g = full["g"][t]
        order = np.lexsort((np.arange(F), -g))
        assert K < F and g[order[K - 1]] - g[order[K]] <= 1e-4, f"{what}: token {t} error {err:.3e} > {tol:.3e}"
        alt = np.sort(np.concatenate([order[: K - 1], order[K: K + 1]])).astype(np.int32)[None]
        ref = orc.forward_given_idx(x64[t: t + 1], wg64, wu64, wd64, alt)["out"][0]
        assert np.abs(out64[t] - ref).max() <= tol, f"{what}: token {t} matches neither pick"


# (tokens, d_model, d_ff, leading dimension of the weights' channel axis, K)
SHAPES = [
    (16, 64, 96, 96, 12),            # one stage per matrix and per column block: the second MMA issuer has nothing to do
    (1, 128, 512, 512, 64),          # a single token (one selector CTA)
    (7, 192, 333, 336, 41),          # ragged channel count, padding rows in the weights, 3 contraction blocks
    (16, 256, 1000, 1000, 125),      # 16 tokens: the 16-column MMA
    (17, 256, 1000, 1000, 125),      # 17 tokens: the 32-column MMA, second chunk of one token
    (32, 264, 520, 520, 65),         # the largest batch; contraction 4 blocks + 8 elements
    (20, 1024, 2048, 2048, 256),     # several stages per matrix: both issuers work, the ring goes round
    (12, 2048, 5461, 5464, 683),     # the LLaMA-1B layer, channel count not a multiple of 8
    (32, 512, 640, 640, 640),        # K = F: dense SwiGLU
    (9, 512, 640, 640, 1),           # a single kept channel
    (8, 128, 20000, 20000, 1500),    # more than 128 channels per CTA: two MMA tiles per streamer
    (30, 64, 24000, 24000, 1500),    # 32 tokens x two tiles: four epilogue items per TMEM lane quarter
    (16, 4096, 11008, 11008, 1376),  # the LLaMA-7B layer of the decode benchmark
]


@pytest.mark.parametrize("T,d,F,F_ld,K", SHAPES)
def test_one_kernel_form_against_oracle_and_three_kernel_form(T, d, F, F_ld, K):
    w = syn.Workload(f"sbf-{T}-{d}-{F}-{K}", "bf16", T, d, F, F_ld, K, seed=1300 + T + d)
    wg, wu, wd = syn.make_weights(w)
    if F_ld > F:
        for m in (wg, wu, wd):
            m[F:] = 3.0    # larger than any real gate value: must never be selected or read as channels
    x = syn.make_x(w)
    xd, wgd, wud, wdd = (t.cuda() for t in (x, wg, wu, wd))
    desc = B.make_desc(T, d, F, K, xd.dtype, d_ff_ld=F_ld)
    ws = B.alloc_workspace(desc, B.MOC_OP_FORWARD, xd.device)
    ws.fill_(0xff)          # nothing may depend on what the workspace held
    outs = []
    for rep in range(3):    # the first run of a workspace prepares the kernel's persistent flags, the others find them ready
        names = _kernels_of(lambda: outs.append(
            B.moc_ffn_forward(xd, wgd, wud, wdd, K, d_ff=F, save=False, workspace=ws)[0].clone()))
        assert "sb_fused" in names and "sb_down" not in names, names
        if rep == 0:
            ws.fill_(0x5a)  # the caller may do what it likes with the workspace between calls
    torch.cuda.synchronize()
    assert B.moc_last_device_status() == B.MOC_OK
    for o in outs:
        _oracle_check(o, x, wg, wu, wd, F, K, f"T={T} d={d} F={F} K={K}")
    # the partial sums of the down projection meet in a different order from run to run: equal up to that
    for o in outs[1:]:
        torch.testing.assert_close(o.float(), outs[0].float(), rtol=2e-2, atol=1e-3 * float(outs[0].float().abs().max()))
    # the three-kernel form (taken when the triple is saved): same selection; it rounds u to bf16 before the product,
    # as the backward pass will see it, so the outputs differ by a few units of bf16's last place of their largest terms
    saved = B.moc_ffn_forward(xd, wgd, wud, wdd, K, d_ff=F, workspace=ws)
    torch.cuda.synchronize()
    torch.testing.assert_close(outs[0].float(), saved[0].float(), rtol=3e-2, atol=6e-3 * float(saved[0].float().abs().max()))


def test_one_kernel_form_ties_and_degenerate_tokens():
    """Duplicated gate rows (equal values: the lower channel wins), an all-zero token (all values tie: channels 0..K-1
    are kept, the output is zero) and a token scaled by 1e4."""
    w = syn.Workload("sbf-ties", "bf16", 12, 128, 512, 512, 65, seed=77)
    wg, wu, wd = syn.make_weights(w)
    wg[1::2] = wg[0::2]
    x = syn.make_x(w)
    x[5] = 0
    x[9] *= 1e4
    xd, wgd, wud, wdd = (t.cuda() for t in (x, wg, wu, wd))
    out = None

    def run():
        nonlocal out
        out = B.moc_ffn_decode(xd, wgd, wud, wdd, w.k)

    names = _kernels_of(run)
    assert "sb_fused" in names, names
    torch.cuda.synchronize()
    assert torch.all(out[5] == 0)
    # against the path that returns its picks
    out_s, idx, tg, tu = B.moc_ffn_forward(xd, wgd, wud, wdd, w.k)
    idx = idx.cpu().numpy().astype(np.int64)
    np.testing.assert_array_equal(idx[5], np.arange(w.k))
    x64, wg64, wu64, wd64 = map(syn.to_f64, (x, wg, wu, wd))
    ref = orc.forward_given_idx(x64, wg64, wu64, wd64, idx.astype(np.int32))["out"]
    tol = parity.REL_TOL["bf16"] * np.abs(ref).max()
    assert np.abs(syn.to_f64(out) - ref).max() <= tol
    assert B.moc_last_device_status() == B.MOC_OK


def test_one_kernel_form_many_workspaces_and_batch_sizes_interleaved():
    """Each workspace address has its own persistent flags; calls on different workspaces, of different batch sizes
    and shapes, interleave freely."""
    w = syn.Workload("sbf-many", "bf16", 32, 256, 1000, 1000, 125, seed=5)
    wg, wu, wd = syn.make_weights(w)
    x = syn.make_x(w)
    xd, wgd, wud, wdd = (t.cuda() for t in (x, wg, wu, wd))
    x64, wg64, wu64, wd64 = map(syn.to_f64, (x, wg, wu, wd))
    spaces = []
    for i in range(5):
        desc = B.make_desc(32, w.d_model, w.d_ff, w.k, xd.dtype)
        spaces.append(B.alloc_workspace(desc, B.MOC_OP_DECODE, xd.device))
    results = []
    for rep in range(3):
        for i, T in enumerate((32, 5, 16, 21, 1)):
            results.append((T, B.moc_ffn_decode(xd[:T], wgd, wud, wdd, w.k, workspace=spaces[(i + rep) % 5])))
    torch.cuda.synchronize()
    assert B.moc_last_device_status() == B.MOC_OK
    full = orc.forward(x64, wg64, wu64, wd64, w.k)["out"]
    tol = parity.REL_TOL["bf16"] * np.abs(full).max()
    for T, out in results:
        if T < 6:
            continue   # (below 6 tokens moc_ffn_decode takes the gathering plans)
        bad = np.abs(syn.to_f64(out) - full[:T]).max(axis=1) > tol
        assert bad.sum() <= 1, f"T={T}: {bad.sum()} tokens off"   # (a near-tie may swap one pick)


@pytest.mark.parametrize("T,d,F", [
    (3, 512, 2048),       # three tokens (half of the channels are in use at K = F / 4)
    (16, 512, 2048),      # the 16-column MMA
    (32, 264, 1000),      # the largest batch; 125 groups, contraction 4 blocks + 8 elements
    (9, 128, 20000),      # more than 128 channels per CTA: groups in the second MMA tile
    (16, 2048, 5504),     # the LLaMA-1B layer (padded width) of the MoC 2:8 benchmark
])
def test_one_kernel_form_with_the_2_of_8_mask(T, d, F):
    """MoC 2:8 (Section 4): the mask is local to groups of 8 channels, so the kernel runs without selector CTAs and its
    streamers pick the two largest of every group themselves.  Picks (from the path that returns them) are checked
    against the oracle's rule, the output against the oracle's forward on those picks; equal gate rows in pairs make
    every group tie."""
    w = syn.Workload(f"sbf-2of8-{T}-{d}-{F}", "bf16", T, d, F, F, F // 4, seed=2100 + T)
    wg, wu, wd = syn.make_weights(w)
    if T == 16 and d == 512:
        wg[1::2] = wg[0::2]    # equal values inside every group: the lower channels win
    x = syn.make_x(w)
    xd, wgd, wud, wdd = (t.cuda() for t in (x, wg, wu, wd))
    outs = []
    for rep in range(2):
        names = _kernels_of(lambda: outs.append(B.moc_ffn_decode(xd, wgd, wud, wdd, None, grouped=True).clone()))
        assert "sb_fused" in names and "sb_select" not in names, names
    _, idx, _, _ = B.moc_ffn_forward(xd, wgd, wud, wdd, None, grouped=True)
    torch.cuda.synchronize()
    assert B.moc_last_device_status() == B.MOC_OK
    x64, wg64, wu64, wd64 = map(syn.to_f64, (x, wg, wu, wd))
    idx_np = idx.cpu().numpy()
    parity.check_picks_grouped(idx_np, orc.gate_projection(x64, wg64))
    ref = orc.forward_given_idx(x64, wg64, wu64, wd64, idx_np.astype(np.int32))["out"]
    for o in outs:
        parity.assert_close(syn.to_f64(o), ref, "bf16", "decode, 2 of 8")


def test_one_kernel_form_gives_up_cleanly_when_a_wait_cannot_complete():
    """The kernel's CTAs wait on one another through counters in global memory.  The test hook tells the selector CTAs
    to wait for one streamer more than exists and shortens every wait's limit to 100 M cycles (about 50 ms): every CTA
    then meets a wait that nothing completes, gives up, raises MOC_ERR_TIMEOUT and returns -- nothing hangs, traps or
    faults, `out` is not written, the context stays usable, and the next calls on the same workspace (which find no
    "clean" mark and prepare the counters themselves) are right."""
    import time
    w = syn.Workload("sbf-stall", "bf16", 8, 256, 1000, 1000, 125, seed=31)
    wg, wu, wd = syn.make_weights(w)
    x = syn.make_x(w)
    xd, wgd, wud, wdd = (t.cuda() for t in (x, wg, wu, wd))
    desc = B.make_desc(w.tokens, w.d_model, w.d_ff, w.k, xd.dtype)
    ws = B.alloc_workspace(desc, B.MOC_OP_DECODE, xd.device)
    first = B.moc_ffn_decode(xd, wgd, wud, wdd, w.k, workspace=ws).clone()   # leaves the workspace's counters marked clean
    assert B.moc_last_device_status() == B.MOC_OK
    out = torch.full_like(xd, 7.0)
    t0 = time.perf_counter()
    B.moc_test_small_batch_stall(xd, wgd, wud, wdd, w.k, 100_000_000, out=out, workspace=ws)
    assert B.moc_last_device_status() == B.MOC_ERR_TIMEOUT          # synchronises, reports, clears
    assert time.perf_counter() - t0 < 5.0
    assert B.moc_last_device_status() == B.MOC_OK
    assert torch.all(out == 7.0)
    with pytest.raises(B.MocError):
        B.moc_test_small_batch_stall(xd, wgd, wud, wdd, w.k, 0, out=out, workspace=ws)   # limit out of range: nothing launched
    for rep in range(2):
        names = _kernels_of(lambda: out.copy_(B.moc_ffn_decode(xd, wgd, wud, wdd, w.k, workspace=ws)))
        assert "sb_fused" in names, names
        torch.cuda.synchronize()
        _oracle_check(out, x, wg, wu, wd, w.d_ff, w.k, f"after the time-out, call {rep}")
        torch.testing.assert_close(out.float(), first.float(), rtol=2e-2, atol=1e-3 * float(first.float().abs().max()))
    assert B.moc_last_device_status() == B.MOC_OK
