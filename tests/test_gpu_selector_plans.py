"""The selectors that the benchmarked plans run, each on its own, bit-exact against the oracle's Top-K rule.

`moc_topk_select` reaches the CTA-per-row selector of the decode / small-batch plans and the gathered plan's selector.
The tensor-core plan's forward pass runs other kernels (teams of two or four warps per row, with separate or shared
row buffers, and a CTA-per-row form for very long rows), and the one-kernel decode form selects without any SM holding
a whole row.  These tests put the same adversarial rows in front of every one of them: non-finite values, NaN,
denormals, rows thinning out over 140 octaves, clusters a few ulps apart, rows of equal values with K cutting the tie.
The mask must be the oracle's, index for index (Section 3.2: exactly K ones per row, the largest signed values; equal
values to the lower channel).
"""
import numpy as np
import pytest
import torch

from oracle import moc_oracle as orc
from paper_2511_09323_b200 import binding as B
from paper_2511_09323_b200 import build as moc_build

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    moc_build.build()
    B.load()
    assert B.moc_last_device_status() == B.MOC_OK
    yield
    assert B.moc_last_device_status() == B.MOC_OK


def _adversarial_rows(n):
    r = np.arange(n, dtype=np.float32)
    rng = np.random.default_rng
    rows = [
        np.zeros(n, np.float32),                                                       # all equal: K cuts the tie
        np.full(n, 3.25, np.float32),
        r.copy(),
        -r,
        np.where(r % 3 == 0, 1.0, -1.0).astype(np.float32),                            # two values
        np.where(r % 2 == 0, 0.0, -0.0).astype(np.float32),                            # +0 equals -0
        np.concatenate([[np.inf, -np.inf], np.linspace(-1, 1, n - 2)]).astype(np.float32),
        np.full(n, -np.inf, np.float32),
        np.where(r % 7 == 0, np.inf, 1.0).astype(np.float32),                          # threshold may be +inf
        np.where(r % 5 == 0, np.nan, np.sin(r)).astype(np.float32),                    # NaN orders as -inf
        np.where(r % 2 == 0, np.nan, -np.inf).astype(np.float32),                      # nothing finite at all
        (np.round(rng(1).standard_normal(n) * 16) / 16).astype(np.float32),            # many duplicates
        rng(2).standard_normal(n).astype(np.float32) * np.float32(1e-30),              # tiny magnitudes
        np.float32(1e30) * rng(3).standard_normal(n).astype(np.float32),               # huge magnitudes
        (np.float32(2.0) ** (-(r % 140))).astype(np.float32),                          # thinning out over 140 octaves
        (np.float32(1.0) + (r % 97) * np.float32(1.2e-7)).astype(np.float32),          # a few ulps apart
        np.where(r == 0, 1e30, np.where(r == 1, -1e30, rng(4).standard_normal(n) * 1e-3)).astype(np.float32),
        (rng(5).standard_normal(n) * 1e-42).astype(np.float32),                        # denormals
        rng(6).standard_normal(n).astype(np.float32),                                  # plain Gaussian rows
        rng(7).standard_normal(n).astype(np.float32) * np.float32(0.55) + np.float32(0.1),
    ]
    return np.stack(rows)


def _k_values(n):
    return sorted({1, 2, max(1, n // 8), max(1, n - 1), n})


# (row length, leading dimension): the LLaMA-130M / 1B / 7B widths, ragged lengths, and the long rows that switch the
# kernel form (shared row buffer from about 14000 channels, a CTA per row beyond what a team's slice holds)
TC_SHAPES = [(300, 304), (2048, 2048), (4096, 4096), (5461, 5464), (5461, 5504), (5504, 5504), (9000, 9000),
             (11008, 11008), (16000, 16000), (24000, 24000), (32768, 32768)]
BRACKETS = [None, (0.6, 0.2), (1.0e6, 1.0), (-3.0, 1.0e-20), (0.0, 1.0e30), (float("nan"), 1.0), (1.0, float("inf"))]


@pytest.mark.parametrize("n,n_ld", TC_SHAPES)
def test_tensor_core_plan_selector_bit_exact_adversarial(n, n_ld):
    rows = _adversarial_rows(n)
    # Gaussian rows in between, as in a real batch: the launch's running bracket then sees ordinary and odd rows mixed
    rows = np.concatenate([rows, np.random.default_rng(8).standard_normal((44, n)).astype(np.float32), rows[::-1]])
    g = np.full((rows.shape[0], n_ld), 1e9, np.float32)   # padding columns hold large values: must be ignored
    g[:, :n] = rows
    gd = torch.from_numpy(g).cuda()
    ran = 0
    for k in _k_values(n):
        if B.load().moc_topk_select_tc_workspace_bytes(g.shape[0], n, n_ld, k) == 0:
            continue      # (n + k) words do not fit the selector's shared memory: the forward pass takes another plan
        ref = orc.topk(g, k, F=n)
        for bracket in BRACKETS:
            got, variant = B.moc_topk_select_tc(gd, k, n=n, bracket=bracket)
            got = got.cpu().numpy().astype(np.int32)
            np.testing.assert_array_equal(got, ref, err_msg=f"n={n} k={k} bracket={bracket} variant={variant}")
            ran += 1
    assert ran >= len(BRACKETS) * 3
    assert B.moc_last_device_status() == B.MOC_OK


def test_every_form_of_the_tensor_core_selector_is_reached():
    """The shapes above, with their K values, run all four kernel forms (asked from the library without a launch)."""
    import ctypes
    lib = B.load()
    seen = set()
    for n, n_ld in TC_SHAPES:
        for k in _k_values(n):
            if lib.moc_topk_select_tc_workspace_bytes(0, n, n_ld, k) == 0:
                continue
            v = ctypes.c_int(-1)
            assert lib.moc_topk_select_tc(0, n, n_ld, k, None, None, None, ctypes.byref(v), None, 0, None) == B.MOC_OK
            seen.add(B.SELECT_VARIANTS[v.value])
    assert seen == set(B.SELECT_VARIANTS), seen


def test_tensor_core_selector_many_rows_and_running_bracket():
    """More rows than teams in flight (grid-stride over rows), thresholds drifting along the batch so that the
    bracket a team carries from row to row keeps missing."""
    rng = np.random.default_rng(9)
    n, rows = 2048, 5000
    g = rng.standard_normal((rows, n)).astype(np.float32) * np.linspace(0.01, 30.0, rows, dtype=np.float32)[:, None]
    g += np.linspace(-5.0, 5.0, rows, dtype=np.float32)[:, None]
    gd = torch.from_numpy(g).cuda()
    for k in (1, 256, 2047):
        got, variant = B.moc_topk_select_tc(gd, k, bracket=(0.3, 0.05))
        assert variant == "team2"
        np.testing.assert_array_equal(got.cpu().numpy().astype(np.int32), orc.topk(g, k))


def test_selector_hook_rejects_bad_shapes():
    lib = B.load()
    assert lib.moc_topk_select_tc_workspace_bytes(4, 100, 100, 10) == 0        # leading dimension not a multiple of 8
    assert lib.moc_topk_select_tc_workspace_bytes(4, 100, 256, 10) == 0        # more padding than one 128-channel group
    assert lib.moc_topk_select_tc_workspace_bytes(4, 100, 104, 101) == 0       # k > n
    assert lib.moc_topk_select_tc_workspace_bytes(4, 32768, 32768, 32768) == 0  # keys + kept list exceed shared memory
    assert lib.moc_topk_select_tc(4, 100, 100, 10, None, None, None, None, None, 0, None) == B.MOC_ERR_INVALID_ARG


# ---------------------------------------------------------------- the one-kernel decode form


def _bf16_rows(n):
    """Adversarial rows that bf16 holds exactly (the gate values reach the kernel through a bf16 weight matrix)."""
    r = np.arange(n, dtype=np.float32)
    rows = _adversarial_rows(n)
    rows = torch.from_numpy(rows).to(torch.bfloat16).to(torch.float32).numpy()
    extra = np.stack([
        (np.float32(1.0) + (r % 5) * np.float32(2.0 ** -7)).astype(np.float32),       # adjacent bf16 values
        np.where(r % 2 == 0, np.float32(9.2e-41), np.float32(-9.2e-41)),              # bf16 denormals
    ])
    return np.concatenate([rows, extra])


def _probe(rows_f32, F, F_ld, d, K, cols):
    """Runs the one-kernel decode form on tokens x_t = e_{cols[t]} with row t stored as column cols[t] of W_gate, so
    that the kernel's gate values ARE the rows; returns its mask [T, F]."""
    T = rows_f32.shape[0]
    wg = torch.zeros((F_ld, d), dtype=torch.bfloat16)
    for t, c in enumerate(cols):
        wg[:F, c] = torch.from_numpy(rows_f32[t]).to(torch.bfloat16)
    if F_ld > F:
        wg[F:] = 7.0      # junk in the padding rows: never channels
    gen = torch.Generator().manual_seed(11)
    wu = (torch.randn(F_ld, d, generator=gen) * 0.02).to(torch.bfloat16)
    wd = (torch.randn(F_ld, d, generator=gen) * 0.02).to(torch.bfloat16)
    x = torch.zeros((T, d), dtype=torch.bfloat16)
    for t, c in enumerate(cols):
        x[t, c] = 1.0
    out, kept = B.moc_ffn_decode_probe(x.cuda(), wg.cuda(), wu.cuda(), wd.cuda(), K, d_ff=F)
    torch.cuda.synchronize()
    return kept.cpu().numpy()


def _mask_of(idx, F):
    m = np.zeros((idx.shape[0], F), np.uint8)
    np.put_along_axis(m, idx.astype(np.int64), 1, axis=1)
    return m


@pytest.mark.parametrize("F,F_ld", [(2048, 2048), (5461, 5504), (11008, 11008), (32768, 32768)])
def test_one_kernel_decode_selection_bit_exact_single_token(F, F_ld):
    rows = _bf16_rows(F)
    d = 64
    for k in _k_values(F):
        ref = _mask_of(orc.topk(rows, k), F)
        for i in range(rows.shape[0]):
            kept = _probe(rows[i: i + 1], F, F_ld, d, k, cols=[i % d])
            assert kept.max() <= 1, "the kernel did not write the whole mask"
            np.testing.assert_array_equal(kept[0], ref[i], err_msg=f"F={F} k={k} row {i}")
    assert B.moc_last_device_status() == B.MOC_OK


@pytest.mark.parametrize("F,F_ld", [(2048, 2048), (5461, 5504), (11008, 11008)])
def test_one_kernel_decode_selection_bit_exact_two_tokens(F, F_ld):
    """Two tokens share the kernel's histogram and candidate arrays.  Only finite rows here: a one-hot x multiplies
    the other token's column by zero, and 0 * inf would leak a NaN into this token's gate values."""
    rows = _bf16_rows(F)
    rows = rows[np.isfinite(rows).all(axis=1)]
    d = 128
    for k in _k_values(F):
        ref = _mask_of(orc.topk(rows, k), F)
        for i in range(0, rows.shape[0] - 1):
            pair = np.stack([rows[i], rows[(i + 5) % rows.shape[0]]])
            kept = _probe(pair, F, F_ld, d, k, cols=[3, 77])
            np.testing.assert_array_equal(kept[0], ref[i], err_msg=f"F={F} k={k} rows {i} (token 0)")
            np.testing.assert_array_equal(kept[1], ref[(i + 5) % rows.shape[0]], err_msg=f"F={F} k={k} (token 1)")
    assert B.moc_last_device_status() == B.MOC_OK
