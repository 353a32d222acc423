"""Pins for the CPU oracle: each check ties it to something other than itself.

* closed forms and textbook constants for SiLU and its derivative;
* numpy ``lexsort`` brute force for the Top-K mask (all K on tiny rows, adversarial rows);
* dense SwiGLU through numpy matmul + scipy ``expit`` for the K = d_ff special case;
* a literal dense-masked numpy evaluation of the forward and backward equations;
* central finite differences of the forward for every gradient;
* structural invariants (token independence, channel permutation, linearity, zero rows);
* the counting formulas and ratios the paper prints (tests/golden/paper_counts.txt).
"""
import math
import os

import numpy as np
import pytest
from scipy.special import expit

from oracle import moc_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_counts.txt")


def _rand_problem(seed, T, d, F, scale_w=0.3):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((T, d))
    wg = rng.standard_normal((F, d)) * scale_w
    wu = rng.standard_normal((F, d)) * scale_w
    wd = rng.standard_normal((F, d)) * scale_w
    return x, wg, wu, wd


def _np_topk_sets(g, K):
    """Brute force with numpy only: order by (value descending, channel ascending); NaN -> -inf."""
    g = np.where(np.isnan(g), -np.inf, g) + 0.0  # +0.0 folds -0.0 into +0.0
    out = np.empty((g.shape[0], K), dtype=np.int32)
    for t in range(g.shape[0]):
        order = np.lexsort((np.arange(g.shape[1]), -g[t]))
        out[t] = np.sort(order[:K])
    return out


def _np_silu(g):
    return g * expit(g)


def _np_dsilu(g):
    s = expit(g)
    return s * (1.0 + g * (1.0 - s))


def _dense_masked_forward(x, wg, wu, wd, K):
    """Eqs. (Moc-1), mask, (MoC-2) literally as dense matrices."""
    G = x @ wg.T
    U = x @ wu.T
    idx = _np_topk_sets(G, K)
    M = np.zeros_like(G)
    np.put_along_axis(M, idx.astype(np.int64), 1.0, axis=1)
    S = _np_silu(G)
    Sp = S * M
    Zp = Sp * U
    D = Zp @ wd
    return dict(G=G, U=U, M=M, S=S, Sp=Sp, Zp=Zp, D=D, idx=idx)


def _dense_masked_backward(x, wg, wu, wd, f, dD):
    """Eqs. (bp-1)..(bp-5) literally."""
    dWd = f["Zp"].T @ dD
    dZp = dD @ wd.T
    dSp = (f["U"] * f["M"]) * dZp
    dU = f["Sp"] * dZp
    dG = dSp * _np_dsilu(f["G"])
    dWg = (x.T @ dG).T        # paper's W is [d, d_ffn]; ours is its transpose (channel-major)
    dWu = (x.T @ dU).T
    dX = dG @ wg + dU @ wu
    return dict(grad_x=dX, grad_w_gate=dWg, grad_w_up=dWu, grad_w_down=dWd)


# ------------------------------------------------------------------ SiLU


def test_silu_textbook_values():
    # sigma(1), sigma(2) are textbook constants; SiLU(x) = x sigma(x) = x (1 + tanh(x/2)) / 2
    assert orc.silu(0.0) == 0.0
    assert orc.dsilu(0.0) == 0.5
    assert orc.silu(1.0) == pytest.approx(0.7310585786300049, rel=1e-15)
    assert orc.silu(-1.0) == pytest.approx(-0.2689414213699951, rel=1e-15)
    assert orc.silu(2.0) == pytest.approx(2 * 0.8807970779778823, rel=1e-15)
    # (1 + tanh) cancels for very negative arguments, so the identity is checked on a moderate range
    for v in (-6.0, -3.3, -0.1, 1e-9, 0.7, 5.0, 40.0):
        assert orc.silu(v) == pytest.approx(v * (1.0 + math.tanh(v / 2.0)) / 2.0, rel=1e-12, abs=1e-300)
    assert orc.silu(-30.0) == pytest.approx(-30.0 * math.exp(-30.0), rel=1e-12)  # sigma(-30) = e^-30 (1 - O(e^-30))


def test_silu_extremes_do_not_overflow():
    assert orc.silu(800.0) == 800.0
    assert orc.silu(-800.0) <= 0.0 and orc.silu(-800.0) > -1e-300
    assert orc.dsilu(800.0) == pytest.approx(1.0)
    assert abs(orc.dsilu(-800.0)) < 1e-300
    assert math.isfinite(orc.silu(1e308)) and math.isfinite(orc.dsilu(-1e308))


def test_dsilu_is_derivative_of_tanh_form():
    # derivative pinned by central differences of the independent tanh closed form
    f = lambda v: v * (1.0 + math.tanh(v / 2.0)) / 2.0
    for v in (-6.0, -1.2785, -0.5, 0.0, 0.3, 1.0, 4.0):
        h = 1e-5
        fd = (f(v + h) - f(v - h)) / (2 * h)
        assert orc.dsilu(v) == pytest.approx(fd, abs=1e-9)
    # SiLU's minimum is near -1.2785: derivative changes sign there
    assert orc.dsilu(-1.27) > 0 > orc.dsilu(-1.29)


# ------------------------------------------------------------------ selection


@pytest.mark.parametrize("F", [1, 2, 7, 33, 64])
def test_topk_brute_force_all_k(F):
    rng = np.random.default_rng(F)
    g = rng.standard_normal((5, F))
    # quantise so that duplicates occur and the tie rule matters
    gq = np.round(g * 4) / 4
    for arr in (g, gq):
        for K in range(1, F + 1):
            np.testing.assert_array_equal(orc.topk(arr, K), _np_topk_sets(arr, K))


def test_topk_adversarial_rows():
    F = 45  # not a multiple of 32
    rows = np.stack([
        np.zeros(F),                                     # all equal -> 0..K-1
        np.arange(F, dtype=float),                       # ascending -> last K
        -np.arange(F, dtype=float),                      # descending -> first K
        np.where(np.arange(F) % 3 == 0, 1.0, -1.0),      # two-valued
        np.where(np.arange(F) % 2 == 0, 0.0, -0.0),      # +-0 are equal
        np.concatenate([[np.inf, -np.inf], np.linspace(-1, 1, F - 2)]),
    ])
    for K in (1, 2, 15, F - 1, F):
        got = orc.topk(rows, K)
        np.testing.assert_array_equal(got, _np_topk_sets(rows, K))
        np.testing.assert_array_equal(got[0], np.arange(K))
        np.testing.assert_array_equal(got[1], np.arange(F - K, F))
        np.testing.assert_array_equal(got[2], np.arange(K))
        np.testing.assert_array_equal(got[4], np.arange(K))
    # signed, not absolute: a large negative value is never preferred to a small positive one
    r = np.array([[-100.0, 0.1, -0.2, 0.05]])
    np.testing.assert_array_equal(orc.topk(r, 2), [[1, 3]])


def test_topk_nan_is_lowest_and_padding_ignored():
    g = np.array([[0.5, np.nan, -3.0, np.nan, 0.1, 99.0, 98.0]])
    # only the first 5 columns are channels (F=5, ld=7): the large tail must not be picked
    np.testing.assert_array_equal(orc.topk(g, 3, F=5), [[0, 2, 4]])
    np.testing.assert_array_equal(orc.topk(g, 4, F=5), [[0, 1, 2, 4]])  # NaN ties -> lower index
    np.testing.assert_array_equal(orc.topk(g, 5, F=5), [[0, 1, 2, 3, 4]])


def test_topk_f32_path_matches_f64_on_same_values():
    rng = np.random.default_rng(3)
    g32 = rng.standard_normal((64, 300)).astype(np.float32)
    g32[:, ::7] = g32[:, 1::7][:, : g32[:, ::7].shape[1]]  # duplicates
    np.testing.assert_array_equal(orc.topk(g32, 37), _np_topk_sets(g32.astype(np.float64), 37))


def test_topk_invariants():
    rng = np.random.default_rng(11)
    F, K = 257, 40
    g = np.round(rng.standard_normal((32, F)) * 8) / 8
    idx = orc.topk(g, K)
    for t in range(g.shape[0]):
        row = idx[t]
        assert len(set(row.tolist())) == K and row.min() >= 0 and row.max() < F
        assert np.all(np.diff(row) > 0)
        sel = np.zeros(F, bool)
        sel[row] = True
        thr = g[t, sel].min()
        assert thr >= g[t, ~sel].max()
        # an unselected channel equal to the threshold must have a higher index than every selected equal one
        eq_unsel = np.where((~sel) & (g[t] == thr))[0]
        eq_sel = np.where(sel & (g[t] == thr))[0]
        if len(eq_unsel):
            assert eq_sel.max() < eq_unsel.min()


# ------------------------------------------------------------------ forward


def test_k_equals_dff_is_dense_swiglu():
    x, wg, wu, wd = _rand_problem(1, 9, 12, 20)
    dense = (_np_silu(x @ wg.T) * (x @ wu.T)) @ wd
    r = orc.forward(x, wg, wu, wd, K=20)
    np.testing.assert_allclose(r["out"], dense, rtol=1e-12, atol=1e-13)
    np.testing.assert_array_equal(r["idx"], np.tile(np.arange(20), (9, 1)))
    np.testing.assert_allclose(r["gval"], x @ wg.T, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(r["uval"], x @ wu.T, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("T,d,F,K", [(7, 5, 11, 3), (16, 24, 40, 1), (5, 8, 33, 32), (3, 16, 64, 8)])
def test_forward_matches_dense_masked_equations(T, d, F, K):
    x, wg, wu, wd = _rand_problem(T * 100 + K, T, d, F)
    f = _dense_masked_forward(x, wg, wu, wd, K)
    r = orc.forward(x, wg, wu, wd, K=K, want_g=True)
    np.testing.assert_array_equal(r["idx"], f["idx"])
    np.testing.assert_allclose(r["out"], f["D"], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(r["g"], f["G"], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(r["gval"], np.take_along_axis(f["G"], f["idx"].astype(np.int64), 1), rtol=1e-12)
    np.testing.assert_allclose(r["uval"], np.take_along_axis(f["U"], f["idx"].astype(np.int64), 1), rtol=1e-12,
                               atol=1e-13)
    # each mask row has exactly K ones
    assert np.all(f["M"].sum(axis=1) == K)


def test_forward_one_hot_input_hand_computed():
    # x = e_i  =>  g_j = Wg[j,i], u_j = Wu[j,i]; pick the two largest g by hand
    d, F = 4, 5
    wg = np.array([[0.1, 2.0, 0, 0], [0.2, -1.0, 0, 0], [0.3, 0.5, 0, 0], [0.4, 3.0, 0, 0], [0.5, 0.4, 0, 0]])
    wu = np.arange(F * d, dtype=float).reshape(F, d) / 10
    wd = np.ones((F, d)) * np.arange(1, F + 1)[:, None]
    x = np.zeros((1, d))
    x[0, 1] = 1.0
    r = orc.forward(x, wg, wu, wd, K=2)
    np.testing.assert_array_equal(r["idx"], [[0, 3]])  # g = [2,-1,.5,3,.4]
    z0 = 2.0 / (1 + math.exp(-2.0)) * wu[0, 1]
    z3 = 3.0 / (1 + math.exp(-3.0)) * wu[3, 1]
    np.testing.assert_allclose(r["out"][0], np.full(d, z0 * 1 + z3 * 4), rtol=1e-14)


def test_gate_projection_one_hot_rows_and_library_matmul():
    # x = e_i picks column i of every channel's weight row: G[t, j] = Wg[j, i] exactly; a padded tail is not projected
    d, F = 6, 9
    rng = np.random.default_rng(17)
    wg = rng.standard_normal((F + 3, d))
    x = np.eye(d)
    np.testing.assert_array_equal(orc.gate_projection(x, wg, F), wg[:F].T)
    # general rows against the library routine (numpy matmul), and against the dense g the full forward reports
    x, wg, wu, wd = _rand_problem(23, 7, 11, 20)
    g = orc.gate_projection(x, wg)
    assert g.shape == (7, 20)
    np.testing.assert_allclose(g, x @ wg.T, rtol=1e-13, atol=1e-14)
    np.testing.assert_array_equal(g, orc.forward(x, wg, wu, wd, K=5, want_g=True)["g"])
    with pytest.raises(ValueError):
        orc.gate_projection(x, wg[:, :5])


def test_forward_structure_token_independence_permutation_linearity():
    T, d, F, K = 12, 10, 30, 7
    x, wg, wu, wd = _rand_problem(5, T, d, F)
    full = orc.forward(x, wg, wu, wd, K=K)
    # token independence
    for t in (0, 5, 11):
        one = orc.forward(x[t:t + 1], wg, wu, wd, K=K)
        np.testing.assert_array_equal(one["out"][0], full["out"][t])
        np.testing.assert_array_equal(one["idx"][0], full["idx"][t])
    # channel permutation: same function (no ties in random data), indices map through the permutation
    perm = np.random.default_rng(0).permutation(F)
    p = orc.forward(x, wg[perm], wu[perm], wd[perm], K=K)
    np.testing.assert_allclose(p["out"], full["out"], rtol=1e-11, atol=1e-13)
    for t in range(T):
        assert set(perm[p["idx"][t]].tolist()) == set(full["idx"][t].tolist())
    # linear in W_down and in W_up (selection depends on W_gate only)
    a = orc.forward(x, wg, wu, 2.5 * wd, K=K)
    np.testing.assert_allclose(a["out"], 2.5 * full["out"], rtol=1e-12, atol=1e-13)
    b = orc.forward(x, wg, -3.0 * wu, wd, K=K)
    np.testing.assert_allclose(b["out"], -3.0 * full["out"], rtol=1e-12, atol=1e-13)
    np.testing.assert_array_equal(b["idx"], full["idx"])


def test_forward_given_idx_agrees_and_ignores_order():
    T, d, F, K = 6, 9, 21, 5
    x, wg, wu, wd = _rand_problem(8, T, d, F)
    full = orc.forward(x, wg, wu, wd, K=K)
    g = orc.forward_given_idx(x, wg, wu, wd, full["idx"])
    np.testing.assert_allclose(g["out"], full["out"], rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(g["gval"], full["gval"], rtol=1e-13)
    # forced (different) mask equals the dense-masked formula with that mask
    rng = np.random.default_rng(1)
    forced = np.stack([np.sort(rng.choice(F, K, replace=False)) for _ in range(T)]).astype(np.int32)
    M = np.zeros((T, F))
    np.put_along_axis(M, forced.astype(np.int64), 1.0, axis=1)
    D = ((_np_silu(x @ wg.T) * M) * (x @ wu.T)) @ wd
    np.testing.assert_allclose(orc.forward_given_idx(x, wg, wu, wd, forced)["out"], D, rtol=1e-12, atol=1e-13)


def test_padded_weights_equal_unpadded_problem():
    T, d, F, K, ld = 5, 8, 19, 6, 24
    x, wg, wu, wd = _rand_problem(21, T, d, F)
    pad = lambda w: np.concatenate([w, np.zeros((ld - F, d))])
    a = orc.forward(x, wg, wu, wd, K=K)
    b = orc.forward(x, pad(wg), pad(wu), pad(wd), K=K, F=F)
    np.testing.assert_array_equal(a["idx"], b["idx"])
    np.testing.assert_array_equal(a["out"], b["out"])


# ------------------------------------------------------------------ backward


@pytest.mark.parametrize("T,d,F,K", [(7, 5, 11, 3), (6, 12, 20, 20), (4, 16, 64, 9)])
def test_backward_matches_dense_masked_equations(T, d, F, K):
    x, wg, wu, wd = _rand_problem(T + F + K, T, d, F)
    dD = np.random.default_rng(9).standard_normal((T, d))
    f = _dense_masked_forward(x, wg, wu, wd, K)
    ref = _dense_masked_backward(x, wg, wu, wd, f, dD)
    r = orc.forward(x, wg, wu, wd, K=K)
    got = orc.backward(x, wg, wu, wd, r["idx"], r["gval"], r["uval"], dD)
    for k in ref:
        np.testing.assert_allclose(got[k], ref[k], rtol=1e-11, atol=1e-12, err_msg=k)


def test_backward_k_equals_dff_is_dense_swiglu_backward():
    T, d, F = 5, 7, 13
    x, wg, wu, wd = _rand_problem(2, T, d, F)
    dD = np.random.default_rng(4).standard_normal((T, d))
    G, U = x @ wg.T, x @ wu.T
    S = _np_silu(G)
    dZ = dD @ wd.T
    dG = dZ * U * _np_dsilu(G)
    dU = dZ * S
    r = orc.forward(x, wg, wu, wd, K=F)
    got = orc.backward(x, wg, wu, wd, r["idx"], r["gval"], r["uval"], dD)
    np.testing.assert_allclose(got["grad_w_down"], (S * U).T @ dD, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(got["grad_w_gate"], dG.T @ x, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(got["grad_w_up"], dU.T @ x, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(got["grad_x"], dG @ wg + dU @ wu, rtol=1e-11, atol=1e-12)


def test_backward_finite_differences_fixed_mask():
    """L = sum(out * R) with the mask held constant; central differences on every input."""
    T, d, F, K = 4, 6, 14, 5
    x, wg, wu, wd = _rand_problem(33, T, d, F)
    rng = np.random.default_rng(34)
    R = rng.standard_normal((T, d))
    r = orc.forward(x, wg, wu, wd, K=K)
    idx = r["idx"]
    got = orc.backward(x, wg, wu, wd, idx, r["gval"], r["uval"], R)

    def loss(x_, wg_, wu_, wd_):
        return float(np.sum(orc.forward_given_idx(x_, wg_, wu_, wd_, idx)["out"] * R))

    h = 1e-6
    args = [x, wg, wu, wd]
    names = ["grad_x", "grad_w_gate", "grad_w_up", "grad_w_down"]
    for a_i, name in enumerate(names):
        arr = args[a_i]
        fd = np.zeros_like(arr)
        for pos in np.ndindex(arr.shape):
            plus = [a.copy() for a in args]
            minus = [a.copy() for a in args]
            plus[a_i][pos] += h
            minus[a_i][pos] -= h
            fd[pos] = (loss(*plus) - loss(*minus)) / (2 * h)
        scale = np.abs(fd).max()
        np.testing.assert_allclose(got[name], fd, rtol=0, atol=1e-6 * scale + 1e-9, err_msg=name)


def test_backward_finite_differences_full_forward_with_margin():
    """With a clear Top-K margin the mask is locally constant, so FD of the full forward applies."""
    T, d, F, K = 3, 5, 12, 4
    x, wg, wu, wd = _rand_problem(71, T, d, F)
    r = orc.forward(x, wg, wu, wd, K=K, want_g=True)
    srt = -np.sort(-r["g"], axis=1)
    margin = (srt[:, K - 1] - srt[:, K]).min()
    h = 1e-6
    assert margin > 100 * h
    R = np.random.default_rng(72).standard_normal((T, d))
    got = orc.backward(x, wg, wu, wd, r["idx"], r["gval"], r["uval"], R)
    fd = np.zeros_like(x)
    for pos in np.ndindex(x.shape):
        xp, xm = x.copy(), x.copy()
        xp[pos] += h
        xm[pos] -= h
        fd[pos] = (np.sum(orc.forward(xp, wg, wu, wd, K=K)["out"] * R) -
                   np.sum(orc.forward(xm, wg, wu, wd, K=K)["out"] * R)) / (2 * h)
    np.testing.assert_allclose(got["grad_x"], fd, atol=1e-6 * np.abs(fd).max())


def test_backward_unselected_rows_are_exactly_zero_and_row_sampler_agrees():
    T, d, F, K = 6, 8, 40, 3
    x, wg, wu, wd = _rand_problem(55, T, d, F)
    dD = np.random.default_rng(56).standard_normal((T, d))
    r = orc.forward(x, wg, wu, wd, K=K)
    got = orc.backward(x, wg, wu, wd, r["idx"], r["gval"], r["uval"], dD)
    used = np.zeros(F, bool)
    used[r["idx"].ravel()] = True
    assert (~used).any()
    for name in ("grad_w_gate", "grad_w_up", "grad_w_down"):
        assert np.all(got[name][~used] == 0.0)
        assert np.all(np.abs(got[name][used]).sum(axis=1) > 0)
    rows = np.unique(np.array([0, 7, 39, int(r["idx"][0, 0])], dtype=np.int32))
    part = orc.backward_weight_rows(x, wd, r["idx"], r["gval"], r["uval"], dD, rows, F)
    for name in ("grad_w_gate", "grad_w_up", "grad_w_down"):
        np.testing.assert_allclose(part[name], got[name][rows], rtol=1e-13, atol=1e-15)


def test_backward_skips_null_outputs():
    T, d, F, K = 3, 4, 9, 2
    x, wg, wu, wd = _rand_problem(5, T, d, F)
    dD = np.ones((T, d))
    r = orc.forward(x, wg, wu, wd, K=K)
    full = orc.backward(x, wg, wu, wd, r["idx"], r["gval"], r["uval"], dD)
    part = orc.backward(x, wg, wu, wd, r["idx"], r["gval"], r["uval"], dD, want=("w_up",))
    assert part["grad_x"] is None and part["grad_w_down"] is None
    np.testing.assert_array_equal(part["grad_w_up"], full["grad_w_up"])


# ------------------------------------------------------------------ counting formulas (paper's printed figures)


def _golden():
    vals = {}
    with open(GOLDEN) as fh:
        for line in fh:
            line = line.split("#")[0].split()
            if len(line) == 2:
                vals[line[0]] = float(line[1])
    return vals


def test_counts_reproduce_table_1_and_section_5():
    gold = _golden()
    d = 3000
    F = 8 * d // 3
    K = int(round(gold["kept_fraction"] * F))
    assert orc.saved_elems("ffn", d, F) / d == pytest.approx(gold["ffn_over_bsd"], abs=5e-3)
    assert orc.saved_elems("ffn_gcp", d, F) / d == pytest.approx(gold["ffn_gcp_over_bsd"], abs=5e-3)
    assert orc.saved_elems("moc", d, K) / d == pytest.approx(gold["moc_over_bsd"], abs=5e-3)
    assert orc.saved_elems("moc_gcp", d, K) / d == pytest.approx(gold["moc_gcp_over_bsd"], abs=5e-3)
    assert orc.saved_elems("ffn", d, F) == gold["ffn_elems_coeff_dffn"] * F + d
    assert orc.macs_dense(d, F) == gold["dense_macs_coeff"] * d * F
    assert orc.macs_moc(d, F, K) == gold["moc_macs_gate_coeff"] * d * F + gold["moc_macs_topk_coeff"] * K * d
    # the compact form kept for backward is 3K elements per token (plus the output D)
    assert orc.saved_elems("moc_gcp", 0, K) == 3 * K


def test_bad_arguments_are_rejected():
    x, wg, wu, wd = _rand_problem(1, 2, 3, 4)
    with pytest.raises(RuntimeError):
        orc.forward(x, wg, wu, wd, K=5)
    with pytest.raises(RuntimeError):
        orc.forward_given_idx(x, wg, wu, wd, np.array([[0, 4], [1, 2]], dtype=np.int32))


# ------------------------------------------------------------------ grouped selection (MoC 2:8, Section 4; Theorem 1)


def _np_grouped_sets(g, group, keep):
    """Brute force by counting: a channel is kept when fewer than `keep` channels of its group precede it in
    (value descending, channel ascending) order.  No sort involved."""
    g = np.where(np.isnan(g), -np.inf, g) + 0.0
    rows, F = g.shape
    out = []
    for t in range(rows):
        kept = []
        for q in range(F // group):
            for e in range(group):
                j = q * group + e
                before = sum(1 for f in range(group)
                             if g[t, q * group + f] > g[t, j] or (g[t, q * group + f] == g[t, j] and f < e))
                if before < keep:
                    kept.append(j)
        out.append(kept)
    return np.asarray(out, dtype=np.int32)


@pytest.mark.parametrize("group,keep", [(8, 2), (4, 1), (8, 8), (2, 1)])
def test_grouped_selection_brute_force(group, keep):
    rng = np.random.default_rng(group * 10 + keep)
    g = rng.standard_normal((7, 8 * group))
    g[1, :] = 0.5                                   # all equal: the first `keep` channels of every group
    g[2, ::2] = g[2, 1::2]                          # pairs of equal values
    g[3, 3] = np.nan
    g[3, 4] = np.inf
    g[4, :group] = [-0.0, 0.0] * (group // 2) if group % 2 == 0 else 0.0
    g[5] = np.round(g[5] * 2) / 2                   # many ties
    got = orc.topk_grouped(g, group, keep)
    assert np.array_equal(got, _np_grouped_sets(g, group, keep))
    assert np.array_equal(got[1], np.concatenate([np.arange(q * group, q * group + keep) for q in range(8)]))
    # exactly `keep` per group, ascending
    assert np.all(np.diff(got, axis=1) > 0)
    assert np.all((got // group) == np.repeat(np.arange(8), keep)[None, :])


def test_grouped_selection_with_one_group_is_the_global_rule():
    rng = np.random.default_rng(5)
    g = rng.standard_normal((9, 24))
    g[0, 5] = g[0, 17]
    assert np.array_equal(orc.topk_grouped(g, group=24, keep=7), orc.topk(g, 7))
    assert np.array_equal(orc.topk_grouped(g, group=24, keep=7), _np_topk_sets(g, 7))


def test_grouped_forward_keep_all_is_dense_swiglu_and_matches_dense_masked_form():
    x, wg, wu, wd = _rand_problem(21, T=6, d=10, F=32)
    full = orc.forward_grouped(x, wg, wu, wd, group=8, keep=8)
    dense = (_np_silu(x @ wg.T) * (x @ wu.T)) @ wd
    np.testing.assert_allclose(full["out"], dense, rtol=1e-12, atol=1e-13)
    # 2 of 8: Eqs. (Moc-1), mask, (MoC-2) written as dense matrices with the grouped mask
    res = orc.forward_grouped(x, wg, wu, wd, group=8, keep=2)
    G, U = x @ wg.T, x @ wu.T
    M = np.zeros_like(G)
    np.put_along_axis(M, _np_grouped_sets(G, 8, 2).astype(np.int64), 1.0, axis=1)
    np.testing.assert_allclose(res["out"], (_np_silu(G) * M * U) @ wd, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(res["gval"], np.take_along_axis(G, res["idx"].astype(np.int64), axis=1), rtol=1e-13)


def test_theorem_1_embedding_dense_ffn_into_2_of_8():
    """Theorem 1 with a:b = 2:8: a dense SwiGLU FFN of width d_ffn is reproduced exactly by MoC 2:8 of width
    8 * ceil(d_ffn / 2) whose groups hold two real channels and six zero channels.  With the input-based key the
    zero channels must not beat the real ones, so the inputs are chosen with all real gate values positive."""
    rng = np.random.default_rng(8)
    d, d_ffn = 6, 7
    x = rng.uniform(0.1, 1.0, (5, d))
    wg = rng.uniform(0.05, 0.5, (d_ffn, d))          # x, wg > 0: every real gate value exceeds the padded channels' 0
    wu = rng.standard_normal((d_ffn, d))
    wd = rng.standard_normal((d_ffn, d))
    groups = -(-d_ffn // 2)
    wg2, wu2, wd2 = (np.zeros((8 * groups, d)) for _ in range(3))
    for j in range(d_ffn):
        q, r = divmod(j, 2)
        wg2[q * 8 + r], wu2[q * 8 + r], wd2[q * 8 + r] = wg[j], wu[j], wd[j]
    dense = (_np_silu(x @ wg.T) * (x @ wu.T)) @ wd
    moc = orc.forward_grouped(x, wg2, wu2, wd2, group=8, keep=2)
    np.testing.assert_allclose(moc["out"], dense, rtol=1e-12, atol=1e-13)
    # a group whose second real slot is padding keeps a zero channel, which contributes nothing
    assert moc["idx"].shape == (5, 2 * groups)


# --------------------------------------------------------------------------- the block around the layer (Section 2)

def test_rmsnorm_worked_example_and_closed_forms():
    """Section 2, item "RMSNorm": y = x / sqrt(mean(x^2) + eps) . g."""
    # x = (3, 4): mean square 12.5, RMS 3.5355339059..., so y = (0.848528137.., 1.131370849..) before the weight
    y = orc.rmsnorm(np.array([[3.0, 4.0]]), np.array([1.0, 2.0]), 0.0)
    np.testing.assert_allclose(y, [[0.8485281374238570, 2.2627416997969520]], rtol=1e-15)
    # eps enters under the root: x = (1, 1, 1, 1), eps = 3 gives RMS 2
    y = orc.rmsnorm(np.ones((1, 4)), np.array([1.0, -2.0, 4.0, 0.5]), 3.0)
    np.testing.assert_allclose(y, [[0.5, -1.0, 2.0, 0.25]], rtol=1e-15)
    # a zero row stays zero (eps keeps the division finite)
    assert np.all(orc.rmsnorm(np.zeros((2, 8)), np.ones(8), 1e-6) == 0.0)
    rng = np.random.default_rng(21)
    x = rng.standard_normal((7, 96)) * rng.uniform(0.01, 100.0, (7, 1))
    g = rng.standard_normal(96)
    # unit weight, eps = 0: every row has mean square exactly 1; rows are invariant to their scale
    y1 = orc.rmsnorm(x, np.ones(96), 0.0)
    np.testing.assert_allclose((y1 * y1).mean(axis=1), 1.0, rtol=1e-13)
    np.testing.assert_allclose(orc.rmsnorm(-3.5 * x, np.ones(96), 0.0), -y1, rtol=1e-13)
    # the weight multiplies element by element
    np.testing.assert_allclose(orc.rmsnorm(x, g, 0.0), y1 * g, rtol=1e-13)


def test_rmsnorm_matches_the_library_routine():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(22)
    x = rng.standard_normal((5, 160))
    g = rng.standard_normal(160)
    for eps in (0.0, 1e-6, 0.3):
        ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (160,), torch.from_numpy(g), eps).numpy()
        np.testing.assert_allclose(orc.rmsnorm(x, g, eps), ref, rtol=1e-13, atol=1e-15)


def test_residual_and_block_composition():
    """Section 2, item "Residual connections" (Z = X + Y) and "LLM structure": out = h + FFN(RMSNorm(h))."""
    np.testing.assert_array_equal(orc.residual(np.array([[1.0, -2.0], [0.5, 4.0]]), np.array([[10.0, 20.0], [30.0, 40.0]])),
                                  [[11.0, 18.0], [30.5, 44.0]])
    rng = np.random.default_rng(23)
    T, d, F, K = 4, 24, 40, 7
    h = rng.standard_normal((T, d)) * 3.0
    g = rng.uniform(0.5, 1.5, d)
    wg, wu, wd = (rng.standard_normal((F, d)) * 0.2 for _ in range(3))
    # a zero down projection leaves the residual stream untouched
    out, x, _ = orc.decode_block(h, g, 1e-5, wg, wu, np.zeros_like(wd), K)
    np.testing.assert_array_equal(out, h)
    # the layer sees the normalised rows: unit-ish mean square whatever the scale of h
    np.testing.assert_allclose(((x / g) ** 2).mean(axis=1), 1.0, rtol=1e-4)
    # scaling h by a positive constant changes only the residual term (eps = 0: the norm removes the scale)
    out1, _, f1 = orc.decode_block(h, g, 0.0, wg, wu, wd, K)
    out2, _, f2 = orc.decode_block(7.0 * h, g, 0.0, wg, wu, wd, K)
    np.testing.assert_array_equal(f1["idx"], f2["idx"])
    np.testing.assert_allclose(out2 - 7.0 * h, out1 - h, rtol=1e-10, atol=1e-12)
    # `store` is applied to what the layer reads: a coarse rounding changes the layer's input and nothing else
    coarse = lambda a: np.round(a * 8.0) / 8.0
    out3, x3, f3 = orc.decode_block(h, g, 1e-5, wg, wu, wd, K, store=coarse)
    np.testing.assert_array_equal(x3, coarse(orc.rmsnorm(h, g, 1e-5)))
    np.testing.assert_allclose(out3, h + orc.forward(x3, wg, wu, wd, K)["out"], rtol=1e-13, atol=1e-14)


# --------------------------------------------------------------------------- Top-K after the activation (Section 6.5)

def test_post_silu_selection_equals_pre_silu_when_enough_gates_are_positive():
    """SiLU is increasing and positive on g > 0 and negative on g < 0, so with at least K positive gate values the
    K largest SiLU(g) are the K largest g."""
    rng = np.random.default_rng(31)
    T, d, F, K = 6, 16, 48, 9
    x = rng.standard_normal((T, d))
    wg, wu, wd = (rng.standard_normal((F, d)) * 0.3 for _ in range(3))
    G = x @ wg.T
    assert (G > 0).sum(axis=1).min() >= K
    post, pre = orc.forward_post_silu(x, wg, wu, wd, K), orc.forward(x, wg, wu, wd, K)
    np.testing.assert_array_equal(post["idx"], pre["idx"])
    np.testing.assert_allclose(post["out"], pre["out"], rtol=1e-13, atol=1e-14)
    # the keys are SiLU of the gate values the oracle itself formed (sequential dot products; numpy's matmul sums in
    # another order, which shows as ~1e-17 absolute on values that cancel to nearly zero)
    np.testing.assert_allclose(post["g"], G, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(post["s"], post["g"] * expit(post["g"]), rtol=1e-13, atol=1e-300)


def test_post_silu_selection_differs_where_it_must():
    """One token, hand-made gate values through an identity gate matrix.  Only two are positive; with K = 4 the other
    two picks are the negative values whose SiLU is closest to zero: g = -0.01 (SiLU -0.00497..) and g = -12
    (SiLU -7.4e-5), not g = -0.5 (-0.189) or g = -1.3 (-0.279), while the pre-SiLU rule takes -0.01 and -0.5."""
    g = np.array([[2.0, -0.5, -12.0, 0.3, -1.3, -0.01, -3.0, -0.8]])
    F = g.shape[1]
    eye = np.eye(F)
    wu, wd = np.ones((F, F)), np.eye(F)
    post = orc.forward_post_silu(g, eye, wu, wd, 4)
    pre = orc.forward(g, eye, wu, wd, 4)
    np.testing.assert_array_equal(post["idx"], [[0, 2, 3, 5]])
    np.testing.assert_array_equal(pre["idx"], [[0, 1, 3, 5]])
    # brute force over all subsets of size 4: the kept set maximises the sum of SiLU(g)
    import itertools
    s = g[0] * expit(g[0])
    best = max(itertools.combinations(range(F), 4), key=lambda c: s[list(c)].sum())
    assert list(best) == post["idx"][0].tolist()
    # the output is Eq. (MoC-2) on that mask: u = sum(g) for every channel, W_down = I
    expect = np.zeros(F)
    expect[list(best)] = s[list(best)] * g.sum()
    np.testing.assert_allclose(post["out"][0], expect, rtol=1e-13, atol=1e-15)
    # equal keys: the lower channel (two channels with the same gate value on the threshold)
    tie = orc.forward_post_silu(np.array([[1.0, -2.0, -2.0, -0.1]]), np.eye(4), np.ones((4, 4)), np.eye(4), 3)
    np.testing.assert_array_equal(tie["idx"], [[0, 1, 3]])
