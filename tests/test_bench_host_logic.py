"""Host-side logic of bench.py that the multi-GPU launch relies on, exercised with two gloo ranks on CPU."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402


def test_shard_plan_and_aggregate_single_process():
    assert bench.shard_plan(1, 0, 16384) == (0, 16384)
    assert bench.shard_plan(4, 3, 100) == (300, 100)
    with pytest.raises(ValueError):
        bench.shard_plan(2, 2, 8)
    value, ms = bench.aggregate([100.0, 125.0], [16384, 16384], steps=10)
    assert ms == pytest.approx(12.5)
    assert value == pytest.approx(2 * 16384 * 10 / 0.125)


def test_kernel_work_table_matches_per_token_formulas():
    T, d, F, K, e = 16384, 768, 2048, 256, 2
    assert bench.kernel_work("gate_gemm_alu", T, d, F, K, e)[:2] == ("tensor", 2.0 * T * d * F)
    assert bench.kernel_work("select_rows", T, d, F, K, e)[1] == T * F * 4 + T * K * 4
    # gathered plan: forward + backward sparse work adds up to the 16 T K d of the operator
    total = sum(bench.kernel_work(k, T, d, F, K, e)[1] for k in ("forward_token", "backward_token", "wgrad_rows"))
    assert total == 16.0 * T * K * d
    # tensor-core plan: algorithmic flops = gate 2TdF + 16TKd; executed flops = 18TdF (every contraction dense)
    gemms = ("tc_gate_up_gemm", "tc_down_gemm", "tc_dz_gemm", "tc_wgrad_gemm", "tc_dx_gemm")
    assert sum(bench.kernel_work(k, T, d, F, K, e)[1] for k in gemms) == 2.0 * T * d * F + 16.0 * T * K * d
    assert sum(bench.kernel_work(k, T, d, F, K, e)[2] for k in gemms) == 18.0 * T * d * F
    for k in gemms:
        bound, algo, executed, unit = bench.kernel_work(k, T, d, F, K, e)
        assert bound == "tensor" and unit == "flop" and executed >= algo
    assert bench.kernel_work("nonexistent", T, d, F, K, e) is None


def test_roofline_report_picks_the_largest_kernel_and_fills_every_key():
    from paper_2511_09323_b200 import synthetic as syn
    w, steps = syn.C2, 4
    peaks = {"hbm_gbs": 6550.7, "bf16_tflops": 1647.5, "bf16_tflops_sustained": 1388.1, "source": "measured"}
    prof = {"tc_wgrad_gemm": (steps, 0.48), "tc_select_mask": (steps, 0.36), "_hidden": (1, 9.0)}
    at_max = {"sm_mhz": 1965.0, "sm_max_mhz": 1965.0, "reasons": []}
    roof, kernels = bench.roofline_report(prof, steps, w.tokens, w, 2, peaks, at_max)
    assert roof["kernel"] == "tc_wgrad_gemm" and set(kernels) == {"tc_wgrad_gemm", "tc_select_mask"}
    # the SM clock sat at its maximum while the kernels were timed: the burst figure is the denominator
    assert roof["bound"] == "tensor" and roof["peak"] == 1647.5 and roof["unit"] == "TFLOP/s"
    assert "burst" in roof["peak_source"]
    assert roof["frac"] == pytest.approx(roof["achieved"] / roof["peak"])
    assert roof["achieved"] == pytest.approx(6.0 * w.tokens * w.k * w.d_model / 0.12e-3 / 1e12)
    assert roof["avg_ms_x_sm_mhz"] == pytest.approx(0.12 * 1965.0)
    assert roof["traffic"] == bench.NCU_DRAM_BYTES_C2["tc_wgrad_gemm"]          # that workload: measured bytes
    roof2, _ = bench.roofline_report(prof, steps, 1024, w, 2, peaks, at_max)    # any other size: no measurement
    assert roof2["traffic"] is None
    assert kernels["tc_select_mask"]["share"] == pytest.approx(0.36 / 0.84, abs=1e-3)
    # a clock that sagged under the power cap: the sustained figure
    sagged = {"sm_mhz": 1400.0, "sm_max_mhz": 1965.0, "reasons": ["sw_power_cap"]}
    roof3, _ = bench.roofline_report(prof, steps, w.tokens, w, 2, peaks, sagged)
    assert roof3["peak"] == 1388.1 and "sustained" in roof3["peak_source"]
    assert bench.choose_tensor_peak(peaks, {}) == (1647.5, "burst")


def test_measured_traffic_is_linear_in_tokens_where_two_captures_exist(monkeypatch):
    from paper_2511_09323_b200 import synthetic as syn
    monkeypatch.setitem(bench.NCU_DRAM_BYTES, ("C5", "tc_wgrad_gemm"), (100.0, 3.0))
    got, src = bench.measured_traffic(syn.C5, 1000, "tc_wgrad_gemm", 4, 4)
    assert got == 100.0 + 3.0 * 1000 and "linear" in src
    assert bench.measured_traffic(syn.C5, 1000, "tc_wgrad_gemm", 8, 4)[0] is None     # several launches per step
    assert bench.measured_traffic(syn.C2, 1000, "tc_wgrad_gemm", 4, 4)[0] is None     # another shape at another size
    assert bench.measured_traffic(syn.C5, 1000, "tc_dz_gemm", 4, 4)[0] is None        # a kernel without a capture


def test_strict_roofline_matches_the_hand_computed_figures():
    from paper_2511_09323_b200 import synthetic as syn
    peaks = {"hbm_gbs": 6550.7, "bf16_tflops": 1647.5, "bf16_tflops_sustained": 1388.1, "source": "measured"}
    w = syn.C5
    r = bench.strict_roofline(w, w.tokens, 2, 10.0, peaks, {"sm_mhz": 1965.0, "sm_max_mhz": 1965.0})
    gate = 2.0 * 65536 * 2048 * 5504
    assert r["r_gate_ms"] == pytest.approx(gate / 1647.5e12 * 1e3)            # 0.897 ms
    assert r["r_gate_ms"] == pytest.approx(0.897, abs=2e-3)
    assert r["r_bytes_ms"] == pytest.approx(0.319, abs=5e-3)
    assert r["strict_frac"] == pytest.approx(r["r_gate_ms"] / 10.0)
    assert r["dense_equiv_tflops"] == pytest.approx(9 * gate / 10e-3 / 1e12)


# ---- two gloo ranks run the functions the NCCL ranks run -------------------------------------------------------------
# Each rank owns one shard of a seeded batch (the shard seeds of the input module), computes the oracle's weight
# gradients of its shard, and the job's exchange -- bench.allreduce_weight_grads on the flat [3, F, d] buffer -- must
# give the oracle's weight gradients of the whole batch; timings go through bench.max_over_ranks / job_throughput.

_SHARD_W = dict(dtype="f32", d=24, F=40, K=7, tokens_per_rank=9)


def _shard_problem(rank):
    from oracle import moc_oracle as orc
    from paper_2511_09323_b200 import synthetic as syn
    p = _SHARD_W
    w = syn.Workload("shard-test", p["dtype"], p["tokens_per_rank"], p["d"], p["F"], p["F"], p["K"], seed=77)
    wg, wu, wd = (syn.to_f64(t) for t in syn.make_weights(w))
    x = syn.to_f64(syn.make_x(w, shard=rank))
    dD = syn.to_f64(syn.make_grad_out(w, shard=rank))
    f = orc.forward(x, wg, wu, wd, w.k)
    g = orc.backward(x, wg, wu, wd, f["idx"], f["gval"], f["uval"], dD)
    return w, (wg, wu, wd), x, dD, f, g


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist, world_seen, rank_seen = bench.init_distributed("gloo")
    try:
        assert (world_seen, rank_seen) == (world, rank)
        off, n = bench.shard_plan(world, rank, _SHARD_W["tokens_per_rank"])
        w, _, x, dD, f, g = _shard_problem(rank)
        like = torch.empty((w.d_ff_ld, w.d_model), dtype=torch.float64)
        flat, views = bench.flat_weight_grads(torch, like)
        for name in ("grad_w_gate", "grad_w_up", "grad_w_down"):
            views[name].copy_(torch.from_numpy(g[name]))
        sent = bench.allreduce_weight_grads(dist, flat)
        worst = bench.max_over_ranks(dist, [10.0 + 5.0 * rank, 20.0 + rank])
        dist.barrier()
        q.put((rank, off, n, worst, sent, flat.numpy().copy(), bench.job_throughput(world, n, 2, worst[0])))
    finally:
        dist.destroy_process_group()


def test_two_rank_gloo_job_sums_weight_gradients_and_takes_the_slowest_rank():
    import numpy as np
    from oracle import moc_oracle as orc
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted((q.get(timeout=180) for _ in procs), key=lambda r: r[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    n = _SHARD_W["tokens_per_rank"]
    assert [(r[1], r[2]) for r in res] == [(0, n), (n, n)]     # disjoint, contiguous token ranges
    assert all(r[3] == [15.0, 21.0] for r in res)              # every rank sees the slowest rank's times
    assert all(r[4] == 3 * _SHARD_W["F"] * _SHARD_W["d"] * 8 for r in res)   # bytes one rank contributes
    assert all(r[6] == pytest.approx(2 * n * 2 / 0.015) for r in res)
    # the whole batch = the shards one after the other; the mask is per token, so shards add (Eqs. (bp-1), (bp-4))
    parts = [_shard_problem(r) for r in range(2)]
    wg, wu, wd = parts[0][1]
    x = np.concatenate([p[2] for p in parts])
    dD = np.concatenate([p[3] for p in parts])
    assert not np.array_equal(parts[0][2], parts[1][2])        # the shards are different tokens
    f = orc.forward(x, wg, wu, wd, _SHARD_W["K"])
    np.testing.assert_array_equal(f["idx"], np.concatenate([p[4]["idx"] for p in parts]))
    whole = orc.backward(x, wg, wu, wd, f["idx"], f["gval"], f["uval"], dD)
    for r in res:
        for i, name in enumerate(("grad_w_gate", "grad_w_up", "grad_w_down")):
            np.testing.assert_allclose(r[5][i], whole[name], rtol=1e-12, atol=1e-13)
    # grad_x stays local: a shard's rows are the whole batch's rows
    np.testing.assert_allclose(np.concatenate([p[5]["grad_x"] for p in parts]), whole["grad_x"], rtol=1e-12, atol=1e-14)


def test_single_process_helpers_need_no_process_group(monkeypatch):
    monkeypatch.setenv("WORLD_SIZE", "1")
    assert bench.init_distributed("gloo") == (None, 1, 0)
    assert bench.max_over_ranks(None, [3.0, 4.0]) == [3.0, 4.0]
    flat, views = bench.flat_weight_grads(torch, torch.empty((6, 4)))
    assert flat.shape == (3, 6, 4) and views["grad_w_down"].data_ptr() == flat[2].data_ptr()
    assert all(v.is_contiguous() for v in views.values())
    assert bench.allreduce_weight_grads(None, flat) == 3 * 6 * 4 * 4
