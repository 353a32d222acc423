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
    roof, kernels = bench.roofline_report(prof, steps, w.tokens, w, 2, peaks)
    assert roof["kernel"] == "tc_wgrad_gemm" and set(kernels) == {"tc_wgrad_gemm", "tc_select_mask"}
    assert roof["bound"] == "tensor" and roof["peak"] == 1388.1 and roof["unit"] == "TFLOP/s"
    assert roof["frac"] == pytest.approx(roof["achieved"] / roof["peak"])
    assert roof["achieved"] == pytest.approx(6.0 * w.tokens * w.k * w.d_model / 0.12e-3 / 1e12)
    assert roof["traffic"] == bench.NCU_DRAM_BYTES_C2["tc_wgrad_gemm"]          # default workload: measured bytes
    roof2, _ = bench.roofline_report(prof, steps, 1024, w, 2, peaks)            # any other size: no measurement
    assert roof2["traffic"] is None
    assert kernels["tc_select_mask"]["share"] == pytest.approx(0.36 / 0.84, abs=1e-3)


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        off, n = bench.shard_plan(world, rank, 1000)
        # each rank "times" its shard; the job time is the slowest rank's (MAX all-reduce), tokens add up
        t = torch.tensor([10.0 + 5.0 * rank, 20.0 + rank], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        tok = torch.tensor([n], dtype=torch.int64)
        dist.all_reduce(tok, op=dist.ReduceOp.SUM)
        dist.barrier()
        q.put((rank, off, n, t.tolist(), int(tok.item())))
    finally:
        dist.destroy_process_group()


def test_two_rank_gloo_sharding_and_max_over_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [0, 1000]               # disjoint token offsets
    assert all(r[3] == [15.0, 21.0] for r in res)          # every rank sees the slowest rank's times
    assert all(r[4] == 2000 for r in res)                  # whole-job tokens
    value, _ = bench.aggregate([res[0][3][0]] * 2, [1000, 1000], steps=1)
    assert value == pytest.approx(2000 / 0.015)
