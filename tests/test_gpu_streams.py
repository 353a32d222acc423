"""Calls from several host threads on different streams with separate buffers (what the header allows) give the same
results as the same calls made one after the other."""
import threading

import pytest
import torch

from paper_2511_09323_b200 import binding as B
from paper_2511_09323_b200 import build as moc_build
from paper_2511_09323_b200 import synthetic as syn

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    moc_build.build()
    B.load()
    yield
    assert B.moc_last_device_status() == B.MOC_OK


def _job(w, seed_shift):
    wk = syn.Workload(w.name, w.dtype, w.tokens, w.d_model, w.d_ff, w.d_ff_ld, w.k, seed=w.seed + seed_shift)
    wg, wu, wd = (t.cuda() for t in syn.make_weights(wk))
    return dict(w=wk, x=syn.make_x(wk).cuda(), dD=syn.make_grad_out(wk).cuda(), wg=wg, wu=wu, wd=wd)


def _run(job, stream, rounds):
    w = job["w"]
    with torch.cuda.stream(stream):
        for _ in range(rounds):
            out, idx, tg, tu = B.moc_ffn_forward(job["x"], job["wg"], job["wu"], job["wd"], w.k, stream=stream)
            grads = B.moc_ffn_backward(job["x"], job["wg"], job["wu"], job["wd"], idx, tg, tu, job["dD"], stream=stream)
            dec = B.moc_ffn_decode(job["x"][:3], job["wg"], job["wu"], job["wd"], w.k, stream=stream)
        stream.synchronize()
    return dict(out=out, idx=idx, tg=tg, tu=tu, dec=dec, **grads)


@pytest.mark.parametrize("T,exact", [(320, True), (40, False)])   # tensor-core plan (deterministic); small-batch plan
def test_two_threads_two_streams(T, exact):
    base = syn.Workload("streams", "bf16", T, 256, 1024, 1024, 128, seed=6100 + T)
    jobs = [_job(base, 0), _job(base, 1)]
    ref = [_run(j, torch.cuda.current_stream(), 1) for j in jobs]
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream() for _ in jobs]
    got = [None, None]
    errs = []

    def work(i):
        try:
            got[i] = _run(jobs[i], streams[i], 20)
        except Exception as exc:  # surfaces in the main thread below
            errs.append(exc)

    threads = [threading.Thread(target=work, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errs, errs
    torch.cuda.synchronize()
    for r, g in zip(ref, got):
        assert torch.equal(r["idx"], g["idx"])
        for k in ("out", "tg", "tu", "grad_x", "grad_w_gate", "grad_w_up", "grad_w_down", "dec"):
            if exact and k != "dec":
                assert torch.equal(r[k], g[k]), k
            else:   # partial sums of the down projection meet in an order that is not fixed: the last bit may differ
                torch.testing.assert_close(r[k].float(), g[k].float(), rtol=2e-2, atol=2e-4, msg=k)
