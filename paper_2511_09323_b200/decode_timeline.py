"""Device-clock timeline of one moc_ffn_decode call on the LLaMA-7B shape (development aid).

The timeline needs a library built with the stamps compiled in (without them the script still runs the calls: a small
target for a profiler):

    MOC_FFN_NVCC_FLAGS=-DMOC_TIMELINE python -m paper_2511_09323_b200.build --force
    python -m paper_2511_09323_b200.decode_timeline 16            # (a second argument `grouped`: the MoC 2:8 mask)
    python -m paper_2511_09323_b200.build --force          # back to the normal build

Eight calls rotating four weight sets are replayed from one CUDA graph; every CTA of the small-batch kernels notes the
GPU's nanosecond timer at a few points (the last call's stamps survive).  Printed: minimum / median / maximum over the
CTAs of a kernel, relative to the moment the previous call had completed.
"""
import ctypes
import sys

import numpy as np
import torch

from . import binding as B
from . import synthetic as syn

REGIONS = [(256, "gate start"), (512, "gate mma done"), (768, "gate end"), (1024, "select after wait"),
           (1280, "select end"), (1536, "up start"), (1792, "up mma done"), (2048, "up end"), (2304, "down start"),
           (2560, "down after wait"), (2816, "down mma done"), (3072, "down end")]
# the one-kernel form (streamer CTAs, then the selector CTAs, in one grid)
REGIONS_FUSED = [(256, "start"), (512, "after grid barrier"), (768, "gate mma done"), (1024, "gate values stored"),
                 (1280, "select: row wait over"), (3072, "select: row staged"), (3328, "select: threshold found"),
                 (3840, "select: bitmap signalled"), (1536, "select end"), (1792, "up mma done"), (2048, "Z' stored"),
                 (2304, "down: Z' complete"), (2560, "down mma done"), (2816, "end")]
# the one-kernel decode form for one or two tokens
REGIONS_COOP = [(256, "start"), (512, "x staged, arrays cleared"), (768, "gate rows done, barrier 0"), (1024, "histogram complete (barrier 1)"),
                (1280, "candidate lists complete (barrier 2)"), (1536, "kept channels ranked"), (1792, "rows of W_up, W_down done"),
                (2048, "barrier 3"), (2304, "end")]


def main():
    T = int(sys.argv[1]) if len(sys.argv) > 1 else 16
    grouped = len(sys.argv) > 2 and sys.argv[2] == "grouped"   # the MoC 2:8 mask (K = d_ff / 4)
    lib = B.load()
    stamps = hasattr(lib, "moc_debug_timeline")
    w = syn.C4
    sets = [tuple(t.cuda() for t in syn.make_weights(w, seed_offset=s)) for s in range(4)]
    x = syn.make_x(w, tokens=T).cuda()
    out = torch.empty_like(x)
    k = None if grouped else w.k
    desc = B.make_desc(T, w.d_model, w.d_ff, w.d_ff // 4 if grouped else w.k, x.dtype,
                       flags=B.MOC_FLAG_SELECT_2_OF_8 if grouped else 0)
    ws = B.alloc_workspace(desc, B.MOC_OP_DECODE)
    stream = torch.cuda.Stream()
    for i in range(4):
        B.moc_ffn_decode(x, *sets[i % 4], k, out=out, workspace=ws, grouped=grouped)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            for i in range(8):
                B.moc_ffn_decode(x, *sets[i % 4], k, out=out, workspace=ws, stream=stream, grouped=grouped)
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    if B.moc_last_device_status() != B.MOC_OK:
        raise SystemExit("device status raised")
    if not stamps:   # (still a small, self-contained run of the decode call: a target for a profiler)
        print("this build has no stamps: rebuild with MOC_FFN_NVCC_FLAGS=-DMOC_TIMELINE to see the timeline")
        return
    buf = (ctypes.c_ulonglong * 4096)()
    lib.moc_debug_timeline.argtypes = [ctypes.c_void_p, ctypes.c_int]
    if lib.moc_debug_timeline(buf, 4096) != 0:
        raise SystemExit("reading the stamps failed")
    a = np.array(buf, dtype=np.uint64).astype(np.int64)
    ref = a[3] if a[3] else min(v for v in a[256:512] if v > 0)   # the first kernel's wait for the previous call returned
    if a[4095]:
        starts = np.sort(a[3584:3648][a[3584:3648] > 0])
        print("one-kernel form: us between the starts of successive calls:", np.round(np.diff(starts[-8:]) / 1000.0, 2))
    print(f"T = {T}: us after the previous call completed -- min / median / max over CTAs (n)")
    for base, name in (REGIONS if a[3] else REGIONS_COOP if T <= 2 else REGIONS_FUSED):
        v = a[base:base + 256]
        v = v[v > 0]
        if len(v):
            r = (v - ref) / 1000.0
            print(f"{name:38s} {r.min():8.2f} {np.median(r):8.2f} {r.max():8.2f}   ({len(v)})")


if __name__ == "__main__":
    main()
