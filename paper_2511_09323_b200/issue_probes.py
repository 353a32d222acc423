"""Two device probes behind design decisions of the small-batch kernels (development aid).

Needs a library built with the probes compiled in:

    MOC_FFN_NVCC_FLAGS=-DMOC_TIMELINE python -m paper_2511_09323_b200.build --force
    python -m paper_2511_09323_b200.issue_probes
    python -m paper_2511_09323_b200.build --force          # back to the normal build

1. What a short tcgen05.mma and a tcgen05.commit cost the thread that issues them, and whether a second issuing thread
   is slowed by the first one's commits.
2. Streaming one LLaMA-7B weight matrix (11008 x 4096 bf16, 90 MB) as TMA boxes of `rows` x 128 bytes, `boxes`
   adjacent boxes per stage, against the number of stages: whether the strided box pattern of a weights-as-MMA-rows
   kernel reads HBM as fast as large contiguous copies.
"""
import ctypes

import torch

from . import binding as B


def main():
    lib = B.load()
    if not hasattr(lib, "moc_debug_mma_cycles"):
        raise SystemExit("this build has no probes: rebuild with MOC_FFN_NVCC_FLAGS=-DMOC_TIMELINE")
    torch.zeros(1, device="cuda")
    lib.moc_debug_mma_cycles.restype = ctypes.c_longlong
    lib.moc_debug_mma_cycles.argtypes = [ctypes.c_int] * 5
    print("cycles per MMA for the issuing thread (4096 MMAs, K = 16)")
    print("   M    N  MMAs/commit   unwaited commits   waited commits   unwaited, two issuers")
    for m, n in ((128, 16), (128, 32), (128, 64), (128, 128), (128, 256), (64, 16)):
        for pc in (8, 16, 64, 256):
            row = []
            for mode in (0, 1, 2):
                lib.moc_debug_mma_cycles(m, n, 256, pc, mode)
                row.append(lib.moc_debug_mma_cycles(m, n, 4096, pc, mode) / 4096)
            print(f"{m:4d} {n:4d} {pc:8d} {row[0]:18.1f} {row[1]:16.1f} {row[2]:18.1f}", flush=True)

    F, d = 11008, 4096
    ws = [torch.randn(F, d, device="cuda").to(torch.bfloat16) for _ in range(8)]   # 8 x 90 MB > L2
    lib.moc_debug_stream_boxes.argtypes = [ctypes.c_void_p] + [ctypes.c_int] * 5 + [ctypes.c_void_p]

    def run(rows, boxes, stages):
        def once(i):
            rc = lib.moc_debug_stream_boxes(ws[i % 8].data_ptr(), F, d, rows, boxes, stages, None)
            assert rc == 0, rc
        for i in range(8):
            once(i)
        torch.cuda.synchronize()
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record()
        for i in range(40):
            once(i)
        e.record()
        torch.cuda.synchronize()
        return s.elapsed_time(e) * 1e3 / 40

    print("\nbox streaming: one kernel launch per matrix, back to back (the time includes the launch's ramps)")
    print("rows/CTA boxes/stage stages  KiB in flight/SM   us    TB/s")
    for rows in (84, 128, 256):
        for boxes in (1, 2, 4, 8):
            pitch = (rows * 128 + 1023) // 1024 * 1024
            for inflight in (100, 150, 200):
                stages = min(32, inflight * 1024 // (boxes * pitch))
                if stages < 2:
                    continue
                us = run(rows, boxes, stages)
                print(f"{rows:8d} {boxes:11d} {stages:6d} {stages * boxes * rows * 128 / 1024:14.0f} {us:8.2f} {F * d * 2 / us / 1e6:6.2f}",
                      flush=True)
    assert B.moc_last_device_status() == B.MOC_OK


if __name__ == "__main__":
    main()
