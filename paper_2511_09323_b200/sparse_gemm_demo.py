"""The 2:4-sparse down projection next to the dense one (the commands under profiles/ run this).

    python -m paper_2511_09323_b200.sparse_gemm_demo [tokens] [d_model] [d_ff] [repeats]

A [tokens, d_ff] masked hidden state with the 2-of-8 structure of MoC 2:8 (Section 4) is contracted with a
[d_ff, d_model] weight matrix twice: by moc_tc_gemm_sp_dense_bf16 (compression + tcgen05.mma.sp on CTA pairs) and by
moc_tc_gemm_bf16 (the dense tcgen05 kernel).  Prints the library's per-kernel event times of both.
"""
import sys

import torch

from . import binding as B


def main():
    T, d, F, reps = (int(a) for a in (sys.argv[1:5] + ["8192", "2048", "5504", "5"][len(sys.argv) - 1:]))
    gen = torch.Generator().manual_seed(0)
    z = torch.zeros(T, F // 8, 8)
    keep = torch.rand(T, F // 8, 8, generator=gen).argsort(dim=-1) < 2          # 2 of every 8 channels
    z = torch.where(keep, torch.randn(T, F // 8, 8, generator=gen), z).reshape(T, F).to(torch.bfloat16).cuda()
    w = (torch.randn(F, d, generator=gen) * 0.02).to(torch.bfloat16).cuda()
    B.load()
    for _ in range(2):
        out, left_out = B.moc_tc_gemm_sp_dense_bf16(z, w)
        ref = B.moc_tc_gemm_bf16(z, w, b_mn_major=True)
    torch.cuda.synchronize()
    err = (out.float() - ref).abs().max().item() / ref.abs().max().item()
    B.moc_profile_enable(True)
    for _ in range(reps):
        B.moc_tc_gemm_sp_dense_bf16(z, w, out=out)
    sparse = B.moc_profile_collect()
    B.moc_profile_enable(True)
    for _ in range(reps):
        B.moc_tc_gemm_bf16(z, w, b_mn_major=True)
    dense = B.moc_profile_collect()
    B.moc_profile_enable(False)
    ms = lambda prof, name: prof[name][1] / prof[name][0]
    print(f"tokens {T}, d_model {d}, d_ff {F}: sparse GEMM {ms(sparse, 'tc_test_gemm'):.4f} ms (+ compression "
          f"{ms(sparse, 'tc_compress_2of4'):.4f} ms), dense GEMM {ms(dense, 'tc_test_gemm'):.4f} ms; "
          f"values left out {left_out}; max |sparse - dense| / max |dense| = {err:.2e}")
    if B.moc_last_device_status() != B.MOC_OK:
        raise SystemExit("device status raised")


if __name__ == "__main__":
    main()
