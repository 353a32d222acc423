"""Seeded synthetic inputs for the MoC FFN operator.

This module holds the workload shapes and the random-input recipe only; it contains none
of the operator's arithmetic, so both the CUDA binding's callers and the CPU oracle's tests
may draw their inputs from it.  All draws come from a CPU ``torch.Generator`` so that the
same seed gives the same arrays on every machine; values are drawn in fp32 and then rounded
once to the storage dtype, and that rounded array is what both sides consume.

Shapes follow the LLaMA configurations of the paper's pre-training table (hidden /
intermediate sizes 768/2048 for 130M, 2048/5461 for 1B) and LLaMA-7B (4096/11008) for decode.
The paper trains on C4 with learned weights; neither is available, so Gaussian tensors of the
same shapes stand in: the operator's cost depends on the shapes and on K, not on token content.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    dtype: str          # "f32" | "bf16" : storage type of x, weights, outputs, saved values, grads
    tokens: int         # T = batch * seq
    d_model: int        # d
    d_ff: int           # F, logical channel count
    d_ff_ld: int        # rows allocated per weight array (>= d_ff; the tail rows are zero)
    k: int              # channels kept per token
    seed: int
    rms_norm_x: bool = False   # per-token x / sqrt(mean(x^2) + 1e-6) before rounding
    decode: bool = False
    batch: int = 0
    seq: int = 0

    def with_tokens(self, tokens: int) -> "Workload":
        return replace(self, tokens=tokens, batch=0, seq=0)


# The five benchmark configurations.  C1 is the tiny fp32 case the oracle finishes at once; C2 and C3 are the
# LLaMA-130M and LLaMA-1B training shapes; C4 is the LLaMA-7B decode shape; C5 (65536 tokens on the 1B shape, three K)
# is the largest single-GPU training case and the one the benchmark's headline line runs.
C1 = Workload("C1-tiny-f32", "f32", 256, 128, 512, 512, 64, seed=0)
C2 = Workload("C2-llama130m-bf16", "bf16", 64 * 256, 768, 2048, 2048, 256, seed=2, rms_norm_x=True,
              batch=64, seq=256)
C3 = Workload("C3-llama1b-bf16", "bf16", 32 * 1024, 2048, 5461, 5504, 688, seed=3, batch=32, seq=1024)
C4 = Workload("C4-llama7b-decode-bf16", "bf16", 1, 4096, 11008, 11008, 1376, seed=4, decode=True)
C5 = Workload("C5-llama1b-sweep-bf16", "bf16", 65536, 2048, 5504, 5504, 688, seed=5)

WORKLOADS = {w.name.split("-")[0]: w for w in (C1, C2, C3, C4, C5)}
C4_BATCHES = (1, 4, 16)
C5_K = (344, 688, 1376)
C5_BATCH_SEQ = ((256, 256), (128, 512), (64, 1024), (32, 2048), (16, 4096))


def torch_dtype(name: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return g


def make_weights(w: Workload, seed_offset: int = 0):
    """(w_gate, w_up, w_down), each [d_ff_ld, d] channel-major, N(0, 0.02^2), zero rows beyond d_ff."""
    g = _gen(1000003 * (w.seed + 1) + 17 + 7919 * seed_offset)
    out = []
    for _ in range(3):
        m = torch.randn(w.d_ff_ld, w.d_model, generator=g, dtype=torch.float32) * 0.02
        if w.d_ff_ld > w.d_ff:
            m[w.d_ff:] = 0.0
        out.append(m.to(torch_dtype(w.dtype)).contiguous())
    return tuple(out)


def make_x(w: Workload, tokens: int | None = None, shard: int = 0):
    """x [T, d] ~ N(0,1), optionally RMS-normalised per token, rounded to the storage dtype.

    `shard`: a batch sharded by tokens over several GPUs is the concatenation of its shards, each drawn from its own
    seed (shard 0 is the single-GPU batch), so no rank has to draw the other ranks' tokens."""
    T = w.tokens if tokens is None else tokens
    g = _gen(1000003 * (w.seed + 1) + 1 + 104729 * shard)
    x = torch.randn(T, w.d_model, generator=g, dtype=torch.float32)
    if w.rms_norm_x:
        x = x / torch.sqrt(x.pow(2).mean(dim=1, keepdim=True) + 1e-6)
    return x.to(torch_dtype(w.dtype)).contiguous()


def make_grad_out(w: Workload, tokens: int | None = None, shard: int = 0):
    """Upstream gradient [T, d] ~ N(0,1), rounded to the storage dtype; `shard` as in make_x."""
    T = w.tokens if tokens is None else tokens
    g = _gen(1000003 * (w.seed + 1) + 2 + 104729 * shard)
    return torch.randn(T, w.d_model, generator=g, dtype=torch.float32).to(torch_dtype(w.dtype)).contiguous()


def to_f64(t: torch.Tensor) -> np.ndarray:
    """Widen a (possibly bf16) CPU/GPU tensor to a float64 numpy array without changing its values."""
    return t.detach().to("cpu").to(torch.float64).numpy()


def round_to(a: np.ndarray, dtype: str) -> np.ndarray:
    """Round a float64 array to the storage dtype (round-to-nearest-even) and widen it back."""
    return torch.from_numpy(np.ascontiguousarray(a)).to(torch_dtype(dtype)).to(torch.float64).numpy()
