"""Small-batch decode through the C ABI on the LLaMA-7B FFN shape: a few calls of `moc_ffn_decode` that rotate four weight sets
(1.08 GB, more than the L2 holds) so that every call streams its weights from HBM, as a decoding loop over many layers does.

    python -m paper_2511_09323_b200.decode_demo [tokens] [calls]

Prints the device status word.  Used as the small, self-contained command for profiler captures of the decode kernels.
"""
import sys

import torch

from . import binding as B
from . import synthetic as syn


def main(argv):
    tokens = int(argv[1]) if len(argv) > 1 else 1
    calls = int(argv[2]) if len(argv) > 2 else 8
    B.load()
    w = syn.C4
    wg, wu, wd = (t.cuda() for t in syn.make_weights(w))
    sets = [(wg, wu, wd)] + [tuple(t.clone() for t in (wg, wu, wd)) for _ in range(3)]
    x = syn.make_x(w, tokens=tokens).cuda()
    out = torch.empty_like(x)
    desc = B.make_desc(tokens, w.d_model, w.d_ff, w.k, x.dtype)
    ws = B.alloc_workspace(desc, B.MOC_OP_DECODE)
    for i in range(calls):
        B.moc_ffn_decode(x, *sets[i % 4], w.k, out=out, workspace=ws)
    torch.cuda.synchronize()
    print("decode calls:", calls, "tokens:", tokens, "device status:", B.moc_last_device_status())
    return 0


if __name__ == "__main__":
    sys.exit(main(sys.argv))
