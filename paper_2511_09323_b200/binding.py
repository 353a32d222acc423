"""ctypes binding of the MoC FFN C ABI (``include/moc_ffn.h``).

Argument marshalling only: every step of the operator runs in the CUDA library.  PyTorch is
used for device memory and streams.  There is no fallback: if ``libmoc_ffn.so`` has not been
built (``python -m paper_2511_09323_b200.build``) or cannot be loaded, the first call raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmoc_ffn.so")

MOC_OK = 0
MOC_ERR_INVALID_ARG = -1
MOC_ERR_UNSUPPORTED = -2
MOC_ERR_WORKSPACE = -3
MOC_ERR_CUDA = -4
MOC_ERR_TIMEOUT = -5
MOC_ERR_BAD_INDEX = -6
MOC_ERR_STATIC_LIMIT = -7
MOC_STATIC_MAX_TOKENS, MOC_STATIC_MAX_DFF = 16, 16384
MOC_F32, MOC_BF16 = 0, 1
MOC_OP_FORWARD, MOC_OP_BACKWARD, MOC_OP_DECODE, MOC_OP_DECODE_BLOCK = 0, 1, 2, 3
MOC_FLAG_ACCUMULATE_WGRAD = 1
MOC_FLAG_SELECT_2_OF_8 = 2
MOC_FLAG_SELECT_POST_SILU = 4

EXPORTED = (
    "moc_ffn_workspace_bytes", "moc_ffn_forward", "moc_ffn_backward", "moc_ffn_decode", "moc_topk_select",
    "moc_last_device_status", "moc_ffn_saved_bytes_per_token", "moc_status_string", "moc_launch_count",
    "moc_profile_enable", "moc_profile_collect", "moc_profile_kernel_count", "moc_profile_kernel_name",
    "moc_profile_read", "moc_ffn_decode_static", "moc_tc_gemm_bf16", "moc_ffn_recompute_up",
    "moc_ffn_backward_overlap", "moc_topk_select_tc", "moc_topk_select_tc_workspace_bytes", "moc_ffn_decode_probe",
    "moc_ffn_decode_probe_workspace_bytes", "moc_tc_gemm_sp_bf16", "moc_tc_gemm_sp_dense_bf16",
    "moc_tc_gemm_sp_dense_workspace_bytes", "moc_profile_stream_read", "moc_test_small_batch_stall",
)


class MocFfnDesc(ctypes.Structure):
    _fields_ = [
        ("tokens", ctypes.c_int64), ("d_model", ctypes.c_int32), ("d_ff", ctypes.c_int32),
        ("d_ff_ld", ctypes.c_int32), ("k", ctypes.c_int32), ("dtype", ctypes.c_int32),
        ("flags", ctypes.c_uint32),
    ]


class MocError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


_lib = None


def load() -> ctypes.CDLL:
    """Loads the CUDA library; raises if it is missing (there is no CPU path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_2511_09323_b200.build`")
        lib = ctypes.CDLL(LIB_PATH)
        vp, sz = ctypes.c_void_p, ctypes.c_size_t
        dp = ctypes.POINTER(MocFfnDesc)
        lib.moc_ffn_workspace_bytes.restype = sz
        lib.moc_ffn_workspace_bytes.argtypes = [dp, ctypes.c_int]
        lib.moc_ffn_saved_bytes_per_token.restype = sz
        lib.moc_ffn_saved_bytes_per_token.argtypes = [dp]
        lib.moc_ffn_forward.restype = ctypes.c_int
        lib.moc_ffn_forward.argtypes = [dp] + [vp] * 9 + [sz, vp]
        lib.moc_ffn_backward.restype = ctypes.c_int
        lib.moc_ffn_backward.argtypes = [dp] + [vp] * 13 + [sz, vp]
        lib.moc_ffn_backward_overlap.restype = ctypes.c_int
        lib.moc_ffn_backward_overlap.argtypes = [dp] + [vp] * 13 + [sz, vp, vp]
        lib.moc_ffn_decode.restype = ctypes.c_int
        lib.moc_ffn_decode.argtypes = [dp] + [vp] * 6 + [sz, vp]
        lib.moc_ffn_decode_block.restype = ctypes.c_int
        lib.moc_ffn_decode_block.argtypes = [dp, vp, vp, ctypes.c_float] + [vp] * 5 + [sz, vp]
        lib.moc_ffn_recompute_up.restype = ctypes.c_int
        lib.moc_ffn_recompute_up.argtypes = [dp] + [vp] * 5 + [sz, vp]
        lib.moc_ffn_decode_static.restype = ctypes.c_int
        lib.moc_ffn_decode_static.argtypes = [dp] + [vp] * 5 + [vp]
        lib.moc_tc_gemm_bf16.restype = ctypes.c_int
        lib.moc_tc_gemm_bf16.argtypes = [ctypes.c_int64] * 3 + [vp, ctypes.c_int, ctypes.c_int64, vp, ctypes.c_int,
                                                                ctypes.c_int64, vp, ctypes.c_int64, vp]
        lib.moc_topk_select.restype = ctypes.c_int
        lib.moc_topk_select.argtypes = [ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, vp, vp, vp]
        lib.moc_topk_select_tc_workspace_bytes.restype = sz
        lib.moc_topk_select_tc_workspace_bytes.argtypes = [ctypes.c_int64] + [ctypes.c_int32] * 3
        lib.moc_topk_select_tc.restype = ctypes.c_int
        lib.moc_topk_select_tc.argtypes = [ctypes.c_int64] + [ctypes.c_int32] * 3 + [vp, vp, ctypes.POINTER(ctypes.c_float),
                                                                                  ctypes.POINTER(ctypes.c_int), vp, sz, vp]
        lib.moc_ffn_decode_probe_workspace_bytes.restype = sz
        lib.moc_ffn_decode_probe_workspace_bytes.argtypes = [dp]
        lib.moc_ffn_decode_probe.restype = ctypes.c_int
        lib.moc_ffn_decode_probe.argtypes = [dp] + [vp] * 7 + [sz, vp]
        lib.moc_tc_gemm_sp_bf16.restype = ctypes.c_int
        lib.moc_tc_gemm_sp_bf16.argtypes = [ctypes.c_int64] * 3 + [vp, vp, vp, ctypes.c_int, ctypes.c_int64, vp,
                                                                  ctypes.c_int64, vp]
        lib.moc_tc_gemm_sp_dense_workspace_bytes.restype = sz
        lib.moc_tc_gemm_sp_dense_workspace_bytes.argtypes = [ctypes.c_int64] * 2
        lib.moc_tc_gemm_sp_dense_bf16.restype = ctypes.c_int
        lib.moc_tc_gemm_sp_dense_bf16.argtypes = [ctypes.c_int64] * 3 + [vp, ctypes.c_int64, vp, ctypes.c_int64, vp,
                                                                        ctypes.c_int64, ctypes.c_int,
                                                                        ctypes.POINTER(ctypes.c_int64), vp, sz, vp]
        lib.moc_profile_stream_read.restype = ctypes.c_int
        lib.moc_profile_stream_read.argtypes = [vp, sz, vp, sz, vp, sz, vp]
        lib.moc_last_device_status.restype = ctypes.c_int
        lib.moc_test_bounded_wait.argtypes = [ctypes.c_int64, vp]
        lib.moc_test_bounded_wait.restype = ctypes.c_int
        lib.moc_test_small_batch_stall.argtypes = [dp] + [vp] * 6 + [sz, ctypes.c_int64, vp]
        lib.moc_test_small_batch_stall.restype = ctypes.c_int
        lib.moc_last_device_status.argtypes = [vp]
        lib.moc_status_string.restype = ctypes.c_char_p
        lib.moc_status_string.argtypes = [ctypes.c_int]
        lib.moc_launch_count.restype = ctypes.c_int64
        lib.moc_launch_count.argtypes = []
        lib.moc_profile_enable.restype = ctypes.c_int
        lib.moc_profile_enable.argtypes = [ctypes.c_int]
        lib.moc_profile_collect.restype = ctypes.c_int
        lib.moc_profile_collect.argtypes = [vp]
        lib.moc_profile_kernel_count.restype = ctypes.c_int
        lib.moc_profile_kernel_count.argtypes = []
        lib.moc_profile_kernel_name.restype = ctypes.c_char_p
        lib.moc_profile_kernel_name.argtypes = [ctypes.c_int]
        lib.moc_profile_read.restype = ctypes.c_int
        lib.moc_profile_read.argtypes = [ctypes.c_int, ctypes.POINTER(ctypes.c_int64),
                                         ctypes.POINTER(ctypes.c_double)]
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load().moc_status_string(int(status)).decode()


def _dtype_code(t: torch.dtype) -> int:
    if t == torch.float32:
        return MOC_F32
    if t == torch.bfloat16:
        return MOC_BF16
    raise TypeError(f"unsupported storage dtype {t}")


def make_desc(tokens, d_model, d_ff, k, dtype, d_ff_ld=None, flags=0) -> MocFfnDesc:
    code = dtype if isinstance(dtype, int) else _dtype_code(dtype)
    return MocFfnDesc(int(tokens), int(d_model), int(d_ff), int(d_ff if d_ff_ld is None else d_ff_ld), int(k),
                      code, int(flags))


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream_ptr(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check_dev(*tensors):
    for t in tensors:
        if t is None:
            continue
        if not t.is_cuda:
            raise ValueError("expected CUDA tensors")
        if not t.is_contiguous():
            raise ValueError("expected contiguous tensors")


def moc_ffn_workspace_bytes(desc: MocFfnDesc, op: int) -> int:
    return int(load().moc_ffn_workspace_bytes(ctypes.byref(desc), int(op)))


def moc_ffn_saved_bytes_per_token(desc: MocFfnDesc) -> int:
    return int(load().moc_ffn_saved_bytes_per_token(ctypes.byref(desc)))


def alloc_workspace(desc: MocFfnDesc, op: int, device=None) -> torch.Tensor:
    n = moc_ffn_workspace_bytes(desc, op)
    return torch.empty(max(n, 16), dtype=torch.uint8, device=device or torch.device("cuda"))


def _grouped_k(k, d_ff):
    """k of the 2-of-8 mask (d_ff / 4); a caller may pass it or leave it None."""
    if d_ff % 8:
        raise ValueError("the 2-of-8 mask needs d_ff to be a multiple of 8")
    if k is not None and int(k) != d_ff // 4:
        raise ValueError("the 2-of-8 mask keeps d_ff / 4 channels")
    return d_ff // 4


def moc_ffn_forward(x, w_gate, w_up, w_down, k, d_ff=None, save=True, out=None, saved=None, workspace=None,
                    stream=None, grouped=False, post_silu=False):
    """Returns (out, topk_idx, topk_gate, topk_up); the last three are None when save=False.
    grouped=True: the 2-of-8 mask (MOC_FLAG_SELECT_2_OF_8) instead of the row Top-K; k is then d_ff / 4.
    post_silu=True: the Top-K on SiLU(g) instead of g (MOC_FLAG_SELECT_POST_SILU, the ablation variant)."""
    _check_dev(x, w_gate, w_up, w_down, out, workspace)
    T, d = x.shape
    F_ld = w_gate.shape[0]
    if grouped:
        k = _grouped_k(k, F_ld if d_ff is None else d_ff)
    desc = make_desc(T, d, F_ld if d_ff is None else d_ff, k, x.dtype, d_ff_ld=F_ld,
                     flags=(MOC_FLAG_SELECT_2_OF_8 if grouped else 0) | (MOC_FLAG_SELECT_POST_SILU if post_silu else 0))
    if out is None:
        out = torch.empty_like(x)
    if save:
        if saved is None:
            saved = (torch.empty((T, k), dtype=torch.int16, device=x.device),
                     torch.empty((T, k), dtype=x.dtype, device=x.device),
                     torch.empty((T, k), dtype=x.dtype, device=x.device))
        idx, tg, tu = saved
    else:
        idx = tg = tu = None
    if workspace is None:
        workspace = alloc_workspace(desc, MOC_OP_FORWARD, x.device)
    rc = load().moc_ffn_forward(ctypes.byref(desc), _ptr(x), _ptr(w_gate), _ptr(w_up), _ptr(w_down), _ptr(out),
                                _ptr(idx), _ptr(tg), _ptr(tu), _ptr(workspace), workspace.numel(),
                                _stream_ptr(stream))
    if rc != MOC_OK:
        raise MocError(rc, "moc_ffn_forward")
    return out, idx, tg, tu


def moc_ffn_backward(x, w_gate, w_up, w_down, topk_idx, topk_gate, topk_up, grad_out, d_ff=None,
                     want=("x", "w_gate", "w_up", "w_down"), grads=None, accumulate=False, workspace=None,
                     stream=None, wgrad_event=None, grouped=False):
    """Returns dict(grad_x, grad_w_gate, grad_w_up, grad_w_down) (None for entries not in `want`).
    `wgrad_event`: a torch.cuda.Event that the library records once the weight gradients are complete in stream
    order and before the grad_x kernel (moc_ffn_backward_overlap): a side stream that waits on it can all-reduce the
    weight gradients of a token-sharded batch while grad_x is still being computed."""
    _check_dev(x, w_gate, w_up, w_down, topk_idx, topk_gate, topk_up, grad_out, workspace)
    T, d = x.shape
    F_ld = w_gate.shape[0]
    k = topk_idx.shape[1]
    # grouped=True tells the library that the saved indices come from the 2-of-8 mask (slots 2q, 2q + 1 hold channels of
    # group q): grad_x may then run on the 2:4-sparse tensor-core MMA
    desc = make_desc(T, d, F_ld if d_ff is None else d_ff, k, x.dtype, d_ff_ld=F_ld,
                     flags=(MOC_FLAG_ACCUMULATE_WGRAD if accumulate else 0) | (MOC_FLAG_SELECT_2_OF_8 if grouped else 0))
    grads = dict(grads or {})
    res = {}
    for name, like in (("x", x), ("w_gate", w_gate), ("w_up", w_up), ("w_down", w_down)):
        key = "grad_" + name
        if name in want:
            res[key] = grads.get(key)
            if res[key] is None:
                res[key] = torch.empty_like(like)
        else:
            res[key] = None
    _check_dev(*res.values())
    if workspace is None:
        workspace = alloc_workspace(desc, MOC_OP_BACKWARD, x.device)
    args = (ctypes.byref(desc), _ptr(x), _ptr(w_gate), _ptr(w_up), _ptr(w_down), _ptr(topk_idx), _ptr(topk_gate),
            _ptr(topk_up), _ptr(grad_out), _ptr(res["grad_x"]), _ptr(res["grad_w_gate"]), _ptr(res["grad_w_up"]),
            _ptr(res["grad_w_down"]), _ptr(workspace), workspace.numel(), _stream_ptr(stream))
    if wgrad_event is None:
        rc = load().moc_ffn_backward(*args)
    else:
        if not wgrad_event.cuda_event:       # torch creates the underlying cudaEvent_t lazily: force it with a record
            wgrad_event.record(torch.cuda.current_stream(x.device) if stream is None else stream)
        rc = load().moc_ffn_backward_overlap(*args, ctypes.c_void_p(wgrad_event.cuda_event))
    if rc != MOC_OK:
        raise MocError(rc, "moc_ffn_backward")
    return res


def moc_ffn_recompute_up(x, w_up, topk_idx, d_ff=None, out=None, workspace=None, stream=None):
    """topk_up [T, k] again from x, w_up and the saved indices (for callers that kept only indices and gate values).
    `workspace`: a MOC_OP_BACKWARD workspace (the one the backward call takes next can be passed to both)."""
    _check_dev(x, w_up, topk_idx, out, workspace)
    T, d = x.shape
    F_ld = w_up.shape[0]
    k = topk_idx.shape[1]
    desc = make_desc(T, d, F_ld if d_ff is None else d_ff, k, x.dtype, d_ff_ld=F_ld)
    if out is None:
        out = torch.empty((T, k), dtype=x.dtype, device=x.device)
    if workspace is None:
        workspace = alloc_workspace(desc, MOC_OP_BACKWARD, x.device)
    rc = load().moc_ffn_recompute_up(ctypes.byref(desc), _ptr(x), _ptr(w_up), _ptr(topk_idx), _ptr(out),
                                     _ptr(workspace), workspace.numel(), _stream_ptr(stream))
    if rc != MOC_OK:
        raise MocError(rc, "moc_ffn_recompute_up")
    return out


def moc_ffn_decode(x, w_gate, w_up, w_down, k, d_ff=None, out=None, workspace=None, stream=None, grouped=False,
                   post_silu=False):
    _check_dev(x, w_gate, w_up, w_down, out, workspace)
    T, d = x.shape
    F_ld = w_gate.shape[0]
    if grouped:
        k = _grouped_k(k, F_ld if d_ff is None else d_ff)
    desc = make_desc(T, d, F_ld if d_ff is None else d_ff, k, x.dtype, d_ff_ld=F_ld,
                     flags=(MOC_FLAG_SELECT_2_OF_8 if grouped else 0) | (MOC_FLAG_SELECT_POST_SILU if post_silu else 0))
    if out is None:
        out = torch.empty_like(x)
    if workspace is None:
        workspace = alloc_workspace(desc, MOC_OP_DECODE, x.device)
    rc = load().moc_ffn_decode(ctypes.byref(desc), _ptr(x), _ptr(w_gate), _ptr(w_up), _ptr(w_down), _ptr(out),
                               _ptr(workspace), workspace.numel(), _stream_ptr(stream))
    if rc != MOC_OK:
        raise MocError(rc, "moc_ffn_decode")
    return out


def moc_ffn_decode_block(h, rms_weight, rms_eps, w_gate, w_up, w_down, k, d_ff=None, out=None, workspace=None,
                         stream=None, grouped=False):
    """out = h + MoC_FFN(RMSNorm(h; rms_weight, rms_eps)) for up to 256 bf16 tokens; `out` may be `h`."""
    _check_dev(h, rms_weight, w_gate, w_up, w_down, out, workspace)
    T, d = h.shape
    if rms_weight.dtype != h.dtype or tuple(rms_weight.shape) != (d,):
        raise TypeError("rms_weight must be a [d_model] tensor of the activations' dtype")
    F_ld = w_gate.shape[0]
    if grouped:
        k = _grouped_k(k, F_ld if d_ff is None else d_ff)
    desc = make_desc(T, d, F_ld if d_ff is None else d_ff, k, h.dtype, d_ff_ld=F_ld,
                     flags=MOC_FLAG_SELECT_2_OF_8 if grouped else 0)
    if out is None:
        out = torch.empty_like(h)
    if workspace is None:
        workspace = alloc_workspace(desc, MOC_OP_DECODE_BLOCK, h.device)
    rc = load().moc_ffn_decode_block(ctypes.byref(desc), _ptr(h), _ptr(rms_weight), float(rms_eps), _ptr(w_gate),
                                     _ptr(w_up), _ptr(w_down), _ptr(out), _ptr(workspace), workspace.numel(),
                                     _stream_ptr(stream))
    if rc != MOC_OK:
        raise MocError(rc, "moc_ffn_decode_block")
    return out


def moc_ffn_decode_static(x, w_gate, w_up, w_down, k, out, d_ff=None, stream=None, grouped=False, post_silu=False):
    """Decode for callers that cannot allocate: no workspace argument, and `out` must be supplied, so that
    nothing on this call path asks any allocator (torch's included) for memory.  The transient buffers
    live in an array inside the library; see the limits and the sharing rules in include/moc_ffn.h."""
    _check_dev(x, w_gate, w_up, w_down, out)
    T, d = x.shape
    F_ld = w_gate.shape[0]
    if grouped:
        k = _grouped_k(k, F_ld if d_ff is None else d_ff)
    desc = make_desc(T, d, F_ld if d_ff is None else d_ff, k, x.dtype, d_ff_ld=F_ld,
                     flags=(MOC_FLAG_SELECT_2_OF_8 if grouped else 0) | (MOC_FLAG_SELECT_POST_SILU if post_silu else 0))
    rc = load().moc_ffn_decode_static(ctypes.byref(desc), _ptr(x), _ptr(w_gate), _ptr(w_up), _ptr(w_down),
                                      _ptr(out), _stream_ptr(stream))
    if rc != MOC_OK:
        raise MocError(rc, "moc_ffn_decode_static")
    return out


def moc_topk_select(gate: torch.Tensor, k: int, n: int | None = None, stream=None) -> torch.Tensor:
    """gate [rows, n_ld] fp32 on the device -> idx [rows, k] int16 (ascending)."""
    _check_dev(gate)
    if gate.dtype != torch.float32 or gate.dim() != 2:
        raise TypeError("gate must be a 2-D fp32 tensor")
    rows, n_ld = gate.shape
    n = n_ld if n is None else n
    idx = torch.empty((rows, k), dtype=torch.int16, device=gate.device)
    rc = load().moc_topk_select(rows, n, n_ld, k, _ptr(gate), _ptr(idx), _stream_ptr(stream))
    if rc != MOC_OK:
        raise MocError(rc, "moc_topk_select")
    return idx


SELECT_VARIANTS = ("cta_per_row", "team2", "team4", "team4_shared")


def moc_topk_select_tc(gate: torch.Tensor, k: int, n: int | None = None, bracket=None, stream=None):
    """The tensor-core plan's selector alone: gate [rows, n_ld] fp32 -> (idx [rows, k] int16, variant name).
    `bracket`: (center, half width) the launch starts from, None = the state of a first call."""
    _check_dev(gate)
    if gate.dtype != torch.float32 or gate.dim() != 2:
        raise TypeError("gate must be a 2-D fp32 tensor")
    rows, n_ld = gate.shape
    n = n_ld if n is None else n
    lib = load()
    need = lib.moc_topk_select_tc_workspace_bytes(rows, n, n_ld, k)
    if need == 0:
        raise MocError(MOC_ERR_UNSUPPORTED, "moc_topk_select_tc")
    ws = torch.empty(need, dtype=torch.uint8, device=gate.device)
    idx = torch.empty((rows, k), dtype=torch.int16, device=gate.device)
    variant = ctypes.c_int(-1)
    br = None if bracket is None else (ctypes.c_float * 2)(float(bracket[0]), float(bracket[1]))
    rc = lib.moc_topk_select_tc(rows, n, n_ld, k, _ptr(gate), _ptr(idx), br, ctypes.byref(variant), _ptr(ws), need,
                                _stream_ptr(stream))
    if rc != MOC_OK:
        raise MocError(rc, "moc_topk_select_tc")
    return idx, SELECT_VARIANTS[variant.value]


def moc_ffn_decode_probe(x, w_gate, w_up, w_down, k, d_ff=None, stream=None, grouped=False):
    """The one-kernel decode form for one or two tokens with its mask: (out [T, d], kept [T, d_ff] uint8)."""
    _check_dev(x, w_gate, w_up, w_down)
    T, d = x.shape
    F_ld = w_gate.shape[0]
    F = F_ld if d_ff is None else d_ff
    if grouped:
        k = _grouped_k(k, F)
    desc = make_desc(T, d, F, k, x.dtype, d_ff_ld=F_ld, flags=MOC_FLAG_SELECT_2_OF_8 if grouped else 0)
    out = torch.empty_like(x)
    kept = torch.full((T, F), 255, dtype=torch.uint8, device=x.device)
    need = load().moc_ffn_decode_probe_workspace_bytes(ctypes.byref(desc))
    if need == 0:
        raise MocError(MOC_ERR_UNSUPPORTED, "moc_ffn_decode_probe")
    ws = torch.empty(need, dtype=torch.uint8, device=x.device)
    rc = load().moc_ffn_decode_probe(ctypes.byref(desc), _ptr(x), _ptr(w_gate), _ptr(w_up), _ptr(w_down), _ptr(out),
                                     _ptr(kept), _ptr(ws), ws.numel(), _stream_ptr(stream))
    if rc != MOC_OK:
        raise MocError(rc, "moc_ffn_decode_probe")
    return out, kept


def moc_tc_gemm_sp_bf16(a_compressed: torch.Tensor, metadata: torch.Tensor, b: torch.Tensor, k: int,
                        b_mn_major: bool = False, stream=None) -> torch.Tensor:
    """The one-CTA sparse GEMM on caller-built operands: a_compressed [m, k/2] bf16, metadata int32 words in the
    tensor-memory arrangement (include/moc_ffn.h), b [n, k] (or [k, n] when b_mn_major) -> C [m, n] fp32."""
    _check_dev(a_compressed, metadata, b)
    m = a_compressed.shape[0]
    n = b.shape[1] if b_mn_major else b.shape[0]
    c = torch.empty((m, n), dtype=torch.float32, device=b.device)
    rc = load().moc_tc_gemm_sp_bf16(m, n, k, _ptr(a_compressed), _ptr(metadata), _ptr(b), int(b_mn_major), b.stride(0),
                                    _ptr(c), n, _stream_ptr(stream))
    if rc != MOC_OK:
        raise MocError(rc, "moc_tc_gemm_sp_bf16")
    return c


def moc_tc_gemm_sp_dense_bf16(a: torch.Tensor, b: torch.Tensor, out=None, accumulate: bool = False, stream=None):
    """a [m, k] bf16 with at most 2 non-zero values per 4 consecutive elements, b [k, n] bf16 -> (C [m, n] bf16, number
    of values that did not fit the 2:4 pattern and were left out)."""
    _check_dev(a, b, out)
    m, k = a.shape
    n = b.shape[1]
    lib = load()
    need = lib.moc_tc_gemm_sp_dense_workspace_bytes(m, k)
    if need == 0:
        raise MocError(MOC_ERR_INVALID_ARG, "moc_tc_gemm_sp_dense_bf16")
    ws = torch.empty(need, dtype=torch.uint8, device=a.device)
    if out is None:
        out = torch.empty((m, n), dtype=torch.bfloat16, device=a.device)
    left_out = ctypes.c_int64(-1)
    rc = lib.moc_tc_gemm_sp_dense_bf16(m, n, k, _ptr(a), a.stride(0), _ptr(b), b.stride(0), _ptr(out), out.stride(0),
                                       int(accumulate), ctypes.byref(left_out), _ptr(ws), need, _stream_ptr(stream))
    if rc != MOC_OK:
        raise MocError(rc, "moc_tc_gemm_sp_dense_bf16")
    return out, int(left_out.value)


def moc_last_device_status(stream=None) -> int:
    return int(load().moc_last_device_status(_stream_ptr(stream)))


def moc_test_bounded_wait(limit_cycles: int, stream=None) -> None:
    """Launches the probe whose bounded wait runs out after `limit_cycles` SM cycles (the status word then reads
    MOC_ERR_TIMEOUT)."""
    rc = load().moc_test_bounded_wait(int(limit_cycles), _stream_ptr(stream))
    if rc != MOC_OK:
        raise MocError(rc, "moc_test_bounded_wait")


def moc_test_small_batch_stall(x, w_gate, w_up, w_down, k, limit_cycles: int, d_ff=None, out=None, workspace=None,
                               stream=None):
    """moc_ffn_decode's call for up to 32 tokens, run so that every CTA of its cooperative kernel meets a wait that nothing
    completes and gives up after `limit_cycles` SM cycles (the status word then reads MOC_ERR_TIMEOUT; `out` is not
    written).  Returns `out`."""
    _check_dev(x, w_gate, w_up, w_down, out, workspace)
    T, d = x.shape
    F_ld = w_gate.shape[0]
    desc = make_desc(T, d, F_ld if d_ff is None else d_ff, k, x.dtype, d_ff_ld=F_ld)
    if out is None:
        out = torch.empty_like(x)
    if workspace is None:
        workspace = alloc_workspace(desc, MOC_OP_DECODE, x.device)
    rc = load().moc_test_small_batch_stall(ctypes.byref(desc), _ptr(x), _ptr(w_gate), _ptr(w_up), _ptr(w_down), _ptr(out),
                                           _ptr(workspace), workspace.numel(), int(limit_cycles), _stream_ptr(stream))
    if rc != MOC_OK:
        raise MocError(rc, "moc_test_small_batch_stall")
    return out


def moc_launch_count() -> int:
    return int(load().moc_launch_count())


def moc_profile_enable(on: bool) -> None:
    rc = load().moc_profile_enable(1 if on else 0)
    if rc != MOC_OK:
        raise MocError(rc, "moc_profile_enable")


def moc_profile_stream_read(ranges, stream=None) -> None:
    """A bare streaming read of up to three (tensor, bytes) ranges: the floor under any kernel that has to read them."""
    flat = []
    for t, n in list(ranges) + [(None, 0)] * (3 - len(ranges)):
        flat += [_ptr(t) if t is not None else None, int(n) // 16 * 16]
    rc = load().moc_profile_stream_read(*flat, _stream_ptr(stream))
    if rc != MOC_OK:
        raise MocError(rc, "moc_profile_stream_read")


def moc_profile_collect(stream=None) -> dict:
    """Synchronises the stream and returns {kernel name: (launches, total_ms)} for the open window."""
    lib = load()
    rc = lib.moc_profile_collect(_stream_ptr(stream))
    if rc < 0:
        raise MocError(rc, "moc_profile_collect")
    out = {}
    for i in range(lib.moc_profile_kernel_count()):
        n, ms = ctypes.c_int64(0), ctypes.c_double(0.0)
        lib.moc_profile_read(i, ctypes.byref(n), ctypes.byref(ms))
        if n.value:
            out[lib.moc_profile_kernel_name(i).decode()] = (int(n.value), float(ms.value))
    out["_dropped"] = (rc, 0.0)
    return out


def moc_tc_gemm_bf16(a: torch.Tensor, b: torch.Tensor, a_mn_major: bool = False, b_mn_major: bool = False,
                     stream=None) -> torch.Tensor:
    """C[m,n] fp32 = sum_k A(m,k) B(n,k).  a is [m,k] (or [k,m] when a_mn_major), b is [n,k] (or [k,n])."""
    _check_dev(a, b)
    if a.dtype != torch.bfloat16 or b.dtype != torch.bfloat16:
        raise TypeError("bf16 operands expected")
    m, k = (a.shape[1], a.shape[0]) if a_mn_major else a.shape
    n, kb = (b.shape[1], b.shape[0]) if b_mn_major else b.shape
    if k != kb:
        raise ValueError("contraction sizes differ")
    c = torch.empty((m, n), dtype=torch.float32, device=a.device)
    rc = load().moc_tc_gemm_bf16(m, n, k, _ptr(a), int(a_mn_major), a.stride(0), _ptr(b), int(b_mn_major),
                                 b.stride(0), _ptr(c), n, _stream_ptr(stream))
    if rc != MOC_OK:
        raise MocError(rc, "moc_tc_gemm_bf16")
    return c
