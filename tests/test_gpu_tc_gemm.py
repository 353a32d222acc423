"""The tcgen05 GEMM on its own, against a float64 matmul of the same bf16 inputs."""
import pytest
import torch

from paper_2511_09323_b200 import binding as B
from paper_2511_09323_b200 import build as moc_build

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    moc_build.build()
    B.load()
    yield
    assert B.moc_last_device_status() == B.MOC_OK


def _operand(rows_mn, k, mn_major, gen, pad=0):
    """Returns (storage tensor handed to the library, logical [mn, k] float64 matrix)."""
    logical = torch.randn(rows_mn, k, generator=gen, dtype=torch.float32).to(torch.bfloat16)
    up8 = lambda v: (v + 7) // 8 * 8          # leading dimensions must be multiples of 8 elements (16 bytes)
    if mn_major:
        store = torch.full((k, up8(rows_mn + pad)), 7.0, dtype=torch.bfloat16)   # padding holds junk, not zeros
        store[:, :rows_mn] = logical.t()
        dev = store.cuda()[:, :rows_mn]
    else:
        store = torch.full((rows_mn, up8(k + pad)), 7.0, dtype=torch.bfloat16)
        store[:, :k] = logical
        dev = store.cuda()[:, :k]
    return dev, logical.double()


def _run(m, n, k, a_mn, b_mn, pad=0):
    gen = torch.Generator().manual_seed(m * 7 + n * 3 + k + 2 * a_mn + b_mn)
    a_dev, a64 = _operand(m, k, a_mn, gen, pad)
    b_dev, b64 = _operand(n, k, b_mn, gen, pad)
    lib = B.load()
    c = torch.full((m, n), float("nan"), dtype=torch.float32, device="cuda")
    import ctypes
    rc = lib.moc_tc_gemm_bf16(m, n, k, ctypes.c_void_p(a_dev.data_ptr()), int(a_mn), a_dev.stride(0),
                              ctypes.c_void_p(b_dev.data_ptr()), int(b_mn), b_dev.stride(0),
                              ctypes.c_void_p(c.data_ptr()), n, ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert rc == B.MOC_OK
    torch.cuda.synchronize()
    assert B.moc_last_device_status() == B.MOC_OK
    ref = a64 @ b64.t()
    err = (c.double().cpu() - ref).abs().max().item()
    scale = ref.abs().max().item()
    # fp32 accumulation of exact bf16 products: error ~ k * 2^-24 relative to the partial sums
    assert err <= 2e-5 * scale * max(1.0, (k / 64) ** 0.5), f"m={m} n={n} k={k} a_mn={a_mn} b_mn={b_mn}: err {err:.3e} scale {scale:.3e}"


@pytest.mark.parametrize("a_mn,b_mn", [(False, False), (False, True), (True, True), (True, False)])
@pytest.mark.parametrize("m,n,k", [(128, 256, 64), (128, 256, 256), (256, 512, 128)])
def test_exact_tiles(m, n, k, a_mn, b_mn):
    _run(m, n, k, a_mn, b_mn)


@pytest.mark.parametrize("a_mn,b_mn", [(False, False), (False, True), (True, True), (True, False)])
@pytest.mark.parametrize("m,n,k", [(1, 8, 8), (130, 264, 72), (300, 520, 200), (77, 1000, 1000)])
def test_ragged_edges(m, n, k, a_mn, b_mn):
    _run(m, n, k, a_mn, b_mn)


@pytest.mark.parametrize("a_mn,b_mn", [(False, False), (False, True), (True, True)])
def test_many_tiles_persistent_schedule_and_padding(a_mn, b_mn):
    # more tiles than SMs, long contraction (pipeline wraps many times), leading dimension > extent
    _run(2500, 1300, 1544, a_mn, b_mn, pad=8)


def test_output_pitch_a_tensor_map_cannot_describe():
    # 250 fp32 columns = 1000-byte rows: not a multiple of 16 bytes, so the epilogue stores rows thread by thread
    _run(200, 250, 136, False, False)
    _run(200, 250, 136, True, True)


def test_single_cta_kernel_selected_by_environment():
    """MOC_FFN_GEMM=single (read once per process) routes every GEMM to the one-CTA kernel: run the exact-tile and
    ragged cases again in a child process with it set."""
    import os
    import subprocess
    import sys
    env = dict(os.environ, MOC_FFN_GEMM="single")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(root, "tests", "test_gpu_tc_gemm.py"), "-q", "-x",
                        "-m", "gpu", "-k", "exact_tiles or ragged_edges or output_pitch"],
                       cwd=root, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]
