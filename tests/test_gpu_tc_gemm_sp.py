"""The 2:4-sparse tensor-core contraction (tcgen05.mma.sp) against a float64 matmul.

Section 4 ("MoC with structured 2:8 sparsity"): a row of the 2:8-masked hidden state has at most 2 non-zero values in
every 4 consecutive channels, so the down projection can run on the sparse MMA.  Two entry points are checked: the
one-CTA kernel on operands this test compresses itself (which pins the metadata arrangement stated in the header), and
the CTA-pair kernel behind the library's own compression of a dense 2:4 array.
"""
import numpy as np
import pytest
import torch

from paper_2511_09323_b200 import binding as B
from paper_2511_09323_b200 import build as moc_build

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    moc_build.build()
    B.load()
    assert B.moc_last_device_status() == B.MOC_OK
    yield
    assert B.moc_last_device_status() == B.MOC_OK


def _sparse_2of4(m, k, gen, max_kept=2, small_ints=False):
    """[m, k] with 0..max_kept non-zero values at random positions of every group of 4."""
    cnt = torch.randint(0, max_kept + 1, (m, k // 4, 1), generator=gen)
    order = torch.rand(m, k // 4, 4, generator=gen).argsort(dim=-1)
    vals = torch.randint(-4, 5, (m, k // 4, 4), generator=gen).float() if small_ints else torch.randn(m, k // 4, 4, generator=gen)
    return torch.where(order < cnt, vals, torch.zeros(())).reshape(m, k).to(torch.bfloat16)


def _compress(a):
    """numpy restatement of the operand format: values [m, k/2] and one nibble per group of 4 [m, k/4]."""
    a = a.float().numpy()
    m, k = a.shape
    g = a.reshape(m, k // 4, 4)
    comp = np.zeros((m, k // 4, 2), np.float32)
    nib = np.zeros((m, k // 4), np.uint32)
    for i in range(m):
        for j in range(k // 4):
            nz = np.nonzero(g[i, j])[0].tolist()
            assert len(nz) <= 2
            pos = [0, 1] if not nz else ([nz[0], 3] if nz[0] < 3 else [2, 3]) if len(nz) == 1 else nz
            comp[i, j] = g[i, j, pos]
            nib[i, j] = pos[0] | (pos[1] << 2)
    return comp.reshape(m, k // 2), nib


def _metadata_words(nib, m, k):
    """[ceil(m/128)][ceil(k/128)][128 lanes][4 columns]: lane l, column c hold rows (l % 8) + 16 (l / 16) (bits 0..15)
    and + 8 (bits 16..31), groups 4 ((l / 8) % 2) .. + 3 of the 8 groups of elements 32 c .. 32 c + 31."""
    mt, ks = (m + 127) // 128, (k + 127) // 128
    full = np.full((mt * 128, ks * 32), 0x4, np.uint32)
    full[:m, :k // 4] = nib
    full = full.reshape(mt, 128, ks, 4, 2, 4)           # [tile, row, stage, column, half, group]
    out = np.zeros((mt, ks, 128, 4), np.uint32)
    for lane in range(128):
        r, half = (lane % 8) + 16 * (lane // 16), (lane // 8) % 2
        for q in range(4):
            out[:, :, lane, :] |= full[:, r, :, :, half, q] << (4 * q)
            out[:, :, lane, :] |= full[:, r + 8, :, :, half, q] << (16 + 4 * q)
    return out


@pytest.mark.parametrize("m,n,k", [(128, 128, 128), (200, 136, 400), (256, 256, 512)])
@pytest.mark.parametrize("b_mn_major", [False, True])
def test_sparse_mma_on_hand_compressed_operands(m, n, k, b_mn_major):
    gen = torch.Generator().manual_seed(m + n + k)
    a = _sparse_2of4(m, k, gen, small_ints=True)
    b = torch.randint(-4, 5, (k, n), generator=gen).float()
    comp, nib = _compress(a)
    words = torch.from_numpy(_metadata_words(nib, m, k).view(np.int32)).cuda().contiguous()
    bt = (b if b_mn_major else b.T.contiguous()).to(torch.bfloat16).cuda()
    got = B.moc_tc_gemm_sp_bf16(torch.from_numpy(comp).to(torch.bfloat16).cuda().contiguous(), words, bt, k,
                                b_mn_major=b_mn_major)
    torch.cuda.synchronize()
    ref = a.double() @ b.double()
    assert torch.equal(got.cpu().double(), ref), "small integers: the products and sums are exact"


@pytest.mark.parametrize("m,n,k", [(77, 136, 64), (300, 520, 1000), (512, 768, 2048), (1000, 2048, 5504)])
def test_sparse_pair_gemm_with_library_compression(m, n, k):
    gen = torch.Generator().manual_seed(7 * m + k)
    a = _sparse_2of4(m, k, gen).cuda()
    b = (torch.randn(k, n, generator=gen) * 0.05).to(torch.bfloat16).cuda()
    ref = a.double() @ b.double()
    got, left_out = B.moc_tc_gemm_sp_dense_bf16(a, b)
    torch.cuda.synchronize()
    assert left_out == 0
    scale = ref.abs().max().item()
    assert (got.double() - ref).abs().max().item() <= 1e-2 * scale
    prev = torch.randn(m, n, generator=gen).to(torch.bfloat16).cuda()
    got2, _ = B.moc_tc_gemm_sp_dense_bf16(a, b, out=prev.clone(), accumulate=True)
    torch.cuda.synchronize()
    ref2 = ref + prev.double()
    assert (got2.double() - ref2).abs().max().item() <= 1e-2 * ref2.abs().max().item()


def test_values_beyond_two_per_group_are_counted_not_silently_used():
    gen = torch.Generator().manual_seed(3)
    m, n, k = 256, 256, 512
    a = torch.where(torch.rand(m, k, generator=gen) < 0.3, torch.randn(m, k, generator=gen), torch.zeros(())).to(torch.bfloat16)
    extra = int((((a != 0).reshape(m, k // 4, 4).sum(-1) - 2).clamp(min=0)).sum())
    assert extra > 0
    b = (torch.randn(k, n, generator=gen) * 0.05).to(torch.bfloat16)
    got, left_out = B.moc_tc_gemm_sp_dense_bf16(a.cuda(), b.cuda())
    assert left_out == extra
    # what was computed is the product with the first two non-zero values of every group
    kept = a.clone().reshape(m, k // 4, 4)
    seen = (kept != 0).cumsum(-1)
    kept[seen > 2] = 0
    ref = kept.reshape(m, k).double() @ b.double()
    assert (got.cpu().double() - ref).abs().max().item() <= 1e-2 * ref.abs().max().item()
