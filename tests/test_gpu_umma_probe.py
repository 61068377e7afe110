"""Bring-up checks of the tcgen05 / TMA / TMEM building blocks against a host matmul."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mdn():
    import paper_2605_05838_b200 as m
    m.lib()
    return m


def bf16_mat(rng, shape):
    import torch
    return torch.from_numpy(rng.standard_normal(shape).astype(np.float32)).to(torch.bfloat16)


def run(mdn, mode, a, b, out_shape):
    import torch
    out = torch.full(out_shape, float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    mdn.selftest_umma(mode, a.cuda(), None if b is None else b.cuda(), out, status)
    torch.cuda.synchronize()
    assert int(status[0]) == 0, "device-side wait timed out"
    return out.cpu()


def test_tma_swizzle128_layout(mdn):
    import torch
    a = torch.arange(64 * 128, dtype=torch.float32).reshape(64, 128).remainder(251).to(torch.bfloat16)
    raw = run(mdn, 0, a, None, (4096,)).view(torch.int16).numpy().view(np.uint16)        # 8192 bf16
    expect = np.zeros(8192, dtype=np.uint16)
    bits = a.view(torch.int16).numpy().view(np.uint16)
    for r in range(64):
        for c in range(128):
            blk, cc = divmod(c, 64)
            off = blk * 8192 + r * 128 + (((cc >> 3) ^ (r & 7)) * 16) + (cc & 7) * 2
            expect[off // 2] = bits[r, c]
    assert np.array_equal(raw, expect)


def test_mma_smem_smem_kmajor(mdn):
    rng = np.random.default_rng(0)
    a, b = bf16_mat(rng, (128, 128)), bf16_mat(rng, (64, 128))
    out = run(mdn, 1, a, b, (128, 64))
    ref = a.float() @ b.float().T
    assert (out - ref).abs().max() < 1e-3


def test_mma_tmem_a_kmajor_b(mdn):
    rng = np.random.default_rng(1)
    a, b = bf16_mat(rng, (128, 64)), bf16_mat(rng, (64, 64))
    out = run(mdn, 2, a, b, (128, 64))
    ref = a.float() @ b.float().T
    assert (out - ref).abs().max() < 1e-3


def test_mma_tmem_a_mnmajor_b_negate_accumulate(mdn):
    rng = np.random.default_rng(2)
    a, b = bf16_mat(rng, (128, 64)), bf16_mat(rng, (64, 128))
    out = run(mdn, 3, a, b, (128, 128))
    ref = 1.0 - a.float() @ b.float()
    assert (out - ref).abs().max() < 1e-3


def test_mma_m64_data_path_layout(mdn):
    """M = 64 (a 64-row product, e.g. the 64 tokens of a chunk as rows): row r of the result lies in tensor-memory
    lane 32 (r // 16) + r % 16 - sixteen lanes of each 32-lane quarter - and the other lanes are left untouched."""
    rng = np.random.default_rng(5)
    a, b = bf16_mat(rng, (64, 128)), bf16_mat(rng, (128, 128))
    out = run(mdn, 4, a, b, (128, 128)).numpy()
    ref = (a.float() @ b.float().T).numpy()
    for lane in range(128):
        q, i = divmod(lane, 32)
        if i < 16:
            assert np.abs(out[lane] - ref[16 * q + i]).max() < 1e-3, lane
        else:
            assert np.all(out[lane] == -777.0), lane


def test_mma_m64_state_image_as_mn_major_b(mdn):
    """A 64-row product against a kept chunk state read in place: B[j][d] in the state's shared-memory image (two
    blocks of key-index halves, 128-byte swizzle) through an MN-major descriptor, sixteen rows of j per K step."""
    rng = np.random.default_rng(6)
    a, b = bf16_mat(rng, (64, 128)), bf16_mat(rng, (128, 128))
    out = run(mdn, 5, a, b, (64, 128))
    ref = a.float() @ b.float()
    assert (out - ref).abs().max() < 1e-3
