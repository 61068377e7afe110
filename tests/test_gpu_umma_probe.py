"""Bring-up checks of the tcgen05 / TMA / TMEM building blocks against a host matmul, and a bounded device-side
wait that is made to run out.  The probes live in a test-only library (tests/probe), not in libmdn.so."""
import ctypes
import os
import sys

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

PROBE_DIR = os.path.join(os.path.dirname(os.path.abspath(__file__)), "probe")


@pytest.fixture(scope="module")
def probe():
    sys.path.insert(0, PROBE_DIR)
    import build_probe
    L = ctypes.CDLL(build_probe.build())
    vp = ctypes.c_void_p
    L.mdn_selftest_umma.restype = ctypes.c_int
    L.mdn_selftest_umma.argtypes = [ctypes.c_int32, vp, vp, vp, vp, vp]
    L.mdn_probe_tf32.restype = ctypes.c_int
    L.mdn_probe_tf32.argtypes = [ctypes.c_int32, vp, vp, vp, vp, vp, vp]
    L.mdn_probe_mma_timing.restype = ctypes.c_int
    L.mdn_probe_mma_timing.argtypes = [ctypes.c_int32] * 5 + [vp, vp, vp]
    L.mdn_probe_bounded_wait.restype = ctypes.c_int
    L.mdn_probe_bounded_wait.argtypes = [ctypes.c_uint32, vp, vp]
    return L


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    import torch
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def bf16_mat(rng, shape):
    import torch
    return torch.from_numpy(rng.standard_normal(shape).astype(np.float32)).to(torch.bfloat16)


def run(probe, mode, a, b, out_shape):
    import torch
    out = torch.full(out_shape, float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    a, b = a.cuda(), (None if b is None else b.cuda())
    assert probe.mdn_selftest_umma(mode, _ptr(a), _ptr(b), _ptr(out), _ptr(status), _stream()) == 0
    torch.cuda.synchronize()
    assert int(status[0]) == 0, "device-side wait timed out"
    return out.cpu()


def run_tf32(probe, mode, a, b, c, out_shape):
    import torch
    out = torch.full(out_shape, float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    dev = [None if x is None else torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda() for x in (a, b, c)]
    assert probe.mdn_probe_tf32(mode, _ptr(dev[0]), _ptr(dev[1]), _ptr(dev[2]), _ptr(out), _ptr(status), _stream()) == 0
    torch.cuda.synchronize()
    assert int(status[0]) == 0, "device-side wait timed out"
    return out.cpu().numpy().astype(np.float64)


def tf32_trunc(x):
    """fp32 -> tf32 as the tensor core reads it: the low 13 mantissa bits dropped."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32) & np.uint32(0xFFFFE000)
    return u.view(np.float32).astype(np.float64)


def test_tma_swizzle128_layout(probe):
    import torch
    a = torch.arange(64 * 128, dtype=torch.float32).reshape(64, 128).remainder(251).to(torch.bfloat16)
    raw = run(probe, 0, a, None, (4096,)).view(torch.int16).numpy().view(np.uint16)        # 8192 bf16
    expect = np.zeros(8192, dtype=np.uint16)
    bits = a.view(torch.int16).numpy().view(np.uint16)
    for r in range(64):
        for c in range(128):
            blk, cc = divmod(c, 64)
            off = blk * 8192 + r * 128 + (((cc >> 3) ^ (r & 7)) * 16) + (cc & 7) * 2
            expect[off // 2] = bits[r, c]
    assert np.array_equal(raw, expect)


def test_mma_smem_smem_kmajor(probe):
    rng = np.random.default_rng(0)
    a, b = bf16_mat(rng, (128, 128)), bf16_mat(rng, (64, 128))
    out = run(probe, 1, a, b, (128, 64))
    ref = a.float() @ b.float().T
    assert (out - ref).abs().max() < 1e-3


def test_mma_tmem_a_kmajor_b(probe):
    rng = np.random.default_rng(1)
    a, b = bf16_mat(rng, (128, 64)), bf16_mat(rng, (64, 64))
    out = run(probe, 2, a, b, (128, 64))
    ref = a.float() @ b.float().T
    assert (out - ref).abs().max() < 1e-3


def test_mma_tmem_a_mnmajor_b_negate_accumulate(probe):
    rng = np.random.default_rng(2)
    a, b = bf16_mat(rng, (128, 64)), bf16_mat(rng, (64, 128))
    out = run(probe, 3, a, b, (128, 128))
    ref = 1.0 - a.float() @ b.float()
    assert (out - ref).abs().max() < 1e-3


def test_mma_m64_data_path_layout(probe):
    """M = 64 (a 64-row product, e.g. the 64 tokens of a chunk as rows): row r of the result lies in tensor-memory
    lane 32 (r // 16) + r % 16 - sixteen lanes of each 32-lane quarter - and the other lanes are left untouched."""
    rng = np.random.default_rng(5)
    a, b = bf16_mat(rng, (64, 128)), bf16_mat(rng, (128, 128))
    out = run(probe, 4, a, b, (128, 128)).numpy()
    ref = (a.float() @ b.float().T).numpy()
    for lane in range(128):
        q, i = divmod(lane, 32)
        if i < 16:
            assert np.abs(out[lane] - ref[16 * q + i]).max() < 1e-3, lane
        else:
            assert np.all(out[lane] == -777.0), lane


def test_mma_m64_state_image_as_mn_major_b(probe):
    """A 64-row product against a kept chunk state read in place: B[j][d] in the state's shared-memory image (two
    blocks of key-index halves, 128-byte swizzle) through an MN-major descriptor, sixteen rows of j per K step."""
    rng = np.random.default_rng(6)
    a, b = bf16_mat(rng, (64, 128)), bf16_mat(rng, (128, 128))
    out = run(probe, 5, a, b, (64, 128))
    ref = a.float() @ b.float()
    assert (out - ref).abs().max() < 1e-3


# ------------------------------------------------------------------------------------------ kind::tf32
def test_tf32_tmem_a_kmajor_b(probe):
    """fp32 operands read as tf32 (10-bit mantissa): A from tensor memory, B K-major fp32 blocks."""
    rng = np.random.default_rng(7)
    a, b = rng.standard_normal((128, 128)), rng.standard_normal((64, 128))
    out = run_tf32(probe, 0, a, b, None, (128, 64))
    exact = a.astype(np.float32).astype(np.float64) @ b.astype(np.float32).astype(np.float64).T
    trunc = tf32_trunc(a) @ tf32_trunc(b).T
    scale = np.sqrt(128.0)
    assert np.abs(out - exact).max() < 4e-3 * scale          # tf32 rounding of both operands
    print("tf32 product: max |out - truncated-operand product| %.3e, |out - exact| %.3e"
          % (np.abs(out - trunc).max(), np.abs(out - exact).max()))


def test_tf32_tmem_a_mnmajor_b(probe):
    rng = np.random.default_rng(8)
    a, b = rng.standard_normal((128, 64)), rng.standard_normal((64, 128))
    out = run_tf32(probe, 1, a, b, None, (128, 128))
    exact = a.astype(np.float32).astype(np.float64) @ b.astype(np.float32).astype(np.float64)
    # reported, not asserted: no kernel of the library reads a tf32 operand MN-major (measured on B200: this
    # descriptor form gives an all-zero result, so the kernels keep fp32 tiles K-major)
    print("tf32 MN-major B: max |out - exact| %.3e, max |out| %.3e" % (np.abs(out - exact).max(), np.abs(out).max()))


def test_tf32_product_reading_the_previous_accumulator(probe):
    """Y = (A B^T) C^T with the second product's A operand = the first one's accumulator in tensor memory.
    With a commit + wait in between (mode 3) the result must be right; issued back to back (mode 2) it must be the
    same bit for bit: the tensor pipe runs one thread's products in issue order."""
    rng = np.random.default_rng(9)
    a, b, c = rng.standard_normal((128, 128)), rng.standard_normal((64, 128)), rng.standard_normal((64, 64))
    x = a.astype(np.float32).astype(np.float64) @ b.astype(np.float32).astype(np.float64).T
    exact = x @ c.astype(np.float32).astype(np.float64).T
    tol = 4e-3 * np.sqrt(128.0 * 64.0) * 2
    waited = run_tf32(probe, 3, a, b, c, (128, 64))
    assert np.abs(waited - exact).max() < tol
    chained = run_tf32(probe, 2, a, b, c, (128, 64))
    print("back-to-back dependent products: max |chained - waited| %.3e (0 = the pipe ordered them)"
          % np.abs(chained - waited).max())
    assert np.array_equal(chained, waited)          # the chain kernel relies on it (chain_tf32.cu, MMA issuer)


def test_product_overwriting_the_previous_products_operand(probe):
    """Write-after-read through the pipe: a product issued right behind another one overwrites the columns that one
    reads its A operand from; the first result must still be the product of the ORIGINAL operand (the chain kernel
    issues dependent products back to back and relies on the pipe running them in issue order)."""
    rng = np.random.default_rng(10)
    a, b = rng.standard_normal((128, 128)), rng.standard_normal((64, 128))
    plain = run_tf32(probe, 0, a, b, None, (128, 64))
    raced = run_tf32(probe, 9, a, b, None, (128, 64))
    assert np.array_equal(plain, raced)


def test_tf32_issue_to_completion_timings(probe):
    names = {4: "tf32 A=tmem N=64", 5: "tf32 A=tmem N=128 MN-major B", 6: "bf16 A=smem N=64",
             7: "tf32 A=tmem N=64, commit+wait per 16"}
    for mode, name in names.items():
        out = run_tf32(probe, mode, None, None, None, (2,))
        assert out[1] > 0 and out[0] > 0
        print("%-40s %6.1f cycles per product (%d products)" % (name, out[0] / out[1], int(out[1])))


def test_issuer_timeline_around_a_commit(probe):
    out = run_tf32(probe, 8, None, None, None, (20,))
    print("issuing thread, cycles since first issue: 8 products issued %d, commit %d, wait on a complete barrier %d, "
          "fence %d, 8 more issued %d, first commit seen %d, second %d" % tuple(int(x) for x in out[:7]))
    print("nothing in flight: wait on a complete barrier %d, one poll %d; 8 products issued %d, then a relaxed poll %d, "
          "an acquire poll %d" % tuple(int(x) for x in out[7:12]))
    print("in flight: 8 issued %d, commit %d, fence %d, 8 more issued %d, commit %d, poll %d, fence %d, one more issued %d"
          % tuple(int(x) for x in out[12:20]))
    assert out[6] > 0


def test_product_cost_by_shape(probe):
    """Cycles per tcgen05 product (M = 128) by kind, A source and N: printed for the design notes; asserts only that
    every shape completes and that a product never gets cheaper when N grows."""
    import torch
    for m in (128, 64):
        for tf32 in (0, 1):
            for a_tmem in (0, 1):
                row, issue = [], []
                for n in (32, 64, 128, 256):
                    out = torch.zeros(4, dtype=torch.float32, device="cuda")
                    status = torch.zeros(4, dtype=torch.int32, device="cuda")
                    assert probe.mdn_probe_mma_timing(tf32, a_tmem, n, m, 256, _ptr(out), _ptr(status), _stream()) == 0
                    torch.cuda.synchronize()
                    assert int(status[0]) == 0
                    row.append(float(out[0]) / float(out[1]))
                    issue.append(float(out[2]) / float(out[1]))
                print("M = %3d, %s, A from %s: cycles per product at N = 32, 64, 128, 256: %s"
                      % (m, "tf32 K=8 " if tf32 else "bf16 K=16", "tensor memory" if a_tmem else "shared memory",
                         ", ".join("%.1f" % x for x in row)) + "  (issuing thread alone: %s)" % ", ".join("%.1f" % x for x in issue))
                assert row[3] >= row[1] * 0.9
    # the state update's form: bf16, A from tensor memory, B a [64 x 128] tile read MN-major (N = 128 only)
    out = torch.zeros(4, dtype=torch.float32, device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    assert probe.mdn_probe_mma_timing(0, 2, 128, 128, 256, _ptr(out), _ptr(status), _stream()) == 0
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    print("M = 128, bf16 K=16, A from tensor memory, B MN-major, N = 128: %.1f cycles per product" % (float(out[0]) / float(out[1])))
    assert probe.mdn_probe_mma_timing(1, 3, 128, 128, 256, _ptr(out), _ptr(status), _stream()) == 0
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    print("M = 128, tf32, A = 128 columns of tensor memory, B = 64 KB in four panels (the chain kernel's first product), "
          "N = 128: %.1f cycles per product" % (float(out[0]) / float(out[1])))


# ------------------------------------------------------------------------------------------ bounded waits
def test_bounded_wait_runs_out_and_the_context_stays_usable(probe):
    """Every device-side wait of the library is bounded: a wait whose partner never arrives gives up, sets the
    status word and lets the kernel return.  Here nothing ever arrives at the barrier; afterwards an ordinary
    forward gives bit-identical results to one run before."""
    import torch
    import mdn_workloads as wl
    import paper_2605_05838_b200 as mdn
    from helpers import run_gpu
    w = wl.Workload("after_timeout", B=1, T=200, H=2, dk=128, dv=128, dtype="bf16", seed=5)
    inp = wl.make_inputs(w)
    before = run_gpu(mdn, inp)
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    assert probe.mdn_probe_bounded_wait(2000, _ptr(status), _stream()) == 0
    torch.cuda.synchronize()                          # returns: the kernel ended by itself
    assert int(status[0]) == 2 and int(status[1]) == 1          # kDevTimeout; the second waiter saw the abort flag
    assert mdn.status_string(5) == "device-side wait timed out"
    after = run_gpu(mdn, inp)
    for x, y in zip(before, after):
        assert np.array_equal(x, y)
