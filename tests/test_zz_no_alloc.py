"""mdn_chunk_fwd_static_scratch, the entry point for callers that cannot allocate device memory
(an inference server whose arena owns all device memory, a plugin whose host forbids allocator
calls): same result as mdn_chunk_fwd, scratch taken from the library's built-in array.

Collected last on purpose: a run that stops at the first failure has then already run every other
test.  Two calls in a row check that whatever the first call left in the shared array does not
leak into the second."""
import numpy as np
import pytest

import mdn_workloads as wl
from helpers import to_torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mdn():
    import paper_2605_05838_b200 as m
    m.lib()
    return m


first_call = [True]


def both_ways(mdn, inp, path):
    import torch
    t = to_torch(inp)
    kw = dict(initial_S=t["initial_S"], initial_M=t["initial_M"], cu_seqlens=t["cu_seqlens"], scale=inp["scale"],
              path=path)
    o_ref, S_ref, M_ref = mdn.chunk_fwd(t["q"], t["k"], t["v"], t["beta"], t["log_alpha"], t["log_mu"], t["eta"], **kw)
    o = torch.full_like(o_ref, float("nan"))
    S = torch.full_like(S_ref, float("nan"))
    M = torch.full_like(M_ref, float("nan"))
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    free_before = torch.cuda.mem_get_info()[0]
    mdn.chunk_fwd_static_scratch(t["q"], t["k"], t["v"], t["beta"], t["log_alpha"], t["log_mu"], t["eta"],
                                 out=o, final_S=S, final_M=M, **kw)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before          # nothing was allocated through torch ...
    # ... nor behind its back: the driver's count of free device memory has not gone down (the very first call
    # of a process may load the kernels' code, so the comparison is made on a repeat call)
    if not first_call[0]:
        assert torch.cuda.mem_get_info()[0] >= free_before
    first_call[0] = False
    return (o.float().cpu().numpy(), S.cpu().numpy(), M.cpu().numpy(),
            o_ref.float().cpu().numpy(), S_ref.cpu().numpy(), M_ref.cpu().numpy())


def test_static_scratch_matches_workspace_entry_point_twice_in_a_row(mdn):
    first = wl.Workload("noalloc_a", B=2, T=200, H=3, dk=64, dv=64, dtype="f32", init_state_std=0.3, seed=21)
    lens = np.array([70, 1, 129, 300])
    second = wl.Workload("noalloc_b", B=1, T=int(lens.sum()), H=2, dk=128, dv=128, dtype="bf16", varlen=True, seed=22)
    for w, inp in ((first, wl.make_inputs(first)), (second, wl.make_inputs(second, lengths=lens))):
        paths = ["simt"] + (["tensor"] if w.dtype == "bf16" else [])
        for path in paths:
            for _ in range(2):      # twice in a row: what the first call left in the shared array must not leak
                o, S, M, o_ref, S_ref, M_ref = both_ways(mdn, inp, path)
                assert np.isfinite(o).all() and np.isfinite(S).all() and np.isfinite(M).all()
                # the same kernels on the same inputs, and the forward is bit-reproducible: the tolerance the
                # parity tests use for this dtype (1e-4 / 2e-2 of the RMS) is met with zero difference
                assert np.array_equal(o, o_ref) and np.array_equal(S, S_ref) and np.array_equal(M, M_ref)


def test_static_scratch_rejects_problems_beyond_its_fixed_size(mdn):
    import torch
    w = wl.Workload("noalloc_big", B=8, T=4096, H=16, dk=128, dv=128, dtype="bf16")
    q = torch.empty((w.B, w.T, w.H, w.dk), dtype=torch.bfloat16, device="cuda")
    g = torch.empty((w.B, w.T, w.H), dtype=torch.float32, device="cuda")
    o = torch.empty_like(q)
    assert mdn.workspace_bytes(mdn.make_params(q, q)) > mdn.STATIC_SCRATCH_BYTES
    with pytest.raises(mdn.MdnError) as e:
        mdn.chunk_fwd_static_scratch(q, q, q, g, g, g, None, out=o)
    assert e.value.status == 6 and "static" in str(e.value)


def test_static_scratch_reports_bad_parameters_like_the_workspace_entry_point(mdn):
    import ctypes
    import torch
    q = torch.empty((1, 64, 2, 64), dtype=torch.float32, device="cuda")
    g = torch.empty((1, 64, 2), dtype=torch.float32, device="cuda")
    ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    vp = lambda t: ctypes.c_void_p(t.data_ptr())
    for field, value in (("B", 0), ("chunk", 32), ("io_dtype", 7), ("num_seqs", 3)):
        p = mdn.make_params(q, q)
        setattr(p, field, value)
        a = mdn.lib().mdn_chunk_fwd(ctypes.byref(p), vp(q), vp(q), vp(q), vp(g), vp(g), vp(g), None, None, None, None,
                                    vp(q), None, None, vp(ws), ws.numel(), None)
        b = mdn.lib().mdn_chunk_fwd_static_scratch(ctypes.byref(p), vp(q), vp(q), vp(q), vp(g), vp(g), vp(g), None, None,
                                                   None, None, vp(q), None, None, None)
        assert a == b and a in (1, 2), (field, a, b)
