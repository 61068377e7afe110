"""Canary words around everything the forward writes: the workspace, `o` and the two final states each sit inside a
larger buffer filled with a pattern, and after the call every byte outside the region handed to the library must
still hold the pattern.  A kernel that stores past the end of a short chunk, of the last sequence, of a segment's
scratch or of its slice of the workspace shows up here (compute-sanitizer is not available on the test machines)."""
import ctypes

import numpy as np
import pytest

import mdn_workloads as wl
from helpers import to_torch

pytestmark = pytest.mark.gpu

GUARD = 4096        # bytes on each side, a multiple of the 256-byte workspace alignment
PATTERN = 0xA5


@pytest.fixture(scope="module")
def mdn():
    import paper_2605_05838_b200 as m
    m.lib()
    return m


def guarded(nbytes, dtype, shape):
    import torch
    buf = torch.full((nbytes + 2 * GUARD,), PATTERN, dtype=torch.uint8, device="cuda")
    return buf, buf[GUARD:GUARD + nbytes].view(dtype).view(shape)


def guards_intact(buf, nbytes):
    return bool((buf[:GUARD] == PATTERN).all()) and bool((buf[GUARD + nbytes:] == PATTERN).all())


CASES = [
    ("fixed bf16, ragged T", dict(B=2, T=200, H=3, dk=128, dv=128, dtype="bf16", seed=31), None, 0, "tensor"),
    ("fixed bf16, one short chunk", dict(B=1, T=5, H=2, dk=128, dv=128, dtype="bf16", seed=32), None, 0, "tensor"),
    ("packed bf16", dict(B=1, T=70 + 1 + 129 + 300 + 64, H=2, dk=128, dv=128, dtype="bf16", varlen=True, seed=33),
     [70, 1, 129, 300, 64], 0, "tensor"),
    ("segments forced", dict(B=1, T=64 * 40, H=2, dk=128, dv=128, dtype="bf16", seed=34, init_state_std=0.1), None, 4, "tensor"),
    ("fp32 SIMT", dict(B=2, T=130, H=2, dk=64, dv=64, dtype="f32", seed=35), None, 0, "simt"),
    ("packed fp32 SIMT", dict(B=1, T=63 + 65 + 2, H=2, dk=64, dv=64, dtype="f32", varlen=True, seed=36), [63, 65, 2], 0, "simt"),
]


@pytest.mark.parametrize("name,wkw,lens,segments,path", CASES, ids=[c[0] for c in CASES])
def test_nothing_is_written_outside_the_buffers_handed_over(mdn, name, wkw, lens, segments, path):
    import torch
    w = wl.Workload("canary", **wkw)
    inp = wl.make_inputs(w, lengths=np.array(lens)) if lens is not None else wl.make_inputs(w)
    t = to_torch(inp)
    N = len(inp["seq_len"])
    o_dtype = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    p = mdn.make_params(t["q"], t["v"], num_seqs=(N if w.varlen else 0), scale=inp["scale"], o_dtype=o_dtype, path=path,
                        segments=segments)
    es = 2 if w.dtype == "bf16" else 4
    ws_bytes = mdn.workspace_bytes(p)
    o_bytes = w.B * w.T * w.H * w.dv * es
    st_bytes = N * w.H * w.dk * w.dv * 4
    ws_buf, ws = guarded(ws_bytes, torch.uint8, (ws_bytes,))
    o_buf, o = guarded(o_bytes, o_dtype, (w.B, w.T, w.H, w.dv))
    S_buf, S = guarded(st_bytes, torch.float32, (N, w.H, w.dk, w.dv))
    M_buf, M = guarded(st_bytes, torch.float32, (N, w.H, w.dk, w.dv))
    vp = lambda x: None if x is None else ctypes.c_void_p(x.data_ptr())
    for _ in range(2):
        st = mdn.lib().mdn_chunk_fwd(ctypes.byref(p), vp(t["q"]), vp(t["k"]), vp(t["v"]), vp(t["beta"]), vp(t["log_alpha"]),
                                     vp(t["log_mu"]), vp(t["eta"]), vp(t["initial_S"]), vp(t["initial_M"]),
                                     vp(t["cu_seqlens"]), vp(o), vp(S), vp(M), vp(ws), ws_bytes, None)
        assert st == 0
        torch.cuda.synchronize()
        assert mdn.read_status(p, ws) == 0
    assert guards_intact(ws_buf, ws_bytes), "workspace"
    assert guards_intact(o_buf, o_bytes), "o"
    assert guards_intact(S_buf, st_bytes) and guards_intact(M_buf, st_bytes), "final states"
    # and the call wrote what it should: the same result as through the binding's own buffers
    o_ref, S_ref, M_ref = mdn.chunk_fwd(t["q"], t["k"], t["v"], t["beta"], t["log_alpha"], t["log_mu"], t["eta"],
                                        initial_S=t["initial_S"], initial_M=t["initial_M"], cu_seqlens=t["cu_seqlens"],
                                        scale=inp["scale"], o_dtype=o_dtype, path=path, segments=segments)
    assert torch.equal(o, o_ref) and torch.equal(S, S_ref) and torch.equal(M, M_ref)


@pytest.mark.parametrize("o_bf16", [True, False])
def test_fused_layer_operations_stay_inside_their_buffers(mdn, o_bf16):
    """The forward with all three layer operations inside the kernels (the output step stages an fp32 tile over
    several areas of a stage and, for a short chunk, stores row by row): a batch whose last chunk is short."""
    import torch
    w = wl.Workload("canary_layer", B=2, T=200, H=2, dk=128, dv=128, dtype="bf16", seed=41)
    inp = wl.make_layer_inputs(w)
    dt = torch.bfloat16
    dev = lambda x, d=torch.float32: torch.from_numpy(np.ascontiguousarray(x)).to("cuda").to(d)
    q, k, v, g = dev(inp["q"], dt), dev(inp["k"], dt), dev(inp["v"], dt), dev(inp["g"], dt)
    gates = [dev(inp[n]) for n in ("x_beta", "x_alpha", "x_mu", "x_eta")]
    gp = dict(a_alpha=dev(inp["a_alpha"]), b_alpha=dev(inp["b_alpha"]), a_mu=dev(inp["a_mu"]), b_mu=dev(inp["b_mu"]),
              s=inp["s"], tau=inp["tau"], log_mu_min=inp["log_mu_min"])
    ops = mdn.make_layer_ops(q, v, gate_param=gp, qk_norm=dict(d=dev(inp["d"]), eps=inp["qk_eps"]),
                             out_norm_gate=dict(g=g, w=dev(inp["w_norm"]), eps=inp["rms_eps"]), placement="fused")
    o_dtype = torch.bfloat16 if o_bf16 else torch.float32
    p = mdn.make_params(q, v, scale=inp["scale"], o_dtype=o_dtype, path="tensor")
    ws_bytes = int(mdn.lib().mdn_chunk_fwd_fused_workspace_bytes(ctypes.byref(p), ctypes.byref(ops)))
    o_bytes = w.B * w.T * w.H * w.dv * (2 if o_bf16 else 4)
    ws_buf, ws = guarded(ws_bytes, torch.uint8, (ws_bytes,))
    o_buf, o = guarded(o_bytes, o_dtype, (w.B, w.T, w.H, w.dv))
    for _ in range(2):
        mdn.chunk_fwd(q, k, v, *gates, scale=inp["scale"], o_dtype=o_dtype, path="tensor", layer_ops=ops,
                      workspace=ws, out=o)
        torch.cuda.synchronize()
    assert guards_intact(ws_buf, ws_bytes), "workspace"
    assert guards_intact(o_buf, o_bytes), "o"
    assert torch.isfinite(o.float()).all()
