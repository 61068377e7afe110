"""Shared test plumbing: numpy inputs -> torch CUDA tensors, error metric, oracle calls."""
from __future__ import annotations

import numpy as np

import mdn_workloads as wl


def to_torch(inp, device="cuda", host_pinned=False):
    """Device (or pinned host) tensors for the CUDA path from make_inputs() output."""
    import torch
    w = inp["workload"]

    def place(t):
        if host_pinned:
            return t.pin_memory()
        return t.to(device)

    def data(x):
        t = torch.from_numpy(np.ascontiguousarray(x))
        if w.dtype == "bf16":
            t = t.to(torch.bfloat16)     # exact: values are already bf16-representable
        return place(t)

    def f32(x):
        return None if x is None else place(torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)))

    out = dict(q=data(inp["q"]), k=data(inp["k"]), v=data(inp["v"]), beta=f32(inp["beta"]),
               log_alpha=f32(inp["log_alpha"]), log_mu=f32(inp["log_mu"]), eta=f32(inp["eta"]),
               initial_S=f32(inp["S0"]), initial_M=f32(inp["M0"]), cu_seqlens=None)
    if inp["cu_seqlens"] is not None:
        out["cu_seqlens"] = place(torch.from_numpy(inp["cu_seqlens"].astype(np.int32)))
    return out


def run_gpu(mdn, inp, **kw):
    t = to_torch(inp)
    o, S, M = mdn.chunk_fwd(t["q"], t["k"], t["v"], t["beta"], t["log_alpha"], t["log_mu"], t["eta"],
                            initial_S=t["initial_S"], initial_M=t["initial_M"], cu_seqlens=t["cu_seqlens"],
                            scale=inp["scale"], **kw)
    import torch
    torch.cuda.synchronize()
    return (o.float().cpu().numpy().astype(np.float64), S.cpu().numpy().astype(np.float64),
            M.cpu().numpy().astype(np.float64))


def run_oracle(inp, chains=None):
    import oracle
    return oracle.stepwise(inp["q"], inp["k"], inp["v"], inp["beta"], inp["log_alpha"], inp["log_mu"], inp["eta"],
                           scale=inp["scale"], S0=inp["S0"], M0=inp["M0"], seq_start=inp["seq_start"],
                           seq_len=inp["seq_len"], chains=chains)


def rel_err(x, ref):
    """max |x - ref| / RMS(ref) over the entries the oracle evaluated (non-NaN in ref)."""
    mask = ~np.isnan(ref)
    assert mask.any()
    assert np.isfinite(x[mask]).all(), "non-finite value in the result"
    rms = np.sqrt(np.mean(ref[mask] ** 2))
    diff = np.abs(x[mask] - ref[mask]).max()
    if rms == 0.0:
        assert diff == 0.0
        return 0.0
    return float(diff / rms)


def bf16_floor(ref):
    """max |bf16(ref) - ref| / RMS(ref): what storing the exact result in bf16 already costs."""
    mask = ~np.isnan(ref)
    r = ref[mask]
    rb = wl.round_to_bf16(r.astype(np.float32)).astype(np.float64)
    return float(np.abs(rb - r).max() / np.sqrt(np.mean(r ** 2)))


def chain_mask_tokens(inp, chains):
    """Boolean [B,T,H] mask of the (token, head) pairs that belong to the given chains."""
    w = inp["workload"]
    m = np.zeros((w.B * w.T, w.H), dtype=bool)
    for c in chains:
        n, h = divmod(int(c), w.H)
        s, l = int(inp["seq_start"][n]), int(inp["seq_len"][n])
        m[s:s + l, h] = True
    return m.reshape(w.B, w.T, w.H)
