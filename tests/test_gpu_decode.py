"""Recurrent decode step (one token, carried S and M) against the fp64 oracle of the same recurrence."""
import dataclasses

import numpy as np
import pytest

import mdn_workloads as wl
from helpers import rel_err, run_gpu, run_oracle, to_torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mdn():
    import paper_2605_05838_b200 as m
    m.lib()
    return m


def decode_all(mdn, inp, S0, M0, o_dtype=None):
    """Feeds the tokens of `inp` one by one through mdn_decode_step."""
    import torch
    w = inp["workload"]
    t = to_torch(inp)
    S = torch.from_numpy(S0.astype(np.float32)).cuda().contiguous()
    M = torch.from_numpy(M0.astype(np.float32)).cuda().contiguous()
    outs = []
    for i in range(w.T):
        sl = slice(i, i + 1)
        eta = None if t["eta"] is None else t["eta"][:, sl].contiguous()
        o = mdn.decode_step(t["q"][:, sl].contiguous(), t["k"][:, sl].contiguous(), t["v"][:, sl].contiguous(),
                            t["beta"][:, sl].contiguous(), t["log_alpha"][:, sl].contiguous(),
                            t["log_mu"][:, sl].contiguous(), eta, S, M, scale=inp["scale"], o_dtype=o_dtype)
        outs.append(o.float())
    torch.cuda.synchronize()
    return (torch.cat(outs, dim=1).cpu().numpy().astype(np.float64), S.cpu().numpy().astype(np.float64),
            M.cpu().numpy().astype(np.float64))


@pytest.mark.parametrize("dtype,dk,dv", [("f32", 64, 64), ("f32", 128, 64), ("bf16", 128, 128), ("bf16", 64, 128)])
def test_decode_steps_match_oracle(mdn, dtype, dk, dv):
    import torch
    w = wl.Workload("decode", B=3, T=40, H=2, dk=dk, dv=dv, dtype=dtype, init_state_std=0.3, seed=41, preset="F")
    inp = wl.make_inputs(w)
    inp["log_mu"][:, 7] = -np.inf          # a mu = 0 token
    inp["beta"][:, 11] = 0.0               # a beta = 0 token
    o_ref, S_ref, M_ref = run_oracle(inp)
    o, S, M = decode_all(mdn, inp, inp["S0"], inp["M0"], o_dtype=torch.float32)
    errs = rel_err(o, o_ref), rel_err(S, S_ref), rel_err(M, M_ref)
    print("decode %s dk%d dv%d: o %.3e S %.3e M %.3e" % (dtype, dk, dv, *errs))
    assert max(errs) <= 1e-4               # fp32 arithmetic on exactly representable inputs


def test_decode_continues_chunk_prefill(mdn):
    """Prefill 200 tokens with mdn_chunk_fwd, decode 8 more: same as the oracle on all 208 tokens."""
    w = wl.Workload("prefill_decode", B=2, T=208, H=2, dk=64, dv=64, dtype="f32", seed=42)
    inp = wl.make_inputs(w)
    o_ref, S_ref, M_ref = run_oracle(inp)
    pre = dict(inp); dec = dict(inp)
    for name in ("q", "k", "v", "beta", "log_alpha", "log_mu", "eta"):
        pre[name] = inp[name][:, :200]; dec[name] = inp[name][:, 200:]
    pre["workload"] = dataclasses.replace(w, T=200); dec["workload"] = dataclasses.replace(w, T=8)
    o_pre, S_pre, M_pre = run_gpu(mdn, pre, path="simt")
    o_dec, S, M = decode_all(mdn, dec, S_pre, M_pre)
    assert rel_err(np.concatenate([o_pre, o_dec], axis=1), o_ref) <= 1e-4
    assert rel_err(S, S_ref) <= 1e-4 and rel_err(M, M_ref) <= 1e-4


def test_decode_rejects_more_than_one_token(mdn):
    import torch
    q = torch.zeros((1, 2, 1, 64), device="cuda")
    g = torch.zeros((1, 2, 1), device="cuda")
    S = torch.zeros((1, 1, 64, 64), device="cuda")
    with pytest.raises(ValueError):
        mdn.decode_step(q, q, q, g, g, g, None, S, S.clone())
