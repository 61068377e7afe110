"""The forward that keeps the chunk-start states (what a chunk-parallel backward starts from) against the fp64
oracle: the state at the start of chunk c of a sequence is the oracle's final state after the sequence's first
64 c tokens."""
import numpy as np
import pytest

import mdn_workloads as wl
from helpers import bf16_floor, rel_err, run_oracle, to_torch

pytestmark = pytest.mark.gpu

# The kept states are the forward's own bf16 operand copies: storing the EXACT state in bf16 already costs
# bf16_floor(ref) in the max-abs / RMS metric; on top of that the forward's state error (about 1e-3) is allowed.
TOL_OVER_FLOOR = 5e-3


@pytest.fixture(scope="module")
def mdn():
    import paper_2605_05838_b200 as m
    m.lib()          # raises if the CUDA library is missing: no fallback
    return m


def oracle_chunk_start_states(inp):
    """[slots][H][dk][dv] in the workspace's slot order (sequence after sequence, chunk after chunk)."""
    lens = np.asarray(inp["seq_len"])
    nch = (lens + 63) // 64
    S_all, M_all = [], []
    for c in range(int(nch.max())):
        cut = dict(inp)
        cut["seq_len"] = np.minimum(lens, 64 * c).astype(lens.dtype)
        _, S, M = run_oracle(cut)
        S_all.append(S)
        M_all.append(M)
    S_out, M_out = [], []
    for s in range(len(lens)):
        for c in range(int(nch[s])):
            S_out.append(S_all[c][s])
            M_out.append(M_all[c][s])
    return np.stack(S_out), np.stack(M_out)


@pytest.mark.parametrize("name, kw", [
    ("fixed", dict(B=2, T=64 * 5 + 17, init_state_std=0.1)),
    ("packed", dict(B=1, T=700, varlen=True, len_lo=30, len_hi=260, init_state_std=0.1)),
])
def test_keep_chunk_states(mdn, name, kw):
    import torch
    w = wl.Workload("keep_" + name, H=2, dk=128, dv=128, dtype="bf16", seed=81, **kw)
    inp = wl.make_inputs(w)
    t = to_torch(inp)
    o, S, M, states, _ = mdn.chunk_fwd(t["q"], t["k"], t["v"], t["beta"], t["log_alpha"], t["log_mu"], t["eta"],
                                       initial_S=t["initial_S"], initial_M=t["initial_M"], cu_seqlens=t["cu_seqlens"],
                                       scale=inp["scale"], path="tensor", o_dtype=torch.float32, keep_chunk_states=True)
    o1, S1, M1 = mdn.chunk_fwd(t["q"], t["k"], t["v"], t["beta"], t["log_alpha"], t["log_mu"], t["eta"],
                               initial_S=t["initial_S"], initial_M=t["initial_M"], cu_seqlens=t["cu_seqlens"],
                               scale=inp["scale"], path="tensor", o_dtype=torch.float32, segments=1)
    # the kept states change nothing else
    assert torch.equal(o, o1) and torch.equal(S, S1) and torch.equal(M, M1)
    Sc, Mc = mdn.unpack_chunk_states(states, w.H)
    S_ref, M_ref = oracle_chunk_start_states(inp)
    n = S_ref.shape[0]
    es, em = rel_err(Sc[:n].cpu().numpy(), S_ref), rel_err(Mc[:n].cpu().numpy(), M_ref)
    fs, fm = bf16_floor(S_ref), bf16_floor(M_ref)
    print("chunk-start states (%s, %d slots): S %.3e (bf16 floor %.3e) M %.3e (floor %.3e)" % (name, n, es, fs, em, fm))
    assert es <= fs + TOL_OVER_FLOOR and em <= fm + TOL_OVER_FLOOR
