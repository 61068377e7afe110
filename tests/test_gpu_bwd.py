"""mdn_chunk_bwd against the fp64 backward oracle (reverse mode through the stepwise recurrence), element by
element on the same seeded inputs.  The CUDA backward computes in fp32 whatever the i/o dtype, so every case is held
to the fp32 bound: max |g - ref| / RMS(ref) <= 1e-4 per gradient tensor."""
import numpy as np
import pytest

import mdn_workloads as wl
from helpers import rel_err

pytestmark = pytest.mark.gpu

TOL = 1e-4
NAMES = [("dq", "dq"), ("dk", "dk"), ("dv", "dv"), ("dbeta", "dbeta"), ("dlog_alpha", "dlog_alpha"),
         ("dlog_mu", "dlog_mu"), ("deta", "deta"), ("d_initial_S", "dS0"), ("d_initial_M", "dM0")]


@pytest.fixture(scope="module")
def mdn():
    import paper_2605_05838_b200 as m
    m.lib()
    return m


def upstream(w, inp, seed):
    """Seeded upstream gradients dL/do, dL/dS_T, dL/dM_T (inputs of the backward, not part of the method)."""
    r = np.random.default_rng([seed, 77])
    N = len(inp["seq_len"])
    d_o = r.standard_normal((w.B, w.T, w.H, w.dv)).astype(np.float32)
    if w.dtype == "bf16":
        d_o = wl.round_to_bf16(d_o)
    dS = (0.1 * r.standard_normal((N, w.H, w.dk, w.dv))).astype(np.float32)
    dM = (0.1 * r.standard_normal((N, w.H, w.dk, w.dv))).astype(np.float32)
    return d_o, dS, dM


def run_both(mdn, inp, d_o, dS, dM, chains=None, eta_none=False):
    import oracle
    import torch
    w = inp["workload"]
    eta = None if eta_none else inp["eta"]
    ref = oracle.stepwise_bwd(inp["q"], inp["k"], inp["v"], inp["beta"], inp["log_alpha"], inp["log_mu"], eta, d_o,
                              scale=inp["scale"], S0=inp["S0"], M0=inp["M0"], dS_final=dS, dM_final=dM,
                              seq_start=inp["seq_start"], seq_len=inp["seq_len"], chains=chains)
    dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    dev = lambda x, d=torch.float32: None if x is None else torch.from_numpy(np.ascontiguousarray(x)).to("cuda").to(d)
    cu = None if inp["cu_seqlens"] is None else torch.from_numpy(inp["cu_seqlens"]).to("cuda")
    got = mdn.chunk_bwd(dev(inp["q"], dt), dev(inp["k"], dt), dev(inp["v"], dt), dev(inp["beta"]), dev(inp["log_alpha"]),
                        dev(inp["log_mu"]), dev(eta), dev(d_o, dt), initial_S=dev(inp["S0"]), initial_M=dev(inp["M0"]),
                        cu_seqlens=cu, d_final_S=dev(dS), d_final_M=dev(dM), scale=inp["scale"])
    torch.cuda.synchronize()
    return got, ref


def check(got, ref, label):
    errs = {}
    for gname, rname in NAMES:
        if ref[rname] is None:
            assert got[gname] is None
            continue
        errs[gname] = rel_err(got[gname].cpu().numpy().astype(np.float64), ref[rname])
    print(label, " ".join("%s %.2e" % kv for kv in errs.items()))
    assert max(errs.values()) <= TOL, errs


@pytest.mark.parametrize("T", [1, 2, 63, 64, 65, 150, 257])
def test_fp32_lengths(mdn, T):
    w = wl.Workload("bwd_f32", B=2, T=T, H=3, dk=64, dv=64, dtype="f32", init_state_std=0.3, seed=60)
    inp = wl.make_inputs(w)
    check(*run_both(mdn, inp, *upstream(w, inp, T)), "fp32 T=%d" % T)


@pytest.mark.parametrize("dk,dv,dtype", [(64, 128, "f32"), (128, 64, "f32"), (128, 128, "f32"), (128, 128, "bf16"),
                                         (64, 64, "bf16")])
def test_head_dims_and_dtypes(mdn, dk, dv, dtype):
    w = wl.Workload("bwd_dims", B=1, T=200, H=2, dk=dk, dv=dv, dtype=dtype, init_state_std=0.2, seed=61)
    inp = wl.make_inputs(w)
    check(*run_both(mdn, inp, *upstream(w, inp, dk + dv)), "%s dk%d dv%d" % (dtype, dk, dv))


def test_no_eta_no_state_no_final_grads(mdn):
    w = wl.Workload("bwd_plain", B=2, T=130, H=2, dk=64, dv=64, dtype="f32", seed=62)
    inp = wl.make_inputs(w)
    d_o, _, _ = upstream(w, inp, 1)
    check(*run_both(mdn, inp, d_o, None, None, eta_none=True), "eta=None, zero states")


def test_packed_varlen(mdn):
    w = wl.Workload("bwd_packed", B=1, T=700, H=3, dk=64, dv=64, dtype="f32", varlen=True, len_lo=1, len_hi=200,
                    init_state_std=0.2, seed=63)
    inp = wl.make_inputs(w)
    check(*run_both(mdn, inp, *upstream(w, inp, 2)), "packed")


def test_fast_forgetting_preset_and_degenerate_gates(mdn):
    w = wl.Workload("bwd_F", B=1, T=160, H=2, dk=64, dv=64, dtype="f32", preset="F", init_state_std=0.2, seed=64)
    inp = wl.make_inputs(w)
    inp["k"] = wl.correlated_keys(w, 0.8)
    inp["beta"][:, 10:20] = 0.0
    inp["log_mu"][:, 30:50] = -np.inf          # mu = 0: the division-free formulas must not produce NaN
    check(*run_both(mdn, inp, *upstream(w, inp, 3)), "preset F, beta=0, mu=0 tokens")


def test_config2_full_size_two_chains(mdn):
    """The launch configuration bench.py --backward times (B=8, H=16, T=4096, dk=dv=128, bf16), two sampled chains."""
    w = wl.CONFIGS[2]
    inp = wl.make_inputs(w)
    d_o, dS, dM = upstream(w, inp, 5)
    got, ref = run_both(mdn, inp, d_o, dS, dM, chains=np.array([3, 126]))
    check(got, ref, "config 2 (2 of 128 chains)")


def test_config1_sampled_chains_and_repeatability(mdn):
    import torch
    w = wl.CONFIGS[1]
    inp = wl.make_inputs(w)
    d_o, dS, dM = upstream(w, inp, 4)
    chains = np.array([0, 9, 18, 31])
    got, ref = run_both(mdn, inp, d_o, dS, dM, chains=chains)
    check(got, ref, "config 1 (4 of 32 chains)")
    # a second run differs at most in the last bits (shared-memory floating-point atomics in the column sums)
    again, _ = run_both(mdn, inp, d_o, dS, dM, chains=chains[:1])
    for n, _ in NAMES:
        assert torch.allclose(got[n], again[n], rtol=1e-4, atol=1e-6 * float(got[n].abs().max()))
    for n in ("dv", "d_initial_S", "d_initial_M"):        # no cross-warp sums in these: bit-identical
        assert torch.equal(got[n], again[n])
