"""mdn_chunk_fwd_fused (Section 3.3 element-wise operations absorbed by the forward) against the fp64 oracle:
oracle.layer_ops (gate parameterisation, q/k pre-processing, output norm + gate) around oracle.stepwise.

Tolerances as for the plain forward: fp32 i/o <= 1e-4, bf16 i/o <= 2e-2, as max |x - ref| / RMS(ref) taken PER HEAD
(max over heads): with per-head decay parameters the heads' outputs differ several-fold in magnitude, each head is
an independent problem, and one global RMS would loosen the bound for the quiet heads and tighten it for the loud
ones.  The "separate passes" mode stores the normalised q, k in the i/o dtype; its reference rounds them the same way
(that intermediate tensor is part of what an unfused pipeline computes)."""
import dataclasses

import numpy as np
import pytest

import mdn_workloads as wl
from helpers import rel_err


def head_err(x, ref, axis):
    """max over heads of max |x - ref| / RMS(ref) within the head (`axis` is the head axis)."""
    return max(rel_err(np.take(x, h, axis=axis), np.take(ref, h, axis=axis)) for h in range(ref.shape[axis])
               if not np.isnan(np.take(ref, h, axis=axis)).all())


def errs3(got, ref):
    return [head_err(got[0], ref[0], 2), head_err(got[1], ref[1], 1), head_err(got[2], ref[2], 1)]


pytestmark = pytest.mark.gpu

TOL_F32 = 1e-4
TOL_BF16 = 2e-2


@pytest.fixture(scope="module")
def mdn():
    import paper_2605_05838_b200 as m
    m.lib()
    return m


def oracle_layer(inp, which, chains=None, round_qk=False):
    """which: subset of {"gates", "qk", "out"}; the rest of the pipeline is the plain forward.
    round_qk: the normalised q, k pass through a bf16 tensor (reference of the separate-passes mode)."""
    import oracle
    from oracle import layer_ops as lo
    q, k = inp["q"], inp["k"]
    if "gates" in which:
        la, lm, be, et = lo.gate_parameterisation(inp["x_alpha"], inp["x_mu"], inp["x_beta"], inp["x_eta"],
                                                  inp["a_alpha"], inp["b_alpha"], inp["a_mu"], inp["b_mu"],
                                                  inp["s"], inp["tau"], inp["log_mu_min"])
    else:
        la, lm, be, et = inp["log_alpha"], inp["log_mu"], inp["beta"], inp["eta"]
    if "qk" in which:
        q, k = lo.qk_preprocess(q, k, inp["d"], inp["qk_eps"])
        if round_qk:
            q, k = wl.round_to_bf16(q.astype(np.float32)), wl.round_to_bf16(k.astype(np.float32))
    o, S, M = oracle.stepwise(q, k, inp["v"], be, la, lm, et, scale=inp["scale"], S0=inp["S0"], M0=inp["M0"],
                              seq_start=inp["seq_start"], seq_len=inp["seq_len"], chains=chains)
    if "out" in which:
        o = lo.output_norm_gate(o, inp["g"], inp["w_norm"], inp["rms_eps"])
    return o, S, M


def run_fused(mdn, inp, which, *, path="auto", placement="fused", o_dtype=None, segments=0):
    import torch
    w = inp["workload"]
    dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    dev = lambda x, d=torch.float32: None if x is None else torch.from_numpy(np.ascontiguousarray(x)).to("cuda").to(d)
    q, k, v = dev(inp["q"], dt), dev(inp["k"], dt), dev(inp["v"], dt)
    if "gates" in which:
        gates = [dev(inp[n]) for n in ("x_beta", "x_alpha", "x_mu", "x_eta")]
        gp = dict(a_alpha=dev(inp["a_alpha"]), b_alpha=dev(inp["b_alpha"]), a_mu=dev(inp["a_mu"]),
                  b_mu=dev(inp["b_mu"]), s=inp["s"], tau=inp["tau"], log_mu_min=inp["log_mu_min"])
    else:
        gates = [dev(inp[n]) for n in ("beta", "log_alpha", "log_mu", "eta")]
        gp = None
    qk = dict(d=dev(inp["d"]), eps=inp["qk_eps"]) if "qk" in which else None
    out = dict(g=dev(inp["g"], dt), w=dev(inp["w_norm"]), eps=inp["rms_eps"]) if "out" in which else None
    ops = mdn.make_layer_ops(q, v, gate_param=gp, qk_norm=qk, out_norm_gate=out, placement=placement)
    cu = None if inp["cu_seqlens"] is None else torch.from_numpy(inp["cu_seqlens"]).to("cuda")
    o, S, M = mdn.chunk_fwd(q, k, v, *gates, initial_S=dev(inp["S0"]), initial_M=dev(inp["M0"]), cu_seqlens=cu,
                            scale=inp["scale"], path=path, o_dtype=o_dtype, layer_ops=ops, segments=segments)
    torch.cuda.synchronize()
    f = lambda t: t.float().cpu().numpy().astype(np.float64)
    return f(o), f(S), f(M)


def compose(w, which, s=0.25):
    """Inputs for a call with the operations in `which` on: un-normalised q, k only when the q/k step is part of
    the call (the recurrence needs |k| = 1), plain gates from the seeded generator when raw_gates is off."""
    inp = wl.make_layer_inputs(w, s=s)
    base = wl.make_inputs(w)
    if "qk" not in which:
        inp["q"], inp["k"] = base["q"], base["k"]
    for name in ("beta", "log_alpha", "log_mu", "eta"):
        inp[name] = base[name]
    return inp


ALL = ("gates", "qk", "out")


@pytest.mark.parametrize("which", [("gates",), ("qk",), ("out",), ALL])
def test_fp32_each_operation_and_all(mdn, which):
    w = wl.Workload("layer_f32", B=2, T=150, H=3, dk=64, dv=64, dtype="f32", init_state_std=0.3, seed=50)
    inp = compose(w, which)
    ref = oracle_layer(inp, which)
    got = run_fused(mdn, inp, which)
    errs = errs3(got, ref)
    print("fp32 %s: o %.3e S %.3e M %.3e" % ("+".join(which), *errs))
    assert max(errs) <= TOL_F32


@pytest.mark.parametrize("dk,dv", [(128, 64), (64, 128), (128, 128)])
def test_fp32_head_dims_all_operations(mdn, dk, dv):
    w = wl.Workload("layer_f32_dims", B=1, T=130, H=2, dk=dk, dv=dv, dtype="f32", seed=51)
    inp = wl.make_layer_inputs(w, s=1.0)
    ref = oracle_layer(inp, ALL)
    got = run_fused(mdn, inp, ALL)
    errs = errs3(got, ref)
    print("fp32 dk%d dv%d: o %.3e S %.3e M %.3e" % (dk, dv, *errs))
    assert max(errs) <= TOL_F32


def tensor_ok(mdn, w):
    p = mdn.MdnParams(w.B, w.T, w.H, w.dk, w.dv, 64, 0, 1, 1, 2, 1.0, 0)
    return w.dtype == "bf16" and mdn.workspace_bytes(p) > 0


@pytest.mark.parametrize("which", [("gates",), ("qk",), ("out",), ALL])
@pytest.mark.parametrize("placement", ["fused", "separate"])
def test_tensor_path_each_operation_and_all(mdn, which, placement):
    import torch
    w = wl.Workload("layer_bf16", B=2, T=300, H=3, dk=128, dv=128, dtype="bf16", init_state_std=0.05, seed=52)
    if not tensor_ok(mdn, w):
        pytest.skip("tensor path not built")
    inp = compose(w, which)
    ref = oracle_layer(inp, which, round_qk=placement == "separate")
    got = run_fused(mdn, inp, which, path="tensor", placement=placement, o_dtype=torch.float32)
    errs = errs3(got, ref)
    print("bf16 %s %s: o %.3e S %.3e M %.3e" % ("+".join(which), placement, *errs))
    assert max(errs) <= TOL_BF16


@pytest.mark.parametrize("T", [1, 63, 64, 65, 129, 200])
def test_tensor_path_fused_ragged_lengths(mdn, T):
    import torch
    w = wl.Workload("layer_ragged", B=2, T=T, H=2, dk=128, dv=128, dtype="bf16", init_state_std=0.2, seed=53)
    if not tensor_ok(mdn, w):
        pytest.skip("tensor path not built")
    inp = wl.make_layer_inputs(w)
    ref = oracle_layer(inp, ALL)
    got = run_fused(mdn, inp, ALL, path="tensor", o_dtype=torch.float32)
    errs = errs3(got, ref)
    print("fused T=%d: o %.3e S %.3e M %.3e" % (T, *errs))
    assert max(errs) <= TOL_BF16
    gb = run_fused(mdn, inp, ALL, path="tensor")                  # bf16 store of y
    for h in range(w.H):
        r, x = ref[0][:, :, h], gb[0][:, :, h]
        assert (np.abs(x - r) - 2.0 ** -8 * np.abs(r)).max() <= TOL_BF16 * np.sqrt(np.mean(r ** 2))


def test_tensor_path_fused_packed_varlen_and_s1(mdn):
    import torch
    w = wl.Workload("layer_packed", B=1, T=1500, H=4, dk=128, dv=128, dtype="bf16", varlen=True, len_lo=1, len_hi=400,
                    init_state_std=0.2, seed=54)
    if not tensor_ok(mdn, w):
        pytest.skip("tensor path not built")
    inp = wl.make_layer_inputs(w, s=1.0)       # theta up to arctan 2: strong forgetting, large beta
    ref = oracle_layer(inp, ALL)
    got = run_fused(mdn, inp, ALL, path="tensor", o_dtype=torch.float32)
    errs = errs3(got, ref)
    print("fused packed: o %.3e S %.3e M %.3e" % tuple(errs))
    assert max(errs) <= TOL_BF16


def test_tensor_path_fused_with_parallel_scan_and_determinism(mdn):
    import torch
    w = wl.Workload("layer_seg", B=1, T=64 * 24 + 9, H=2, dk=128, dv=128, dtype="bf16", init_state_std=0.02, seed=55)
    if not tensor_ok(mdn, w):
        pytest.skip("tensor path not built")
    inp = wl.make_layer_inputs(w)
    ref = oracle_layer(inp, ALL)
    got = run_fused(mdn, inp, ALL, path="tensor", o_dtype=torch.float32, segments=4)
    assert mdn.last_launch_count() == 5       # status clear, intra-chunk, segment runs, combine, real runs
    errs = errs3(got, ref)
    print("fused, 4 segments: o %.3e S %.3e M %.3e" % tuple(errs))
    assert max(errs) <= TOL_BF16
    serial = run_fused(mdn, inp, ALL, path="tensor", o_dtype=torch.float32, segments=1)
    print("fused, serial chain: o %.3e S %.3e M %.3e" % tuple(errs3(serial, ref)))
    per = (24 + 1 + 3) // 4 * 64                                  # segment 0 is the same real run in both
    assert np.array_equal(serial[0][:, :per], got[0][:, :per])
    again = run_fused(mdn, inp, ALL, path="tensor", o_dtype=torch.float32, segments=4)
    assert all(np.array_equal(a, b) for a, b in zip(got, again))


def test_config1_full_size_fused(mdn):
    import torch
    w = dataclasses.replace(wl.CONFIGS[1], name="cfg1_layer")
    if not tensor_ok(mdn, w):
        pytest.skip("tensor path not built")
    inp = wl.make_layer_inputs(w)
    chains = np.array([0, 7, 13, 22, 31])
    ref = oracle_layer(inp, ALL, chains=chains)
    got = run_fused(mdn, inp, ALL, path="tensor", o_dtype=torch.float32)
    errs = errs3(got, ref)
    print("cfg1 fused: o %.3e S %.3e M %.3e" % tuple(errs))
    assert max(errs) <= TOL_BF16


@pytest.mark.parametrize("dtype,dk,dv", [("f32", 64, 64), ("f32", 128, 128), ("bf16", 128, 128), ("bf16", 64, 128)])
def test_decode_step_with_layer_operations(mdn, dtype, dk, dv):
    """mdn_decode_step_fused token by token (serving path) against the oracle pipeline on the whole sequence."""
    import torch
    w = wl.Workload("layer_decode", B=3, T=24, H=2, dk=dk, dv=dv, dtype=dtype, init_state_std=0.2, seed=57)
    inp = wl.make_layer_inputs(w, s=1.0)
    ref = oracle_layer(inp, ALL)
    dt = torch.bfloat16 if dtype == "bf16" else torch.float32
    dev = lambda x, d=torch.float32: torch.from_numpy(np.ascontiguousarray(x)).to("cuda").to(d)
    q, k, v, g = dev(inp["q"], dt), dev(inp["k"], dt), dev(inp["v"], dt), dev(inp["g"], dt)
    xb, xa, xm, xe = (dev(inp[n]) for n in ("x_beta", "x_alpha", "x_mu", "x_eta"))
    gp = dict(a_alpha=dev(inp["a_alpha"]), b_alpha=dev(inp["b_alpha"]), a_mu=dev(inp["a_mu"]), b_mu=dev(inp["b_mu"]),
              s=inp["s"], tau=inp["tau"], log_mu_min=inp["log_mu_min"])
    dvec, wn = dev(inp["d"]), dev(inp["w_norm"])
    S, M = dev(inp["S0"]), dev(inp["M0"])
    outs = []
    for t in range(w.T):
        sl = slice(t, t + 1)
        c = lambda x: x[:, sl].contiguous()
        gt = c(g)
        ops = mdn.make_layer_ops(c(q), c(v), gate_param=gp, qk_norm=dict(d=dvec, eps=inp["qk_eps"]),
                                 out_norm_gate=dict(g=gt, w=wn, eps=inp["rms_eps"]))
        outs.append(mdn.decode_step(c(q), c(k), c(v), c(xb), c(xa), c(xm), c(xe), S, M, scale=inp["scale"],
                                    o_dtype=torch.float32, layer_ops=ops))
    torch.cuda.synchronize()
    f = lambda x: x.float().cpu().numpy().astype(np.float64)
    got = (f(torch.cat(outs, dim=1)), f(S), f(M))
    errs = errs3(got, ref)
    print("decode + layer ops %s dk%d dv%d: o %.3e S %.3e M %.3e" % (dtype, dk, dv, *errs))
    assert max(errs) <= 1e-4          # the decode kernel computes in fp32 whatever the i/o dtype


def test_fused_argument_validation(mdn):
    import torch
    w = wl.Workload("layer_args", B=1, T=64, H=2, dk=64, dv=64, dtype="f32", seed=56)
    inp = wl.make_layer_inputs(w)
    bad = dict(inp, qk_eps=0.0)
    with pytest.raises(mdn.MdnError):
        run_fused(mdn, bad, ("qk",) + ("gates",))
    bad = dict(inp, tau=0.0)
    with pytest.raises(mdn.MdnError):
        run_fused(mdn, bad, ("gates",))
