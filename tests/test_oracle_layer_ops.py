"""Pins for oracle/layer_ops.py (gate parameterisation, q/k pre-processing, output norm + gate of
Section 3.3): closed forms, identities and library routines, never the oracle's own formula retyped.
All CPU, fp64, seconds."""
import numpy as np
import torch

from oracle import layer_ops as lo


def test_softplus_and_sigmoid_closed_forms_and_library():
    assert np.isclose(lo.softplus(0.0), np.log(2.0), rtol=0, atol=1e-15)
    x = np.linspace(-40, 40, 401)
    assert np.allclose(lo.softplus(x) - lo.softplus(-x), x, rtol=0, atol=1e-12)       # log(1+e^x) - log(1+e^-x) = x
    assert np.allclose(lo.softplus(np.array([800.0, -800.0])), [800.0, 0.0])          # no overflow
    assert np.allclose(lo.sigmoid(x) + lo.sigmoid(-x), 1.0, rtol=0, atol=1e-15)
    h = 1e-5                                                                          # softplus' = sigmoid
    assert np.allclose((lo.softplus(x + h) - lo.softplus(x - h)) / (2 * h), lo.sigmoid(x), atol=1e-9)
    xt = torch.tensor(x, dtype=torch.float64)
    assert np.allclose(lo.softplus(x), torch.nn.functional.softplus(xt, threshold=1e9).numpy(), atol=1e-13)
    assert np.allclose(lo.sigmoid(x), torch.sigmoid(xt).numpy(), atol=1e-15)


def test_gate_bounds_at_known_angles():
    """theta = arctan(eta s): eta = 1 (x_eta = 0) with s = 1 gives pi/4, with s = sqrt 3 gives pi/3."""
    H = 2
    one, zero = np.ones(H), np.zeros(H)
    big = np.full((1, H), 60.0)
    for s, amax, bmax in [(1.0, 0.5, 0.5), (np.sqrt(3.0), 0.25, 0.75), (1.0 / np.sqrt(3.0), 0.75, 0.25)]:
        # x_alpha -> -inf: softplus -> 0, alpha -> alpha_max;  x_beta -> +inf: sigmoid -> 1, beta -> beta_max
        la, lm, be, et = lo.gate_parameterisation(-big * 20, zero[None], big, zero[None], one, zero, one, zero, s, 4.0)
        assert np.allclose(et, 1.0) and np.allclose(np.exp(la), amax, atol=1e-12) and np.allclose(be, bmax, atol=1e-12)
    # x_alpha = 0, a = 1, b = 0: f = -ln 2, so alpha = alpha_max / 2;  x_beta = 0: beta = beta_max / 2
    la, lm, be, et = lo.gate_parameterisation(zero[None], zero[None], zero[None], zero[None], one, zero, one, zero, 1.0, 4.0)
    assert np.allclose(np.exp(la), 0.25) and np.allclose(be, 0.25) and np.allclose(np.exp(lm), 0.5)


def test_gate_invariants_random():
    r = np.random.default_rng(0)
    B, T, H = 2, 50, 4
    xa, xm, xb, xe = (3 * r.standard_normal((B, T, H)) for _ in range(4))
    aa, am = r.uniform(0.1, 4, H), r.uniform(0.1, 4, H)
    ba, bm = r.standard_normal(H), r.standard_normal(H)
    s, tau = 0.7, 8.0
    la, lm, be, et = lo.gate_parameterisation(xa, xm, xb, xe, aa, ba, am, bm, s, tau)
    assert (et > 0).all() and (et < 2).all()
    # tanh is odd: eta(x) + eta(-x) = 2
    _, _, _, et_neg = lo.gate_parameterisation(xa, xm, xb, -xe, aa, ba, am, bm, s, tau)
    assert np.allclose(et + et_neg, 2.0, atol=1e-14)
    # cos^2(arctan z) = 1 / (1 + z^2): the bounds by the rational route, and alpha_max + beta_max = 1
    z = et * s
    amax, bmax = 1.0 / (1.0 + z * z), z * z / (1.0 + z * z)
    f_alpha = la - np.log(amax)
    assert (f_alpha <= 0).all()                                   # the decay function is non-positive
    assert (np.exp(la) <= amax + 1e-15).all() and (be <= bmax + 1e-15).all() and (be >= 0).all()
    assert (np.exp(la) + be <= 1.0 + 1e-14).all()                 # the stability region of Section 3.3
    # the decay function through the library softplus: -a softplus(x + b)
    f_lib = -aa * torch.nn.functional.softplus(torch.tensor(xa + ba), threshold=1e9).numpy()
    assert np.allclose(f_alpha, f_lib, atol=1e-12)
    assert np.allclose(be / bmax, torch.sigmoid(torch.tensor(xb)).numpy(), atol=1e-13)
    # momentum floor: never below -1, equal to f where f is above it
    f_mu = -am * torch.nn.functional.softplus(torch.tensor(xm + bm), threshold=1e9).numpy()
    assert (lm >= -1.0).all() and np.allclose(lm, np.maximum(f_mu, -1.0), atol=1e-12)
    assert (f_mu < -1.0).any() and (f_mu > -1.0).any()            # both branches exercised
    # each head uses its own (a, b): permuting heads permutes the result
    perm = np.array([2, 0, 3, 1])
    la_p, lm_p, be_p, et_p = lo.gate_parameterisation(xa[..., perm], xm[..., perm], xb[..., perm], xe[..., perm],
                                                      aa[perm], ba[perm], am[perm], bm[perm], s, tau)
    assert np.allclose(la_p, la[..., perm]) and np.allclose(lm_p, lm[..., perm]) and np.allclose(be_p, be[..., perm])


def test_qk_preprocess_geometry():
    r = np.random.default_rng(1)
    q, k = r.standard_normal((3, 7, 4, 16)), r.standard_normal((3, 7, 4, 16))
    d = r.uniform(-0.5, 0.5, 4)
    qn, kn = lo.qk_preprocess(q, k, d, 0.0)
    assert np.allclose(np.linalg.norm(qn, axis=-1), 1.0) and np.allclose(np.linalg.norm(kn, axis=-1), 1.0)
    # direction: k' parallel to k, q' parallel to q - d k (Cauchy-Schwarz equality)
    assert np.allclose(np.sum(kn * k, -1), np.linalg.norm(k, axis=-1))
    diff = q - d[None, None, :, None] * k
    assert np.allclose(np.sum(qn * diff, -1), np.linalg.norm(diff, axis=-1))
    # library route (eps -> 0)
    kt = torch.nn.functional.normalize(torch.tensor(k), dim=-1, eps=1e-300).numpy()
    assert np.allclose(kn, kt, atol=1e-14)
    # d = (q.k)/(k.k) removes the k component: q' is orthogonal to k'
    dd = np.sum(q[0, 0] * k[0, 0], -1) / np.sum(k[0, 0] * k[0, 0], -1)
    qo, ko = lo.qk_preprocess(q[0, 0], k[0, 0], dd, 0.0)
    assert np.allclose(np.sum(qo * ko, -1), 0.0, atol=1e-14)
    # d = None is d = 0; scaling the inputs changes nothing at eps = 0; eps sits inside the root
    q0, k0 = lo.qk_preprocess(q, k, None, 0.0)
    qz, kz = lo.qk_preprocess(q, k, np.zeros(4), 0.0)
    assert np.array_equal(q0, qz) and np.array_equal(k0, kz)
    q5, k5 = lo.qk_preprocess(5 * q, 5 * k, d, 0.0)
    assert np.allclose(q5, qn) and np.allclose(k5, kn)
    x = np.array([[3.0, 4.0]])
    assert np.allclose(lo.l2norm(x, 11.0), x / 6.0)               # sqrt(25 + 11) = 6


def test_output_norm_gate():
    r = np.random.default_rng(2)
    o, g = 3 * r.standard_normal((2, 9, 4, 32)), r.standard_normal((2, 9, 4, 32))
    w = r.uniform(0.5, 1.5, 32)
    open_gate = np.full_like(g, 80.0)                             # sigmoid -> 1
    y = lo.output_norm_gate(o, open_gate, None, 0.0)
    assert np.allclose(np.mean(y * y, -1), 1.0)                   # unit RMS per head
    assert np.allclose(lo.output_norm_gate(7 * o, open_gate, None, 0.0), y)
    # library RMSNorm with weight and eps
    eps = 1e-3
    ref = torch.nn.functional.rms_norm(torch.tensor(o), (32,), torch.tensor(w), eps).numpy()
    assert np.allclose(lo.output_norm_gate(o, open_gate, w, eps), ref, atol=1e-13)
    # the gate multiplies element-wise: g = 0 halves, g = -inf closes
    assert np.allclose(lo.output_norm_gate(o, np.zeros_like(g), w, eps), 0.5 * ref)
    assert np.allclose(lo.output_norm_gate(o, -open_gate, w, eps), 0.0, atol=1e-30)
    assert np.allclose(lo.output_norm_gate(o, g, w, eps), torch.sigmoid(torch.tensor(g)).numpy() * ref, atol=1e-13)
    # heads are normalised independently
    o2 = o.copy(); o2[:, :, 1] *= 100.0
    y2 = lo.output_norm_gate(o2, g, w, 0.0)
    assert np.allclose(y2, lo.output_norm_gate(o, g, w, 0.0))
