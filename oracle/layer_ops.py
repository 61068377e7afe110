"""fp64 oracle of the element-wise operations that surround the MDN recurrence inside a layer
(Section 3.3, "Model Architecture" and "Stability Aware Gating Parameterization").

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's CPU-baseline leg may import this;
the CUDA library never does and shares no code with it.

Every function is the printed formula written out in numpy float64, one line per symbol of the paper:

  gate_parameterisation   alpha^log = f(x_alpha) + log alpha_max,  mu^log = max(f(x_mu), floor),
                          beta = sigmoid(x_beta) * beta_max,       eta = tanh(x_eta / tau) + 1,
                          alpha_max = cos^2 theta, beta_max = sin^2 theta, theta = arctan(eta * s),
                          f(x) = -a * softplus(x + b)
  qk_preprocess           q <- L2Norm(q - d k),  k <- L2Norm(k)     (output correction before the norm)
  output_norm_gate        y = sigmoid(g) * RMSNorm(o)               (head-wise: over the dv entries of a head)

Readings where the text leaves a choice (each is a parameter here, not a constant):
  * a, b of the decay function are per-head vectors; alpha and mu have their own pair (passing the same
    arrays gives a shared one);
  * L2Norm(x) = x / sqrt(sum x^2 + eps) and RMSNorm(x) = x / sqrt(mean x^2 + eps) * w, eps inside the root;
  * d is a per-head scalar.
"""
import numpy as np


def softplus(x):
    """log(1 + e^x), evaluated without overflow."""
    x = np.asarray(x, dtype=np.float64)
    return np.maximum(x, 0.0) + np.log1p(np.exp(-np.abs(x)))


def sigmoid(x):
    x = np.asarray(x, dtype=np.float64)
    return np.where(x >= 0, 1.0 / (1.0 + np.exp(-np.abs(x))), np.exp(-np.abs(x)) / (1.0 + np.exp(-np.abs(x))))


def decay(x, a, b):
    """f(x) = -a * softplus(x + b); x: [..., H], a, b: [H]."""
    return -np.asarray(a, dtype=np.float64) * softplus(np.asarray(x, dtype=np.float64) + np.asarray(b, dtype=np.float64))


def gate_parameterisation(x_alpha, x_mu, x_beta, x_eta, a_alpha, b_alpha, a_mu, b_mu, s, tau, log_mu_min=-1.0):
    """Raw per-head projections [..., H] -> (log_alpha, log_mu, beta, eta), all float64."""
    eta = np.tanh(np.asarray(x_eta, dtype=np.float64) / tau) + 1.0
    theta = np.arctan(eta * s)
    alpha_max = np.cos(theta) ** 2
    beta_max = np.sin(theta) ** 2
    log_alpha = decay(x_alpha, a_alpha, b_alpha) + np.log(alpha_max)
    log_mu = np.maximum(decay(x_mu, a_mu, b_mu), log_mu_min)
    beta = sigmoid(x_beta) * beta_max
    return log_alpha, log_mu, beta, eta


def l2norm(x, eps):
    x = np.asarray(x, dtype=np.float64)
    return x / np.sqrt(np.sum(x * x, axis=-1, keepdims=True) + eps)


def qk_preprocess(q, k, d, eps):
    """q, k: [..., H, dk]; d: [H] (or None = 0).  Returns (L2Norm(q - d k), L2Norm(k))."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    if d is not None:
        q = q - np.asarray(d, dtype=np.float64)[:, None] * k
    return l2norm(q, eps), l2norm(k, eps)


def output_norm_gate(o, g, w, eps):
    """o, g: [..., H, dv]; w: [dv] (or None = ones).  y = sigmoid(g) * o / sqrt(mean(o^2) + eps) * w."""
    o = np.asarray(o, dtype=np.float64)
    rms = np.sqrt(np.mean(o * o, axis=-1, keepdims=True) + eps)
    y = o / rms
    if w is not None:
        y = y * np.asarray(w, dtype=np.float64)
    return sigmoid(g) * y
