"""Seeded synthetic inputs for the MDN chunkwise forward.

This module only *draws inputs*.  It holds none of the method's arithmetic
(no recurrence, no coefficients, no solve): the CPU oracle and the CUDA path
both take what it returns, and neither imports the other.

The tensors stand in for one MDN layer's inputs during language-model
training (the paper trains on 4k-token sequences with 400M / 1.3B models);
that data is not available here, so the shapes, dtypes and value structure
are reproduced instead:

* q, k: float32 N(0,1) draws, L2-normalised per (token, head) vector (the layer
  applies L2Norm to q and k, Section 3.3), then rounded once to the storage
  dtype.  v: N(0,1) (no normalisation in the layer).
* gates: raw logits z ~ N(0,1) pushed through the stability-aware gate
  parameterisation of Section 3.3:
      eta       = tanh(z_eta / tau) + 1
      theta     = arctan(eta * s)
      alpha_max = cos^2(theta),  beta_max = sin^2(theta)
      log_alpha = -a * softplus(z_alpha + b) + log(alpha_max)
      log_mu    = max(-a * softplus(z_mu + b), clamp)
      beta      = sigmoid(z_beta) * beta_max
  which guarantees beta <= 1 - alpha, mu in [e^clamp, 1), eta in (0, 2).
  The paper gives no values for a, b, s; two presets are provided.
* all per-token scalars are float32; states are float32.

Streams: numpy.random.default_rng([seed, stream]) with stream ids
0..9 = q, k, v, z_beta, z_alpha, z_mu, z_eta, S0, M0, lengths.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional

import numpy as np

CHUNK = 64

# Constants of the gate parameterisation the paper leaves open.
#   "S": long-memory regime (mean alpha ~0.92, mu ~0.97, beta ~0.03): the inter-chunk
#        state matters over thousands of tokens.  Default for all named configs.
#   "F": fast-forgetting stress preset (mean alpha ~0.27, mu ~0.53, beta ~0.23).
GATE_PRESETS: Dict[str, Dict[str, float]] = {
    "S": dict(a=1.0, b=-4.0, s=0.25, clamp=-1.0),
    "F": dict(a=1.0, b=0.0, s=1.0, clamp=-1.0),
}


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    B: int                      # batch rows (1 when packed / varlen)
    T: int                      # tokens per row (total tokens when varlen)
    H: int
    dk: int
    dv: int
    dtype: str                  # "f32" or "bf16": storage dtype of q, k, v, o
    varlen: bool = False        # split T into sequences via cu_seqlens
    len_lo: int = 128
    len_hi: int = 8192
    init_state_std: float = 0.0  # >0: nonzero initial S and M ~ N(0, std)
    seed: int = 0
    preset: str = "S"

    @property
    def scale(self) -> float:
        return float(self.dk) ** -0.5


# The five named configurations (index = config number).
CONFIGS: List[Workload] = [
    Workload("cfg0_tiny_f32", B=1, H=2, T=256, dk=64, dv=64, dtype="f32"),
    Workload("cfg1_400m_bf16", B=4, H=8, T=2048, dk=128, dv=128, dtype="bf16"),
    Workload("cfg2_1p3b_bf16", B=8, H=16, T=4096, dk=128, dv=128, dtype="bf16"),
    Workload("cfg3_long_bf16", B=1, H=16, T=65536, dk=128, dv=128, dtype="bf16",
             init_state_std=0.02),
    Workload("cfg4_varlen_bf16", B=1, H=16, T=32768, dk=128, dv=128, dtype="bf16",
             varlen=True),
]


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); returns float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    with np.errstate(over="ignore"):
        rounded = (u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) & np.uint32(0xFFFF0000)
    return rounded.view(np.float32).reshape(x.shape)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of float32 values that are already exactly bfloat16."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> 16).astype(np.uint16).reshape(x.shape)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32).reshape(bits.shape)


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.default_rng([seed, stream])


def _store(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round draws once to the storage dtype; returned as float32 (exact)."""
    x32 = np.asarray(x, dtype=np.float32)
    return round_to_bf16(x32) if dtype == "bf16" else x32


def _unit_rows(rng: np.random.Generator, shape, dtype: str) -> np.ndarray:
    x = rng.standard_normal(shape, dtype=np.float32)
    x /= np.sqrt(np.einsum("...d,...d->...", x, x, dtype=np.float64))[..., None].astype(np.float32)
    return _store(x, dtype)


def _softplus(x: np.ndarray) -> np.ndarray:
    return np.logaddexp(0.0, x)


def draw_gates(shape, seed: int, preset: str, dk: int,
               tau: Optional[float] = None, clamp: Optional[float] = None):
    """(beta, log_alpha, log_mu, eta) as float32 arrays of `shape` from N(0,1) logits."""
    p = GATE_PRESETS[preset]
    tau = math.sqrt(dk) if tau is None else tau
    clamp = p["clamp"] if clamp is None else clamp
    z_beta = _rng(seed, 3).standard_normal(shape)
    z_alpha = _rng(seed, 4).standard_normal(shape)
    z_mu = _rng(seed, 5).standard_normal(shape)
    z_eta = _rng(seed, 6).standard_normal(shape)
    eta = np.tanh(z_eta / tau) + 1.0
    theta = np.arctan(eta * p["s"])
    log_alpha_max = 2.0 * np.log(np.cos(theta))
    beta_max = np.sin(theta) ** 2
    log_alpha = -p["a"] * _softplus(z_alpha + p["b"]) + log_alpha_max
    log_mu = np.maximum(-p["a"] * _softplus(z_mu + p["b"]), clamp)
    beta = beta_max / (1.0 + np.exp(-z_beta))
    f32 = np.float32
    return beta.astype(f32), log_alpha.astype(f32), log_mu.astype(f32), eta.astype(f32)


def draw_lengths(total: int, lo: int, hi: int, seed: int) -> np.ndarray:
    """Integer lengths uniform in [lo, hi], drawn until they cover `total`; the last
    one is truncated so that the sum is exactly `total`."""
    rng = _rng(seed, 9)
    lens, acc = [], 0
    while acc < total:
        n = int(rng.integers(lo, hi + 1))
        n = min(n, total - acc)
        lens.append(n)
        acc += n
    return np.asarray(lens, dtype=np.int64)


def make_inputs(w: Workload, lengths: Optional[np.ndarray] = None) -> Dict[str, object]:
    """Draw every input of one call.

    Returns float32 arrays (values exactly representable in w.dtype for q, k, v):
      q, k [B,T,H,dk]; v [B,T,H,dv]; beta, log_alpha, log_mu, eta [B,T,H];
      S0, M0 [N,H,dk,dv] or None; cu_seqlens int32 [N+1] or None;
      seq_start, seq_len int64 [N]  (token ranges in the flattened [B*T] token axis).
    """
    B, T, H, dk, dv = w.B, w.T, w.H, w.dk, w.dv
    q = _unit_rows(_rng(w.seed, 0), (B, T, H, dk), w.dtype)
    k = _unit_rows(_rng(w.seed, 1), (B, T, H, dk), w.dtype)
    v = _store(_rng(w.seed, 2).standard_normal((B, T, H, dv), dtype=np.float32), w.dtype)
    beta, log_alpha, log_mu, eta = draw_gates((B, T, H), w.seed, w.preset, dk)

    if w.varlen:
        assert B == 1
        if lengths is None:
            lengths = draw_lengths(T, w.len_lo, w.len_hi, w.seed)
        lengths = np.asarray(lengths, dtype=np.int64)
        assert lengths.sum() == T and (lengths > 0).all()
        cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
        seq_start = cu[:-1].astype(np.int64)
        seq_len = lengths
    else:
        cu = None
        seq_start = np.arange(B, dtype=np.int64) * T
        seq_len = np.full(B, T, dtype=np.int64)
    N = len(seq_len)

    if w.init_state_std > 0:
        S0 = (_rng(w.seed, 7).standard_normal((N, H, dk, dv)) * w.init_state_std).astype(np.float32)
        M0 = (_rng(w.seed, 8).standard_normal((N, H, dk, dv)) * w.init_state_std).astype(np.float32)
    else:
        S0 = M0 = None

    return dict(q=q, k=k, v=v, beta=beta, log_alpha=log_alpha, log_mu=log_mu, eta=eta,
                S0=S0, M0=M0, cu_seqlens=cu, seq_start=seq_start, seq_len=seq_len,
                scale=w.scale, workload=w)


def make_layer_inputs(w: Workload, s: float = 0.25, d_in: int = 2048) -> Dict[str, object]:
    """Inputs of the forward WITH the layer's element-wise operations (Section 3.3): un-normalised q, k (stand-ins
    for the activations after ShortConv + SiLU), the raw per-head gate projections, the per-head parameters and
    the output gate.  Draws only: none of the operations is evaluated here.

    Adds to make_inputs(w): q, k replaced by N(0, sigma_h^2) rows (sigma_h in [0.5, 2] per head);
      x_beta, x_alpha, x_mu, x_eta [B,T,H] float32;  a_alpha, b_alpha, a_mu, b_mu, d [H] float32;
      s, tau = sqrt(d_in / H), log_mu_min = -1;  g [B,T,H,dv] (stored in w.dtype), w_norm [dv] float32;
      qk_eps = 1e-6, rms_eps = 1e-5.
    """
    inp = make_inputs(w)
    B, T, H, dk, dv = w.B, w.T, w.H, w.dk, w.dv
    sig = _rng(w.seed, 20).uniform(0.5, 2.0, (1, 1, H, 1)).astype(np.float32)
    inp["q"] = _store(_rng(w.seed, 21).standard_normal((B, T, H, dk), dtype=np.float32) * sig, w.dtype)
    inp["k"] = _store(_rng(w.seed, 22).standard_normal((B, T, H, dk), dtype=np.float32) * sig, w.dtype)
    f32 = np.float32
    inp["x_beta"] = _rng(w.seed, 23).standard_normal((B, T, H), dtype=f32)
    inp["x_alpha"] = _rng(w.seed, 24).standard_normal((B, T, H), dtype=f32)
    inp["x_mu"] = _rng(w.seed, 25).standard_normal((B, T, H), dtype=f32)
    inp["x_eta"] = (8.0 * _rng(w.seed, 26).standard_normal((B, T, H), dtype=f32)).astype(f32)
    inp["a_alpha"] = _rng(w.seed, 27).uniform(0.5, 8.0, H).astype(f32)
    inp["b_alpha"] = (-4.0 + 0.5 * _rng(w.seed, 28).standard_normal(H)).astype(f32)
    inp["a_mu"] = _rng(w.seed, 29).uniform(0.5, 8.0, H).astype(f32)
    inp["b_mu"] = (-3.0 + 0.5 * _rng(w.seed, 30).standard_normal(H)).astype(f32)
    inp["d"] = _rng(w.seed, 31).uniform(-0.2, 0.5, H).astype(f32)
    inp["s"], inp["tau"], inp["log_mu_min"] = float(s), float(math.sqrt(d_in / H)), -1.0
    inp["g"] = _store(1.5 * _rng(w.seed, 32).standard_normal((B, T, H, dv), dtype=f32), w.dtype)
    inp["w_norm"] = _rng(w.seed, 33).uniform(0.5, 1.5, dv).astype(f32)
    inp["qk_eps"], inp["rms_eps"] = 1e-6, 1e-5
    for name in ("beta", "log_alpha", "log_mu", "eta"):
        del inp[name]
    return inp


def correlated_keys(w: Workload, rho: float = 0.8) -> np.ndarray:
    """Unit keys sharing a common direction per head (pairwise cosine ~ rho): with
    i.i.d. keys the intra-chunk triangular system is nearly the identity, so this
    variant is what actually exercises the solve."""
    rng = _rng(w.seed, 1)
    x = rng.standard_normal((w.B, w.T, w.H, w.dk))
    x /= np.sqrt((x * x).sum(axis=-1, keepdims=True))
    c = _rng(w.seed, 11).standard_normal((1, 1, w.H, w.dk))
    c /= np.sqrt((c * c).sum(axis=-1, keepdims=True))
    y = math.sqrt(rho) * c + math.sqrt(1.0 - rho) * x
    y /= np.sqrt((y * y).sum(axis=-1, keepdims=True))
    return _store(y, w.dtype)
