// Element-wise operations of the MDN layer that the forward can absorb (Section 3.3): parameter bundles passed to
// the kernels by value, and the gate formulas as a device function shared by every kernel that evaluates them.
#pragma once

#include <cuda_runtime.h>

namespace mdn {

// Stability-aware gate parameterisation.  raw == 0: the gate arrays already hold beta, log_alpha, log_mu, eta.
struct GateParam {
  int raw;
  const float* a_alpha;   // [H]  f(x) = -a softplus(x + b)
  const float* b_alpha;
  const float* a_mu;
  const float* b_mu;
  float s, inv_tau, log_mu_min;
};

// q <- L2Norm(q - d k), k <- L2Norm(k), applied to accumulators inside the kernels.
struct QkNorm {
  int on;
  const float* d;   // [H] or NULL
  float eps;
};

// o <- sigmoid(g) * RMSNorm(o) * w in the output epilogue.
struct OutPost {
  int on;
  const void* g;    // [B,T,H,dv], i/o dtype
  const float* w;   // [dv] or NULL
  float eps;
};

__device__ __forceinline__ float softplus_f32(float x) { return fmaxf(x, 0.f) + log1pf(expf(-fabsf(x))); }

// Raw projections of one (token, head) -> eta, the two bounds' common factor, and the decay exponents.
//   eta = tanh(x_eta / tau) + 1;  z = eta s = tan(theta);  cos^2 = 1 / (1 + z^2);  sin^2 = z^2 / (1 + z^2)
struct GateValues { float log_alpha, log_mu, beta, eta; };
__device__ __forceinline__ GateValues gate_transform(const GateParam& gp, int h, float x_alpha, float x_mu, float x_beta,
                                                     float x_eta) {
  GateValues gv;
  gv.eta = tanhf(x_eta * gp.inv_tau) + 1.f;
  const float z = gv.eta * gp.s, z2 = z * z;
  gv.log_alpha = -__ldg(gp.a_alpha + h) * softplus_f32(x_alpha + __ldg(gp.b_alpha + h)) - log1pf(z2);
  gv.log_mu = fmaxf(-__ldg(gp.a_mu + h) * softplus_f32(x_mu + __ldg(gp.b_mu + h)), gp.log_mu_min);
  gv.beta = z2 / ((1.f + z2) * (1.f + expf(-x_beta)));
  return gv;
}

}  // namespace mdn
