// Per-(chunk, head) coefficient scan shared by the stand-alone scan kernel and the fused tensor-path
// intra-chunk kernel: one warp, two consecutive positions per lane (r = 2 lane, 2 lane + 1).
#pragma once

#include <cuda_runtime.h>

namespace mdn {

// Affine map x -> a*x + c; compose(f_later, f_earlier).
struct Affine { float a, c; };
__device__ __forceinline__ Affine compose(Affine later, Affine earlier) {
  return Affine{later.a * earlier.a, fmaf(later.a, earlier.c, later.c)};
}

// Inclusive scan over lanes in increasing order: result(l) = f_l o ... o f_0.
__device__ __forceinline__ Affine warp_scan_up(Affine f, int lane) {
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    Affine o;
    o.a = __shfl_up_sync(0xffffffffu, f.a, off);
    o.c = __shfl_up_sync(0xffffffffu, f.c, off);
    if (lane >= off) f = compose(f, o);
  }
  return f;
}
// Inclusive scan in decreasing order: result(l) = f_l o f_{l+1} o ... o f_31.
__device__ __forceinline__ Affine warp_scan_down(Affine f, int lane) {
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    Affine o;
    o.a = __shfl_down_sync(0xffffffffu, f.a, off);
    o.c = __shfl_down_sync(0xffffffffu, f.c, off);
    if (lane + off < 32) f = compose(f, o);
  }
  return f;
}

// Chain-kernel coefficient vectors of one (chunk, head); element e belongs to position 2 lane + e.
struct HeadCoefs { float abar[2], b[2], ab_prev[2], gs[2], gm[2], mubar[2]; };

// al, mu, be, et: alpha, mu, beta, eta at the lane's two positions (exact no-ops past the end of a short
// chunk: alpha = mu = 1, beta = eta = 0).  All 32 lanes must call.
__device__ __forceinline__ HeadCoefs scan_head(const float (&al)[2], const float (&mu)[2], const float (&be)[2],
                                               const float (&et)[2], int lane) {
    // forward products abar, mubar
    Affine pa = warp_scan_up(Affine{al[0] * al[1], 0.f}, lane);
    Affine pm = warp_scan_up(Affine{mu[0] * mu[1], 0.f}, lane);
    float ea = __shfl_up_sync(0xffffffffu, pa.a, 1), em = __shfl_up_sync(0xffffffffu, pm.a, 1);
    if (lane == 0) { ea = 1.f; em = 1.f; }
    const float abar0 = ea * al[0], abar1 = abar0 * al[1];
    const float mbar0 = em * mu[0], mbar1 = mbar0 * mu[1];
    // b_r = alpha_r b_{r-1} + beta_r mubar_r
    const Affine f0{al[0], be[0] * mbar0}, f1{al[1], be[1] * mbar1};
    Affine fb = warp_scan_up(compose(f1, f0), lane);
    float bprev = __shfl_up_sync(0xffffffffu, fb.c, 1);
    if (lane == 0) bprev = 0.f;
    const float b0 = fmaf(al[0], bprev, f0.c), b1 = fmaf(al[1], b0, f1.c);
    // backward: A_i = prod_{l>i} alpha_l, m_i = prod_{l>i} mu_l
    Affine sa = warp_scan_down(Affine{al[0] * al[1], 0.f}, lane);
    Affine smu = warp_scan_down(Affine{mu[0] * mu[1], 0.f}, lane);
    float xa = __shfl_down_sync(0xffffffffu, sa.a, 1), xm = __shfl_down_sync(0xffffffffu, smu.a, 1);
    if (lane == 31) { xa = 1.f; xm = 1.f; }
    const float A1 = xa, A0 = xa * al[1];
    const float m1 = xm, m0 = xm * mu[1];
    // g_i = A_i beta_i + mu_{i+1} g_{i+1}
    float mu_next = __shfl_down_sync(0xffffffffu, mu[0], 1);
    if (lane == 31) mu_next = 0.f;
    const Affine h1{mu_next, A1 * be[1]}, h0{mu[1], A0 * be[0]};
    Affine fg = warp_scan_down(compose(h0, h1), lane);
    float gnext = __shfl_down_sync(0xffffffffu, fg.c, 1);
    if (lane == 31) gnext = 0.f;
    const float g1 = fmaf(mu_next, gnext, h1.c), g0 = fmaf(mu[1], g1, h0.c);

    HeadCoefs hc;
    hc.abar[0] = abar0; hc.abar[1] = abar1;
    hc.b[0] = b0; hc.b[1] = b1;
    hc.ab_prev[0] = al[0] * bprev; hc.ab_prev[1] = al[1] * b0;
    hc.gs[0] = g0 * et[0]; hc.gs[1] = g1 * et[1];
    hc.gm[0] = m0 * et[0]; hc.gm[1] = m1 * et[1];
    hc.mubar[0] = mbar0; hc.mubar[1] = mbar1;
    return hc;
}

}  // namespace mdn
