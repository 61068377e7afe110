// Recurrent decode step: the stepwise recurrence of Section 3.1 (Eq. 5-6) applied to ONE new token per
// sequence with the carried state (S, M), updated in place:
//     v~ = v - alpha S^T k;   M <- mu M - eta k v~^T;   S <- alpha S - beta M;   o = scale S^T q
// The paper uses this form for autoregressive decoding (Section 3.3).  Pure streaming work: each (sequence,
// head) reads and writes its two dk x dv fp32 matrices once (4 * dk * dv * 4 bytes), so the kernel is
// HBM-bound; all arithmetic fp32.
//
// grid = (sequences * heads, dv / 32); block = 128 threads = 32 value columns x 4 groups of dk / 4 rows (with the
// layer operations of Section 3.3 the gate formulas and the q / k norms run here, the output norm and gate after it).
// A thread keeps its S entries in registers between the two passes (prediction, then update), so S and M
// each cross HBM exactly twice (one read, one write); row reads are 128-byte coalesced.
#include "mdn_common.cuh"

namespace mdn {
namespace {

constexpr int kGroups = 4;

// Block-wide sums of two values per thread (blockDim = 32 * nwarps <= 512); `buf` holds 2 x 16 floats and is used
// for this one reduction only (no barrier needed before it is written).
__device__ __forceinline__ float2 block_sum2(float x, float y, float* buf) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    x += __shfl_xor_sync(0xffffffffu, x, off);
    y += __shfl_xor_sync(0xffffffffu, y, off);
  }
  const int warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  if ((threadIdx.x & 31) == 0) { buf[warp] = x; buf[16 + warp] = y; }
  __syncthreads();
  float tx = 0.f, ty = 0.f;
  for (int w = 0; w < nw; ++w) { tx += buf[w]; ty += buf[16 + w]; }
  return make_float2(tx, ty);
}

// 32 value columns per CTA (4 CTAs per (sequence, head) at dv = 128: many small CTAs keep a pure streaming kernel at
// HBM speed).  kLayer adds the gate formulas and the q / k step of Section 3.3 (measured: free and +1 us); the output
// norm and gate need the whole head row and run as a second, tiny kernel over o (0.5 MB, L2-resident: +3 us) -
// forming thread-block clusters of the head's CTAs and reducing through distributed shared memory cost +20 us,
// one 512-thread CTA per head +36 us.
template <typename TIn, typename TO, int DK, int DV, int kCols, bool kLayer>
__global__ void __launch_bounds__(kCols * kGroups) decode_step_kernel(int H, const TIn* __restrict__ q,
                                                                    const TIn* __restrict__ k,
                                                                    const TIn* __restrict__ v,
                                                                    const float* __restrict__ beta,
                                                                    const float* __restrict__ log_alpha,
                                                                    const float* __restrict__ log_mu,
                                                                    const float* __restrict__ eta, float scale,
                                                                    float* __restrict__ S, float* __restrict__ M,
                                                                    TO* __restrict__ o, GateParam gp, QkNorm qk) {
  constexpr int RPT = DK / kGroups;   // rows of S, M per thread
  constexpr int kThreads = kCols * kGroups;
  __shared__ float ks[DK], qs[DK];
  __shared__ float red[kGroups][kCols];
  __shared__ float rbuf[32];
  const int chain = blockIdx.x;       // sequence * H + head
  const int jj = threadIdx.x % kCols;
  const int j = blockIdx.y * kCols + jj;
  const int dg = threadIdx.x / kCols;
  const int tid = threadIdx.x;
  for (int d = tid; d < DK; d += kThreads) {
    ks[d] = to_f32<TIn>(k[(size_t)chain * DK + d]);
    qs[d] = to_f32<TIn>(q[(size_t)chain * DK + d]);
  }
  float alpha, mu, be, et;
  {
    const TokenGates tg = load_token_gates(gp, chain % H, log_alpha[chain], log_mu[chain], beta[chain],
                                           eta ? eta[chain] : 1.f);
    alpha = tg.alpha; mu = tg.mu; be = tg.beta; et = tg.eta;
  }
  float* Sp = S + (size_t)chain * DK * DV + (size_t)(dg * RPT) * DV + j;
  float* Mp = M + (size_t)chain * DK * DV + (size_t)(dg * RPT) * DV + j;
  float sreg[RPT], mreg[RPT];   // both loads are issued up front: the prediction needs S only, but M's
#pragma unroll                  // latency then hides behind it
  for (int i = 0; i < RPT; ++i) sreg[i] = Sp[(size_t)i * DV];
#pragma unroll
  for (int i = 0; i < RPT; ++i) mreg[i] = Mp[(size_t)i * DV];
  __syncthreads();
  if (kLayer && qk.on) {
    // q <- L2Norm(q - d k), k <- L2Norm(k) (Section 3.3), on the staged vectors
    const float dh = qk.d ? __ldg(qk.d + chain % H) : 0.f;
    float pk = 0.f, pq = 0.f;
    for (int d = tid; d < DK; d += kThreads) {
      const float kv = ks[d], qv = qs[d] - dh * kv;
      pk = fmaf(kv, kv, pk);
      pq = fmaf(qv, qv, pq);
    }
    const float2 nrm = block_sum2(pk, pq, rbuf);
    const float rk = 1.f / sqrtf(nrm.x + qk.eps), rq = 1.f / sqrtf(nrm.y + qk.eps);
    for (int d = tid; d < DK; d += kThreads) {
      const float kv = ks[d];
      qs[d] = (qs[d] - dh * kv) * rq;
      ks[d] = kv * rk;
    }
    __syncthreads();
  }
  float part = 0.f;
#pragma unroll
  for (int i = 0; i < RPT; ++i) part = fmaf(sreg[i], ks[dg * RPT + i], part);
  red[dg][jj] = part;
  __syncthreads();
  const float pred = red[0][jj] + red[1][jj] + red[2][jj] + red[3][jj];     // (S^T k)_j, same order in every group
  const float vt = to_f32<TIn>(v[(size_t)chain * DV + j]) - alpha * pred;
  __syncthreads();
  float opart = 0.f;
#pragma unroll
  for (int i = 0; i < RPT; ++i) {
    const float m_new = mu * mreg[i] - et * ks[dg * RPT + i] * vt;
    const float s_new = alpha * sreg[i] - be * m_new;
    Mp[(size_t)i * DV] = m_new;
    Sp[(size_t)i * DV] = s_new;
    opart = fmaf(s_new, qs[dg * RPT + i], opart);
  }
  red[dg][jj] = opart;
  __syncthreads();
  const float ov = scale * (red[0][jj] + red[1][jj] + red[2][jj] + red[3][jj]);
  if (dg == 0) o[(size_t)chain * DV + j] = from_f32<TO>(ov);
}

template <typename TIn, typename TO>
cudaError_t dispatch(const mdn_params& p, const void* q, const void* k, const void* v, const float* beta,
                     const float* log_alpha, const float* log_mu, const float* eta, float* S, float* M, void* o,
                     const GateParam& gp, const QkNorm& qk, cudaStream_t st) {
  const bool layer = gp.raw || qk.on;
#define MDN_DECODE_CASE(DKV, DVV)                                                                              \
  if (p.dk == DKV && p.dv == DVV) {                                                                            \
    if (!layer) {                                                                                              \
      const dim3 grid((unsigned)p.B * p.H, (unsigned)p.dv / 32);                                               \
      decode_step_kernel<TIn, TO, DKV, DVV, 32, false><<<grid, 32 * kGroups, 0, st>>>(                         \
          p.H, static_cast<const TIn*>(q), static_cast<const TIn*>(k), static_cast<const TIn*>(v), beta, log_alpha, \
          log_mu, eta, p.scale, S, M, static_cast<TO*>(o), gp, qk);                                            \
    } else {                                                                                                   \
      const dim3 grid((unsigned)p.B * p.H, (unsigned)p.dv / 32);                                               \
      decode_step_kernel<TIn, TO, DKV, DVV, 32, true><<<grid, 32 * kGroups, 0, st>>>(                          \
          p.H, static_cast<const TIn*>(q), static_cast<const TIn*>(k), static_cast<const TIn*>(v), beta, log_alpha, \
          log_mu, eta, p.scale, S, M, static_cast<TO*>(o), gp, qk);                                            \
    }                                                                                                          \
    return cudaGetLastError();                                                                                 \
  }
  MDN_DECODE_CASE(64, 64)
  MDN_DECODE_CASE(64, 128)
  MDN_DECODE_CASE(128, 64)
  MDN_DECODE_CASE(128, 128)
#undef MDN_DECODE_CASE
  return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t launch_decode_step(const mdn_params& p, const void* q, const void* k, const void* v, const float* beta,
                               const float* log_alpha, const float* log_mu, const float* eta, float* S, float* M,
                               void* o, const GateParam& gp, const QkNorm& qk, cudaStream_t st) {
  const bool in_bf16 = p.io_dtype == MDN_BF16, o_bf16 = p.o_dtype == MDN_BF16;
  if (!in_bf16 && !o_bf16)
    return dispatch<float, float>(p, q, k, v, beta, log_alpha, log_mu, eta, S, M, o, gp, qk, st);
  if (in_bf16 && o_bf16)
    return dispatch<__nv_bfloat16, __nv_bfloat16>(p, q, k, v, beta, log_alpha, log_mu, eta, S, M, o, gp, qk, st);
  if (in_bf16) return dispatch<__nv_bfloat16, float>(p, q, k, v, beta, log_alpha, log_mu, eta, S, M, o, gp, qk, st);
  return dispatch<float, __nv_bfloat16>(p, q, k, v, beta, log_alpha, log_mu, eta, S, M, o, gp, qk, st);
}

}  // namespace mdn
