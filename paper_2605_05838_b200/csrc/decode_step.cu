// Recurrent decode step: the stepwise recurrence of Section 3.1 (Eq. 5-6) applied to ONE new token per
// sequence with the carried state (S, M), updated in place:
//     v~ = v - alpha S^T k;   M <- mu M - eta k v~^T;   S <- alpha S - beta M;   o = scale S^T q
// The paper uses this form for autoregressive decoding (Section 3.3).  Pure streaming work: each (sequence,
// head) reads and writes its two dk x dv fp32 matrices once (4 * dk * dv * 4 bytes), so the kernel is
// HBM-bound; all arithmetic fp32.
//
// grid = (sequences * heads, dv / 32); block = 128 threads = 32 value columns x 4 groups of dk / 4 rows.
// A thread keeps its S entries in registers between the two passes (prediction, then update), so S and M
// each cross HBM exactly twice (one read, one write); row reads are 128-byte coalesced.
#include "mdn_common.cuh"

namespace mdn {
namespace {

constexpr int kCols = 32, kGroups = 4, kThreads = kCols * kGroups;

template <typename TIn, typename TO, int DK, int DV>
__global__ void __launch_bounds__(kThreads) decode_step_kernel(int H, const TIn* __restrict__ q,
                                                              const TIn* __restrict__ k, const TIn* __restrict__ v,
                                                              const float* __restrict__ beta,
                                                              const float* __restrict__ log_alpha,
                                                              const float* __restrict__ log_mu,
                                                              const float* __restrict__ eta, float scale,
                                                              float* __restrict__ S, float* __restrict__ M,
                                                              TO* __restrict__ o) {
  constexpr int RPT = DK / kGroups;   // rows of S, M per thread
  __shared__ float ks[DK], qs[DK];
  __shared__ float red[kGroups][kCols];
  const int chain = blockIdx.x;       // sequence * H + head
  const int j = blockIdx.y * kCols + (threadIdx.x & (kCols - 1));
  const int dg = threadIdx.x / kCols;
  const int tid = threadIdx.x;
  for (int d = tid; d < DK; d += kThreads) {
    ks[d] = to_f32<TIn>(k[(size_t)chain * DK + d]);
    qs[d] = to_f32<TIn>(q[(size_t)chain * DK + d]);
  }
  const float alpha = expf(log_alpha[chain]), mu = expf(log_mu[chain]);
  const float be = beta[chain], et = eta ? eta[chain] : 1.f;
  float* Sp = S + (size_t)chain * DK * DV + (size_t)(dg * RPT) * DV + j;
  float* Mp = M + (size_t)chain * DK * DV + (size_t)(dg * RPT) * DV + j;
  float sreg[RPT], mreg[RPT];   // both loads are issued up front: the prediction needs S only, but M's
#pragma unroll                  // latency then hides behind it
  for (int i = 0; i < RPT; ++i) sreg[i] = Sp[(size_t)i * DV];
#pragma unroll
  for (int i = 0; i < RPT; ++i) mreg[i] = Mp[(size_t)i * DV];
  __syncthreads();
  float part = 0.f;
#pragma unroll
  for (int i = 0; i < RPT; ++i) part = fmaf(sreg[i], ks[dg * RPT + i], part);
  red[dg][tid & (kCols - 1)] = part;
  __syncthreads();
  const int jj = tid & (kCols - 1);
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
  if (dg == 0) o[(size_t)chain * DV + j] = from_f32<TO>(scale * (red[0][jj] + red[1][jj] + red[2][jj] + red[3][jj]));
}

template <typename TIn, typename TO>
cudaError_t dispatch(const mdn_params& p, const void* q, const void* k, const void* v, const float* beta,
                     const float* log_alpha, const float* log_mu, const float* eta, float* S, float* M, void* o,
                     cudaStream_t st) {
  const dim3 grid((unsigned)p.B * p.H, (unsigned)p.dv / kCols);
#define MDN_DECODE_CASE(DKV, DVV)                                                                              \
  if (p.dk == DKV && p.dv == DVV) {                                                                            \
    decode_step_kernel<TIn, TO, DKV, DVV><<<grid, kThreads, 0, st>>>(                                          \
        p.H, static_cast<const TIn*>(q), static_cast<const TIn*>(k), static_cast<const TIn*>(v), beta, log_alpha, \
        log_mu, eta, p.scale, S, M, static_cast<TO*>(o));                                                      \
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
                               void* o, cudaStream_t st) {
  const bool in_bf16 = p.io_dtype == MDN_BF16, o_bf16 = p.o_dtype == MDN_BF16;
  if (!in_bf16 && !o_bf16) return dispatch<float, float>(p, q, k, v, beta, log_alpha, log_mu, eta, S, M, o, st);
  if (in_bf16 && o_bf16)
    return dispatch<__nv_bfloat16, __nv_bfloat16>(p, q, k, v, beta, log_alpha, log_mu, eta, S, M, o, st);
  if (in_bf16) return dispatch<__nv_bfloat16, float>(p, q, k, v, beta, log_alpha, log_mu, eta, S, M, o, st);
  return dispatch<float, __nv_bfloat16>(p, q, k, v, beta, log_alpha, log_mu, eta, S, M, o, st);
}

}  // namespace mdn
