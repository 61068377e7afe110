// The layer's element-wise operations (Section 3.3) as passes of their own: the reference the fused forms are
// measured against, and the way the fp32 SIMT path runs the q/k pre-processing and the output step.
//   gate_param_kernel      raw projections -> beta, log_alpha, log_mu, eta          (one thread per (token, head))
//   qk_prep_kernel         q <- L2Norm(q - d k), k <- L2Norm(k)                     (one warp per (token, head))
//   out_norm_gate_kernel   o <- sigmoid(g) * RMSNorm(o) * w, in place               (one warp per (token, head))
// All three are single passes over their tensors: HBM-bound, coalesced (a warp reads one contiguous head row).
#include "mdn_common.cuh"

namespace mdn {
namespace {

__global__ void __launch_bounds__(256) gate_param_kernel(GateParam gp, int H, size_t n, const float* __restrict__ x_beta,
                                                        const float* __restrict__ x_alpha,
                                                        const float* __restrict__ x_mu,
                                                        const float* __restrict__ x_eta, float* __restrict__ beta,
                                                        float* __restrict__ log_alpha, float* __restrict__ log_mu,
                                                        float* __restrict__ eta) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    const GateValues gv = gate_transform(gp, (int)(i % H), __ldg(x_alpha + i), __ldg(x_mu + i), __ldg(x_beta + i),
                                         __ldg(x_eta + i));
    beta[i] = gv.beta; log_alpha[i] = gv.log_alpha; log_mu[i] = gv.log_mu; eta[i] = gv.eta;
  }
}

// E consecutive elements moved as one access of up to 16 bytes (two when TG is wider than TO).
template <typename T, int E> struct alignas(sizeof(T) * E <= 16 ? sizeof(T) * E : 16) Pack { T v[E]; };

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
  return x;
}

// rows = B*T*H head rows of D elements.  Every lane moves 16 bytes per access (E = 16 / sizeof(T) consecutive
// elements), so a row takes LPR = D / E lanes and a warp covers 32 / LPR rows per access; kRowsPerIter such accesses
// are issued before the first reduction, so that enough bytes are in flight per SM to approach HBM bandwidth.
constexpr int kRowsPerIter = 4;

template <int LPR> __device__ __forceinline__ float row_sum(float x) {
#pragma unroll
  for (int off = LPR / 2; off > 0; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
  return x;
}

template <typename T, int D>
__global__ void __launch_bounds__(256) qk_prep_kernel(size_t rows, int H, QkNorm qk, const T* __restrict__ q,
                                                     const T* __restrict__ k, T* __restrict__ q_out,
                                                     T* __restrict__ k_out) {
  constexpr int E = 16 / sizeof(T), LPR = D / E, RPW = 32 / LPR, R = kRowsPerIter;
  const int lane = threadIdx.x & 31, sub = lane / LPR, l = lane % LPR;
  const size_t warps = (size_t)gridDim.x * (blockDim.x >> 5);
  const size_t warp_id = (size_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  for (size_t row0 = warp_id * (RPW * R); row0 < rows; row0 += warps * (RPW * R)) {
    Pack<T, E> kp[R], qp[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const size_t row = row0 + (size_t)r * RPW + sub;
      if (row < rows) {
        kp[r] = *reinterpret_cast<const Pack<T, E>*>(k + row * D + l * E);
        qp[r] = *reinterpret_cast<const Pack<T, E>*>(q + row * D + l * E);
      }
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const size_t row = row0 + (size_t)r * RPW + sub;
      const bool live = row < rows;     // (all lanes take part in the shuffles)
      const float d = (live && qk.d) ? __ldg(qk.d + (int)(row % H)) : 0.f;
      float qv[E], kv[E];
      float sq = 0.f, sk = 0.f;
#pragma unroll
      for (int e = 0; e < E; ++e) {
        kv[e] = live ? to_f32<T>(kp[r].v[e]) : 0.f;
        qv[e] = live ? to_f32<T>(qp[r].v[e]) - d * kv[e] : 0.f;
        sq = fmaf(qv[e], qv[e], sq);
        sk = fmaf(kv[e], kv[e], sk);
      }
      const float rq = rsqrtf(row_sum<LPR>(sq) + qk.eps), rk = rsqrtf(row_sum<LPR>(sk) + qk.eps);
      if (live) {
        Pack<T, E> qo, ko;
#pragma unroll
        for (int e = 0; e < E; ++e) {
          qo.v[e] = from_f32<T>(qv[e] * rq);
          ko.v[e] = from_f32<T>(kv[e] * rk);
        }
        *reinterpret_cast<Pack<T, E>*>(q_out + row * D + l * E) = qo;
        *reinterpret_cast<Pack<T, E>*>(k_out + row * D + l * E) = ko;
      }
    }
  }
}

// TO and TG may differ in size: the lane's E = 16 / sizeof(TO) elements are one 16-byte access of o and one 16- or
// 8-byte (or two 16-byte) access of g.
template <typename TO, typename TG, int D>
__global__ void __launch_bounds__(256) out_norm_gate_kernel(size_t rows, OutPost post, TO* __restrict__ o) {
  constexpr int E = 16 / sizeof(TO), LPR = D / E, RPW = 32 / LPR, R = kRowsPerIter;
  const int lane = threadIdx.x & 31, sub = lane / LPR, l = lane % LPR;
  const TG* __restrict__ g = static_cast<const TG*>(post.g);
  float wv[E];
#pragma unroll
  for (int e = 0; e < E; ++e) wv[e] = post.w ? __ldg(post.w + l * E + e) : 1.f;
  const size_t warps = (size_t)gridDim.x * (blockDim.x >> 5);
  const size_t warp_id = (size_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  for (size_t row0 = warp_id * (RPW * R); row0 < rows; row0 += warps * (RPW * R)) {
    Pack<TO, E> op[R];
    Pack<TG, E> gp[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const size_t row = row0 + (size_t)r * RPW + sub;
      if (row < rows) {
        op[r] = *reinterpret_cast<const Pack<TO, E>*>(o + row * D + l * E);
        gp[r] = *reinterpret_cast<const Pack<TG, E>*>(g + row * D + l * E);
      }
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const size_t row = row0 + (size_t)r * RPW + sub;
      const bool live = row < rows;
      float ov[E];
      float ss = 0.f;
#pragma unroll
      for (int e = 0; e < E; ++e) {
        ov[e] = live ? to_f32<TO>(op[r].v[e]) : 0.f;
        ss = fmaf(ov[e], ov[e], ss);
      }
      const float rstd = rsqrtf(row_sum<LPR>(ss) * (1.f / D) + post.eps);
      if (live) {
        Pack<TO, E> yo;
#pragma unroll
        for (int e = 0; e < E; ++e) {
          const float gate = __fdividef(1.f, 1.f + __expf(-to_f32<TG>(gp[r].v[e])));   // 2 special-function ops
          yo.v[e] = from_f32<TO>(gate * ov[e] * rstd * wv[e]);
        }
        *reinterpret_cast<Pack<TO, E>*>(o + row * D + l * E) = yo;
      }
    }
  }
}

inline unsigned blocks_for(size_t items, int per_block) {
  const size_t b = (items + per_block - 1) / per_block;
  return (unsigned)(b < 148 * 32 ? (b ? b : 1) : 148 * 32);
}

}  // namespace

cudaError_t launch_gate_param(const Plan& pl, const float* x_beta, const float* x_alpha, const float* x_mu,
                              const float* x_eta, float* beta, float* log_alpha, float* log_mu, float* eta,
                              int* launches) {
  const size_t n = (size_t)pl.p.B * pl.p.T * pl.p.H;
  gate_param_kernel<<<blocks_for(n, 256), 256, 0, pl.stream>>>(pl.gp, pl.p.H, n, x_beta, x_alpha, x_mu, x_eta, beta,
                                                              log_alpha, log_mu, eta);
  ++*launches;
  return cudaGetLastError();
}

cudaError_t launch_qk_prep(const Plan& pl, const QkNorm& qk, const void* q, const void* k, void* q_out, void* k_out,
                           int* launches) {
  const size_t rows = (size_t)pl.p.B * pl.p.T * pl.p.H;
  const unsigned grid = blocks_for(rows, 16 * kRowsPerIter);
  const bool bf = pl.p.io_dtype == MDN_BF16;
#define MDN_QK_CASE(T, D)                                                                                   \
  qk_prep_kernel<T, D><<<grid, 256, 0, pl.stream>>>(rows, pl.p.H, qk, static_cast<const T*>(q),             \
                                                    static_cast<const T*>(k), static_cast<T*>(q_out),       \
                                                    static_cast<T*>(k_out))
  if (pl.p.dk == 64) {
    if (bf) MDN_QK_CASE(__nv_bfloat16, 64); else MDN_QK_CASE(float, 64);
  } else {
    if (bf) MDN_QK_CASE(__nv_bfloat16, 128); else MDN_QK_CASE(float, 128);
  }
#undef MDN_QK_CASE
  ++*launches;
  return cudaGetLastError();
}

cudaError_t launch_out_norm_gate(const Plan& pl, const OutPost& post, void* o, int* launches) {
  const size_t rows = (size_t)pl.p.B * pl.p.T * pl.p.H;
  const unsigned grid = blocks_for(rows, 16 * kRowsPerIter);
  const bool obf = pl.p.o_dtype == MDN_BF16, gbf = pl.p.io_dtype == MDN_BF16;
#define MDN_OUT_CASE(TO, TG, D) out_norm_gate_kernel<TO, TG, D><<<grid, 256, 0, pl.stream>>>(rows, post, static_cast<TO*>(o))
#define MDN_OUT_D(D)                                                   \
  if (obf && gbf) MDN_OUT_CASE(__nv_bfloat16, __nv_bfloat16, D);       \
  else if (obf) MDN_OUT_CASE(__nv_bfloat16, float, D);                 \
  else if (gbf) MDN_OUT_CASE(float, __nv_bfloat16, D);                 \
  else MDN_OUT_CASE(float, float, D)
  if (pl.p.dv == 64) { MDN_OUT_D(64); } else { MDN_OUT_D(128); }
#undef MDN_OUT_D
#undef MDN_OUT_CASE
  ++*launches;
  return cudaGetLastError();
}

}  // namespace mdn
