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

// E consecutive elements moved as one 4-, 8- or 16-byte access.
template <typename T, int E> struct alignas(sizeof(T) * E) Pack { T v[E]; };

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
  return x;
}

// rows = B*T*H head rows of D elements; lane l owns elements l*E .. l*E+E-1 (E = D / 32, contiguous).  A warp takes
// kRowsPerIter consecutive rows per iteration and issues all their loads before the first reduction, so that enough
// bytes are in flight per SM to reach HBM bandwidth.
constexpr int kRowsPerIter = 4;

template <typename T, int D>
__global__ void __launch_bounds__(256) qk_prep_kernel(size_t rows, int H, QkNorm qk, const T* __restrict__ q,
                                                     const T* __restrict__ k, T* __restrict__ q_out,
                                                     T* __restrict__ k_out) {
  constexpr int E = D / 32, R = kRowsPerIter;
  const int lane = threadIdx.x & 31;
  const size_t warps = (size_t)gridDim.x * (blockDim.x >> 5);
  for (size_t row0 = ((size_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * R; row0 < rows; row0 += warps * R) {
    Pack<T, E> kp[R], qp[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      if (row0 + r < rows) {
        kp[r] = *reinterpret_cast<const Pack<T, E>*>(k + (row0 + r) * D + lane * E);
        qp[r] = *reinterpret_cast<const Pack<T, E>*>(q + (row0 + r) * D + lane * E);
      }
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      if (row0 + r >= rows) break;
      const size_t row = row0 + r;
      const float d = qk.d ? __ldg(qk.d + (int)(row % H)) : 0.f;
      float qv[E], kv[E];
      float sq = 0.f, sk = 0.f;
#pragma unroll
      for (int e = 0; e < E; ++e) {
        kv[e] = to_f32<T>(kp[r].v[e]);
        qv[e] = to_f32<T>(qp[r].v[e]) - d * kv[e];
        sq = fmaf(qv[e], qv[e], sq);
        sk = fmaf(kv[e], kv[e], sk);
      }
      const float rq = 1.f / sqrtf(warp_sum(sq) + qk.eps), rk = 1.f / sqrtf(warp_sum(sk) + qk.eps);
      Pack<T, E> qo, ko;
#pragma unroll
      for (int e = 0; e < E; ++e) {
        qo.v[e] = from_f32<T>(qv[e] * rq);
        ko.v[e] = from_f32<T>(kv[e] * rk);
      }
      *reinterpret_cast<Pack<T, E>*>(q_out + row * D + lane * E) = qo;
      *reinterpret_cast<Pack<T, E>*>(k_out + row * D + lane * E) = ko;
    }
  }
}

template <typename TO, typename TG, int D>
__global__ void __launch_bounds__(256) out_norm_gate_kernel(size_t rows, OutPost post, TO* __restrict__ o) {
  constexpr int E = D / 32, R = kRowsPerIter;
  const int lane = threadIdx.x & 31;
  const TG* __restrict__ g = static_cast<const TG*>(post.g);
  float wv[E];
#pragma unroll
  for (int e = 0; e < E; ++e) wv[e] = post.w ? __ldg(post.w + lane * E + e) : 1.f;
  const size_t warps = (size_t)gridDim.x * (blockDim.x >> 5);
  for (size_t row0 = ((size_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * R; row0 < rows; row0 += warps * R) {
    Pack<TO, E> op[R];
    Pack<TG, E> gp[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      if (row0 + r < rows) {
        op[r] = *reinterpret_cast<const Pack<TO, E>*>(o + (row0 + r) * D + lane * E);
        gp[r] = *reinterpret_cast<const Pack<TG, E>*>(g + (row0 + r) * D + lane * E);
      }
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      if (row0 + r >= rows) break;
      const size_t row = row0 + r;
      float ov[E];
      float ss = 0.f;
#pragma unroll
      for (int e = 0; e < E; ++e) {
        ov[e] = to_f32<TO>(op[r].v[e]);
        ss = fmaf(ov[e], ov[e], ss);
      }
      const float rstd = 1.f / sqrtf(warp_sum(ss) * (1.f / D) + post.eps);
      Pack<TO, E> yo;
#pragma unroll
      for (int e = 0; e < E; ++e) {
        const float gate = 1.f / (1.f + expf(-to_f32<TG>(gp[r].v[e])));
        yo.v[e] = from_f32<TO>(gate * ov[e] * rstd * wv[e]);
      }
      *reinterpret_cast<Pack<TO, E>*>(o + row * D + lane * E) = yo;
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
  const unsigned grid = blocks_for(rows, 8 * kRowsPerIter);
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
  const unsigned grid = blocks_for(rows, 8 * kRowsPerIter);
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
