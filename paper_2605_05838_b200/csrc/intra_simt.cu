// a2, fp32 SIMT version: per (chunk, head) the intra-chunk system of Eq. 15 and the masked
// query-key matrix of Eq. 12.
//
//   Gamma[r][i]   = gamma_{r,i}              (i <= r)   built column by column from
//                   gamma_{r,i} = alpha_r gamma_{r-1,i} + beta_r m_{r,i},  m_{r,i} = mu_r m_{r-1,i}, m_{i,i} = 1
//   A[r][i]       = alpha_r gamma_{r-1,i} eta_i (k_r . k_i)       (i < r)    = ((P K^T) .* Gamma^-)[r][i]
//   T             = (I + A)^{-1}             forward substitution, one column per thread
//   W[r][i]       = scale gamma_{r,i} eta_i (q_r . k_i)           (i <= r)
//
// Gamma^- is Gamma shifted down one row (the derivation substitutes S_{t-1}); with
// p_r = alpha_r k_r its entry is alpha_r gamma_{r-1,i}, which the column recurrence
// produces directly, with no subtraction.  All arithmetic fp32; q, k are widened on load.
#include "mdn_common.cuh"

namespace mdn {

constexpr int kIntraThreads = 256;

template <typename TIn, int DK>
__device__ __forceinline__ void load_tile_f32(float* dst /*[64][DK+1]*/, const TIn* src, int row_stride, int n,
                                              int tid) {
  constexpr int VEC = 16 / sizeof(TIn);
  constexpr int VPR = DK / VEC;  // vectors per row
  for (int idx = tid; idx < C * VPR; idx += kIntraThreads) {
    const int r = idx / VPR, c = (idx % VPR) * VEC;
    float vals[VEC];
    if (r < n) {
      const uint4 raw = __ldg(reinterpret_cast<const uint4*>(src + (size_t)r * row_stride + c));
      const TIn* e = reinterpret_cast<const TIn*>(&raw);
#pragma unroll
      for (int x = 0; x < VEC; ++x) vals[x] = to_f32<TIn>(e[x]);
    } else {
#pragma unroll
      for (int x = 0; x < VEC; ++x) vals[x] = 0.f;
    }
#pragma unroll
    for (int x = 0; x < VEC; ++x) dst[r * (DK + 1) + c + x] = vals[x];
  }
}

template <typename TOut> __device__ __forceinline__ void store_mat(TOut* dst, int idx, float x);
template <> __device__ __forceinline__ void store_mat<float>(float* dst, int idx, float x) { dst[idx] = x; }
template <> __device__ __forceinline__ void store_mat<__nv_bfloat16>(__nv_bfloat16* dst, int idx, float x) {
  dst[idx] = __float2bfloat16_rn(x);
}

// TOut = float: T and W fp32.  TOut = bf16: T bf16; W as hi part at Wout and the
// residual lo part (W - hi, rounded to bf16) at Wout + total_mats*4096.
template <typename TIn, typename TOut, int DK>
__global__ void __launch_bounds__(kIntraThreads) intra_simt_kernel(ChunkGeom g, const TIn* __restrict__ q,
                                                                  const TIn* __restrict__ k,
                                                                  const float* __restrict__ coef, float scale,
                                                                  TOut* __restrict__ Tout, TOut* __restrict__ Wout,
                                                                  size_t w_lo_offset) {
  extern __shared__ float sm[];
  const int slot = blockIdx.x / g.H, h = blockIdx.x % g.H;
  const SlotInfo si = slot_info(g, slot);
  if (si.seq < 0) return;
  const int tid = threadIdx.x;
  constexpr int LD = DK + 1, LM = C + 1;
  float* Ks = sm;                  // [64][DK+1]
  float* Qs = Ks + C * LD;         // [64][DK+1]
  float* Gs = Qs + C * LD;         // [64][65]  gamma, then W
  float* As = Gs + C * LM;         // [64][65]  alpha_r gamma_{r-1,i}, then A
  float* Ts = As + C * LM;         // [64][65]
  float* cv = Ts + C * LM;         // [4][64]   alpha, beta, mu, eta

  const size_t tok = (size_t)si.tok0 * g.H + h;
  load_tile_f32<TIn, DK>(Ks, k + tok * DK, g.H * DK, si.n, tid);
  load_tile_f32<TIn, DK>(Qs, q + tok * DK, g.H * DK, si.n, tid);
  const float* cf = coef + ((size_t)slot * g.H + h) * MDN_NUM_COEF * C;
  {
    const int which = tid >> 6, r = tid & 63;   // 4 vectors x 64
    cv[which * C + r] = cf[(kAlpha + which) * C + r];
  }
  for (int idx = tid; idx < C * LM; idx += kIntraThreads) { Gs[idx] = 0.f; As[idx] = 0.f; }
  __syncthreads();

  if (tid < C) {   // column i of Gamma and of the shifted mask
    const int i = tid;
    float m = 1.f, gprev = 0.f;
    for (int r = i; r < C; ++r) {
      const float al = cv[0 * C + r], be = cv[1 * C + r], mu = cv[2 * C + r];
      if (r > i) m *= mu;
      const float shifted = al * gprev;          // alpha_r gamma_{r-1,i}
      const float gam = fmaf(be, m, shifted);    // gamma_{r,i}
      Gs[r * LM + i] = gam;
      As[r * LM + i] = shifted;
      gprev = gam;
    }
  }
  __syncthreads();

  for (int idx = tid; idx < C * C; idx += kIntraThreads) {
    const int r = idx >> 6, i = idx & 63;
    if (i <= r) {
      const float* kr = Ks + r * LD;
      const float* ki = Ks + i * LD;
      const float* qr = Qs + r * LD;
      float kk = 0.f, qk = 0.f;
#pragma unroll 8
      for (int d = 0; d < DK; ++d) {
        const float kid = ki[d];
        kk = fmaf(kr[d], kid, kk);
        qk = fmaf(qr[d], kid, qk);
      }
      const float et = cv[3 * C + i];
      Gs[r * LM + i] = scale * Gs[r * LM + i] * et * qk;         // W
      As[r * LM + i] = (i < r) ? As[r * LM + i] * et * kk : 0.f;  // A (strictly lower)
    }
  }
  __syncthreads();

  if (tid < C) {   // T = (I + A)^{-1}: column j by forward substitution
    const int j = tid;
    for (int r = 0; r < C; ++r) {
      float acc = (r == j) ? 1.f : 0.f;
      const float* ar = As + r * LM;
      for (int i = 0; i < r; ++i) acc = fmaf(-ar[i], Ts[i * LM + j], acc);
      Ts[r * LM + j] = acc;
    }
  }
  __syncthreads();

  const size_t mat = ((size_t)slot * g.H + h) * C * C;
  for (int idx = tid; idx < C * C; idx += kIntraThreads) {
    const int r = idx >> 6, i = idx & 63;
    const float t = Ts[r * LM + i], w = Gs[r * LM + i];
    store_mat<TOut>(Tout + mat, idx, t);
    store_mat<TOut>(Wout + mat, idx, w);
    if (sizeof(TOut) == 2) {
      const float hi = to_f32<TOut>(from_f32<TOut>(w));
      store_mat<TOut>(Wout + w_lo_offset + mat, idx, w - hi);
    }
  }
}

template <typename TIn, typename TOut, int DK>
static cudaError_t launch_one(const Plan& pl, const void* q, const void* k) {
  const size_t smem = (size_t)(2 * C * (DK + 1) + 3 * C * (C + 1) + 4 * C) * sizeof(float);
  auto kern = intra_simt_kernel<TIn, TOut, DK>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const size_t n_mats = (size_t)pl.geom.num_slots * pl.p.H;
  kern<<<(unsigned)n_mats, kIntraThreads, smem, pl.stream>>>(
      pl.geom, static_cast<const TIn*>(q), static_cast<const TIn*>(k),
      reinterpret_cast<const float*>(pl.ws + pl.lay.off_coef), pl.p.scale,
      reinterpret_cast<TOut*>(pl.ws + pl.lay.off_T), reinterpret_cast<TOut*>(pl.ws + pl.lay.off_W),
      n_mats * C * C);
  return cudaGetLastError();
}

cudaError_t launch_intra_simt(const Plan& pl, const void* q, const void* k, int* launches) {
  const bool in_bf16 = pl.p.io_dtype == MDN_BF16, out_bf16 = pl.lay.mat_dtype == MDN_BF16;
  cudaError_t e = cudaErrorInvalidValue;
  if (pl.p.dk == 64) {
    if (!in_bf16 && !out_bf16) e = launch_one<float, float, 64>(pl, q, k);
    else if (in_bf16 && !out_bf16) e = launch_one<__nv_bfloat16, float, 64>(pl, q, k);
    else if (in_bf16 && out_bf16) e = launch_one<__nv_bfloat16, __nv_bfloat16, 64>(pl, q, k);
  } else if (pl.p.dk == 128) {
    if (!in_bf16 && !out_bf16) e = launch_one<float, float, 128>(pl, q, k);
    else if (in_bf16 && !out_bf16) e = launch_one<__nv_bfloat16, float, 128>(pl, q, k);
    else if (in_bf16 && out_bf16) e = launch_one<__nv_bfloat16, __nv_bfloat16, 128>(pl, q, k);
  }
  if (e == cudaSuccess) ++*launches;
  return e;
}

}  // namespace mdn
