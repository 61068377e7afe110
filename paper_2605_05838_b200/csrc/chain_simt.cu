// a3 + a4, fp32 SIMT version: one CTA walks the chunks of one (sequence, head, block of
// NV value columns) in order, carrying its slices of S and M in shared memory.
//
// Per chunk (state equations and Eq. 11-12 of Section 3.1, in the form that applies T once):
//   R   = V - Diag(abar) (K S) + Diag(alpha b^-) (K M)          right-hand side of the solve
//   V~  = T R                                                    (T from the intra-chunk stage)
//   O   = scale (Diag(abar) (Q S) - Diag(b) (Q M)) + W V~        (W carries scale, Gamma, eta)
//   S' = abar_C S - b_C M + K^T Diag(gamma_C eta) V~
//   M' = mubar_C M - K^T Diag((mubar_C/mubar) eta) V~
// This equals the paper's U - Y S + Z M because T is linear and alpha_r abar_{r-1} = abar_r.
// Columns of S, M, V, V~, O never mix, so value-column blocks are independent CTAs.
#include "mdn_common.cuh"

namespace mdn {

constexpr int kChainThreads = 256;
constexpr int kNV = 32;   // value columns per CTA

template <typename TIn, int D>
__device__ __forceinline__ void load_rows_f32(float* dst, int ld, const TIn* src, int row_stride, int n, int tid) {
  constexpr int VEC = 16 / sizeof(TIn);
  constexpr int VPR = D / VEC;
  for (int idx = tid; idx < C * VPR; idx += kChainThreads) {
    const int r = idx / VPR, c = (idx % VPR) * VEC;
    if (r < n) {
      const uint4 raw = __ldg(reinterpret_cast<const uint4*>(src + (size_t)r * row_stride + c));
      const TIn* e = reinterpret_cast<const TIn*>(&raw);
#pragma unroll
      for (int x = 0; x < VEC; ++x) dst[r * ld + c + x] = to_f32<TIn>(e[x]);
    } else {
#pragma unroll
      for (int x = 0; x < VEC; ++x) dst[r * ld + c + x] = 0.f;
    }
  }
}

template <typename TIn, typename TO, int DK, int DV>
__global__ void __launch_bounds__(kChainThreads) chain_simt_kernel(
    ChunkGeom g, const TIn* __restrict__ q, const TIn* __restrict__ k, const TIn* __restrict__ v,
    const float* __restrict__ coef, const float* __restrict__ Tmat, const float* __restrict__ Wmat,
    const float* __restrict__ S0, const float* __restrict__ M0, float scale, TO* __restrict__ o,
    float* __restrict__ Sf, float* __restrict__ Mf) {
  extern __shared__ float sm[];
  constexpr int NV = kNV, LD = DK + 1, LM = C + 1, NVB = DV / NV;
  constexpr int RPT = C / 8;    // rows per thread in the row phases (8 row groups)
  constexpr int DPT = DK / 8;   // state rows per thread in the update phase
  float* Ss = sm;                 // [DK][NV]
  float* Ms = Ss + DK * NV;       // [DK][NV]
  float* Ks = Ms + DK * NV;       // [64][DK+1]
  float* Qs = Ks + C * LD;        // [64][DK+1]
  float* Rs = Qs + C * LD;        // [64][NV]
  float* Vt = Rs + C * NV;        // [64][NV]
  float* Tm = Vt + C * NV;        // [64][65]
  float* Wm = Tm + C * LM;        // [64][65]
  float* cv = Wm + C * LM;        // [6][64] abar, b, alpha*b_prev, gS, gM, mubar

  const int tid = threadIdx.x, j = tid % NV, rg = tid / NV;
  const int vb = blockIdx.x % NVB, h = (blockIdx.x / NVB) % g.H, seq = blockIdx.x / (NVB * g.H);
  const int j0 = vb * NV;
  const SeqInfo sq = seq_info(g, seq);
  const size_t st_off = ((size_t)seq * g.H + h) * DK * DV;

  for (int idx = tid; idx < DK * NV; idx += kChainThreads) {
    const int d = idx / NV, jj = idx % NV;
    Ss[idx] = S0 ? S0[st_off + (size_t)d * DV + j0 + jj] : 0.f;
    Ms[idx] = M0 ? M0[st_off + (size_t)d * DV + j0 + jj] : 0.f;
  }

  for (int c = 0; c < sq.nchunks; ++c) {
    const int slot = sq.slot0 + c;
    const int tok0 = sq.tok0 + c * C;
    const int n = min(C, sq.len - c * C);
    const size_t tok = (size_t)tok0 * g.H + h;
    __syncthreads();   // previous chunk's readers of Ks/Qs/Tm/Wm/cv/Vt are done; state is written
    load_rows_f32<TIn, DK>(Ks, LD, k + tok * DK, g.H * DK, n, tid);
    load_rows_f32<TIn, DK>(Qs, LD, q + tok * DK, g.H * DK, n, tid);
    const size_t mat = ((size_t)slot * g.H + h) * C * C;
    for (int idx = tid; idx < C * C; idx += kChainThreads) {
      Tm[(idx >> 6) * LM + (idx & 63)] = Tmat[mat + idx];
      Wm[(idx >> 6) * LM + (idx & 63)] = Wmat[mat + idx];
    }
    const float* cf = coef + ((size_t)slot * g.H + h) * MDN_NUM_COEF * C;
    for (int idx = tid; idx < kChainCoefs * C; idx += kChainThreads) cv[idx] = cf[idx];   // vectors 0..5 are contiguous
    __syncthreads();

    // ---- phase 1: K S, K M, Q S, Q M for rows rg + 8 i, column j
    float ks[RPT], km[RPT], qs[RPT], qm[RPT];
#pragma unroll
    for (int i = 0; i < RPT; ++i) ks[i] = km[i] = qs[i] = qm[i] = 0.f;
#pragma unroll 4
    for (int d = 0; d < DK; ++d) {
      const float s = Ss[d * NV + j], m = Ms[d * NV + j];
#pragma unroll
      for (int i = 0; i < RPT; ++i) {
        const int r = rg + 8 * i;
        const float kd = Ks[r * LD + d], qd = Qs[r * LD + d];
        ks[i] = fmaf(kd, s, ks[i]); km[i] = fmaf(kd, m, km[i]);
        qs[i] = fmaf(qd, s, qs[i]); qm[i] = fmaf(qd, m, qm[i]);
      }
    }
    float oacc[RPT];
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
      const int r = rg + 8 * i;
      const float abar = cv[kAbar * C + r], b = cv[kB * C + r], ab = cv[kAlphaBPrev * C + r];
      float vv = 0.f;
      if (r < n) vv = to_f32<TIn>(v[(tok + (size_t)r * g.H) * DV + j0 + j]);
      Rs[r * NV + j] = vv - abar * ks[i] + ab * km[i];
      oacc[i] = scale * (abar * qs[i] - b * qm[i]);
    }
    __syncthreads();

    // ---- phase 2: V~ = T R   (T is lower triangular with unit diagonal)
    float vt[RPT];
#pragma unroll
    for (int i = 0; i < RPT; ++i) vt[i] = 0.f;
    for (int x = 0; x < C; ++x) {
      const float rx = Rs[x * NV + j];
#pragma unroll
      for (int i = 0; i < RPT; ++i) vt[i] = fmaf(Tm[(rg + 8 * i) * LM + x], rx, vt[i]);
    }
#pragma unroll
    for (int i = 0; i < RPT; ++i) Vt[(rg + 8 * i) * NV + j] = vt[i];
    __syncthreads();

    // ---- phase 3: O = inter + W V~
    for (int x = 0; x < C; ++x) {
      const float vx = Vt[x * NV + j];
#pragma unroll
      for (int i = 0; i < RPT; ++i) oacc[i] = fmaf(Wm[(rg + 8 * i) * LM + x], vx, oacc[i]);
    }
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
      const int r = rg + 8 * i;
      if (r < n) o[(tok + (size_t)r * g.H) * DV + j0 + j] = from_f32<TO>(oacc[i]);
    }

    // ---- phase 4: state hand-over for rows rg + 8 i of S and M, column j
    float dS[DPT], dM[DPT];
#pragma unroll
    for (int i = 0; i < DPT; ++i) dS[i] = dM[i] = 0.f;
    for (int r = 0; r < C; ++r) {
      const float x = Vt[r * NV + j];
      const float xs = cv[kGS * C + r] * x, xm = cv[kGM * C + r] * x;
#pragma unroll
      for (int i = 0; i < DPT; ++i) {
        const float kd = Ks[r * LD + rg + 8 * i];
        dS[i] = fmaf(kd, xs, dS[i]);
        dM[i] = fmaf(kd, xm, dM[i]);
      }
    }
    // every thread finished reading the old state two barriers ago, and each (d, j) entry is
    // updated by the one thread that owns it: no barrier needed before the write
    const float abar_l = cv[kAbar * C + C - 1], b_l = cv[kB * C + C - 1], mubar_l = cv[kMubar * C + C - 1];
#pragma unroll
    for (int i = 0; i < DPT; ++i) {
      const int d = rg + 8 * i;
      const float s = Ss[d * NV + j], m = Ms[d * NV + j];
      Ss[d * NV + j] = abar_l * s - b_l * m + dS[i];
      Ms[d * NV + j] = mubar_l * m - dM[i];
    }
  }
  __syncthreads();
  for (int idx = tid; idx < DK * NV; idx += kChainThreads) {
    const int d = idx / NV, jj = idx % NV;
    if (Sf) Sf[st_off + (size_t)d * DV + j0 + jj] = Ss[idx];
    if (Mf) Mf[st_off + (size_t)d * DV + j0 + jj] = Ms[idx];
  }
}

template <typename TIn, typename TO, int DK, int DV>
static cudaError_t launch_one(const Plan& pl, const void* q, const void* k, const void* v, const float* S0,
                              const float* M0, void* o, float* Sf, float* Mf) {
  const size_t smem = (size_t)(2 * DK * kNV + 2 * C * (DK + 1) + 2 * C * kNV + 2 * C * (C + 1) + kChainCoefs * C) * sizeof(float);
  auto kern = chain_simt_kernel<TIn, TO, DK, DV>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const unsigned grid = (unsigned)pl.geom.num_seqs * pl.p.H * (DV / kNV);
  kern<<<grid, kChainThreads, smem, pl.stream>>>(
      pl.geom, static_cast<const TIn*>(q), static_cast<const TIn*>(k), static_cast<const TIn*>(v),
      reinterpret_cast<const float*>(pl.ws + pl.lay.off_coef), reinterpret_cast<const float*>(pl.ws + pl.lay.off_T),
      reinterpret_cast<const float*>(pl.ws + pl.lay.off_W), S0, M0, pl.p.scale, static_cast<TO*>(o), Sf, Mf);
  return cudaGetLastError();
}

template <typename TIn, typename TO>
static cudaError_t dispatch_dims(const Plan& pl, const void* q, const void* k, const void* v, const float* S0,
                                 const float* M0, void* o, float* Sf, float* Mf) {
  const int dk = pl.p.dk, dv = pl.p.dv;
  if (dk == 64 && dv == 64) return launch_one<TIn, TO, 64, 64>(pl, q, k, v, S0, M0, o, Sf, Mf);
  if (dk == 64 && dv == 128) return launch_one<TIn, TO, 64, 128>(pl, q, k, v, S0, M0, o, Sf, Mf);
  if (dk == 128 && dv == 64) return launch_one<TIn, TO, 128, 64>(pl, q, k, v, S0, M0, o, Sf, Mf);
  if (dk == 128 && dv == 128) return launch_one<TIn, TO, 128, 128>(pl, q, k, v, S0, M0, o, Sf, Mf);
  return cudaErrorInvalidValue;
}

cudaError_t launch_chain_simt(const Plan& pl, const void* q, const void* k, const void* v, const float* S0,
                              const float* M0, void* o, float* Sf, float* Mf, int* launches) {
  const bool in_bf16 = pl.p.io_dtype == MDN_BF16, o_bf16 = pl.p.o_dtype == MDN_BF16;
  cudaError_t e;
  if (!in_bf16 && !o_bf16) e = dispatch_dims<float, float>(pl, q, k, v, S0, M0, o, Sf, Mf);
  else if (in_bf16 && o_bf16) e = dispatch_dims<__nv_bfloat16, __nv_bfloat16>(pl, q, k, v, S0, M0, o, Sf, Mf);
  else if (in_bf16 && !o_bf16) e = dispatch_dims<__nv_bfloat16, float>(pl, q, k, v, S0, M0, o, Sf, Mf);
  else e = dispatch_dims<float, __nv_bfloat16>(pl, q, k, v, S0, M0, o, Sf, Mf);
  if (e == cudaSuccess) ++*launches;
  return e;
}

}  // namespace mdn
