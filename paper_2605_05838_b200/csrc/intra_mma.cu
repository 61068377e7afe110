// a2 for the tensor-core path: per (chunk, head)
//   kk = K K^T, qk = Q K^T            warp-level bf16 tensor-core MMAs (fp32 accumulate), lower triangle only
//   Gamma (Eq. 10)                     column recurrences  gamma_{r,i} = alpha_r gamma_{r-1,i} + beta_r m_{r,i}
//   A = tril(alpha_r gamma_{r-1,i} eta_i kk, -1)          = (P K^T) .* Gamma^-   (Gamma^- = Gamma shifted one row down)
//   W = scale gamma_{r,i} eta_i qk                          written as bf16 hi + lo
//   T = (I + A)^{-1}                   fp32, blocked: invert the four 16x16 diagonal blocks by forward
//                                      substitution, then  T_21 = -T_22 A_21 T_11  at block sizes 16 and 32
//                                      (Eq. 15; the paper substitutes row by row over all 64 rows)
// One 128-thread CTA per (chunk, head); ~53 KB of shared memory, so four CTAs share an SM.
// The K.K^T / Q.K^T products here are 12 % of the path's FLOPs and the kernel is bound by reading
// q, k once and writing T, W: warp-level mma.sync is enough, the big contractions are in the chain kernel.
#include "mdn_common.cuh"

namespace mdn {
namespace {

constexpr int kThreads = 128;
constexpr int kD = 128;
constexpr int LDK = kD + 8;   // bf16 elements per smem row (272 B: 16-byte aligned, conflict-free for ldmatrix)
constexpr int LM = C + 1;     // fp32 elements per row of the 64x64 matrices

constexpr uint32_t kOffK = 0;
constexpr uint32_t kOffQ = C * LDK * 2;              // 17408
constexpr uint32_t kOffG = 2 * C * LDK * 2;          // 34816
constexpr uint32_t kOffCv = kOffG + C * LM * 4;      // 51456
constexpr uint32_t kSmem = kOffCv + 4 * C * 4;       // 52480
static_assert(C * LM * 4 <= C * LDK * 2, "fp32 64x64 matrices alias the bf16 tiles");

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void load_tile(__nv_bfloat16* dst, const __nv_bfloat16* src, int row_stride, int n, int tid) {
  for (int idx = tid; idx < C * (kD / 8); idx += kThreads) {
    const int r = idx >> 4, c8 = idx & 15;
    uint4 val = make_uint4(0, 0, 0, 0);
    if (r < n) val = __ldg(reinterpret_cast<const uint4*>(src + (size_t)r * row_stride) + c8);
    *reinterpret_cast<uint4*>(dst + r * LDK + c8 * 8) = val;
  }
}

__global__ void __launch_bounds__(kThreads) intra_mma_kernel(ChunkGeom g, const __nv_bfloat16* __restrict__ q,
                                                            const __nv_bfloat16* __restrict__ k,
                                                            const float* __restrict__ coef, float scale,
                                                            __nv_bfloat16* __restrict__ Tout,
                                                            __nv_bfloat16* __restrict__ Wout, size_t w_lo_offset) {
  extern __shared__ __align__(16) uint8_t smem[];
  const int slot = blockIdx.x / g.H, h = blockIdx.x % g.H;
  const SlotInfo si = slot_info(g, slot);
  if (si.seq < 0) return;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  __nv_bfloat16* Ks = reinterpret_cast<__nv_bfloat16*>(smem + kOffK);
  __nv_bfloat16* Qs = reinterpret_cast<__nv_bfloat16*>(smem + kOffQ);
  float* Gs = reinterpret_cast<float*>(smem + kOffG);     // Gamma; later T
  float* cv = reinterpret_cast<float*>(smem + kOffCv);    // alpha, beta, mu, eta
  float* Af = reinterpret_cast<float*>(smem + kOffK);     // A    (aliases the K tile once the MMAs are done)
  float* Wf = reinterpret_cast<float*>(smem + kOffQ);     // W    (aliases the Q tile); later product scratch
  float* Tf = Gs;

  const size_t tok = (size_t)si.tok0 * g.H + h;
  load_tile(Ks, k + tok * kD, g.H * kD, si.n, tid);
  load_tile(Qs, q + tok * kD, g.H * kD, si.n, tid);
  const float* cf = coef + ((size_t)slot * g.H + h) * MDN_NUM_COEF * C;
  for (int idx = tid; idx < 4 * C; idx += kThreads) cv[idx] = cf[kAlpha * C + idx];
  __syncthreads();

  // ---- Gamma columns (threads 0..63) ahead of the light MMA share of warps 0 and 1
  if (tid < C) {
    const int i = tid;
    float m = 1.f, gam = 0.f;
    for (int r = i; r < C; ++r) {
      const float al = cv[0 * C + r], be = cv[1 * C + r], mu = cv[2 * C + r];
      if (r > i) m *= mu;
      gam = fmaf(be, m, al * gam);
      Gs[r * LM + i] = gam;
    }
  }

  // ---- kk, qk for rows 16*warp .. +15, columns 0 .. 16*warp+15 (n-tiles of 8)
  float kk[8][4], qk[8][4];
#pragma unroll
  for (int t = 0; t < 8; ++t)
#pragma unroll
    for (int e = 0; e < 4; ++e) kk[t][e] = qk[t][e] = 0.f;
  {
    const int r0 = warp * 16;
    const uint32_t a_row = r0 + (lane & 7) + ((lane >> 3) & 1) * 8, a_col = (lane >> 4) * 8;
    const uint32_t b_row = (lane & 7) + (lane >> 4) * 8, b_col = ((lane >> 3) & 1) * 8;
    const uint32_t ks_base = static_cast<uint32_t>(__cvta_generic_to_shared(Ks));
    const uint32_t qs_base = static_cast<uint32_t>(__cvta_generic_to_shared(Qs));
#pragma unroll 2
    for (int ks = 0; ks < kD / 16; ++ks) {
      uint32_t ka0, ka1, ka2, ka3, qa0, qa1, qa2, qa3;
      ldmatrix_x4(ks_base + (a_row * LDK + ks * 16 + a_col) * 2, ka0, ka1, ka2, ka3);
      ldmatrix_x4(qs_base + (a_row * LDK + ks * 16 + a_col) * 2, qa0, qa1, qa2, qa3);
#pragma unroll
      for (int tp = 0; tp < 4; ++tp) {
        if (tp <= warp) {   // n-tiles 2tp, 2tp+1 cover columns 16tp .. 16tp+15
          uint32_t b0, b1, b2, b3;
          ldmatrix_x4(ks_base + ((tp * 16 + b_row) * LDK + ks * 16 + b_col) * 2, b0, b1, b2, b3);
          mma_bf16(kk[2 * tp], ka0, ka1, ka2, ka3, b0, b1);
          mma_bf16(kk[2 * tp + 1], ka0, ka1, ka2, ka3, b2, b3);
          mma_bf16(qk[2 * tp], qa0, qa1, qa2, qa3, b0, b1);
          mma_bf16(qk[2 * tp + 1], qa0, qa1, qa2, qa3, b2, b3);
        }
      }
    }
  }
  __syncthreads();   // Gamma complete; every warp is done reading the K and Q tiles

  // ---- A and W from the accumulator fragments (rows lane/4 and lane/4+8, column pairs)
  {
    const int rbase = warp * 16 + (lane >> 2), cbase = (lane & 3) * 2;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int r = rbase + (e >> 1) * 8, i = t * 8 + cbase + (e & 1);
        float av = 0.f, wv = 0.f;
        if (i <= r) {
          const float et = cv[3 * C + i];
          wv = scale * Gs[r * LM + i] * et * qk[t][e];
          if (i < r) av = cv[0 * C + r] * Gs[(r - 1) * LM + i] * et * kk[t][e];
        }
        Af[r * LM + i] = av;
        Wf[r * LM + i] = wv;
      }
    }
  }
  __syncthreads();   // A, W complete; Gamma no longer needed (T takes its place)

  const size_t mat = ((size_t)slot * g.H + h) * C * C;
  // ---- W out as bf16 hi + lo (16-byte stores), and step 1 of the inverse on threads 0..63
  for (int idx = tid; idx < C * 8; idx += kThreads) {
    const int r = idx >> 3, c0 = (idx & 7) * 8;
    __align__(16) __nv_bfloat16 hi[8], lo[8];
#pragma unroll
    for (int x = 0; x < 8; ++x) {
      const float w = Wf[r * LM + c0 + x];
      hi[x] = __float2bfloat16_rn(w);
      lo[x] = __float2bfloat16_rn(w - __bfloat162float(hi[x]));
    }
    *reinterpret_cast<uint4*>(Wout + mat + r * C + c0) = *reinterpret_cast<const uint4*>(hi);
    *reinterpret_cast<uint4*>(Wout + w_lo_offset + mat + r * C + c0) = *reinterpret_cast<const uint4*>(lo);
  }
  for (int idx = tid; idx < C * LM; idx += kThreads) Tf[idx] = 0.f;
  __syncthreads();   // W is out (its buffer becomes scratch); T zeroed

  // step 1: D_b = (I + A_bb)^{-1} for the four 16x16 diagonal blocks; thread = (block, column)
  if (tid < C) {
    const int b0 = (tid >> 4) * 16, j = tid & 15;
    float x[16];
#pragma unroll
    for (int r = 0; r < 16; ++r) {
      float acc = (r == j) ? 1.f : 0.f;
#pragma unroll
      for (int m = 0; m < r; ++m) acc = fmaf(-Af[(b0 + r) * LM + b0 + m], x[m], acc);
      x[r] = acc;
    }
#pragma unroll
    for (int r = 0; r < 16; ++r) Tf[(b0 + r) * LM + b0 + j] = x[r];
  }
  __syncthreads();

  float* Pf = Wf;   // product scratch, row stride LM
  // step 2: inside each 32x32 diagonal block s: T_lo = -D_hi (A_lo D_lo), 16x16 blocks
  {
    const int s = tid >> 6, rr = (tid & 63) >> 2, c0 = (tid & 3) * 4;
    const int R0 = 32 * s + 16, C0 = 32 * s;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
    for (int m = 0; m < 16; ++m) {
      const float av = Af[(R0 + rr) * LM + C0 + m];
#pragma unroll
      for (int x = 0; x < 4; ++x) acc[x] = fmaf(av, Tf[(C0 + m) * LM + C0 + c0 + x], acc[x]);
    }
#pragma unroll
    for (int x = 0; x < 4; ++x) Pf[(R0 + rr) * LM + c0 + x] = acc[x];
    __syncthreads();
#pragma unroll
    for (int x = 0; x < 4; ++x) acc[x] = 0.f;
#pragma unroll 4
    for (int m = 0; m < 16; ++m) {
      const float tv = Tf[(R0 + rr) * LM + R0 + m];
#pragma unroll
      for (int x = 0; x < 4; ++x) acc[x] = fmaf(tv, Pf[(R0 + m) * LM + c0 + x], acc[x]);
    }
#pragma unroll
    for (int x = 0; x < 4; ++x) Tf[(R0 + rr) * LM + C0 + c0 + x] = -acc[x];
  }
  __syncthreads();
  // step 3: T[32:64, 0:32] = -T[32:64, 32:64] (A[32:64, 0:32] T[0:32, 0:32])
  {
    const int rr = tid >> 2, c0 = (tid & 3) * 8;
    float acc[8];
#pragma unroll
    for (int x = 0; x < 8; ++x) acc[x] = 0.f;
#pragma unroll 4
    for (int m = 0; m < 32; ++m) {
      const float av = Af[(32 + rr) * LM + m];
#pragma unroll
      for (int x = 0; x < 8; ++x) acc[x] = fmaf(av, Tf[m * LM + c0 + x], acc[x]);
    }
#pragma unroll
    for (int x = 0; x < 8; ++x) Pf[rr * LM + c0 + x] = acc[x];
    __syncthreads();
#pragma unroll
    for (int x = 0; x < 8; ++x) acc[x] = 0.f;
#pragma unroll 4
    for (int m = 0; m < 32; ++m) {
      const float tv = Tf[(32 + rr) * LM + 32 + m];
#pragma unroll
      for (int x = 0; x < 8; ++x) acc[x] = fmaf(tv, Pf[m * LM + c0 + x], acc[x]);
    }
#pragma unroll
    for (int x = 0; x < 8; ++x) Tf[(32 + rr) * LM + c0 + x] = -acc[x];
  }
  __syncthreads();

  for (int idx = tid; idx < C * 8; idx += kThreads) {
    const int r = idx >> 3, c0 = (idx & 7) * 8;
    __align__(16) __nv_bfloat16 tv[8];
#pragma unroll
    for (int x = 0; x < 8; ++x) tv[x] = __float2bfloat16_rn(Tf[r * LM + c0 + x]);
    *reinterpret_cast<uint4*>(Tout + mat + r * C + c0) = *reinterpret_cast<const uint4*>(tv);
  }
}

}  // namespace

cudaError_t launch_intra_mma(const Plan& pl, const void* q, const void* k, int* launches) {
  cudaError_t e = cudaFuncSetAttribute(intra_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem);
  if (e != cudaSuccess) return e;
  const size_t n_mats = (size_t)pl.geom.num_slots * pl.p.H;
  intra_mma_kernel<<<(unsigned)n_mats, kThreads, kSmem, pl.stream>>>(
      pl.geom, static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(k),
      reinterpret_cast<const float*>(pl.ws + pl.lay.off_coef), pl.p.scale,
      reinterpret_cast<__nv_bfloat16*>(pl.ws + pl.lay.off_T), reinterpret_cast<__nv_bfloat16*>(pl.ws + pl.lay.off_W),
      n_mats * C * C);
  e = cudaGetLastError();
  if (e == cudaSuccess) ++*launches;
  return e;
}

}  // namespace mdn
