// a2 for the tensor-core path: per (chunk, head)
//   kk = K K^T, qk = Q K^T            warp-level bf16 tensor-core MMAs (fp32 accumulate), lower triangle only;
//                                      K, Q tiles arrive by TMA (128-byte swizzle), fragments by swizzled ldmatrix
//   Gamma (Eq. 10)                     column recurrences  gamma_{r,i} = alpha_r gamma_{r-1,i} + beta_r m_{r,i}
//   A = tril(alpha_r gamma_{r-1,i} eta_i kk, -1)          = (P K^T) .* Gamma^-   (Gamma^- = Gamma shifted one row down)
//   W = scale gamma_{r,i} eta_i qk                          written from the fragments as bf16 hi + lo
//   T = (I + A)^{-1}                   blocked: the four 16x16 diagonal blocks by fp32 forward substitution, then
//                                      T_21 = -T_22 A_21 T_11 at block sizes 16 and 32 with tf32 tensor-core MMAs
//                                      (Eq. 15; the paper substitutes row by row over all 64 rows).  T leaves as bf16,
//                                      so tf32 (10-bit mantissa) block products cost nothing visible.
// One 128-thread CTA per (chunk, head); ~51 KB of shared memory, four CTAs per SM.
// The K K^T / Q K^T products are 12 % of the path's FLOPs and this kernel is bound by reading q, k
// once and writing T, W: warp-level mma.sync is enough here, the big contractions are in the chain kernel.
#include <cstring>

#include "coeff_scan.cuh"
#include "mdn_common.cuh"
#include "tc_utils.cuh"

namespace mdn {
namespace {

using namespace tc;

constexpr int kThreads = 128;
constexpr int kD = 128;
constexpr int LM = C + 4;     // fp32 elements per row of the 64x64 matrices (16-byte aligned rows)

constexpr uint32_t kOffK = 0, kOffQ = 16384;                 // bf16 tiles, two [64 x 128 B] swizzled blocks each
constexpr uint32_t kOffG = 32768;                            // Gamma [64][68] fp32; later T
constexpr uint32_t kOffCv = kOffG + C * LM * 4;              // alpha, beta, mu, eta, then the q/k-norm vectors
constexpr int kCvVecs = 12;                                  // + gamma_C eta, (mubar_C/mubar) eta, 1/|k|, 1/|q - dk|, |q|^2, q.k, |k|^2
// the tile area is reused once the MMAs are done: first as the bf16 staging of W_hi / W_lo, then for A and scratch
constexpr int LW = C + 8;                                    // bf16 elements per staged W row (144 B: conflict-free)
constexpr uint32_t kOffWh = 0, kOffWl = C * LW * 2;          // W_hi, W_lo staging [64][72] bf16
constexpr uint32_t kOffA = 0;                                // A [64][68] fp32
constexpr int LD16 = 16 * 16 + 4;                            // floats per compact 16x16 diagonal block (+4: bank shift)
constexpr uint32_t kOffAd = C * LM * 4;                      // the four diagonal blocks of A, compact
constexpr uint32_t kOffP = kOffAd + 4 * LD16 * 4;            // product scratch [32][68] fp32
constexpr uint32_t kSmem = kOffCv + kCvVecs * C * 4 + 1024;        // + slack for the 1024-byte alignment
static_assert(kOffP + 32 * LM * 4 <= kOffG && kOffWl + C * LW * 2 <= kOffG, "reuse of the tile area");

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
__device__ __forceinline__ uint32_t to_tf32(float x) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ void mma_tf32(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Byte offset of the 16-byte chunk `c16` (0..15 over the 128 columns) of row `row` in a swizzled tile.
__device__ __forceinline__ uint32_t tile_chunk(uint32_t row, uint32_t c16) {
  return (c16 >> 3) * 8192 + row * 128 + (((c16 & 7) ^ (row & 7)) << 4);
}

// C[16 x 8*NT] (+)= A[16 x 8*KS] * B[8*KS x 8*NT], fp32 matrices in shared memory (row stride LM), tf32 MMAs.
// a: &A[row0][k0], b: &B[k0][col0].  Fragment coordinates: g = lane / 4, t = lane % 4.
template <int KS, int NT>
__device__ __forceinline__ void block_mma_tf32(float (&acc)[NT][4], const float* a, const float* b, int g, int t) {
#pragma unroll
  for (int ks = 0; ks < KS; ++ks) {
    uint32_t af[4];
    af[0] = to_tf32(a[g * LM + ks * 8 + t]);
    af[1] = to_tf32(a[(g + 8) * LM + ks * 8 + t]);
    af[2] = to_tf32(a[g * LM + ks * 8 + t + 4]);
    af[3] = to_tf32(a[(g + 8) * LM + ks * 8 + t + 4]);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const uint32_t b0 = to_tf32(b[(ks * 8 + t) * LM + nt * 8 + g]);
      const uint32_t b1 = to_tf32(b[(ks * 8 + t + 4) * LM + nt * 8 + g]);
      mma_tf32(acc[nt], af, b0, b1);
    }
  }
}

__global__ void __launch_bounds__(kThreads) intra_mma_kernel(ChunkGeom g, const __grid_constant__ CUtensorMap map_q,
                                                            const __grid_constant__ CUtensorMap map_k,
                                                            float* __restrict__ coef, GateArgs gates, GateParam gp,
                                                            QkNorm qkn, float scale,
                                                            __nv_bfloat16* __restrict__ Tout,
                                                            __nv_bfloat16* __restrict__ Wout, size_t w_lo_offset,
                                                            int32_t* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ __align__(8) uint64_t bar_tiles;
  __shared__ int abort_flag;
  const int slot = blockIdx.x / g.H, h = blockIdx.x % g.H;
  grid_dependency_wait();   // chunk map and coefficients come from the previous kernels
  const SlotInfo si = slot_info(g, slot);
  if (si.seq < 0) return;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int fg = lane >> 2, ft = lane & 3;   // MMA fragment coordinates
  float* Gs = reinterpret_cast<float*>(smem + kOffG);     // Gamma; later T
  float* cv = reinterpret_cast<float*>(smem + kOffCv);
  float* Af = reinterpret_cast<float*>(smem + kOffA);
  float* Ad = reinterpret_cast<float*>(smem + kOffAd);
  float* Pf = reinterpret_cast<float*>(smem + kOffP);
  __nv_bfloat16* Wsh = reinterpret_cast<__nv_bfloat16*>(smem + kOffWh);
  __nv_bfloat16* Wsl = reinterpret_cast<__nv_bfloat16*>(smem + kOffWl);
  float* Tf = Gs;
  const uint32_t bar = smem_u32(&bar_tiles);
  const uint32_t s_base = smem_u32(smem);

  if (tid == 0) {
    abort_flag = 0;
    mbar_init(bar, 1);
    mbar_fence_init();
    mbar_arrive_expect_tx(bar, 32768);
    tma_load_2d(s_base + kOffK, &map_k, h * kD, si.tok0, bar);
    tma_load_2d(s_base + kOffK + 8192, &map_k, h * kD + 64, si.tok0, bar);
    tma_load_2d(s_base + kOffQ, &map_q, h * kD, si.tok0, bar);
    tma_load_2d(s_base + kOffQ + 8192, &map_q, h * kD + 64, si.tok0, bar);
  }
  float* cf = coef + ((size_t)slot * g.H + h) * MDN_NUM_COEF * C;
  if (gates.log_alpha == nullptr) {
    for (int idx = tid; idx < 4 * C; idx += kThreads) cv[idx] = cf[kAlpha * C + idx];
    if (qkn.on)
      for (int idx = tid; idx < 2 * C; idx += kThreads) {   // gamma_C eta, (mubar_C/mubar) eta; alpha b^-
        cv[4 * C + idx] = cf[kGS * C + idx];
        if (idx < C) cv[11 * C + idx] = cf[kAlphaBPrev * C + idx];
      }
    __syncthreads();   // coefficients in smem; barrier initialised before anyone waits on it
  } else {
    // fused coefficient scan (Eq. 10): this head's gates (stride H floats), then one warp runs the scans,
    // keeps alpha, beta, mu, eta in smem for the Gamma recurrence and writes the chain kernel's six vectors
    if (tid < C) {
      const bool valid = tid < si.n;
      const size_t gi = ((size_t)si.tok0 + tid) * g.H + h;
      TokenGates tg{1.f, 1.f, 0.f, 0.f};
      if (valid)
        tg = load_token_gates(gp, h, __ldg(gates.log_alpha + gi), __ldg(gates.log_mu + gi), __ldg(gates.beta + gi),
                              gates.eta ? __ldg(gates.eta + gi) : 1.f);
      cv[0 * C + tid] = tg.alpha;
      cv[1 * C + tid] = tg.beta;
      cv[2 * C + tid] = tg.mu;
      cv[3 * C + tid] = tg.eta;
    }
    __syncthreads();   // gates in smem; barrier initialised before anyone waits on it
    if (warp == 3) {   // an otherwise idle warp, concurrently with the Gamma recurrence of warps 0 and 1
      const float2 a2 = reinterpret_cast<const float2*>(cv + 0 * C)[lane], b2 = reinterpret_cast<const float2*>(cv + 1 * C)[lane];
      const float2 m2 = reinterpret_cast<const float2*>(cv + 2 * C)[lane], e2 = reinterpret_cast<const float2*>(cv + 3 * C)[lane];
      const float al[2] = {a2.x, a2.y}, be[2] = {b2.x, b2.y}, mu[2] = {m2.x, m2.y}, et[2] = {e2.x, e2.y};
      const HeadCoefs hc = scan_head(al, mu, be, et, lane);
      auto put = [&](int which, float x0, float x1) { reinterpret_cast<float2*>(cf + which * C)[lane] = make_float2(x0, x1); };
      put(kAbar, hc.abar[0], hc.abar[1]);
      put(kB, hc.b[0], hc.b[1]);
      put(kAlphaBPrev, hc.ab_prev[0], hc.ab_prev[1]);
      put(kGS, hc.gs[0], hc.gs[1]);
      put(kGM, hc.gm[0], hc.gm[1]);
      put(kMubar, hc.mubar[0], hc.mubar[1]);
      if (qkn.on) {   // the last-row weights get their 1/|k| factor once the norms are known
        reinterpret_cast<float2*>(cv + 4 * C)[lane] = make_float2(hc.gs[0], hc.gs[1]);
        reinterpret_cast<float2*>(cv + 5 * C)[lane] = make_float2(hc.gm[0], hc.gm[1]);
        reinterpret_cast<float2*>(cv + 11 * C)[lane] = make_float2(hc.ab_prev[0], hc.ab_prev[1]);
      } else {
        put(kRk, 1.f, 1.f);
        put(kRq, 1.f, 1.f);
      }
    }
  }

  // ---- Gamma columns (threads 0..63) while the tiles are in flight
  if (tid < C) {
    const int i = tid;
    float m = 1.f, gam = 0.f;
    int r4 = i & ~3;
    {   // first group of four: rows below i are skipped
      const float4 al = *reinterpret_cast<const float4*>(cv + 0 * C + r4);
      const float4 be = *reinterpret_cast<const float4*>(cv + 1 * C + r4);
      const float4 mu = *reinterpret_cast<const float4*>(cv + 2 * C + r4);
      const float alv[4] = {al.x, al.y, al.z, al.w}, bev[4] = {be.x, be.y, be.z, be.w}, muv[4] = {mu.x, mu.y, mu.z, mu.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int r = r4 + e;
        if (r >= i) {
          if (r > i) m *= muv[e];
          gam = fmaf(bev[e], m, alv[e] * gam);
          Gs[r * LM + i] = gam;
        }
      }
    }
    for (r4 += 4; r4 < C; r4 += 4) {
      const float4 al = *reinterpret_cast<const float4*>(cv + 0 * C + r4);
      const float4 be = *reinterpret_cast<const float4*>(cv + 1 * C + r4);
      const float4 mu = *reinterpret_cast<const float4*>(cv + 2 * C + r4);
      float* grow = Gs + r4 * LM + i;
      m *= mu.x; gam = fmaf(be.x, m, al.x * gam); grow[0] = gam;
      m *= mu.y; gam = fmaf(be.y, m, al.y * gam); grow[LM] = gam;
      m *= mu.z; gam = fmaf(be.z, m, al.z * gam); grow[2 * LM] = gam;
      m *= mu.w; gam = fmaf(be.w, m, al.w * gam); grow[3 * LM] = gam;
    }
  }

  bool ok = mbar_wait(bar, 0, &abort_flag);
  __syncwarp();

  // ---- kk, qk for rows 16*warp .. +15, columns 0 .. 16*warp+15 (n-tiles of 8)
  float kk[8][4], qk[8][4];
#pragma unroll
  for (int t = 0; t < 8; ++t)
#pragma unroll
    for (int e = 0; e < 4; ++e) kk[t][e] = qk[t][e] = 0.f;
  if (ok) {
    const uint32_t a_row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, a_c = lane >> 4;
    const uint32_t b_row = (lane & 7) + (lane >> 4) * 8, b_c = (lane >> 3) & 1;
    const uint32_t ks_base = s_base + kOffK, qs_base = s_base + kOffQ;
#pragma unroll 2
    for (int ks = 0; ks < kD / 16; ++ks) {
      uint32_t ka0, ka1, ka2, ka3, qa0, qa1, qa2, qa3;
      ldmatrix_x4(ks_base + tile_chunk(a_row, ks * 2 + a_c), ka0, ka1, ka2, ka3);
      ldmatrix_x4(qs_base + tile_chunk(a_row, ks * 2 + a_c), qa0, qa1, qa2, qa3);
#pragma unroll
      for (int tp = 0; tp < 4; ++tp) {
        if (tp <= warp) {   // n-tiles 2tp, 2tp+1 cover columns 16tp .. 16tp+15
          uint32_t b0, b1, b2, b3;
          ldmatrix_x4(ks_base + tile_chunk(tp * 16 + b_row, ks * 2 + b_c), b0, b1, b2, b3);
          mma_bf16(kk[2 * tp], ka0, ka1, ka2, ka3, b0, b1);
          mma_bf16(kk[2 * tp + 1], ka0, ka1, ka2, ka3, b2, b3);
          mma_bf16(qk[2 * tp], qa0, qa1, qa2, qa3, b0, b1);
          mma_bf16(qk[2 * tp + 1], qa0, qa1, qa2, qa3, b2, b3);
        }
      }
    }
  }
  if (qkn.on) {
    // fused q/k norm: |k_r|^2 and q_r . k_r are the diagonals of the two products; |q_r|^2 is summed from the
    // Q tile (two threads per row); then  |q - d k|^2 = |q|^2 - 2 d q.k + d^2 |k|^2
    if (ok) {
      const int row = tid >> 1, hb = tid & 1;
      float ssq = 0.f;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint4 u = *reinterpret_cast<const uint4*>(smem + kOffQ + tile_chunk(row, hb * 8 + j));
        const uint32_t w4[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float lo = __uint_as_float(w4[e] << 16), hi = __uint_as_float(w4[e] & 0xffff0000u);
          ssq = fmaf(lo, lo, fmaf(hi, hi, ssq));
        }
      }
      ssq += __shfl_xor_sync(0xffffffffu, ssq, 1);
      if (hb == 0) cv[8 * C + row] = ssq;
    }
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      if ((t >> 1) == warp) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int r = warp * 16 + fg + (e >> 1) * 8, i = t * 8 + ft * 2 + (e & 1);
          if (r == i) { cv[9 * C + r] = qk[t][e]; cv[10 * C + r] = kk[t][e]; }
        }
      }
    }
    __syncthreads();
    if (tid < C) {
      const float dh = qkn.d ? __ldg(qkn.d + h) : 0.f;
      const float nk2 = cv[10 * C + tid], nq2 = cv[8 * C + tid], qkd = cv[9 * C + tid];
      const float rk = 1.f / sqrtf(nk2 + qkn.eps);
      const float rq = 1.f / sqrtf(fmaxf(nq2 - 2.f * dh * qkd + dh * dh * nk2, 0.f) + qkn.eps);
      cv[6 * C + tid] = rk;
      cv[7 * C + tid] = rq;
      cf[kGS * C + tid] = cv[4 * C + tid] * rk;
      cf[kGM * C + tid] = cv[5 * C + tid] * rk;
      cf[kAlphaBPrev * C + tid] = cv[11 * C + tid] * rk;
      cf[kRk * C + tid] = rk;
      cf[kRq * C + tid] = rq;
    }
  }
  __syncthreads();   // Gamma complete; every warp is done reading the K and Q tiles

  // ---- W and A from the accumulator fragments (rows fg and fg + 8 of the warp's 16, column pairs), one pass:
  // W goes to the bf16 staging, A stays in the kk registers until the staging has been written out.
  // Tiles left of the warp's diagonal block need no mask, tiles right of it are zero; tokens past the end of a
  // short chunk (rows >= n hold another sequence's data) are masked.
  const size_t mat = ((size_t)slot * g.H + h) * C * C;
  const int rbase = warp * 16 + fg, cbase = ft * 2;
#pragma unroll
  for (int t = 0; t < 8; ++t) {
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const int r = rbase + half * 8, i0 = t * 8 + cbase;
      float wv0 = 0.f, wv1 = 0.f, av0 = 0.f, av1 = 0.f;
      if ((t >> 1) <= warp && r < si.n) {
        const float2 gw = *reinterpret_cast<const float2*>(Gs + r * LM + i0);
        const float2 et = *reinterpret_cast<const float2*>(cv + 3 * C + i0);
        const float alr = cv[0 * C + r];
        float2 ga = make_float2(0.f, 0.f);
        if (r > 0) ga = *reinterpret_cast<const float2*>(Gs + (r - 1) * LM + i0);
        float q0 = qk[t][half * 2], q1 = qk[t][half * 2 + 1], k0 = kk[t][half * 2], k1 = kk[t][half * 2 + 1];
        if (qkn.on) {   // (q_r - d k_r) . k_i / (|q_r - d k_r| |k_i|)  and  k_r . k_i / (|k_r| |k_i|)
          const float dh = qkn.d ? __ldg(qkn.d + h) : 0.f;
          const float2 rki = *reinterpret_cast<const float2*>(cv + 6 * C + i0);
          const float rkr = cv[6 * C + r], rqr = cv[7 * C + r];
          q0 = (q0 - dh * k0) * rqr * rki.x; q1 = (q1 - dh * k1) * rqr * rki.y;
          k0 *= rkr * rki.x; k1 *= rkr * rki.y;
        }
        wv0 = scale * gw.x * et.x * q0;
        wv1 = scale * gw.y * et.y * q1;
        av0 = alr * ga.x * et.x * k0;
        av1 = alr * ga.y * et.y * k1;
        if ((t >> 1) == warp) {   // diagonal block: W keeps i <= r, A keeps i < r
          if (i0 > r) { wv0 = 0.f; }
          if (i0 + 1 > r) { wv1 = 0.f; }
          if (i0 >= r) { av0 = 0.f; }
          if (i0 + 1 >= r) { av1 = 0.f; }
        }
      }
      kk[t][half * 2] = av0;
      kk[t][half * 2 + 1] = av1;
      uint32_t hi, lo;
      split_pack_bf16(wv0, wv1, hi, lo);
      *reinterpret_cast<uint32_t*>(Wsh + r * LW + i0) = hi;
      *reinterpret_cast<uint32_t*>(Wsl + r * LW + i0) = lo;
    }
  }
  __syncthreads();
  for (int idx = tid; idx < C * 8; idx += kThreads) {   // coalesced 16-byte stores of W_hi, W_lo
    const int r = idx >> 3, c0 = (idx & 7) * 8;
    *reinterpret_cast<uint4*>(Wout + mat + r * C + c0) = *reinterpret_cast<const uint4*>(Wsh + r * LW + c0);
    *reinterpret_cast<uint4*>(Wout + w_lo_offset + mat + r * C + c0) = *reinterpret_cast<const uint4*>(Wsl + r * LW + c0);
  }
  __syncthreads();   // staging read out; the area now takes A
#pragma unroll
  for (int t = 0; t < 8; ++t) {
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const int r = rbase + half * 8, i0 = t * 8 + cbase;
      const float2 av = make_float2(kk[t][half * 2], kk[t][half * 2 + 1]);
      *reinterpret_cast<float2*>(Af + r * LM + i0) = av;
      if ((t >> 1) == warp)   // the warp's diagonal 16x16 block, kept compact for the forward substitution
        *reinterpret_cast<float2*>(Ad + warp * LD16 + (r - warp * 16) * 16 + (i0 - warp * 16)) = av;
    }
  }
  __syncthreads();   // A complete; Gamma no longer needed (T takes its place)
  for (int idx = tid; idx < C * LM / 4; idx += kThreads) reinterpret_cast<float4*>(Tf)[idx] = make_float4(0.f, 0.f, 0.f, 0.f);
  __syncthreads();

  // step 1: D_b = (I + A_bb)^{-1} for the four 16x16 diagonal blocks; thread = (block, column), fp32
  if (tid < C) {
    const int b0 = (tid >> 4) * 16, j = tid & 15;
    float x[16];
#pragma unroll
    for (int r = 0; r < 16; ++r) {
      float arow[16];
#pragma unroll
      for (int m4 = 0; m4 < 16; m4 += 4) {
        if (m4 < r) {
          const float4 v4 = *reinterpret_cast<const float4*>(Ad + (tid >> 4) * LD16 + r * 16 + m4);
          arow[m4] = v4.x; arow[m4 + 1] = v4.y; arow[m4 + 2] = v4.z; arow[m4 + 3] = v4.w;
        }
      }
      float acc = (r == j) ? 1.f : 0.f;
#pragma unroll
      for (int m = 0; m < r; ++m) acc = fmaf(-arow[m], x[m], acc);
      x[r] = acc;
    }
#pragma unroll
    for (int r = 0; r < 16; ++r) Tf[(b0 + r) * LM + b0 + j] = x[r];
  }
  __syncthreads();

  // step 2: inside each 32x32 diagonal block s: T_lo = -D_hi (A_lo D_lo); 16x16 blocks, warp s does block s
  if (warp < 2) {
    const int R0 = 32 * warp + 16, C0 = 32 * warp;
    float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    block_mma_tf32<2, 2>(acc, Af + R0 * LM + C0, Tf + C0 * LM + C0, fg, ft);
    float* P = Pf + warp * 16 * LM;
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      *reinterpret_cast<float2*>(P + fg * LM + nt * 8 + 2 * ft) = make_float2(acc[nt][0], acc[nt][1]);
      *reinterpret_cast<float2*>(P + (fg + 8) * LM + nt * 8 + 2 * ft) = make_float2(acc[nt][2], acc[nt][3]);
    }
    __syncwarp();
    float acc2[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    block_mma_tf32<2, 2>(acc2, Tf + R0 * LM + R0, P, fg, ft);
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      *reinterpret_cast<float2*>(Tf + (R0 + fg) * LM + C0 + nt * 8 + 2 * ft) = make_float2(-acc2[nt][0], -acc2[nt][1]);
      *reinterpret_cast<float2*>(Tf + (R0 + fg + 8) * LM + C0 + nt * 8 + 2 * ft) = make_float2(-acc2[nt][2], -acc2[nt][3]);
    }
  }
  __syncthreads();
  // step 3: T[32:64, 0:32] = -T[32:64, 32:64] (A[32:64, 0:32] T[0:32, 0:32]); warp = (row tile, column half)
  {
    const int mt = warp & 1, n0 = (warp >> 1) * 16;
    float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    block_mma_tf32<4, 2>(acc, Af + (32 + 16 * mt) * LM, Tf + n0, fg, ft);
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      *reinterpret_cast<float2*>(Pf + (16 * mt + fg) * LM + n0 + nt * 8 + 2 * ft) = make_float2(acc[nt][0], acc[nt][1]);
      *reinterpret_cast<float2*>(Pf + (16 * mt + fg + 8) * LM + n0 + nt * 8 + 2 * ft) = make_float2(acc[nt][2], acc[nt][3]);
    }
    __syncthreads();
    float acc2[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    block_mma_tf32<4, 2>(acc2, Tf + (32 + 16 * mt) * LM + 32, Pf + n0, fg, ft);
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      *reinterpret_cast<float2*>(Tf + (32 + 16 * mt + fg) * LM + n0 + nt * 8 + 2 * ft) = make_float2(-acc2[nt][0], -acc2[nt][1]);
      *reinterpret_cast<float2*>(Tf + (32 + 16 * mt + fg + 8) * LM + n0 + nt * 8 + 2 * ft) = make_float2(-acc2[nt][2], -acc2[nt][3]);
    }
  }
  __syncthreads();

  for (int idx = tid; idx < C * 8; idx += kThreads) {
    const int r = idx >> 3, c0 = (idx & 7) * 8;
    const float4 t0 = *reinterpret_cast<const float4*>(Tf + r * LM + c0);
    const float4 t1 = *reinterpret_cast<const float4*>(Tf + r * LM + c0 + 4);
    uint4 packed;
    packed.x = pack_bf16(t0.x, t0.y); packed.y = pack_bf16(t0.z, t0.w);
    packed.z = pack_bf16(t1.x, t1.y); packed.w = pack_bf16(t1.z, t1.w);
    *reinterpret_cast<uint4*>(Tout + mat + r * C + c0) = packed;
  }
  if (!ok && tid == 0) atomicCAS(status, kDevOk, kDevTimeout);
  grid_launch_dependents();
}

}  // namespace

cudaError_t launch_intra_mma(const Plan& pl, const void* q, const void* k, const GateArgs& gates, int* launches) {
  cudaError_t e = cudaFuncSetAttribute(intra_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem);
  if (e != cudaSuccess) return e;
  const size_t n_mats = (size_t)pl.geom.num_slots * pl.p.H;
  const uint64_t tokens = (uint64_t)pl.p.B * pl.p.T, row = (uint64_t)pl.p.H * kD;
  CUtensorMap mq, mk;
  if (!encode_tma_2d_bf16(&mq, TmaMap2D{q, row, tokens, row * 2, 64, 64, true}) ||
      !encode_tma_2d_bf16(&mk, TmaMap2D{k, row, tokens, row * 2, 64, 64, true}))
    return cudaErrorInvalidValue;
  e = launch_pdl(intra_mma_kernel, dim3((unsigned)n_mats), dim3(kThreads), kSmem, pl.stream, pl.geom, mq, mk,
                 reinterpret_cast<float*>(pl.ws + pl.lay.off_coef), gates, pl.gp, pl.qk, pl.p.scale,
                 reinterpret_cast<__nv_bfloat16*>(pl.ws + pl.lay.off_T),
                 reinterpret_cast<__nv_bfloat16*>(pl.ws + pl.lay.off_W), n_mats * C * C,
                 reinterpret_cast<int32_t*>(pl.ws + pl.lay.off_status));
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e == cudaSuccess) ++*launches;
  return e;
}

}  // namespace mdn
