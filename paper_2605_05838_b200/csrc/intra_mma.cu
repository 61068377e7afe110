// a2 for the tensor-core path: per (chunk, head)
//   [K K^T ; Q K^T]                    ONE tcgen05 product: A = the K tile stacked on the Q tile (128 rows), B = the K
//                                      tile, fp32 accumulator in tensor memory (128 lanes x 64 columns); K, Q arrive
//                                      by TMA (128-byte swizzle) laid out so that the stack is one K-major operand.
//                                      Lane r holds row r of K K^T, lane 64 + r row r of Q K^T: the threads of
//                                      warps 0, 1 each turn one row into A, those of warps 2, 3 one row into W.
//   Gamma (Eq. 10)                     each thread builds ITS row of Gamma in registers, right to left:
//                                      gamma_{r,i} = mu_{i+1} gamma_{r,i+1} + beta_i prod_{i<l<=r} alpha_l
//                                      (the column recurrence gamma_{r,i} = alpha_r gamma_{r-1,i} + beta_r m_{r,i}
//                                      unrolled along the row), while the tiles and the product are in flight
//   A = tril(alpha_r gamma_{r-1,i} eta_i kk, -1)          = (P K^T) .* Gamma^-   (Gamma^- = Gamma shifted one row down)
//   W = scale gamma_{r,i} eta_i qk                          staged as bf16 hi + lo, written out in 16-byte pieces
//   T = (I + A)^{-1}                   blocked: the four 16x16 diagonal blocks by fp32 forward substitution, then
//                                      T_21 = -T_22 A_21 T_11 at block sizes 16 and 32 with tf32 tensor-core MMAs
//                                      (Eq. 15; the paper substitutes row by row over all 64 rows).  T leaves as bf16,
//                                      so tf32 (10-bit mantissa) block products cost nothing visible.
// With the fused q/k norm a W thread also needs its row of K K^T ((q - d k) . k_i = Q K^T - d K K^T), which the product
// leaves in another warp's lanes: the A thread of that row passes it through the row's slot of the W staging area
// (one block barrier; a first version loaded the K tile a second time and ran a second product: 52 KB, 128 columns,
// four CTAs per SM).
// One 128-thread CTA per (chunk, head); 36 KB of shared memory (the operand tiles, reused for the W staging, A and
// T) and 64 columns of tensor memory.  Tensor memory is released before the CTA signals its dependents, so the chain kernel
// (which takes all 512 columns of an SM) can never be resident beside a CTA of this kernel that still has to allocate.
#include <cstring>
#include <type_traits>

#include "coeff_scan.cuh"
#include "mdn_common.cuh"
#include "tc_utils.cuh"

namespace mdn {
namespace {

using namespace tc;

constexpr int kThreads = 128;
constexpr int kCtasPerSm = 5;
constexpr int kD = 128;
constexpr int LM = C + 4;     // fp32 elements per row of T (16-byte aligned rows)

// operand tiles, bf16, [64 rows x 128 B] swizzled blocks: K (dk 0..63) | Q (dk 0..63) | K (dk 64..127) | Q (..)
// so that rows 0..127 of each 16 KB half are K stacked on Q
struct Lay {
  uint32_t k1, cv, tiles, smem;   // offset of the second half, of the vectors; tile bytes; dynamic shared memory
};
constexpr uint32_t kOffK0 = 0, kOffQ0 = 8192;
constexpr int kCvVecs = 12;                                  // + gamma_C eta, (mubar_C/mubar) eta, 1/|k|, 1/|q - dk|, |q|^2, q.k, |k|^2
// the tile area is reused once the product is done:
constexpr uint32_t kOffT = 0;                                // T [64][68] fp32
constexpr uint32_t kOffWh = 0, kOffWl = 8192;                // before T: W_hi, W_lo staging, [64] rows of 128 B, 16-byte
                                                             // pieces XOR-swizzled with (row % 8) (conflict-free both ways)
// A is kept only where the inversion reads it, in compact blocks (strides chosen for conflict-free row-per-thread stores)
constexpr int LA = 36, LB = 20;                              // row strides (floats) of the 32x32 and the 16x16 blocks
constexpr int LD16 = 16 * LB + 4;                            // floats per diagonal block (+4: bank shift between blocks)
constexpr uint32_t kOffA21 = C * LM * 4;                     // A[32:64, 0:32]
constexpr uint32_t kOffB10 = kOffA21 + 32 * LA * 4;          // A[16:32, 0:16]
constexpr uint32_t kOffB32 = kOffB10 + 16 * LB * 4;          // A[48:64, 32:48]
constexpr uint32_t kOffAd = kOffB32 + 16 * LB * 4;           // the four diagonal blocks; dead after step 1:
constexpr uint32_t kOffP = kOffAd;                           // product scratch, 2 x [16][LB] in step 2, [32][LA] in step 3
__host__ __device__ constexpr Lay lay_of(bool qk) {
  const uint32_t half = 16384u; (void)qk;
  return Lay{half, 2 * half, 2 * half, 2 * half + kCvVecs * C * 4 + 1024};   // + slack for the 1024-byte alignment
}
static_assert(kOffAd + 4 * LD16 * 4 <= 32768 && 32 * LA * 4 <= 4 * LD16 * 4, "reuse of the tile area");

__device__ __forceinline__ float4 lds_f4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}
// Operands of the tf32 block products.  Their fragments are loaded as plain fp32 bits (a conversion per fragment
// element cost 320 warp instructions per chunk-head); what the products themselves produce and consume again - the
// inverted diagonal blocks, the intermediate products, the lower blocks of T - is rounded to tf32 (to nearest) once,
// where it is written to shared memory; only the blocks of A, written by the row pass, stay unrounded (the tensor
// core truncates them).  Measured where T is far from I (correlated keys), max error of o / RMS: everything
// truncated 1.9e-2, this 1.2e-2, a conversion per fragment element 1.2e-2; the A blocks rounded at their write as
// well was the slowest of all.
__device__ __forceinline__ uint32_t to_tf32(float x) { return __float_as_uint(x); }
__device__ __forceinline__ float rnd_tf32(float x) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
  return __uint_as_float(r);
}
__device__ __forceinline__ float2 rnd_tf32(float a, float b) { return make_float2(rnd_tf32(a), rnd_tf32(b)); }
__device__ __forceinline__ void mma_tf32(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Byte offset of the 16-byte chunk `c16` (0..15 over the 128 columns) of row `row` of the Q tile.
__device__ __forceinline__ uint32_t q_tile_chunk(uint32_t half_bytes, uint32_t row, uint32_t c16) {
  return kOffQ0 + (c16 >> 3) * half_bytes + row * 128 + (((c16 & 7) ^ (row & 7)) << 4);
}

// C[16 x 8*NT] (+)= A[16 x 8*KS] * B[8*KS x 8*NT], fp32 matrices in shared memory (row strides LDA, LDB), tf32 MMAs.
// a: &A[row0][k0], b: &B[k0][col0].  Fragment coordinates: g = lane / 4, t = lane % 4.
template <int KS, int NT, int LDA, int LDB>
__device__ __forceinline__ void block_mma_tf32(float (&acc)[NT][4], const float* a, const float* b, int g, int t) {
  static_assert((LDA * 4) % 16 == 0, "ldmatrix rows are 16-byte pieces");
  // The 16 x 8 fp32 A fragment of one k-step in ONE instruction: ldmatrix moves 8 x 8 tiles of 16-bit elements, i.e.
  // 8 rows of 16 bytes = 8 x 4 fp32, and hands thread (g, t) the 32 bits at row g, piece t - exactly the tf32
  // fragment layout.  Lane l supplies the row address of tile l / 8: rows 0..7 / 8..15 at columns 0..3, then 4..7.
  const int lane = g * 4 + t;
  const uint32_t a_lane = smem_u32(a + ((lane & 7) + 8 * ((lane >> 3) & 1)) * LDA + 4 * (lane >> 4));
#pragma unroll
  for (int ks = 0; ks < KS; ++ks) {
    uint32_t af[4];
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(af[0]), "=r"(af[1]), "=r"(af[2]), "=r"(af[3])
                 : "r"(a_lane + ks * 32));
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const uint32_t b0 = to_tf32(b[(ks * 8 + t) * LDB + nt * 8 + g]);
      const uint32_t b1 = to_tf32(b[(ks * 8 + t + 4) * LDB + nt * 8 + g]);
      mma_tf32(acc[nt], af, b0, b1);
    }
  }
}

// 16 consecutive columns of the thread's lane of tensor memory (zeros after a failed wait); warp-wide.
__device__ __forceinline__ void load16(uint32_t taddr, float (&x)[16], bool ok) {
  uint32_t u[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) u[j] = 0u;
  if (ok) {
    tmem_ld16(taddr, u);
    tmem_wait_ld();
  }
#pragma unroll
  for (int j = 0; j < 16; ++j) x[j] = __uint_as_float(u[j]);
}
// kWf32: W leaves as one fp32 matrix (what the kind::tf32 output product of chain_tf32.cu reads) instead of the bf16
// hi + lo pair; same bytes, same staging area.
template <bool kQk, bool kWf32>
__global__ void __launch_bounds__(kThreads, kCtasPerSm) intra_mma_kernel(ChunkGeom g, const __grid_constant__ CUtensorMap map_q,
                                                            const __grid_constant__ CUtensorMap map_k,
                                                            float* __restrict__ coef, GateArgs gates, GateParam gp,
                                                            QkNorm qkn, float scale,
                                                            __nv_bfloat16* __restrict__ Tout,
                                                            __nv_bfloat16* __restrict__ Wout, size_t w_lo_offset,
                                                            int32_t* __restrict__ status) {
  static_assert(!kQk || kWf32, "the q/k-norm variant uses the fp32 W staging slots");
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ __align__(8) uint64_t bars[2];   // tiles landed; product done
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  const int slot = blockIdx.x / g.H, h = blockIdx.x % g.H;
  grid_dependency_wait();   // chunk map and coefficients come from the previous kernels
  const SlotInfo si = slot_info(g, slot);
  if (si.seq < 0) return;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr Lay L = lay_of(kQk);
  constexpr uint32_t kOffK1 = L.k1, kOffQ1 = L.k1 + 8192, kOffCv = L.cv, kTmemCols = 64;
  const int fg = lane >> 2, ft = lane & 3;   // MMA fragment coordinates of the tf32 block products
  float* Tf = reinterpret_cast<float*>(smem + kOffT);
  float* cv = reinterpret_cast<float*>(smem + kOffCv);
  float* A21 = reinterpret_cast<float*>(smem + kOffA21);
  float* B10 = reinterpret_cast<float*>(smem + kOffB10);
  float* B32 = reinterpret_cast<float*>(smem + kOffB32);
  float* Ad = reinterpret_cast<float*>(smem + kOffAd);
  float* Pf = reinterpret_cast<float*>(smem + kOffP);
  const uint32_t bar_t = smem_u32(&bars[0]), bar_p = smem_u32(&bars[1]);
  const uint32_t s_base = smem_u32(smem);

  if (warp == 2) {   // the warp with no gate loads of its own: barriers, tile loads, tensor memory
    if (lane == 0) {
      abort_flag = 0;
      mbar_init(bar_t, 1);
      mbar_init(bar_p, 1);
      mbar_fence_init();
      mbar_arrive_expect_tx(bar_t, L.tiles);
      tma_load_2d(s_base + kOffK0, &map_k, h * kD, si.tok0, bar_t);
      tma_load_2d(s_base + kOffK1, &map_k, h * kD + 64, si.tok0, bar_t);
      tma_load_2d(s_base + kOffQ0, &map_q, h * kD, si.tok0, bar_t);
      tma_load_2d(s_base + kOffQ1, &map_q, h * kD + 64, si.tok0, bar_t);
    }
    __syncwarp();
    tmem_alloc(smem_u32(&tmem_slot), kTmemCols);
    tc_fence_before_sync();
  }
  float* cf = coef + ((size_t)slot * g.H + h) * MDN_NUM_COEF * C;
  if (gates.log_alpha == nullptr) {
    for (int idx = tid; idx < 4 * C; idx += kThreads) cv[idx] = cf[kAlpha * C + idx];
    if constexpr (kQk)
      for (int idx = tid; idx < 2 * C; idx += kThreads) {   // gamma_C eta, (mubar_C/mubar) eta; alpha b^-
        cv[4 * C + idx] = cf[kGS * C + idx];
        if (idx < C) cv[11 * C + idx] = cf[kAlphaBPrev * C + idx];
      }
    __syncthreads();   // coefficients in smem; barriers initialised and tensor memory allocated
  } else {
    // fused coefficient scan (Eq. 10): this head's gates (stride H floats), then one warp runs the scans,
    // keeps alpha, beta, mu, eta in smem for the Gamma rows and writes the chain kernel's six vectors
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
    __syncthreads();   // gates in smem; barriers initialised and tensor memory allocated
    if (warp == 0) {   // (the warp with the least to do afterwards: rows 0..31 of A) while the others build their rows of Gamma
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
      if constexpr (kQk) {   // the last-row weights get their 1/|k| factor once the norms are known
        reinterpret_cast<float2*>(cv + 4 * C)[lane] = make_float2(hc.gs[0], hc.gs[1]);
        reinterpret_cast<float2*>(cv + 5 * C)[lane] = make_float2(hc.gm[0], hc.gm[1]);
        reinterpret_cast<float2*>(cv + 11 * C)[lane] = make_float2(hc.ab_prev[0], hc.ab_prev[1]);
      } else {
        put(kRk, 1.f, 1.f);
        put(kRq, 1.f, 1.f);
      }
    }
  }
  tc_fence_after_sync();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);

  // ---- the product, issued by one thread as soon as the tiles have landed: eight k-steps of 16 over dk
  if (tid == 2 * 32) {
    if (mbar_wait(bar_t, 0, &abort_flag)) {
      tc_fence_after_sync();
      constexpr uint32_t idesc = idesc_bf16(128, 64, false, false, false);
      const uint64_t d0 = smem_desc_sw128(s_base + kOffK0, 16, 1024), d1 = smem_desc_sw128(s_base + kOffK1, 16, 1024);
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const uint64_t d = ((k >> 2) ? d1 : d0) + 2 * (k & 3);   // A: 128 rows from here (K, then Q); B: the first 64 (K)
        umma_ss(tmem, d, d, idesc, k > 0);
      }
      umma_commit(bar_p);
    }
  }


  // ---- the thread's row of Gamma, times eta (and scale or alpha_r), in registers: f[i] ~ gamma_{rp,i} eta_i for i <= rp, else 0, where
  // rp = r for a W row (mask i <= r) and r - 1 for an A row (Gamma shifted one row down, mask i < r).  Tokens past
  // the end of a short chunk (they hold another sequence's data) get empty rows.  Walking i from 63 down,
  //   G <- mu_{i+1} G + beta_i a,   a <- a alpha_i      (a = prod_{i<l<=rp} alpha_l; both idle while i > rp)
  const bool w_thread = tid >= C;          // warps 2, 3: one row of W each; warps 0, 1: one row of A each
  const int r = tid & (C - 1);
  const int rp = (r < si.n) ? (w_thread ? r : r - 1) : -1;
  float f[C];
  {
    float G = 0.f, a = 0.f, mu_next = 0.f;
    // the row's constant factor rides on the seed of a (G is linear in it): scale for a W row, alpha_r for an A row
    const float seed = w_thread ? scale : cv[0 * C + r];
    const uint32_t cv_s = s_base + kOffCv;
    auto walk = [&](auto from_tag, auto to_tag) {   // columns from + 3 down to `to`, in groups of four
      constexpr int kFrom = decltype(from_tag)::value, kTo = decltype(to_tag)::value;
      float4 al = lds_f4(cv_s + kFrom * 4), be = lds_f4(cv_s + (C + kFrom) * 4), mu = lds_f4(cv_s + (2 * C + kFrom) * 4),
             et = lds_f4(cv_s + (3 * C + kFrom) * 4);
#pragma unroll
      for (int i4 = kFrom; i4 >= kTo; i4 -= 4) {
        const float alv[4] = {al.x, al.y, al.z, al.w}, bev[4] = {be.x, be.y, be.z, be.w}, muv[4] = {mu.x, mu.y, mu.z, mu.w},
                    etv[4] = {et.x, et.y, et.z, et.w};
        if (i4 >= kTo + 4) {   // the next group's gate values, fetched ahead of the dependent chain
          al = lds_f4(cv_s + (i4 - 4) * 4); be = lds_f4(cv_s + (C + i4 - 4) * 4); mu = lds_f4(cv_s + (2 * C + i4 - 4) * 4);
          et = lds_f4(cv_s + (3 * C + i4 - 4) * 4);
        }
#pragma unroll
        for (int e = 3; e >= 0; --e) {
          const int i = i4 + e;
          a = (i == rp) ? seed : a;   // a (and with it G) stays 0 until the walk reaches the row's last column
          G = fmaf(mu_next, G, bev[e] * a);
          a *= alv[e];
          f[i] = G * etv[e];
          mu_next = muv[e];
        }
      }
    };
    if (warp & 1) {   // rows 32..63; the rows 0..31 of the other warps are empty right of column 31
      walk(std::integral_constant<int, C - 4>{}, std::integral_constant<int, C / 2>{});
    } else {
#pragma unroll
      for (int i = C / 2; i < C; ++i) f[i] = 0.f;
      mu_next = 0.f;
    }
    walk(std::integral_constant<int, C / 2 - 4>{}, std::integral_constant<int, 0>{});
  }

  bool ok = true;
  float rn_r = 1.f;                        // 1/|k_r| for an A row, 1/|q_r - d k_r| for a W row
  float dh = 0.f;
  if constexpr (kQk) {
    // fused q/k norm, while the products run: |k|^2, |q|^2 and q . k of every token from the tiles, two threads
    // per token (one per half of dk);  |q - d k|^2 = |q|^2 - 2 d q.k + d^2 |k|^2
    dh = qkn.d ? __ldg(qkn.d + h) : 0.f;
    ok = mbar_wait(bar_t, 0, &abort_flag);
    if (ok) {
      const int row = tid >> 1, hb = tid & 1;
      float nq2 = 0.f, qkd = 0.f, nk2 = 0.f;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint32_t off = q_tile_chunk(L.k1, row, hb * 8 + j);
        const uint4 uq = *reinterpret_cast<const uint4*>(smem + off);
        const uint4 uk = *reinterpret_cast<const uint4*>(smem + off - kOffQ0);
        const uint32_t q4[4] = {uq.x, uq.y, uq.z, uq.w}, k4[4] = {uk.x, uk.y, uk.z, uk.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float ql = __uint_as_float(q4[e] << 16), qh = __uint_as_float(q4[e] & 0xffff0000u);
          const float kl = __uint_as_float(k4[e] << 16), kh = __uint_as_float(k4[e] & 0xffff0000u);
          nq2 = fmaf(ql, ql, fmaf(qh, qh, nq2));
          qkd = fmaf(ql, kl, fmaf(qh, kh, qkd));
          nk2 = fmaf(kl, kl, fmaf(kh, kh, nk2));
        }
      }
      nq2 += __shfl_xor_sync(0xffffffffu, nq2, 1);
      qkd += __shfl_xor_sync(0xffffffffu, qkd, 1);
      nk2 += __shfl_xor_sync(0xffffffffu, nk2, 1);
      if (hb == 0) {
        cv[6 * C + row] = 1.f / sqrtf(nk2 + qkn.eps);
        cv[7 * C + row] = 1.f / sqrtf(fmaxf(nq2 - 2.f * dh * qkd + dh * dh * nk2, 0.f) + qkn.eps);
      }
    }
    __syncthreads();   // the norms of every token known; the coefficient scans are done
    rn_r = cv[(w_thread ? 7 : 6) * C + r];
    if (!w_thread) {
      cf[kGS * C + r] = cv[4 * C + r] * rn_r;
      cf[kGM * C + r] = cv[5 * C + r] * rn_r;
      cf[kAlphaBPrev * C + r] = cv[11 * C + r] * rn_r;
      cf[kRk * C + r] = rn_r;
    } else {
      cf[kRq * C + r] = rn_r;
    }
  }

  // ---- the product: lanes 0..63 of tensor memory hold the rows of K K^T, lanes 64..127 those of Q K^T; a thread
  // reads its row 16 columns at a time; the rows 0..31 of a warp never look past column 31
  ok = mbar_wait(bar_p, 0, &abort_flag) && ok;
  ok = __all_sync(0xffffffffu, ok);   // warp-uniform: the tensor-memory loads below are warp-wide
  tc_fence_after_sync();
  const uint32_t trow = tmem + (static_cast<uint32_t>(warp * 32) << 16);
  const int reach = (warp & 1) ? 4 : 2;    // 16-column groups the warp's rows can reach

  // ---- one row of A (into the compact blocks the inversion reads) or of W (into the bf16 staging) per thread
  const size_t mat = ((size_t)slot * g.H + h) * C * C;
  if (!w_thread) {
    const int rbk = r >> 4, rl = r & 15;
#pragma unroll
    for (int cb = 0; cb < 4; ++cb) {
      if (cb < reach) {
        float x[16];
        load16(trow + cb * 16, x, ok);
        if constexpr (kQk) {
          // fused q/k norm: the W thread of row r needs this row of K K^T as well ((q - d k) . k_i = Q K^T - d K K^T): it
          // goes through row r's slot of the W staging area (the tiles there are dead), which that thread reads below
          // and then overwrites with its row of W
#pragma unroll
          for (int p4 = 0; p4 < 4; ++p4)
            *reinterpret_cast<float4*>(smem + kOffWh + r * 256 + (((cb * 4 + p4) ^ (r & 7)) * 16)) =
                make_float4(x[p4 * 4], x[p4 * 4 + 1], x[p4 * 4 + 2], x[p4 * 4 + 3]);
        }
        if (cb <= rbk) {
          float* dst = (cb == rbk) ? Ad + rbk * LD16 + rl * LB
                                   : (rbk >= 2 && cb < 2) ? A21 + (r - 32) * LA + cb * 16 : (rbk == 1 ? B10 : B32) + rl * LB;
#pragma unroll
          for (int j4 = 0; j4 < 16; j4 += 4) {
            const int i = cb * 16 + j4;
            float4 av;
            if constexpr (kQk) {
              const float4 rki = *reinterpret_cast<const float4*>(cv + 6 * C + i);
              av = make_float4(rn_r * f[i] * rki.x * x[j4], rn_r * f[i + 1] * rki.y * x[j4 + 1], rn_r * f[i + 2] * rki.z * x[j4 + 2],
                               rn_r * f[i + 3] * rki.w * x[j4 + 3]);
            } else {
              const float2 p0 = __fmul2_rn(make_float2(f[i], f[i + 1]), make_float2(x[j4], x[j4 + 1]));
              const float2 p1 = __fmul2_rn(make_float2(f[i + 2], f[i + 3]), make_float2(x[j4 + 2], x[j4 + 3]));
              av = make_float4(p0.x, p0.y, p1.x, p1.y);
            }
            *reinterpret_cast<float4*>(dst + j4) = av;
          }
        }
      }
    }
  }
  if constexpr (kQk) __syncthreads();   // the rows of K K^T are in their slots
  if (w_thread) {
    uint8_t* w_hi = smem + kOffWh + r * 128;
    uint8_t* w_lo = smem + kOffWl + r * 128;
    uint8_t* w_f32 = smem + kOffWh + r * 256;   // fp32 staging: [64] rows of 256 B, 16-byte pieces XOR-swizzled with (row % 8)
#pragma unroll
    for (int cb = 0; cb < 4; ++cb) {
      uint4 hi4[2] = {make_uint4(0u, 0u, 0u, 0u), make_uint4(0u, 0u, 0u, 0u)};
      uint4 lo4[2] = {make_uint4(0u, 0u, 0u, 0u), make_uint4(0u, 0u, 0u, 0u)};
      float4 wf[4] = {make_float4(0.f, 0.f, 0.f, 0.f), make_float4(0.f, 0.f, 0.f, 0.f), make_float4(0.f, 0.f, 0.f, 0.f),
                      make_float4(0.f, 0.f, 0.f, 0.f)};
      if (cb < reach) {
        float x[16];
        if constexpr (kQk) {   // (q_r - d k_r) . k_i / |k_i|; this row of K K^T waits in the row's staging slot
          float y[16];
          load16(trow + cb * 16, x, ok);
#pragma unroll
          for (int p4 = 0; p4 < 4; ++p4) {
            const float4 y4 = *reinterpret_cast<const float4*>(w_f32 + (((cb * 4 + p4) ^ (r & 7)) * 16));
            y[p4 * 4] = y4.x; y[p4 * 4 + 1] = y4.y; y[p4 * 4 + 2] = y4.z; y[p4 * 4 + 3] = y4.w;
          }
#pragma unroll
          for (int j4 = 0; j4 < 16; j4 += 4) {
            const float4 rki = *reinterpret_cast<const float4*>(cv + 6 * C + cb * 16 + j4);
            x[j4] = (x[j4] - dh * y[j4]) * rki.x; x[j4 + 1] = (x[j4 + 1] - dh * y[j4 + 1]) * rki.y;
            x[j4 + 2] = (x[j4 + 2] - dh * y[j4 + 2]) * rki.z; x[j4 + 3] = (x[j4 + 3] - dh * y[j4 + 3]) * rki.w;
          }
        } else {
          load16(trow + cb * 16, x, ok);
        }
        float w[16];
        if constexpr (kQk) {
#pragma unroll
          for (int j = 0; j < 16; ++j) w[j] = rn_r * f[cb * 16 + j] * x[j];
        } else {
#pragma unroll
          for (int j = 0; j < 16; j += 2) {
            const float2 p = __fmul2_rn(make_float2(f[cb * 16 + j], f[cb * 16 + j + 1]), make_float2(x[j], x[j + 1]));
            w[j] = p.x; w[j + 1] = p.y;
          }
        }
        if constexpr (kWf32) {
#pragma unroll
          for (int p4 = 0; p4 < 4; ++p4) wf[p4] = make_float4(w[p4 * 4], w[p4 * 4 + 1], w[p4 * 4 + 2], w[p4 * 4 + 3]);
        } else {
#pragma unroll
          for (int hf = 0; hf < 2; ++hf) {
            split_pack_bf16(w[hf * 8 + 0], w[hf * 8 + 1], hi4[hf].x, lo4[hf].x);
            split_pack_bf16(w[hf * 8 + 2], w[hf * 8 + 3], hi4[hf].y, lo4[hf].y);
            split_pack_bf16(w[hf * 8 + 4], w[hf * 8 + 5], hi4[hf].z, lo4[hf].z);
            split_pack_bf16(w[hf * 8 + 6], w[hf * 8 + 7], hi4[hf].w, lo4[hf].w);
          }
        }
      }
      if constexpr (kWf32) {
#pragma unroll
        for (int p4 = 0; p4 < 4; ++p4) *reinterpret_cast<float4*>(w_f32 + (((cb * 4 + p4) ^ (r & 7)) * 16)) = wf[p4];
      } else {
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          const int sw = ((cb * 2 + hf) ^ (r & 7)) * 16;
          *reinterpret_cast<uint4*>(w_hi + sw) = hi4[hf];
          *reinterpret_cast<uint4*>(w_lo + sw) = lo4[hf];
        }
      }
    }
  }
  tc_fence_before_sync();
  __syncthreads();   // A and the W staging complete
  if (warp == 2) {   // every warp's tensor-memory loads completed before the barrier
    tc_fence_after_sync();
    tmem_dealloc(tmem, kTmemCols);
  }
  if constexpr (kWf32) {
    float* Wf = reinterpret_cast<float*>(Wout);   // [slot][H][64][64] fp32
    for (int idx = tid; idx < C * 16; idx += kThreads) {   // coalesced 16-byte stores
      const int rr = idx >> 4, c = idx & 15;
      *reinterpret_cast<uint4*>(Wf + mat + rr * C + c * 4) =
          *reinterpret_cast<const uint4*>(smem + kOffWh + rr * 256 + ((c ^ (rr & 7)) * 16));
    }
  } else {
    for (int idx = tid; idx < C * 8; idx += kThreads) {   // coalesced 16-byte stores of W_hi, W_lo
      const int rr = idx >> 3, c = idx & 7, sw = rr * 128 + ((c ^ (rr & 7)) * 16);
      *reinterpret_cast<uint4*>(Wout + mat + rr * C + c * 8) = *reinterpret_cast<const uint4*>(smem + kOffWh + sw);
      *reinterpret_cast<uint4*>(Wout + w_lo_offset + mat + rr * C + c * 8) = *reinterpret_cast<const uint4*>(smem + kOffWl + sw);
    }
  }
  __syncthreads();   // staging read out: T takes its place

  // step 1: D_b = (I + A_bb)^{-1} for the four 16x16 diagonal blocks; thread = (block, column), fp32
  if (tid < C) {
    const int b0 = (tid >> 4) * 16, j = tid & 15;
    float x[16];
#pragma unroll
    for (int rr = 0; rr < 16; ++rr) {
      float arow[16];
#pragma unroll
      for (int m4 = 0; m4 < 16; m4 += 4) {
        if (m4 < rr) {
          const float4 v4 = *reinterpret_cast<const float4*>(Ad + (tid >> 4) * LD16 + rr * LB + m4);
          arow[m4] = v4.x; arow[m4 + 1] = v4.y; arow[m4 + 2] = v4.z; arow[m4 + 3] = v4.w;
        }
      }
      float acc = (rr == j) ? 1.f : 0.f;
#pragma unroll
      for (int m = 0; m < rr; ++m) acc = fmaf(-arow[m], x[m], acc);
      x[rr] = acc;
    }
#pragma unroll
    for (int rr = 0; rr < 16; ++rr) Tf[(b0 + rr) * LM + b0 + j] = rnd_tf32(x[rr]);   // (an operand of steps 2, 3)
    if (((tid >> 4) & 1) == 0) {   // the zero block right of D_0 (D_2): step 3 reads T_11 and T_22 as full 32x32 blocks
#pragma unroll
      for (int rr = 0; rr < 16; ++rr) Tf[(b0 + rr) * LM + b0 + 16 + j] = 0.f;
    }
  }
  __syncthreads();

  // step 2: inside each 32x32 diagonal block s: T_lo = -D_hi (A_lo D_lo); 16x16 blocks, warp s does block s
  if (warp < 2) {
    const int R0 = 32 * warp + 16, C0 = 32 * warp;
    float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    block_mma_tf32<2, 2, LB, LM>(acc, warp == 0 ? B10 : B32, Tf + C0 * LM + C0, fg, ft);
    float* P = Pf + warp * 16 * LB;
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      *reinterpret_cast<float2*>(P + fg * LB + nt * 8 + 2 * ft) = rnd_tf32(acc[nt][0], acc[nt][1]);
      *reinterpret_cast<float2*>(P + (fg + 8) * LB + nt * 8 + 2 * ft) = rnd_tf32(acc[nt][2], acc[nt][3]);
    }
    __syncwarp();
    float acc2[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    block_mma_tf32<2, 2, LM, LB>(acc2, Tf + R0 * LM + R0, P, fg, ft);
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      *reinterpret_cast<float2*>(Tf + (R0 + fg) * LM + C0 + nt * 8 + 2 * ft) = rnd_tf32(-acc2[nt][0], -acc2[nt][1]);
      *reinterpret_cast<float2*>(Tf + (R0 + fg + 8) * LM + C0 + nt * 8 + 2 * ft) = rnd_tf32(-acc2[nt][2], -acc2[nt][3]);
    }
  }
  __syncthreads();
  // step 3: T[32:64, 0:32] = -T[32:64, 32:64] (A[32:64, 0:32] T[0:32, 0:32]); warp = (row tile, column half)
  {
    const int mt = warp & 1, n0 = (warp >> 1) * 16;
    float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    block_mma_tf32<4, 2, LA, LM>(acc, A21 + 16 * mt * LA, Tf + n0, fg, ft);
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      *reinterpret_cast<float2*>(Pf + (16 * mt + fg) * LA + n0 + nt * 8 + 2 * ft) = rnd_tf32(acc[nt][0], acc[nt][1]);
      *reinterpret_cast<float2*>(Pf + (16 * mt + fg + 8) * LA + n0 + nt * 8 + 2 * ft) = rnd_tf32(acc[nt][2], acc[nt][3]);
    }
    __syncthreads();
    float acc2[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    block_mma_tf32<4, 2, LM, LA>(acc2, Tf + (32 + 16 * mt) * LM + 32, Pf + n0, fg, ft);
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      *reinterpret_cast<float2*>(Tf + (32 + 16 * mt + fg) * LM + n0 + nt * 8 + 2 * ft) = make_float2(-acc2[nt][0], -acc2[nt][1]);
      *reinterpret_cast<float2*>(Tf + (32 + 16 * mt + fg + 8) * LM + n0 + nt * 8 + 2 * ft) = make_float2(-acc2[nt][2], -acc2[nt][3]);
    }
  }
  __syncthreads();

  for (int idx = tid; idx < C * 8; idx += kThreads) {   // T as bf16; the blocks above the diagonal are zero and were never written
    const int rr = idx >> 3, c0 = (idx & 7) * 8;
    uint4 packed = make_uint4(0u, 0u, 0u, 0u);
    if ((c0 >> 4) <= (rr >> 4)) {
      const float4 t0 = *reinterpret_cast<const float4*>(Tf + rr * LM + c0);
      const float4 t1 = *reinterpret_cast<const float4*>(Tf + rr * LM + c0 + 4);
      packed.x = pack_bf16(t0.x, t0.y); packed.y = pack_bf16(t0.z, t0.w);
      packed.z = pack_bf16(t1.x, t1.y); packed.w = pack_bf16(t1.z, t1.w);
    }
    *reinterpret_cast<uint4*>(Tout + mat + rr * C + c0) = packed;
  }
  if (!ok && tid == 0) atomicCAS(status, kDevOk, kDevTimeout);
  grid_launch_dependents();   // after the tensor memory has been released (see the head of this file)
}

}  // namespace

template <bool kQk, bool kWf32>
static cudaError_t launch_intra_variant(const Plan& pl, const CUtensorMap& mq, const CUtensorMap& mk, const GateArgs& gates,
                                        size_t n_mats) {
  constexpr uint32_t smem_bytes = lay_of(kQk).smem;
  cudaError_t e = cudaFuncSetAttribute(intra_mma_kernel<kQk, kWf32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
  if (e != cudaSuccess) return e;
  return launch_pdl(intra_mma_kernel<kQk, kWf32>, dim3((unsigned)n_mats), dim3(kThreads), smem_bytes, pl.stream, pl.geom, mq, mk,
                    reinterpret_cast<float*>(pl.ws + pl.lay.off_coef), gates, pl.gp, pl.qk, pl.p.scale,
                    reinterpret_cast<__nv_bfloat16*>(pl.ws + pl.lay.off_T),
                    reinterpret_cast<__nv_bfloat16*>(pl.ws + pl.lay.off_W), n_mats * C * C,
                    reinterpret_cast<int32_t*>(pl.ws + pl.lay.off_status));
}

cudaError_t launch_intra_mma(const Plan& pl, const void* q, const void* k, const GateArgs& gates, int* launches) {
  const size_t n_mats = (size_t)pl.geom.num_slots * pl.p.H;
  const uint64_t tokens = (uint64_t)pl.p.B * pl.p.T, row = (uint64_t)pl.p.H * kD;
  CUtensorMap mq, mk;
  if (!encode_tma_2d_bf16(&mq, TmaMap2D{q, row, tokens, row * 2, 64, 64, true}) ||
      !encode_tma_2d_bf16(&mk, TmaMap2D{k, row, tokens, row * 2, 64, 64, true}))
    return cudaErrorInvalidValue;
  // (the q/k-norm variant passes rows of K K^T through the fp32 W staging slots: it exists with the fp32 W only, which is
  // what every caller that can switch the q/k norm on uses)
  if (pl.qk.on && !pl.w_f32) return cudaErrorInvalidValue;
  cudaError_t e = pl.qk.on ? launch_intra_variant<true, true>(pl, mq, mk, gates, n_mats)
                           : (pl.w_f32 ? launch_intra_variant<false, true>(pl, mq, mk, gates, n_mats)
                                       : launch_intra_variant<false, false>(pl, mq, mk, gates, n_mats));
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e == cudaSuccess) ++*launches;
  return e;
}

}  // namespace mdn
