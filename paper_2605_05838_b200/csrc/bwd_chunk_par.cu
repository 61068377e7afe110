// Chunk-parallel backward, stage 2: per (chunk, head), from the kept forward states (S, M at the chunk's start) and
// the adjoint pair (dS', dM' at its end), the gradients of q, k, v and of the four gates.  Section 3.1-3.2: the chunk
// form in the notation of chain_tensor.cu,
//     X = K S,  Y = K M,  R = V - abar.X + p.Y,  V~ = T R,  T = (I + A)^-1,  A = G^- o (K K^T),  W = scale Geta o (Q K^T),
//     O = scale (abar.(Q S) - b.(Q M)) + W V~,   S' = abar_C S - b_C M + K^T (g_S.V~),   M' = mubar_C M - K^T (g_M.V~),
// differentiated matrix by matrix:
//     dV~ = W^T dO + g_S.(K dS') - g_M.(K dM'),   dR = T^T dV~ = dV,
//     dQ  = scale (abar.(dO S^T) - b.(dO M^T)) + DW K,                    DW = scale Geta o tril(dO V~^T),
//     dK  = -abar.(dR S^T) + p.(dR M^T) + g_S.(V~ dS'^T) - g_M.(V~ dM'^T) + DW^T Q + (DA + DA^T) K,
//                                                                         DA = G^- o dA,  dA = -tril(dR V~^T, -1),
// the adjoints of the coefficient vectors as row sums (e.g. d abar_r = -sum_j dR X + scale sum_j dO (Q S), where
// sum_j dR_rj X_rj = sum_d K_rd (dR S^T)_rd reuses a product that dK needs anyway), the adjoints of the two masks
// d Geta = scale tril(dO V~^T) o (Q K^T), d G^- = dA o (K K^T), and from those the gate gradients by running the
// coefficient recurrences of Eq. 10 in reverse.
// All products are tf32 tensor-core MMAs (fp32 accumulate) on operands in shared memory: q, k, dO and the states as
// the bf16 values they are, the intermediates (V~, dR, DW, DA, T, W) in fp32.  One 256-thread CTA per (chunk, head).
#include "mdn_common.cuh"
#include "tc_utils.cuh"

namespace mdn {
namespace {

using namespace tc;

constexpr int kD = 128;
constexpr int kThreads = 256;
constexpr int LT = kD + 8;    // bf16 elements per row of a 64 x 128 bf16 tile and of a state (row = value index)
constexpr int LF = kD + 4;    // floats per row of a 64 x 128 fp32 tile
constexpr int L64 = C + 4;    // floats per row of a 64 x 64 matrix

// shared memory map (bytes)
constexpr uint32_t kOffSt = 0;                                   // state, bf16 [128 (value j)][LT (key d)]; later d Geta, d G^-
constexpr uint32_t kOffK = kOffSt + kD * LT * 2;                 // k, q, dO tiles, bf16 [64][LT]
constexpr uint32_t kOffQ = kOffK + C * LT * 2;
constexpr uint32_t kOffDO = kOffQ + C * LT * 2;
constexpr uint32_t kOffVt = kOffDO + C * LT * 2;                 // V~, fp32 [64][LF]; later DW
constexpr uint32_t kOffDR = kOffVt + C * LF * 4;                 // dR, fp32 [64][LF]; later DA
constexpr uint32_t kOffT = kOffDR + C * LF * 4;                  // T, fp32 [64][L64]
constexpr uint32_t kOffTmp = kOffT + C * L64 * 4;                // R / dV~ (fp32 [64][LF]); later gamma and m ([64][L64] each)
constexpr uint32_t kOffVec = kOffTmp + 2 * C * L64 * 4;          // vectors, 24 x [64] floats
constexpr uint32_t kSmem = kOffVec + 24 * C * 4;
static_assert(2 * C * L64 * 4 >= C * LF * 4 && kD * LT * 2 >= 2 * C * L64 * 4, "overlays");
static_assert(kSmem <= 232448, "shared memory");

// vectors
enum Vec : int { vAbar = 0, vB, vP, vGS, vGM, vMubar, vAlpha, vBeta, vMu, vEta, vBprev,
                 vdAbar, vdB, vdP, vdGS, vdGM, vdMubar, vdAlpha, vdBeta, vdMu, vdEta, vRed };

struct ParArgs {
  ChunkGeom g;
  const __nv_bfloat16* q; const __nv_bfloat16* k; const __nv_bfloat16* v; const __nv_bfloat16* d_o;
  const float* beta; const float* log_alpha; const float* log_mu; const float* eta;
  const float* coef; const __nv_bfloat16* T; const __nv_bfloat16* W; size_t w_lo_offset;
  const uint8_t* fwd_states; const uint8_t* adj_states; const __nv_bfloat16* v_ext;
  float scale;
  float* dq; float* dk; float* dv; float* dbeta; float* dlog_alpha; float* dlog_mu; float* deta;
};

__device__ __forceinline__ uint32_t tf32_of(float x) {
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

// acc[mt][nt] (+)= A[m0 + 16 mt .., k] B[k, n0 + 8 nt ..] over k < K.  A(m, k), B(k, n) return floats from shared
// memory (any layout: a transposed operand is an accessor with its indices exchanged).  g = lane / 4, t = lane % 4.
template <int MT, int NT, class FA, class FB>
__device__ __forceinline__ void warp_mma(float (&acc)[MT][NT][4], FA A, FB B, int K, int m0, int n0, int g, int t) {
  for (int k0 = 0; k0 < K; k0 += 8) {
    uint32_t af[MT][4], bf[NT][2];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      const int m = m0 + 16 * mt + g;
      af[mt][0] = tf32_of(A(m, k0 + t)); af[mt][1] = tf32_of(A(m + 8, k0 + t));
      af[mt][2] = tf32_of(A(m, k0 + t + 4)); af[mt][3] = tf32_of(A(m + 8, k0 + t + 4));
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const int n = n0 + 8 * nt + g;
      bf[nt][0] = tf32_of(B(k0 + t, n)); bf[nt][1] = tf32_of(B(k0 + t + 4, n));
    }
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) mma_tf32(acc[mt][nt], af[mt], bf[nt][0], bf[nt][1]);
  }
}

template <int MT, int NT> __device__ __forceinline__ void zero(float (&acc)[MT][NT][4]) {
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[mt][nt][e] = 0.f;
}

// visit the elements of a warp's fragment block: f(mt, nt, e, row, col)
template <int MT, int NT, class F> __device__ __forceinline__ void for_frag(int m0, int n0, int g, int t, F f) {
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) f(mt, nt, e, m0 + 16 * mt + g + 8 * (e >> 1), n0 + 8 * nt + 2 * t + (e & 1));
}

__global__ void __launch_bounds__(kThreads, 1) bwd_chunk_par_kernel(ParArgs a) {
  extern __shared__ __align__(16) uint8_t smem[];
  __nv_bfloat16* sSt = reinterpret_cast<__nv_bfloat16*>(smem + kOffSt);
  __nv_bfloat16* sK = reinterpret_cast<__nv_bfloat16*>(smem + kOffK);
  __nv_bfloat16* sQ = reinterpret_cast<__nv_bfloat16*>(smem + kOffQ);
  __nv_bfloat16* sDO = reinterpret_cast<__nv_bfloat16*>(smem + kOffDO);
  float* sVt = reinterpret_cast<float*>(smem + kOffVt);
  float* sDR = reinterpret_cast<float*>(smem + kOffDR);
  float* sT = reinterpret_cast<float*>(smem + kOffT);
  float* sTmp = reinterpret_cast<float*>(smem + kOffTmp);
  float* sGam = sTmp;                       // gamma [64][L64] (after R / dV~ are done with the area)
  float* sMm = sTmp + C * L64;              // m [64][L64]
  float* sDW = sVt;                         // DW [64][L64] (after V~ is done)
  float* sDA = sDR;                         // DA
  float* sdGe = reinterpret_cast<float*>(smem + kOffSt);            // d Geta [64][L64] (after the states are done)
  float* sdGm = sdGe + C * L64;             // d G^-
  float* vec = reinterpret_cast<float*>(smem + kOffVec);
  auto V = [&](int which) { return vec + which * C; };

  const int slot = blockIdx.x / a.g.H, h = blockIdx.x % a.g.H, H = a.g.H;
  const SlotInfo si = slot_info(a.g, slot);
  if (si.seq < 0) return;
  const int n = si.n, nch = a.g.chunks_per_seq;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int m0 = 32 * (warp & 1), n0 = 32 * (warp >> 1), n064 = 16 * (warp >> 1);   // the warp's block of a 64x128 / 64x64 result
  const size_t mat = ((size_t)slot * H + h) * C * C;
  const uint8_t* imgS = a.fwd_states + ((size_t)slot * H + h) * 65536;
  const uint8_t* imgM = imgS + 32768;
  const int e_real = si.seq * 2 * nch + 2 * (nch - 1 - si.local);
  const uint8_t* imgdM = a.adj_states + ((size_t)e_real * H + h) * 65536;   // roles exchanged in the adjoint run
  const uint8_t* imgdS = imgdM + 32768;
  const float scale = a.scale;

  auto tok = [&](int r) { return (size_t)(si.tok0 + r) * H + h; };
  auto load_tile = [&](__nv_bfloat16* dst, const __nv_bfloat16* src) {
    for (int idx = tid; idx < C * 16; idx += kThreads) {
      const int r = idx >> 4, c8 = (idx & 15) * 8;
      uint4 x = make_uint4(0u, 0u, 0u, 0u);
      if (r < n) x = *reinterpret_cast<const uint4*>(src + tok(r) * kD + c8);
      *reinterpret_cast<uint4*>(dst + r * LT + c8) = x;
    }
  };
  // state image (value index j x key index d, two swizzled blocks) -> sSt[j][d]
  auto load_state = [&](const uint8_t* img) {
    for (int idx = tid; idx < 2 * kD * 8; idx += kThreads) {
      const int half = idx >> 10, j = (idx >> 3) & 127, pp = idx & 7, c = pp ^ (j & 7);
      *reinterpret_cast<uint4*>(sSt + j * LT + half * 64 + c * 8) =
          *reinterpret_cast<const uint4*>(img + half * 16384 + j * 128 + pp * 16);
    }
  };
  auto dot_images = [&](const uint8_t* x, const uint8_t* y) {   // sum of the element-wise product (same layout)
    float s = 0.f;
    for (int idx = tid; idx < 2048; idx += kThreads) {
      const uint4 ux = *reinterpret_cast<const uint4*>(x + idx * 16), uy = *reinterpret_cast<const uint4*>(y + idx * 16);
      const uint32_t xs[4] = {ux.x, ux.y, ux.z, ux.w}, ys[4] = {uy.x, uy.y, uy.z, uy.w};
#pragma unroll
      for (int e = 0; e < 4; ++e)
        s += __uint_as_float(xs[e] << 16) * __uint_as_float(ys[e] << 16) +
             __uint_as_float(xs[e] & 0xffff0000u) * __uint_as_float(ys[e] & 0xffff0000u);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    return s;   // per warp; lane 0 adds it where it belongs
  };
  auto bfv = [](const __nv_bfloat16* p, int i) { return __bfloat162float(p[i]); };
  auto AK = [&](int m, int k) { return bfv(sK, m * LT + k); };
  auto AQ = [&](int m, int k) { return bfv(sQ, m * LT + k); };
  auto ADO = [&](int m, int k) { return bfv(sDO, m * LT + k); };
  auto AVt = [&](int m, int k) { return sVt[m * LF + k]; };
  auto ADR = [&](int m, int k) { return sDR[m * LF + k]; };
  auto BSt_dk = [&](int k, int nn) { return bfv(sSt, nn * LT + k); };   // contraction over the key index: B(d, j) = S[d][j]
  auto BSt_dv = [&](int k, int nn) { return bfv(sSt, k * LT + nn); };   // contraction over the value index: B(j, d) = S[d][j]
  // row sums of G o X over the warp's 32 columns, added to a vector (X(r, c) from a tile)
  auto add_rowsum = [&](float (&G)[2][4][4], auto X, float* dst, float sign) {
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        const int r = m0 + 16 * mt + g + 8 * hf;
        float s = 0.f;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
          const int c = n0 + 8 * nt + 2 * t;
          s = fmaf(G[mt][nt][2 * hf], X(r, c), s);
          s = fmaf(G[mt][nt][2 * hf + 1], X(r, c + 1), s);
        }
        s += __shfl_xor_sync(0xffffffffu, s, 1);
        s += __shfl_xor_sync(0xffffffffu, s, 2);
        if (t == 0) atomicAdd(dst + r, sign * s);
      }
  };

  // ---- vectors: the chain's coefficient vectors, the gates, zeroed adjoints
  const float* cf = a.coef + ((size_t)slot * H + h) * MDN_NUM_COEF * C;
  for (int idx = tid; idx < 24 * C; idx += kThreads) vec[idx] = 0.f;
  __syncthreads();
  if (tid < C) {
    const int r = tid;
    const bool live = r < n;
    V(vAbar)[r] = cf[kAbar * C + r]; V(vB)[r] = cf[kB * C + r]; V(vP)[r] = cf[kAlphaBPrev * C + r];
    V(vGS)[r] = live ? cf[kGS * C + r] : 0.f; V(vGM)[r] = live ? cf[kGM * C + r] : 0.f; V(vMubar)[r] = cf[kMubar * C + r];
    const size_t gi = tok(r);
    V(vAlpha)[r] = live ? expf(a.log_alpha[gi]) : 1.f; V(vMu)[r] = live ? expf(a.log_mu[gi]) : 1.f;
    V(vBeta)[r] = live ? a.beta[gi] : 0.f; V(vEta)[r] = live ? (a.eta ? a.eta[gi] : 1.f) : 0.f;
  }
  load_tile(sK, a.k);
  load_tile(sQ, a.q);
  load_tile(sDO, a.d_o);
  for (int idx = tid; idx < C * C; idx += kThreads) sT[(idx >> 6) * L64 + (idx & 63)] = __bfloat162float(a.T[mat + idx]);
  load_state(imgS);
  __syncthreads();
  if (tid < C) V(vBprev)[tid] = tid > 0 ? V(vB)[tid - 1] : 0.f;

  float dQ[2][4][4], dK[2][4][4];
  zero(dQ); zero(dK);

  // ---- forward quantities again: X = K S, Y = K M, R = V - abar.X + p.Y, V~ = T R
  {
    float X[2][4][4], Y[2][4][4];
    zero(X); zero(Y);
    warp_mma(X, AK, BSt_dk, kD, m0, n0, g, t);
    __syncthreads();
    load_state(imgM);
    __syncthreads();
    warp_mma(Y, AK, BSt_dk, kD, m0, n0, g, t);
    for_frag<2, 4>(m0, n0, g, t, [&](int mt, int nt, int e, int r, int c) {
      const float v = r < n ? __bfloat162float(a.v[tok(r) * kD + c]) : 0.f;
      sTmp[r * LF + c] = v - V(vAbar)[r] * X[mt][nt][e] + V(vP)[r] * Y[mt][nt][e];
    });
    __syncthreads();
    float Vt[2][4][4];
    zero(Vt);
    warp_mma(Vt, [&](int m, int k) { return sT[m * L64 + k]; }, [&](int k, int nn) { return sTmp[k * LF + nn]; }, C, m0, n0, g, t);
    for_frag<2, 4>(m0, n0, g, t, [&](int mt, int nt, int e, int r, int c) { sVt[r * LF + c] = r < n ? Vt[mt][nt][e] : 0.f; });
  }
  __syncthreads();

  // ---- with dM' (the end-of-chunk adjoint of M): K dM', the g_M term of dK and its coefficient adjoint
  float KdM[2][4][4];
  zero(KdM);
  load_state(imgdM);
  {
    const float s = dot_images(imgdM, imgM);                         // d mubar_C = <dM', M>
    if (lane == 0) atomicAdd(V(vdMubar) + n - 1, s);
  }
  __syncthreads();
  warp_mma(KdM, AK, BSt_dk, kD, m0, n0, g, t);
  {
    float G[2][4][4];
    zero(G);
    warp_mma(G, AVt, BSt_dv, kD, m0, n0, g, t);                       // V~ dM'^T
    for_frag<2, 4>(m0, n0, g, t, [&](int mt, int nt, int e, int r, int c) { dK[mt][nt][e] -= V(vGM)[r] * G[mt][nt][e]; });
    add_rowsum(G, AK, V(vdGM), -1.f);
  }
  __syncthreads();
  // ---- with dS': K dS', the g_S term of dK, dV~ and dR
  load_state(imgdS);
  {
    const float s1 = dot_images(imgdS, imgS), s2 = dot_images(imgdS, imgM);   // d abar_C = <dS', S>, d b_C = -<dS', M>
    if (lane == 0) { atomicAdd(V(vdAbar) + n - 1, s1); atomicAdd(V(vdB) + n - 1, -s2); }
  }
  __syncthreads();
  // W (hi + lo, fp32) into the free area: W^T dO is formed here in fp32 (the adjoint chain's bf16 copy of it would
  // put one bf16 rounding of the dominant term into dV)
  for (int idx = tid; idx < C * C; idx += kThreads)
    sTmp[(idx >> 6) * L64 + (idx & 63)] = __bfloat162float(a.W[mat + idx]) + __bfloat162float(a.W[a.w_lo_offset + mat + idx]);
  __syncthreads();
  {
    float KdS[2][4][4], G[2][4][4], Vp[2][4][4];
    zero(KdS); zero(G); zero(Vp);
    warp_mma(Vp, [&](int m, int k) { return sTmp[k * L64 + m]; }, [&](int k, int nn) { return bfv(sDO, k * LT + nn); }, C, m0, n0, g, t);
    __syncthreads();   // W has been read: the area takes dV~
    warp_mma(KdS, AK, BSt_dk, kD, m0, n0, g, t);
    warp_mma(G, AVt, BSt_dv, kD, m0, n0, g, t);                       // V~ dS'^T
    for_frag<2, 4>(m0, n0, g, t, [&](int mt, int nt, int e, int r, int c) { dK[mt][nt][e] += V(vGS)[r] * G[mt][nt][e]; });
    add_rowsum(G, AK, V(vdGS), 1.f);
    for_frag<2, 4>(m0, n0, g, t, [&](int mt, int nt, int e, int r, int c) {
      sTmp[r * LF + c] = Vp[mt][nt][e] + V(vGS)[r] * KdS[mt][nt][e] - V(vGM)[r] * KdM[mt][nt][e];
    });
  }
  __syncthreads();
  {
    float dR[2][4][4];
    zero(dR);
    warp_mma(dR, [&](int m, int k) { return sT[k * L64 + m]; }, [&](int k, int nn) { return sTmp[k * LF + nn]; }, C, m0, n0, g, t);
    for_frag<2, 4>(m0, n0, g, t, [&](int mt, int nt, int e, int r, int c) {
      const float x = r < n ? dR[mt][nt][e] : 0.f;
      sDR[r * LF + c] = x;
      if (r < n) a.dv[tok(r) * kD + c] = x;
    });
  }
  __syncthreads();

  // ---- with S: dO S^T (dQ, d abar), dR S^T (dK, d abar)
  load_state(imgS);
  __syncthreads();
  {
    float G[2][4][4];
    zero(G);
    warp_mma(G, ADO, BSt_dv, kD, m0, n0, g, t);
    for_frag<2, 4>(m0, n0, g, t, [&](int mt, int nt, int e, int r, int c) { dQ[mt][nt][e] += scale * V(vAbar)[r] * G[mt][nt][e]; });
    add_rowsum(G, AQ, V(vdAbar), scale);
    zero(G);
    warp_mma(G, ADR, BSt_dv, kD, m0, n0, g, t);
    for_frag<2, 4>(m0, n0, g, t, [&](int mt, int nt, int e, int r, int c) { dK[mt][nt][e] -= V(vAbar)[r] * G[mt][nt][e]; });
    add_rowsum(G, AK, V(vdAbar), -1.f);
  }
  __syncthreads();
  // ---- with M: dO M^T (dQ, d b), dR M^T (dK, d p)
  load_state(imgM);
  __syncthreads();
  {
    float G[2][4][4];
    zero(G);
    warp_mma(G, ADO, BSt_dv, kD, m0, n0, g, t);
    for_frag<2, 4>(m0, n0, g, t, [&](int mt, int nt, int e, int r, int c) { dQ[mt][nt][e] -= scale * V(vB)[r] * G[mt][nt][e]; });
    add_rowsum(G, AQ, V(vdB), -scale);
    zero(G);
    warp_mma(G, ADR, BSt_dv, kD, m0, n0, g, t);
    for_frag<2, 4>(m0, n0, g, t, [&](int mt, int nt, int e, int r, int c) { dK[mt][nt][e] += V(vP)[r] * G[mt][nt][e]; });
    add_rowsum(G, AK, V(vdP), 1.f);
  }

  // ---- gamma and m by the column recurrences of Eq. 10 (thread = column), into the area R / dV~ used
  if (tid < C) {
    const int i = tid;
    float m = 1.f, gam = 0.f;
    for (int r = 0; r < C; ++r) {
      if (r > i) m *= V(vMu)[r];
      if (r >= i) gam = V(vAlpha)[r] * gam + V(vBeta)[r] * m;
      sGam[r * L64 + i] = r >= i ? gam : 0.f;
      sMm[r * L64 + i] = r >= i ? m : 0.f;
    }
  }
  // ---- the four 64 x 64 products
  float P1[2][2][4], P2[2][2][4], QK[2][2][4], KK[2][2][4];
  zero(P1); zero(P2); zero(QK); zero(KK);
  warp_mma(P1, ADO, [&](int k, int nn) { return sVt[nn * LF + k]; }, kD, m0, n064, g, t);   // dO V~^T
  warp_mma(P2, ADR, [&](int k, int nn) { return sVt[nn * LF + k]; }, kD, m0, n064, g, t);   // dR V~^T
  warp_mma(QK, AQ, [&](int k, int nn) { return bfv(sK, nn * LT + k); }, kD, m0, n064, g, t);
  warp_mma(KK, AK, [&](int k, int nn) { return bfv(sK, nn * LT + k); }, kD, m0, n064, g, t);
  __syncthreads();   // V~, dR and the state are no longer read; gamma, m complete
  for_frag<2, 2>(m0, n064, g, t, [&](int mt, int nt, int e, int r, int i) {
    const bool live = r < n;
    const float dOVt = (live && i <= r) ? P1[mt][nt][e] : 0.f;
    const float dA = (live && i < r) ? -P2[mt][nt][e] : 0.f;
    const float geta = sGam[r * L64 + i] * V(vEta)[i];
    const float gmin = (r > 0) ? V(vAlpha)[r] * sGam[(r - 1) * L64 + i] * V(vEta)[i] : 0.f;
    sDW[r * L64 + i] = scale * geta * dOVt;
    sDA[r * L64 + i] = gmin * dA;
    sdGe[r * L64 + i] = scale * dOVt * QK[mt][nt][e];
    sdGm[r * L64 + i] = dA * KK[mt][nt][e];
  });
  __syncthreads();
  // ---- dQ += DW K;  dK += DW^T Q + (DA + DA^T) K
  warp_mma(dQ, [&](int m, int k) { return sDW[m * L64 + k]; }, [&](int k, int nn) { return bfv(sK, k * LT + nn); }, C, m0, n0, g, t);
  warp_mma(dK, [&](int m, int k) { return sDW[k * L64 + m]; }, [&](int k, int nn) { return bfv(sQ, k * LT + nn); }, C, m0, n0, g, t);
  warp_mma(dK, [&](int m, int k) { return sDA[m * L64 + k] + sDA[k * L64 + m]; }, [&](int k, int nn) { return bfv(sK, k * LT + nn); }, C, m0, n0, g, t);
  for_frag<2, 4>(m0, n0, g, t, [&](int mt, int nt, int e, int r, int c) {
    if (r < n) {
      a.dq[tok(r) * kD + c] = dQ[mt][nt][e];
      a.dk[tok(r) * kD + c] = dK[mt][nt][e];
    }
  });

  // ---- gate gradients: the recurrences of Eq. 10 in reverse.  Thread i walks column i of gamma / m from the last
  // row up, carrying the adjoints of gamma_{r,i} and m_{r,i}; what belongs to a row goes to the row's accumulators.
  __syncthreads();   // d Geta, d G^- written; all row sums in
  if (tid < C) {
    const int i = tid;
    const float eta_i = V(vEta)[i];
    float dg = 0.f, dm = 0.f, deta_i = 0.f;
    for (int r = C - 1; r >= i; --r) {
      const float gam = sGam[r * L64 + i], mm = sMm[r * L64 + i];
      const float gam_up = r > i ? sGam[(r - 1) * L64 + i] : 0.f;
      const float al = V(vAlpha)[r], dge = sdGe[r * L64 + i], dgm = sdGm[r * L64 + i];
      // gamma_{r,i} feeds Geta_{r,i}, G^-_{r+1,i} (carried in dg from the row below) and, in the last row, g_S
      float dgam = dg + dge * eta_i;
      float dmm = dm;
      if (r == C - 1) {
        dgam += V(vdGS)[i] * eta_i;
        dmm += V(vdGM)[i] * eta_i;
        deta_i += V(vdGS)[i] * gam + V(vdGM)[i] * mm;
      }
      deta_i += dge * gam + dgm * al * gam_up;
      dmm += dgam * V(vBeta)[r];
      atomicAdd(V(vdAlpha) + r, dgam * gam_up + dgm * gam_up * eta_i);
      atomicAdd(V(vdBeta) + r, dgam * mm);
      if (r > i) atomicAdd(V(vdMu) + r, dmm * sMm[(r - 1) * L64 + i]);
      // to the row above: gamma_{r-1,i} through the recurrence and through G^-_{r,i} = alpha_r gamma_{r-1,i} eta_i
      dg = dgam * al + dgm * al * eta_i;
      dm = dmm * V(vMu)[r];
    }
    V(vdEta)[i] = deta_i;
  }
  __syncthreads();
  if (tid == 0) {   // the three vector recurrences (p_r = alpha_r b_{r-1}; b; the cumulative products), serial
    float* dAl = V(vdAlpha); float* dBe = V(vdBeta); float* dMu = V(vdMu);
    float* dAb = V(vdAbar); float* dB = V(vdB); float* dMb = V(vdMubar);
    for (int r = 0; r < C; ++r) {
      dAl[r] += V(vdP)[r] * V(vBprev)[r];
      if (r > 0) dB[r - 1] += V(vdP)[r] * V(vAlpha)[r];
    }
    for (int r = C - 1; r >= 0; --r) {
      dAl[r] += dB[r] * V(vBprev)[r];
      dBe[r] += dB[r] * V(vMubar)[r];
      dMb[r] += dB[r] * V(vBeta)[r];
      if (r > 0) dB[r - 1] += dB[r] * V(vAlpha)[r];
    }
    for (int r = C - 1; r >= 0; --r) {
      dAl[r] += dAb[r] * (r > 0 ? V(vAbar)[r - 1] : 1.f);
      dMu[r] += dMb[r] * (r > 0 ? V(vMubar)[r - 1] : 1.f);
      if (r > 0) {
        dAb[r - 1] += dAb[r] * V(vAlpha)[r];
        dMb[r - 1] += dMb[r] * V(vMu)[r];
      }
    }
  }
  __syncthreads();
  if (tid < n) {
    const size_t gi = tok(tid);
    a.dbeta[gi] = V(vdBeta)[tid];
    a.dlog_alpha[gi] = V(vAlpha)[tid] * V(vdAlpha)[tid];
    a.dlog_mu[gi] = V(vMu)[tid] * V(vdMu)[tid];
    if (a.deta) a.deta[gi] = V(vdEta)[tid];
  }
}

}  // namespace

cudaError_t launch_bwd_chunk_par(const Plan& fwd, const void* q, const void* k, const void* v, const void* d_o,
                                 const float* beta, const float* log_alpha, const float* log_mu, const float* eta,
                                 const void* fwd_states, const void* adj_states, const void* v_ext, float* dq, float* dk,
                                 float* dv, float* dbeta, float* dlog_alpha, float* dlog_mu, float* deta, int* launches) {
  ParArgs a;
  a.g = fwd.geom;
  a.q = static_cast<const __nv_bfloat16*>(q); a.k = static_cast<const __nv_bfloat16*>(k);
  a.v = static_cast<const __nv_bfloat16*>(v); a.d_o = static_cast<const __nv_bfloat16*>(d_o);
  a.beta = beta; a.log_alpha = log_alpha; a.log_mu = log_mu; a.eta = eta;
  a.coef = reinterpret_cast<const float*>(fwd.ws + fwd.lay.off_coef);
  a.T = reinterpret_cast<const __nv_bfloat16*>(fwd.ws + fwd.lay.off_T);
  a.W = reinterpret_cast<const __nv_bfloat16*>(fwd.ws + fwd.lay.off_W);
  a.w_lo_offset = (size_t)fwd.geom.num_slots * fwd.p.H * C * C;
  a.fwd_states = static_cast<const uint8_t*>(fwd_states);
  a.adj_states = static_cast<const uint8_t*>(adj_states);
  a.v_ext = static_cast<const __nv_bfloat16*>(v_ext);
  a.scale = fwd.p.scale;
  a.dq = dq; a.dk = dk; a.dv = dv; a.dbeta = dbeta; a.dlog_alpha = dlog_alpha; a.dlog_mu = dlog_mu; a.deta = deta;
  cudaError_t e = cudaFuncSetAttribute(bwd_chunk_par_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem);
  if (e != cudaSuccess) return e;
  bwd_chunk_par_kernel<<<dim3((unsigned)fwd.geom.num_slots * fwd.p.H), dim3(kThreads), kSmem, fwd.stream>>>(a);
  e = cudaGetLastError();
  if (e == cudaSuccess) ++*launches;
  return e;
}

}  // namespace mdn
