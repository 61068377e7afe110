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
// V~ and dR are not recomputed here: the two chain runs (the forward that keeps its states, the adjoint chain) have
// both in their epilogues and leave them in global memory as fp32, so X, Y, R, T R, K dS', K dM' and T^T dV~ cost nothing.
// Every product is a warp-level bf16 tensor-core MMA (m16n8k16, fp32 accumulate) fed by ldmatrix from shared memory:
// q, k, dO and the states are bf16 as they stand.  Of the operands that come out of an accumulator, V~ and DW are
// bf16 hi + lo pairs (16 mantissa bits through two MMAs); dR and DA enter as single bf16 values: measured, their lo
// parts change no gradient's error, while leaving out the lo part of V~ or DW does (dk 5e-2, dq 1.5x).
// One 256-thread CTA per (chunk, head).
#include "mdn_common.cuh"
#include "tc_utils.cuh"
#include "warp_mma.cuh"

namespace mdn {
namespace {

using namespace tc;
typedef __nv_bfloat16 bf16;

constexpr int kD = 128;
constexpr int kThreads = 256;
constexpr int LT = kD + 8;    // bf16 elements per row of a 64 x 128 tile and of a state (272 B: ldmatrix conflict-free)
constexpr int L6 = C + 8;     // bf16 elements per row of a 64 x 64 matrix (144 B)
constexpr int LG = C + 4;     // floats per row of a 64 x 64 fp32 matrix

// shared memory map (bytes)
constexpr uint32_t kTile = C * LT * 2, kMat6 = C * L6 * 2, kMatF = C * LG * 4;
constexpr uint32_t kOffSt = 0;                        // state, bf16 [128 (value j)][LT (key d)]; later d Geta, d G^- (fp32)
constexpr uint32_t kOffK = kOffSt + kD * LT * 2;      // k, q, dO
constexpr uint32_t kOffQ = kOffK + kTile;
constexpr uint32_t kOffDO = kOffQ + kTile;
constexpr uint32_t kOffVt = kOffDO + kTile;           // V~ hi, lo; later DW hi, lo
constexpr uint32_t kOffDR = kOffVt + 2 * kTile;       // dR; later DA
constexpr uint32_t kOffTmp = kOffDR + 2 * kTile;      // dS', then M again; later gamma, m (fp32 [64][LG] each)
constexpr uint32_t kOffVec = kOffTmp + 2 * kTile;     // vectors, 24 x [64] floats
constexpr uint32_t kOffGam = kOffVec + 24 * C * 4;    // gamma, fp32 [64][LG]: built while the first loads are in flight
constexpr uint32_t kSmem = kOffGam + kMatF;
constexpr uint32_t kR0 = kOffSt, kR1 = kOffVt, kR2 = kOffDR, kR3 = kOffTmp;   // the four reusable areas (see the kernel)
static_assert(kD * LT * 2 == 2 * kTile, "a state and a hi + lo tile pair have the same size");
static_assert(2 * kTile >= 2 * kMatF && kD * LT * 2 >= 2 * kMatF && 2 * kTile >= 2 * kMat6, "overlays");
static_assert(kSmem <= 232448, "shared memory");

constexpr int kIssuer = kThreads - 32;   // the thread that issues the bulk copies
constexpr int kBarSlot = 22;   // vector slot that holds the two mbarriers and the abort flag instead
enum Vec : int { vAbar = 0, vB, vP, vGS, vGM, vMubar, vAlpha, vBeta, vMu, vEta, vBprev,
                 vdAbar, vdB, vdP, vdGS, vdGM, vdMubar, vdAlpha, vdBeta, vdMu, vdEta, vRed };

struct ParArgs {
  ChunkGeom g;
  const bf16* q; const bf16* k; const bf16* d_o;
  const float* beta; const float* log_alpha; const float* log_mu; const float* eta;
  const float* coef;
  const uint8_t* fwd_states; const uint8_t* adj_states;   // state images per chunk slot
  const float* fwd_vt; const float* adj_dr;               // V~ and dR per chunk slot, fp32 [slot][64][H][dv]
  int32_t* status;                                        // the forward workspace's status word
  float scale;
  float* dq; float* dk; float* dv; float* dbeta; float* dlog_alpha; float* dlog_mu; float* deta;
};

__global__ void __launch_bounds__(kThreads, 1) bwd_chunk_par_kernel(ParArgs a) {
  extern __shared__ __align__(16) uint8_t smem[];
  const uint32_t sb = smem_u32(smem);
  bf16* sK = reinterpret_cast<bf16*>(smem + kOffK);
  bf16* sQ = reinterpret_cast<bf16*>(smem + kOffQ);
  float* sGam = reinterpret_cast<float*>(smem + kOffGam);     // gamma (own place), m
  float* sMm = reinterpret_cast<float*>(smem + kR2);
  bf16* sDWH = reinterpret_cast<bf16*>(smem + kR1);           // DW (hi, lo), DA
  bf16* sDWL = sDWH + C * L6;
  bf16* sDAH = reinterpret_cast<bf16*>(smem + kR3);
  float* sdGe = reinterpret_cast<float*>(smem + kR0);         // d Geta, d G^-
  float* sdGm = sdGe + C * LG;
  float* vec = reinterpret_cast<float*>(smem + kOffVec);
  auto V = [&](int which) { return vec + which * C; };

  const int slot = blockIdx.x / a.g.H, h = blockIdx.x % a.g.H, H = a.g.H;
  const SlotInfo si = slot_info(a.g, slot);
  if (si.seq < 0) return;
  const int n = si.n;
  int slot0, nch;
  seq_chunks(a.g, si.seq, &slot0, &nch);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int m0 = 32 * (warp & 1), n0 = 32 * (warp >> 1), n064 = 16 * (warp >> 1);   // the warp's block of a 64x128 / 64x64 result
  const uint8_t* imgS = a.fwd_states + ((size_t)slot * H + h) * 65536;
  const uint8_t* imgM = imgS + 32768;
  const int e_real = slot0 + (nch - 1 - si.local);   // this chunk in the adjoint chain's mirrored order
  const uint8_t* imgdM = a.adj_states + ((size_t)e_real * H + h) * 65536;   // roles exchanged in the adjoint run
  const uint8_t* imgdS = imgdM + 32768;
  const float scale = a.scale;

  // operands
  const Opnd oK{sb + kOffK, LT * 2, false}, oK_t{sb + kOffK, LT * 2, true};
  const Opnd oQ{sb + kOffQ, LT * 2, false}, oQ_t{sb + kOffQ, LT * 2, true};
  const Opnd oDO{sb + kOffDO, LT * 2, false};
  // a state in an area: B(k = key d, n = value j) = S[d][j], stored [j][d]; or B(k = value j, n = key d)
  auto st_dv = [&](uint32_t base) { return Opnd{sb + base, 0, true, true}; };
  // a 64 x 128 tile in an area, stored [row][column]: as A it is [m][k], as B it is [n][k]; tile_kn reads it as B [k][n]
  auto tile_mk = [&](uint32_t base) { return Opnd{sb + base, LT * 2, false}; };
  const Opnd oDWH{sb + kR1, L6 * 2, false}, oDWL{sb + kR1 + kMat6, L6 * 2, false};
  const Opnd oDWH_t{sb + kR1, L6 * 2, true}, oDWL_t{sb + kR1 + kMat6, L6 * 2, true};
  const Opnd oDAH{sb + kR3, L6 * 2, false}, oDAH_t{sb + kR3, L6 * 2, true};

  auto tok = [&](int r) { return (size_t)(si.tok0 + r) * H + h; };
  // everything arrives by cp.async (no registers in between, nothing blocks until the wait); rows past the chunk's
  // end are zero-filled (source size 0)
  auto cp16 = [&](uint32_t dst, const void* src, bool live) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(live ? 16 : 0));
  };
  auto load_tile = [&](uint32_t base, const bf16* src) {
    for (int idx = tid; idx < C * 16; idx += kThreads) {
      const int r = idx >> 4, c8 = (idx & 15) * 8;
      cp16(sb + base + (r * LT + c8) * 2, src + tok(r < n ? r : 0) * kD + c8, r < n);
    }
  };
  // a chunk's V~ or dR (fp32 rows of one head, H * dv floats apart) -> [64][128] fp32 at the start of an area
  auto load_f32 = [&](uint32_t base, const float* src) {
    for (int idx = tid; idx < C * 32; idx += kThreads) {
      const int r = idx >> 5, c4 = (idx & 31) * 4;
      cp16(sb + base + idx * 16, src + (size_t)(r < n ? r : 0) * H * kD + c4, r < n);
    }
  };
  // ... and from there, in place, to the bf16 hi + lo tiles the products read (every thread holds its 32 values across
  // the barrier; with_lo = false: the hi tile only); `out`, if given, receives the fp32 values of the live rows (dv = dR)
  auto split_in_place = [&](uint32_t base, float* out, bool with_lo) {
    float4 x[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) x[i] = *reinterpret_cast<const float4*>(smem + base + (tid + kThreads * i) * 16);
    __syncthreads();
    bf16* hi = reinterpret_cast<bf16*>(smem + base);
    bf16* lo = hi + C * LT;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int idx = tid + kThreads * i, r = idx >> 5, c4 = (idx & 31) * 4;
      uint2 ph, pl;
      split_pack_bf16(x[i].x, x[i].y, ph.x, pl.x);
      split_pack_bf16(x[i].z, x[i].w, ph.y, pl.y);
      *reinterpret_cast<uint2*>(hi + r * LT + c4) = ph;
      if (with_lo) *reinterpret_cast<uint2*>(lo + r * LT + c4) = pl;
      if (out != nullptr && r < n) *reinterpret_cast<float4*>(out + tok(r) * kD + c4) = x[i];
    }
  };
  // a state image (value index j x key index d, two swizzled blocks) goes into an area as it is, by two bulk copies
  // from one thread; the products address it through the swizzle (Opnd::swz)
  auto load_state = [&](const uint8_t* img, uint32_t base, uint32_t bar) {
    bulk_load(sb + base, img, 16384, bar);
    bulk_load(sb + base + 16384, img + 16384, 16384, bar);
  };
  auto cp_async_commit = []() { asm volatile("cp.async.commit_group;" ::: "memory"); };
  auto cp_async_wait = []() { asm volatile("cp.async.wait_group 0;" ::: "memory"); };
  // the three inner products of state images that the end-of-chunk adjoints need, in one pass over the four areas
  // (32768-byte images): <dM', M>, <dS', S>, <dS', M>, summed per warp
  auto state_dots = [&](float& dmm, float& dss, float& dsm) {
    float s0 = 0.f, s1 = 0.f, s2 = 0.f;
#pragma unroll 2
    for (int idx = tid - C; idx < kD * 16; idx += kThreads - C) {   // threads C.. (the first two warps are elsewhere)
      const uint32_t off = idx * 16;   // the four images have the same layout: any common order will do
      const uint4 uS = *reinterpret_cast<const uint4*>(smem + kR0 + off), uM = *reinterpret_cast<const uint4*>(smem + kR1 + off);
      const uint4 udS = *reinterpret_cast<const uint4*>(smem + kR2 + off), udM = *reinterpret_cast<const uint4*>(smem + kR3 + off);
      const uint32_t xS[4] = {uS.x, uS.y, uS.z, uS.w}, xM[4] = {uM.x, uM.y, uM.z, uM.w};
      const uint32_t xdS[4] = {udS.x, udS.y, udS.z, udS.w}, xdM[4] = {udM.x, udM.y, udM.z, udM.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float S0 = __uint_as_float(xS[e] << 16), S1 = __uint_as_float(xS[e] & 0xffff0000u);
        const float M0 = __uint_as_float(xM[e] << 16), M1 = __uint_as_float(xM[e] & 0xffff0000u);
        const float dS0 = __uint_as_float(xdS[e] << 16), dS1 = __uint_as_float(xdS[e] & 0xffff0000u);
        const float dM0 = __uint_as_float(xdM[e] << 16), dM1 = __uint_as_float(xdM[e] & 0xffff0000u);
        s0 = fmaf(dM0, M0, fmaf(dM1, M1, s0));
        s1 = fmaf(dS0, S0, fmaf(dS1, S1, s1));
        s2 = fmaf(dS0, M0, fmaf(dS1, M1, s2));
      }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      s0 += __shfl_xor_sync(0xffffffffu, s0, off);
      s1 += __shfl_xor_sync(0xffffffffu, s1, off);
      s2 += __shfl_xor_sync(0xffffffffu, s2, off);
    }
    dmm = s0; dss = s1; dsm = s2;   // per warp; lane 0 adds them where they belong
  };
  // row sums of G o X over the warp's 32 columns, added to a vector (X: a bf16 tile, k or q)
  auto add_rowsum = [&](float (&G)[2][4][4], const bf16* X, float* dst, float sign) {
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        const int r = m0 + 16 * mt + g + 8 * hf;
        float s = 0.f;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
          const uint32_t x2 = *reinterpret_cast<const uint32_t*>(X + r * LT + n0 + 8 * nt + 2 * t);
          s = fmaf(G[mt][nt][2 * hf], __uint_as_float(x2 << 16), s);
          s = fmaf(G[mt][nt][2 * hf + 1], __uint_as_float(x2 & 0xffff0000u), s);
        }
        s += __shfl_xor_sync(0xffffffffu, s, 1);
        s += __shfl_xor_sync(0xffffffffu, s, 2);
        if (t == 0) atomicAdd(dst + r, sign * s);
      }
  };

  const float* vt_rows = a.fwd_vt + (((size_t)slot * C) * H + h) * kD;
  const float* dr_rows = a.adj_dr + (((size_t)e_real * C) * H + h) * kD;
  // ---- what this CTA fetches later (V~, dR), towards L2 now (one CTA per SM: nothing else hides the latency)
  {
    const int r = tid >> 2, part = (tid & 3) * 32;
    if (r < n) {
      asm volatile("prefetch.global.L2 [%0];" ::"l"(vt_rows + (size_t)r * H * kD + part));
      asm volatile("prefetch.global.L2 [%0];" ::"l"(dr_rows + (size_t)r * H * kD + part));
    }
  }
  // Four areas of 34816 bytes (a state, or the hi + lo pair of a 64 x 128 tile) are reused through the phases:
  //   R0: S                                               | later d Geta, d G^-
  //   R1: M    | V~ (fp32, then hi, lo)                   | later DW (hi, lo), then two contribution matrices
  //   R2: dS'  | M again                                  | m
  //   R3: dM'  | dR (fp32, then bf16)                     | DA, then a contribution matrix
  // All four states arrive at the start by cp.async (no registers in between); M is fetched a second time later.
  const uint32_t bar0 = smem_u32(vec + kBarSlot * C), bar1 = bar0 + 8;   // mbarriers: the four states; M again
  volatile int* abort_flag = reinterpret_cast<volatile int*>(vec + kBarSlot * C + 4);
  if (tid == kIssuer) {   // a thread of the last warp: the first two warps have the vectors and gamma to set up
    *abort_flag = 0;
    mbar_init(bar0, 1);
    mbar_init(bar1, 1);
    mbar_fence_init();
    mbar_arrive_expect_tx(bar0, 4 * 32768);
    load_state(imgS, kR0, bar0);
    load_state(imgM, kR1, bar0);
    load_state(imgdS, kR2, bar0);
    load_state(imgdM, kR3, bar0);
  }
  load_tile(kOffK, a.k);
  load_tile(kOffQ, a.q);
  load_tile(kOffDO, a.d_o);
  cp_async_commit();
  // ---- vectors: the chain's coefficient vectors, the gates, zeroed adjoints
  const float* cf = a.coef + ((size_t)slot * H + h) * MDN_NUM_COEF * C;
  for (int idx = tid; idx < kBarSlot * C; idx += kThreads) vec[idx] = 0.f;
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
  cp_async_wait();
  {   // the states: a bounded wait; if it runs out the CTA reports it and leaves (all threads together)
    const bool ok = mbar_wait(bar0, 0, abort_flag);
    if (!__syncthreads_and(ok)) {
      if (tid == 0) atomicCAS(a.status, kDevOk, kDevTimeout);
      return;
    }
  }
  if (tid < C) {
    // two warps: gamma by the column recurrence of Eq. 10 (thread = column) ...
    V(vBprev)[tid] = tid > 0 ? V(vB)[tid - 1] : 0.f;
    const int i = tid;
    float m = 1.f, gam = 0.f;
    for (int rb = 0; rb < C; rb += 4) {
      const float4 al = *reinterpret_cast<const float4*>(V(vAlpha) + rb), be = *reinterpret_cast<const float4*>(V(vBeta) + rb);
      const float4 mu = *reinterpret_cast<const float4*>(V(vMu) + rb);
      const float a4[4] = {al.x, al.y, al.z, al.w}, b4[4] = {be.x, be.y, be.z, be.w}, m4[4] = {mu.x, mu.y, mu.z, mu.w};
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int rr = rb + u;
        if (rr > i) m *= m4[u];
        if (rr >= i) gam = fmaf(a4[u], gam, b4[u] * m);
        sGam[rr * LG + i] = rr >= i ? gam : 0.f;
      }
    }
  } else {
    // ... six warps: the end-of-chunk adjoints d mubar_C = <dM', M>, d abar_C = <dS', S>, d b_C = -<dS', M>
    float s0, s1, s2;
    state_dots(s0, s1, s2);
    if (lane == 0) {
      atomicAdd(V(vdMubar) + n - 1, s0);
      atomicAdd(V(vdAbar) + n - 1, s1);
      atomicAdd(V(vdB) + n - 1, -s2);
    }
  }

  float dQ[2][4][4], dK[2][4][4];
  zero(dQ); zero(dK);

  // ---- phase 1: dO S^T, dO M^T (dQ, d abar, d b)
  {
    float Y[2][4][4];
    zero(Y);
    warp_mma(Y, oDO, st_dv(kR0), kD, m0, n0, lane);                   // dO S^T
    for_frag<2, 4>(m0, n0, g, t, [&](int mt, int nt, int e, int r, int c) { dQ[mt][nt][e] += scale * V(vAbar)[r] * Y[mt][nt][e]; });
    add_rowsum(Y, sQ, V(vdAbar), scale);
    zero(Y);
    warp_mma(Y, oDO, st_dv(kR1), kD, m0, n0, lane);                   // dO M^T
    for_frag<2, 4>(m0, n0, g, t, [&](int mt, int nt, int e, int r, int c) { dQ[mt][nt][e] -= scale * V(vB)[r] * Y[mt][nt][e]; });
    add_rowsum(Y, sQ, V(vdB), -scale);
  }
  __syncthreads();   // M has been read: V~ takes its place
  load_f32(kR1, vt_rows);
  cp_async_commit();
  float QK[2][2][4], KK[2][2][4];   // Q K^T, K K^T while V~ arrives
  zero(QK); zero(KK);
  warp_mma(QK, oQ, oK, kD, m0, n064, lane);
  warp_mma(KK, oK, oK, kD, m0, n064, lane);
  cp_async_wait();
  __syncthreads();
  split_in_place(kR1, nullptr, true);
  __syncthreads();

  // ---- phase 2: the g_M and g_S terms of dK from V~ dM'^T, V~ dS'^T; dR arrives under the second
  {
    float G[2][4][4];
    zero(G);
    warp_mma(G, tile_mk(kR1), st_dv(kR3), kD, m0, n0, lane);          // V~ dM'^T
    warp_mma(G, tile_mk(kR1 + kTile), st_dv(kR3), kD, m0, n0, lane);
    for_frag<2, 4>(m0, n0, g, t, [&](int mt, int nt, int e, int r, int c) { dK[mt][nt][e] -= V(vGM)[r] * G[mt][nt][e]; });
    add_rowsum(G, sK, V(vdGM), -1.f);
    __syncthreads();   // dM' has been read: dR takes its place
    load_f32(kR3, dr_rows);
    cp_async_commit();
    zero(G);
    warp_mma(G, tile_mk(kR1), st_dv(kR2), kD, m0, n0, lane);          // V~ dS'^T
    warp_mma(G, tile_mk(kR1 + kTile), st_dv(kR2), kD, m0, n0, lane);
    for_frag<2, 4>(m0, n0, g, t, [&](int mt, int nt, int e, int r, int c) { dK[mt][nt][e] += V(vGS)[r] * G[mt][nt][e]; });
    add_rowsum(G, sK, V(vdGS), 1.f);
  }
  __syncthreads();   // dS' has been read: M takes its place
  if (tid == kIssuer) {
    fence_proxy_async_smem();
    mbar_arrive_expect_tx(bar1, 32768);
    load_state(imgM, kR2, bar1);
  }
  cp_async_wait();   // dR is in (M may still be on its way)
  __syncthreads();
  split_in_place(kR3, a.dv, false);   // no product reads dR's lo part
  __syncthreads();

  // ---- phase 3: dR S^T (dK, d abar) while M arrives again, then dR M^T (dK, d p)
  {
    float G[2][4][4];
    zero(G);
    // dR enters these two products as its hi part alone: S and M are single bf16 values themselves, and the lo part
    // changes no gradient's error (measured; V~ in the two products above does need its lo part)
    warp_mma(G, tile_mk(kR3), st_dv(kR0), kD, m0, n0, lane);
    for_frag<2, 4>(m0, n0, g, t, [&](int mt, int nt, int e, int r, int c) { dK[mt][nt][e] -= V(vAbar)[r] * G[mt][nt][e]; });
    add_rowsum(G, sK, V(vdAbar), -1.f);
    {
      const bool ok = mbar_wait(bar1, 0, abort_flag);
      if (!__syncthreads_and(ok)) {
        if (tid == 0) atomicCAS(a.status, kDevOk, kDevTimeout);
        return;
      }
    }
    zero(G);
    warp_mma(G, tile_mk(kR3), st_dv(kR2), kD, m0, n0, lane);
    for_frag<2, 4>(m0, n0, g, t, [&](int mt, int nt, int e, int r, int c) { dK[mt][nt][e] += V(vP)[r] * G[mt][nt][e]; });
    add_rowsum(G, sK, V(vdP), 1.f);
  }
  __syncthreads();   // M has been read: its area takes m

  // ---- m by its column recurrence (thread = column): m_{r,i} = mu_{i+1} .. mu_r
  if (tid < C) {
    const int i = tid;
    float m = 1.f;
    for (int rb = 0; rb < C; rb += 4) {
      const float4 mu = *reinterpret_cast<const float4*>(V(vMu) + rb);
      const float m4[4] = {mu.x, mu.y, mu.z, mu.w};
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int rr = rb + u;
        if (rr > i) m *= m4[u];
        sMm[rr * LG + i] = rr >= i ? m : 0.f;
      }
    }
  }
  // ---- the four 64 x 64 products
  float P1[2][2][4], P2[2][2][4];
  zero(P1); zero(P2);
  warp_mma(P1, oDO, tile_mk(kR1), kD, m0, n064, lane);                        // dO V~^T  (V~ as B: [n][k])
  warp_mma(P1, oDO, tile_mk(kR1 + kTile), kD, m0, n064, lane);
  warp_mma(P2, tile_mk(kR3), tile_mk(kR1), kD, m0, n064, lane);               // dR V~^T
  warp_mma(P2, tile_mk(kR3), tile_mk(kR1 + kTile), kD, m0, n064, lane);
  __syncthreads();   // V~, dR and S are no longer read; gamma, m complete
  for_pair<2, 2>(m0, n064, g, t, [&](int mt, int nt, int hf, int r, int i0) {
    float dw[2], da[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int i = i0 + e;
      const bool live = r < n;
      const float dOVt = (live && i <= r) ? P1[mt][nt][2 * hf + e] : 0.f;
      const float dA = (live && i < r) ? -P2[mt][nt][2 * hf + e] : 0.f;
      const float geta = sGam[r * LG + i] * V(vEta)[i];
      const float gmin = (r > 0) ? V(vAlpha)[r] * sGam[(r - 1) * LG + i] * V(vEta)[i] : 0.f;
      dw[e] = scale * geta * dOVt;
      da[e] = gmin * dA;
      sdGe[r * LG + i] = scale * dOVt * QK[mt][nt][2 * hf + e];
      sdGm[r * LG + i] = dA * KK[mt][nt][2 * hf + e];
    }
    uint32_t ph, pl;
    split_pack_bf16(dw[0], dw[1], ph, pl);
    *reinterpret_cast<uint32_t*>(sDWH + r * L6 + i0) = ph;
    *reinterpret_cast<uint32_t*>(sDWL + r * L6 + i0) = pl;
    *reinterpret_cast<uint32_t*>(sDAH + r * L6 + i0) = pack_bf16(da[0], da[1]);
  });
  __syncthreads();
  // ---- dQ += DW K;  dK += DW^T Q + (DA + DA^T) K
  warp_mma(dQ, oDWH, oK_t, C, m0, n0, lane);
  warp_mma(dQ, oDWL, oK_t, C, m0, n0, lane);
  warp_mma(dK, oDWH_t, oQ_t, C, m0, n0, lane);
  warp_mma(dK, oDWL_t, oQ_t, C, m0, n0, lane);
  warp_mma(dK, oDAH, oK_t, C, m0, n0, lane);
  warp_mma(dK, oDAH_t, oK_t, C, m0, n0, lane);
  for_pair<2, 4>(m0, n0, g, t, [&](int mt, int nt, int hf, int r, int c) {
    if (r < n) {
      *reinterpret_cast<float2*>(a.dq + tok(r) * kD + c) = make_float2(dQ[mt][nt][2 * hf], dQ[mt][nt][2 * hf + 1]);
      *reinterpret_cast<float2*>(a.dk + tok(r) * kD + c) = make_float2(dK[mt][nt][2 * hf], dK[mt][nt][2 * hf + 1]);
    }
  });

  // ---- gate gradients: the recurrences of Eq. 10 in reverse, column i of gamma / m from the last row up, carrying
  // the adjoints of gamma_{r,i} and m_{r,i}.
  __syncthreads();   // d Geta, d G^- written; all row sums in; DW, DA have been read
  // In two passes.  Serial (thread i = column i, from the last row up): only the two carried adjoints
  //     d gamma_{r,i} = dg + dGeta_{r,i} eta_i,      dg <- alpha_r (d gamma_{r,i} + dG^-_{r,i} eta_i)
  //     d m_{r,i}     = dm + d gamma_{r,i} beta_r,   dm <- mu_r d m_{r,i}
  // (g_S, g_M enter in the last row), written to two matrices in the area DW used.  Everything that is a sum over a
  // row (d alpha_r, d beta_r, d mu_r) or over a column (d eta_i) of products with these follows on all threads:
  // shared-memory atomics from the serial walk would serialise 64-way, and the walk itself is one instruction stream.
  float* sDg = reinterpret_cast<float*>(smem + kR1);
  float* sDm = sDg + C * LG;
  float* sPart = reinterpret_cast<float*>(smem + kR3);   // [3][64] partial column sums
  static_assert(2 * kMatF <= 2 * kTile, "adjoint matrices");
  if (tid < C) {
    const int i = tid;
    const float eta_i = V(vEta)[i];
    float dg = V(vdGS)[i] * eta_i, dm = V(vdGM)[i] * eta_i;   // what g_S, g_M give to the last row
    for (int rb = C - 4; rb >= 0; rb -= 4) {   // four rows' loads first: the walk itself is a chain of three FMAs per row
      float dge[4], dgm[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) { dge[u] = sdGe[(rb + u) * LG + i]; dgm[u] = sdGm[(rb + u) * LG + i]; }   // zero above the diagonal
      const float4 al4 = *reinterpret_cast<const float4*>(V(vAlpha) + rb), be4 = *reinterpret_cast<const float4*>(V(vBeta) + rb);
      const float4 mu4 = *reinterpret_cast<const float4*>(V(vMu) + rb);
      const float al[4] = {al4.x, al4.y, al4.z, al4.w}, be[4] = {be4.x, be4.y, be4.z, be4.w}, mu[4] = {mu4.x, mu4.y, mu4.z, mu4.w};
#pragma unroll
      for (int u = 3; u >= 0; --u) {
        const float dgam = fmaf(dge[u], eta_i, dg);
        const float dmm = fmaf(dgam, be[u], dm);
        sDg[(rb + u) * LG + i] = dgam;
        sDm[(rb + u) * LG + i] = dmm;
        dg = al[u] * fmaf(dgm[u], eta_i, dgam);
        dm = dmm * mu[u];
      }
    }
  } else {
    // meanwhile on the other six warps, column sums that do not need the walk: d eta_i = sum_r dGeta gamma_{r,i} +
    // dG^- alpha_r gamma_{r-1,i}, and the last row's g_S, g_M terms (three threads per column, a third of the rows each)
    const int i = (tid - C) & 63, part = (tid - C) >> 6, r0 = 22 * part, r1 = min(C, r0 + 22);
    float s = 0.f;
#pragma unroll 4
    for (int r = max(r0, i); r < r1; ++r) {
      s = fmaf(sdGe[r * LG + i], sGam[r * LG + i], s);
      if (r > i) s = fmaf(sdGm[r * LG + i] * V(vAlpha)[r], sGam[(r - 1) * LG + i], s);
    }
    if (part == 2) s += V(vdGS)[i] * sGam[(C - 1) * LG + i] + V(vdGM)[i] * sMm[(C - 1) * LG + i];
    sPart[part * C + i] = s;
  }
  __syncthreads();
  {   // row sums, four threads per row: d alpha_r += sum_i gamma_{r-1,i} (d gamma + dG^- eta_i), d beta_r += sum_i
      // d gamma m_{r,i}, d mu_r += sum_i d m m_{r-1,i}   (columns i <= r; the terms with gamma_{r-1,i}, m_{r-1,i}: i < r)
    const int r = tid >> 2, part = tid & 3;
    float sa = 0.f, sbe = 0.f, sm = 0.f;
#pragma unroll 4
    for (int i = part; i < C; i += 4) {   // columns interleaved over the row's four threads: conflict-free
      if (i <= r) {
        const float dgam = sDg[r * LG + i], dmm = sDm[r * LG + i];
        sbe = fmaf(dgam, sMm[r * LG + i], sbe);
        if (i < r) {
          sa = fmaf(sGam[(r - 1) * LG + i], fmaf(sdGm[r * LG + i], V(vEta)[i], dgam), sa);
          sm = fmaf(dmm, sMm[(r - 1) * LG + i], sm);
        }
      }
    }
    sa += __shfl_xor_sync(0xffffffffu, sa, 1); sa += __shfl_xor_sync(0xffffffffu, sa, 2);
    sbe += __shfl_xor_sync(0xffffffffu, sbe, 1); sbe += __shfl_xor_sync(0xffffffffu, sbe, 2);
    sm += __shfl_xor_sync(0xffffffffu, sm, 1); sm += __shfl_xor_sync(0xffffffffu, sm, 2);
    if (part == 0) { V(vdAlpha)[r] += sa; V(vdBeta)[r] += sbe; V(vdMu)[r] += sm; }
  }
  __syncthreads();
  // The three vector recurrences (p_r = alpha_r b_{r-1};  b_r = alpha_r b_{r-1} + beta_r mubar_r;  the cumulative
  // products) in reverse, on one warp with two rows per lane and everything in registers.  Each reverse chain
  // x_{r-1} = d_{r-1} + c_r x_r is a suffix scan of affine maps: the lane's two rows compose to x_{2l} = B + A x_{2l+2},
  // five shuffle steps compose the lanes.
  if (warp == 0) {
    const int e0 = 2 * lane, e1 = e0 + 1;
    auto rev_scan = [&](float& d0, float& d1, float c1, float c2) {   // c1 = c_{e1}, c2 = c_{e1+1} (0 past the end)
      float A = c1 * c2, B = fmaf(c1, d1, d0);
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const float A2 = __shfl_down_sync(0xffffffffu, A, o), B2 = __shfl_down_sync(0xffffffffu, B, o);
        if (lane + o < 32) { B = fmaf(A, B2, B); A *= A2; }
      }
      float xn = __shfl_down_sync(0xffffffffu, B, 1);
      if (lane == 31) xn = 0.f;
      d1 = fmaf(c2, xn, d1);
      d0 = B;
    };
    const float2 al = *reinterpret_cast<const float2*>(V(vAlpha) + e0), mu = *reinterpret_cast<const float2*>(V(vMu) + e0);
    const float al2 = lane < 31 ? V(vAlpha)[e0 + 2] : 0.f, mu2 = lane < 31 ? V(vMu)[e0 + 2] : 0.f;
    const float2 be = *reinterpret_cast<const float2*>(V(vBeta) + e0), bp = *reinterpret_cast<const float2*>(V(vBprev) + e0);
    const float2 mb = *reinterpret_cast<const float2*>(V(vMubar) + e0), dP = *reinterpret_cast<const float2*>(V(vdP) + e0);
    const float dP2 = lane < 31 ? V(vdP)[e0 + 2] : 0.f;
    float2 dAl = *reinterpret_cast<const float2*>(V(vdAlpha) + e0), dBe = *reinterpret_cast<const float2*>(V(vdBeta) + e0);
    float2 dMu = *reinterpret_cast<const float2*>(V(vdMu) + e0), dAb = *reinterpret_cast<const float2*>(V(vdAbar) + e0);
    float2 dB = *reinterpret_cast<const float2*>(V(vdB) + e0), dMb = *reinterpret_cast<const float2*>(V(vdMubar) + e0);
    const float ab_prev0 = lane > 0 ? V(vAbar)[e0 - 1] : 1.f, mb_prev0 = lane > 0 ? V(vMubar)[e0 - 1] : 1.f;
    const float ab0 = V(vAbar)[e0];
    // p_r = alpha_r b_{r-1}
    dAl.x = fmaf(dP.x, bp.x, dAl.x); dAl.y = fmaf(dP.y, bp.y, dAl.y);
    dB.x = fmaf(dP.y, al.y, dB.x); dB.y = fmaf(dP2, al2, dB.y);
    rev_scan(dB.x, dB.y, al.y, al2);                      // b_r = alpha_r b_{r-1} + beta_r mubar_r
    dAl.x = fmaf(dB.x, bp.x, dAl.x); dAl.y = fmaf(dB.y, bp.y, dAl.y);
    dBe.x = fmaf(dB.x, mb.x, dBe.x); dBe.y = fmaf(dB.y, mb.y, dBe.y);
    dMb.x = fmaf(dB.x, be.x, dMb.x); dMb.y = fmaf(dB.y, be.y, dMb.y);
    rev_scan(dAb.x, dAb.y, al.y, al2);                    // abar_r = alpha_r abar_{r-1},  mubar_r = mu_r mubar_{r-1}
    rev_scan(dMb.x, dMb.y, mu.y, mu2);
    dAl.x = fmaf(dAb.x, ab_prev0, dAl.x); dAl.y = fmaf(dAb.y, ab0, dAl.y);
    dMu.x = fmaf(dMb.x, mb_prev0, dMu.x); dMu.y = fmaf(dMb.y, mb.x, dMu.y);
    const float de0 = sPart[e0] + sPart[C + e0] + sPart[2 * C + e0], de1 = sPart[e1] + sPart[C + e1] + sPart[2 * C + e1];
    if (e0 < n) {
      const size_t gi = tok(e0);
      a.dbeta[gi] = dBe.x; a.dlog_alpha[gi] = al.x * dAl.x; a.dlog_mu[gi] = mu.x * dMu.x;
      if (a.deta) a.deta[gi] = de0;
    }
    if (e1 < n) {
      const size_t gi = tok(e1);
      a.dbeta[gi] = dBe.y; a.dlog_alpha[gi] = al.y * dAl.y; a.dlog_mu[gi] = mu.y * dMu.y;
      if (a.deta) a.deta[gi] = de1;
    }
  }
}

}  // namespace

cudaError_t launch_bwd_chunk_par(const Plan& fwd, const void* q, const void* k, const void* d_o, const float* beta,
                                 const float* log_alpha, const float* log_mu, const float* eta, const void* fwd_states,
                                 const float* fwd_vt, const void* adj_states, const float* adj_dr, float* dq, float* dk,
                                 float* dv, float* dbeta, float* dlog_alpha, float* dlog_mu, float* deta, int* launches) {
  ParArgs a;
  a.g = fwd.geom;
  a.q = static_cast<const __nv_bfloat16*>(q); a.k = static_cast<const __nv_bfloat16*>(k);
  a.d_o = static_cast<const __nv_bfloat16*>(d_o);
  a.beta = beta; a.log_alpha = log_alpha; a.log_mu = log_mu; a.eta = eta;
  a.coef = reinterpret_cast<const float*>(fwd.ws + fwd.lay.off_coef);
  a.fwd_states = static_cast<const uint8_t*>(fwd_states);
  a.adj_states = static_cast<const uint8_t*>(adj_states);
  a.fwd_vt = fwd_vt; a.adj_dr = adj_dr;
  a.status = reinterpret_cast<int32_t*>(fwd.ws + fwd.lay.off_status);
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
