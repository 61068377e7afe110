// a3 + a4 on the 5th-generation tensor cores (tcgen05, sm_100a): one CTA walks the chunks of
// one (sequence, head) in order.  bf16 q/k/v, dk = dv = 128, chunk 64.
//
// Everything is kept TRANSPOSED so that the value dimension (128) is the MMA M dimension and
// fills all 128 tensor-memory lanes; the 64 tokens of a chunk are the N (or K) dimension:
//
//   MMA-1a  X = S_b K^T, Y = M_b K^T              [dv x C]   A = bf16 copy of S^T / M^T in smem (K-major),
//   MMA-1b  Z = S_b Q^T, U = M_b Q^T                          B = the TMA-loaded K / Q tile as it is
//   EPI-1   R^T = V^T - abar .* X + (alpha b^-) .* Y          (per-token scalars act on COLUMNS here)
//   MMA-2   Y = R^T T^T                           [dv x C]   A = R^T from tensor memory (bf16 hi + lo),
//                                                             B = T, row-major = K-major
//   EPI-2   V~_S = (gamma_C eta) .* V~ , V~_M = ((mubar_C/mubar) eta) .* V~ , V~ ; each as bf16 hi + lo
//   MMA-3   S^T += V~_S^T K ,  M^T -= V~_M^T K    [dv x dk]  fp32 masters live in tensor memory, already
//                                                             scaled by (abar_C, b_C, mubar_C); B = the same
//                                                             K tile read MN-major; "-=" via the A-negate bit
//   MMA-3'  U = V~^T W^T                          [dv x C]   intra-chunk output, W = hi + lo
//   EPI-o   o^T = scale (abar .* Z - b .* U_old) + U          written straight from registers (rows < n)
//   P(c+1)  read S^T, M^T (fp32) once: write their bf16 copies to smem for the next MMA-1 and store them
//           back scaled by the next chunk's (abar_C, b_C, mubar_C); after the last chunk: final states.
//
// The bf16 hi + lo splits keep R, V~ and W at ~16 mantissa bits through the tensor cores (their
// rounding to plain bf16 would dominate the error budget); raw q/k tiles are never rescaled before
// an MMA - every row/column scaling is applied to fp32 accumulators.
//
// Warp roles: 0-3 critical-path epilogue (P, EPI-1, EPI-2); 4-7 output epilogue (EPI-o);
// 8 TMA producer (2-stage ring: K, Q, V, T, W_hi, W_lo, 6 coefficient vectors per chunk);
// 9 MMA issuer (one elected lane) and tensor-memory owner.  All hand-offs are mbarriers with
// bounded waits; tensor-memory column reuse is ordered by those same barriers.
#include <cstdlib>
#include <cstring>

#include "mdn_common.cuh"
#include "tc_utils.cuh"

namespace mdn {
namespace {

using namespace tc;

constexpr int kD = 128;
constexpr int kThreads = 320;
constexpr int kWarpTma = 8, kWarpMma = 9;

// shared memory (offsets from a 1024-byte aligned base)
constexpr uint32_t kOffSb = 0, kOffMb = 32768, kOffStage = 65536;
constexpr uint32_t kStK = 0, kStQ = 16384, kStV = 32768, kStT = 49152, kStWh = 57344, kStWl = 65536, kStCoef = 73728;
constexpr uint32_t kCoefBytes = kChainCoefs * C * sizeof(float);
constexpr uint32_t kStageBytes = 75776;
constexpr uint32_t kTxBytes = 3 * 16384 + 3 * 8192 + kCoefBytes;
constexpr uint32_t kSmemBytes = kOffStage + 2 * kStageBytes + 1024;
static_assert(kStCoef + kCoefBytes <= kStageBytes, "stage layout");

// tensor memory columns (512 x 128 lanes x 32 bit)
constexpr uint32_t kColS = 0, kColM = 128, kColX = 256, kColY = 320, kColZ = 384, kColU = 448;

struct Bars {
  uint64_t full[2], empty[2];
  uint64_t sb;   // P(c) done: S_b, M_b in smem, scaled masters in tensor memory     (128 arrivals)
  uint64_t m1;   // MMA-1a done                                                      (commit)
  uint64_t mq;   // MMA-1b done                                                      (commit)
  uint64_t r;    // EPI-1 done: R^T hi/lo in X                                        (128)
  uint64_t m2;   // MMA-2 done                                                       (commit)
  uint64_t zq;   // output epilogue has read Z, U (Q S, Q M)                          (128)
  uint64_t v;    // EPI-2 done: V~_S, V~_M, V~ operands in X, Y, Z                    (128)
  uint64_t m3;   // MMA-3 done                                                       (commit)
  uint64_t mo;   // MMA-3' done                                                      (commit)
  uint64_t zu;   // output epilogue has read U (intra-chunk output)                   (128)
};

struct ChainArgs {
  ChunkGeom g;
  const float* coef;
  const float* S0;
  const float* M0;
  void* o;
  float* Sf;
  float* Mf;
  int32_t* status;
  float scale;
  uint32_t w_lo_row_offset;   // rows between the hi and lo parts in the W tensor map
  uint32_t drop_lo;           // debug: bit 0 R, 1 V~_S/V~_M, 2 V~ (output), 3 W: leave that operand's lo part out
  long long* timeline;        // debug: CTA 0 writes clock64() at [chunk*32 + event] (NULL = off)
};

// Timeline events (debug).
enum Ev : int { kEvMmaStart = 0, kEvM1Seen, kEvRArrive, kEvM2Seen, kEvVArrive, kEvM3Seen, kEvSbArrive, kEvMqSeen,
                kEvZqArrive, kEvMoSeen, kEvZuArrive, kEvMmaIssued, kEvRSeen, kEvVSeen, kEvTmaIssued, kEvFullSeen, kEvStoresDone };

__device__ __forceinline__ void split_bf16(float x, float& hi, float& lo) {
  hi = bf16_round(x);
  lo = x - hi;
}

template <typename TO> __device__ __forceinline__ void store_o(TO* p, float x);
template <> __device__ __forceinline__ void store_o<float>(float* p, float x) { *p = x; }
template <> __device__ __forceinline__ void store_o<__nv_bfloat16>(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

template <typename TO>
__global__ void __launch_bounds__(kThreads, 1) chain_tensor_kernel(const ChainArgs a,
                                                                  const __grid_constant__ CUtensorMap map_q,
                                                                  const __grid_constant__ CUtensorMap map_k,
                                                                  const __grid_constant__ CUtensorMap map_v,
                                                                  const __grid_constant__ CUtensorMap map_t,
                                                                  const __grid_constant__ CUtensorMap map_w) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ __align__(8) Bars bars;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int H = a.g.H;
  const int seq = blockIdx.x / H, h = blockIdx.x % H;
  const SeqInfo sq = seq_info(a.g, seq);
  const int nch = sq.nchunks;
  const size_t st_off = ((size_t)seq * H + h) * kD * kD;

  const uint32_t s_base = smem_u32(smem);
  const uint32_t b_full0 = smem_u32(&bars.full[0]), b_full1 = smem_u32(&bars.full[1]);
  const uint32_t b_empty0 = smem_u32(&bars.empty[0]), b_empty1 = smem_u32(&bars.empty[1]);
  const uint32_t b_sb = smem_u32(&bars.sb), b_m1 = smem_u32(&bars.m1), b_mq = smem_u32(&bars.mq);
  const uint32_t b_r = smem_u32(&bars.r), b_m2 = smem_u32(&bars.m2), b_zq = smem_u32(&bars.zq);
  const uint32_t b_v = smem_u32(&bars.v), b_m3 = smem_u32(&bars.m3), b_mo = smem_u32(&bars.mo);
  const uint32_t b_zu = smem_u32(&bars.zu);

  if (tid == 0) {
    abort_flag = 0;
    mbar_init(b_full0, 1); mbar_init(b_full1, 1);
    mbar_init(b_empty0, 256); mbar_init(b_empty1, 256);
    mbar_init(b_sb, 128); mbar_init(b_r, 128); mbar_init(b_zq, 128); mbar_init(b_v, 128); mbar_init(b_zu, 128);
    mbar_init(b_m1, 1); mbar_init(b_mq, 1); mbar_init(b_m2, 1); mbar_init(b_m3, 1); mbar_init(b_mo, 1);
    mbar_fence_init();
  }
  if (warp == kWarpMma) tmem_alloc(smem_u32(&tmem_slot), 512);
  if (warp == kWarpTma && lane == 0) {
    prefetch_tensormap(&map_q); prefetch_tensormap(&map_k); prefetch_tensormap(&map_v);
    prefetch_tensormap(&map_t); prefetch_tensormap(&map_w);
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = tmem_slot;
  bool ok = true;
  volatile int* abortp = &abort_flag;
#define MDN_WAIT(bar, par)                         \
  if (!mbar_wait((bar), (par), abortp)) {          \
    ok = false;                                    \
    break;                                         \
  }

  long long* const tline = (blockIdx.x == 0) ? a.timeline : nullptr;
#define MDN_MARK(c, ev)                                                      \
  if (tline != nullptr && lane == 0 && (warp & 3) == ((warp < 8) ? 0 : (warp & 3))) tline[(c) * 32 + (ev)] = clock64();

  if (warp == kWarpTma) {
    // ================================================================== TMA producer
    if (lane == 0) {
      int issued = 0;
      for (int c = 0; c < nch; ++c) {
        const int s = c & 1;
        MDN_WAIT(s ? b_empty1 : b_empty0, ((c >> 1) & 1) ^ 1);
        const uint32_t fb = s ? b_full1 : b_full0;
        const uint32_t st = s_base + kOffStage + s * kStageBytes;
        const int tok0 = sq.tok0 + c * C;
        const int mat = (sq.slot0 + c) * H + h;
        mbar_arrive_expect_tx(fb, kTxBytes);
        tma_load_2d(st + kStK, &map_k, h * kD, tok0, fb);
        tma_load_2d(st + kStK + 8192, &map_k, h * kD + 64, tok0, fb);
        bulk_load(st + kStCoef, a.coef + (size_t)mat * MDN_NUM_COEF * C, kCoefBytes, fb);
        tma_load_2d(st + kStV, &map_v, h * kD, tok0, fb);
        tma_load_2d(st + kStT, &map_t, 0, mat * C, fb);
        tma_load_2d(st + kStQ, &map_q, h * kD, tok0, fb);
        tma_load_2d(st + kStQ + 8192, &map_q, h * kD + 64, tok0, fb);
        tma_load_2d(st + kStWh, &map_w, 0, mat * C, fb);
        tma_load_2d(st + kStWl, &map_w, 0, mat * C + (int)a.w_lo_row_offset, fb);
        MDN_MARK(c, kEvTmaIssued);
        issued = c + 1;
      }
      if (!ok) {   // giving up: let the copies already in flight land before the CTA exits
        for (int c = max(0, issued - 2); c < issued; ++c)
          for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait((c & 1) ? b_full1 : b_full0, (c >> 1) & 1); ++it) {}
      }
    }
  } else if (warp == kWarpMma) {
    // ================================================================== MMA issuer
    if (lane == 0) {
      const uint32_t id64 = idesc_bf16(128, 64, false, false, false);
      const uint32_t id128_mn = idesc_bf16(128, 128, false, true, false);
      const uint32_t id128_mn_neg = idesc_bf16(128, 128, false, true, true);
      const uint32_t sSb = s_base + kOffSb, sMb = s_base + kOffMb;
      for (int c = 0; c < nch; ++c) {
        const int s = c & 1;
        const uint32_t ph = c & 1;
        const uint32_t st = s_base + kOffStage + s * kStageBytes;
        const uint32_t sK = st + kStK, sQ = st + kStQ, sT = st + kStT, sWh = st + kStWh, sWl = st + kStWl;
        MDN_WAIT(s ? b_full1 : b_full0, (c >> 1) & 1);
        MDN_WAIT(b_sb, ph);
        tc_fence_after_sync();
        MDN_MARK(c, kEvMmaStart);
        // ---- MMA-1a: X = S_b K^T, Y = M_b K^T
#pragma unroll
        for (int k = 0; k < 8; ++k)
          umma_ss(tmem + kColX, smem_desc_sw128(sSb + (k >> 2) * 16384 + (k & 3) * 32, 16, 1024),
                  smem_desc_sw128(sK + (k >> 2) * 8192 + (k & 3) * 32, 16, 1024), id64, k > 0);
#pragma unroll
        for (int k = 0; k < 8; ++k)
          umma_ss(tmem + kColY, smem_desc_sw128(sMb + (k >> 2) * 16384 + (k & 3) * 32, 16, 1024),
                  smem_desc_sw128(sK + (k >> 2) * 8192 + (k & 3) * 32, 16, 1024), id64, k > 0);
        umma_commit(b_m1);
        // ---- MMA-1b: Z = S_b Q^T, U = M_b Q^T (Z, U must have been drained by the output epilogue)
        MDN_WAIT(b_zu, ph ^ 1);
        tc_fence_after_sync();
#pragma unroll
        for (int k = 0; k < 8; ++k)
          umma_ss(tmem + kColZ, smem_desc_sw128(sSb + (k >> 2) * 16384 + (k & 3) * 32, 16, 1024),
                  smem_desc_sw128(sQ + (k >> 2) * 8192 + (k & 3) * 32, 16, 1024), id64, k > 0);
#pragma unroll
        for (int k = 0; k < 8; ++k)
          umma_ss(tmem + kColU, smem_desc_sw128(sMb + (k >> 2) * 16384 + (k & 3) * 32, 16, 1024),
                  smem_desc_sw128(sQ + (k >> 2) * 8192 + (k & 3) * 32, 16, 1024), id64, k > 0);
        umma_commit(b_mq);
        // ---- MMA-2: Y = (R_hi + R_lo)^T T^T
        MDN_WAIT(b_r, ph);
        tc_fence_after_sync();
        MDN_MARK(c, kEvRSeen);
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_ts(tmem + kColY, tmem + kColX + k * 8, smem_desc_sw128(sT + k * 32, 16, 1024), id64, k > 0);
        if (!(a.drop_lo & 1u)) {
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma_ts(tmem + kColY, tmem + kColX + 32 + k * 8, smem_desc_sw128(sT + k * 32, 16, 1024), id64, true);
        }
        umma_commit(b_m2);
        // ---- MMA-3: S^T += V~_S^T K, M^T -= V~_M^T K   (K tile read MN-major: N = dk, K = tokens)
        MDN_WAIT(b_v, ph);
        tc_fence_after_sync();
        MDN_MARK(c, kEvVSeen);
        const int n3 = (a.drop_lo & 2u) ? 4 : 8;
        for (int k = 0; k < n3; ++k)
          umma_ts(tmem + kColS, tmem + kColX + (k >> 2) * 32 + (k & 3) * 8,
                  smem_desc_sw128(sK + (k & 3) * 2048, 8192, 1024), id128_mn, true);
        for (int k = 0; k < n3; ++k)
          umma_ts(tmem + kColM, tmem + kColY + (k >> 2) * 32 + (k & 3) * 8,
                  smem_desc_sw128(sK + (k & 3) * 2048, 8192, 1024), id128_mn_neg, true);
        umma_commit(b_m3);
        // ---- MMA-3': U = V~^T W^T  with  V~ = hi + lo, W = hi + lo (lo*lo dropped)
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_ts(tmem + kColU, tmem + kColZ + k * 8, smem_desc_sw128(sWh + k * 32, 16, 1024), id64, k > 0);
        if (!(a.drop_lo & 4u)) {
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma_ts(tmem + kColU, tmem + kColZ + 32 + k * 8, smem_desc_sw128(sWh + k * 32, 16, 1024), id64, true);
        }
        if (!(a.drop_lo & 8u)) {
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma_ts(tmem + kColU, tmem + kColZ + k * 8, smem_desc_sw128(sWl + k * 32, 16, 1024), id64, true);
        }
        umma_commit(b_mo);
        MDN_MARK(c, kEvMmaIssued);
      }
    }
  } else if (warp < 4) {
    // ================================================================== critical-path epilogue (P, EPI-1, EPI-2)
    const int d = tid;                                              // value column = tensor-memory lane
    const uint32_t tl = tmem + (static_cast<uint32_t>(warp * 32) << 16);
    for (int c = 0; c <= nch; ++c) {
      // ---------------- P(c)
      float al = 0.f, bl = 0.f, ml = 0.f;
      if (c > 0) {
        MDN_WAIT(b_m3, (c - 1) & 1);
        MDN_MARK(c - 1, kEvM3Seen);
      }
      if (c < nch) {
        MDN_WAIT((c & 1) ? b_full1 : b_full0, (c >> 1) & 1);
        const float* cf = reinterpret_cast<const float*>(smem + kOffStage + (c & 1) * kStageBytes + kStCoef);
        al = cf[kAbar * C + C - 1]; bl = cf[kB * C + C - 1]; ml = cf[kMubar * C + C - 1];
        MDN_MARK(c, kEvFullSeen);
      }
      __syncwarp();
      tc_fence_after_sync();
#pragma unroll 1
      for (int cs = 0; cs < 4; ++cs) {
        uint32_t sr[32], mr[32];
        if (c == 0) {
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            sr[j] = __float_as_uint(a.S0 ? __ldg(a.S0 + st_off + (size_t)(cs * 32 + j) * kD + d) : 0.f);
            mr[j] = __float_as_uint(a.M0 ? __ldg(a.M0 + st_off + (size_t)(cs * 32 + j) * kD + d) : 0.f);
          }
        } else {
          tmem_ld32(tl + kColS + cs * 32, sr);
          tmem_ld32(tl + kColM + cs * 32, mr);
          tmem_wait_ld();
        }
        if (c < nch) {
          uint8_t* sb = smem + kOffSb + (cs >> 1) * 16384;
          uint8_t* mb = smem + kOffMb + (cs >> 1) * 16384;
#pragma unroll
          for (int j8 = 0; j8 < 4; ++j8) {
            uint4 ps, pm;
            ps.x = pack_bf16(__uint_as_float(sr[j8 * 8 + 0]), __uint_as_float(sr[j8 * 8 + 1]));
            ps.y = pack_bf16(__uint_as_float(sr[j8 * 8 + 2]), __uint_as_float(sr[j8 * 8 + 3]));
            ps.z = pack_bf16(__uint_as_float(sr[j8 * 8 + 4]), __uint_as_float(sr[j8 * 8 + 5]));
            ps.w = pack_bf16(__uint_as_float(sr[j8 * 8 + 6]), __uint_as_float(sr[j8 * 8 + 7]));
            pm.x = pack_bf16(__uint_as_float(mr[j8 * 8 + 0]), __uint_as_float(mr[j8 * 8 + 1]));
            pm.y = pack_bf16(__uint_as_float(mr[j8 * 8 + 2]), __uint_as_float(mr[j8 * 8 + 3]));
            pm.z = pack_bf16(__uint_as_float(mr[j8 * 8 + 4]), __uint_as_float(mr[j8 * 8 + 5]));
            pm.w = pack_bf16(__uint_as_float(mr[j8 * 8 + 6]), __uint_as_float(mr[j8 * 8 + 7]));
            const uint32_t off = sw128_offset(d, (cs & 1) * 32 + j8 * 8);
            *reinterpret_cast<uint4*>(sb + off) = ps;
            *reinterpret_cast<uint4*>(mb + off) = pm;
          }
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float sv = __uint_as_float(sr[j]), mv = __uint_as_float(mr[j]);
            sr[j] = __float_as_uint(al * sv - bl * mv);
            mr[j] = __float_as_uint(ml * mv);
          }
          tmem_st32(tl + kColS + cs * 32, sr);
          tmem_st32(tl + kColM + cs * 32, mr);
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            if (a.Sf) a.Sf[st_off + (size_t)(cs * 32 + j) * kD + d] = __uint_as_float(sr[j]);
            if (a.Mf) a.Mf[st_off + (size_t)(cs * 32 + j) * kD + d] = __uint_as_float(mr[j]);
          }
        }
      }
      if (c == nch) break;
      tmem_wait_st();
      fence_proxy_async_smem();
      tc_fence_before_sync();
      mbar_arrive(b_sb);
      MDN_MARK(c, kEvSbArrive);

      const uint32_t ph = c & 1;
      const uint8_t* stg = smem + kOffStage + (c & 1) * kStageBytes;
      const float* cf = reinterpret_cast<const float*>(stg + kStCoef);
      const __nv_bfloat16* sV = reinterpret_cast<const __nv_bfloat16*>(stg + kStV);
      // ---------------- EPI-1: R^T = V^T - abar .* X + (alpha b^-) .* Y  -> bf16 hi, lo in X
      MDN_WAIT(b_m1, ph);
      __syncwarp();
      tc_fence_after_sync();
      MDN_MARK(c, kEvM1Seen);
      {
        uint32_t hi[32], lo[32];
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          uint32_t x[32], y[32];
          tmem_ld32(tl + kColX + hh * 32, x);
          tmem_ld32(tl + kColY + hh * 32, y);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; j += 2) {
            const int r = hh * 32 + j;
            const float2 ab = *reinterpret_cast<const float2*>(cf + kAbar * C + r);
            const float2 pb = *reinterpret_cast<const float2*>(cf + kAlphaBPrev * C + r);
            const float v0 = __bfloat162float(sV[r * kD + d]), v1 = __bfloat162float(sV[(r + 1) * kD + d]);
            const float r0 = v0 - ab.x * __uint_as_float(x[j]) + pb.x * __uint_as_float(y[j]);
            const float r1 = v1 - ab.y * __uint_as_float(x[j + 1]) + pb.y * __uint_as_float(y[j + 1]);
            float h0, l0, h1, l1;
            split_bf16(r0, h0, l0);
            split_bf16(r1, h1, l1);
            hi[r >> 1] = pack_bf16(h0, h1);
            lo[r >> 1] = pack_bf16(l0, l1);
          }
        }
        tmem_st32(tl + kColX, hi);
        tmem_st32(tl + kColX + 32, lo);
        tmem_wait_st();
      }
      tc_fence_before_sync();
      mbar_arrive(b_r);
      MDN_MARK(c, kEvRArrive);
      // ---------------- EPI-2: V~ -> (gamma_C eta) V~, ((mubar_C/mubar) eta) V~, V~ as bf16 hi, lo
      MDN_WAIT(b_m2, ph);
      MDN_WAIT(b_zq, ph);
      __syncwarp();
      tc_fence_after_sync();
      MDN_MARK(c, kEvM2Seen);
      {
        uint32_t vt[64];
        tmem_ld32(tl + kColY, *reinterpret_cast<uint32_t(*)[32]>(&vt[0]));
        tmem_ld32(tl + kColY + 32, *reinterpret_cast<uint32_t(*)[32]>(&vt[32]));
        tmem_wait_ld();
#pragma unroll
        for (int gq = 0; gq < 4; ++gq) {
          uint32_t sh[8], sl[8], mh[8], mlo[8], vh[8], vl[8];
#pragma unroll
          for (int jj = 0; jj < 8; ++jj) {
            const int r = gq * 16 + 2 * jj;
            const float2 gs = *reinterpret_cast<const float2*>(cf + kGS * C + r);
            const float2 gm = *reinterpret_cast<const float2*>(cf + kGM * C + r);
            const float v0 = __uint_as_float(vt[r]), v1 = __uint_as_float(vt[r + 1]);
            float h0, l0, h1, l1;
            split_bf16(gs.x * v0, h0, l0); split_bf16(gs.y * v1, h1, l1);
            sh[jj] = pack_bf16(h0, h1); sl[jj] = pack_bf16(l0, l1);
            split_bf16(gm.x * v0, h0, l0); split_bf16(gm.y * v1, h1, l1);
            mh[jj] = pack_bf16(h0, h1); mlo[jj] = pack_bf16(l0, l1);
            split_bf16(v0, h0, l0); split_bf16(v1, h1, l1);
            vh[jj] = pack_bf16(h0, h1); vl[jj] = pack_bf16(l0, l1);
          }
          tmem_st8(tl + kColX + gq * 8, sh); tmem_st8(tl + kColX + 32 + gq * 8, sl);
          tmem_st8(tl + kColY + gq * 8, mh); tmem_st8(tl + kColY + 32 + gq * 8, mlo);
          tmem_st8(tl + kColZ + gq * 8, vh); tmem_st8(tl + kColZ + 32 + gq * 8, vl);
        }
        tmem_wait_st();
      }
      tc_fence_before_sync();
      mbar_arrive(b_v);
      MDN_MARK(c, kEvVArrive);
      mbar_arrive((c & 1) ? b_empty1 : b_empty0);
    }
  } else {
    // ================================================================== output epilogue
    const int d = tid - 128;
    const uint32_t tl = tmem + (static_cast<uint32_t>((warp - 4) * 32) << 16);
    TO* o = static_cast<TO*>(a.o);
    for (int c = 0; c < nch; ++c) {
      const uint32_t ph = c & 1;
      const int n = min(C, sq.len - c * C);
      const size_t tok = (size_t)(sq.tok0 + c * C) * H + h;
      const float* cf = reinterpret_cast<const float*>(smem + kOffStage + (c & 1) * kStageBytes + kStCoef);
      MDN_WAIT((c & 1) ? b_full1 : b_full0, (c >> 1) & 1);
      MDN_WAIT(b_mq, ph);
      __syncwarp();
      tc_fence_after_sync();
      MDN_MARK(c, kEvMqSeen);
      float oi[64];
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        uint32_t z[32], u[32];
        tmem_ld32(tl + kColZ + hh * 32, z);
        tmem_ld32(tl + kColU + hh * 32, u);
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const int r = hh * 32 + j;
          oi[r] = a.scale * (cf[kAbar * C + r] * __uint_as_float(z[j]) - cf[kB * C + r] * __uint_as_float(u[j]));
        }
      }
      tc_fence_before_sync();
      mbar_arrive(b_zq);
      MDN_MARK(c, kEvZqArrive);
      MDN_WAIT(b_mo, ph);
      __syncwarp();
      tc_fence_after_sync();
      MDN_MARK(c, kEvMoSeen);
      {
        uint32_t u[64];
        tmem_ld32(tl + kColU, *reinterpret_cast<uint32_t(*)[32]>(&u[0]));
        tmem_ld32(tl + kColU + 32, *reinterpret_cast<uint32_t(*)[32]>(&u[32]));
        tmem_wait_ld();
        // U and this stage's coefficients are in registers: hand both back before the global stores
        tc_fence_before_sync();
        mbar_arrive(b_zu);
        mbar_arrive((c & 1) ? b_empty1 : b_empty0);
        MDN_MARK(c, kEvZuArrive);
        if (!(a.drop_lo & 16u)) {
#pragma unroll
          for (int r = 0; r < 64; ++r)
            if (r < n) store_o<TO>(o + (tok + (size_t)r * H) * kD + d, oi[r] + __uint_as_float(u[r]));
        } else {   // debug: one store per thread instead of 64
          float acc = 0.f;
#pragma unroll
          for (int r = 0; r < 64; ++r) acc += oi[r] + __uint_as_float(u[r]);
          store_o<TO>(o + tok * kD + d, acc);
        }
        MDN_MARK(c, kEvStoresDone);
      }
    }
  }
#undef MDN_WAIT
#undef MDN_MARK

  if (!ok && lane == 0) atomicCAS(a.status, kDevOk, kDevTimeout);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == kWarpMma) tmem_dealloc(tmem, 512);
}

}  // namespace

bool tensor_path_supported(const mdn_params& p) {
  return p.io_dtype == MDN_BF16 && p.dk == kD && p.dv == kD && p.chunk == C;
}

cudaError_t launch_intra_tensor(const Plan& pl, const void* q, const void* k, int* launches) {
  return launch_intra_mma(pl, q, k, launches);
}

cudaError_t launch_chain_tensor(const Plan& pl, const void* q, const void* k, const void* v, const float* S0,
                                const float* M0, void* o, float* Sf, float* Mf, int* launches) {
  const mdn_params& p = pl.p;
  const uint64_t tokens = (uint64_t)p.B * p.T;
  const uint64_t mats = (uint64_t)pl.geom.num_slots * p.H;
  CUtensorMap mq, mk, mv, mt, mw;
  const uint64_t row = (uint64_t)p.H * kD;
  if (!encode_tma_2d_bf16(&mq, TmaMap2D{q, row, tokens, row * 2, 64, 64, true}) ||
      !encode_tma_2d_bf16(&mk, TmaMap2D{k, row, tokens, row * 2, 64, 64, true}) ||
      !encode_tma_2d_bf16(&mv, TmaMap2D{v, row, tokens, row * 2, 128, 64, false}) ||
      !encode_tma_2d_bf16(&mt, TmaMap2D{pl.ws + pl.lay.off_T, 64, mats * C, 128, 64, 64, true}) ||
      !encode_tma_2d_bf16(&mw, TmaMap2D{pl.ws + pl.lay.off_W, 64, 2 * mats * C, 128, 64, 64, true}))
    return cudaErrorInvalidValue;
  ChainArgs a;
  a.g = pl.geom;
  a.coef = reinterpret_cast<const float*>(pl.ws + pl.lay.off_coef);
  a.S0 = S0; a.M0 = M0; a.o = o; a.Sf = Sf; a.Mf = Mf;
  a.status = reinterpret_cast<int32_t*>(pl.ws + pl.lay.off_status);
  a.scale = p.scale;
  a.w_lo_row_offset = (uint32_t)(mats * C);
  const char* drop = getenv("MDN_DEBUG_DROP_LO");
  a.drop_lo = drop ? (uint32_t)atoi(drop) : 0u;
  const char* tl = getenv("MDN_DEBUG_TIMELINE");   // device address of an int64 buffer, [chunks][32]
  a.timeline = tl ? reinterpret_cast<long long*>(strtoull(tl, nullptr, 0)) : nullptr;
  const unsigned grid = (unsigned)pl.geom.num_seqs * p.H;
  cudaError_t e;
  if (p.o_dtype == MDN_BF16) {
    auto kern = chain_tensor_kernel<__nv_bfloat16>;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    kern<<<grid, kThreads, kSmemBytes, pl.stream>>>(a, mq, mk, mv, mt, mw);
  } else {
    auto kern = chain_tensor_kernel<float>;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    kern<<<grid, kThreads, kSmemBytes, pl.stream>>>(a, mq, mk, mv, mt, mw);
  }
  e = cudaGetLastError();
  if (e == cudaSuccess) ++*launches;
  return e;
}

}  // namespace mdn
