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
// Layer operations (template flag kLayer; Section 3.3): with the fused q/k step the accumulators X, Y are scaled by
// 1 / |k| (folded into the coefficient vectors), EPI-1 leaves -d K S, -d K M in Z, U and MMA-1b runs after MMA-2,
// accumulating onto them; with the fused output step the staged fp32 tile is re-read row-wise for RMSNorm, weight
// and sigmoid gate before the TMA store.  kLayer = false is the plain forward, compiled without any of it.
//
// Warp roles: 8 (plain forward) or 16 (with layer operations) epilogue warps, lane quarter x token group, every one
// running P, EPI-o, EPI-1, EPI-2 on its share; then the TMA producer (2-stage ring: K, Q, V, T, W_hi, W_lo, 8 coefficient vectors per chunk; it also
// issues the output stores) and the MMA issuer (one elected lane, tensor-memory owner).  All hand-offs are
// mbarriers with bounded waits; tensor-memory column reuse is ordered by those same barriers.
#include <cstdlib>
#include <cstring>

#include "mdn_common.cuh"
#include "tc_utils.cuh"

namespace mdn {
namespace {

using namespace tc;

constexpr int kD = 128;
// Epilogue warps: 4 lane quarters (value rows 32 q .. +31 = the tensor-memory lanes a warp may touch) x TG token
// groups of 64 / TG tokens, followed by the TMA producer warp and the MMA issuer warp.  The epilogue steps are bound
// by fixed latencies (tensor-memory round trips, group barriers), not by instruction issue: the plain forward is
// as fast with 8 epilogue warps (TG = 2, 168 registers per thread) as with 16; the variant with the layer
// operations, whose output step is instruction-heavy, gains 3 % from 16 (TG = 4, 96 registers).
template <int TG> struct Roles {
  static_assert(TG == 2 || TG == 4, "token groups");
  static constexpr int kTG = TG;
  static constexpr int kTok = C / TG;          // tokens per epilogue warp in the per-token steps
  static constexpr int kPk = kTok / 2;         // 32-bit words of packed bf16 pairs for those tokens
  static constexpr int kEpiWarps = 4 * TG;
  static constexpr int kThreads = (kEpiWarps + 2) * 32;
};
constexpr int token_groups(bool layer) { return layer ? 4 : 2; }

// shared memory (offsets from a 1024-byte aligned base)
constexpr uint32_t kOffSb = 0, kOffMb = 32768, kOffStage = 65536;
constexpr uint32_t kStK = 0, kStQ = 16384, kStV = 32768, kStT = 49152, kStWh = 57344, kStWl = 65536, kStCoef = 73728;
constexpr uint32_t kCoefBytes = kChainCoefs * C * sizeof(float);
constexpr uint32_t kStageBytes = 75776;
constexpr uint32_t kTxBytes = 3 * 16384 + 3 * 8192 + kCoefBytes;
constexpr uint32_t kTxQW = 16384 + 2 * 8192, kTxV = 16384;   // bytes of the Q + W_hi + W_lo tiles, of the V tile
constexpr uint32_t kSmemBytes = kOffStage + 2 * kStageBytes + 1024;
static_assert(kStCoef + kCoefBytes <= kStageBytes, "stage layout");

// tensor memory columns (512 x 128 lanes x 32 bit)
constexpr uint32_t kColS = 0, kColM = 128, kColX = 256, kColY = 320, kColZ = 384, kColU = 448;

struct Bars {
  uint64_t full[2];   // TMA loads of a stage landed                                   (1 + tx bytes)
  uint64_t go[2];     // a stage's output tile is staged and nobody reads the stage any more (256)
  uint64_t sb;        // P part 1: S_b, M_b in smem                                    (256)
  uint64_t m1;        // MMA-1a done                                                   (commit)
  uint64_t mq;        // MMA-1b done                                                   (commit)
  uint64_t r;         // EPI-1 done: R^T hi/lo in X                                     (256)
  uint64_t m2;        // MMA-2 done                                                    (commit)
  uint64_t v1;        // EPI-2a done: V~_S, V~_M operands in X, Y; masters pre-scaled   (256)
  uint64_t v2;        // EPI-2b done: V~ operand in Z                                   (256)
  uint64_t m3;        // MMA-3 done                                                    (commit)
  uint64_t mo;        // MMA-3' done                                                   (commit)
  uint64_t zu;        // U (intra-chunk output) has been read                           (256)
  uint64_t dump;      // the producer has copied S_b, M_b of a chunk out (chunk-state dump only)   (1)
  uint64_t pn[4];     // fused output step: the staged rows of a token group are in shared memory (128 each)
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
  // parallel inter-chunk scan (seg_G = 0: off, one CTA walks all chunks of its chain)
  int seg_G;                  // segments per sequence
  int seg_phase;              // 1: segment 0 + the Psi / Phi runs of the middle segments; 3: segments 1.. from E
  float* seg_E;               // [chains][G-1][2][dk*dv]  state at the END of segment g (start of g+1)
  float* seg_Psi;             // [chains][G-2][2][dk*dv]  segment run from a zero state
  float* seg_PhiS;            // [chains][G-2][2][dk*dv]  segment run with V = 0 from (S, M) = (I, 0)
  float* seg_PhiM;            // [chains][G-2][2][dk*dv]  ... from (0, I)
  // layer operations absorbed by this kernel (Section 3.3)
  int qk_on;                  // q <- L2Norm(q - d k), k <- L2Norm(k): coefficient vectors 6, 7 hold 1/|k|, 1/|q - d k|
  const float* qk_d;          // [H] or NULL
  int post_on;                // o <- sigmoid(g) * RMSNorm(o) * w in the output epilogue
  const float* post_w;        // [dv] or NULL
  const void* post_g;         // [B,T,H,dv] bf16
  float post_eps;
  // training / backward support
  uint8_t* dump;              // NULL, or [slot][H][65536]: the bf16 copies S_b^T | M_b^T of the state at the START of
                              // every chunk, as they lie in shared memory (two [128 x 128 B] swizzled blocks each)
  int state_only;             // no output terms (no Q, W loads, no output MMAs): states (and the dump) only
  int end_scalars_in_rk;      // (abar_C, b_C, mubar_C) of a chunk are entries 0..2 of coefficient vector 6, not the
                              // last entries of vectors 0, 1, 5 (the adjoint chain decouples them)
  float* vt_dump;             // NULL, or [chunk slot][64][H][dv] fp32: V~ of every chunk as EPI-2 reads it
  int mirror;                 // with inject: q, k, G and T are the ORIGINAL tensors of a problem whose chunks this run
  ChunkGeom mirror_g;         // walks in reverse order (geometry mirror_g): chunk c of this run reads the rows of
                              // original chunk nchunks - 1 - c (rows past a short chunk's end meet zero coefficients)
                              // and uses that chunk's T transposed (the tile is read MN-major)
  int inject;                 // state-only runs: a second rank-64 update of the pair per chunk, S^T += G_S^T Q,
                              // M^T -= G_M^T Q with G_S = (-scale b) . G, G_M = (-scale g_M) . G (b, g_M: coefficient
                              // vectors 1 and 4), G the [B,T,H,dv] bf16 tensor passed as `o`, Q the q tensor: the two Q
                              // terms of the adjoint state recurrence
  uint32_t drop_lo;           // debug: bit 0 R, 1 V~_S/V~_M, 2 V~ (output), 3 W: leave that operand's lo part out
  long long* timeline;        // debug: CTA 0 writes clock64() at [chunk*32 + event] (NULL = off)
};

// Timeline events (debug).
enum Ev : int { kEvMmaStart = 0, kEvM1Seen, kEvRArrive, kEvM2Seen, kEvVArrive, kEvM3Seen, kEvSbArrive, kEvMqSeen,
                kEvZqArrive, kEvMoSeen, kEvZuArrive, kEvMmaIssued, kEvRSeen, kEvVSeen, kEvTmaIssued, kEvFullSeen,
                kEvStoresDone, kEvV2Arrive, kEvPrescaled };

// sigmoid(x) = (1 + tanh(x / 2)) / 2 with the one-instruction tanh approximation (relative error ~2^-11)
__device__ __forceinline__ float sigmoid_fast(float x) {
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(0.5f * x));
  return fmaf(0.5f, t, 0.5f);
}

template <typename TO> __device__ __forceinline__ void stage_o(uint8_t* tile, int r, int d, float x);
template <> __device__ __forceinline__ void stage_o<float>(uint8_t* tile, int r, int d, float x) {
  reinterpret_cast<float*>(tile)[r * kD + d] = x;
}
template <> __device__ __forceinline__ void stage_o<__nv_bfloat16>(uint8_t* tile, int r, int d, float x) {
  reinterpret_cast<__nv_bfloat16*>(tile)[r * kD + d] = __float2bfloat16_rn(x);
}

// kTrain compiles in the chunk-state dump, the state-only switch and the decoupled end-of-chunk scalars (the plain
// forward's instantiation stays as it is: its schedule is fragile, a runtime test of these options cost it 2 %)
template <typename TO, bool kLayer, bool kTrain = false>
__global__ void __launch_bounds__(Roles<token_groups(kLayer)>::kThreads, 1) chain_tensor_kernel(const ChainArgs a,
                                                                  const __grid_constant__ CUtensorMap map_q,
                                                                  const __grid_constant__ CUtensorMap map_k,
                                                                  const __grid_constant__ CUtensorMap map_v,
                                                                  const __grid_constant__ CUtensorMap map_t,
                                                                  const __grid_constant__ CUtensorMap map_w,
                                                                  const __grid_constant__ CUtensorMap map_o) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ __align__(8) Bars bars;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  __shared__ __align__(16) float w_sm[kLayer ? kD : 4];   // RMSNorm weight of the fused output step

  using R = Roles<token_groups(kLayer)>;
  constexpr int kTG = R::kTG, kTok = R::kTok, kPk = R::kPk, kEpiWarps = R::kEpiWarps;
  constexpr int kWarpTma = kEpiWarps, kWarpMma = kEpiWarps + 1;
  constexpr bool kWarpArrive = kLayer;   // epilogue hand-overs: one mbarrier arrival per warp, or one per thread
  constexpr int kArrivals = kWarpArrive ? kEpiWarps : kEpiWarps * 32;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int H = a.g.H;
  // ---- work item: which chain, which segment of it, which kind of run
  int chain = blockIdx.x, seg = 0, run = 0;   // run 0: the real thing; 1: Psi; 2: Phi from (I, 0); 3: Phi from (0, I)
  if (a.seg_G > 0) {
    if (a.seg_phase == 1) {
      const int items = 1 + 3 * (a.seg_G - 2);
      chain = blockIdx.x / items;
      const int w = blockIdx.x % items;
      if (w > 0) { seg = 1 + (w - 1) / 3; run = 1 + (w - 1) % 3; }
    } else {
      chain = blockIdx.x / (a.seg_G - 1);
      seg = 1 + blockIdx.x % (a.seg_G - 1);
    }
  }
  const int seq = chain / H, h = chain % H;
  grid_dependency_wait();   // chunk map, coefficients, T and W (and segment states) come from the previous kernels
  SeqInfo sq = seq_info(a.g, seq);
  if (a.seg_G > 0) {        // restrict the view to this segment's chunks
    const int per = (sq.nchunks + a.seg_G - 1) / a.seg_G;
    const int cb = min(sq.nchunks, seg * per), ce = min(sq.nchunks, (seg + 1) * per);
    sq.slot0 += cb;
    sq.tok0 += cb * C;
    sq.len = (ce > cb) ? min(sq.len - cb * C, (ce - cb) * C) : 0;
    sq.nchunks = ce - cb;
  }
  const int nch = sq.nchunks;
  const size_t st_off = (size_t)chain * kD * kD;
  // ---- where the start state comes from, where the end state goes, whether V counts, whether o is written
  const float* S0p = a.S0 ? a.S0 + st_off : nullptr;
  const float* M0p = a.M0 ? a.M0 + st_off : nullptr;
  float* Sfp = a.Sf ? a.Sf + st_off : nullptr;
  float* Mfp = a.Mf ? a.Mf + st_off : nullptr;
  bool id_s = false, id_m = false, v_zero = false, write_o = true;
  if (a.seg_G > 0) {
    constexpr size_t kMat = (size_t)kD * kD;
    auto e_ptr = [&](int gi, int which) { return a.seg_E + (((size_t)chain * (a.seg_G - 1) + gi) * 2 + which) * kMat; };
    if (run == 0) {
      if (seg > 0) { S0p = e_ptr(seg - 1, 0); M0p = e_ptr(seg - 1, 1); }
      if (seg < a.seg_G - 1) {
        Sfp = (seg == 0) ? e_ptr(0, 0) : nullptr;
        Mfp = (seg == 0) ? e_ptr(0, 1) : nullptr;
      }
    } else {
      write_o = false;
      S0p = M0p = nullptr;
      id_s = run == 2; id_m = run == 3; v_zero = run >= 2;
      float* base = (run == 1 ? a.seg_Psi : run == 2 ? a.seg_PhiS : a.seg_PhiM) +
                    (((size_t)chain * (a.seg_G - 2) + (seg - 1)) * 2) * kMat;
      Sfp = base; Mfp = base + kMat;
    }
  }
  if constexpr (kTrain) {
    if (a.state_only) write_o = false;
  }

  const uint32_t s_base = smem_u32(smem);
  const uint32_t b_full0 = smem_u32(&bars.full[0]), b_full1 = smem_u32(&bars.full[1]);
  const uint32_t b_go0 = smem_u32(&bars.go[0]), b_go1 = smem_u32(&bars.go[1]);
  const uint32_t b_sb = smem_u32(&bars.sb), b_m1 = smem_u32(&bars.m1), b_mq = smem_u32(&bars.mq);
  const uint32_t b_r = smem_u32(&bars.r), b_m2 = smem_u32(&bars.m2);
  const uint32_t b_v1 = smem_u32(&bars.v1), b_v2 = smem_u32(&bars.v2), b_m3 = smem_u32(&bars.m3);
  const uint32_t b_mo = smem_u32(&bars.mo), b_zu = smem_u32(&bars.zu), b_dump = smem_u32(&bars.dump);
  // kLayer = false compiles the layer operations out: the plain forward keeps its instruction count
  const bool qk_on = kLayer && a.qk_on;
  const bool post = kLayer && a.post_on && write_o;
  const float dh = (qk_on && a.qk_d) ? __ldg(a.qk_d + h) : 0.f;

  if (tid == 0) {
    abort_flag = 0;
    mbar_init(b_full0, 1); mbar_init(b_full1, 1);
    mbar_init(b_go0, kArrivals); mbar_init(b_go1, kArrivals);
    mbar_init(b_sb, kArrivals); mbar_init(b_r, kArrivals); mbar_init(b_v1, kArrivals);
    mbar_init(b_v2, kArrivals);
    mbar_init(b_zu, kArrivals);
    mbar_init(b_dump, 1);
    mbar_init(b_m1, 1); mbar_init(b_mq, 1); mbar_init(b_m2, 1); mbar_init(b_m3, 1); mbar_init(b_mo, 1);
    for (int i = 0; i < kTG; ++i) mbar_init(smem_u32(&bars.pn[i]), 128);
    mbar_fence_init();
  }
  if (kLayer && tid < kD) w_sm[tid] = (a.post_on && a.post_w) ? __ldg(a.post_w + tid) : 1.f;
  if (warp == kWarpMma) tmem_alloc(smem_u32(&tmem_slot), 512);
  if (warp == kWarpTma && lane == 0) {
    prefetch_tensormap(&map_q); prefetch_tensormap(&map_k); prefetch_tensormap(&map_v);
    prefetch_tensormap(&map_t); prefetch_tensormap(&map_w); prefetch_tensormap(&map_o);
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
#ifdef MDN_DEBUG
  long long* const tline = (blockIdx.x == 0) ? a.timeline : nullptr;
#endif
  // Hand-over arrivals of the epilogue.  With 16 epilogue warps (layer variant) one arrival per warp, after the warp
  // has converged (every lane's stores and fences precede it): 32 x fewer shared-memory atomics in front of every
  // hand-over, 2 % of the step.  The 8-warp plain forward measured 1 % slower that way and keeps one per thread.
#define MDN_WARP_ARRIVE(bar)             \
  {                                      \
    if constexpr (kWarpArrive) {         \
      __syncwarp();                      \
      if (lane == 0) mbar_arrive(bar);   \
    } else {                             \
      mbar_arrive(bar);                  \
    }                                    \
  }
#ifdef MDN_DEBUG
#define MDN_MARK(c, ev) \
  if (tline != nullptr && lane == 0 && (warp == 0 || warp >= kEpiWarps)) tline[(c) * 32 + (ev)] = clock64();
#else
#define MDN_MARK(c, ev)
#endif

  if (warp == kWarpTma) {
    // ================================================================== TMA producer + output stores
    // Stage s = c & 1 serves chunk c, then (as the staged output tile) is written out and refilled for chunk c + 2.
    if (lane == 0) {
      int issued = 0;
      for (int c = 0; c < nch + 2; ++c) {
        const int s = c & 1;
        const uint32_t st = s_base + kOffStage + s * kStageBytes;
        if (c >= 2) {
          const int co = c - 2;
          MDN_WAIT(s ? b_go1 : b_go0, (co >> 1) & 1);
          const int n = min(C, sq.len - co * C);
          const int tok0 = sq.tok0 + co * C;
          // the finished tile: at the start of the stage, except the bf16 tile of the fused output step (T / W area)
          const uint32_t src = st + ((post && sizeof(TO) == 2) ? kStT : 0u);
          if (!write_o) {
            // Psi / Phi runs of the parallel scan produce states only
          } else if (n == C) {
            tma_store_2d(&map_o, h * kD, tok0, src);
          } else {   // short chunk: rows >= n belong to another sequence; one bulk copy per valid row
            for (int r = 0; r < n; ++r)
              bulk_store(static_cast<uint8_t*>(a.o) + (((size_t)(tok0 + r) * H + h) * kD) * sizeof(TO),
                         src + r * kD * (uint32_t)sizeof(TO), kD * (uint32_t)sizeof(TO));
          }
          tma_store_commit();
          tma_store_wait_read();
          MDN_MARK(co, kEvStoresDone);
        }
        if (c < nch) {
          const uint32_t fb = s ? b_full1 : b_full0;
          const int tok0 = sq.tok0 + c * C;
          const int mat = (sq.slot0 + c) * H + h;
          // state-only runs need neither Q nor W, and the V = 0 runs no V either
          const bool inj = kTrain && a.inject;   // Q and G (into the W area) instead of Q and W
          int tok0k = tok0;                      // rows of k, q, G
          int mat_t = mat;                       // which T
          if (kTrain && a.mirror) {
            tok0k = seq_info(a.mirror_g, seq).tok0 + (nch - 1 - c) * C;
            mat_t = (sq.slot0 + nch - 1 - c) * H + h;
          }
          mbar_arrive_expect_tx(fb, kTxBytes - ((write_o || inj) ? 0u : kTxQW) - (v_zero ? kTxV : 0u));
          tma_load_2d(st + kStK, &map_k, h * kD, tok0k, fb);
          tma_load_2d(st + kStK + 8192, &map_k, h * kD + 64, tok0k, fb);
          bulk_load(st + kStCoef, a.coef + (size_t)mat * MDN_NUM_COEF * C, kCoefBytes, fb);
          if (!v_zero) tma_load_2d(st + kStV, &map_v, h * kD, tok0, fb);
          tma_load_2d(st + kStT, &map_t, 0, mat_t * C, fb);
          if (write_o) {
            tma_load_2d(st + kStQ, &map_q, h * kD, tok0, fb);
            tma_load_2d(st + kStQ + 8192, &map_q, h * kD + 64, tok0, fb);
            tma_load_2d(st + kStWh, &map_w, 0, mat * C, fb);
            tma_load_2d(st + kStWl, &map_w, 0, mat * C + (int)a.w_lo_row_offset, fb);
          } else if (inj) {
            tma_load_2d(st + kStQ, &map_q, h * kD, tok0k, fb);
            tma_load_2d(st + kStQ + 8192, &map_q, h * kD + 64, tok0k, fb);
            tma_load_2d(st + kStWh, &map_o, h * kD, tok0k, fb);   // G: the tensor map of `o`, used for a load
          }
          MDN_MARK(c, kEvTmaIssued);
          issued = c + 1;
        }
        if (kTrain && a.dump != nullptr && c >= 1 && c <= nch) {   // the state copies of chunk c - 1 (handed over long ago)
          MDN_WAIT(b_sb, (c - 1) & 1);
          uint8_t* dst = a.dump + ((size_t)(sq.slot0 + c - 1) * H + h) * 65536;
          for (int b = 0; b < 4; ++b) bulk_store(dst + b * 16384, s_base + kOffSb + b * 16384, 16384);
          tma_store_commit();
          tma_store_wait_read();
          mbar_arrive(b_dump);
        }
      }
      if (!ok) {   // giving up: let the copies already in flight land before the CTA exits
        for (int c = max(0, issued - 2); c < issued; ++c)
          for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait((c & 1) ? b_full1 : b_full0, (c >> 1) & 1); ++it) {}
      }
      tma_store_wait_all();
    }
  } else if (warp == kWarpMma) {
    // ================================================================== MMA issuer
    if (lane == 0) {
      // Column of the bf16 A operands the epilogue leaves in X, Y, Z: K-step k covers tokens 16k .. 16k + 15; the
      // epilogue warp that owns those tokens keeps hi (part 0) and lo (part 1) inside its own kTok columns
      auto a_col = [](int part, int k) {
        return static_cast<uint32_t>(kTok * ((16 * k) / kTok) + kPk * part + ((16 * k) % kTok) / 2);
      };
      const uint32_t id64 = idesc_bf16(128, 64, false, false, false);
      const uint32_t id128_mn = idesc_bf16(128, 128, false, true, false);
      const uint32_t id128_mn_neg = idesc_bf16(128, 128, false, true, true);
      // descriptors: bases are fixed; stepping K by 16 elements = +32 bytes = +2 in the address field
      const uint64_t dSb0 = smem_desc_sw128(s_base + kOffSb, 16, 1024), dSb1 = smem_desc_sw128(s_base + kOffSb + 16384, 16, 1024);
      const uint64_t dMb0 = smem_desc_sw128(s_base + kOffMb, 16, 1024), dMb1 = smem_desc_sw128(s_base + kOffMb + 16384, 16, 1024);
      for (int c = 0; c < nch; ++c) {
        const int s = c & 1;
        const uint32_t ph = c & 1;
        const uint32_t st = s_base + kOffStage + s * kStageBytes;
        const uint64_t dK0 = smem_desc_sw128(st + kStK, 16, 1024), dK1 = smem_desc_sw128(st + kStK + 8192, 16, 1024);
        const uint64_t dQ0 = smem_desc_sw128(st + kStQ, 16, 1024), dQ1 = smem_desc_sw128(st + kStQ + 8192, 16, 1024);
        const uint64_t dT = smem_desc_sw128(st + kStT, 16, 1024);
        const uint64_t dWh = smem_desc_sw128(st + kStWh, 16, 1024), dWl = smem_desc_sw128(st + kStWl, 16, 1024);
        const uint64_t dKmn = smem_desc_sw128(st + kStK, 8192, 1024);   // K tile read MN-major; +2048 B per 16 tokens
        MDN_WAIT(s ? b_full1 : b_full0, (c >> 1) & 1);
        MDN_WAIT(b_sb, ph);
        tc_fence_after_sync();
        MDN_MARK(c, kEvMmaStart);
        // ---- MMA-1a: X = S_b K^T, Y = M_b K^T
#pragma unroll
        for (int k = 0; k < 8; ++k)
          umma_ss(tmem + kColX, ((k >> 2) ? dSb1 : dSb0) + 2 * (k & 3), ((k >> 2) ? dK1 : dK0) + 2 * (k & 3), id64, k > 0);
#pragma unroll
        for (int k = 0; k < 8; ++k)
          umma_ss(tmem + kColY, ((k >> 2) ? dMb1 : dMb0) + 2 * (k & 3), ((k >> 2) ? dK1 : dK0) + 2 * (k & 3), id64, k > 0);
        umma_commit(b_m1);
        // ---- MMA-1b: Z = S_b Q^T, U = M_b Q^T (U of the previous chunk must have been read).  With the fused q/k
        // step it runs after MMA-2 instead and ACCUMULATES onto -d K S, -d K M, which EPI-1 has put into Z, U.
#define MDN_MMA_1B(onto)                                                                                                  \
  {                                                                                                                        \
    MDN_WAIT(b_zu, ph ^ 1);                                                                                                \
    tc_fence_after_sync();                                                                                                 \
    _Pragma("unroll") for (int k = 0; k < 8; ++k)                                                                          \
        umma_ss(tmem + kColZ, ((k >> 2) ? dSb1 : dSb0) + 2 * (k & 3), ((k >> 2) ? dQ1 : dQ0) + 2 * (k & 3), id64, (onto) || k > 0); \
    _Pragma("unroll") for (int k = 0; k < 8; ++k)                                                                          \
        umma_ss(tmem + kColU, ((k >> 2) ? dMb1 : dMb0) + 2 * (k & 3), ((k >> 2) ? dQ1 : dQ0) + 2 * (k & 3), id64, (onto) || k > 0); \
    umma_commit(b_mq);                                                                                                     \
  }
        // ---- MMA-1b (output terms, off the critical path).  The tensor pipe runs its MMAs in issue order, so a group
        // issued here delays MMA-2 by whatever of it is still running when EPI-1 is done: only Z = S_b Q^T is issued
        // here (it fits under EPI-1) ...
        if constexpr (!kLayer) {
          if (write_o) {
#pragma unroll
            for (int k = 0; k < 8; ++k)
              umma_ss(tmem + kColZ, ((k >> 2) ? dSb1 : dSb0) + 2 * (k & 3), ((k >> 2) ? dQ1 : dQ0) + 2 * (k & 3), id64, k > 0);
          }
        } else {
          if (write_o && !qk_on) MDN_MMA_1B(false);
        }
        // ---- MMA-2: Y = (R_hi + R_lo)^T T^T
        MDN_WAIT(b_r, ph);
        tc_fence_after_sync();
        MDN_MARK(c, kEvRSeen);
        if (kTrain && a.mirror) {   // T^T: the same tile read MN-major (16 rows = 2048 bytes per K step)
          const uint64_t dTmn = smem_desc_sw128(st + kStT, 8192, 1024);
          const uint32_t id64_mn = idesc_bf16(128, 64, false, true, false);
          for (int k = 0; k < 8; ++k)
            umma_ts(tmem + kColY, tmem + kColX + a_col(k >> 2, k & 3), dTmn + 128 * (k & 3), id64_mn, k > 0);
        } else {
#pragma unroll
          for (int k = 0; k < 4; ++k) umma_ts(tmem + kColY, tmem + kColX + a_col(0, k), dT + 2 * k, id64, k > 0);
          if (!(a.drop_lo & 1u)) {
#pragma unroll
            for (int k = 0; k < 4; ++k) umma_ts(tmem + kColY, tmem + kColX + a_col(1, k), dT + 2 * k, id64, true);
          }
        }
        umma_commit(b_m2);
        // ... and U = M_b Q^T here: it fits under EPI-2 and is done before MMA-3 can start
        if constexpr (!kLayer) {
          if (write_o) {
            MDN_WAIT(b_zu, ph ^ 1);
            tc_fence_after_sync();
#pragma unroll
            for (int k = 0; k < 8; ++k)
              umma_ss(tmem + kColU, ((k >> 2) ? dMb1 : dMb0) + 2 * (k & 3), ((k >> 2) ? dQ1 : dQ0) + 2 * (k & 3), id64, k > 0);
            umma_commit(b_mq);
          }
        } else {
          if (write_o && qk_on) MDN_MMA_1B(true);
        }
        if constexpr (kTrain) {
          if (a.inject) {
            // the second update (operands in Z, U and the pre-scaled masters ready since the start of the chunk, Q
            // read MN-major) needs nothing of this chunk's V~: issued here it runs while EPI-2 works, before MMA-3
            const uint64_t dQmn = smem_desc_sw128(st + kStQ, 8192, 1024);
            MDN_WAIT(b_v2, ph);
            tc_fence_after_sync();
            for (int k = 0; k < 8; ++k)
              umma_ts(tmem + kColS, tmem + kColZ + a_col(k >> 2, k & 3), dQmn + 128 * (k & 3), id128_mn, true);
            for (int k = 0; k < 8; ++k)
              umma_ts(tmem + kColM, tmem + kColU + a_col(k >> 2, k & 3), dQmn + 128 * (k & 3), id128_mn_neg, true);
          }
        }
        // ---- MMA-3: S^T += V~_S^T K, M^T -= V~_M^T K   (K tile read MN-major: N = dk, K = tokens)
        MDN_WAIT(b_v1, ph);
        tc_fence_after_sync();
        MDN_MARK(c, kEvVSeen);
        const int n3 = (a.drop_lo & 2u) ? 4 : 8;
        for (int k = 0; k < n3; ++k)
          umma_ts(tmem + kColS, tmem + kColX + a_col(k >> 2, k & 3), dKmn + 128 * (k & 3), id128_mn, true);
        for (int k = 0; k < n3; ++k)
          umma_ts(tmem + kColM, tmem + kColY + a_col(k >> 2, k & 3), dKmn + 128 * (k & 3), id128_mn_neg, true);
        umma_commit(b_m3);
        if (!write_o) continue;   // state-only run: no output terms
        // ---- MMA-3': U = V~^T W^T  with  V~ = hi + lo, W = hi + lo (lo*lo dropped)
        MDN_WAIT(b_v2, ph);
        tc_fence_after_sync();
#pragma unroll
        for (int k = 0; k < 4; ++k) umma_ts(tmem + kColU, tmem + kColZ + a_col(0, k), dWh + 2 * k, id64, k > 0);
        if (!(a.drop_lo & 4u)) {
#pragma unroll
          for (int k = 0; k < 4; ++k) umma_ts(tmem + kColU, tmem + kColZ + a_col(1, k), dWh + 2 * k, id64, true);
        }
        if (!(a.drop_lo & 8u)) {
#pragma unroll
          for (int k = 0; k < 4; ++k) umma_ts(tmem + kColU, tmem + kColZ + a_col(0, k), dWl + 2 * k, id64, true);
        }
        umma_commit(b_mo);
        MDN_MARK(c, kEvMmaIssued);
      }
    }
  } else {
    // ================================================================== epilogue warps
    // lane quarter q4 = warp & 3 (value columns 32 q4 .. +31 = this warp's tensor-memory lanes),
    // token group hf = warp >> 2 (tokens kTok hf .. +kTok-1 in the per-token steps, a share of the dk columns in P).
    const int q4 = warp & 3, hf = warp >> 2;   // hf: token group
    const int d = q4 * 32 + lane;
    const int r0 = kTok * hf;
    const uint32_t tl = tmem + (static_cast<uint32_t>(q4 * 32) << 16);
    uint32_t pn_phase = 0;
    const uint32_t b_pn = smem_u32(&bars.pn[hf]);
    float oi[kTok];   // scale (abar .* Q S - b .* Q M) for this thread's tokens, carried to the output step

#pragma unroll
    for (int j = 0; j < kTok; ++j) oi[j] = 0.f;
    for (int c = 0; c <= nch; ++c) {
      // ---------------- P(c): bf16 copies of S^T, M^T for MMA-1 (after the last chunk: final states)
      float al = 0.f, bl = 0.f, ml = 0.f;
      if (c > 0) {
        MDN_WAIT(b_m3, (c - 1) & 1);
        MDN_MARK(c - 1, kEvM3Seen);
      }
      if (c < nch) {
        MDN_WAIT((c & 1) ? b_full1 : b_full0, (c >> 1) & 1);
        const float* cf = reinterpret_cast<const float*>(smem + kOffStage + (c & 1) * kStageBytes + kStCoef);
        if (kTrain && a.end_scalars_in_rk) {
          al = cf[kRk * C + 0]; bl = cf[kRk * C + 1]; ml = cf[kRk * C + 2];
        } else {
          al = cf[kAbar * C + C - 1]; bl = cf[kB * C + C - 1]; ml = cf[kMubar * C + C - 1];
        }
        if (kTrain && a.dump != nullptr && c > 0) MDN_WAIT(b_dump, (c - 1) & 1);
        MDN_MARK(c, kEvFullSeen);
      }
      __syncwarp();
      tc_fence_after_sync();
      if constexpr (kTG == 2) {   // two passes of 32 dk columns (kept textually apart: the plain forward's schedule is fragile)
#pragma unroll 1
        for (int i = 0; i < 2; ++i) {
          const int cs = 2 * hf + i;   // 32-column slice of dk
          uint32_t sr[32], mr[32];
          if (c == 0) {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const float unit = (cs * 32 + j == d) ? 1.f : 0.f;
              sr[j] = __float_as_uint(S0p ? __ldg(S0p + (size_t)(cs * 32 + j) * kD + d) : (id_s ? unit : 0.f));
              mr[j] = __float_as_uint(M0p ? __ldg(M0p + (size_t)(cs * 32 + j) * kD + d) : (id_m ? unit : 0.f));
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
            // masters scaled by this chunk's (abar_C, b_C, mubar_C) so that MMA-3 can accumulate straight into
            // them; the stores are asynchronous and only waited for before V~_S, V~_M are handed over
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
              if (Sfp) Sfp[(size_t)(cs * 32 + j) * kD + d] = __uint_as_float(sr[j]);
              if (Mfp) Mfp[(size_t)(cs * 32 + j) * kD + d] = __uint_as_float(mr[j]);
            }
          }
        }
      } else {
        constexpr int kPw = (kTG == 4) ? 16 : 32;   // dk columns per pass (a warp owns 128 / kTG of them)
#pragma unroll 1
        for (int i = 0; i < 128 / kTG / kPw; ++i) {
          const int col0 = hf * (128 / kTG) + i * kPw;
          uint32_t sr[kPw], mr[kPw];
          if (c == 0) {
#pragma unroll
            for (int j = 0; j < kPw; ++j) {
              const float unit = (col0 + j == d) ? 1.f : 0.f;
              sr[j] = __float_as_uint(S0p ? __ldg(S0p + (size_t)(col0 + j) * kD + d) : (id_s ? unit : 0.f));
              mr[j] = __float_as_uint(M0p ? __ldg(M0p + (size_t)(col0 + j) * kD + d) : (id_m ? unit : 0.f));
            }
          } else {
            tmem_ld_n<kPw>(tl + kColS + col0, sr);
            tmem_ld_n<kPw>(tl + kColM + col0, mr);
            tmem_wait_ld();
          }
          if (c < nch) {
            uint8_t* sb = smem + kOffSb + (col0 >> 6) * 16384;
            uint8_t* mb = smem + kOffMb + (col0 >> 6) * 16384;
#pragma unroll
            for (int j8 = 0; j8 < kPw / 8; ++j8) {
              uint4 ps, pm;
              ps.x = pack_bf16(__uint_as_float(sr[j8 * 8 + 0]), __uint_as_float(sr[j8 * 8 + 1]));
              ps.y = pack_bf16(__uint_as_float(sr[j8 * 8 + 2]), __uint_as_float(sr[j8 * 8 + 3]));
              ps.z = pack_bf16(__uint_as_float(sr[j8 * 8 + 4]), __uint_as_float(sr[j8 * 8 + 5]));
              ps.w = pack_bf16(__uint_as_float(sr[j8 * 8 + 6]), __uint_as_float(sr[j8 * 8 + 7]));
              pm.x = pack_bf16(__uint_as_float(mr[j8 * 8 + 0]), __uint_as_float(mr[j8 * 8 + 1]));
              pm.y = pack_bf16(__uint_as_float(mr[j8 * 8 + 2]), __uint_as_float(mr[j8 * 8 + 3]));
              pm.z = pack_bf16(__uint_as_float(mr[j8 * 8 + 4]), __uint_as_float(mr[j8 * 8 + 5]));
              pm.w = pack_bf16(__uint_as_float(mr[j8 * 8 + 6]), __uint_as_float(mr[j8 * 8 + 7]));
              const uint32_t off = sw128_offset(d, (col0 & 63) + j8 * 8);
              *reinterpret_cast<uint4*>(sb + off) = ps;
              *reinterpret_cast<uint4*>(mb + off) = pm;
            }
            // masters scaled by this chunk's (abar_C, b_C, mubar_C) so that MMA-3 can accumulate straight into
            // them; the stores are asynchronous and only waited for before V~_S, V~_M are handed over
#pragma unroll
            for (int j = 0; j < kPw; ++j) {
              const float sv = __uint_as_float(sr[j]), mv = __uint_as_float(mr[j]);
              sr[j] = __float_as_uint(al * sv - bl * mv);
              mr[j] = __float_as_uint(ml * mv);
            }
            tmem_st_n<kPw>(tl + kColS + col0, sr);
            tmem_st_n<kPw>(tl + kColM + col0, mr);
          } else {
#pragma unroll
            for (int j = 0; j < kPw; ++j) {
              if (Sfp) Sfp[(size_t)(col0 + j) * kD + d] = __uint_as_float(sr[j]);
              if (Mfp) Mfp[(size_t)(col0 + j) * kD + d] = __uint_as_float(mr[j]);
            }
          }
        }
      }
      if (c < nch) {
        fence_proxy_async_smem();
        MDN_WARP_ARRIVE(b_sb);
        MDN_MARK(c, kEvSbArrive);
      }
      // ---------------- output of the previous chunk (under MMA-1a): o^T = oi + U, staged as a [64 x 128] tile in
      // the previous chunk's stage (all its MMAs are done and nobody reads its tiles any more)
      if (c > 0 && !write_o) {
        // state-only run: MMA-3 of the previous chunk (waited for above) was the last reader of its stage
        MDN_WARP_ARRIVE(((c - 1) & 1) ? b_go1 : b_go0);
      } else if (c > 0) {
        const int cp = c - 1;
        uint8_t* stp = smem + kOffStage + (cp & 1) * kStageBytes;
        // fused output step: this thread's share of the chunk's output-gate rows is four threads per token, 8-byte
        // pieces (each warp-load covers eight full 32-byte sectors); the rows are pulled towards L2 here and read
        // once the tile is staged, when registers are free again
        constexpr int kTpr = 128 / kTok, kPieces = 32 / kTpr;   // threads per row, 16-byte pieces per thread
        const int t128 = q4 * 32 + lane, prow = r0 + t128 / kTpr, part = t128 % kTpr;
        const bool g_live = post && cp * C + prow < sq.len;
        const uint2* gp = reinterpret_cast<const uint2*>(static_cast<const __nv_bfloat16*>(a.post_g) +
                                                         ((size_t)(sq.tok0 + cp * C + prow) * H + h) * kD) + part;
        if (g_live && part < 2) asm volatile("prefetch.global.L2 [%0];" ::"l"(gp + 15 * part));   // bytes 0 and 128 of the row (parts 0, 1)
        MDN_WAIT(b_mo, cp & 1);
        __syncwarp();
        tc_fence_after_sync();
        MDN_MARK(cp, kEvMoSeen);
        {
          uint32_t u[kTok];
          tmem_ld_n<kTok>(tl + kColU + r0, u);
          tmem_wait_ld();
          tc_fence_before_sync();
          MDN_WARP_ARRIVE(b_zu);
          MDN_MARK(cp, kEvZuArrive);
          if (!post) {
#pragma unroll
            for (int j = 0; j < kTok; ++j) stage_o<TO>(stp, r0 + j, d, oi[j] + __uint_as_float(u[j]));
          } else {
            // fused output step: y = sigmoid(g) * o / sqrt(mean_d o^2 + eps) * w_d.  The fp32 tile is staged first
            // (value columns across lanes), then re-read row-wise: four threads per token sum its 128 squares,
            // rescale, gate and write the final tile (in place for fp32 output, into the T / W area for bf16).
            float* tile = reinterpret_cast<float*>(stp);
#pragma unroll
            for (int j = 0; j < kTok; ++j) tile[(r0 + j) * kD + d] = oi[j] + __uint_as_float(u[j]);
            uint2 graw[kPieces];
#pragma unroll
            for (int i = 0; i < kPieces; ++i) graw[i] = g_live ? __ldg(gp + kTpr * i) : make_uint2(0u, 0u);
            mbar_arrive(b_pn);
            MDN_WAIT(b_pn, pn_phase);
            pn_phase ^= 1;
            __syncwarp();
            const int row = prow;
            float4 ov[kPieces];
            float ss = 0.f;
#pragma unroll
            for (int i = 0; i < kPieces; ++i) {   // interleaved 16-byte pieces: a row's threads cover contiguous bytes
              ov[i] = *reinterpret_cast<const float4*>(tile + row * kD + (part + kTpr * i) * 4);
              ss = fmaf(ov[i].x, ov[i].x, fmaf(ov[i].y, ov[i].y, fmaf(ov[i].z, ov[i].z, fmaf(ov[i].w, ov[i].w, ss))));
            }
#pragma unroll
            for (int off = 1; off < kTpr; off <<= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
            const float rstd = rsqrtf(ss * (1.f / kD) + a.post_eps);
#pragma unroll
            for (int i = 0; i < kPieces; ++i) {
              const int col = (part + kTpr * i) * 4;
              const float4 wv = *reinterpret_cast<const float4*>(w_sm + col);
              const uint2 gr = graw[i];
              const float g0 = __uint_as_float(gr.x << 16), g1 = __uint_as_float(gr.x & 0xffff0000u);
              const float g2 = __uint_as_float(gr.y << 16), g3 = __uint_as_float(gr.y & 0xffff0000u);
              const float y0 = ov[i].x * rstd * wv.x * sigmoid_fast(g0), y1 = ov[i].y * rstd * wv.y * sigmoid_fast(g1);
              const float y2 = ov[i].z * rstd * wv.z * sigmoid_fast(g2), y3 = ov[i].w * rstd * wv.w * sigmoid_fast(g3);
              if (sizeof(TO) == 4) {
                *reinterpret_cast<float4*>(tile + row * kD + col) = make_float4(y0, y1, y2, y3);
              } else {
                uint2 pk;
                pk.x = pack_bf16(y0, y1); pk.y = pack_bf16(y2, y3);
                *reinterpret_cast<uint2*>(stp + kStT + (row * kD + col) * 2) = pk;
              }
            }
          }
        }
        fence_proxy_async_smem();
        MDN_WARP_ARRIVE((cp & 1) ? b_go1 : b_go0);
      }
      if (c == nch) break;
      MDN_MARK(c, kEvPrescaled);

      const uint32_t ph = c & 1;
      const uint8_t* stg = smem + kOffStage + (c & 1) * kStageBytes;
      const float* cf = reinterpret_cast<const float*>(stg + kStCoef);
      const __nv_bfloat16* sV = reinterpret_cast<const __nv_bfloat16*>(stg + kStV);
      if constexpr (kTrain) {
        if (a.inject) {
          // operands of the second update: they depend on nothing the chain computes, so they are made here, while
          // MMA-1a runs.  Z, U are free in a state-only run; the previous chunk's MMA-3 (waited for in P) was their
          // last reader.
          const __nv_bfloat16* sG = reinterpret_cast<const __nv_bfloat16*>(stg + kStWh);
          float gv[kTok];
#pragma unroll
          for (int j = 0; j < kTok; ++j) gv[j] = __bfloat162float(sG[(r0 + j) * kD + d]);
#pragma unroll
          for (int which = 0; which < 2; ++which) {
            uint32_t oh[kPk], ol[kPk];
            const float* vecp = cf + (which ? kGM : kB) * C + r0;
#pragma unroll
            for (int j = 0; j < kTok; j += 4) {
              const float4 w4 = *reinterpret_cast<const float4*>(vecp + j);
              split_pack_bf16(-a.scale * w4.x * gv[j], -a.scale * w4.y * gv[j + 1], oh[j >> 1], ol[j >> 1]);
              split_pack_bf16(-a.scale * w4.z * gv[j + 2], -a.scale * w4.w * gv[j + 3], oh[(j >> 1) + 1], ol[(j >> 1) + 1]);
            }
            tmem_st_n<kPk>(tl + (which ? kColU : kColZ) + r0, oh);
            tmem_st_n<kPk>(tl + (which ? kColU : kColZ) + r0 + kPk, ol);
          }
          tmem_wait_st();
          tc_fence_before_sync();
          MDN_WARP_ARRIVE(b_v2);
        }
      }
      // ---------------- EPI-1: R^T = V^T - abar .* X + (alpha b^-) .* Y  -> bf16 hi, lo in X
      {
        // V and the coefficients do not depend on the MMA: fetch them while MMA-1a runs
        float vv[kTok];
#pragma unroll
        for (int j = 0; j < kTok; ++j) vv[j] = v_zero ? 0.f : __bfloat162float(sV[(r0 + j) * kD + d]);
        MDN_WAIT(b_m1, ph);
        __syncwarp();
        tc_fence_after_sync();
        MDN_MARK(c, kEvM1Seen);
        uint32_t hi[kPk], lo[kPk];
        {
          uint32_t x[kTok], y[kTok];
          tmem_ld_n<kTok>(tl + kColX + r0, x);
          tmem_ld_n<kTok>(tl + kColY + r0, y);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < kTok; j += 4) {
            const float4 ab = *reinterpret_cast<const float4*>(cf + kAbar * C + r0 + j);
            const float4 pb = *reinterpret_cast<const float4*>(cf + kAlphaBPrev * C + r0 + j);
            float e0, e1, e2, e3;
            if (qk_on) {
              // k' = k / |k|: X, Y are products with the raw k tile, so the norm scales the accumulators (vector 2
              // already carries the factor); the output correction q - d k turns Q S into Q S - d K S (same for M):
              // its K terms are X, Y themselves, handed to the tensor core as the start value of Z, U
              const float4 rk = *reinterpret_cast<const float4*>(cf + kRk * C + r0 + j);
              const float x0 = __uint_as_float(x[j + 0]), x1 = __uint_as_float(x[j + 1]);
              const float x2 = __uint_as_float(x[j + 2]), x3 = __uint_as_float(x[j + 3]);
              const float y0 = __uint_as_float(y[j + 0]), y1 = __uint_as_float(y[j + 1]);
              const float y2 = __uint_as_float(y[j + 2]), y3 = __uint_as_float(y[j + 3]);
              e0 = vv[j + 0] - (rk.x * ab.x) * x0 + pb.x * y0;
              e1 = vv[j + 1] - (rk.y * ab.y) * x1 + pb.y * y1;
              e2 = vv[j + 2] - (rk.z * ab.z) * x2 + pb.z * y2;
              e3 = vv[j + 3] - (rk.w * ab.w) * x3 + pb.w * y3;
              // -d K S, -d K M: MMA-1b will accumulate Q S, Q M onto them
              x[j + 0] = __float_as_uint(-dh * x0); x[j + 1] = __float_as_uint(-dh * x1);
              x[j + 2] = __float_as_uint(-dh * x2); x[j + 3] = __float_as_uint(-dh * x3);
              y[j + 0] = __float_as_uint(-dh * y0); y[j + 1] = __float_as_uint(-dh * y1);
              y[j + 2] = __float_as_uint(-dh * y2); y[j + 3] = __float_as_uint(-dh * y3);
            } else {
              e0 = vv[j + 0] - ab.x * __uint_as_float(x[j + 0]) + pb.x * __uint_as_float(y[j + 0]);
              e1 = vv[j + 1] - ab.y * __uint_as_float(x[j + 1]) + pb.y * __uint_as_float(y[j + 1]);
              e2 = vv[j + 2] - ab.z * __uint_as_float(x[j + 2]) + pb.z * __uint_as_float(y[j + 2]);
              e3 = vv[j + 3] - ab.w * __uint_as_float(x[j + 3]) + pb.w * __uint_as_float(y[j + 3]);
            }
            split_pack_bf16(e0, e1, hi[j >> 1], lo[j >> 1]);
            split_pack_bf16(e2, e3, hi[(j >> 1) + 1], lo[(j >> 1) + 1]);
          }
          if (qk_on && write_o) {   // own lanes only; MMA-3' of the previous chunk and this thread's read of U are done
            tmem_st_n<kTok>(tl + kColZ + r0, x);
            tmem_st_n<kTok>(tl + kColU + r0, y);
          }
        }
        // hi and lo both go into the columns this warp has just read (its own kTok columns of X): no other warp
        // touches them, so no group barrier is needed before overwriting
        tmem_st_n<kPk>(tl + kColX + r0, hi);
        tmem_st_n<kPk>(tl + kColX + r0 + kPk, lo);
        tmem_wait_st();
      }
      tc_fence_before_sync();
      MDN_WARP_ARRIVE(b_r);
      MDN_MARK(c, kEvRArrive);
      // ---------------- inter-chunk output terms: oi = scale (abar .* Q S - b .* Q M), under MMA-2; with the fused
      // q/k step Z, U arrive later (MMA-1b follows MMA-2) and already hold Q S - d K S, Q M - d K M: then this
      // step runs under MMA-3 instead
#define MDN_INTER_CHUNK_TERMS()                                                                              \
  {                                                                                                          \
    MDN_WAIT(b_mq, ph);                                                                                      \
    __syncwarp();                                                                                            \
    tc_fence_after_sync();                                                                                   \
    MDN_MARK(c, kEvMqSeen);                                                                                  \
    uint32_t z[kTok], u[kTok];                                                                               \
    tmem_ld_n<kTok>(tl + kColZ + r0, z);                                                                     \
    tmem_ld_n<kTok>(tl + kColU + r0, u);                                                                     \
    tmem_wait_ld();                                                                                          \
    tc_fence_before_sync();                                                                                  \
    MDN_MARK(c, kEvZqArrive);                                                                                \
    _Pragma("unroll") for (int j = 0; j < kTok; j += 4) {                                                    \
      const float4 ab = *reinterpret_cast<const float4*>(cf + kAbar * C + r0 + j);                           \
      const float4 bb = *reinterpret_cast<const float4*>(cf + kB * C + r0 + j);                              \
      float4 sc = make_float4(a.scale, a.scale, a.scale, a.scale);                                           \
      if (qk_on) { /* q' = (q - d k) / |q - d k| */                                                          \
        const float4 rq = *reinterpret_cast<const float4*>(cf + kRq * C + r0 + j);                           \
        sc.x *= rq.x; sc.y *= rq.y; sc.z *= rq.z; sc.w *= rq.w;                                              \
      }                                                                                                      \
      oi[j + 0] = sc.x * (ab.x * __uint_as_float(z[j + 0]) - bb.x * __uint_as_float(u[j + 0]));              \
      oi[j + 1] = sc.y * (ab.y * __uint_as_float(z[j + 1]) - bb.y * __uint_as_float(u[j + 1]));              \
      oi[j + 2] = sc.z * (ab.z * __uint_as_float(z[j + 2]) - bb.z * __uint_as_float(u[j + 2]));              \
      oi[j + 3] = sc.w * (ab.w * __uint_as_float(z[j + 3]) - bb.w * __uint_as_float(u[j + 3]));              \
    }                                                                                                        \
  }
      if constexpr (kLayer) {
        if (write_o && !qk_on) MDN_INTER_CHUNK_TERMS();
      }
      // ---------------- EPI-2: V~ -> (gamma_C eta) V~, ((mubar_C/mubar) eta) V~ [part a], V~ [part b]; bf16 hi, lo
      MDN_WAIT(b_m2, ph);
      __syncwarp();
      tc_fence_after_sync();
      MDN_MARK(c, kEvM2Seen);
      {
        uint32_t vt[kTok];
        tmem_ld_n<kTok>(tl + kColY + r0, vt);
        tmem_wait_ld();
        {
          uint32_t sh[kPk], sl[kPk];
#pragma unroll
          for (int j = 0; j < kTok; j += 4) {
            const float4 gs = *reinterpret_cast<const float4*>(cf + kGS * C + r0 + j);
            split_pack_bf16(gs.x * __uint_as_float(vt[j]), gs.y * __uint_as_float(vt[j + 1]), sh[j >> 1], sl[j >> 1]);
            split_pack_bf16(gs.z * __uint_as_float(vt[j + 2]), gs.w * __uint_as_float(vt[j + 3]), sh[(j >> 1) + 1],
                            sl[(j >> 1) + 1]);
          }
          tmem_st_n<kPk>(tl + kColX + r0, sh);          // X is free: MMA-2 has consumed R
          tmem_st_n<kPk>(tl + kColX + r0 + kPk, sl);
        }
        {
          uint32_t mh[kPk], mlo[kPk];
#pragma unroll
          for (int j = 0; j < kTok; j += 4) {
            const float4 gm = *reinterpret_cast<const float4*>(cf + kGM * C + r0 + j);
            split_pack_bf16(gm.x * __uint_as_float(vt[j]), gm.y * __uint_as_float(vt[j + 1]), mh[j >> 1], mlo[j >> 1]);
            split_pack_bf16(gm.z * __uint_as_float(vt[j + 2]), gm.w * __uint_as_float(vt[j + 3]), mh[(j >> 1) + 1],
                            mlo[(j >> 1) + 1]);
          }
          // over this warp's own columns of Y (the V~ it has loaded above)
          tmem_st_n<kPk>(tl + kColY + r0, mh);
          tmem_st_n<kPk>(tl + kColY + r0 + kPk, mlo);
        }
        tmem_wait_st();          // also covers the pre-scaled masters stored in P part 2
        tc_fence_before_sync();
        MDN_WARP_ARRIVE(b_v1);
        MDN_MARK(c, kEvVArrive);
        if constexpr (!kLayer) {
          if (write_o) {
            MDN_WAIT(b_mq, ph);
            __syncwarp();
            tc_fence_after_sync();
            MDN_MARK(c, kEvMqSeen);
            uint32_t z[kTok], u[kTok];
            tmem_ld_n<kTok>(tl + kColZ + r0, z);
            tmem_ld_n<kTok>(tl + kColU + r0, u);
            tmem_wait_ld();
            tc_fence_before_sync();
            MDN_MARK(c, kEvZqArrive);
#pragma unroll
            for (int j = 0; j < kTok; j += 4) {
              const float4 ab = *reinterpret_cast<const float4*>(cf + kAbar * C + r0 + j);
              const float4 bb = *reinterpret_cast<const float4*>(cf + kB * C + r0 + j);
              oi[j + 0] = a.scale * (ab.x * __uint_as_float(z[j + 0]) - bb.x * __uint_as_float(u[j + 0]));
              oi[j + 1] = a.scale * (ab.y * __uint_as_float(z[j + 1]) - bb.y * __uint_as_float(u[j + 1]));
              oi[j + 2] = a.scale * (ab.z * __uint_as_float(z[j + 2]) - bb.z * __uint_as_float(u[j + 2]));
              oi[j + 3] = a.scale * (ab.w * __uint_as_float(z[j + 3]) - bb.w * __uint_as_float(u[j + 3]));
            }
          }
        } else {
          if (write_o && qk_on) MDN_INTER_CHUNK_TERMS();
        }
        // part b (under MMA-3): V~ itself for the intra-chunk output, into Z
        if (write_o) {
          uint32_t vh[kPk], vl[kPk];
#pragma unroll
          for (int j = 0; j < kTok; j += 2) split_pack_bf16(__uint_as_float(vt[j]), __uint_as_float(vt[j + 1]), vh[j >> 1], vl[j >> 1]);
          tmem_st_n<kPk>(tl + kColZ + r0, vh);          // own columns of Z: this thread has read its Q S entries
          tmem_st_n<kPk>(tl + kColZ + r0 + kPk, vl);
          tmem_wait_st();
          tc_fence_before_sync();
          MDN_WARP_ARRIVE(b_v2);
        }
        MDN_MARK(c, kEvV2Arrive);
        if constexpr (kTrain) {   // off the chain's critical path: MMA-3 is running
          const int slot_c = sq.slot0 + c;
          if (a.vt_dump != nullptr) {
            const int live = min(C, sq.len - c * C) - r0;   // this thread's tokens inside the chunk
            float* dst = a.vt_dump + (((size_t)slot_c * C + r0) * H + h) * kD + d;
            const size_t stride = (size_t)H * kD;
            if (live >= kTok) {   // the usual case: no per-store predicate
#pragma unroll
              for (int j = 0; j < kTok; ++j, dst += stride) *dst = __uint_as_float(vt[j]);
            } else {
#pragma unroll
              for (int j = 0; j < kTok; ++j, dst += stride)
                if (j < live) *dst = __uint_as_float(vt[j]);
            }
          }
        }
      }
    }
  }
#undef MDN_INTER_CHUNK_TERMS
#undef MDN_MMA_1B
#undef MDN_WARP_ARRIVE
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

cudaError_t launch_intra_tensor(const Plan& pl, const void* q, const void* k, const GateArgs& gates, int* launches) {
  return launch_intra_mma(pl, q, k, gates, launches);
}

bool chain_uses_tf32_kernel(const Plan& pl) {
  const bool train = pl.chain_dump != nullptr || pl.chain_state_only || pl.chain_end_scalars_in_rk ||
                     pl.chain_vt_dump != nullptr || pl.chain_inject || pl.chain_mirror_geom != nullptr;
  return pl.p.path == MDN_PATH_TENSOR && !train;
}

cudaError_t launch_chain_tensor(const Plan& pl, const void* q, const void* k, const void* v, const float* S0,
                                const float* M0, void* o, float* Sf, float* Mf, int* launches) {
  if (pl.w_f32) return launch_chain_tf32(pl, q, k, v, S0, M0, o, Sf, Mf, launches);
  const mdn_params& p = pl.p;
  const uint64_t tokens = (uint64_t)p.B * p.T;
  // mirrored run: q, k, o are another problem's tensors (its geometry in chain_mirror_geom)
  const uint64_t tokens_qko = pl.chain_mirror_geom ? (uint64_t)pl.chain_mirror_geom->B * pl.chain_mirror_geom->T : tokens;
  const uint64_t mats = (uint64_t)pl.geom.num_slots * p.H;
  CUtensorMap mq, mk, mv, mt, mw, mo;
  const uint64_t row = (uint64_t)p.H * kD;
  if (!encode_tma_2d_bf16(&mq, TmaMap2D{q, row, tokens_qko, row * 2, 64, 64, true}) ||
      !encode_tma_2d_bf16(&mk, TmaMap2D{k, row, tokens_qko, row * 2, 64, 64, true}) ||
      !encode_tma_2d_bf16(&mv, TmaMap2D{v, row, tokens, row * 2, 128, 64, false}) ||
      !encode_tma_2d_bf16(&mt, TmaMap2D{pl.chain_mirror_T ? pl.chain_mirror_T : pl.ws + pl.lay.off_T, 64, mats * C, 128, 64,
                                        64, true}) ||
      !encode_tma_2d_bf16(&mw, TmaMap2D{pl.ws + pl.lay.off_W, 64, 2 * mats * C, 128, 64, 64, true}))
    return cudaErrorInvalidValue;
  const bool o_bf16 = p.o_dtype == MDN_BF16;
  if (!encode_tma_2d(&mo, TmaMap2D{o, row, tokens_qko, row * (o_bf16 ? 2u : 4u), 128, 64, false}, !o_bf16))
    return cudaErrorInvalidValue;
  ChainArgs a;
  a.qk_on = pl.qk.on; a.qk_d = pl.qk.d;
  a.post_on = pl.post.on; a.post_w = pl.post.w; a.post_g = pl.post.g; a.post_eps = pl.post.eps;
  a.g = pl.geom;
  a.coef = reinterpret_cast<const float*>(pl.ws + pl.lay.off_coef);
  a.S0 = S0; a.M0 = M0; a.o = o; a.Sf = Sf; a.Mf = Mf;
  a.status = reinterpret_cast<int32_t*>(pl.ws + pl.lay.off_status);
  a.scale = p.scale;
  a.w_lo_row_offset = (uint32_t)(mats * C);
  a.drop_lo = 0u;
  a.timeline = nullptr;
#ifdef MDN_DEBUG   // debug builds only (-DMDN_DEBUG): the product library reads nothing from the environment
  const char* drop = getenv("MDN_DEBUG_DROP_LO");
  a.drop_lo = drop ? (uint32_t)atoi(drop) : 0u;
  const char* tl = getenv("MDN_DEBUG_TIMELINE");   // device address of an int64 buffer, [chunks][32]
  a.timeline = tl ? reinterpret_cast<long long*>(strtoull(tl, nullptr, 0)) : nullptr;
#endif
  a.dump = pl.chain_dump; a.state_only = pl.chain_state_only; a.end_scalars_in_rk = pl.chain_end_scalars_in_rk;
  a.vt_dump = pl.chain_vt_dump; a.inject = pl.chain_inject;
  a.mirror = pl.chain_mirror_geom != nullptr;
  if (a.mirror) a.mirror_g = *pl.chain_mirror_geom; else a.mirror_g = pl.geom;
  a.seg_G = 0; a.seg_phase = 0;
  a.seg_E = a.seg_Psi = a.seg_PhiS = a.seg_PhiM = nullptr;
  const unsigned chains = (unsigned)pl.geom.num_seqs * p.H;
  const bool layer = a.qk_on || a.post_on;
  auto launch_as = [&](auto kern, unsigned grid) -> cudaError_t {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    const unsigned threads = layer ? Roles<token_groups(true)>::kThreads : Roles<token_groups(false)>::kThreads;
    e = launch_pdl(kern, dim3(grid), dim3(threads), kSmemBytes, pl.stream, a, mq, mk, mv, mt, mw, mo);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e == cudaSuccess) ++*launches;
    return e;
  };
  auto launch = [&](unsigned grid) -> cudaError_t {
    const bool train = a.dump != nullptr || a.state_only || a.end_scalars_in_rk || a.vt_dump != nullptr || a.inject;
    if ((a.inject && !a.state_only) || (a.mirror && !a.inject)) return cudaErrorInvalidValue;
    if (train) {   // plain forward with the training options (no layer operations there)
      if (layer) return cudaErrorInvalidValue;
      return p.o_dtype == MDN_BF16 ? launch_as(chain_tensor_kernel<__nv_bfloat16, false, true>, grid)
                                   : launch_as(chain_tensor_kernel<float, false, true>, grid);
    }
    if (p.o_dtype == MDN_BF16)
      return layer ? launch_as(chain_tensor_kernel<__nv_bfloat16, true>, grid)
                   : launch_as(chain_tensor_kernel<__nv_bfloat16, false>, grid);
    return layer ? launch_as(chain_tensor_kernel<float, true>, grid) : launch_as(chain_tensor_kernel<float, false>, grid);
  };
  const int G = pl.lay.segments;
  if (G <= 1) return launch(chains);

  // ---- parallel inter-chunk scan: Psi / Phi of the middle segments, serial combine, then all segments for real
  constexpr size_t kMat = (size_t)kD * kD;
  float* seg = reinterpret_cast<float*>(pl.ws + pl.lay.off_seg);
  a.seg_G = G;
  a.seg_E = seg;
  a.seg_Psi = a.seg_E + (size_t)chains * (G - 1) * 2 * kMat;
  a.seg_PhiS = a.seg_Psi + (size_t)chains * (G - 2) * 2 * kMat;
  a.seg_PhiM = a.seg_PhiS + (size_t)chains * (G - 2) * 2 * kMat;
  a.seg_phase = 1;
  cudaError_t e = launch(chains * (1 + 3 * (G - 2)));
  if (e != cudaSuccess) return e;
  e = launch_seg_combine(pl, G, a.seg_E, a.seg_Psi, a.seg_PhiS, a.seg_PhiM, launches);
  if (e != cudaSuccess) return e;
  a.seg_phase = 3;
  return launch(chains * (G - 1));
}

size_t seg_scratch_bytes(const mdn_params& p, int segments) {
  if (segments <= 1) return 0;
  const size_t chains = (size_t)p.B * p.H, mat = (size_t)p.dk * p.dv * sizeof(float);
  return chains * ((size_t)(segments - 1) * 2 + (size_t)(segments - 2) * 6) * mat;
}

// Segments per sequence for the parallel scan, from a wave-count model of the two chain launches (one CTA per
// SM, every CTA walks ceil(nch / G) chunks; a middle segment costs three extra runs) plus about four chunk-times
// per step of the serial combine.  The scan is used only where the model predicts at most 0.7 of the serial
// chain's time and every segment keeps at least 8 chunks; otherwise 1 (off).
int choose_segments(const mdn_params& p) {
  if (!tensor_path_supported(p) || p.num_seqs > 0) return 1;
  if (p.segments == 1) return 1;
  if (p.segments >= 3) return p.segments;
  constexpr long kSMs = 148;
  const long nch = (p.T + C - 1) / C, chains = (long)p.B * p.H;
  auto waves = [&](long ctas) { return (ctas + kSMs - 1) / kSMs; };
  const long serial = waves(chains) * nch;
  long best_cost = serial;
  int best = 1;
  for (int g = 3; g <= 32 && nch / g >= 8; ++g) {
    const long per = (nch + g - 1) / g;
    // (a state-only run takes about 0.9 of a full one: it skips the output terms, which mostly hide anyway)
    const long cost = (waves(chains * (1 + 3 * (g - 2))) * 9 * per) / 10 + waves(chains * (g - 1)) * per + 4 * (g - 2);
    if (cost * 10 <= serial * 7 && cost < best_cost) { best_cost = cost; best = g; }
  }
  return best;
}

}  // namespace mdn
