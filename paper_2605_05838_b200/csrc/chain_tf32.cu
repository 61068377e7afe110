// a3 + a4 of the plain forward on the 5th-generation tensor cores (tcgen05, sm_100a), second design: one CTA walks
// the chunks of one (sequence, head) in order; bf16 q/k/v, dk = dv = 128, chunk 64.  (The first design,
// chain_tensor.cu, stays for the training / backward runs.)  Template flag kLayer: the layer's element-wise operations
// of Section 3.3 inside this kernel (q/k norm through the coefficient vectors and the converter warps, RMSNorm and
// sigmoid gate in the output step); kLayer = false compiles them out.
//
// Everything is kept TRANSPOSED: the value dimension (128) is the MMA M dimension and fills the 128 tensor-memory
// lanes, tokens are N (or K).  What is different here:
//
//  * No per-chunk pass over the state.  The fp32 masters S^T, M^T in tensor memory are read by the tensor core as
//    they are, as the A operand of kind::tf32 products (fp32 storage read as tf32), against fp32 copies of the K and
//    Q tiles that two converter warps write one chunk ahead.  No bf16 copy of the state is ever made.
//  * Lazy scaling of the state.  The chunk hand-over  S' = abar_C S - b_C M + dS,  M' = mubar_C M - dM  (state equations
//    below Eq. 12) is a 2 x 2 upper-triangular scalar map D_c on the pair [S; M].  Instead of rescaling the masters
//    every chunk, the masters hold [Sh; Mh] with  [S; M] = G [Sh; Mh],  G = [[g11, g12], [0, g22]]  kept as three
//    scalars:  G' = D_c G  and the update is added in hat coordinates,  [Sh'; Mh'] = [Sh; Mh] + G'^-1 [dS; -dM].
//    Every use of the state then only changes per-token coefficients (all products are linear in the state):
//        K S = g11 (K Sh) + g12 (K Mh),  K M = g22 (K Mh)        ->  R = V - cX .* X + cY .* Y
//        Q S, Q M likewise                                       ->  o_inter = cZ .* Z + cU .* U
//        dS / g11' + (g12' / (g11' g22')) dM,  dM / g22'         ->  per-token weights wS, wM of V~ in the updates
//    with cX = abar g11, cY = (alpha b^-) g22 - abar g12, cZ = scale abar g11, cU = scale (abar g12 - b g22),
//    wS = (gS + (g12'/g22') gM) / g11', wM = gM / g22' (gS = gamma_C eta, gM = (mubar_C/mubar) eta).  The producer
//    warp runs the scalar recurrence of G and writes these six vectors per chunk.  When G' would leave a safe range
//    (g11' or g22' below 2^-64, or |g12'| above g22': fast-decaying gates, mu = 0 tokens, S decaying slower than M) the chunk is "eager":
//    the epilogue warps rescale the masters once by G' (the first design's pre-scaling, with G folded in) and G
//    returns to the identity.  The result is the same recurrence either way; only rounding differs.
//  * One product gives the state terms of the correction AND of the output: B = the K tile stacked on the Q tile
//    (128 rows), so [X | Z] = Sh [K; Q]^T and [Y | U] = Mh [K; Q]^T are two N = 128 products (a product costs the
//    same up to N = 128: measured 54 / 54 / 64 / 128 cycles at N = 32 / 64 / 128 / 256 with A in tensor memory).
//  * The intra-chunk output product reads V~ straight from the accumulator of V~ = T R (kind::tf32 against an fp32 W
//    tile the intra-chunk kernel writes), accumulating onto the inter-chunk terms the epilogue has left there: no
//    operand conversion for it, and it runs under the epilogue's work on the state update.
//
// Per chunk:  MMA-1 [X|Z], [Y|U]  ->  EPI-1 R^T (bf16 hi + lo)  ->  MMA-2 Y = R^T T^T  ->  EPI-2 wS .* V~, wM .* V~ (bf16 hi + lo)
//             ->  MMA-3 Sh^T += (wS V~)^T K, Mh^T -= (wM V~)^T K (K tile read MN-major)  ->  next chunk's MMA-1.
// Off that path: o_inter into U (under MMA-2), MMA-3' U += V~^T W^T (under EPI-2), output tile + TMA store (under MMA-3).
//
// Warps: MMA issuer (one elected lane, tensor-memory owner), TMA producer (also issues the output stores), 8 epilogue
// warps (lane quarter x token half), 2 converter warps.  All hand-offs are mbarriers with bounded waits.
#include <cstdlib>
#include <cstring>

#include "mdn_common.cuh"
#include "tc_utils.cuh"

namespace mdn {
namespace {

using namespace tc;

constexpr int kD = 128;
constexpr int kEpiWarps = 8, kTok = 32, kPk = 16;
// Warp roles: warp 0 MMA issuer, warp 1 TMA producer (it also runs the scalar recurrence of G and writes each chunk's
// coefficient vectors), warps 2..9 epilogue (lane quarter = warp % 4, as tensor memory demands), warps 10, 11 converters
// (fp32 copies of the next chunk's K and Q tiles; they sit on the two schedulers that hold neither the MMA nor the
// TMA warp).  Three warps per scheduler: 168 registers each.  Measured alternatives: the conversion inside the
// epilogue warps (behind the hand-over of the state-update operands) put its 1.5 k cycles of shared-memory traffic
// on the chain's critical path; four converter warps cost the epilogue its registers.
constexpr int kWarpMma = 0, kWarpTma = 1, kWarpEpi = 2, kWarpCvt = 10, kCvtWarps = 2;
constexpr int kThreads = (kEpiWarps + 2 + kCvtWarps) * 32;
constexpr int kEpiThreads = kEpiWarps * 32, kCvtThreads = kCvtWarps * 32;

// shared memory (offsets from a 1024-byte aligned base)
// The K tile is loaded twice: early into a buffer of its own (with the Q tile), where it is free again as soon as
// its fp32 copy is made, so that the next chunk's arrives a whole chunk ahead; and into the stage, where MMA-3 reads
// it (MN-major) at the end of the chunk.  The second load hits the L2.
constexpr uint32_t kOffKQ32 = 0;        // fp32 [K; Q]: four dk quarters x [128 rows (K tokens, then Q tokens) x 128 B], swizzled
constexpr uint32_t kOffCvt = 65536;     // bf16 K and Q tiles waiting for their fp32 copies: [K 16 KB | Q 16 KB], single buffer
constexpr uint32_t kOffStage = 98304;
constexpr uint32_t kStK = 0, kStV = 16384, kStT = 32768, kStW = 40960, kStCoef = 57344;
constexpr uint32_t kCoefBytes = kChainCoefs * C * sizeof(float);
constexpr uint32_t kStageBytes = 59392;
constexpr uint32_t kTxBytes = 2 * 16384 + 8192 + 16384 + kCoefBytes;
constexpr uint32_t kTxW = 16384, kTxV = 16384;   // bytes of the W tile, of the V tile
constexpr uint32_t kStOut = kStV;       // the finished output tile: V area (bf16), V + T + half of W (fp32); all dead by then
constexpr uint32_t kOffAdj = kOffStage + 2 * kStageBytes;
constexpr uint32_t kAdjBytes = 2048;
constexpr uint32_t kSmemBytes = kOffAdj + 2 * kAdjBytes + 1024;
static_assert(kStCoef + kCoefBytes <= kStageBytes && kSmemBytes <= 232448, "shared-memory layout");

// per-chunk block the producer warp publishes (float indices)
enum Adj : int { kCx = 0, kCy = 64, kCz = 128, kCu = 192, kWs = 256, kWm = 320, kN11 = 384, kN12, kN22, kLazy };
constexpr float kLazyMin = 5.421010862427522e-20f;   // 2^-64: smallest g11', g22' a lazy chunk may leave
constexpr float kLazyMix = 1.f;                      // largest |g12'| / g22' (beyond it the two hat terms of S cancel too much)

// tensor memory columns (512 x 128 lanes x 32 bit)
constexpr uint32_t kColS = 0, kColM = 128, kColX = 256, kColZ = 320, kColY = 384, kColU = 448;

struct Bars {
  uint64_t full[2];   // TMA loads of a stage landed                                      (1 + tx bytes)
  uint64_t go[2];     // a stage's output tile is staged and nothing reads the stage any more (256)
  uint64_t cfull;     // bf16 K, Q of a chunk landed in their buffer                         (1 + tx bytes)
  uint64_t cfree;     // ... and read: the next chunk's may be loaded                       (64)
  uint64_t kq;        // fp32 [K; Q] of a chunk written                                   (64)
  uint64_t adj[2];    // a chunk's coefficient block written                              (32)
  uint64_t fin;       // G after the last chunk written                                   (32)
  uint64_t init;      // masters of chunk 0 stored                                        (256)
  uint64_t mx;        // first half of MMA-1 done: X, Z                                    (commit)
  uint64_t m1;        // MMA-1 done: X, Z, Y, U                                            (commit)
  uint64_t r;         // EPI-1 done: R^T hi/lo in X                                        (256)
  uint64_t m2;        // MMA-2 done                                                       (commit)
  uint64_t oi;        // inter-chunk output terms stored in U                             (256)
  uint64_t v1a;       // EPI-2, first part: wS V~ in X (eager chunks: Sh rescaled)         (256)
  uint64_t v1b;       // EPI-2, second part: wM V~ in Y (eager chunks: Mh rescaled)        (256)
  uint64_t m3s;       // MMA-3, Sh part done                                              (commit)
  uint64_t m3;        // MMA-3 done                                                       (commit)
  uint64_t mo;        // MMA-3' done                                                      (commit)
  uint64_t zu;        // U (the chunk's output) has been read                              (256)
  uint64_t pn;        // fused output step: the fp32 tile is staged / has been read            (256)
};

struct Args {
  ChunkGeom g;
  const float* coef;
  const float* S0;
  const float* M0;
  void* o;
  float* Sf;
  float* Mf;
  int32_t* status;
  float scale;
  // parallel inter-chunk scan (seg_G = 0: off, one CTA walks all chunks of its chain)
  int seg_G;
  int seg_phase;
  float* seg_E;
  float* seg_Psi;
  float* seg_PhiS;
  float* seg_PhiM;
  long long* timeline;   // debug builds: CTA 0 writes clock64() at [chunk * 32 + event]
  // layer operations (Section 3.3), kLayer instantiation only
  int qk_on;             // q <- L2Norm(q - d k), k <- L2Norm(k): 1/|k|, 1/|q - d k| arrive as coefficient vectors 6, 7
  const float* qk_d;     // [H] or NULL
  int post_on;           // o <- sigmoid(g) * RMSNorm(o) * w in the output step
  const float* post_w;   // [dv] or NULL
  const void* post_g;    // [B,T,H,dv] bf16
  float post_eps;
};

__device__ __forceinline__ float sigmoid_fast(float x) {
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(0.5f * x));
  return fmaf(0.5f, t, 0.5f);
}

enum Ev : int { kEvMma1 = 0, kEvM1Seen, kEvRArrive, kEvOiArrive, kEvM2Seen, kEvV1Arrive, kEvOutDone, kEvM3Seen, kEvRSeen,
                kEvV1Seen, kEvCvtStart, kEvCvtDone, kEvTmaIssued, kEvStoresDone, kEvM2Own, kEvEager,
                kEvXzIssued, kEvYuIssued, kEvM2Issued, kEvSIssued, kEvMIssued, kEvV1bSeen, kEvV1bArrive, kEvZuArrive, kEvMoIssued, kEvM3sOwn, kEvKqSeen, kEvLoopTop, kEvRArrive2, kEvV1Arrive2 };

template <typename TO> __device__ __forceinline__ void stage_o(uint8_t* tile, int r, int d, float x);
template <> __device__ __forceinline__ void stage_o<float>(uint8_t* tile, int r, int d, float x) {
  reinterpret_cast<float*>(tile)[r * kD + d] = x;
}
template <> __device__ __forceinline__ void stage_o<__nv_bfloat16>(uint8_t* tile, int r, int d, float x) {
  reinterpret_cast<__nv_bfloat16*>(tile)[r * kD + d] = __float2bfloat16_rn(x);
}

template <typename TO, bool kLayer>
__global__ void __launch_bounds__(kThreads, 1) chain_tf32_kernel(const Args a, const __grid_constant__ CUtensorMap map_q,
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
  __shared__ float g_final[4];   // G after the last chunk: what the final states are read through
  __shared__ __align__(16) float w_sm[kLayer ? kD : 4];   // RMSNorm weight of the fused output step

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

  const uint32_t s_base = smem_u32(smem);
  const uint32_t b_full0 = smem_u32(&bars.full[0]), b_full1 = smem_u32(&bars.full[1]);
  const uint32_t b_go0 = smem_u32(&bars.go[0]), b_go1 = smem_u32(&bars.go[1]);
  const uint32_t b_kq = smem_u32(&bars.kq), b_adj0 = smem_u32(&bars.adj[0]), b_adj1 = smem_u32(&bars.adj[1]);
  const uint32_t b_init = smem_u32(&bars.init), b_m1 = smem_u32(&bars.m1), b_r = smem_u32(&bars.r);
  const uint32_t b_m2 = smem_u32(&bars.m2), b_oi = smem_u32(&bars.oi), b_v1a = smem_u32(&bars.v1a);
  const uint32_t b_v1b = smem_u32(&bars.v1b), b_mx = smem_u32(&bars.mx), b_m3s = smem_u32(&bars.m3s);
  const uint32_t b_m3 = smem_u32(&bars.m3), b_mo = smem_u32(&bars.mo), b_zu = smem_u32(&bars.zu);
  const uint32_t b_fin = smem_u32(&bars.fin), b_cfull = smem_u32(&bars.cfull), b_cfree = smem_u32(&bars.cfree);
  const uint32_t b_pn = smem_u32(&bars.pn);
  // kLayer = false compiles the layer operations out
  const bool qk_on = kLayer && a.qk_on;
  const float qk_dh = (qk_on && a.qk_d) ? __ldg(a.qk_d + h) : 0.f;

  if (tid == 0) {
    abort_flag = 0;
    mbar_init(b_full0, 1); mbar_init(b_full1, 1);
    mbar_init(b_go0, kEpiThreads); mbar_init(b_go1, kEpiThreads);
    mbar_init(b_kq, kCvtThreads); mbar_init(b_adj0, 32); mbar_init(b_adj1, 32);
    mbar_init(b_fin, 32); mbar_init(b_cfull, 1); mbar_init(b_cfree, kCvtThreads);
    mbar_init(b_init, kEpiThreads); mbar_init(b_r, kEpiThreads); mbar_init(b_oi, kEpiThreads);
    mbar_init(b_v1a, kEpiThreads); mbar_init(b_v1b, kEpiThreads); mbar_init(b_zu, kEpiThreads);
    if constexpr (kLayer) mbar_init(b_pn, kEpiThreads);
    mbar_init(b_m1, 1); mbar_init(b_m2, 1); mbar_init(b_m3, 1); mbar_init(b_mo, 1); mbar_init(b_mx, 1); mbar_init(b_m3s, 1);
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
  // waits on the chain's critical path poll without suspending
#define MDN_SPIN(bar, par)                         \
  if (!mbar_wait_spin((bar), (par), abortp)) {     \
    ok = false;                                    \
    break;                                         \
  }
#ifdef MDN_DEBUG
  // Stamps go to shared memory (a global store per stamp slows the stamping thread by hundreds of cycles) for the
  // chunks kTlFirst .. kTlFirst + 7 and are copied out when the kernel ends.
  long long* const tline = (blockIdx.x == 0) ? a.timeline : nullptr;
  constexpr int kTlFirst = 16;
  __shared__ long long tl_sm[8][32];
#define MDN_MARK(c, ev) \
  if (tline != nullptr && lane == 0 && (c) >= kTlFirst && (c) < kTlFirst + 8 && \
      (warp < kWarpEpi || warp == kWarpEpi + 2 || warp >= kWarpCvt)) tl_sm[(c) - kTlFirst][(ev)] = clock64();
#define MDN_MARK2(c, ev) \
  if (tline != nullptr && lane == 0 && (c) >= kTlFirst && (c) < kTlFirst + 8 && warp == 7) tl_sm[(c) - kTlFirst][(ev)] = clock64();
#else
#define MDN_MARK(c, ev)
#define MDN_MARK2(c, ev)
#endif

#ifdef MDN_DEBUG
  if (tline != nullptr && tid == 0) {   // clock rate of this run: cycle and nanosecond stamps at both ends
    unsigned long long ns;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns));
    tline[30] = clock64(); tline[31] = (long long)ns;
  }
#endif
  if (warp == kWarpTma) {
    // ================================================================== TMA producer + output stores + coefficients
    // Stage s = c & 1 serves chunk c, then (as the staged output tile) is written out and refilled for chunk c + 2.
    // The whole warp walks the loop; lane 0 issues the copies; every lane writes the coefficients of two tokens.
    {
      int issued = 0, issued_kq = 0;
      float g11 = 1.f, g12 = 0.f, g22 = 1.f;
      for (int c = 0; c < nch + 2; ++c) {
        const int s = c & 1;
        const uint32_t st = s_base + kOffStage + s * kStageBytes;
        if (c < nch) {
          // the chunk's K and Q tiles for the converters first: their buffer is free long before the stage is, and
          // with the fused q/k norm the converters need the head start
          if (c > 0) MDN_WAIT(b_cfree, (c - 1) & 1);   // the previous chunk's bf16 K, Q have been read
          if (lane == 0) {
            const int tok0 = sq.tok0 + c * C;
            mbar_arrive_expect_tx(b_cfull, write_o ? 32768u : 16384u);
            tma_load_2d(s_base + kOffCvt, &map_k, h * kD, tok0, b_cfull);
            tma_load_2d(s_base + kOffCvt + 8192, &map_k, h * kD + 64, tok0, b_cfull);
            if (write_o) {
              tma_load_2d(s_base + kOffCvt + 16384, &map_q, h * kD, tok0, b_cfull);
              tma_load_2d(s_base + kOffCvt + 24576, &map_q, h * kD + 64, tok0, b_cfull);
            }
          }
          __syncwarp();
          issued_kq = c + 1;
        }
        if (c >= 2) {
          const int co = c - 2;
          MDN_WAIT(s ? b_go1 : b_go0, (co >> 1) & 1);
          if (lane == 0) {
            const int n = min(C, sq.len - co * C);
            const int tok0 = sq.tok0 + co * C;
            const uint32_t src = st + kStOut;
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
          }
          __syncwarp();
          MDN_MARK(co, kEvStoresDone);
        }
        if (c < nch) {
          const uint32_t fb = s ? b_full1 : b_full0;
          if (lane == 0) {
            const int tok0 = sq.tok0 + c * C;
            const int mat = (sq.slot0 + c) * H + h;
            mbar_arrive_expect_tx(fb, kTxBytes - (write_o ? 0u : kTxW) - (v_zero ? kTxV : 0u));
            bulk_load(st + kStCoef, a.coef + (size_t)mat * MDN_NUM_COEF * C, kCoefBytes, fb);
            if (!v_zero) tma_load_2d(st + kStV, &map_v, h * kD, tok0, fb);
            tma_load_2d(st + kStT, &map_t, 0, mat * C, fb);
            if (write_o) {
              tma_load_2d(st + kStW, &map_w, 0, mat * C, fb);
              tma_load_2d(st + kStW + 8192, &map_w, 32, mat * C, fb);
            }
            tma_load_2d(st + kStK, &map_k, h * kD, tok0, fb);          // for MMA-3 at the end of the chunk (L2 hit)
            tma_load_2d(st + kStK + 8192, &map_k, h * kD + 64, tok0, fb);
          }
          __syncwarp();
          MDN_MARK(c, kEvTmaIssued);
          issued = c + 1;
          // ---- the scalar recurrence of G and the chunk's six coefficient vectors (two tokens per lane), as soon as the
          // chunk's coefficient vectors have landed: about a chunk before the epilogue needs them
          MDN_WAIT(fb, (c >> 1) & 1);
          float* aj = reinterpret_cast<float*>(smem + kOffAdj + s * kAdjBytes);
          const float* cf = reinterpret_cast<const float*>(smem + kOffStage + s * kStageBytes + kStCoef);
          const float aC = cf[kAbar * C + C - 1], bC = cf[kB * C + C - 1], mC = cf[kMubar * C + C - 1];
          const float n11 = __fmul_rn(aC, g11), n12 = __fsub_rn(__fmul_rn(aC, g12), __fmul_rn(bC, g22)), n22 = __fmul_rn(mC, g22);
          const bool lazy = n11 >= kLazyMin && n22 >= kLazyMin && fabsf(n12) <= kLazyMix * n22;
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int t = 2 * lane + e;
            const float ab = cf[kAbar * C + t], bb = cf[kB * C + t], pp = cf[kAlphaBPrev * C + t];
            const float gs = cf[kGS * C + t], gm = cf[kGM * C + t];
            // fused q/k norm: k^ = k / |k| scales the rows of K S, K M (vectors 2, 3, 4 carry that factor already),
            // q^ = (q - d k) / |q - d k| those of the output terms (the converter warps subtract d k from the Q tile)
            float cx, cy, cz, cu;
            if constexpr (kLayer) {
              const float rk = cf[kRk * C + t], sq_ = a.scale * cf[kRq * C + t];
              cx = ab * rk * g11; cy = pp * g22 - ab * rk * g12;
              cz = sq_ * (ab * g11); cu = sq_ * (ab * g12 - bb * g22);
            } else {
              cx = ab * g11; cy = pp * g22 - ab * g12;
              cz = a.scale * cx; cu = a.scale * (ab * g12 - bb * g22);
            }
            aj[kCx + t] = -cx;     // stored negated: the epilogue's first step is one packed FMA per token pair
            aj[kCy + t] = cy;
            aj[kCz + t] = cz;
            aj[kCu + t] = cu;
            aj[kWs + t] = lazy ? (gs + (n12 / n22) * gm) / n11 : gs;
            aj[kWm + t] = lazy ? gm / n22 : gm;
          }
          if (lane == 0) { aj[kN11] = n11; aj[kN12] = n12; aj[kN22] = n22; aj[kLazy] = lazy ? 1.f : 0.f; }
          if (lazy) { g11 = n11; g12 = n12; g22 = n22; } else { g11 = 1.f; g12 = 0.f; g22 = 1.f; }
          mbar_arrive(s ? b_adj1 : b_adj0);
        } else if (c == nch) {
          if (lane == 0) { g_final[0] = g11; g_final[1] = g12; g_final[2] = g22; }
          mbar_arrive(b_fin);
        }
      }
      if (!ok && lane == 0) {   // giving up: let the copies already in flight land before the CTA exits
        for (int c = max(0, issued - 2); c < issued; ++c)
          for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait((c & 1) ? b_full1 : b_full0, (c >> 1) & 1); ++it) {}
        for (uint32_t it = 0; it < (1u << 16) && issued_kq > 0 && !mbar_try_wait(b_cfull, (issued_kq - 1) & 1); ++it) {}
      }
      if (lane == 0) tma_store_wait_all();
    }
  } else if (warp == kWarpMma) {
    // ================================================================== MMA issuer
    // The whole warp walks the loop and waits (warp-uniform control flow and operands: the descriptors can live in
    // uniform registers); one elected lane issues the products and the commits.
    {
      const uint32_t tm = __shfl_sync(0xffffffffu, tmem, 0);
      const uint32_t sb = __shfl_sync(0xffffffffu, s_base, 0);
      const bool lead = elect_one();
      // Column of the bf16 A operands the epilogue leaves in X, Y: K-step k covers tokens 16k .. 16k + 15; the
      // epilogue warp that owns those tokens keeps hi (part 0) and lo (part 1) inside its own kTok columns
      auto a_col = [](int part, int k) {
        return static_cast<uint32_t>(kTok * ((16 * k) / kTok) + kPk * part + ((16 * k) % kTok) / 2);
      };
      const uint32_t id64 = idesc_bf16(128, 64, false, false, false);
      const uint32_t id128_mn = idesc_bf16(128, 128, false, true, false);
      const uint32_t id128_mn_neg = idesc_bf16(128, 128, false, true, true);
      const uint32_t id1 = idesc_tf32(128, write_o ? 128 : 64, false, false, false);
      const uint32_t id64_tf32 = idesc_tf32(128, 64, false, false, false);
      const uint64_t dKQ = smem_desc_sw128(sb + kOffKQ32, 16, 1024);   // + (j >> 2) * 16384 bytes + (j & 3) * 32 bytes per K step
      // per stage: T, the two halves of W, the K tile read MN-major (+2048 B per 16 tokens)
      const uint64_t dT_0 = smem_desc_sw128(sb + kOffStage + kStT, 16, 1024), dT_1 = dT_0 + (kStageBytes >> 4);
      const uint64_t dW0_0 = smem_desc_sw128(sb + kOffStage + kStW, 16, 1024), dW0_1 = dW0_0 + (kStageBytes >> 4);
      const uint64_t dKmn_0 = smem_desc_sw128(sb + kOffStage + kStK, 8192, 1024), dKmn_1 = dKmn_0 + (kStageBytes >> 4);
      for (int c = 0; c < nch; ++c) {
        const int s = c & 1;
        const uint32_t ph = c & 1;
        const uint64_t dT = s ? dT_1 : dT_0, dW0 = s ? dW0_1 : dW0_0, dW1 = dW0 + (8192 >> 4), dKmn = s ? dKmn_1 : dKmn_0;
        MDN_MARK(c, kEvLoopTop);
        MDN_SPIN(b_kq, ph);
        MDN_MARK(c, kEvKqSeen);
        if (c == 0) MDN_WAIT(b_init, 0);
        tc_fence_after_sync();
        MDN_MARK(c, kEvMma1);
        // ---- MMA-1: [X | Z] = Sh [K; Q]^T, [Y | U] = Mh [K; Q]^T  (state-only runs: X, Y against K alone).  Issued right
        // behind the previous chunk's updates of Sh, Mh, without waiting for their commits: the tensor pipe runs this
        // thread's products in issue order, a product that reads another's accumulator (or overwrites another's
        // operand) included - the probe library's chained-product tests show it.  Commits are for the epilogue.
        if (lead) {
#pragma unroll
          for (int j = 0; j < 16; ++j)
            umma_ts_tf32(tm + kColX, tm + kColS + 8 * j, dKQ + (uint64_t)((j >> 2) * 1024 + (j & 3) * 2), id1, j > 0);
          umma_commit(b_mx);
        }
        MDN_MARK(c, kEvXzIssued);
        if (write_o) MDN_SPIN(b_zu, ph ^ 1);   // the previous chunk's output has been read out of U
        tc_fence_after_sync();
        if (lead) {
#pragma unroll
          for (int j = 0; j < 16; ++j)
            umma_ts_tf32(tm + kColY, tm + kColM + 8 * j, dKQ + (uint64_t)((j >> 2) * 1024 + (j & 3) * 2), id1, j > 0);
          umma_commit(b_m1);
        }
        MDN_MARK(c, kEvYuIssued);
        // (T, W and the bf16 K tile of the stage have landed: the producer warp waited for them before it published the
        // coefficients the epilogue has used by the time it hands R over)
        // ---- MMA-2: Y = (R_hi + R_lo)^T T^T
        MDN_SPIN(b_r, ph);
        tc_fence_after_sync();
        MDN_MARK(c, kEvRSeen);
        if (lead) {
#pragma unroll
          for (int k = 0; k < 4; ++k) umma_ts(tm + kColY, tm + kColX + a_col(0, k), dT + 2 * k, id64, k > 0);
#pragma unroll
          for (int k = 0; k < 4; ++k) umma_ts(tm + kColY, tm + kColX + a_col(1, k), dT + 2 * k, id64, true);
          umma_commit(b_m2);
        }
        MDN_MARK(c, kEvM2Issued);
        // ---- MMA-3': U += V~^T W^T, V~ read as tf32 from the accumulator MMA-2 has just filled, W an fp32 tile;
        // U holds the inter-chunk terms.  Runs while the epilogue makes the state-update operands.
        if (write_o) {
          MDN_SPIN(b_oi, ph);
          tc_fence_after_sync();
          MDN_MARK(c, kEvM2Own);
          if (lead) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
              umma_ts_tf32(tm + kColU, tm + kColY + 8 * j, ((j >> 2) ? dW1 : dW0) + 2 * (j & 3), id64_tf32, true);
            umma_commit(b_mo);
          }
          MDN_MARK(c, kEvMoIssued);
        }
        // ---- MMA-3: Sh^T += (wS V~)^T K, then Mh^T -= (wM V~)^T K   (K tile read MN-major: N = dk, K = tokens); the
        // first starts while the epilogue still makes the second one's operand
        MDN_SPIN(b_v1a, ph);
        tc_fence_after_sync();
        MDN_MARK(c, kEvV1Seen);
        if (lead) {
#pragma unroll
          for (int k = 0; k < 8; ++k)
            umma_ts(tm + kColS, tm + kColX + a_col(k >> 2, k & 3), dKmn + 128 * (k & 3), id128_mn, true);
          umma_commit(b_m3s);
        }
        MDN_MARK(c, kEvSIssued);
        MDN_SPIN(b_v1b, ph);
        tc_fence_after_sync();
        MDN_MARK(c, kEvV1bSeen);
        if (lead) {
#pragma unroll
          for (int k = 0; k < 8; ++k)
            umma_ts(tm + kColM, tm + kColY + a_col(k >> 2, k & 3), dKmn + 128 * (k & 3), id128_mn_neg, true);
          umma_commit(b_m3);
        }
        MDN_MARK(c, kEvMIssued);
      }
    }
  } else if (warp >= kWarpCvt) {
    // ================================================================== converter warps
    // One chunk ahead of the chain: fp32 copies of the K and Q tiles.  bf16 tile: two dk halves of [64 rows x 128 B];
    // fp32 tile: four dk quarters of [128 rows x 128 B].  A thread takes one token row (rows across the lanes:
    // minimal wavefronts in both swizzled layouts): the sixteen loads of a tile first, then its thirty-two stores.
    const uint32_t row = static_cast<uint32_t>(tid - kWarpCvt * 32), sw = row & 7;
    for (int c = 0; c < nch; ++c) {
      MDN_WAIT(b_cfull, c & 1);
      if (c > 0) MDN_WAIT(b_m1, (c - 1) & 1);   // the previous chunk's products have read the fp32 tiles
      MDN_MARK(c, kEvCvtStart);
#pragma unroll 1
      for (int which = 0; which < (write_o ? 2 : 1); ++which) {
        const uint32_t src = s_base + kOffCvt + which * 16384 + row * 128;
        const uint32_t dst = s_base + kOffKQ32 + (which * 64 + row) * 128;
        uint4 u[16];
#pragma unroll
        for (int c16 = 0; c16 < 16; ++c16)
          asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                       : "=r"(u[c16].x), "=r"(u[c16].y), "=r"(u[c16].z), "=r"(u[c16].w)
                       : "r"(src + (c16 >> 3) * 8192 + ((static_cast<uint32_t>(c16 & 7) ^ sw) << 4)));
        if (kLayer && which == 1 && qk_dh != 0.f) {   // (kLayer = false: compiled out)
          // fused q/k norm: the Q tile's copy is q - d k (fp32, from the two bf16 rows): the output terms then come out
          // of the same products as for a plain q (their 1/|q - d k| rides on the coefficients)
#pragma unroll
          for (int c16 = 0; c16 < 16; ++c16) {
            uint4 kk;
            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(kk.x), "=r"(kk.y), "=r"(kk.z), "=r"(kk.w)
                         : "r"(src - 16384 + (c16 >> 3) * 8192 + ((static_cast<uint32_t>(c16 & 7) ^ sw) << 4)));
            const uint32_t qw[4] = {u[c16].x, u[c16].y, u[c16].z, u[c16].w}, kw[4] = {kk.x, kk.y, kk.z, kk.w};
            uint32_t f[8];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              f[2 * e] = __float_as_uint(fmaf(-qk_dh, __uint_as_float(kw[e] << 16), __uint_as_float(qw[e] << 16)));
              f[2 * e + 1] = __float_as_uint(fmaf(-qk_dh, __uint_as_float(kw[e] & 0xffff0000u), __uint_as_float(qw[e] & 0xffff0000u)));
            }
            const uint32_t d0 = dst + (c16 >> 2) * 16384, ch = static_cast<uint32_t>((c16 & 3) * 2);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(d0 + ((ch ^ sw) << 4)), "r"(f[0]), "r"(f[1]), "r"(f[2]), "r"(f[3]) : "memory");
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(d0 + (((ch + 1) ^ sw) << 4)), "r"(f[4]), "r"(f[5]), "r"(f[6]), "r"(f[7]) : "memory");
          }
        } else {
#pragma unroll
        for (int c16 = 0; c16 < 16; ++c16) {
          const uint32_t d0 = dst + (c16 >> 2) * 16384, ch = static_cast<uint32_t>((c16 & 3) * 2);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(d0 + ((ch ^ sw) << 4)), "r"(u[c16].x << 16),
                       "r"(u[c16].x & 0xffff0000u), "r"(u[c16].y << 16), "r"(u[c16].y & 0xffff0000u) : "memory");
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(d0 + (((ch + 1) ^ sw) << 4)), "r"(u[c16].z << 16),
                       "r"(u[c16].z & 0xffff0000u), "r"(u[c16].w << 16), "r"(u[c16].w & 0xffff0000u) : "memory");
        }
        }
      }
      mbar_arrive(b_cfree);          // the bf16 tiles have been read: the next chunk's may land
      fence_proxy_async_smem();
      mbar_arrive(b_kq);
      MDN_MARK(c, kEvCvtDone);
    }
  } else {
    // ================================================================== epilogue warps
    // lane quarter q4 = warp & 3 (value columns 32 q4 .. +31 = this warp's tensor-memory lanes),
    // token half hf = warp >> 2 (tokens 32 hf .. +31 in the per-token steps, dk columns 64 hf .. +63 of the masters)
    const int q4 = warp & 3, hf = (warp - kWarpEpi) >> 2;
    const int d = q4 * 32 + lane;
    const int r0 = kTok * hf;
    const uint32_t tl = tmem + (static_cast<uint32_t>(q4 * 32) << 16);
    const bool post = kLayer && a.post_on && write_o;
    uint32_t pn_phase = 0;
    for (int c = 0; c <= nch; ++c) {
      const float* aj = reinterpret_cast<const float*>(smem + kOffAdj + (c & 1) * kAdjBytes);
      if constexpr (kLayer) {
        if (post && c > 0) {
          // Fused output step of the previous chunk, second half: y = sigmoid(g) * o / sqrt(mean_d o^2 + eps) * w_d.
          // The staged fp32 tile is re-read row-wise: four threads per token sum its 128 squares, rescale and gate.
          // fp32 output: written back in place (a thread rewrites only the pieces it has read); bf16 output: the final
          // tile goes over the start of the fp32 one, once every row has been read.  Then the stage is handed back.
          const int cp = c - 1;
          uint8_t* stp = smem + kOffStage + (cp & 1) * kStageBytes;
          constexpr int kTpr = 4, kPieces = 8;   // threads per token, 16-byte fp32 pieces (8-byte gate pieces) per thread
          float* tile = reinterpret_cast<float*>(stp + kStOut);
          const int t128 = q4 * 32 + lane, prow = r0 + t128 / kTpr, part = t128 % kTpr;
          const bool g_live = cp * C + prow < sq.len;
          const uint2* gp = reinterpret_cast<const uint2*>(static_cast<const __nv_bfloat16*>(a.post_g) +
                                                           ((size_t)(sq.tok0 + cp * C + prow) * H + h) * kD) + part;
          uint2 graw[kPieces];
#pragma unroll
          for (int i = 0; i < kPieces; ++i) graw[i] = g_live ? __ldg(gp + kTpr * i) : make_uint2(0u, 0u);
          MDN_WAIT(b_pn, pn_phase);
          pn_phase ^= 1;
          float4 ov[kPieces];
          float ss = 0.f;
#pragma unroll
          for (int i = 0; i < kPieces; ++i) {   // interleaved 16-byte pieces: a row's threads cover contiguous bytes
            ov[i] = *reinterpret_cast<const float4*>(tile + prow * kD + (part + kTpr * i) * 4);
            ss = fmaf(ov[i].x, ov[i].x, fmaf(ov[i].y, ov[i].y, fmaf(ov[i].z, ov[i].z, fmaf(ov[i].w, ov[i].w, ss))));
          }
          ss += __shfl_xor_sync(0xffffffffu, ss, 1);
          ss += __shfl_xor_sync(0xffffffffu, ss, 2);
          const float rstd = rsqrtf(ss * (1.f / kD) + a.post_eps);
          if (sizeof(TO) == 2) {   // every row read before any bf16 row lands on top of the fp32 tile
            mbar_arrive(b_pn);
            MDN_WAIT(b_pn, pn_phase);
            pn_phase ^= 1;
          }
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
              *reinterpret_cast<float4*>(tile + prow * kD + col) = make_float4(y0, y1, y2, y3);
            } else {
              uint2 pk;
              pk.x = pack_bf16(y0, y1); pk.y = pack_bf16(y2, y3);
              *reinterpret_cast<uint2*>(stp + kStOut + (prow * kD + col) * 2) = pk;
            }
          }
          fence_proxy_async_smem();
          mbar_arrive((cp & 1) ? b_go1 : b_go0);
        }
      }
      if (c == 0) {
        // ---------------- the start state into the masters
#pragma unroll 1
        for (int i = 0; i < 2; ++i) {
          const int col0 = hf * 64 + i * 32;
          uint32_t sr[32], mr[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float unit = (col0 + j == d) ? 1.f : 0.f;
            sr[j] = __float_as_uint(S0p ? __ldg(S0p + (size_t)(col0 + j) * kD + d) : (id_s ? unit : 0.f));
            mr[j] = __float_as_uint(M0p ? __ldg(M0p + (size_t)(col0 + j) * kD + d) : (id_m ? unit : 0.f));
          }
          tmem_st32(tl + kColS + col0, sr);
          tmem_st32(tl + kColM + col0, mr);
        }
        tmem_wait_st();
        tc_fence_before_sync();
        mbar_arrive(b_init);
      }
      if (c == nch) {
        // ---------------- final states: [S; M] = G [Sh; Mh]  (the last chunk's MMA-3 was waited for below)
        MDN_WAIT(b_fin, 0);
        const float g11 = g_final[0], g12 = g_final[1], g22 = g_final[2];
        tc_fence_after_sync();
#pragma unroll 1
        for (int i = 0; i < 2; ++i) {
          const int col0 = hf * 64 + i * 32;
          uint32_t sr[32], mr[32];
          tmem_ld32(tl + kColS + col0, sr);
          tmem_ld32(tl + kColM + col0, mr);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float sv = __uint_as_float(sr[j]), mv = __uint_as_float(mr[j]);
            if (Sfp) Sfp[(size_t)(col0 + j) * kD + d] = g11 * sv + g12 * mv;
            if (Mfp) Mfp[(size_t)(col0 + j) * kD + d] = g22 * mv;
          }
        }
        break;
      }
      const uint32_t ph = c & 1;
      uint8_t* stg = smem + kOffStage + (c & 1) * kStageBytes;
      const __nv_bfloat16* sV = reinterpret_cast<const __nv_bfloat16*>(stg + kStV);
      if constexpr (kLayer) if (post) {   // the chunk's output-gate rows towards L2: read at the end of the chunk
        const int t128 = q4 * 32 + lane, prow = r0 + t128 / 4, part = t128 % 4;
        if (part < 2 && c * C + prow < sq.len)
          asm volatile("prefetch.global.L2 [%0];" ::"l"(static_cast<const __nv_bfloat16*>(a.post_g) +
                                                        ((size_t)(sq.tok0 + c * C + prow) * H + h) * kD + 64 * part));
      }
      MDN_WAIT((c & 1) ? b_full1 : b_full0, (c >> 1) & 1);
      MDN_WAIT((c & 1) ? b_adj1 : b_adj0, (c >> 1) & 1);
      // ---------------- EPI-1: R^T = V^T - cX .* X + cY .* Y  -> bf16 hi, lo in X
      {
        // V and the coefficients are fetched BEFORE the waits: shared-memory loads issued after a wait would sit on the
        // chain's critical path, behind whatever the converter warps have queued in the shared-memory pipe
        // (token pairs as float2: the per-token arithmetic runs on the packed two-lane fp32 instructions)
        float2 vv[kTok / 2], cf1[kTok / 2];
#pragma unroll
        for (int j = 0; j < kTok; j += 2)
          vv[j >> 1] = v_zero ? make_float2(0.f, 0.f)
                              : make_float2(__bfloat162float(sV[(r0 + j) * kD + d]), __bfloat162float(sV[(r0 + j + 1) * kD + d]));
#pragma unroll
        for (int j = 0; j < kTok; j += 4) {
          const float4 cx = *reinterpret_cast<const float4*>(aj + kCx + r0 + j);   // -cX
          cf1[j >> 1] = make_float2(cx.x, cx.y); cf1[(j >> 1) + 1] = make_float2(cx.z, cx.w);
        }
        MDN_WAIT(b_mx, ph);          // X is there; Y is still being computed
        __syncwarp();
        tc_fence_after_sync();
        {
          uint32_t x[kTok];
          tmem_ld32(tl + kColX + r0, x);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < kTok; j += 2)
            vv[j >> 1] = __ffma2_rn(cf1[j >> 1], make_float2(__uint_as_float(x[j]), __uint_as_float(x[j + 1])), vv[j >> 1]);
        }
#pragma unroll
        for (int j = 0; j < kTok; j += 4) {
          const float4 cy = *reinterpret_cast<const float4*>(aj + kCy + r0 + j);
          cf1[j >> 1] = make_float2(cy.x, cy.y); cf1[(j >> 1) + 1] = make_float2(cy.z, cy.w);
        }
        MDN_WAIT(b_m1, ph);
        __syncwarp();
        tc_fence_after_sync();
        MDN_MARK(c, kEvM1Seen);
        uint32_t hi[kPk], lo[kPk];
        {
          uint32_t y[kTok];
          tmem_ld32(tl + kColY + r0, y);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < kTok; j += 2)
            split_pack_bf16(__ffma2_rn(cf1[j >> 1], make_float2(__uint_as_float(y[j]), __uint_as_float(y[j + 1])), vv[j >> 1]),
                            hi[j >> 1], lo[j >> 1]);
        }
        // hi and lo both go into the columns this warp has just read (its own kTok columns of X)
        tmem_st16(tl + kColX + r0, hi);
        tmem_st16(tl + kColX + r0 + kPk, lo);
        tmem_wait_st();
      }
      tc_fence_before_sync();
      mbar_arrive(b_r);
      MDN_MARK(c, kEvRArrive);
      MDN_MARK2(c, kEvRArrive2);
      // ---------------- inter-chunk output terms cZ .* Z + cU .* U, left in U for MMA-3' to accumulate onto (under MMA-2)
      if (write_o) {
        uint32_t z[kTok], u[kTok];
        tmem_ld32(tl + kColZ + r0, z);
        tmem_ld32(tl + kColU + r0, u);
        float2 cz[kTok / 2], cu[kTok / 2];   // (their loads run while the tensor-memory loads are in flight)
#pragma unroll
        for (int j = 0; j < kTok; j += 4) {
          const float4 a4 = *reinterpret_cast<const float4*>(aj + kCz + r0 + j);
          const float4 b4 = *reinterpret_cast<const float4*>(aj + kCu + r0 + j);
          cz[j >> 1] = make_float2(a4.x, a4.y); cz[(j >> 1) + 1] = make_float2(a4.z, a4.w);
          cu[j >> 1] = make_float2(b4.x, b4.y); cu[(j >> 1) + 1] = make_float2(b4.z, b4.w);
        }
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < kTok; j += 2) {
          const float2 t2 = __fmul2_rn(cu[j >> 1], make_float2(__uint_as_float(u[j]), __uint_as_float(u[j + 1])));
          const float2 o2 = __ffma2_rn(cz[j >> 1], make_float2(__uint_as_float(z[j]), __uint_as_float(z[j + 1])), t2);
          u[j] = __float_as_uint(o2.x); u[j + 1] = __float_as_uint(o2.y);
        }
        tmem_st32(tl + kColU + r0, u);
        tmem_wait_st();
        tc_fence_before_sync();
        mbar_arrive(b_oi);
        MDN_MARK(c, kEvOiArrive);
      }
      // ---------------- EPI-2: wS .* V~ -> X (handed over first), wM .* V~ -> Y, each as bf16 hi, lo.  V~ itself stays
      // in Y for MMA-3' until that product has read it.  Eager chunks: the masters take G' = D_c G here (MMA-1 of this
      // chunk, their last reader, is done) and the update is added in true coordinates.
      const bool eager = aj[kLazy] == 0.f;
      const float n11 = aj[kN11], n12 = aj[kN12], n22 = aj[kN22];
      // (the first operand's weights are fetched before the wait: shared-memory loads issued after it sit on the
      // chain's critical path behind whatever the converter warps have queued)
      float2 wsv[kTok / 2];
#pragma unroll
      for (int j = 0; j < kTok; j += 4) {
        float4 a4;
        asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(a4.x), "=f"(a4.y), "=f"(a4.z), "=f"(a4.w) : "r"(smem_u32(aj + kWs + r0 + j)));
        wsv[j >> 1] = make_float2(a4.x, a4.y); wsv[(j >> 1) + 1] = make_float2(a4.z, a4.w);
      }
      MDN_WAIT(b_m2, ph);
      __syncwarp();
      tc_fence_after_sync();
      MDN_MARK(c, kEvM2Seen);
      {
        uint32_t vt[kTok];
        tmem_ld32(tl + kColY + r0, vt);
        float2 wmv[kTok / 2];   // (their loads run while the tensor-memory load is in flight)
#pragma unroll
        for (int j = 0; j < kTok; j += 4) {
          const float4 b4 = *reinterpret_cast<const float4*>(aj + kWm + r0 + j);
          wmv[j >> 1] = make_float2(b4.x, b4.y); wmv[(j >> 1) + 1] = make_float2(b4.z, b4.w);
        }
        tmem_wait_ld();
        {
          uint32_t sh[kPk], sl[kPk];
#pragma unroll
          for (int j = 0; j < kTok; j += 2)
            split_pack_bf16(__fmul2_rn(wsv[j >> 1], make_float2(__uint_as_float(vt[j]), __uint_as_float(vt[j + 1]))),
                            sh[j >> 1], sl[j >> 1]);
          tmem_st16(tl + kColX + r0, sh);          // X is free: MMA-2 has consumed R
          tmem_st16(tl + kColX + r0 + kPk, sl);
        }
        if (eager) {   // Sh <- n11 Sh + n12 Mh (Mh still the old one)
          MDN_MARK(c, kEvEager);
#pragma unroll 1
          for (int i = 0; i < 2; ++i) {
            const int col0 = hf * 64 + i * 32;
            uint32_t sr[32], mr[32];
            tmem_ld32(tl + kColS + col0, sr);
            tmem_ld32(tl + kColM + col0, mr);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 32; ++j) sr[j] = __float_as_uint(n11 * __uint_as_float(sr[j]) + n12 * __uint_as_float(mr[j]));
            tmem_st32(tl + kColS + col0, sr);
          }
        }
        tmem_wait_st();
        tc_fence_before_sync();
        mbar_arrive(b_v1a);
        MDN_MARK(c, kEvV1Arrive);
        MDN_MARK2(c, kEvV1Arrive2);
        uint32_t mh[kPk], mlo[kPk];
#pragma unroll
        for (int j = 0; j < kTok; j += 2)
          split_pack_bf16(__fmul2_rn(wmv[j >> 1], make_float2(__uint_as_float(vt[j]), __uint_as_float(vt[j + 1]))),
                          mh[j >> 1], mlo[j >> 1]);
        if (write_o) {   // MMA-3' reads V~ from Y: it must be done before Y is overwritten
          MDN_WAIT(b_mo, ph);
          __syncwarp();
          tc_fence_after_sync();
        }
        tmem_st16(tl + kColY + r0, mh);          // own columns of Y
        tmem_st16(tl + kColY + r0 + kPk, mlo);
      }
      if (eager) {   // Mh <- n22 Mh
#pragma unroll 1
        for (int i = 0; i < 2; ++i) {
          const int col0 = hf * 64 + i * 32;
          uint32_t mr[32];
          tmem_ld32(tl + kColM + col0, mr);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j) mr[j] = __float_as_uint(n22 * __uint_as_float(mr[j]));
          tmem_st32(tl + kColM + col0, mr);
        }
      }
      tmem_wait_st();
      tc_fence_before_sync();
      mbar_arrive(b_v1b);
      MDN_MARK(c, kEvV1bArrive);
      // ---------------- the chunk's output tile (under MMA-3): U -> [64 x 128] tile in the stage's Q / V area
      if (write_o) {   // (MMA-3' was waited for above)
        uint32_t u[kTok];
        tmem_ld32(tl + kColU + r0, u);
        tmem_wait_ld();
        tc_fence_before_sync();
        mbar_arrive(b_zu);
        MDN_MARK(c, kEvZuArrive);
        bool plain_out = true;
        if constexpr (kLayer) plain_out = !post;
        if (plain_out) {
#pragma unroll
          for (int j = 0; j < kTok; ++j) stage_o<TO>(stg + kStOut, r0 + j, d, __uint_as_float(u[j]));
        } else if constexpr (kLayer) {
          // fused output step, first half: the fp32 tile (value columns across the lanes; V, T and half of the W area,
          // all dead by now).  The rest runs at the top of the next iteration, under the next chunk's MMA-1.
          float* tile = reinterpret_cast<float*>(stg + kStOut);
#pragma unroll
          for (int j = 0; j < kTok; ++j) tile[(r0 + j) * kD + d] = __uint_as_float(u[j]);
          mbar_arrive(b_pn);
        }
        fence_proxy_async_smem();
        MDN_MARK(c, kEvOutDone);
      }
      // the stage may be refilled once MMA-3, the last reader of its K tile, is done
      MDN_WAIT(b_m3, ph);
      MDN_MARK(c, kEvM3Seen);
      if (!post) mbar_arrive((c & 1) ? b_go1 : b_go0);   // (fused output step: after its second half)
    }
  }
#undef MDN_WAIT
#undef MDN_SPIN
#undef MDN_MARK
#undef MDN_MARK2

  if (!ok && lane == 0) atomicCAS(a.status, kDevOk, kDevTimeout);
  tc_fence_before_sync();
  __syncthreads();
#ifdef MDN_DEBUG
  if (tline != nullptr && tid == 0) {
    unsigned long long ns;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns));
    tline[62] = clock64(); tline[63] = (long long)ns;
  }
  if (tline != nullptr && tid < 256) tline[(kTlFirst + (tid >> 5)) * 32 + (tid & 31)] = (tid & 31) < 30 ? tl_sm[tid >> 5][tid & 31] : 0;
#endif
  if (warp == kWarpMma) tmem_dealloc(tmem, 512);
}

}  // namespace

cudaError_t launch_chain_tf32(const Plan& pl, const void* q, const void* k, const void* v, const float* S0,
                              const float* M0, void* o, float* Sf, float* Mf, int* launches) {
  const mdn_params& p = pl.p;
  const uint64_t tokens = (uint64_t)p.B * p.T;
  const uint64_t mats = (uint64_t)pl.geom.num_slots * p.H;
  CUtensorMap mq, mk, mv, mt, mw, mo;
  const uint64_t row = (uint64_t)p.H * kD;
  if (!encode_tma_2d_bf16(&mq, TmaMap2D{q, row, tokens, row * 2, 64, 64, true}) ||
      !encode_tma_2d_bf16(&mk, TmaMap2D{k, row, tokens, row * 2, 64, 64, true}) ||
      !encode_tma_2d_bf16(&mv, TmaMap2D{v, row, tokens, row * 2, 128, 64, false}) ||
      !encode_tma_2d_bf16(&mt, TmaMap2D{pl.ws + pl.lay.off_T, 64, mats * C, 128, 64, 64, true}) ||
      !encode_tma_2d(&mw, TmaMap2D{pl.ws + pl.lay.off_W, 64, mats * C, 256, 32, 64, true}, true))
    return cudaErrorInvalidValue;
  const bool o_bf16 = p.o_dtype == MDN_BF16;
  if (!encode_tma_2d(&mo, TmaMap2D{o, row, tokens, row * (o_bf16 ? 2u : 4u), 128, 64, false}, !o_bf16))
    return cudaErrorInvalidValue;
  Args a;
  a.g = pl.geom;
  a.coef = reinterpret_cast<const float*>(pl.ws + pl.lay.off_coef);
  a.S0 = S0; a.M0 = M0; a.o = o; a.Sf = Sf; a.Mf = Mf;
  a.status = reinterpret_cast<int32_t*>(pl.ws + pl.lay.off_status);
  a.scale = p.scale;
  a.seg_G = 0; a.seg_phase = 0;
  a.seg_E = a.seg_Psi = a.seg_PhiS = a.seg_PhiM = nullptr;
  a.qk_on = pl.qk.on; a.qk_d = pl.qk.d;
  a.post_on = pl.post.on; a.post_w = pl.post.w; a.post_g = pl.post.g; a.post_eps = pl.post.eps;
  const bool layer = a.qk_on || a.post_on;
  a.timeline = nullptr;
#ifdef MDN_DEBUG   // debug builds only (-DMDN_DEBUG): the product library reads nothing from the environment
  const char* tl = getenv("MDN_DEBUG_TIMELINE");   // device address of an int64 buffer, [chunks][32]
  a.timeline = tl ? reinterpret_cast<long long*>(strtoull(tl, nullptr, 0)) : nullptr;
#endif
  const unsigned chains = (unsigned)pl.geom.num_seqs * p.H;
  auto launch = [&](unsigned grid) -> cudaError_t {
    auto kern = layer ? (o_bf16 ? chain_tf32_kernel<__nv_bfloat16, true> : chain_tf32_kernel<float, true>)
                      : (o_bf16 ? chain_tf32_kernel<__nv_bfloat16, false> : chain_tf32_kernel<float, false>);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    e = launch_pdl(kern, dim3(grid), dim3(kThreads), kSmemBytes, pl.stream, a, mq, mk, mv, mt, mw, mo);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e == cudaSuccess) ++*launches;
    return e;
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

}  // namespace mdn
