// Backward of the MDN recurrence (Section 3.1, Eq. 5-6): reverse-mode, token by token, with the states recomputed
// chunk by chunk from checkpoints (the paper's training kernels also keep no per-token states and rebuild them in
// the backward pass).  fp32 throughout; this is the exact CUDA form of the backward - every gradient, any dk, dv in
// {64, 128}, fixed-length or packed input.  (The chunk-parallel matrix form on the tensor cores is bwd_chunk*.cu.)
//
// The value columns of S, M and of their adjoints GS, GM are independent; only dq, dk and the gate gradients sum over
// columns.  One WARP owns 4 value columns of one (sequence, head): lane l holds rows l, l + 32, .. of those columns of
// all four matrices in registers, sums over rows are warp shuffles, and nothing inside a chunk needs a block barrier.
// A CTA is 16 such warps (64 columns); its dq, dk and gate-gradient contributions meet in shared-memory accumulators
// (floating-point atomics: the summation order, hence the last bits, may differ from run to run), are written per
// chunk as one partial result per CTA, and bwd_finish_kernel adds the CTAs' partials in a fixed order.
//   phase 1  forward sweep, keeping (S, M) every kBlk tokens (global scratch);
//   phase 2  blocks in reverse: recompute the block forward, parking S_{t-1}, M_{t-1} of every token (global
//            scratch that stays in L2, fetched back one token ahead) and v~_t, S_{t-1}^T k_t (shared memory); then
//            the adjoint steps of the block, last token first:
//     GS += scale q do^T;  dq = scale S_t do;  dbeta = -<GS, M_t>;  GM -= beta GS;  a = GM v~;  deta = -k.a;
//     dv~ = -eta GM^T k = dv;  dalpha = <GS, S_{t-1}> - dv~.(S_{t-1}^T k);  dmu = <GM, M_{t-1}>;
//     dk = -eta a - alpha S_{t-1} dv~;  GS <- alpha (GS - k dv~^T);  GM <- mu GM.
#include "mdn_common.cuh"

namespace mdn {
namespace {

constexpr int kCW = 4;             // value columns per warp
constexpr int kWarps = 16;         // warps per CTA
constexpr int kNV = kCW * kWarps;  // value columns per CTA
constexpr int kBT = kWarps * 32;
// Recomputation block: (S, M) is kept every kBlk tokens and the states before each token are parked for one block
// at a time.  Parking a whole 64-token chunk made the pass HBM-bound (2 x dk x dv x 4 bytes written and read back
// per token and chain: 137 GB at B=8, H=16, T=4096); with short blocks the parked states of all resident CTAs
// (148 x kBlk x 64 KB) stay in the 126 MB L2 and only the checkpoints (1 / kBlk of that traffic) reach HBM.
constexpr int kBlk = 8;
static_assert(C % kBlk == 0, "blocks tile a chunk");

struct BwdArgs {
  ChunkGeom g;
  const void* q; const void* k; const void* v;
  const float* beta; const float* log_alpha; const float* log_mu; const float* eta;
  const float* S0; const float* M0;
  const void* d_o; const float* dSf; const float* dMf;
  float scale;
  int DV;
  float* dv_out; float* dS0; float* dM0;
  float* part_q; float* part_k; float* part_g;   // [NCB][tokens][H][dk] x2, [NCB][tokens][H][4]
  float* ck;      // [slot][C/kBlk][H][dv/4][2][dk][4]  state at the start of every block, per warp
  float* prev;    // [chain][dv/4][kBlk][2][dk][4] S_{t-1}, M_{t-1} of the block being processed, per warp
};

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
  return x;
}

template <typename TIn, typename TDo, int DK>
__global__ void __launch_bounds__(kBT, 1) bwd_stepwise_kernel(BwdArgs a) {
  constexpr int RW = DK / 32;   // rows per lane
  extern __shared__ __align__(16) uint8_t smem_raw[];
  TIn* ks = reinterpret_cast<TIn*>(smem_raw);                                 // [C][DK]
  TIn* qs = ks + C * DK;                                                      // [C][DK]
  float* vs = reinterpret_cast<float*>(smem_raw + 2 * C * DK * sizeof(TIn));  // [C][64]
  float* dos = vs + C * kNV;                                                  // [C][64]
  float* vts = dos + C * kNV;                                                 // [C][64]  v~_t            (warp-private columns)
  float* preds = vts + C * kNV;                                               // [C][64]  S_{t-1}^T k_t   (warp-private columns)
  float* gts = preds + C * kNV;                                               // [4][C]   alpha, mu, beta, eta
  float* dq_acc = gts + 4 * C;                                                // [C][DK]
  float* dk_acc = dq_acc + C * DK;                                            // [C][DK]
  float* g_acc = dk_acc + C * DK;                                             // [C][4]   dbeta, dlog_alpha, dlog_mu, deta

  const int tid = threadIdx.x, lane = tid & 31, wp = tid >> 5;
  const int chain = blockIdx.x, cb = blockIdx.y;
  const int H = a.g.H, seq = chain / H, h = chain % H;
  const int DV = a.DV, NW = DV / kCW;            // warps (column groups) per chain
  const int wcol = cb * kWarps + wp;             // this warp's column group
  const int j0 = wcol * kCW;                     // its first value column
  const int cl = wp * kCW;                       // ... within the CTA's 64
  const SeqInfo sq = seq_info(a.g, seq);
  const int nch = sq.nchunks;
  const size_t st_off = (size_t)chain * DK * DV;
  const TIn* qg = static_cast<const TIn*>(a.q);
  const TIn* kg = static_cast<const TIn*>(a.k);
  const TIn* vg = static_cast<const TIn*>(a.v);
  const TDo* dog = static_cast<const TDo*>(a.d_o);
  const size_t n_tok = (size_t)a.g.B * a.g.T;

  float S[RW][kCW], M[RW][kCW];
#pragma unroll
  for (int r = 0; r < RW; ++r) {
    const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
    const size_t i = st_off + (size_t)(lane + 32 * r) * DV + j0;
    const float4 s4 = a.S0 ? __ldg(reinterpret_cast<const float4*>(a.S0 + i)) : z;
    const float4 m4 = a.M0 ? __ldg(reinterpret_cast<const float4*>(a.M0 + i)) : z;
    S[r][0] = s4.x; S[r][1] = s4.y; S[r][2] = s4.z; S[r][3] = s4.w;
    M[r][0] = m4.x; M[r][1] = m4.y; M[r][2] = m4.z; M[r][3] = m4.w;
  }

  // stage the k (and q) rows, the CTA's v (and dO) columns and the gates of chunk c; zero the accumulators
  auto stage = [&](int c, bool adjoint) {
    const int n = min(C, sq.len - c * C);
    const size_t tok0 = (size_t)sq.tok0 + (size_t)c * C;
    for (int idx = tid; idx < n * DK; idx += kBT) {
      const int t = idx / DK, d = idx - t * DK;
      ks[idx] = kg[((tok0 + t) * H + h) * DK + d];
      if (adjoint) qs[idx] = qg[((tok0 + t) * H + h) * DK + d];
    }
    for (int idx = tid; idx < n * kNV; idx += kBT) {
      const int t = idx / kNV, jj = idx - t * kNV;
      vs[idx] = to_f32<TIn>(vg[((tok0 + t) * H + h) * DV + cb * kNV + jj]);
      if (adjoint) dos[idx] = to_f32<TDo>(dog[((tok0 + t) * H + h) * DV + cb * kNV + jj]);
    }
    if (tid < n) {
      const size_t gi = (tok0 + tid) * H + h;
      gts[0 * C + tid] = expf(__ldg(a.log_alpha + gi));
      gts[1 * C + tid] = expf(__ldg(a.log_mu + gi));
      gts[2 * C + tid] = __ldg(a.beta + gi);
      gts[3 * C + tid] = a.eta ? __ldg(a.eta + gi) : 1.f;
    }
    if (adjoint) {
      for (int idx = tid; idx < C * DK; idx += kBT) { dq_acc[idx] = 0.f; dk_acc[idx] = 0.f; }
      for (int idx = tid; idx < C * 4; idx += kBT) g_acc[idx] = 0.f;
    }
    return n;
  };

  // one forward token on the warp's columns; vt = v~, pred = S_{t-1}^T k (both for the 4 columns, on every lane)
  auto forward_token = [&](int t, float (&vt)[kCW], float (&pred)[kCW]) {
    float kr[RW];
#pragma unroll
    for (int r = 0; r < RW; ++r) kr[r] = to_f32<TIn>(ks[t * DK + lane + 32 * r]);
#pragma unroll
    for (int c4 = 0; c4 < kCW; ++c4) {
      float w = 0.f;
#pragma unroll
      for (int r = 0; r < RW; ++r) w = fmaf(S[r][c4], kr[r], w);
      pred[c4] = warp_sum(w);
    }
    const float al = gts[0 * C + t], mu = gts[1 * C + t], be = gts[2 * C + t], et = gts[3 * C + t];
    const float4 v4 = *reinterpret_cast<const float4*>(vs + t * kNV + cl);
    vt[0] = v4.x - al * pred[0]; vt[1] = v4.y - al * pred[1]; vt[2] = v4.z - al * pred[2]; vt[3] = v4.w - al * pred[3];
#pragma unroll
    for (int r = 0; r < RW; ++r)
#pragma unroll
      for (int c4 = 0; c4 < kCW; ++c4) {
        const float m_new = mu * M[r][c4] - et * kr[r] * vt[c4];
        M[r][c4] = m_new;
        S[r][c4] = al * S[r][c4] - be * m_new;
      }
  };
  auto store_state = [&](float* dst) {   // [2][DK][4]
#pragma unroll
    for (int r = 0; r < RW; ++r) {
      reinterpret_cast<float4*>(dst)[lane + 32 * r] = make_float4(S[r][0], S[r][1], S[r][2], S[r][3]);
      reinterpret_cast<float4*>(dst)[DK + lane + 32 * r] = make_float4(M[r][0], M[r][1], M[r][2], M[r][3]);
    }
  };

  // ------------------------------------------------------------------ phase 1: checkpoints
  auto ck_ptr = [&](int c, int b) {
    return a.ck + (((((size_t)(sq.slot0 + c) * (C / kBlk) + b) * H + h) * NW + wcol) * 2) * DK * kCW;
  };
  for (int c = 0; c < nch; ++c) {
    __syncthreads();   // every warp is done with the previous chunk's staged tiles
    const int n = stage(c, false);
    __syncthreads();
    for (int t = 0; t < n; ++t) {
      if (t % kBlk == 0) store_state(ck_ptr(c, t / kBlk));
      float vt[kCW], pred[kCW];
      forward_token(t, vt, pred);
    }
  }

  // ------------------------------------------------------------------ phase 2: reverse over chunks
  float GS[RW][kCW], GM[RW][kCW];
#pragma unroll
  for (int r = 0; r < RW; ++r) {
    const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
    const size_t i = st_off + (size_t)(lane + 32 * r) * DV + j0;
    const float4 s4 = a.dSf ? __ldg(reinterpret_cast<const float4*>(a.dSf + i)) : z;
    const float4 m4 = a.dMf ? __ldg(reinterpret_cast<const float4*>(a.dMf + i)) : z;
    GS[r][0] = s4.x; GS[r][1] = s4.y; GS[r][2] = s4.z; GS[r][3] = s4.w;
    GM[r][0] = m4.x; GM[r][1] = m4.y; GM[r][2] = m4.z; GM[r][3] = m4.w;
  }
  float* prevp = a.prev + ((size_t)chain * NW + wcol) * kBlk * 2 * DK * kCW;
  for (int c = nch - 1; c >= 0; --c) {
    __syncthreads();   // the previous chunk's accumulators have been written out
    const int n = stage(c, true);
    __syncthreads();
    const size_t tok0 = (size_t)sq.tok0 + (size_t)c * C;
    for (int b = (n - 1) / kBlk; b >= 0; --b) {
    const int tb = b * kBlk, te = min(n, tb + kBlk);
    {
      const float4* ckp = reinterpret_cast<const float4*>(ck_ptr(c, b));
#pragma unroll
      for (int r = 0; r < RW; ++r) {
        const float4 s4 = ckp[lane + 32 * r], m4 = ckp[DK + lane + 32 * r];
        S[r][0] = s4.x; S[r][1] = s4.y; S[r][2] = s4.z; S[r][3] = s4.w;
        M[r][0] = m4.x; M[r][1] = m4.y; M[r][2] = m4.z; M[r][3] = m4.w;
      }
    }
    // recompute, parking the state BEFORE every token
    for (int t = tb; t < te; ++t) {
      store_state(prevp + (size_t)(t - tb) * 2 * DK * kCW);
      float vt[kCW], pred[kCW];
      forward_token(t, vt, pred);
      if (lane == 0) {
        *reinterpret_cast<float4*>(vts + t * kNV + cl) = make_float4(vt[0], vt[1], vt[2], vt[3]);
        *reinterpret_cast<float4*>(preds + t * kNV + cl) = make_float4(pred[0], pred[1], pred[2], pred[3]);
      }
    }
    __syncwarp();
    // adjoint steps; S_{t-1}, M_{t-1} of the next token to be processed are fetched one token ahead
    float Sp[RW][kCW], Mp[RW][kCW];
    auto fetch_prev = [&](int t) {
      const float4* pp = reinterpret_cast<const float4*>(prevp + (size_t)(t - tb) * 2 * DK * kCW);
#pragma unroll
      for (int r = 0; r < RW; ++r) {
        const float4 s4 = pp[lane + 32 * r], m4 = pp[DK + lane + 32 * r];
        Sp[r][0] = s4.x; Sp[r][1] = s4.y; Sp[r][2] = s4.z; Sp[r][3] = s4.w;
        Mp[r][0] = m4.x; Mp[r][1] = m4.y; Mp[r][2] = m4.z; Mp[r][3] = m4.w;
      }
    };
    fetch_prev(te - 1);
    for (int t = te - 1; t >= tb; --t) {
      const float al = gts[0 * C + t], mu = gts[1 * C + t], be = gts[2 * C + t], et = gts[3 * C + t];
      const float4 do4 = *reinterpret_cast<const float4*>(dos + t * kNV + cl);
      const float4 vt4 = *reinterpret_cast<const float4*>(vts + t * kNV + cl);
      const float4 pr4 = *reinterpret_cast<const float4*>(preds + t * kNV + cl);
      const float dov[kCW] = {do4.x, do4.y, do4.z, do4.w}, vtv[kCW] = {vt4.x, vt4.y, vt4.z, vt4.w};
      const float prv[kCW] = {pr4.x, pr4.y, pr4.z, pr4.w};
      float kr[RW], dqr[RW], ar[RW];
      float nb = 0.f, na = 0.f, nm = 0.f, ke = 0.f;
      float wv[kCW] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int r = 0; r < RW; ++r) {
        kr[r] = to_f32<TIn>(ks[t * DK + lane + 32 * r]);
        const float qr = a.scale * to_f32<TIn>(qs[t * DK + lane + 32 * r]);
        float dq_r = 0.f, a_r = 0.f;
#pragma unroll
        for (int c4 = 0; c4 < kCW; ++c4) {
          const float m_t = mu * Mp[r][c4] - et * kr[r] * vtv[c4];
          const float s_t = al * Sp[r][c4] - be * m_t;
          GS[r][c4] = fmaf(qr, dov[c4], GS[r][c4]);
          dq_r = fmaf(s_t, dov[c4], dq_r);
          nb = fmaf(GS[r][c4], m_t, nb);
          na = fmaf(GS[r][c4], Sp[r][c4], na);
          GM[r][c4] = fmaf(-be, GS[r][c4], GM[r][c4]);
          nm = fmaf(GM[r][c4], Mp[r][c4], nm);
          a_r = fmaf(GM[r][c4], vtv[c4], a_r);
          wv[c4] = fmaf(GM[r][c4], kr[r], wv[c4]);
        }
        dqr[r] = a.scale * dq_r;
        ar[r] = a_r;
        ke = fmaf(kr[r], a_r, ke);
      }
      float dvt[kCW];
#pragma unroll
      for (int c4 = 0; c4 < kCW; ++c4) dvt[c4] = -et * warp_sum(wv[c4]);
      float dp = 0.f;
#pragma unroll
      for (int c4 = 0; c4 < kCW; ++c4) dp = fmaf(dvt[c4], prv[c4], dp);
#pragma unroll
      for (int r = 0; r < RW; ++r) {
        float e_r = 0.f;
#pragma unroll
        for (int c4 = 0; c4 < kCW; ++c4) {
          e_r = fmaf(Sp[r][c4], dvt[c4], e_r);
          GS[r][c4] = al * (GS[r][c4] - kr[r] * dvt[c4]);
          GM[r][c4] *= mu;
        }
        atomicAdd(dq_acc + t * DK + lane + 32 * r, dqr[r]);
        atomicAdd(dk_acc + t * DK + lane + 32 * r, -et * ar[r] - al * e_r);
      }
      if (t > tb) fetch_prev(t - 1);   // in flight while the reductions below finish this token
      nb = warp_sum(nb); na = warp_sum(na); nm = warp_sum(nm); ke = warp_sum(ke);
      if (lane == 0) {
        *reinterpret_cast<float4*>(a.dv_out + ((tok0 + t) * H + h) * DV + j0) = make_float4(dvt[0], dvt[1], dvt[2], dvt[3]);
        atomicAdd(g_acc + t * 4 + 0, -nb);
        atomicAdd(g_acc + t * 4 + 1, al * (na - dp));
        atomicAdd(g_acc + t * 4 + 2, mu * nm);
        atomicAdd(g_acc + t * 4 + 3, -ke);
      }
    }
    }   // blocks of the chunk
    __syncthreads();   // all warps' contributions of this chunk are in the accumulators
    for (int idx = tid; idx < n * DK; idx += kBT) {
      const int t = idx / DK, d = idx - t * DK;
      const size_t pi = (((size_t)cb * n_tok + (tok0 + t)) * H + h) * DK + d;
      a.part_q[pi] = dq_acc[idx];
      a.part_k[pi] = dk_acc[idx];
    }
    for (int idx = tid; idx < n * 4; idx += kBT)
      a.part_g[(((size_t)cb * n_tok + (tok0 + (idx >> 2))) * H + h) * 4 + (idx & 3)] = g_acc[idx];
  }
#pragma unroll
  for (int r = 0; r < RW; ++r) {
    const size_t i = st_off + (size_t)(lane + 32 * r) * DV + j0;
    if (a.dS0) *reinterpret_cast<float4*>(a.dS0 + i) = make_float4(GS[r][0], GS[r][1], GS[r][2], GS[r][3]);
    if (a.dM0) *reinterpret_cast<float4*>(a.dM0 + i) = make_float4(GM[r][0], GM[r][1], GM[r][2], GM[r][3]);
  }
}

// Sums the CTAs' partial results in a fixed order.
__global__ void __launch_bounds__(256) bwd_finish_kernel(size_t n_qk, size_t n_g, int NCB, const float* __restrict__ part_q,
                                                        const float* __restrict__ part_k,
                                                        const float* __restrict__ part_g, float* __restrict__ dq,
                                                        float* __restrict__ dk, float* __restrict__ dbeta,
                                                        float* __restrict__ dlog_alpha, float* __restrict__ dlog_mu,
                                                        float* __restrict__ deta) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_qk; i += stride) {
    float sq = 0.f, sk = 0.f;
    for (int b = 0; b < NCB; ++b) { sq += part_q[(size_t)b * n_qk + i]; sk += part_k[(size_t)b * n_qk + i]; }
    dq[i] = sq; dk[i] = sk;
  }
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_g; i += stride) {
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int b = 0; b < NCB; ++b) {
      const float4 p = reinterpret_cast<const float4*>(part_g)[(size_t)b * n_g + i];
      s.x += p.x; s.y += p.y; s.z += p.z; s.w += p.w;
    }
    dbeta[i] = s.x; dlog_alpha[i] = s.y; dlog_mu[i] = s.z;
    if (deta) deta[i] = s.w;
  }
}

template <typename TIn, int DK>
size_t bwd_smem_bytes() {
  return (size_t)2 * C * DK * sizeof(TIn) + sizeof(float) * ((size_t)4 * C * kNV + 4 * C + 2 * C * DK + 4 * C);
}

template <typename TIn, typename TDo, int DK>
cudaError_t launch_one(const BwdArgs& a, dim3 grid, cudaStream_t st) {
  auto kern = bwd_stepwise_kernel<TIn, TDo, DK>;
  const size_t smem = bwd_smem_bytes<TIn, DK>();
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  kern<<<grid, kBT, smem, st>>>(a);
  return cudaGetLastError();
}

}  // namespace

void bwd_scratch_layout(const mdn_params& p, int num_slots, BwdScratch* s) {
  const uint64_t ncb = ((uint64_t)p.dv + kNV - 1) / kNV, tokens = (uint64_t)p.B * p.T;
  const uint64_t chains = (uint64_t)(p.num_seqs > 0 ? p.num_seqs : p.B) * p.H;
  auto up = [](uint64_t x) { return (x + 255) / 256 * 256; };
  uint64_t off = 0;
  s->part_q = off; off = up(off + ncb * tokens * p.H * p.dk * 4);
  s->part_k = off; off = up(off + ncb * tokens * p.H * p.dk * 4);
  s->part_g = off; off = up(off + ncb * tokens * p.H * 4 * 4);
  s->ck = off; off = up(off + (uint64_t)num_slots * (C / kBlk) * p.H * 2 * p.dk * p.dv * 4);
  s->prev = off; off = up(off + chains * kBlk * 2 * p.dk * p.dv * 4);
  s->total = off;
}

cudaError_t launch_bwd_stepwise(const Plan& pl, const BwdIo& io, char* scratch, const BwdScratch& sl, int* launches) {
  const mdn_params& p = pl.p;
  BwdArgs a;
  a.g = pl.geom;
  a.q = io.q; a.k = io.k; a.v = io.v;
  a.beta = io.beta; a.log_alpha = io.log_alpha; a.log_mu = io.log_mu; a.eta = io.eta;
  a.S0 = io.S0; a.M0 = io.M0; a.d_o = io.d_o; a.dSf = io.dSf; a.dMf = io.dMf;
  a.scale = p.scale; a.DV = p.dv;
  a.dv_out = io.dv; a.dS0 = io.dS0; a.dM0 = io.dM0;
  a.part_q = reinterpret_cast<float*>(scratch + sl.part_q);
  a.part_k = reinterpret_cast<float*>(scratch + sl.part_k);
  a.part_g = reinterpret_cast<float*>(scratch + sl.part_g);
  a.ck = reinterpret_cast<float*>(scratch + sl.ck);
  a.prev = reinterpret_cast<float*>(scratch + sl.prev);
  const int NCB = p.dv / kNV;
  const dim3 grid((unsigned)pl.geom.num_seqs * p.H, (unsigned)NCB);
  const bool in_bf = p.io_dtype == MDN_BF16, do_bf = p.o_dtype == MDN_BF16;
  cudaError_t e;
#define MDN_BWD_CASE(TI, TD)                                                     \
  e = p.dk == 64 ? launch_one<TI, TD, 64>(a, grid, pl.stream) : launch_one<TI, TD, 128>(a, grid, pl.stream)
  if (in_bf && do_bf) { MDN_BWD_CASE(__nv_bfloat16, __nv_bfloat16); }
  else if (in_bf) { MDN_BWD_CASE(__nv_bfloat16, float); }
  else if (do_bf) { MDN_BWD_CASE(float, __nv_bfloat16); }
  else { MDN_BWD_CASE(float, float); }
#undef MDN_BWD_CASE
  if (e != cudaSuccess) return e;
  ++*launches;
  const size_t n_g = (size_t)p.B * p.T * p.H, n_qk = n_g * p.dk;
  bwd_finish_kernel<<<148 * 8, 256, 0, pl.stream>>>(n_qk, n_g, NCB, a.part_q, a.part_k, a.part_g, io.dq, io.dk, io.dbeta,
                                                    io.dlog_alpha, io.dlog_mu, io.deta);
  e = cudaGetLastError();
  if (e == cudaSuccess) ++*launches;
  return e;
}

}  // namespace mdn
