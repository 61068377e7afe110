// Backward of the MDN recurrence (Section 3.1, Eq. 5-6): reverse-mode, token by token, with the states recomputed
// chunk by chunk from checkpoints (the paper's training kernels also keep no per-token states and rebuild them in
// the backward pass).  fp32 throughout; this is the first, exact CUDA form of the backward - every gradient, any
// dk, dv in {64, 128}, fixed-length or packed input - not yet the chunk-parallel matrix form.
//
// One CTA per (sequence, head, block of 32 value columns): the columns of S, M and of their adjoints GS, GM are
// independent, only dq, dk and the gate gradients sum over columns (partial results per column block, summed by
// bwd_finish_kernel in a fixed order).  256 threads = 8 row groups x 32 columns; a thread owns dk / 8 rows of one
// column of S, M, GS, GM in registers.
//   phase 1  forward sweep, keeping (S, M) at the start of every 64-token chunk (global scratch);
//   phase 2  chunks in reverse: recompute the chunk forward, parking S_{t-1}, M_{t-1} of every token (global
//            scratch, 2 x dk x 32 floats per token) and v~_t, S_{t-1}^T k_t (shared memory); then the adjoint
//            steps t = n-1 .. 0:
//     GS += scale q do^T;  dq = scale S_t do;  dbeta = -<GS, M_t>;  GM -= beta GS;  a = GM v~;  deta = -k.a;
//     dv~ = -eta GM^T k = dv;  dalpha = <GS, S_{t-1}> - dv~.(S_{t-1}^T k);  dmu = <GM, M_{t-1}>;
//     dk = -eta a - alpha S_{t-1} dv~;  GS <- alpha (GS - k dv~^T);  GM <- mu GM.
// Sums over rows (per column) go through an 8 x 32 shared array; sums over the 32 columns (per row) through
// [dk][33] shared tiles read back by two threads per row; two block barriers per adjoint step.
#include "mdn_common.cuh"

namespace mdn {
namespace {

constexpr int kNV = 32;          // value columns per CTA
constexpr int kGroups = 8;       // row groups
constexpr int kBT = kNV * kGroups;
constexpr int kLT = kNV + 1;     // tile row stride (floats)

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
  float* ck;      // [slot][H][NCB][2][dk][32]  state at the start of every chunk
  float* prev;    // [chain][NCB][64][2][dk][32] S_{t-1}, M_{t-1} of the chunk being processed
};

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
  return x;
}

template <typename TIn, typename TDo, int DK>
__global__ void __launch_bounds__(kBT, DK == 128 && sizeof(TIn) == 4 ? 1 : 2) bwd_stepwise_kernel(BwdArgs a) {
  constexpr int RPT = DK / kGroups;
  extern __shared__ __align__(16) uint8_t smem_raw[];
  TIn* ks = reinterpret_cast<TIn*>(smem_raw);                          // [C][DK]
  float* vs = reinterpret_cast<float*>(smem_raw + C * DK * sizeof(TIn)); // [C][32]
  float* dos = vs + C * kNV;                                           // [C][32]
  float* vts = dos + C * kNV;                                          // [C][32]  v~_t
  float* preds = vts + C * kNV;                                        // [C][32]  S_{t-1}^T k_t
  float* gts = preds + C * kNV;                                        // [4][C]   alpha, mu, beta, eta
  float* red8 = gts + 4 * C;                                           // [2][8][32]
  float* tileA = red8 + 2 * kGroups * kNV;                             // [DK][33]
  float* tileB = tileA + DK * kLT;
  float* tileC = tileB + DK * kLT;
  float* scal = tileC + DK * kLT;                                      // [8][4]

  const int tid = threadIdx.x, lane = tid & 31, dg = tid >> 5;
  const int chain = blockIdx.x, cb = blockIdx.y, NCB = gridDim.y;
  const int H = a.g.H, seq = chain / H, h = chain % H;
  const int DV = a.DV, j = cb * kNV + lane;
  const SeqInfo sq = seq_info(a.g, seq);
  const int nch = sq.nchunks;
  const size_t cta = (size_t)chain * NCB + cb;
  const size_t st_off = (size_t)chain * DK * DV;
  const TIn* qg = static_cast<const TIn*>(a.q);
  const TIn* kg = static_cast<const TIn*>(a.k);
  const TIn* vg = static_cast<const TIn*>(a.v);
  const TDo* dog = static_cast<const TDo*>(a.d_o);

  float S[RPT], M[RPT];
#pragma unroll
  for (int r = 0; r < RPT; ++r) {
    const size_t i = st_off + (size_t)(dg * RPT + r) * DV + j;
    S[r] = a.S0 ? __ldg(a.S0 + i) : 0.f;
    M[r] = a.M0 ? __ldg(a.M0 + i) : 0.f;
  }

  // stage the k rows, the v (and dO) columns and the gates of chunk c
  auto stage = [&](int c, bool with_do) {
    const int n = min(C, sq.len - c * C);
    const size_t tok0 = (size_t)sq.tok0 + (size_t)c * C;
    for (int idx = tid; idx < n * DK; idx += kBT) {
      const int t = idx / DK, d = idx - t * DK;
      ks[t * DK + d] = kg[((tok0 + t) * H + h) * DK + d];
    }
    for (int idx = tid; idx < n * kNV; idx += kBT) {
      const int t = idx / kNV, jj = idx - t * kNV;
      vs[idx] = to_f32<TIn>(vg[((tok0 + t) * H + h) * DV + cb * kNV + jj]);
      if (with_do) dos[idx] = to_f32<TDo>(dog[((tok0 + t) * H + h) * DV + cb * kNV + jj]);
    }
    if (tid < n) {
      const size_t gi = (tok0 + tid) * H + h;
      gts[0 * C + tid] = expf(__ldg(a.log_alpha + gi));
      gts[1 * C + tid] = expf(__ldg(a.log_mu + gi));
      gts[2 * C + tid] = __ldg(a.beta + gi);
      gts[3 * C + tid] = a.eta ? __ldg(a.eta + gi) : 1.f;
    }
    return n;
  };

  // one forward token on the thread's rows; returns v~ and the prediction for column j
  auto forward_token = [&](int t, float& vt, float& pred) {
    float w = 0.f;
#pragma unroll
    for (int r = 0; r < RPT; ++r) w = fmaf(S[r], to_f32<TIn>(ks[t * DK + dg * RPT + r]), w);
    float* rb = red8 + (t & 1) * kGroups * kNV;
    rb[dg * kNV + lane] = w;
    __syncthreads();
    pred = 0.f;
#pragma unroll
    for (int g8 = 0; g8 < kGroups; ++g8) pred += rb[g8 * kNV + lane];
    const float al = gts[0 * C + t], mu = gts[1 * C + t], be = gts[2 * C + t], et = gts[3 * C + t];
    vt = vs[t * kNV + lane] - al * pred;
#pragma unroll
    for (int r = 0; r < RPT; ++r) {
      const float m_new = mu * M[r] - et * to_f32<TIn>(ks[t * DK + dg * RPT + r]) * vt;
      M[r] = m_new;
      S[r] = al * S[r] - be * m_new;
    }
  };

  // ------------------------------------------------------------------ phase 1: checkpoints
  for (int c = 0; c < nch; ++c) {
    float* ckp = a.ck + ((((size_t)(sq.slot0 + c) * H + h) * NCB + cb) * 2) * DK * kNV;
#pragma unroll
    for (int r = 0; r < RPT; ++r) {
      ckp[(size_t)(dg * RPT + r) * kNV + lane] = S[r];
      ckp[(size_t)(DK + dg * RPT + r) * kNV + lane] = M[r];
    }
    __syncthreads();   // the previous chunk's tokens are done with the staged tiles
    const int n = stage(c, false);
    __syncthreads();
    for (int t = 0; t < n; ++t) {
      float vt, pred;
      forward_token(t, vt, pred);
    }
  }

  // ------------------------------------------------------------------ phase 2: reverse over chunks
  float GS[RPT], GM[RPT];
#pragma unroll
  for (int r = 0; r < RPT; ++r) {
    const size_t i = st_off + (size_t)(dg * RPT + r) * DV + j;
    GS[r] = a.dSf ? __ldg(a.dSf + i) : 0.f;
    GM[r] = a.dMf ? __ldg(a.dMf + i) : 0.f;
  }
  float* prevp = a.prev + cta * C * 2 * DK * kNV;
  for (int c = nch - 1; c >= 0; --c) {
    const float* ckp = a.ck + ((((size_t)(sq.slot0 + c) * H + h) * NCB + cb) * 2) * DK * kNV;
#pragma unroll
    for (int r = 0; r < RPT; ++r) {
      S[r] = ckp[(size_t)(dg * RPT + r) * kNV + lane];
      M[r] = ckp[(size_t)(DK + dg * RPT + r) * kNV + lane];
    }
    __syncthreads();
    const int n = stage(c, true);
    __syncthreads();
    const size_t tok0 = (size_t)sq.tok0 + (size_t)c * C;
    // recompute, parking the state BEFORE every token
    for (int t = 0; t < n; ++t) {
      float* pp = prevp + (size_t)t * 2 * DK * kNV;
#pragma unroll
      for (int r = 0; r < RPT; ++r) {
        pp[(size_t)(dg * RPT + r) * kNV + lane] = S[r];
        pp[(size_t)(DK + dg * RPT + r) * kNV + lane] = M[r];
      }
      float vt, pred;
      forward_token(t, vt, pred);
      if (dg == 0) { vts[t * kNV + lane] = vt; preds[t * kNV + lane] = pred; }
    }
    __syncthreads();
    // adjoint steps; S_{t-1}, M_{t-1} of the next token to be processed are fetched one token ahead
    float Sp[RPT], Mp[RPT];
    if (n > 0) {
      const float* pp = prevp + (size_t)(n - 1) * 2 * DK * kNV;
#pragma unroll
      for (int r = 0; r < RPT; ++r) {
        Sp[r] = pp[(size_t)(dg * RPT + r) * kNV + lane];
        Mp[r] = pp[(size_t)(DK + dg * RPT + r) * kNV + lane];
      }
    }
    for (int t = n - 1; t >= 0; --t) {
      const float al = gts[0 * C + t], mu = gts[1 * C + t], be = gts[2 * C + t], et = gts[3 * C + t];
      const float doj = dos[t * kNV + lane], vtj = vts[t * kNV + lane];
      const size_t grow = (tok0 + t) * H + h;
      float kr[RPT];
      float nb = 0.f, na = 0.f, nm = 0.f, w = 0.f;
#pragma unroll
      for (int r = 0; r < RPT; ++r) {
        const int row = dg * RPT + r;
        kr[r] = to_f32<TIn>(ks[t * DK + row]);
        const float qr = to_f32<TIn>(__ldg(qg + grow * DK + row));
        const float m_t = mu * Mp[r] - et * kr[r] * vtj;
        const float s_t = al * Sp[r] - be * m_t;
        GS[r] = fmaf(a.scale * qr, doj, GS[r]);
        nb = fmaf(GS[r], m_t, nb);
        na = fmaf(GS[r], Sp[r], na);
        GM[r] = fmaf(-be, GS[r], GM[r]);
        nm = fmaf(GM[r], Mp[r], nm);
        tileA[row * kLT + lane] = s_t * doj;
        tileB[row * kLT + lane] = GM[r] * vtj;
        w = fmaf(GM[r], kr[r], w);
      }
      red8[dg * kNV + lane] = w;
      nb = warp_sum(nb); na = warp_sum(na); nm = warp_sum(nm);
      if (lane == 0) { scal[dg * 4 + 0] = nb; scal[dg * 4 + 1] = na; scal[dg * 4 + 2] = nm; }
      __syncthreads();   // (1)
      float dvt = 0.f;
#pragma unroll
      for (int g8 = 0; g8 < kGroups; ++g8) dvt += red8[g8 * kNV + lane];
      dvt *= -et;
      // sums over the 32 columns: two threads per row
      const int rrow = tid >> 1, half = tid & 1;
      float sa = 0.f, sb = 0.f;
      if (rrow < DK) {
#pragma unroll
        for (int x = 0; x < kNV / 2; ++x) {
          sa += tileA[rrow * kLT + half * (kNV / 2) + x];
          sb += tileB[rrow * kLT + half * (kNV / 2) + x];
        }
      }
      sa += __shfl_xor_sync(0xffffffffu, sa, 1);
      sb += __shfl_xor_sync(0xffffffffu, sb, 1);
#pragma unroll
      for (int r = 0; r < RPT; ++r) tileC[(dg * RPT + r) * kLT + lane] = Sp[r] * dvt;
      if (t > 0) {   // the previous state of token t - 1: in flight while this token is finished
        const float* pp = prevp + (size_t)(t - 1) * 2 * DK * kNV;
#pragma unroll
        for (int r = 0; r < RPT; ++r) {
          Sp[r] = pp[(size_t)(dg * RPT + r) * kNV + lane];
          Mp[r] = pp[(size_t)(DK + dg * RPT + r) * kNV + lane];
        }
      }
      if (tid == 0 && t < n - 1) {   // deta of the token processed before this one (its k . a partials are complete)
        float te = 0.f;
#pragma unroll
        for (int g8 = 0; g8 < kGroups; ++g8) te += scal[g8 * 4 + 3];
        a.part_g[(((size_t)cb * a.g.B * a.g.T + (tok0 + t + 1)) * H + h) * 4 + 3] = -te;
      }
      if (dg == 0) {
        a.dv_out[grow * DV + j] = dvt;
        const float dp = warp_sum(dvt * preds[t * kNV + lane]);
        if (lane == 0) {
          float tb = 0.f, ta = 0.f, tm = 0.f;
#pragma unroll
          for (int g8 = 0; g8 < kGroups; ++g8) { tb += scal[g8 * 4 + 0]; ta += scal[g8 * 4 + 1]; tm += scal[g8 * 4 + 2]; }
          float* pg = a.part_g + (((size_t)cb * a.g.B * a.g.T + (tok0 + t)) * H + h) * 4;
          pg[0] = -tb;              // dbeta
          pg[1] = al * (ta - dp);   // dlog_alpha
          pg[2] = mu * tm;          // dlog_mu
        }
      }
      __syncthreads();   // (2)
      float se = 0.f;
      if (rrow < DK) {
#pragma unroll
        for (int x = 0; x < kNV / 2; ++x) se += tileC[rrow * kLT + half * (kNV / 2) + x];
      }
      se += __shfl_xor_sync(0xffffffffu, se, 1);
      // deta = -k . a  (a = sb per row): rows live in lanes with half == 0; reduce over the block through scal
      float ke = 0.f;
      if (rrow < DK && half == 0) {
        const float krow = to_f32<TIn>(ks[t * DK + rrow]);
        const size_t pi = (((size_t)cb * a.g.B * a.g.T + (tok0 + t)) * H + h) * DK + rrow;
        a.part_q[pi] = a.scale * sa;
        a.part_k[pi] = -et * sb - al * se;
        ke = krow * sb;
      }
      ke = warp_sum(ke);
      if (lane == 0) scal[dg * 4 + 3] = ke;
#pragma unroll
      for (int r = 0; r < RPT; ++r) {
        GS[r] = al * (GS[r] - kr[r] * dvt);
        GM[r] *= mu;
      }
    }
    __syncthreads();   // k . a partials of the chunk's first token; tiles free for the next chunk
    if (tid == 0 && n > 0) {
      float te = 0.f;
#pragma unroll
      for (int g8 = 0; g8 < kGroups; ++g8) te += scal[g8 * 4 + 3];
      a.part_g[(((size_t)cb * a.g.B * a.g.T + tok0) * H + h) * 4 + 3] = -te;
    }
  }
#pragma unroll
  for (int r = 0; r < RPT; ++r) {
    const size_t i = st_off + (size_t)(dg * RPT + r) * DV + j;
    if (a.dS0) a.dS0[i] = GS[r];
    if (a.dM0) a.dM0[i] = GM[r];
  }
}

// Sums the column blocks' partial results in a fixed order.
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
  return (size_t)C * DK * sizeof(TIn) + sizeof(float) * ((size_t)4 * C * kNV + 4 * C + 2 * kGroups * kNV + 3 * DK * kLT + kGroups * 4);
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
  const uint64_t ncb = (uint64_t)p.dv / kNV, tokens = (uint64_t)p.B * p.T;
  const uint64_t chains = (uint64_t)(p.num_seqs > 0 ? p.num_seqs : p.B) * p.H;
  auto up = [](uint64_t x) { return (x + 255) / 256 * 256; };
  uint64_t off = 0;
  s->part_q = off; off = up(off + ncb * tokens * p.H * p.dk * 4);
  s->part_k = off; off = up(off + ncb * tokens * p.H * p.dk * 4);
  s->part_g = off; off = up(off + ncb * tokens * p.H * 4 * 4);
  s->ck = off; off = up(off + (uint64_t)num_slots * p.H * 2 * p.dk * p.dv * 4);
  s->prev = off; off = up(off + chains * C * 2 * p.dk * p.dv * 4);
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
