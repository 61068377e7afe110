// a0: chunk map from cu_seqlens (integer work, no host sync needed).
// a1: per-chunk coefficient scan (Eq. 10), division-free and fp32.
//
// The paper evaluates c_t = sum_i beta_i mubar_i / abar_i in the log domain because the
// ratio mubar_i/abar_i overflows inside a chunk.  The same coefficients follow from
// first-order linear recurrences whose multipliers all lie in [0,1]:
//     abar_r  = alpha_r abar_{r-1}                  mubar_r = mu_r mubar_{r-1}
//     b_r     = alpha_r b_{r-1} + beta_r mubar_r                       (b_{-1} = 0)
//     gamma_{last,i} = A_i beta_i + mu_{i+1} gamma_{last,i+1},  A_i = prod_{l>i} alpha_l
//     mubar_last/mubar_i = prod_{l>i} mu_l
// (expand gamma_{t,i} = abar_t/mubar_i (c_t - c_{i-1}) = sum_{j=i..t} (abar_t/abar_j) beta_j (mubar_j/mubar_i)).
// No logarithm of beta, no division: beta = 0 and mu = 0 give exact zeros.
// Each recurrence is an affine scan evaluated with warp shuffles: one warp per
// (chunk, head), two consecutive positions per lane.
#include "coeff_scan.cuh"
#include "mdn_common.cuh"

namespace mdn {

// ------------------------------------------------------------------------------------ a0
// One CTA.  Validates cu_seqlens (cu[0] = 0, non-decreasing, cu[N] = T), computes the
// chunk count of every sequence, its exclusive prefix sum, and the slot map.
__global__ void __launch_bounds__(1024) chunk_map_kernel(const int32_t* __restrict__ cu, int num_seqs, int T,
                                                        int num_slots, int32_t* __restrict__ chunk_off,
                                                        int32_t* __restrict__ slot_map,
                                                        int32_t* __restrict__ status) {
  __shared__ int s_scan[1024];
  __shared__ int s_carry;
  __shared__ int s_bad;
  const int tid = threadIdx.x;
  if (tid == 0) { s_carry = 0; s_bad = 0; }
  if (tid < 4) status[tid] = 0;   // the call's status word starts clean (this is the call's first kernel)
  __syncthreads();
  // T < 0: the total may fall short of -T (the caller pads its problem to a bound)
  if (tid == 0 && (cu[0] != 0 || (T >= 0 ? cu[num_seqs] != T : cu[num_seqs] > -T))) s_bad = 1;
  for (int base = 0; base < num_seqs; base += 1024) {
    const int i = base + tid;
    int nch = 0;
    if (i < num_seqs) {
      const int len = cu[i + 1] - cu[i];
      if (len < 0) { s_bad = 1; } else { nch = (len + C - 1) / C; }
    }
    s_scan[tid] = nch;
    __syncthreads();
    for (int off = 1; off < 1024; off <<= 1) {   // inclusive Hillis-Steele scan
      const int add = (tid >= off) ? s_scan[tid - off] : 0;
      __syncthreads();
      s_scan[tid] += add;
      __syncthreads();
    }
    const int carry = s_carry;
    if (i < num_seqs) chunk_off[i] = carry + s_scan[tid] - nch;
    __syncthreads();
    if (tid == 1023) s_carry = carry + s_scan[1023];
    __syncthreads();
  }
  const int total = s_carry;
  if (tid == 0) {
    chunk_off[num_seqs] = total;
    if (total > num_slots) s_bad = 1;
  }
  __syncthreads();
  if (s_bad) {
    if (tid == 0) atomicCAS(status, kDevOk, kDevBadCuSeqlens);
    // leave a map that makes every later kernel a no-op
    for (int s = tid; s < num_slots; s += 1024)
      reinterpret_cast<int4*>(slot_map)[s] = make_int4(-1, 0, 0, 0);
    for (int i = tid; i <= num_seqs; i += 1024) chunk_off[i] = 0;
    return;
  }
  for (int s = total + tid; s < num_slots; s += 1024)
    reinterpret_cast<int4*>(slot_map)[s] = make_int4(-1, 0, 0, 0);
  for (int i = tid; i < num_seqs; i += 1024) {
    const int t0 = cu[i], len = cu[i + 1] - t0, s0 = chunk_off[i];
    const int nch = (len + C - 1) / C;
    for (int c = 0; c < nch; ++c)
      reinterpret_cast<int4*>(slot_map)[s0 + c] = make_int4(i, t0 + c * C, min(C, len - c * C), c);
  }
}

// Fixed-length input has no chunk map to build: the call's first kernel only clears the status word.  A kernel rather
// than a memset node so that the next kernel's launch overlaps it (programmatic dependent launch).
__global__ void status_clear_kernel(int32_t* __restrict__ status) {
  grid_dependency_wait();
  if (threadIdx.x < 4) status[threadIdx.x] = 0;
}

cudaError_t launch_chunk_map(const Plan& pl, int* launches) {
  if (pl.geom.cu == nullptr) {
    ++*launches;
    return launch_pdl(status_clear_kernel, dim3(1), dim3(32), 0, pl.stream, reinterpret_cast<int32_t*>(pl.ws + pl.lay.off_status));
  }
  chunk_map_kernel<<<1, 1024, 0, pl.stream>>>(pl.geom.cu, pl.geom.num_seqs, pl.cu_total_may_be_short ? -pl.p.T : pl.p.T,
                                              pl.geom.num_slots,
                                              const_cast<int32_t*>(pl.geom.chunk_off),
                                              const_cast<int32_t*>(pl.geom.slot_map),
                                              reinterpret_cast<int32_t*>(pl.ws + pl.lay.off_status));
  ++*launches;
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------ a1
constexpr int kScanWarps = 8;

// grid = chunk slots; block = 8 warps.  The [n x H] block of each gate is one contiguous
// span in memory: staged through shared memory with coalesced (128-bit when aligned)
// loads, then each warp scans one head at a time.
__global__ void __launch_bounds__(kScanWarps * 32) coeff_scan_kernel(ChunkGeom g, const float* __restrict__ beta,
                                                                    const float* __restrict__ log_alpha,
                                                                    const float* __restrict__ log_mu,
                                                                    const float* __restrict__ eta, GateParam gp,
                                                                    float* __restrict__ coef) {
  extern __shared__ float sm[];   // [4][64*H]: log_alpha, log_mu, beta, eta
  const int slot = blockIdx.x;
  grid_dependency_wait();   // the chunk map (packed input) comes from the previous kernel
  const SlotInfo si = slot_info(g, slot);
  if (si.seq < 0) return;
  const int H = g.H, tid = threadIdx.x;
  const int span = si.n * H;
  const size_t base = (size_t)si.tok0 * H;
  const float* src[4] = {log_alpha + base, log_mu + base, beta + base, eta ? eta + base : nullptr};
#pragma unroll
  for (int a = 0; a < 4; ++a) {
    float* dst = sm + a * C * H;
    if (src[a] == nullptr) {
      for (int i = tid; i < span; i += blockDim.x) dst[i] = 1.0f;
    } else if ((reinterpret_cast<uintptr_t>(src[a]) & 15) == 0 && (span & 3) == 0) {
      const float4* s4 = reinterpret_cast<const float4*>(src[a]);
      for (int i = tid; i < span / 4; i += blockDim.x) reinterpret_cast<float4*>(dst)[i] = __ldg(s4 + i);
    } else {
      for (int i = tid; i < span; i += blockDim.x) dst[i] = __ldg(src[a] + i);
    }
  }
  __syncthreads();

  const int warp = tid >> 5, lane = tid & 31;
  const int r0 = 2 * lane;
  for (int h = warp; h < H; h += kScanWarps) {
    // exact no-ops past the end of a short chunk: alpha = mu = 1, beta = eta = 0
    float al[2], mu[2], be[2], et[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int r = r0 + e;
      al[e] = mu[e] = 1.0f;
      be[e] = et[e] = 0.0f;
      if (r < si.n) {
        const TokenGates tg = load_token_gates(gp, h, sm[0 * C * H + r * H + h], sm[1 * C * H + r * H + h],
                                               sm[2 * C * H + r * H + h], sm[3 * C * H + r * H + h]);
        al[e] = tg.alpha; mu[e] = tg.mu; be[e] = tg.beta; et[e] = tg.eta;
      }
    }
    const HeadCoefs hc = scan_head(al, mu, be, et, lane);
    float* out = coef + ((size_t)slot * H + h) * MDN_NUM_COEF * C;
    auto put = [&](int which, float x0, float x1) {
      reinterpret_cast<float2*>(out + which * C)[lane] = make_float2(x0, x1);
    };
    put(kAbar, hc.abar[0], hc.abar[1]);
    put(kB, hc.b[0], hc.b[1]);
    put(kAlphaBPrev, hc.ab_prev[0], hc.ab_prev[1]);
    put(kGS, hc.gs[0], hc.gs[1]);
    put(kGM, hc.gm[0], hc.gm[1]);
    put(kAlpha, al[0], al[1]);
    put(kBeta, be[0], be[1]);
    put(kMu, mu[0], mu[1]);
    put(kEta, et[0], et[1]);
    put(kMubar, hc.mubar[0], hc.mubar[1]);
    put(kRk, 1.0f, 1.0f);
    put(kRq, 1.0f, 1.0f);
  }
  grid_launch_dependents();
}

cudaError_t launch_coeff_scan(const Plan& pl, const float* beta, const float* log_alpha, const float* log_mu,
                              const float* eta, int* launches) {
  const size_t smem = (size_t)4 * C * pl.p.H * sizeof(float);
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(coeff_scan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  coeff_scan_kernel<<<pl.geom.num_slots, kScanWarps * 32, smem, pl.stream>>>(
      pl.geom, beta, log_alpha, log_mu, eta, pl.gp, reinterpret_cast<float*>(pl.ws + pl.lay.off_coef));
  ++*launches;
  return cudaGetLastError();
}

}  // namespace mdn
