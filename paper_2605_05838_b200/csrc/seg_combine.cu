// Serial combine step of the parallel inter-chunk scan: for every chain, walk its middle segments in order,
//     [S; M]_g = Phi_g [S; M]_{g-1} + Psi_g          (state at the END of segment g = start of segment g + 1)
// with Phi_g = [Phi_SS Phi_SM; Phi_MS Phi_MM] assembled from the two basis runs of the segment (from (I, 0): the
// column blocks Phi_SS, Phi_MS; from (0, I): Phi_SM, Phi_MM) and Psi_g the run from a zero state.  fp32 FMAs: this is
// (G - 2) products of a 256 x 256 by a 256 x dv matrix per chain, a few percent of the segment runs themselves.
//
// grid = (chains, dv / 16); block = 256 threads: thread i owns row i of the stacked state (i < 128: S, else M) for
// 16 value columns.  The previous state's 256 x 16 slice sits in shared memory (read as broadcasts); Phi streams
// through shared memory in 256 x 16 tiles loaded with coalesced float4 reads (next tile prefetched into registers).
#include "mdn_common.cuh"

namespace mdn {
namespace {

constexpr int kD = 128, kCols = 16, kThreads = 2 * kD, kMT = 16, kPad = kMT + 1;

__global__ void __launch_bounds__(kThreads) seg_combine_kernel(int G, float* __restrict__ E,
                                                              const float* __restrict__ Psi,
                                                              const float* __restrict__ PhiS,
                                                              const float* __restrict__ PhiM) {
  __shared__ __align__(16) float prev[2 * kD][kCols];
  __shared__ float phi_t[2 * kD][kPad];
  constexpr size_t kMat = (size_t)kD * kD;
  const int chain = blockIdx.x, j0 = blockIdx.y * kCols;
  const int i = threadIdx.x, half = i >> 7, row = i & (kD - 1);   // half 0: S rows, 1: M rows
  float* e_chain = E + (size_t)chain * (G - 1) * 2 * kMat;
  {  // state at the end of segment 0 (written by its real run)
    const float4* src = reinterpret_cast<const float4*>(e_chain + (size_t)half * kMat + (size_t)row * kD + j0);
#pragma unroll
    for (int c4 = 0; c4 < kCols / 4; ++c4) *reinterpret_cast<float4*>(&prev[i][c4 * 4]) = src[c4];
  }
  // tile loader: element f = i + 256 x covers stacked row f / 4, floats (f % 4) * 4 .. + 3 of the 16-wide tile
  auto tile_src = [&](size_t seg_off, int mt, int x) {
    const int f = i + kThreads * x, r = f >> 2, q4 = f & 3;
    const int m = mt * kMT;                                 // stacked column of the previous state
    const float* base = (m < kD ? PhiS : PhiM) + seg_off;
    return reinterpret_cast<const float4*>(base + (size_t)(r >> 7) * kMat + (size_t)(r & (kD - 1)) * kD + (m & (kD - 1)) +
                                           q4 * 4);
  };
  __syncthreads();
  for (int g = 1; g <= G - 2; ++g) {
    const size_t seg_off = ((size_t)chain * (G - 2) + (g - 1)) * 2 * kMat;
    float acc[kCols];
    {
      const float4* psi = reinterpret_cast<const float4*>(Psi + seg_off + (size_t)half * kMat + (size_t)row * kD + j0);
#pragma unroll
      for (int c4 = 0; c4 < kCols / 4; ++c4) {
        const float4 t = psi[c4];
        acc[c4 * 4] = t.x; acc[c4 * 4 + 1] = t.y; acc[c4 * 4 + 2] = t.z; acc[c4 * 4 + 3] = t.w;
      }
    }
    float4 nxt[4];
#pragma unroll
    for (int x = 0; x < 4; ++x) nxt[x] = *tile_src(seg_off, 0, x);
    constexpr int kTiles = 2 * kD / kMT;
#pragma unroll 1
    for (int mt = 0; mt < kTiles; ++mt) {
      __syncthreads();   // previous tile consumed
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        const int f = i + kThreads * x, r = f >> 2, q4 = f & 3;
        phi_t[r][q4 * 4 + 0] = nxt[x].x; phi_t[r][q4 * 4 + 1] = nxt[x].y;
        phi_t[r][q4 * 4 + 2] = nxt[x].z; phi_t[r][q4 * 4 + 3] = nxt[x].w;
      }
      __syncthreads();
      if (mt + 1 < kTiles) {
#pragma unroll
        for (int x = 0; x < 4; ++x) nxt[x] = *tile_src(seg_off, mt + 1, x);
      }
#pragma unroll
      for (int mm = 0; mm < kMT; ++mm) {
        const float f = phi_t[i][mm];
        const float4* pr = reinterpret_cast<const float4*>(prev[mt * kMT + mm]);
#pragma unroll
        for (int c4 = 0; c4 < kCols / 4; ++c4) {
          const float4 pv = pr[c4];
          acc[c4 * 4 + 0] = fmaf(f, pv.x, acc[c4 * 4 + 0]);
          acc[c4 * 4 + 1] = fmaf(f, pv.y, acc[c4 * 4 + 1]);
          acc[c4 * 4 + 2] = fmaf(f, pv.z, acc[c4 * 4 + 2]);
          acc[c4 * 4 + 3] = fmaf(f, pv.w, acc[c4 * 4 + 3]);
        }
      }
    }
    float4* out = reinterpret_cast<float4*>(e_chain + ((size_t)g * 2 + half) * kMat + (size_t)row * kD + j0);
    __syncthreads();   // everyone is done reading the previous state
#pragma unroll
    for (int c4 = 0; c4 < kCols / 4; ++c4) {
      const float4 t = make_float4(acc[c4 * 4], acc[c4 * 4 + 1], acc[c4 * 4 + 2], acc[c4 * 4 + 3]);
      out[c4] = t;
      *reinterpret_cast<float4*>(&prev[i][c4 * 4]) = t;
    }
    __syncthreads();
  }
}

}  // namespace

cudaError_t launch_seg_combine(const Plan& pl, int G, float* E, const float* Psi, const float* PhiS,
                               const float* PhiM, int* launches) {
  const dim3 grid((unsigned)pl.geom.num_seqs * pl.p.H, kD / kCols);
  seg_combine_kernel<<<grid, kThreads, 0, pl.stream>>>(G, E, Psi, PhiS, PhiM);
  const cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) ++*launches;
  return e;
}

}  // namespace mdn
