// Warp-level bf16 tensor-core products (mma.sync m16n8k16, fp32 accumulate) on operands in shared memory, fed by
// ldmatrix; used by the kernels of the chunk-parallel backward.
#pragma once
#include <cstdint>

namespace mdn {

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// A bf16 operand in shared memory: byte address of element (0, 0), row stride in bytes, and how it is stored:
// for A, trans = false means [m][k] (k contiguous), true means [k][m]; for B, false means [n][k], true means [k][n].
// swz: the operand is a raw 128-byte-swizzled image instead ([.. x 128] bf16 as two blocks of [rows][64 columns],
// 128-byte rows, 16384 bytes per block, the 16-byte piece index XORed with row mod 8); ld is then unused.
struct Opnd { uint32_t base; uint32_t ld; bool trans; bool swz = false; };

// byte address of the 8-element row segment (row, col .. col + 7), col a multiple of 8
__device__ __forceinline__ uint32_t opnd_addr(const Opnd& o, int row, int col) {
  if (!o.swz) return o.base + row * o.ld + col * 2;
  return o.base + (col >> 6) * 16384 + row * 128 + ((((col >> 3) ^ row) & 7) << 4);
}

// acc[mt][nt] += A[m0 + 16 mt .., k] B[k, n0 + 8 nt ..] over k < K (a multiple of 16); NT even.
template <int MT, int NT>
__device__ __forceinline__ void warp_mma(float (&acc)[MT][NT][4], Opnd A, Opnd B, int K, int m0, int n0, int lane) {
  const int l7 = lane & 7, q1 = (lane >> 3) & 1, q2 = lane >> 4;
  for (int k0 = 0; k0 < K; k0 += 16) {
    uint32_t af[MT][4], bfr[NT / 2][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      if (!A.trans) ldsm_x4(opnd_addr(A, m0 + 16 * mt + l7 + q1 * 8, k0 + q2 * 8), af[mt]);
      else ldsm_x4_t(opnd_addr(A, k0 + q2 * 8 + l7, m0 + 16 * mt + q1 * 8), af[mt]);
    }
#pragma unroll
    for (int p = 0; p < NT / 2; ++p) {
      if (!B.trans) ldsm_x4(opnd_addr(B, n0 + 16 * p + l7 + q2 * 8, k0 + q1 * 8), bfr[p]);
      else ldsm_x4_t(opnd_addr(B, k0 + q1 * 8 + l7, n0 + 16 * p + q2 * 8), bfr[p]);
    }
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int p = 0; p < NT / 2; ++p) {
        mma_bf16(acc[mt][2 * p], af[mt], bfr[p][0], bfr[p][1]);
        mma_bf16(acc[mt][2 * p + 1], af[mt], bfr[p][2], bfr[p][3]);
      }
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
// ... and its column pairs: f(mt, nt, half, row, col) with the values acc[mt][nt][2 half], [2 half + 1] at col, col + 1
template <int MT, int NT, class F> __device__ __forceinline__ void for_pair(int m0, int n0, int g, int t, F f) {
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) f(mt, nt, hf, m0 + 16 * mt + g + 8 * hf, n0 + 8 * nt + 2 * t);
}


}  // namespace mdn
