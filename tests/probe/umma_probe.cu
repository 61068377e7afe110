// Test-only bring-up probe for the sm_100a building blocks of the tensor-core kernels: one CTA runs
// one small tcgen05 / TMA case per mode so that descriptor, swizzle and TMEM-layout mistakes show
// up in isolation (checked against a host matmul by the tests).  Built into its own library
// (libmdn_probe.so) by tests/probe/build_probe.py; nothing of it is part of libmdn.so.
#include <cstring>

#include "mdn_common.cuh"
#include "mdn_probe.h"
#include "tc_utils.cuh"

namespace mdn {

namespace {

using namespace tc;

// A [rows x cols] row-major bf16 matrix -> K-major SW128 blocks of 64 columns ([rows x 128 B] each).
__device__ void fill_kmajor(uint8_t* dst, const __nv_bfloat16* src, int rows, int cols, int tid, int nthr) {
  for (int idx = tid; idx < rows * cols; idx += nthr) {
    const int r = idx / cols, c = idx % cols;
    const uint32_t off = (c / 64) * rows * 128 + sw128_offset(r, c % 64);
    *reinterpret_cast<__nv_bfloat16*>(dst + off) = src[idx];
  }
}

__global__ void __launch_bounds__(128) umma_probe_kernel(int mode, const __nv_bfloat16* __restrict__ a,
                                                        const __nv_bfloat16* __restrict__ b, float* __restrict__ out,
                                                        int32_t* __restrict__ status,
                                                        const __grid_constant__ CUtensorMap map) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;                 // up to 32 KB
  uint8_t* sB = smem + 32768;         // up to 16 KB
  __shared__ __align__(8) uint64_t bars[2];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5;
  const uint32_t bar_tma = smem_u32(&bars[0]), bar_mma = smem_u32(&bars[1]);

  if (tid == 0) {
    abort_flag = 0;
    mbar_init(bar_tma, 1);
    mbar_init(bar_mma, 1);
    mbar_fence_init();
  }
  if (warp == 0) tmem_alloc(smem_u32(&tmem_slot), 256);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = tmem_slot;
  const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
  bool ok = true;

  if (mode == 0) {            // TMA SW128 layout: [64 x 128] bf16 as two [64 x 64] boxes
    if (tid == 0) {
      mbar_arrive_expect_tx(bar_tma, 16384);
      tma_load_2d(smem_u32(sA), &map, 0, 0, bar_tma);
      tma_load_2d(smem_u32(sA) + 8192, &map, 64, 0, bar_tma);
    }
    ok = mbar_wait(bar_tma, 0, &abort_flag);
    if (ok)
      for (int i = tid; i < 4096; i += 128) reinterpret_cast<uint32_t*>(out)[i] = reinterpret_cast<uint32_t*>(sA)[i];
  } else if (mode == 1) {     // SS: D[128x64] = A[128x128] * B[64x128]^T, both K-major in smem
    fill_kmajor(sA, a, 128, 128, tid, 128);
    fill_kmajor(sB, b, 64, 128, tid, 128);
    fence_proxy_async_smem();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after_sync();
      const uint32_t id = idesc_bf16(128, 64, false, false, false);
      for (int k = 0; k < 8; ++k) {
        const uint64_t da = smem_desc_sw128(smem_u32(sA) + (k / 4) * 16384 + (k % 4) * 32, 16, 1024);
        const uint64_t db = smem_desc_sw128(smem_u32(sB) + (k / 4) * 8192 + (k % 4) * 32, 16, 1024);
        umma_ss(tmem, da, db, id, k > 0);
      }
      umma_commit(bar_mma);
    }
    ok = mbar_wait(bar_mma, 0, &abort_flag);
    __syncwarp();
    tc_fence_after_sync();
    if (ok) {
      for (int c0 = 0; c0 < 64; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(tmem + lane_base + c0, r);
        tmem_wait_ld();
        for (int j = 0; j < 32; ++j) out[tid * 64 + c0 + j] = __uint_as_float(r[j]);
      }
    }
  } else if (mode == 5) {     // SS with M = 64 and an MN-major B: D[64x128] = A[64x128] * B[128x128], B a kept chunk state
    // B[j][d] (value index j = K, key index d = N) lies as the chain kernel keeps a state: two blocks (d halves) of
    // [128 rows j][64 d], 128-byte swizzle; read MN-major it needs no transposition.  out[64 x 128], rows from the
    // lanes the M = 64 data path uses
    fill_kmajor(sB, a, 64, 128, tid, 128);
    fill_kmajor(sA, b, 128, 128, tid, 128);
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after_sync();
      const uint32_t id = idesc_bf16(64, 128, false, true, false);
      for (int k = 0; k < 8; ++k) {
        const uint64_t da = smem_desc_sw128(smem_u32(sB) + (k / 4) * 8192 + (k % 4) * 32, 16, 1024);
        const uint64_t db = smem_desc_sw128(smem_u32(sA) + k * 2048, 16384, 1024);   // 16 rows of j per K step
        umma_ss(tmem, da, db, id, k > 0);
      }
      umma_commit(bar_mma);
    }
    ok = mbar_wait(bar_mma, 0, &abort_flag);
    __syncwarp();
    tc_fence_after_sync();
    if (ok) {
      for (int c0 = 0; c0 < 128; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(tmem + lane_base + c0, r);
        tmem_wait_ld();
        if ((tid & 31) < 16)
          for (int j = 0; j < 32; ++j) out[(16 * warp + (tid & 31)) * 128 + c0 + j] = __uint_as_float(r[j]);
      }
    }
  } else if (mode == 4) {     // SS with M = 64: D[64x128] = A[64x128] * B[128x128]^T; out = all 128 lanes x 128 columns
    // tensor memory is filled with a sentinel first, so the lanes the 64 rows land in can be read off the result
    {
      uint32_t r[32];
      for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(-777.0f);
      for (int c0 = 0; c0 < 128; c0 += 32) tmem_st32(tmem + lane_base + c0, r);
      tmem_wait_st();
    }
    fill_kmajor(sB, a, 64, 128, tid, 128);    // A: two [64 x 64] blocks (16 KB) in the smaller area
    fill_kmajor(sA, b, 128, 128, tid, 128);   // B: two [128 x 64] blocks (32 KB)
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after_sync();
      const uint32_t id = idesc_bf16(64, 128, false, false, false);
      for (int k = 0; k < 8; ++k) {
        const uint64_t da = smem_desc_sw128(smem_u32(sB) + (k / 4) * 8192 + (k % 4) * 32, 16, 1024);
        const uint64_t db = smem_desc_sw128(smem_u32(sA) + (k / 4) * 16384 + (k % 4) * 32, 16, 1024);
        umma_ss(tmem, da, db, id, k > 0);
      }
      umma_commit(bar_mma);
    }
    ok = mbar_wait(bar_mma, 0, &abort_flag);
    __syncwarp();
    tc_fence_after_sync();
    if (ok) {
      for (int c0 = 0; c0 < 128; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(tmem + lane_base + c0, r);
        tmem_wait_ld();
        for (int j = 0; j < 32; ++j) out[tid * 128 + c0 + j] = __uint_as_float(r[j]);
      }
    }
  } else if (mode == 2 || mode == 3) {
    // A [128 x 64] bf16 -> TMEM columns 128..159, two elements per column (even k in the low half)
    {
      uint32_t r[32];
      for (int j = 0; j < 32; ++j) {
        const __nv_bfloat162 v = __halves2bfloat162(a[tid * 64 + 2 * j], a[tid * 64 + 2 * j + 1]);
        r[j] = *reinterpret_cast<const uint32_t*>(&v);
      }
      tmem_st32(tmem + lane_base + 128, r);
      tmem_wait_st();
    }
    if (mode == 2) {          // TS: D[128x64] = A * B[64x64]^T, B K-major
      fill_kmajor(sB, b, 64, 64, tid, 128);
      fence_proxy_async_smem();
      tc_fence_before_sync();
      __syncthreads();
      if (tid == 0) {
        tc_fence_after_sync();
        const uint32_t id = idesc_bf16(128, 64, false, false, false);
        for (int k = 0; k < 4; ++k)
          umma_ts(tmem, tmem + 128 + k * 8, smem_desc_sw128(smem_u32(sB) + k * 32, 16, 1024), id, k > 0);
        umma_commit(bar_mma);
      }
      ok = mbar_wait(bar_mma, 0, &abort_flag);
      __syncwarp();
      tc_fence_after_sync();
      if (ok) {
        for (int c0 = 0; c0 < 64; c0 += 32) {
          uint32_t r[32];
          tmem_ld32(tmem + lane_base + c0, r);
          tmem_wait_ld();
          for (int j = 0; j < 32; ++j) out[tid * 64 + c0 + j] = __uint_as_float(r[j]);
        }
      }
    } else {                  // TS: D[128x128] = 1 - A[128 x 64 tok] * Kt[64 tok x 128], Kt by TMA, MN-major B
      {
        uint32_t r[32];
        for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(1.0f);
        for (int c0 = 0; c0 < 128; c0 += 32) tmem_st32(tmem + lane_base + c0, r);
        tmem_wait_st();
      }
      if (tid == 0) {
        mbar_arrive_expect_tx(bar_tma, 16384);
        tma_load_2d(smem_u32(sB), &map, 0, 0, bar_tma);
        tma_load_2d(smem_u32(sB) + 8192, &map, 64, 0, bar_tma);
      }
      tc_fence_before_sync();
      __syncthreads();
      if (tid == 0) {
        ok = mbar_wait(bar_tma, 0, &abort_flag);
        if (ok) {
          tc_fence_after_sync();
          const uint32_t id = idesc_bf16(128, 128, false, true, true);
          for (int k = 0; k < 4; ++k)
            umma_ts(tmem, tmem + 128 + k * 8, smem_desc_sw128(smem_u32(sB) + k * 2048, 8192, 1024), id, true);
          umma_commit(bar_mma);
        }
      }
      ok = mbar_wait(bar_mma, 0, &abort_flag);
      __syncwarp();
      tc_fence_after_sync();
      if (ok) {
        for (int c0 = 0; c0 < 128; c0 += 32) {
          uint32_t r[32];
          tmem_ld32(tmem + lane_base + c0, r);
          tmem_wait_ld();
          for (int j = 0; j < 32; ++j) out[tid * 128 + c0 + j] = __uint_as_float(r[j]);
        }
      }
    }
  }
  if (!ok && tid == 0) atomicCAS(status, kDevOk, kDevTimeout);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 256);
}

}  // namespace
}  // namespace mdn

extern "C" mdn_status mdn_selftest_umma(int32_t mode, const void* a, const void* b, float* out, int32_t* status,
                                        void* cuda_stream) {
  using namespace mdn;
  if (mode < 0 || mode > 5 || !a || !out || !status || (mode != 0 && !b)) return MDN_ERR_INVALID_ARG;
  CUtensorMap map;
  std::memset(&map, 0, sizeof(map));
  const void* tma_src = mode == 3 ? b : a;      // [64 x 128] bf16
  if (!encode_tma_2d_bf16(&map, TmaMap2D{tma_src, 128, 64, 256, 64, 64, true})) return MDN_ERR_CUDA;
  const int smem = 49152 + 1024;
  if (cudaFuncSetAttribute(umma_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
    return MDN_ERR_CUDA;
  umma_probe_kernel<<<1, 128, smem, static_cast<cudaStream_t>(cuda_stream)>>>(
      mode, static_cast<const __nv_bfloat16*>(a), static_cast<const __nv_bfloat16*>(b), out, status, map);
  return cudaGetLastError() == cudaSuccess ? MDN_OK : MDN_ERR_CUDA;
}
