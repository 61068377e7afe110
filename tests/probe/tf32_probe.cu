// Test-only probes of the kind::tf32 tcgen05 forms (fp32 operands read as tf32): A from tensor memory against a
// K-major or an MN-major fp32 tile in shared memory, a product whose A operand is the accumulator of the product
// issued just before it, issue-to-completion timings, and a bounded wait that is made to run out.
// One CTA of 128 threads per call; part of libmdn_probe.so only.
#include <cstring>

#include "mdn_common.cuh"
#include "mdn_probe.h"
#include "tc_utils.cuh"

namespace mdn {
namespace {

using namespace tc;

// A [rows x cols] row-major fp32 matrix -> blocks of 32 columns ([rows x 128 B] each, 128-byte swizzle).
__device__ void fill_f32_blocks(uint8_t* dst, const float* src, int rows, int cols, int tid, int nthr) {
  for (int idx = tid; idx < rows * cols; idx += nthr) {
    const int r = idx / cols, c = idx % cols;
    *reinterpret_cast<float*>(dst + (c / 32) * rows * 128 + sw128_offset_f32(r, c % 32)) = src[idx];
  }
}

__global__ void __launch_bounds__(128) tf32_probe_kernel(int mode, const float* __restrict__ a, const float* __restrict__ b,
                                                        const float* __restrict__ c, float* __restrict__ out,
                                                        int32_t* __restrict__ status) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sB = smem;                 // [64 x 128] fp32: four [64 x 32] blocks, 32 KB
  uint8_t* sT = smem + 32768;         // [64 x 64] fp32: two [64 x 32] blocks, 16 KB
  __shared__ __align__(8) uint64_t bars[2];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5;
  const uint32_t bar_a = smem_u32(&bars[0]), bar_b = smem_u32(&bars[1]);
  if (tid == 0) {
    abort_flag = 0;
    mbar_init(bar_a, 1);
    mbar_init(bar_b, 1);
    mbar_fence_init();
  }
  if (warp == 0) tmem_alloc(smem_u32(&tmem_slot), 256);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = tmem_slot;
  const uint32_t tl = tmem + (static_cast<uint32_t>(warp * 32) << 16);
  bool ok = true;
  constexpr uint32_t kColA = 0, kColX = 128, kColY = 192;

  auto store_rows = [&](const float* src, int cols, uint32_t col0) {   // this thread's row of src -> its lane
    for (int c0 = 0; c0 < cols; c0 += 32) {
      uint32_t r[32];
      for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(src[tid * cols + c0 + j]);
      tmem_st32(tl + col0 + c0, r);
    }
    tmem_wait_st();
  };
  auto fill_cols = [&](float x, int cols, uint32_t col0) {
    uint32_t r[32];
    for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(x);
    for (int c0 = 0; c0 < cols; c0 += 32) tmem_st32(tl + col0 + c0, r);
    tmem_wait_st();
  };
  auto read_rows = [&](int cols, uint32_t col0) {
    for (int c0 = 0; c0 < cols; c0 += 32) {
      uint32_t r[32];
      tmem_ld32(tl + col0 + c0, r);
      tmem_wait_ld();
      for (int j = 0; j < 32; ++j) out[tid * cols + c0 + j] = __uint_as_float(r[j]);
    }
  };
  // X[128 x 64] (+)= A[128 x 128] (tensor memory) * B[64 x 128]^T (K-major blocks): 16 K steps of 8
  auto issue_x = [&](bool accumulate) {
    const uint32_t id = idesc_tf32(128, 64, false, false, false);
    for (int k = 0; k < 16; ++k)
      umma_ts_tf32(tmem + kColX, tmem + kColA + 8 * k, smem_desc_sw128(smem_u32(sB) + (k / 4) * 8192 + (k % 4) * 32, 16, 1024), id,
                   accumulate || k > 0);
  };

  if (mode == 0) {            // out[128 x 64] = a[128 x 128] * b[64 x 128]^T
    store_rows(a, 128, kColA);
    fill_f32_blocks(sB, b, 64, 128, tid, 128);
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after_sync();
      issue_x(false);
      umma_commit(bar_a);
    }
    ok = mbar_wait(bar_a, 0, &abort_flag);
    __syncwarp();
    tc_fence_after_sync();
    if (ok) read_rows(64, kColX);
  } else if (mode == 1) {     // out[128 x 128] = a[128 x 64] * b[64 x 128], b read MN-major (N = its 128 columns, K = its rows)
    store_rows(a, 64, kColA);
    fill_f32_blocks(sB, b, 64, 128, tid, 128);
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after_sync();
      const uint32_t id = idesc_tf32(128, 128, false, true, false);
      for (int k = 0; k < 8; ++k)   // eight rows of b per K step = one 1024-byte atom; 8192 bytes to the next 32 columns
        umma_ts_tf32(tmem + kColX, tmem + kColA + 8 * k, smem_desc_sw128(smem_u32(sB) + k * 1024, 8192, 1024), id, k > 0);
      umma_commit(bar_a);
    }
    ok = mbar_wait(bar_a, 0, &abort_flag);
    __syncwarp();
    tc_fence_after_sync();
    if (ok) read_rows(128, kColX);
  } else if (mode == 2 || mode == 3) {
    // out[128 x 64] = (a[128 x 128] * b[64 x 128]^T) * c[64 x 64]^T: the second product reads the first one's
    // accumulator as its A operand.  mode 2 issues it right behind the first; mode 3 waits for the first to complete.
    store_rows(a, 128, kColA);
    fill_cols(1000.f, 64, kColX);    // a stale read would show
    fill_f32_blocks(sB, b, 64, 128, tid, 128);
    fill_f32_blocks(sT, c, 64, 64, tid, 128);
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after_sync();
      issue_x(false);
      if (mode == 3) {
        umma_commit(bar_b);
        ok = mbar_wait(bar_b, 0, &abort_flag);
        tc_fence_after_sync();
      }
      if (ok) {
        const uint32_t id = idesc_tf32(128, 64, false, false, false);
        for (int k = 0; k < 8; ++k)
          umma_ts_tf32(tmem + kColY, tmem + kColX + 8 * k, smem_desc_sw128(smem_u32(sT) + (k / 4) * 8192 + (k % 4) * 32, 16, 1024), id,
                       k > 0);
      }
      umma_commit(bar_a);
    }
    ok = mbar_wait(bar_a, 0, &abort_flag) && ok;
    __syncwarp();
    tc_fence_after_sync();
    if (ok) read_rows(64, kColY);
  } else if (mode >= 4 && mode <= 7) {
    // timings (clock64 on the issuing thread, first issue to completion of the last product); operands are whatever
    // the fills below leave.  out[0] = cycles, out[1] = products issued.
    //   4: tf32, A tensor memory, N = 64, K-major B        5: tf32, A tensor memory, N = 128, MN-major B
    //   6: bf16, A and B shared memory, N = 64 (kind::f16)  7: as 4, every group of 16 followed by commit + wait
    fill_cols(0.5f, 128, kColA);
    for (int i = tid; i < 49152 / 4; i += 128) reinterpret_cast<uint32_t*>(smem)[i] = 0x3c003c00u;
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    constexpr int kReps = 64;
    if (tid == 0) {
      tc_fence_after_sync();
      const long long t0 = clock64();
      int n = 0;
      for (int rep = 0; rep < kReps && ok; ++rep) {
        if (mode == 4 || mode == 7) {
          issue_x(false);
          n += 16;
          if (mode == 7) {
            umma_commit(bar_b);
            ok = mbar_wait(bar_b, rep & 1, &abort_flag);
            tc_fence_after_sync();
          }
        } else if (mode == 5) {
          const uint32_t id = idesc_tf32(128, 128, false, true, false);
          for (int k = 0; k < 8; ++k)
            umma_ts_tf32(tmem + kColX, tmem + kColA + 8 * k, smem_desc_sw128(smem_u32(sB) + k * 1024, 8192, 1024), id, k > 0);
          n += 8;
        } else {
          const uint32_t id = idesc_bf16(128, 64, false, false, false);
          for (int k = 0; k < 8; ++k)
            umma_ss(tmem + kColX, smem_desc_sw128(smem_u32(smem) + (k / 4) * 16384 + (k % 4) * 32, 16, 1024),
                    smem_desc_sw128(smem_u32(smem) + 32768 + (k / 4) * 8192 + (k % 4) * 32, 16, 1024), id, k > 0);
          n += 8;
        }
      }
      umma_commit(bar_a);
      ok = mbar_wait(bar_a, 0, &abort_flag) && ok;
      const long long t1 = clock64();
      out[0] = static_cast<float>(t1 - t0);
      out[1] = static_cast<float>(n);
    }
  }
  else if (mode == 9) {
    // write-after-read through the pipe: out[128 x 64] = a[128 x 128] * b[64 x 128]^T while a second product, issued
    // right behind the first, overwrites the first one's A operand (columns kColA .. +63) with c-independent data
    store_rows(a, 128, kColA);
    fill_f32_blocks(sB, b, 64, 128, tid, 128);
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after_sync();
      issue_x(false);                                           // reads A = columns 0..127
      const uint32_t id = idesc_tf32(128, 64, false, false, false);
      for (int k = 0; k < 16; ++k)                              // D = columns 0..63: overwrites half of that A
        umma_ts_tf32(tmem + kColA, tmem + kColX + 64 + 8 * (k & 7), smem_desc_sw128(smem_u32(sB) + (k / 4) * 8192 + (k % 4) * 32, 16, 1024),
                     id, k > 0);
      umma_commit(bar_a);
    }
    ok = mbar_wait(bar_a, 0, &abort_flag);
    __syncwarp();
    tc_fence_after_sync();
    if (ok) read_rows(64, kColX);
  } else if (mode == 8) {
    // where an issuing thread's time goes around a commit: stamps (cycles since the first issue) after issuing 8
    // products, after the commit, after a wait on a barrier that is already complete, after the tcgen05 fence, after
    // issuing 8 more products, after waiting for the first commit, after waiting for the second
    __shared__ __align__(8) uint64_t bar_c;
    const uint32_t b_c = smem_u32(&bar_c);
    fill_cols(0.5f, 128, kColA);
    for (int i = tid; i < 49152 / 4; i += 128) reinterpret_cast<uint32_t*>(smem)[i] = 0x3c003c00u;
    fence_proxy_async_smem();
    if (tid == 0) { mbar_init(b_c, 1); mbar_fence_init(); mbar_arrive(b_c); }
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after_sync();
      const uint32_t id = idesc_tf32(128, 128, false, false, false);
      const uint64_t db = smem_desc_sw128(smem_u32(sB), 16, 1024);
      const long long t0 = clock64();
#pragma unroll
      for (int k = 0; k < 8; ++k) umma_ts_tf32(tmem + kColX, tmem + kColA + 8 * k, db + 2 * (k & 3), id, k > 0);
      const long long t1 = clock64();
      umma_commit(bar_a);
      const long long t2 = clock64();
      ok = mbar_wait(b_c, 0, &abort_flag);
      const long long t3 = clock64();
      tc_fence_after_sync();
      const long long t4 = clock64();
#pragma unroll
      for (int k = 0; k < 8; ++k) umma_ts_tf32(tmem + kColX, tmem + kColA + 8 * k, db + 2 * (k & 3), id, true);
      const long long t5 = clock64();
      umma_commit(bar_b);
      ok = mbar_wait(bar_a, 0, &abort_flag) && ok;
      const long long t6 = clock64();
      ok = mbar_wait(bar_b, 0, &abort_flag) && ok;
      const long long t7 = clock64();
      out[0] = static_cast<float>(t1 - t0); out[1] = static_cast<float>(t2 - t0); out[2] = static_cast<float>(t3 - t0);
      out[3] = static_cast<float>(t4 - t0); out[4] = static_cast<float>(t5 - t0); out[5] = static_cast<float>(t6 - t0);
      out[6] = static_cast<float>(t7 - t0);
      // the same waits once more, with nothing in flight: what a wait on a complete barrier costs by itself
      const long long u0 = clock64();
      ok = mbar_wait(b_c, 0, &abort_flag) && ok;
      const long long u1 = clock64();
      ok = mbar_test_wait(b_c, 0) && ok;
      const long long u2 = clock64();
      // and with products in flight but a relaxed, non-suspending poll
#pragma unroll
      for (int k = 0; k < 8; ++k) umma_ts_tf32(tmem + kColX, tmem + kColA + 8 * k, db + 2 * (k & 3), id, true);
      const long long u3 = clock64();
      uint32_t done;
      asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.relaxed.cta.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
                   : "=r"(done) : "r"(b_c), "r"(0u) : "memory");
      const long long u4 = clock64();
      ok = mbar_test_wait(b_c, 0) && ok && done != 0;
      const long long u5 = clock64();
      out[7] = static_cast<float>(u1 - u0); out[8] = static_cast<float>(u2 - u1); out[9] = static_cast<float>(u3 - u2);
      out[10] = static_cast<float>(u4 - u3); out[11] = static_cast<float>(u5 - u4);
      // commit and fence with products in flight (both barriers' phases are spent: the arrivals just accumulate)
      ok = mbar_wait_spin(bar_a, 0, &abort_flag) && ok;
      const long long w0 = clock64();
#pragma unroll
      for (int k = 0; k < 8; ++k) umma_ts_tf32(tmem + kColX, tmem + kColA + 8 * k, db + 2 * (k & 3), id, true);
      const long long w1 = clock64();
      umma_commit(bar_a);
      const long long w2 = clock64();
      tc_fence_after_sync();
      const long long w3 = clock64();
#pragma unroll
      for (int k = 0; k < 8; ++k) umma_ts_tf32(tmem + kColX, tmem + kColA + 8 * k, db + 2 * (k & 3), id, true);
      const long long w4 = clock64();
      umma_commit(bar_b);
      const long long w5 = clock64();
      const bool seen = mbar_test_wait(b_c, 0);
      const long long w6 = clock64();
      tc_fence_after_sync();
      const long long w7 = clock64();
      umma_ts_tf32(tmem + kColX, tmem + kColA, db, id, true);
      const long long w8 = clock64();
      ok = ok && seen;
      out[12] = static_cast<float>(w1 - w0); out[13] = static_cast<float>(w2 - w0); out[14] = static_cast<float>(w3 - w0);
      out[15] = static_cast<float>(w4 - w0); out[16] = static_cast<float>(w5 - w0); out[17] = static_cast<float>(w6 - w0);
      out[18] = static_cast<float>(w7 - w0); out[19] = static_cast<float>(w8 - w0);
      umma_commit(bar_b);
      ok = mbar_wait_spin(bar_b, 0, &abort_flag) && ok;   // drain before the common exit (third completion of this barrier)
    }
  }
  if (!ok && tid == 0) atomicCAS(status, kDevOk, kDevTimeout);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 256);
}

// Issue-to-completion time of a stream of tcgen05 products of one shape (operand contents irrelevant): how the
// cost of one product depends on the kind, on where A comes from and on N.  A [128 x K], B [N x K] K-major,
// K = 64 bf16 or 32 tf32 elements per 128-byte row (one swizzle block): 4 products per pass over the block.
__global__ void __launch_bounds__(128) mma_timing_kernel(int tf32, int a_tmem, int N, int M, int reps, float* __restrict__ out,
                                                        int32_t* __restrict__ status) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ __align__(8) uint64_t bar;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5;
  const uint32_t b_done = smem_u32(&bar);
  if (tid == 0) { abort_flag = 0; mbar_init(b_done, 1); mbar_fence_init(); }
  if (warp == 0) tmem_alloc(smem_u32(&tmem_slot), 512);
  for (int i = tid; i < (16384 + 65536) / 4; i += 128) reinterpret_cast<uint32_t*>(smem)[i] = 0x3c003c00u;
  fence_proxy_async_smem();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = tmem_slot;
  {
    uint32_t r[32];
    for (int j = 0; j < 32; ++j) r[j] = 0x3c003c00u;
    for (int c0 = 0; c0 < 128; c0 += 32)
      tmem_st32(tmem + (static_cast<uint32_t>(warp * 32) << 16) + 256 + c0, r);   // A operand columns 256..383
    tmem_wait_st();
  }
  tc_fence_before_sync();
  __syncthreads();
  bool ok = true;
  if (tid == 0) {
    tc_fence_after_sync();
    const uint32_t id = tf32 ? idesc_tf32(M, N, false, false, false) : idesc_bf16(M, N, false, false, false);
    const uint64_t da = smem_desc_sw128(smem_u32(smem), 16, 1024);              // A block: 128 rows x 128 B
    const uint64_t db = smem_desc_sw128(smem_u32(smem) + 16384, 16, 1024);      // B block: up to 256 rows x 128 B
    const uint32_t ta = tmem + 256;
    const uint32_t id_mn = idesc_bf16(M, N, false, true, false);
    const uint64_t db_mn = smem_desc_sw128(smem_u32(smem) + 16384, 8192, 1024);
    // one branch-free, fully unrolled issue loop per variant (a branch inside the loop would time the issuing thread,
    // not the tensor pipe); sixteen products per iteration, as the kernels issue them
    const long long t0 = clock64();
#define MDN_TIMING_LOOP(CALL)                                   \
    for (int rep = 0; rep < reps; rep += 4) {                   \
      _Pragma("unroll") for (int k = 0; k < 16; ++k) { CALL; }  \
    }
    if (tf32 && a_tmem == 3) {   // the chain kernel's MMA-1: sixteen k-steps over 128 columns of A and four 16 KB panels of B
      MDN_TIMING_LOOP(umma_ts_tf32(tmem, ta + 8 * k, db + (uint64_t)((k >> 2) * 1024 + (k & 3) * 2), id, true))
    } else if (tf32 && a_tmem) { MDN_TIMING_LOOP(umma_ts_tf32(tmem, ta + 8 * (k & 3), db + 2 * (k & 3), id, true)) }
    else if (tf32) { MDN_TIMING_LOOP(umma_ss_tf32(tmem, da + 2 * (k & 3), db + 2 * (k & 3), id, true)) }
    else if (a_tmem == 2) { MDN_TIMING_LOOP(umma_ts(tmem, ta + 8 * (k & 3), db_mn + 128 * (k & 3), id_mn, true)) }
    else if (a_tmem) { MDN_TIMING_LOOP(umma_ts(tmem, ta + 8 * (k & 3), db + 2 * (k & 3), id, true)) }
    else { MDN_TIMING_LOOP(umma_ss(tmem, da + 2 * (k & 3), db + 2 * (k & 3), id, true)) }
#undef MDN_TIMING_LOOP
    const long long t_issued = clock64();
    umma_commit(b_done);
    ok = mbar_wait(b_done, 0, &abort_flag);
    const long long t1 = clock64();
    out[2] = static_cast<float>(t_issued - t0);   // until the last product was issued
    out[0] = static_cast<float>(t1 - t0);
    out[1] = static_cast<float>(16 * ((reps + 3) / 4));
  }
  if (!ok && tid == 0) atomicCAS(status, kDevOk, kDevTimeout);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 512);
}

// One CTA waits, at most `spin_limit` polls, on an mbarrier in its own shared memory that nothing ever arrives at
// (no copy, no product and no other thread refers to it): the wait runs out, the status word is set, the CTA leaves
// through the common exit.  What every bounded wait of the library's kernels does when its partner never shows up.
__global__ void __launch_bounds__(64) bounded_wait_kernel(uint32_t spin_limit, int32_t* __restrict__ status) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  const uint32_t b = smem_u32(&bar);
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(b, 1);
    mbar_fence_init();
  }
  __syncthreads();
  bool ok = true;
  if (threadIdx.x == 0) ok = mbar_wait(b, 0, &abort_flag, spin_limit);          // gives up after spin_limit polls
  __syncthreads();
  if (threadIdx.x == 32) ok = mbar_wait(b, 0, &abort_flag, spin_limit + 1024u);  // leaves early: sees the first thread's abort flag
  if (!ok && (threadIdx.x & 31) == 0) atomicCAS(status, kDevOk, kDevTimeout);
  if (threadIdx.x == 32) status[1] = ok ? 0 : 1;
}

}  // namespace
}  // namespace mdn

extern "C" mdn_status mdn_probe_tf32(int32_t mode, const float* a, const float* b, const float* c, float* out,
                                     int32_t* status, void* cuda_stream) {
  using namespace mdn;
  if (mode < 0 || mode > 9 || !out || !status) return MDN_ERR_INVALID_ARG;
  if ((mode <= 3 || mode == 9) && (!a || !b)) return MDN_ERR_INVALID_ARG;
  if ((mode == 2 || mode == 3) && !c) return MDN_ERR_INVALID_ARG;
  const int smem = 49152 + 1024;
  if (cudaFuncSetAttribute(tf32_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
    return MDN_ERR_CUDA;
  tf32_probe_kernel<<<1, 128, smem, static_cast<cudaStream_t>(cuda_stream)>>>(mode, a, b, c, out, status);
  return cudaGetLastError() == cudaSuccess ? MDN_OK : MDN_ERR_CUDA;
}

extern "C" mdn_status mdn_probe_bounded_wait(uint32_t spin_limit, int32_t* status, void* cuda_stream) {
  using namespace mdn;
  if (!status || spin_limit == 0 || spin_limit > (1u << 20)) return MDN_ERR_INVALID_ARG;
  bounded_wait_kernel<<<1, 64, 0, static_cast<cudaStream_t>(cuda_stream)>>>(spin_limit, status);
  return cudaGetLastError() == cudaSuccess ? MDN_OK : MDN_ERR_CUDA;
}

extern "C" mdn_status mdn_probe_mma_timing(int32_t tf32, int32_t a_tmem, int32_t n, int32_t m, int32_t reps, float* out,
                                           int32_t* status, void* cuda_stream) {
  using namespace mdn;
  if (!out || !status || (n != 32 && n != 64 && n != 128 && n != 256) || (m != 64 && m != 128) || reps < 1 || reps > 4096)
    return MDN_ERR_INVALID_ARG;
  const int smem = 16384 + 65536 + 1024;
  if (cudaFuncSetAttribute(mma_timing_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
    return MDN_ERR_CUDA;
  mma_timing_kernel<<<1, 128, smem, static_cast<cudaStream_t>(cuda_stream)>>>(tf32, a_tmem, n, m, reps, out, status);
  return cudaGetLastError() == cudaSuccess ? MDN_OK : MDN_ERR_CUDA;
}
