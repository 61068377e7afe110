// Chunk-parallel backward, first stage: the adjoint of the inter-chunk state recurrence (Section 3.2, the chunk
// form  S' = abar_C S - b_C M + K^T (g_S . V~),  M' = mubar_C M - K^T (g_M . V~),  V~ = T (V - abar . K S + p . K M),
// O = scale (abar . Q S - b . Q M) + W V~, differentiated with respect to the carried pair).
//
// With dS', dM' the adjoints at the END of a chunk,
//     dV~ = W^T dO + g_S . (K dS') - g_M . (K dM'),      dR = T^T dV~,
//     dS  = abar_C dS' - K^T (abar . dR) + scale Q^T (abar . dO),
//     dM  = -b_C dS' + mubar_C dM' + K^T (p . dR) - scale Q^T (b . dO).
// This has the shape of the forward's own chunk step with the roles exchanged (dM for S, dS for M):
//     X = K dM', Y = K dS',  "R" = V' - g_M . X + g_S . Y  with V' = W^T dO,  "V~" = T^T "R" = dR,
//     dM = mubar_C dM' - b_C dS' + K^T (p . dR),   dS = abar_C dS' - K^T (abar . dR),
// plus the two Q terms, a second rank-64 update of the pair: dM -= Q^T ((scale b) . dO), dS += Q^T ((scale abar) . dO).
// So the adjoint chain is run by the forward's chain kernel itself (chain_tensor.cu, training instantiation with the
// second update switched on) on a "mirrored" problem: the chunks of every sequence in REVERSE order, short chunks
// padded to 64 rows.  q, k and dO are read in place (the chain kernel mirrors the chunk index itself; rows past a
// short chunk's end meet zero coefficients), and so is T (its tile is read transposed); this file holds the kernel
// that builds the rest of that problem (W^T dO and the coefficient vectors) from the forward's workspace.
#include "mdn_common.cuh"
#include "tc_utils.cuh"
#include "warp_mma.cuh"

namespace mdn {
namespace {

using namespace tc;

constexpr int kD = 128;
constexpr int kPrepThreads = 256;
constexpr int LT = kD + 8;    // bf16 elements per row of the dO tile in shared memory (272 B: ldmatrix conflict-free)
constexpr int L6 = C + 8;     // ... of a 64 x 64 matrix

struct PrepArgs {
  ChunkGeom g;                      // the forward's geometry (fixed length)
  const __nv_bfloat16* d_o;
  const float* coef;                // forward: [slot][H][MDN_NUM_COEF][64]
  const __nv_bfloat16* W;           // forward: hi part, lo part w_lo_offset elements later
  size_t w_lo_offset;
  float scale;
  // the mirrored problem: sequence s = rows [chunk_off[s] * 64, ..) of v_ext
  __nv_bfloat16* v_ext;             // [slots 64][H][128]
  float* coef_ext;                  // [slots][H][MDN_NUM_COEF][64]
};

__global__ void __launch_bounds__(kPrepThreads) bwd_prep_kernel(PrepArgs a) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  // shared memory: W hi, W lo ([64][L6] each), then the dO tile ([64][LT])
  const int slot = blockIdx.x / a.g.H, h = blockIdx.x % a.g.H, H = a.g.H;
  const SlotInfo si = slot_info(a.g, slot);
  if (si.seq < 0) return;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  int slot0, nch;
  seq_chunks(a.g, si.seq, &slot0, &nch);
  // where this forward chunk lies in the mirrored problem
  const int e_real = slot0 + (nch - 1 - si.local);
  const size_t mat = ((size_t)slot * H + h) * C * C;

  // ---- W (hi, lo) and the dO tile into shared memory by cp.async (rows past the chunk's end zero-filled); the
  // coefficient vectors are remapped while the copies are in flight
  {
    const uint32_t sb = smem_u32(smem_raw);
    auto cp16 = [&](uint32_t dst, const void* src, bool live) {
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(live ? 16 : 0));
    };
    for (int idx = tid; idx < C * 8; idx += kPrepThreads) {
      const int r = idx >> 3, c8 = (idx & 7) * 8;
      cp16(sb + (r * L6 + c8) * 2, a.W + mat + r * C + c8, true);
      cp16(sb + (C * L6 + r * L6 + c8) * 2, a.W + a.w_lo_offset + mat + r * C + c8, true);
    }
    for (int idx = tid; idx < C * (kD / 8); idx += kPrepThreads) {
      const int r = idx >> 4, c8 = (idx & 15) * 8;
      cp16(sb + (2 * C * L6 + r * LT + c8) * 2, a.d_o + ((size_t)(si.tok0 + (r < si.n ? r : 0)) * H + h) * kD + c8, r < si.n);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  }

  // ---- coefficient vectors: abar' = g_M, p' = g_S, g_S' = p, g_M' = abar, end-of-chunk scalars (mubar_C, b_C,
  // abar_C) in vector 6; b stays where it is: with g_M' = abar it scales dO in the second update
  const float* cf = a.coef + ((size_t)slot * H + h) * MDN_NUM_COEF * C;
  float* cr = a.coef_ext + ((size_t)e_real * H + h) * MDN_NUM_COEF * C;
  for (int idx = tid; idx < MDN_NUM_COEF * C; idx += kPrepThreads) {
    const int vec = idx >> 6, r = idx & 63;
    const bool live = r < si.n;
    float xr = 0.f;
    switch (vec) {
      case kAbar: xr = live ? cf[kGM * C + r] : 0.f; break;
      case kB: xr = live ? cf[kB * C + r] : 0.f; break;
      case kAlphaBPrev: xr = live ? cf[kGS * C + r] : 0.f; break;
      case kGS: xr = live ? cf[kAlphaBPrev * C + r] : 0.f; break;
      case kGM: xr = live ? cf[kAbar * C + r] : 0.f; break;
      case kRk:
        xr = r == 0 ? cf[kMubar * C + C - 1] : r == 1 ? cf[kB * C + C - 1] : r == 2 ? cf[kAbar * C + C - 1] : 1.f;
        break;
      case kRq: xr = 1.f; break;
      default: break;   // mubar and the per-token gates are not read by a state-only run
    }
    cr[idx] = xr;
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();

  // ---- V' = W^T dO for the real step: a 64 x 128 result, one 32 x 32 block per warp, bf16 MMAs (W as hi + lo)
  {
    const uint32_t sb = smem_u32(smem_raw);
    const Opnd oWH_t{sb, L6 * 2, true}, oWL_t{sb + C * L6 * 2, L6 * 2, true}, oDO_t{sb + 2 * C * L6 * 2, LT * 2, true};
    const int m0 = 32 * (warp & 1), n0 = 32 * (warp >> 1);
    float Z[2][4][4];
    zero(Z);
    warp_mma(Z, oWH_t, oDO_t, C, m0, n0, lane);
    warp_mma(Z, oWL_t, oDO_t, C, m0, n0, lane);
    for_pair<2, 4>(m0, n0, g, t, [&](int mt, int nt, int hf, int i, int c) {
      const uint32_t packed = i < si.n ? pack_bf16(Z[mt][nt][2 * hf], Z[mt][nt][2 * hf + 1]) : 0u;
      *reinterpret_cast<uint32_t*>(a.v_ext + ((size_t)(e_real * C + i) * H + h) * kD + c) = packed;
    });
  }
}

// cu_seqlens of the mirrored problem (packed input): sequence s has 64 tokens per chunk
__global__ void bwd_ext_cu_kernel(const int32_t* __restrict__ chunk_off, int num_seqs, int32_t* __restrict__ cu_ext) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i <= num_seqs; i += gridDim.x * blockDim.x) cu_ext[i] = C * chunk_off[i];
}

}  // namespace

cudaError_t launch_bwd_ext_cu(const Plan& fwd, int32_t* cu_ext, int* launches) {
  bwd_ext_cu_kernel<<<1, 256, 0, fwd.stream>>>(fwd.geom.chunk_off, fwd.geom.num_seqs, cu_ext);
  ++*launches;
  return cudaGetLastError();
}

size_t bwd_prep_smem_bytes() { return (size_t)2 * C * L6 * 2 + (size_t)C * LT * 2; }

cudaError_t launch_bwd_prep(const Plan& fwd, const void* d_o, void* v_ext, float* coef_ext, int* launches) {
  PrepArgs a;
  a.g = fwd.geom;
  a.d_o = static_cast<const __nv_bfloat16*>(d_o);
  a.coef = reinterpret_cast<const float*>(fwd.ws + fwd.lay.off_coef);
  a.W = reinterpret_cast<const __nv_bfloat16*>(fwd.ws + fwd.lay.off_W);
  a.w_lo_offset = (size_t)fwd.geom.num_slots * fwd.p.H * C * C;
  a.scale = fwd.p.scale;
  a.v_ext = static_cast<__nv_bfloat16*>(v_ext);
  a.coef_ext = coef_ext;
  const size_t smem = bwd_prep_smem_bytes();
  cudaError_t e = cudaFuncSetAttribute(bwd_prep_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  bwd_prep_kernel<<<dim3((unsigned)fwd.geom.num_slots * fwd.p.H), dim3(kPrepThreads), smem, fwd.stream>>>(a);
  e = cudaGetLastError();
  if (e == cudaSuccess) ++*launches;
  return e;
}

}  // namespace mdn
