// Shared declarations of the MDN chunkwise-forward kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "layer_ops.cuh"
#include "mdn.h"

namespace mdn {

constexpr int C = 64;  // chunk size (Section 3.1; the appendix listing's default)

// Indices of the per-(chunk, head) coefficient vectors (Eq. 10 and the state equations).
enum Coef : int {
  kAbar = 0,    // abar_r  = prod_{j<=r} alpha_j
  kB = 1,       // b_r     = abar_r c_r           (weight of -M_[t] in S_r)
  kAlphaBPrev = 2,  // alpha_r * b_{r-1}          (weight of +K M_[t] in the right-hand side)
  kGS = 3,      // gamma_{last,r} * eta_r         (weight of k_r v~_r^T in S_[t+1])
  kGM = 4,      // (mubar_last/mubar_r) * eta_r   (weight of -k_r v~_r^T in M_[t+1])
  kMubar = 5,   // mubar_r = prod_{j<=r} mu_j
  kRk = 6,      // 1 / |k_r|         (fused q/k norm; 1 otherwise)
  kRq = 7,      // 1 / |q_r - d k_r| (vectors 0..7 are what the chain kernels read)
  kAlpha = 8,
  kBeta = 9,
  kMu = 10,
  kEta = 11
};
constexpr int kChainCoefs = 8;
static_assert(kEta + 1 == MDN_NUM_COEF, "coefficient vector count");

// Device-side error codes written to the workspace status word.
enum DevErr : int { kDevOk = 0, kDevBadCuSeqlens = 1, kDevTimeout = 2 };

// Everything a kernel needs to find a chunk: either arithmetic (fixed length) or
// the slot map the prep kernel wrote (packed input).
struct ChunkGeom {
  int B, T, H;
  int num_seqs;          // sequences (B when fixed length)
  int chunks_per_seq;    // fixed length only
  int num_slots;
  const int32_t* cu;         // packed only
  const int32_t* chunk_off;  // packed only: first slot of each sequence [num_seqs+1]
  const int32_t* slot_map;   // packed only: [num_slots][4]
};

struct SlotInfo {
  int seq;      // sequence id, -1 when the slot is unused
  int tok0;     // first token (index into the flattened [B*T] token axis)
  int n;        // valid tokens in this chunk, 1..64
  int local;    // chunk index inside its sequence
};

__device__ __forceinline__ SlotInfo slot_info(const ChunkGeom& g, int slot) {
  SlotInfo s;
  if (g.cu == nullptr) {
    s.seq = slot / g.chunks_per_seq;
    s.local = slot - s.seq * g.chunks_per_seq;
    s.tok0 = s.seq * g.T + s.local * C;
    s.n = min(C, g.T - s.local * C);
  } else {
    const int4 m = reinterpret_cast<const int4*>(g.slot_map)[slot];
    s.seq = m.x; s.tok0 = m.y; s.n = m.z; s.local = m.w;
  }
  return s;
}

// First chunk slot of a sequence and its chunk count (fixed-length or packed), for the per-chunk backward kernels.
__device__ __forceinline__ void seq_chunks(const ChunkGeom& g, int seq, int* slot0, int* nch) {
  if (g.cu == nullptr) { *slot0 = seq * g.chunks_per_seq; *nch = g.chunks_per_seq; }
  else { *slot0 = g.chunk_off[seq]; *nch = g.chunk_off[seq + 1] - *slot0; }
}

// Range of chunk slots and tokens of one sequence (for the chain kernels).
struct SeqInfo { int slot0, nchunks, tok0, len; };

__device__ __forceinline__ SeqInfo seq_info(const ChunkGeom& g, int seq) {
  SeqInfo s;
  if (g.cu == nullptr) {
    s.slot0 = seq * g.chunks_per_seq; s.nchunks = g.chunks_per_seq; s.tok0 = seq * g.T; s.len = g.T;
  } else {
    s.slot0 = g.chunk_off[seq]; s.nchunks = g.chunk_off[seq + 1] - s.slot0;
    s.tok0 = g.cu[seq]; s.len = g.cu[seq + 1] - s.tok0;
  }
  return s;
}

// Programmatic dependent launch (no-ops unless the kernel was launched with the stream-serialization
// attribute): wait for the preceding kernel's results / let the next kernel's prologue start.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Launch `kern` so that its prologue may overlap the tail of the previous kernel in the stream; the kernel
// itself calls grid_dependency_wait() before it touches anything the previous kernel wrote.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// Raw gate pointers ([B,T,H] fp32) for kernels that run the coefficient scan themselves; all NULL = the
// coefficients are already in the workspace.
struct GateArgs { const float* beta; const float* log_alpha; const float* log_mu; const float* eta; };

// One (token, head)'s alpha, mu, beta, eta from the gate arrays (raw projections when gp.raw).
struct TokenGates { float alpha, mu, beta, eta; };
__device__ __forceinline__ TokenGates load_token_gates(const GateParam& gp, int h, float v_log_alpha, float v_log_mu,
                                                       float v_beta, float v_eta) {
  if (gp.raw) {
    const GateValues gv = gate_transform(gp, h, v_log_alpha, v_log_mu, v_beta, v_eta);
    return TokenGates{expf(gv.log_alpha), expf(gv.log_mu), gv.beta, gv.eta};
  }
  return TokenGates{expf(v_log_alpha), expf(v_log_mu), v_beta, v_eta};
}

// Host-side view of one call, filled by the API layer.
struct Plan {
  mdn_params p;
  mdn_ws_layout lay;
  ChunkGeom geom;
  char* ws;
  cudaStream_t stream;
  GateParam gp;    // layer operations the kernels absorb (all off for the plain forward)
  QkNorm qk;
  OutPost post;
  // chain kernel options of the training / backward entry points (all off for the forward)
  uint8_t* chain_dump = nullptr;
  int chain_state_only = 0;
  int chain_end_scalars_in_rk = 0;
  float* chain_vt_dump = nullptr;        // V~ per chunk slot, fp32 [slot][64][H][dv]
  int chain_inject = 0;                  // second update per chunk from q and the tensor passed as o (adjoint chain)
  const ChunkGeom* chain_mirror_geom = nullptr;   // q, k, o belong to this geometry, walked in reverse chunk order
  const char* chain_mirror_T = nullptr;           // ... and T ([slot][H][64][64] bf16 of that problem), used transposed
  int cu_total_may_be_short = 0;   // packed: cu[N] <= T instead of == T (the adjoint chain's padded problem)
  bool w_f32 = false;              // tensor path: the intra-chunk kernel writes W as fp32 (chain_tf32.cu reads it so)
                                   // instead of the bf16 hi + lo pair of chain_tensor.cu
};

// Launchers (one per .cu file).  Each returns the CUDA error of its launches and adds
// the number of kernels it enqueued to *launches.
cudaError_t launch_chunk_map(const Plan& pl, int* launches);
// bwd_chunk_par.cu: gradients of q, k, v and the gates per (chunk, head) from the kept states and the adjoint states
// (state images per chunk slot; fwd_vt = V~, adj_dr = dR per chunk slot as fp32 [slot][64][H][dv]; adj_* in the adjoint
// chain's mirrored order: chunk c of a sequence with n chunks at the sequence's slot n - 1 - c)
cudaError_t launch_bwd_chunk_par(const Plan& fwd, const void* q, const void* k, const void* d_o, const float* beta,
                                 const float* log_alpha, const float* log_mu, const float* eta, const void* fwd_states,
                                 const float* fwd_vt, const void* adj_states, const float* adj_dr, float* dq, float* dk,
                                 float* dv, float* dbeta, float* dlog_alpha, float* dlog_mu, float* deta, int* launches);
// bwd_chunk.cu: W^T dO and the coefficient vectors of the adjoint state chain's mirrored problem, from the forward's workspace
cudaError_t launch_bwd_ext_cu(const Plan& fwd, int32_t* cu_ext, int* launches);
cudaError_t launch_bwd_prep(const Plan& fwd, const void* d_o, void* v_ext, float* coef_ext, int* launches);
cudaError_t launch_coeff_scan(const Plan& pl, const float* beta, const float* log_alpha,
                              const float* log_mu, const float* eta, int* launches);
// The layer operations as passes of their own (layer_ops.cu).
cudaError_t launch_gate_param(const Plan& pl, const float* x_beta, const float* x_alpha, const float* x_mu,
                              const float* x_eta, float* beta, float* log_alpha, float* log_mu, float* eta,
                              int* launches);
cudaError_t launch_qk_prep(const Plan& pl, const QkNorm& qk, const void* q, const void* k, void* q_out, void* k_out,
                           int* launches);
cudaError_t launch_out_norm_gate(const Plan& pl, const OutPost& post, void* o, int* launches);
cudaError_t launch_intra_simt(const Plan& pl, const void* q, const void* k, int* launches);
cudaError_t launch_chain_simt(const Plan& pl, const void* q, const void* k, const void* v,
                              const float* S0, const float* M0, void* o, float* Sf, float* Mf,
                              int* launches);


// Tensor-core (tcgen05) path: bf16 q/k/v, dk = dv = 128.
bool tensor_path_supported(const mdn_params& p);
cudaError_t launch_intra_tensor(const Plan& pl, const void* q, const void* k, const GateArgs& gates, int* launches);
cudaError_t launch_intra_mma(const Plan& pl, const void* q, const void* k, const GateArgs& gates, int* launches);
cudaError_t launch_chain_tensor(const Plan& pl, const void* q, const void* k, const void* v,
                                const float* S0, const float* M0, void* o, float* Sf, float* Mf,
                                int* launches);
// chain_tf32.cu: the plain forward's chain kernel (no layer operations, no training options); expects an fp32 W
cudaError_t launch_chain_tf32(const Plan& pl, const void* q, const void* k, const void* v,
                              const float* S0, const float* M0, void* o, float* Sf, float* Mf,
                              int* launches);
// True when a plan's chain runs in chain_tf32.cu (decided before the intra-chunk stage, which then writes W as fp32).
bool chain_uses_tf32_kernel(const Plan& pl);
// Segment bookkeeping of the parallel inter-chunk scan: per chain (G-1) states E, (G-2) Psi and 2 (G-2) Phi
// halves, each a pair of [dk x dv] fp32 matrices.
size_t seg_scratch_bytes(const mdn_params& p, int segments);
int choose_segments(const mdn_params& p);
cudaError_t launch_seg_combine(const Plan& pl, int G, float* E, const float* Psi, const float* PhiS,
                               const float* PhiM, int* launches);


// Backward (bwd_stepwise.cu).  Scratch offsets are relative to the scratch base the API layer places after the
// forward's workspace regions.
struct BwdScratch { uint64_t part_q, part_k, part_g, ck, prev, total; };
struct BwdIo {
  const void* q; const void* k; const void* v;
  const float* beta; const float* log_alpha; const float* log_mu; const float* eta;
  const float* S0; const float* M0;
  const void* d_o; const float* dSf; const float* dMf;
  float* dq; float* dk; float* dv; float* dbeta; float* dlog_alpha; float* dlog_mu; float* deta;
  float* dS0; float* dM0;
};
void bwd_scratch_layout(const mdn_params& p, int num_slots, BwdScratch* s);
cudaError_t launch_bwd_stepwise(const Plan& pl, const BwdIo& io, char* scratch, const BwdScratch& sl, int* launches);

// Recurrent decode step (one token per sequence, state updated in place).
cudaError_t launch_decode_step(const mdn_params& p, const void* q, const void* k, const void* v, const float* beta,
                               const float* log_alpha, const float* log_mu, const float* eta, float* S, float* M,
                               void* o, const GateParam& gp, const QkNorm& qk, cudaStream_t st);

}  // namespace mdn
