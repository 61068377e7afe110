// C ABI of libmdn: argument validation, workspace layout, kernel sequencing.
// Every computation runs in the kernels; this file only checks and launches.
#include <cstring>

#include "mdn_common.cuh"

namespace mdn {

static thread_local int t_last_launches = 0;
static thread_local int t_last_cuda_error = 0;
static thread_local cudaEvent_t t_stage_events[MDN_NUM_STAGE_EVENTS] = {nullptr, nullptr, nullptr, nullptr};
static thread_local bool t_stage_events_on = false;

static inline bool mark_stage(int i, cudaStream_t s) {
  return !t_stage_events_on || cudaEventRecord(t_stage_events[i], s) == cudaSuccess;
}

static inline uint64_t align_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }
static inline bool aligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

static mdn_path resolve_path(const mdn_params& p) {
  if (p.path == MDN_PATH_AUTO) return p.io_dtype == MDN_BF16 && tensor_path_supported(p) ? MDN_PATH_TENSOR : MDN_PATH_SIMT;
  return static_cast<mdn_path>(p.path);
}

static mdn_status check_params(const mdn_params* p) {
  if (!p) return MDN_ERR_INVALID_ARG;
  if (p->B <= 0 || p->T <= 0 || p->H <= 0) return MDN_ERR_INVALID_ARG;
  if (p->chunk != C) return MDN_ERR_UNSUPPORTED;
  if (!(p->dk == 64 || p->dk == 128) || !(p->dv == 64 || p->dv == 128)) return MDN_ERR_UNSUPPORTED;
  if (p->io_dtype != MDN_F32 && p->io_dtype != MDN_BF16) return MDN_ERR_INVALID_ARG;
  if (p->o_dtype != MDN_F32 && p->o_dtype != MDN_BF16) return MDN_ERR_INVALID_ARG;
  if (p->path < MDN_PATH_AUTO || p->path > MDN_PATH_TENSOR) return MDN_ERR_INVALID_ARG;
  if (p->num_seqs < 0) return MDN_ERR_INVALID_ARG;
  if (p->num_seqs > 0 && p->B != 1) return MDN_ERR_INVALID_ARG;
  if ((int64_t)p->B * p->T >= (int64_t)1 << 31) return MDN_ERR_UNSUPPORTED;
  if (p->H > 1024) return MDN_ERR_UNSUPPORTED;
  if (p->path == MDN_PATH_TENSOR && !tensor_path_supported(*p)) return MDN_ERR_UNSUPPORTED;
  if (!(p->scale == p->scale)) return MDN_ERR_INVALID_ARG;
  if (p->segments < 0 || p->segments == 2 || p->segments > 32) return MDN_ERR_INVALID_ARG;
  return MDN_OK;
}

static mdn_status make_layout(const mdn_params& p, mdn_ws_layout* lay) {
  std::memset(lay, 0, sizeof(*lay));
  const bool packed = p.num_seqs > 0;
  const int64_t slots = packed ? (int64_t)p.T / C + p.num_seqs : (int64_t)p.B * ((p.T + C - 1) / C);
  if (slots >= (int64_t)1 << 30) return MDN_ERR_UNSUPPORTED;
  lay->num_slots = (int32_t)slots;
  const bool tensor = resolve_path(p) == MDN_PATH_TENSOR;
  lay->mat_dtype = tensor ? MDN_BF16 : MDN_F32;
  const uint64_t mats = (uint64_t)slots * p.H * C * C;
  uint64_t off = 0;
  lay->off_status = off; off = align_up(off + 4 * sizeof(int32_t), 256);
  lay->off_chunk_off = off; off = align_up(off + (uint64_t)(p.num_seqs + 1) * sizeof(int32_t), 256);
  lay->off_slot_map = off; off = align_up(off + (packed ? (uint64_t)slots * 4 * sizeof(int32_t) : 0), 256);
  lay->off_coef = off; off = align_up(off + (uint64_t)slots * p.H * MDN_NUM_COEF * C * sizeof(float), 256);
  lay->off_T = off; off = align_up(off + mats * (tensor ? 2 : 4), 256);
  lay->off_W = off; off = align_up(off + mats * 4, 256);   // fp32, or bf16 hi + bf16 lo
  lay->segments = (tensor && !packed) ? choose_segments(p) : 1;
  lay->off_seg = off; off = align_up(off + (lay->segments > 1 ? seg_scratch_bytes(p, lay->segments) : 0), 256);
  lay->total_bytes = off;
  return MDN_OK;
}

static mdn_status make_plan(const mdn_params* p, const int32_t* cu, void* ws, size_t ws_bytes, void* stream,
                            Plan* pl) {
  mdn_status st = check_params(p);
  if (st != MDN_OK) return st;
  if ((p->num_seqs > 0) != (cu != nullptr)) return MDN_ERR_INVALID_ARG;
  pl->p = *p;
  pl->p.path = resolve_path(*p);
  st = make_layout(*p, &pl->lay);
  if (st != MDN_OK) return st;
  if (!ws || ws_bytes < pl->lay.total_bytes || !aligned(ws, 256)) return MDN_ERR_WORKSPACE;
  pl->ws = static_cast<char*>(ws);
  pl->stream = static_cast<cudaStream_t>(stream);
  pl->gp = GateParam{};
  pl->qk = QkNorm{};
  pl->post = OutPost{};
  ChunkGeom& g = pl->geom;
  g.B = p->B; g.T = p->T; g.H = p->H;
  g.num_seqs = cu ? p->num_seqs : p->B;
  g.chunks_per_seq = (p->T + C - 1) / C;
  g.num_slots = pl->lay.num_slots;
  g.cu = cu;
  g.chunk_off = cu ? reinterpret_cast<const int32_t*>(pl->ws + pl->lay.off_chunk_off) : nullptr;
  g.slot_map = cu ? reinterpret_cast<const int32_t*>(pl->ws + pl->lay.off_slot_map) : nullptr;
  return MDN_OK;
}

// with_scan = false: only the status word and the chunk map (the tensor path runs the scan inside its
// intra-chunk kernel).
static mdn_status run_prep_and_scan(const Plan& pl, const float* beta, const float* log_alpha, const float* log_mu,
                                    const float* eta, int* launches, bool with_scan = true) {
  if (!beta || !log_alpha || !log_mu) return MDN_ERR_INVALID_ARG;
  if (!aligned(beta, 4) || !aligned(log_alpha, 4) || !aligned(log_mu, 4) || (eta && !aligned(eta, 4)))
    return MDN_ERR_INVALID_ARG;
  if (launch_chunk_map(pl, launches) != cudaSuccess) return MDN_ERR_CUDA;   // (also clears the status word)
  if (with_scan && launch_coeff_scan(pl, beta, log_alpha, log_mu, eta, launches) != cudaSuccess) return MDN_ERR_CUDA;
  return MDN_OK;
}

static mdn_status run_intra(const Plan& pl, const void* q, const void* k, int* launches,
                            const GateArgs& gates = GateArgs{nullptr, nullptr, nullptr, nullptr}) {
  if (!q || !k || !aligned(q, 16) || !aligned(k, 16)) return MDN_ERR_INVALID_ARG;
  cudaError_t e = pl.p.path == MDN_PATH_TENSOR ? launch_intra_tensor(pl, q, k, gates, launches)
                                               : launch_intra_simt(pl, q, k, launches);
  if (e != cudaSuccess) t_last_cuda_error = (int)e;
  return e == cudaSuccess ? MDN_OK : MDN_ERR_CUDA;
}

}  // namespace mdn

using namespace mdn;

extern "C" {

static bool ops_active(const mdn_layer_ops* ops);
static mdn_status check_ops(const mdn_layer_ops& f);

size_t mdn_chunk_fwd_workspace_bytes(const mdn_params* p) {
  mdn_ws_layout lay;
  if (check_params(p) != MDN_OK || make_layout(*p, &lay) != MDN_OK) return 0;
  return (size_t)lay.total_bytes;
}

mdn_status mdn_workspace_layout(const mdn_params* p, mdn_ws_layout* out) {
  if (!out) return MDN_ERR_INVALID_ARG;
  mdn_status st = check_params(p);
  if (st != MDN_OK) return st;
  return make_layout(*p, out);
}

mdn_status mdn_coeff_scan(const mdn_params* p, const float* beta, const float* log_alpha, const float* log_mu,
                          const float* eta, const int32_t* cu_seqlens, void* workspace, size_t workspace_bytes,
                          void* cuda_stream) {
  t_last_launches = 0;
  Plan pl;
  mdn_status st = make_plan(p, cu_seqlens, workspace, workspace_bytes, cuda_stream, &pl);
  if (st != MDN_OK) return st;
  return run_prep_and_scan(pl, beta, log_alpha, log_mu, eta, &t_last_launches);
}

mdn_status mdn_intra_chunk(const mdn_params* p, const void* q, const void* k, const int32_t* cu_seqlens,
                           void* workspace, size_t workspace_bytes, void* cuda_stream) {
  t_last_launches = 0;
  Plan pl;
  mdn_status st = make_plan(p, cu_seqlens, workspace, workspace_bytes, cuda_stream, &pl);
  if (st != MDN_OK) return st;
  return run_intra(pl, q, k, &t_last_launches);
}

// The forward proper on a finished plan (chunk map, scan, intra-chunk stage, chain); pl.gp / pl.qk / pl.post say
// which layer operations the kernels absorb.
static mdn_status run_forward(const Plan& plan, const void* q, const void* k, const void* v, const float* beta,
                              const float* log_alpha, const float* log_mu, const float* eta, const float* initial_S,
                              const float* initial_M, void* o, float* final_S, float* final_M) {
  Plan pl = plan;
  pl.w_f32 = chain_uses_tf32_kernel(pl);   // the plain forward's chain kernel reads W as fp32
  if (!q || !k || !v || !o) return MDN_ERR_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(k, 16) || !aligned(v, 16) || !aligned(o, 16)) return MDN_ERR_INVALID_ARG;
  if ((initial_S && !aligned(initial_S, 16)) || (initial_M && !aligned(initial_M, 16)) ||
      (final_S && !aligned(final_S, 16)) || (final_M && !aligned(final_M, 16)))
    return MDN_ERR_INVALID_ARG;
  if (!mark_stage(0, pl.stream)) return MDN_ERR_CUDA;
  // tensor path: the intra-chunk kernel runs the coefficient scan itself (one kernel and one round trip of
  // the coefficient vectors less); SIMT path: stand-alone scan kernel
  const bool fused_scan = pl.p.path == MDN_PATH_TENSOR;
  mdn_status st = run_prep_and_scan(pl, beta, log_alpha, log_mu, eta, &t_last_launches, !fused_scan);
  if (st != MDN_OK) return st;
  if (!mark_stage(1, pl.stream)) return MDN_ERR_CUDA;
  st = fused_scan ? run_intra(pl, q, k, &t_last_launches, GateArgs{beta, log_alpha, log_mu, eta})
                  : run_intra(pl, q, k, &t_last_launches);
  if (st != MDN_OK) return st;
  if (!mark_stage(2, pl.stream)) return MDN_ERR_CUDA;
  cudaError_t e = pl.p.path == MDN_PATH_TENSOR
                      ? launch_chain_tensor(pl, q, k, v, initial_S, initial_M, o, final_S, final_M, &t_last_launches)
                      : launch_chain_simt(pl, q, k, v, initial_S, initial_M, o, final_S, final_M, &t_last_launches);
  if (e != cudaSuccess) { t_last_cuda_error = (int)e; return MDN_ERR_CUDA; }
  if (!mark_stage(3, pl.stream)) return MDN_ERR_CUDA;
  return MDN_OK;
}

mdn_status mdn_chunk_fwd(const mdn_params* p, const void* q, const void* k, const void* v, const float* beta,
                         const float* log_alpha, const float* log_mu, const float* eta, const float* initial_S,
                         const float* initial_M, const int32_t* cu_seqlens, void* o, float* final_S,
                         float* final_M, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  t_last_launches = 0;
  Plan pl;
  mdn_status st = make_plan(p, cu_seqlens, workspace, workspace_bytes, cuda_stream, &pl);
  if (st != MDN_OK) return st;
  return run_forward(pl, q, k, v, beta, log_alpha, log_mu, eta, initial_S, initial_M, o, final_S, final_M);
}

// ---- the forward that keeps the chunk-start states (tensor path, serial chain)
// Per (chunk slot, head): the bf16 state images S_b^T | M_b^T (2 x 32 KB), and behind all of them V~ of every chunk
// slot as fp32 [slot][64][H][dv] (32 KB per slot and head).  The adjoint chain's buffer has the same two parts, with
// dR = T^T dV~ in the place of V~.
constexpr uint64_t kStateImageBytes = 65536, kVtSlotBytes = 64 * 128 * 4;
size_t mdn_chunk_states_bytes(const mdn_params* p) {
  mdn_ws_layout lay;
  if (check_params(p) != MDN_OK || make_layout(*p, &lay) != MDN_OK) return 0;
  if (resolve_path(*p) != MDN_PATH_TENSOR) return 0;
  return (size_t)lay.num_slots * p->H * (kStateImageBytes + kVtSlotBytes);
}

mdn_status mdn_chunk_fwd_keep_states(const mdn_params* p, const void* q, const void* k, const void* v,
                                     const float* beta, const float* log_alpha, const float* log_mu,
                                     const float* eta, const float* initial_S, const float* initial_M,
                                     const int32_t* cu_seqlens, void* o, float* final_S, float* final_M,
                                     void* chunk_states, void* workspace, size_t workspace_bytes,
                                     void* cuda_stream) {
  t_last_launches = 0;
  if (check_params(p) != MDN_OK) return check_params(p);
  if (resolve_path(*p) != MDN_PATH_TENSOR) return MDN_ERR_UNSUPPORTED;
  if (!chunk_states || !aligned(chunk_states, 1024)) return MDN_ERR_INVALID_ARG;
  mdn_params ps = *p;
  ps.segments = 1;
  Plan pl;
  mdn_status st = make_plan(&ps, cu_seqlens, workspace, workspace_bytes, cuda_stream, &pl);
  if (st != MDN_OK) return st;
  pl.chain_dump = static_cast<uint8_t*>(chunk_states);
  pl.chain_vt_dump = reinterpret_cast<float*>(pl.chain_dump + (uint64_t)pl.lay.num_slots * p->H * kStateImageBytes);
  return run_forward(pl, q, k, v, beta, log_alpha, log_mu, eta, initial_S, initial_M, o, final_S, final_M);
}

// ---- chunk-parallel backward, stage 1: the adjoint of the inter-chunk state recurrence
struct AdjLayout {
  mdn_params pe; mdn_ws_layout le; uint64_t v_ext, ws_ext, cu_ext, total;
  uint64_t image_bytes() const { return (uint64_t)le.num_slots * pe.H * kStateImageBytes; }
  uint64_t states_bytes() const { return image_bytes() + (uint64_t)le.num_slots * pe.H * kVtSlotBytes; }
};

static mdn_status adj_layout(const mdn_params* p, AdjLayout* a) {
  mdn_status st = check_params(p);
  if (st != MDN_OK) return st;
  if (resolve_path(*p) != MDN_PATH_TENSOR) return MDN_ERR_UNSUPPORTED;
  a->pe = *p;
  a->pe.segments = 1;
  a->pe.path = MDN_PATH_TENSOR;
  if (p->num_seqs > 0) {   // packed: every chunk slot of the forward, padded to 64 rows (host-side bound)
    mdn_params pf = *p;
    pf.segments = 1;
    mdn_ws_layout lf;
    st = make_layout(pf, &lf);
    if (st != MDN_OK) return st;
    a->pe.B = 1;
    a->pe.T = p->chunk * (int)lf.num_slots;
  } else {
    a->pe.T = ((p->T + p->chunk - 1) / p->chunk) * p->chunk;   // short chunks padded to 64 rows
  }
  st = make_layout(a->pe, &a->le);
  if (st != MDN_OK) return st;
  const uint64_t rows = (uint64_t)a->pe.B * a->pe.T * p->H * p->dk * 2;
  uint64_t off = 0;
  auto take = [&](uint64_t bytes) { uint64_t at = off; off = align_up(off + bytes, 1024); return at; };
  a->v_ext = take(rows); a->ws_ext = take(a->le.total_bytes);
  a->cu_ext = take((uint64_t)(p->num_seqs + 1) * 4); a->total = off;
  return MDN_OK;
}

size_t mdn_bwd_state_chain_workspace_bytes(const mdn_params* p) {
  AdjLayout a;
  return adj_layout(p, &a) == MDN_OK ? (size_t)a.total : 0;
}

size_t mdn_bwd_adjoint_states_bytes(const mdn_params* p) {
  AdjLayout a;
  return adj_layout(p, &a) == MDN_OK ? (size_t)a.states_bytes() : 0;
}

mdn_status mdn_bwd_state_chain(const mdn_params* p, const void* q, const void* k, const void* d_o,
                               const float* d_final_S, const float* d_final_M, const int32_t* cu_seqlens,
                               void* fwd_workspace, size_t fwd_workspace_bytes, void* adjoint_states, float* d_initial_S,
                               float* d_initial_M, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  t_last_launches = 0;
  AdjLayout al;
  mdn_status st = adj_layout(p, &al);
  if (st != MDN_OK) return st;
  if (!q || !k || !d_o || !adjoint_states || !aligned(adjoint_states, 1024)) return MDN_ERR_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(k, 16) || !aligned(d_o, 16)) return MDN_ERR_INVALID_ARG;
  if (p->o_dtype != MDN_BF16) return MDN_ERR_UNSUPPORTED;   // d_o is read as bf16
  if (!workspace || workspace_bytes < al.total || !aligned(workspace, 1024)) return MDN_ERR_WORKSPACE;
  mdn_params pf = *p;
  pf.segments = 1;
  Plan fwd;
  st = make_plan(&pf, cu_seqlens, fwd_workspace, fwd_workspace_bytes, cuda_stream, &fwd);
  if (st != MDN_OK) return st;
  char* w = static_cast<char*>(workspace);
  int32_t* cu_ext = p->num_seqs > 0 ? reinterpret_cast<int32_t*>(w + al.cu_ext) : nullptr;
  Plan ext;
  st = make_plan(&al.pe, cu_ext, w + al.ws_ext, al.le.total_bytes, cuda_stream, &ext);
  if (st != MDN_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(ext.ws + ext.lay.off_status, 0, 16, s) != cudaSuccess) return MDN_ERR_CUDA;
  if (cu_ext) {   // the chunk map of the mirrored problem: 64 tokens per chunk of every sequence
    ext.cu_total_may_be_short = 1;
    if (launch_bwd_ext_cu(fwd, cu_ext, &t_last_launches) != cudaSuccess || launch_chunk_map(ext, &t_last_launches) != cudaSuccess)
      return MDN_ERR_CUDA;
  }
  cudaError_t e = launch_bwd_prep(fwd, d_o, w + al.v_ext, reinterpret_cast<float*>(ext.ws + ext.lay.off_coef),
                                  &t_last_launches);
  if (e != cudaSuccess) { t_last_cuda_error = (int)e; return MDN_ERR_CUDA; }
  // the forward's chain kernel on the mirrored problem, roles exchanged: its "S" is dM, its "M" is dS
  ext.chain_dump = static_cast<uint8_t*>(adjoint_states);
  ext.chain_vt_dump = reinterpret_cast<float*>(ext.chain_dump + al.image_bytes());
  ext.chain_inject = 1;   // the two Q terms: q and dO (passed in the place of o) give a second update per chunk
  ext.chain_mirror_geom = &fwd.geom;   // q, k, dO and T are read in place, chunk index mirrored
  ext.chain_mirror_T = fwd.ws + fwd.lay.off_T;
  ext.chain_state_only = 1;
  ext.chain_end_scalars_in_rk = 1;
  e = launch_chain_tensor(ext, q, k, w + al.v_ext, d_final_M, d_final_S, const_cast<void*>(d_o), d_initial_M,
                          d_initial_S, &t_last_launches);
  if (e != cudaSuccess) { t_last_cuda_error = (int)e; return MDN_ERR_CUDA; }
  return MDN_OK;
}

// ---- the chunk-parallel backward: state-only forward keeping the chunk states, adjoint chain, per-chunk stage
struct ChunkedBwdLayout { AdjLayout al; mdn_ws_layout lf; uint64_t ws_fwd, fwd_states, adj_states, stage, total; };

static mdn_status chunked_bwd_layout(const mdn_params* p, ChunkedBwdLayout* c) {
  mdn_status st = adj_layout(p, &c->al);
  if (st != MDN_OK) return st;
  mdn_params pf = *p;
  pf.segments = 1;
  st = make_layout(pf, &c->lf);
  if (st != MDN_OK) return st;
  uint64_t off = 0;
  auto take = [&](uint64_t bytes) { uint64_t at = off; off = align_up(off + bytes, 1024); return at; };
  c->ws_fwd = take(c->lf.total_bytes);
  c->fwd_states = take((uint64_t)c->lf.num_slots * p->H * (kStateImageBytes + kVtSlotBytes));
  c->adj_states = take(c->al.states_bytes());
  c->stage = take(c->al.total);
  c->total = off;
  return MDN_OK;
}

size_t mdn_chunk_bwd_chunked_workspace_bytes(const mdn_params* p) {
  ChunkedBwdLayout c;
  return chunked_bwd_layout(p, &c) == MDN_OK ? (size_t)c.total : 0;
}

size_t mdn_chunk_bwd_saved_workspace_bytes(const mdn_params* p) {
  ChunkedBwdLayout c;
  return chunked_bwd_layout(p, &c) == MDN_OK ? (size_t)(c.total - c.adj_states) : 0;
}

// Steps 2 and 3 on states and a workspace that a mdn_chunk_fwd_keep_states call left behind.
static mdn_status bwd_from_states(const mdn_params* p, const ChunkedBwdLayout& c, const void* q, const void* k,
                                  const void* v, const float* beta, const float* log_alpha, const float* log_mu,
                                  const float* eta, const int32_t* cu_seqlens, const void* d_o, const float* d_final_S,
                                  const float* d_final_M, void* fwd_ws, const void* fwd_states, char* adj_states,
                                  char* stage, float* dq, float* dk, float* dv, float* dbeta, float* dlog_alpha,
                                  float* dlog_mu, float* deta, float* d_initial_S, float* d_initial_M,
                                  void* cuda_stream, int launches_before) {
  mdn_status st = mdn_bwd_state_chain(p, q, k, d_o, d_final_S, d_final_M, cu_seqlens, fwd_ws, c.lf.total_bytes, adj_states,
                                      d_initial_S, d_initial_M, stage, c.al.total, cuda_stream);
  if (st != MDN_OK) return st;
  t_last_launches += launches_before;
  mdn_params pf = *p;
  pf.segments = 1;
  Plan fwd;
  st = make_plan(&pf, cu_seqlens, fwd_ws, c.lf.total_bytes, cuda_stream, &fwd);
  if (st != MDN_OK) return st;
  const char* fs = static_cast<const char*>(fwd_states);
  cudaError_t e = launch_bwd_chunk_par(
      fwd, q, k, d_o, beta, log_alpha, log_mu, eta, fs,
      reinterpret_cast<const float*>(fs + (uint64_t)c.lf.num_slots * p->H * kStateImageBytes), adj_states,
      reinterpret_cast<const float*>(adj_states + c.al.image_bytes()), dq, dk, dv, dbeta, dlog_alpha, dlog_mu, deta,
      &t_last_launches);
  if (e != cudaSuccess) { t_last_cuda_error = (int)e; return MDN_ERR_CUDA; }
  return MDN_OK;
}

mdn_status mdn_chunk_bwd_saved(const mdn_params* p, const void* q, const void* k, const void* v, const float* beta,
                               const float* log_alpha, const float* log_mu, const float* eta,
                               const int32_t* cu_seqlens, void* fwd_workspace, size_t fwd_workspace_bytes,
                               const void* chunk_states, const void* d_o, const float* d_final_S,
                               const float* d_final_M, float* dq, float* dk, float* dv, float* dbeta,
                               float* dlog_alpha, float* dlog_mu, float* deta, float* d_initial_S,
                               float* d_initial_M, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  t_last_launches = 0;
  if (p && (p->num_seqs > 0) != (cu_seqlens != nullptr)) return MDN_ERR_INVALID_ARG;
  ChunkedBwdLayout c;
  mdn_status st = chunked_bwd_layout(p, &c);
  if (st != MDN_OK) return st;
  if (p->o_dtype != MDN_BF16) return MDN_ERR_UNSUPPORTED;
  if (!q || !k || !v || !d_o || !beta || !log_alpha || !log_mu || !dq || !dk || !dv || !dbeta || !dlog_alpha || !dlog_mu)
    return MDN_ERR_INVALID_ARG;
  if (!fwd_workspace || fwd_workspace_bytes < c.lf.total_bytes || !aligned(fwd_workspace, 256)) return MDN_ERR_WORKSPACE;
  if (!chunk_states || !aligned(chunk_states, 1024)) return MDN_ERR_INVALID_ARG;
  if (!workspace || workspace_bytes < c.total - c.adj_states || !aligned(workspace, 1024)) return MDN_ERR_WORKSPACE;
  char* w = static_cast<char*>(workspace);   // [adjoint states | stage scratch], as in the full layout from adj_states on
  return bwd_from_states(p, c, q, k, v, beta, log_alpha, log_mu, eta, cu_seqlens, d_o, d_final_S, d_final_M,
                         fwd_workspace, chunk_states, w, w + (c.stage - c.adj_states), dq, dk, dv, dbeta, dlog_alpha,
                         dlog_mu, deta, d_initial_S, d_initial_M, cuda_stream, 0);
}

mdn_status mdn_chunk_bwd_chunked(const mdn_params* p, const void* q, const void* k, const void* v, const float* beta,
                                 const float* log_alpha, const float* log_mu, const float* eta,
                                 const float* initial_S, const float* initial_M, const int32_t* cu_seqlens,
                                 const void* d_o, const float* d_final_S, const float* d_final_M, float* dq, float* dk,
                                 float* dv,
                                 float* dbeta, float* dlog_alpha, float* dlog_mu, float* deta, float* d_initial_S,
                                 float* d_initial_M, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  t_last_launches = 0;
  if (p && (p->num_seqs > 0) != (cu_seqlens != nullptr)) return MDN_ERR_INVALID_ARG;
  ChunkedBwdLayout c;
  mdn_status st = chunked_bwd_layout(p, &c);
  if (st != MDN_OK) return st;
  if (p->o_dtype != MDN_BF16) return MDN_ERR_UNSUPPORTED;
  if (!q || !k || !v || !d_o || !beta || !log_alpha || !log_mu || !dq || !dk || !dv || !dbeta || !dlog_alpha || !dlog_mu)
    return MDN_ERR_INVALID_ARG;
  if (!workspace || workspace_bytes < c.total || !aligned(workspace, 1024)) return MDN_ERR_WORKSPACE;
  char* w = static_cast<char*>(workspace);
  // 1. the forward's states (no output terms), kept per chunk; T, W and the coefficient vectors stay in ws_fwd
  mdn_params pf = *p;
  pf.segments = 1;
  Plan fwd;
  st = make_plan(&pf, cu_seqlens, w + c.ws_fwd, c.lf.total_bytes, cuda_stream, &fwd);
  if (st != MDN_OK) return st;
  fwd.chain_dump = reinterpret_cast<uint8_t*>(w + c.fwd_states);
  fwd.chain_vt_dump = reinterpret_cast<float*>(w + c.fwd_states + (uint64_t)c.lf.num_slots * p->H * kStateImageBytes);
  fwd.chain_state_only = 1;
  st = run_forward(fwd, q, k, v, beta, log_alpha, log_mu, eta, initial_S, initial_M, w + c.stage /* o: never written */,
                   nullptr, nullptr);
  if (st != MDN_OK) return st;
  // 2. the adjoint state chain;  3. per (chunk, head): dq, dk, dv and the gate gradients
  return bwd_from_states(p, c, q, k, v, beta, log_alpha, log_mu, eta, cu_seqlens, d_o, d_final_S, d_final_M, w + c.ws_fwd,
                         w + c.fwd_states, w + c.adj_states, w + c.stage, dq, dk, dv, dbeta, dlog_alpha, dlog_mu, deta,
                         d_initial_S, d_initial_M, cuda_stream, t_last_launches);
}

// ---- the forward with layer operations
static bool ops_active(const mdn_layer_ops* ops) {
  return ops && (ops->raw_gates || ops->qk_norm || ops->out_norm_gate);
}

static mdn_status check_ops(const mdn_layer_ops& f) {
  if (f.raw_gates) {
    if (!f.decay_a_alpha || !f.decay_b_alpha || !f.decay_a_mu || !f.decay_b_mu) return MDN_ERR_INVALID_ARG;
    if (!(f.tau > 0.f) || !(f.s == f.s) || !(f.log_mu_min == f.log_mu_min)) return MDN_ERR_INVALID_ARG;
  }
  if (f.qk_norm && !(f.qk_eps > 0.f)) return MDN_ERR_INVALID_ARG;
  if (f.out_norm_gate && (!f.g || !aligned(f.g, 16) || !(f.rms_eps >= 0.f))) return MDN_ERR_INVALID_ARG;
  if (f.placement < 0 || f.placement > 1) return MDN_ERR_INVALID_ARG;
  return MDN_OK;
}

// Scratch of the separate passes, appended to the plain workspace: q', k' (i/o dtype) and the four gate arrays.
struct SepLayout { uint64_t q, k, gates[4], total; bool qk_sep, out_sep, gate_sep; };

static mdn_status sep_layout(const mdn_params& p, const mdn_layer_ops& f, const mdn_ws_layout& lay, SepLayout* sl) {
  const bool simt = resolve_path(p) != MDN_PATH_TENSOR;
  // placement 0: inside the kernels wherever the path can (tensor path: all three; SIMT path: the gate formulas);
  // 1: all as passes of their own
  sl->qk_sep = f.qk_norm && (f.placement == 1 || simt);
  sl->out_sep = f.out_norm_gate && (f.placement == 1 || simt);
  sl->gate_sep = f.raw_gates && f.placement == 1;
  const uint64_t tokens = (uint64_t)p.B * p.T, es = p.io_dtype == MDN_BF16 ? 2 : 4;
  uint64_t off = lay.total_bytes;
  auto take = [&](uint64_t bytes) { uint64_t at = off; off = align_up(off + bytes, 256); return at; };
  sl->q = take(sl->qk_sep ? tokens * p.H * p.dk * es : 0);
  sl->k = take(sl->qk_sep ? tokens * p.H * p.dk * es : 0);
  for (int i = 0; i < 4; ++i) sl->gates[i] = take(sl->gate_sep ? tokens * p.H * 4 : 0);
  sl->total = off;
  return MDN_OK;
}

size_t mdn_chunk_fwd_fused_workspace_bytes(const mdn_params* p, const mdn_layer_ops* ops) {
  mdn_ws_layout lay;
  if (check_params(p) != MDN_OK || make_layout(*p, &lay) != MDN_OK) return 0;
  if (!ops_active(ops)) return (size_t)lay.total_bytes;
  if (check_ops(*ops) != MDN_OK) return 0;
  SepLayout sl;
  sep_layout(*p, *ops, lay, &sl);
  return (size_t)sl.total;
}

mdn_status mdn_chunk_fwd_fused(const mdn_params* p, const mdn_layer_ops* ops, const void* q, const void* k,
                               const void* v, const float* beta, const float* log_alpha, const float* log_mu,
                               const float* eta, const float* initial_S, const float* initial_M,
                               const int32_t* cu_seqlens, void* o, float* final_S, float* final_M, void* workspace,
                               size_t workspace_bytes, void* cuda_stream) {
  if (!ops_active(ops))
    return mdn_chunk_fwd(p, q, k, v, beta, log_alpha, log_mu, eta, initial_S, initial_M, cu_seqlens, o, final_S,
                         final_M, workspace, workspace_bytes, cuda_stream);
  t_last_launches = 0;
  mdn_status st = check_params(p);
  if (st != MDN_OK) return st;
  st = check_ops(*ops);
  if (st != MDN_OK) return st;
  Plan pl;
  st = make_plan(p, cu_seqlens, workspace, workspace_bytes, cuda_stream, &pl);
  if (st != MDN_OK) return st;
  SepLayout sl;
  sep_layout(*p, *ops, pl.lay, &sl);
  if (workspace_bytes < sl.total) return MDN_ERR_WORKSPACE;
  if (!q || !k || !aligned(q, 16) || !aligned(k, 16) || !o || !aligned(o, 16)) return MDN_ERR_INVALID_ARG;
  if (ops->raw_gates) {
    if (!beta || !log_alpha || !log_mu || !eta) return MDN_ERR_INVALID_ARG;
    pl.gp = GateParam{1, ops->decay_a_alpha, ops->decay_b_alpha, ops->decay_a_mu, ops->decay_b_mu, ops->s,
                      1.0f / ops->tau, ops->log_mu_min};
  }
  const QkNorm qk{ops->qk_norm ? 1 : 0, ops->d, ops->qk_eps};
  const OutPost post{ops->out_norm_gate ? 1 : 0, ops->g, ops->w, ops->rms_eps};
  char* ws = pl.ws;
  if (sl.gate_sep) {
    float* g4[4];
    for (int i = 0; i < 4; ++i) g4[i] = reinterpret_cast<float*>(ws + sl.gates[i]);
    if (launch_gate_param(pl, beta, log_alpha, log_mu, eta, g4[0], g4[1], g4[2], g4[3], &t_last_launches) != cudaSuccess)
      return MDN_ERR_CUDA;
    beta = g4[0]; log_alpha = g4[1]; log_mu = g4[2]; eta = g4[3];
    pl.gp = GateParam{};
  }
  if (sl.qk_sep) {
    if (launch_qk_prep(pl, qk, q, k, ws + sl.q, ws + sl.k, &t_last_launches) != cudaSuccess) return MDN_ERR_CUDA;
    q = ws + sl.q; k = ws + sl.k;
  } else {
    pl.qk = qk;
  }
  if (!sl.out_sep) pl.post = post;
  st = run_forward(pl, q, k, v, beta, log_alpha, log_mu, eta, initial_S, initial_M, o, final_S, final_M);
  if (st != MDN_OK) return st;
  if (sl.out_sep && launch_out_norm_gate(pl, post, o, &t_last_launches) != cudaSuccess) return MDN_ERR_CUDA;
  return MDN_OK;
}

// ---- backward
static uint64_t bwd_scratch_base(const mdn_ws_layout& lay) { return align_up(lay.off_coef, 256); }

size_t mdn_chunk_bwd_workspace_bytes(const mdn_params* p) {
  mdn_ws_layout lay;
  if (check_params(p) != MDN_OK || make_layout(*p, &lay) != MDN_OK) return 0;
  BwdScratch bs;
  bwd_scratch_layout(*p, lay.num_slots, &bs);
  return (size_t)(bwd_scratch_base(lay) + bs.total);   // status word and chunk map, then the backward's scratch
}

mdn_status mdn_chunk_bwd(const mdn_params* p, const void* q, const void* k, const void* v, const float* beta,
                         const float* log_alpha, const float* log_mu, const float* eta, const float* initial_S,
                         const float* initial_M, const int32_t* cu_seqlens, const void* d_o, const float* d_final_S,
                         const float* d_final_M, float* dq, float* dk, float* dv, float* dbeta, float* dlog_alpha,
                         float* dlog_mu, float* deta, float* d_initial_S, float* d_initial_M, void* workspace,
                         size_t workspace_bytes, void* cuda_stream) {
  t_last_launches = 0;
  mdn_status st = check_params(p);
  if (st != MDN_OK) return st;
  if ((p->num_seqs > 0) != (cu_seqlens != nullptr)) return MDN_ERR_INVALID_ARG;
  const size_t need = mdn_chunk_bwd_workspace_bytes(p);
  if (!workspace || workspace_bytes < need || !aligned(workspace, 256)) return MDN_ERR_WORKSPACE;
  if (!q || !k || !v || !beta || !log_alpha || !log_mu || !d_o || !dq || !dk || !dv || !dbeta || !dlog_alpha || !dlog_mu)
    return MDN_ERR_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(k, 16) || !aligned(v, 16) || !aligned(d_o, 16) || !aligned(dq, 16) ||
      !aligned(dk, 16) || !aligned(dv, 16))
    return MDN_ERR_INVALID_ARG;
  Plan pl;
  pl.p = *p;
  pl.p.path = MDN_PATH_SIMT;
  st = make_layout(*p, &pl.lay);
  if (st != MDN_OK) return st;
  pl.ws = static_cast<char*>(workspace);
  pl.stream = static_cast<cudaStream_t>(cuda_stream);
  pl.gp = GateParam{}; pl.qk = QkNorm{}; pl.post = OutPost{};
  ChunkGeom& g = pl.geom;
  g.B = p->B; g.T = p->T; g.H = p->H;
  g.num_seqs = cu_seqlens ? p->num_seqs : p->B;
  g.chunks_per_seq = (p->T + C - 1) / C;
  g.num_slots = pl.lay.num_slots;
  g.cu = cu_seqlens;
  g.chunk_off = cu_seqlens ? reinterpret_cast<const int32_t*>(pl.ws + pl.lay.off_chunk_off) : nullptr;
  g.slot_map = cu_seqlens ? reinterpret_cast<const int32_t*>(pl.ws + pl.lay.off_slot_map) : nullptr;
  if (cudaMemsetAsync(pl.ws + pl.lay.off_status, 0, 4 * sizeof(int32_t), pl.stream) != cudaSuccess) return MDN_ERR_CUDA;
  if (launch_chunk_map(pl, &t_last_launches) != cudaSuccess) return MDN_ERR_CUDA;
  BwdScratch bs;
  bwd_scratch_layout(*p, pl.lay.num_slots, &bs);
  const BwdIo io{q, k, v, beta, log_alpha, log_mu, eta, initial_S, initial_M, d_o, d_final_S, d_final_M,
                 dq, dk, dv, dbeta, dlog_alpha, dlog_mu, deta, d_initial_S, d_initial_M};
  const cudaError_t e = launch_bwd_stepwise(pl, io, pl.ws + bwd_scratch_base(pl.lay), bs, &t_last_launches);
  if (e != cudaSuccess) { t_last_cuda_error = (int)e; return MDN_ERR_CUDA; }
  return MDN_OK;
}

static mdn_status decode_common(const mdn_params* p, const mdn_layer_ops* ops, const void* q, const void* k,
                                const void* v, const float* beta, const float* log_alpha, const float* log_mu,
                                const float* eta, float* S, float* M, void* o, void* cuda_stream) {
  t_last_launches = 0;
  mdn_status st = check_params(p);
  if (st != MDN_OK) return st;
  if (p->T != 1 || p->num_seqs != 0) return MDN_ERR_INVALID_ARG;
  if (!q || !k || !v || !beta || !log_alpha || !log_mu || !S || !M || !o) return MDN_ERR_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(k, 16) || !aligned(v, 16) || !aligned(o, 16) || !aligned(S, 16) || !aligned(M, 16))
    return MDN_ERR_INVALID_ARG;
  GateParam gp{};
  QkNorm qk{};
  OutPost post{};
  if (ops_active(ops)) {
    st = check_ops(*ops);
    if (st != MDN_OK) return st;
    if (ops->raw_gates) {
      if (!eta) return MDN_ERR_INVALID_ARG;
      gp = GateParam{1, ops->decay_a_alpha, ops->decay_b_alpha, ops->decay_a_mu, ops->decay_b_mu, ops->s,
                     1.0f / ops->tau, ops->log_mu_min};
    }
    qk = QkNorm{ops->qk_norm ? 1 : 0, ops->d, ops->qk_eps};
    post = OutPost{ops->out_norm_gate ? 1 : 0, ops->g, ops->w, ops->rms_eps};
  }
  cudaError_t e = launch_decode_step(*p, q, k, v, beta, log_alpha, log_mu, eta, S, M, o, gp, qk,
                                     static_cast<cudaStream_t>(cuda_stream));
  if (e != cudaSuccess) { t_last_cuda_error = (int)e; return MDN_ERR_CUDA; }
  t_last_launches = 1;
  if (post.on) {   // the output norm and gate over the step's o (one head row per warp; o is L2-resident)
    Plan pl;
    pl.p = *p;
    pl.stream = static_cast<cudaStream_t>(cuda_stream);
    e = launch_out_norm_gate(pl, post, o, &t_last_launches);
    if (e != cudaSuccess) { t_last_cuda_error = (int)e; return MDN_ERR_CUDA; }
  }
  return MDN_OK;
}

mdn_status mdn_decode_step(const mdn_params* p, const void* q, const void* k, const void* v, const float* beta,
                           const float* log_alpha, const float* log_mu, const float* eta, float* S, float* M,
                           void* o, void* cuda_stream) {
  return decode_common(p, nullptr, q, k, v, beta, log_alpha, log_mu, eta, S, M, o, cuda_stream);
}

mdn_status mdn_decode_step_fused(const mdn_params* p, const mdn_layer_ops* ops, const void* q, const void* k,
                                 const void* v, const float* beta, const float* log_alpha, const float* log_mu,
                                 const float* eta, float* S, float* M, void* o, void* cuda_stream) {
  return decode_common(p, ops, q, k, v, beta, log_alpha, log_mu, eta, S, M, o, cuda_stream);
}

mdn_status mdn_set_stage_events(void* const* events, int32_t n) {
  if (events == nullptr) { t_stage_events_on = false; return MDN_OK; }
  if (n < MDN_NUM_STAGE_EVENTS) return MDN_ERR_INVALID_ARG;
  for (int i = 0; i < MDN_NUM_STAGE_EVENTS; ++i) {
    if (events[i] == nullptr) return MDN_ERR_INVALID_ARG;
    t_stage_events[i] = static_cast<cudaEvent_t>(events[i]);
  }
  t_stage_events_on = true;
  return MDN_OK;
}

// ---- host-buffer variant: arena = [q | k | v | 4 gates | S0 | M0 | cu | o | Sf | Mf | one workspace per slice]
// The batch rows are cut into up to kHostSlices slices that are copied in, computed and copied out as a pipeline:
// the uploads run back to back on one internal stream, each slice's kernels start when its upload has landed, and
// its results leave on a second internal stream while the next slice is still arriving (PCIe is full duplex).  The
// caller's stream waits for the last download, so synchronising it covers the whole call, as before.
constexpr int kHostSlices = 8;

struct HostArena {
  uint64_t q, k, v, gates[4], S0, M0, cu, o, Sf, Mf, ws, total;
  uint64_t qk_row, v_row, gate_row, state_row, cu_bytes, o_row;   // bytes per batch row (per sequence for the states)
  uint64_t ws_slice;
  int slices, rows_max;
};

static int host_slices(const mdn_params& p) { return p.num_seqs > 0 ? 1 : (p.B < kHostSlices ? p.B : kHostSlices); }

static bool host_arena(const mdn_params* p, HostArena* a) {
  if (check_params(p) != MDN_OK) return false;
  a->slices = host_slices(*p);
  a->rows_max = (p->B + a->slices - 1) / a->slices;
  // a slice holds rows_max or rows_max - 1 rows, and the smaller one may need the LARGER workspace (with fewer
  // chains the parallel inter-chunk scan can switch on and bring its segment scratch): size for both
  a->ws_slice = 0;
  for (int rows = a->rows_max; rows >= 1 && rows >= p->B / a->slices; --rows) {
    mdn_params ps = *p;
    ps.B = rows;
    mdn_ws_layout lay;
    if (make_layout(ps, &lay) != MDN_OK) return false;
    if (align_up(lay.total_bytes, 256) > a->ws_slice) a->ws_slice = align_up(lay.total_bytes, 256);
  }
  const uint64_t es = p->io_dtype == MDN_BF16 ? 2 : 4, eo = p->o_dtype == MDN_BF16 ? 2 : 4;
  const uint64_t rows = (uint64_t)p->B, nseq = (uint64_t)(p->num_seqs > 0 ? p->num_seqs : p->B);
  a->qk_row = (uint64_t)p->T * p->H * p->dk * es; a->v_row = (uint64_t)p->T * p->H * p->dv * es;
  a->gate_row = (uint64_t)p->T * p->H * 4; a->state_row = (uint64_t)p->H * p->dk * p->dv * 4;
  a->cu_bytes = p->num_seqs > 0 ? (uint64_t)(p->num_seqs + 1) * 4 : 0; a->o_row = (uint64_t)p->T * p->H * p->dv * eo;
  uint64_t off = 0;
  auto take = [&](uint64_t bytes) { uint64_t at = off; off = align_up(off + bytes, 256); return at; };
  a->q = take(rows * a->qk_row); a->k = take(rows * a->qk_row); a->v = take(rows * a->v_row);
  for (int i = 0; i < 4; ++i) a->gates[i] = take(rows * a->gate_row);
  a->S0 = take(nseq * a->state_row); a->M0 = take(nseq * a->state_row); a->cu = take(a->cu_bytes);
  a->o = take(rows * a->o_row); a->Sf = take(nseq * a->state_row); a->Mf = take(nseq * a->state_row);
  a->ws = take((uint64_t)a->slices * a->ws_slice); a->total = off;
  return true;
}

size_t mdn_chunk_fwd_host_arena_bytes(const mdn_params* p) {
  HostArena a;
  return host_arena(p, &a) ? (size_t)a.total : 0;
}

// Internal copy streams and events of the host-buffer pipeline, one set per device and host thread, created on
// first use and kept.
struct HostPipe {
  bool ready;
  cudaStream_t in, out;
  cudaEvent_t begin, in_done[kHostSlices], cmp_done[kHostSlices], out_done;
};
static thread_local HostPipe t_pipes[64] = {};

static HostPipe* host_pipe() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  HostPipe& hp = t_pipes[dev];
  if (!hp.ready) {
    bool ok = cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp.begin, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp.out_done, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; ok && i < kHostSlices; ++i)
      ok = cudaEventCreateWithFlags(&hp.in_done[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&hp.cmp_done[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) return nullptr;
    hp.ready = true;
  }
  return &hp;
}

mdn_status mdn_chunk_fwd_host(const mdn_params* p, const void* q, const void* k, const void* v, const float* beta,
                              const float* log_alpha, const float* log_mu, const float* eta,
                              const float* initial_S, const float* initial_M, const int32_t* cu_seqlens, void* o,
                              float* final_S, float* final_M, void* arena, size_t arena_bytes, void* cuda_stream) {
  HostArena a;
  if (!host_arena(p, &a)) return check_params(p) != MDN_OK ? check_params(p) : MDN_ERR_UNSUPPORTED;
  if (!arena || arena_bytes < a.total || !aligned(arena, 256)) return MDN_ERR_WORKSPACE;
  if (!q || !k || !v || !beta || !log_alpha || !log_mu || !o) return MDN_ERR_INVALID_ARG;
  if ((p->num_seqs > 0) != (cu_seqlens != nullptr)) return MDN_ERR_INVALID_ARG;
  HostPipe* hp = host_pipe();
  if (!hp) return MDN_ERR_CUDA;
  char* d = static_cast<char*>(arena);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  auto ok = [](cudaError_t e) { return e == cudaSuccess; };
  auto h2d = [&](uint64_t off, const void* src, uint64_t bytes) {
    return src == nullptr || bytes == 0 ||
           ok(cudaMemcpyAsync(d + off, static_cast<const char*>(src), bytes, cudaMemcpyHostToDevice, hp->in));
  };
  auto d2h = [&](void* dst, uint64_t off, uint64_t bytes) {
    return dst == nullptr || bytes == 0 || ok(cudaMemcpyAsync(dst, d + off, bytes, cudaMemcpyDeviceToHost, hp->out));
  };
  auto at = [](const void* base, uint64_t bytes) { return base ? static_cast<const char*>(base) + bytes : nullptr; };
  auto at_w = [](void* base, uint64_t bytes) { return base ? static_cast<char*>(base) + bytes : nullptr; };
  // the uploads start after whatever the caller's stream holds at this point (it may still use the arena)
  if (!ok(cudaEventRecord(hp->begin, s)) || !ok(cudaStreamWaitEvent(hp->in, hp->begin, 0))) return MDN_ERR_CUDA;
  if (!h2d(a.cu, cu_seqlens, a.cu_bytes)) return MDN_ERR_CUDA;
  const int per = p->B / a.slices, extra = p->B % a.slices;
  const bool packed = p->num_seqs > 0;
  int row0 = 0;
  int first_row[kHostSlices], n_rows[kHostSlices];
  for (int i = 0; i < a.slices; ++i) {
    const uint64_t nr = (uint64_t)(per + (i < extra ? 1 : 0)), r0 = (uint64_t)row0;
    const uint64_t nst = packed ? (uint64_t)p->num_seqs : nr, s0 = packed ? 0 : r0;
    first_row[i] = row0; n_rows[i] = (int)nr; row0 += (int)nr;
    if (!h2d(a.q + r0 * a.qk_row, at(q, r0 * a.qk_row), nr * a.qk_row) ||
        !h2d(a.k + r0 * a.qk_row, at(k, r0 * a.qk_row), nr * a.qk_row) ||
        !h2d(a.v + r0 * a.v_row, at(v, r0 * a.v_row), nr * a.v_row) ||
        !h2d(a.gates[0] + r0 * a.gate_row, at(beta, r0 * a.gate_row), nr * a.gate_row) ||
        !h2d(a.gates[1] + r0 * a.gate_row, at(log_alpha, r0 * a.gate_row), nr * a.gate_row) ||
        !h2d(a.gates[2] + r0 * a.gate_row, at(log_mu, r0 * a.gate_row), nr * a.gate_row) ||
        !h2d(a.gates[3] + r0 * a.gate_row, at(eta, r0 * a.gate_row), nr * a.gate_row) ||
        !h2d(a.S0 + s0 * a.state_row, at(initial_S, s0 * a.state_row), nst * a.state_row) ||
        !h2d(a.M0 + s0 * a.state_row, at(initial_M, s0 * a.state_row), nst * a.state_row) ||
        !ok(cudaEventRecord(hp->in_done[i], hp->in)))
      return MDN_ERR_CUDA;
  }
  auto fp = [&](uint64_t off, const void* given) { return given ? reinterpret_cast<float*>(d + off) : nullptr; };
  for (int i = 0; i < a.slices; ++i) {
    const uint64_t nr = (uint64_t)n_rows[i], r0 = (uint64_t)first_row[i];
    const uint64_t nst = packed ? (uint64_t)p->num_seqs : nr, s0 = packed ? 0 : r0;
    mdn_params ps = *p;
    ps.B = n_rows[i];
    if (!ok(cudaStreamWaitEvent(s, hp->in_done[i], 0))) return MDN_ERR_CUDA;
    const mdn_status st = mdn_chunk_fwd(
        &ps, d + a.q + r0 * a.qk_row, d + a.k + r0 * a.qk_row, d + a.v + r0 * a.v_row,
        fp(a.gates[0] + r0 * a.gate_row, beta), fp(a.gates[1] + r0 * a.gate_row, log_alpha),
        fp(a.gates[2] + r0 * a.gate_row, log_mu), fp(a.gates[3] + r0 * a.gate_row, eta),
        fp(a.S0 + s0 * a.state_row, initial_S), fp(a.M0 + s0 * a.state_row, initial_M),
        cu_seqlens ? reinterpret_cast<const int32_t*>(d + a.cu) : nullptr, d + a.o + r0 * a.o_row,
        fp(a.Sf + s0 * a.state_row, final_S), fp(a.Mf + s0 * a.state_row, final_M), d + a.ws + (uint64_t)i * a.ws_slice,
        a.ws_slice, cuda_stream);
    if (st != MDN_OK) return st;
    if (!ok(cudaEventRecord(hp->cmp_done[i], s)) || !ok(cudaStreamWaitEvent(hp->out, hp->cmp_done[i], 0)) ||
        !d2h(at_w(o, r0 * a.o_row), a.o + r0 * a.o_row, nr * a.o_row) ||
        !d2h(at_w(final_S, s0 * a.state_row), a.Sf + s0 * a.state_row, nst * a.state_row) ||
        !d2h(at_w(final_M, s0 * a.state_row), a.Mf + s0 * a.state_row, nst * a.state_row))
      return MDN_ERR_CUDA;
  }
  if (!ok(cudaEventRecord(hp->out_done, hp->out)) || !ok(cudaStreamWaitEvent(s, hp->out_done, 0))) return MDN_ERR_CUDA;
  return MDN_OK;
}

mdn_status mdn_read_status(const mdn_params* p, const void* workspace, void* cuda_stream) {
  mdn_ws_layout lay;
  if (!workspace || check_params(p) != MDN_OK || make_layout(*p, &lay) != MDN_OK) return MDN_ERR_INVALID_ARG;
  int32_t word[4] = {0, 0, 0, 0};
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemcpyAsync(word, static_cast<const char*>(workspace) + lay.off_status, sizeof(word),
                      cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return MDN_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return MDN_ERR_CUDA;
  if (word[0] == kDevOk) return MDN_OK;
  return word[0] == kDevBadCuSeqlens ? MDN_ERR_INVALID_ARG : MDN_ERR_DEVICE_TIMEOUT;
}

const char* mdn_status_string(mdn_status s) {
  switch (s) {
    case MDN_OK: return "ok";
    case MDN_ERR_INVALID_ARG: return "invalid argument";
    case MDN_ERR_UNSUPPORTED: return "unsupported configuration";
    case MDN_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case MDN_ERR_CUDA: return "CUDA runtime error";
    case MDN_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    case MDN_ERR_STATIC_SCRATCH: return "problem needs more scratch than the built-in static buffer holds";
  }
  return "unknown status";
}

int32_t mdn_last_launch_count(void) { return t_last_launches; }

const char* mdn_last_cuda_error_string(void) {
  return t_last_cuda_error == 0 ? "no CUDA error recorded" : cudaGetErrorString((cudaError_t)t_last_cuda_error);
}

}  // extern "C"
