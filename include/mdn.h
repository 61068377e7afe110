/*
 * libmdn: chunkwise-parallel forward of the stepwise-momentum delta-rule
 * linear-attention recurrence (MDN), hand-written CUDA for sm_100a.
 *
 * The result is the one the token-by-token recurrence of Section 3.1 defines
 * (Eq. 5-6, with the correction value v~_t = v_t - alpha_t S_{t-1}^T k_t):
 *
 *     M_t = mu_t M_{t-1} - eta_t k_t v~_t^T
 *     S_t = alpha_t S_{t-1} - beta_t M_t
 *     o_t = scale * S_t^T q_t            alpha_t = exp(log_alpha_t), mu_t = exp(log_mu_t)
 *
 * computed chunk by chunk (chunk size C = 64) with the chunkwise algorithm of
 * Section 3.1 / Appendix C-D: per-chunk coefficients (Eq. 10), the intra-chunk
 * unit-lower-triangular solve (Eq. 15), the inter-chunk propagation of S and M,
 * and the chunk output (Eq. 11-12).
 *
 * Conventions for every entry point
 *  - All data pointers are DEVICE pointers unless a comment says "host".
 *  - Dense row-major layouts, innermost index last:
 *      q, k   [B, T, H, dk]      v, o   [B, T, H, dv]
 *      beta, log_alpha, log_mu, eta  [B, T, H]  float32
 *      states [N, H, dk, dv] float32, N = B (fixed length) or num_seqs (packed)
 *  - Packed / variable-length input: B = 1, T = total tokens, cu_seqlens holds
 *    num_seqs+1 increasing token offsets (cu[0] = 0, cu[num_seqs] = T).  State
 *    restarts at every sequence; chunks never straddle sequences; the last chunk
 *    of a sequence may be short.
 *  - The caller owns every buffer, including the workspace.  The library
 *    allocates no device memory and only enqueues work on the given stream
 *    (it never synchronises).  It keeps no state between calls, with three
 *    documented exceptions: mdn_chunk_fwd_host keeps two internal streams and
 *    their events per host thread and device; mdn_chunk_fwd_static_scratch
 *    keeps the device address of its built-in scratch array (and the array
 *    keeps the last call's contents); mdn_set_stage_events keeps the event
 *    handles of the calling host thread until cleared.
 *  - Errors are returned as mdn_status; nothing throws, aborts or traps.
 *    Invalid arguments are rejected on the host before anything is launched.
 */
#ifndef MDN_H_
#define MDN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  MDN_OK = 0,
  MDN_ERR_INVALID_ARG = 1,    /* NULL / misaligned pointer, bad shape                       */
  MDN_ERR_UNSUPPORTED = 2,    /* valid request this build has no kernel for                 */
  MDN_ERR_WORKSPACE = 3,      /* workspace NULL or smaller than mdn_chunk_fwd_workspace_bytes */
  MDN_ERR_CUDA = 4,           /* a CUDA runtime call (launch, attribute) failed             */
  MDN_ERR_DEVICE_TIMEOUT = 5, /* a bounded device-side wait ran out (reported by mdn_read_status) */
  MDN_ERR_STATIC_SCRATCH = 6  /* mdn_chunk_fwd_static_scratch: the problem needs more scratch than  */
                              /* MDN_STATIC_SCRATCH_BYTES                                            */
} mdn_status;

typedef enum { MDN_F32 = 0, MDN_BF16 = 1 } mdn_dtype;

/* Which kernels run the chain (inter-chunk propagation + output). */
typedef enum {
  MDN_PATH_AUTO = 0,    /* fp32 i/o -> SIMT fp32; bf16 i/o -> tensor-core path          */
  MDN_PATH_SIMT = 1,    /* fp32 FMA everywhere (any i/o dtype)                          */
  MDN_PATH_TENSOR = 2   /* tcgen05 MMAs with fp32 TMEM accumulators (bf16 i/o, d=128): the state is read as tf32
                           straight from its fp32 masters, operands made from accumulators are bf16 hi + lo */
} mdn_path;

typedef struct {
  int32_t B, T, H, dk, dv; /* packed input: B = 1, T = total tokens                         */
  int32_t chunk;           /* must be 64                                                     */
  int32_t num_seqs;        /* number of sequences when cu_seqlens != NULL, else 0            */
  int32_t io_dtype;        /* mdn_dtype of q, k, v                                           */
  int32_t o_dtype;         /* mdn_dtype of o                                                 */
  int32_t path;            /* mdn_path                                                       */
  float scale;             /* multiplies q; dk^-0.5 is the appendix listing's default,       */
                           /* 1.0 gives the bare o_t = S_t^T q_t                             */
  int32_t segments;        /* tensor path, fixed-length input: split every sequence into this */
                           /* many segments whose chunk chains run in PARALLEL (see below);   */
                           /* 0 = choose automatically, 1 = off, 3..32 = forced               */
} mdn_params;

/*
 * Parallel inter-chunk scan for long sequences with few (sequence, head) chains (Section 3.2 views the
 * recurrence as a linear dynamical system on the stacked state [S; M]).  With V = 0 a run of chunks
 * maps [S; M] linearly, so for a segment g of a sequence
 *     [S; M]_end = Phi_g [S; M]_start + Psi_g ,
 * where Psi_g is the segment run from a zero state and the two halves of Phi_g (2dk x 2dk) are the
 * segment run with V = 0 from the states (I, 0) and (0, I).  mdn_chunk_fwd then runs
 *   1. in parallel: segment 0 as usual, and for every middle segment the three runs giving Psi, Phi;
 *   2. a short serial combine over segments (fp32) giving every segment's true start state;
 *   3. in parallel: segments 1.. as usual from those start states (outputs and final state).
 * The result is the same recurrence; only rounding differs.  Chosen automatically when the call has
 * too few chains to fill the GPU and the sequences are long (e.g. B=1, H=16, T=65536).
 */

/* Bytes of device workspace mdn_chunk_fwd needs for these parameters (0 on invalid
 * parameters).  Holds the chunk map, the per-chunk coefficient vectors and the
 * per-chunk T and W matrices; contents are scratch. */
size_t mdn_chunk_fwd_workspace_bytes(const mdn_params* p);

/*
 * The whole hot path (Section 3.1 "Chunkwise Algorithm"; Appendix C):
 *   a0  chunk map from cu_seqlens (packed input only)
 *   a1  coefficient scan: abar, mubar, b and the last-row weights per chunk (Eq. 10)
 *   a2  intra-chunk system: A = tril((P K^T) .* Gamma^-, -1), T = (I + A)^-1 (Eq. 15),
 *       W = scale * (Q K^T) .* Gamma (Eq. 12)
 *   a3  per (sequence, head), chunks in order:  V~ = T (V - Diag(abar) K S + Diag(alpha b^-) K M),
 *       S, M updates (state equations below Eq. 12)
 *   a4  O = scale (Diag(abar) Q S - Diag(b) Q M) + W V~   (Eq. 11-12)
 *
 * eta may be NULL (eta = 1).  initial_S / initial_M may be NULL (zeros).
 * final_S / final_M may be NULL (not written).  cu_seqlens NULL = fixed length.
 * q, k, v, o and the states must be 16-byte aligned; workspace 256-byte aligned.
 * Asynchronous on `cuda_stream` (a cudaStream_t; NULL = default stream).
 */
mdn_status mdn_chunk_fwd(const mdn_params* p,
                         const void* q, const void* k, const void* v,
                         const float* beta, const float* log_alpha, const float* log_mu,
                         const float* eta,
                         const float* initial_S, const float* initial_M,
                         const int32_t* cu_seqlens,
                         void* o, float* final_S, float* final_M,
                         void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The same call for HOST buffers (end-to-end use): copies q, k, v, the gates, the
 * initial states and cu_seqlens from host memory into `arena`, runs mdn_chunk_fwd there,
 * and copies o and the final states back.  All data pointers except `arena` are HOST
 * pointers (pinned memory makes the copies asynchronous); `arena` is a DEVICE buffer of at
 * least mdn_chunk_fwd_host_arena_bytes(p) bytes, 256-byte aligned, owned by the caller.
 * The batch rows are cut into up to eight slices that move as a pipeline: uploads back to back on an internal
 * stream, each slice's kernels on `cuda_stream` as soon as its upload has landed, its results downloaded on a
 * second internal stream while the next slice is still arriving.  `cuda_stream` waits for the last download, so
 * the caller synchronises it before reading o, as with any asynchronous call.  The two internal streams and their
 * events are created on the first call of a host thread on a device and kept (this entry point is the one that
 * is not allocation-free on the host side); pageable host memory works but serialises the copies.
 */
size_t mdn_chunk_fwd_host_arena_bytes(const mdn_params* p);

mdn_status mdn_chunk_fwd_host(const mdn_params* p,
                              const void* q, const void* k, const void* v,
                              const float* beta, const float* log_alpha, const float* log_mu,
                              const float* eta,
                              const float* initial_S, const float* initial_M,
                              const int32_t* cu_seqlens,
                              void* o, float* final_S, float* final_M,
                              void* arena /* device */, size_t arena_bytes, void* cuda_stream);

/*
 * Recurrent decode step (Section 3.3: the recurrent form, Eq. 5-6, is what autoregressive decoding
 * uses): one new token per sequence, carried state updated IN PLACE.
 *     v~ = v - alpha S^T k;   M <- mu M - eta k v~^T;   S <- alpha S - beta M;   o = scale S^T q
 * p->T must be 1 and p->num_seqs 0 (one token per batch row); q, k: [B,1,H,dk]; v, o: [B,1,H,dv];
 * beta, log_alpha, log_mu, eta (NULL = 1): [B,1,H] float32; S, M: [B,H,dk,dv] float32, read and
 * written.  No workspace.  Feeding the final states of mdn_chunk_fwd (prefill) into this call
 * continues the same recurrence.  Asynchronous on `cuda_stream`.
 */
mdn_status mdn_decode_step(const mdn_params* p,
                           const void* q, const void* k, const void* v,
                           const float* beta, const float* log_alpha, const float* log_mu,
                           const float* eta,
                           float* S, float* M, void* o, void* cuda_stream);

/* mdn_decode_step with the layer's element-wise operations (mdn_layer_ops, below) applied to the one token:
 * gate formulas, q <- L2Norm(q - d k), k <- L2Norm(k), o <- sigmoid(g) * RMSNorm(o) * w; g: [B,1,H,dv].
 * `placement` is ignored: gates and q / k run inside the step's kernel, the output norm and gate as a second small
 * kernel over the step's o (measured faster than reducing across the head's CTAs).  ops == NULL is mdn_decode_step. */
struct mdn_layer_ops_s;
mdn_status mdn_decode_step_fused(const mdn_params* p, const struct mdn_layer_ops_s* ops,
                                 const void* q, const void* k, const void* v,
                                 const float* beta, const float* log_alpha, const float* log_mu,
                                 const float* eta,
                                 float* S, float* M, void* o, void* cuda_stream);

/*
 * The forward for callers that cannot allocate device memory (the paper has no counterpart: this
 * is a packaging variant of mdn_chunk_fwd, same kernels, same result).
 *
 * Who needs it: code that has no way to obtain a workspace at the time of the call - a server
 * that gave all device memory to its own arena at start-up, a plugin whose host forbids allocator
 * calls, a loop that cannot tolerate the device-wide synchronisation an allocation or free
 * causes.  Instead of a caller-supplied workspace, the scratch lives in a fixed array of
 * MDN_STATIC_SCRATCH_BYTES that is part of the library image; the call allocates nothing
 * (no cudaMalloc, no cudaFree, no allocating library routine).  The caller still passes every
 * input and output buffer, exactly as for mdn_chunk_fwd.
 *
 * Limits and rules:
 *  - mdn_chunk_fwd_workspace_bytes(p) must not exceed MDN_STATIC_SCRATCH_BYTES (32 MiB: about
 *    1200 chunk-head pairs, e.g. 4800 tokens x 16 heads); larger problems return
 *    MDN_ERR_STATIC_SCRATCH and launch nothing.
 *  - Every GPU that loads the library holds the array until the process exits.
 *  - The first call on each device looks up the array's device address (a one-time set-up on the
 *    host, made with that device current); make that first call before any stream capture.
 *  - All calls share the one array, and it keeps the previous call's contents (the call clears the
 *    part that must start at zero itself).  Calls whose kernels can overlap on the GPU - different
 *    streams, or several host threads - race on it: serialise them, or use mdn_chunk_fwd.
 *  - The device-side cu_seqlens check still turns a bad cu_seqlens into a no-op, but its status
 *    word is inside the array and cannot be read back with mdn_read_status.
 */
#define MDN_STATIC_SCRATCH_BYTES (32u << 20)

mdn_status mdn_chunk_fwd_static_scratch(const mdn_params* p,
                                        const void* q, const void* k, const void* v,
                                        const float* beta, const float* log_alpha, const float* log_mu,
                                        const float* eta,
                                        const float* initial_S, const float* initial_M,
                                        const int32_t* cu_seqlens,
                                        void* o, float* final_S, float* final_M,
                                        void* cuda_stream);

/*
 * The forward with the layer's element-wise operations fused in (Section 3.3, "Model Architecture" and
 * "Stability Aware Gating Parameterization"): none of them needs weights beyond per-head scalars, and each
 * would otherwise be a pass of its own over q, k, o or the gates.
 *
 *  raw_gates != 0: the beta / log_alpha / log_mu / eta arguments of the call hold the RAW per-head projections
 *    x_beta, x_alpha, x_mu, x_eta ([B,T,H] float32, all four required) and the gates are
 *        eta       = tanh(x_eta / tau) + 1                  theta = arctan(eta * s)
 *        log_alpha = f_alpha(x_alpha) + log cos^2(theta)    beta  = sigmoid(x_beta) * sin^2(theta)
 *        log_mu    = max(f_mu(x_mu), log_mu_min)            f(x)  = -a_h * softplus(x + b_h)
 *    with per-head a_h, b_h (decay_a_alpha .. decay_b_mu: device float32[H], all four required).
 *  qk_norm != 0:  q <- L2Norm(q - d_h k),  k <- L2Norm(k),  L2Norm(x) = x / sqrt(sum x^2 + qk_eps), qk_eps > 0;
 *    d: device float32[H] or NULL (= 0).  Both use the un-normalised k (the correction comes before the norm).
 *  out_norm_gate != 0: the output written to `o` is  sigmoid(g) * RMSNorm(o) * w  per head, RMSNorm(o) =
 *    o / sqrt(mean_j o_j^2 + rms_eps);  g: device [B,T,H,dv] in the i/o dtype; w: device float32[dv] or NULL (= 1).
 *  placement: 0 = inside the forward's kernels (below); 1 = all three as kernels of their own before / after the
 *    unchanged forward (needs the larger workspace below; the normalised q, k are then stored in the i/o dtype).
 *    1 is what 0 is measured against; the fp32 SIMT path always runs qk_norm and out_norm_gate as passes of
 *    their own, whatever the value.
 *
 * Inside the kernels (tensor path): the gate formulas run inside the coefficient scan; the norms of k and q - d k are
 * summed from the K and Q tiles the intra-chunk kernel holds anyway and ride on per-token coefficients that scale
 * fp32 accumulators; q - d k is formed in fp32 where the chain kernel makes its fp32 copy of the Q tile (q and k are
 * never rewritten or re-rounded in memory); the output step runs in the chain kernel's output epilogue.  All pointers are device pointers; the struct itself is host memory, read during the call.
 */
typedef struct mdn_layer_ops_s {
  int32_t raw_gates;
  const float* decay_a_alpha;
  const float* decay_b_alpha;
  const float* decay_a_mu;
  const float* decay_b_mu;
  float s, tau, log_mu_min;
  int32_t qk_norm;
  const float* d;
  float qk_eps;
  int32_t out_norm_gate;
  const void* g;
  const float* w;
  float rms_eps;
  int32_t placement;
} mdn_layer_ops;

/* Workspace bytes of mdn_chunk_fwd_fused for these parameters and operations (0 on invalid ones);
 * never less than mdn_chunk_fwd_workspace_bytes(p). */
size_t mdn_chunk_fwd_fused_workspace_bytes(const mdn_params* p, const mdn_layer_ops* ops /* host */);

/* mdn_chunk_fwd with `ops` applied; ops == NULL or all switches 0 is mdn_chunk_fwd itself.  Same
 * argument rules, ownership and error behaviour. */
mdn_status mdn_chunk_fwd_fused(const mdn_params* p, const mdn_layer_ops* ops /* host */,
                               const void* q, const void* k, const void* v,
                               const float* beta, const float* log_alpha, const float* log_mu,
                               const float* eta,
                               const float* initial_S, const float* initial_M,
                               const int32_t* cu_seqlens,
                               void* o, float* final_S, float* final_M,
                               void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Forward that also keeps the state at the START of every chunk (Section 3.2: the chunkwise form carries the pair
 * (S, M) from chunk to chunk; a chunk-parallel backward starts from those states).  Arguments as mdn_chunk_fwd,
 * plus `chunk_states`: a DEVICE buffer of mdn_chunk_states_bytes(p) bytes, 1024-byte aligned, owned by the caller.
 * For every (chunk slot, head), in the workspace's slot order, it receives 65536 bytes: the bf16 copy of S^T
 * (value index x key index, 128 x 128) and then that of M^T, each as two blocks (key index 0..63, 64..127) of 128
 * rows x 128 bytes whose 16-byte pieces are XOR-swizzled with (row mod 8) - the image a K-major tcgen05 operand
 * has in shared memory, so a later kernel can fetch a block with one untiled bulk copy.  These are the copies the
 * forward's own tensor-core products read (the fp32 masters stay on chip).  Behind the images of all slots lies a
 * second part: V~ = T (V - abar.(K S) + p.(K M)) of every chunk as float32 [chunk slot][64][H][dv] (rows past the end
 * of a short chunk are not written), which the chunk-parallel backward reads instead of rebuilding it.
 * Tensor path only (bf16 input, dk = dv = 128): MDN_ERR_UNSUPPORTED otherwise.  The serial chain is used
 * (p->segments is ignored).  Workspace as for mdn_chunk_fwd.
 */
size_t mdn_chunk_states_bytes(const mdn_params* p);

mdn_status mdn_chunk_fwd_keep_states(const mdn_params* p,
                                     const void* q, const void* k, const void* v,
                                     const float* beta, const float* log_alpha, const float* log_mu,
                                     const float* eta,
                                     const float* initial_S, const float* initial_M,
                                     const int32_t* cu_seqlens,
                                     void* o, float* final_S, float* final_M,
                                     void* chunk_states,
                                     void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Chunk-parallel backward, stage 1 (Section 3.2 differentiated chunk by chunk): the adjoint of the inter-chunk
 * state recurrence.  With dS', dM' the adjoints of the carried pair at the END of a chunk,
 *     dV~ = W^T dO + g_S . (K dS') - g_M . (K dM'),   dR = T^T dV~,
 *     dS  = abar_C dS' - K^T (abar . dR) + scale Q^T (abar . dO),
 *     dM  = -b_C dS' + mubar_C dM' + K^T (p . dR) - scale Q^T (b . dO)
 * walk the chunks of every sequence from the last to the first.  This has the shape of the forward's own chunk step
 * with the roles of S and M exchanged plus a second rank-64 update for the two Q terms, so it is run by the forward's
 * chain kernel on a mirrored problem (every sequence's chunks in reverse order) built from the forward's workspace.
 *   p, q, k, cu_seqlens: the forward call's (tensor path, o_dtype bf16); d_o = dL/do, [B,T,H,dv] bf16;
 *   d_final_S, d_final_M: dL/d(final states), [N,H,dk,dv] float32 or NULL (zero);
 *   fwd_workspace: the workspace of an mdn_chunk_fwd_keep_states call with the same p and inputs, untouched since
 *     (T, W and the coefficient vectors are read from it);
 *   adjoint_states: DEVICE buffer of mdn_bwd_adjoint_states_bytes(p) bytes, 1024-byte aligned.  Per sequence (in
 *     the workspace's slot order, entries of sequence s starting at its first chunk slot) and head it receives
 *     nchunks entries of 65536 bytes in the layout of mdn_chunk_fwd_keep_states with dM^T in the first half and
 *     dS^T in the second: entry nchunks - 1 - c is the adjoint pair at the END of chunk c; behind all entries, as
 *     float32 [entry][64][H][dv], dR = T^T dV~ (= dL/dv) of the same chunk;
 *   d_initial_S, d_initial_M: dL/d(initial states), [B,H,dk,dv] float32, or NULL;
 *   workspace: mdn_bwd_state_chain_workspace_bytes(p) bytes, 1024-byte aligned, scratch.
 * The gradients of q, k, v and the gates follow from these adjoint states and the kept forward states chunk by chunk,
 * in parallel; that stage is not part of this entry point (mdn_chunk_bwd is the complete backward).
 */
size_t mdn_bwd_state_chain_workspace_bytes(const mdn_params* p);
size_t mdn_bwd_adjoint_states_bytes(const mdn_params* p);

mdn_status mdn_bwd_state_chain(const mdn_params* p,
                               const void* q, const void* k, const void* d_o,
                               const float* d_final_S, const float* d_final_M,
                               const int32_t* cu_seqlens,
                               void* fwd_workspace, size_t fwd_workspace_bytes,
                               void* adjoint_states,
                               float* d_initial_S, float* d_initial_M,
                               void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The chunk-parallel backward (Section 3.2 differentiated chunk by chunk, on the tensor cores): the same gradients
 * as mdn_chunk_bwd, computed as
 *   1. the forward's state recurrence again, keeping (S, M) at the start of every chunk (mdn_chunk_fwd_keep_states
 *      without the output terms),
 *   2. the adjoint state recurrence (mdn_bwd_state_chain),
 *   3. per (chunk, head), in parallel: dQ, dK, the adjoints of the coefficient vectors and of the two masks, and
 *      from those the gate gradients by the recurrences of Eq. 10 in reverse (V~ and dR = dV are left behind by the
 *      chain runs of steps 1 and 2).
 * Arguments as mdn_chunk_bwd (fixed-length or packed input).  Tensor path only: bf16 q, k, v, bf16 d_o,
 * dk = dv = 128; MDN_ERR_UNSUPPORTED otherwise.  Operands are bf16 / tf32 with fp32 accumulation, so the gradients
 * carry the forward's bf16-level error (see the tests), not mdn_chunk_bwd's fp32 exactness; d_final_S, d_final_M
 * enter the tensor-core products through a bf16 copy (one rounding, up to 2^-8 of their largest element).  deta,
 * d_initial_S, d_initial_M may be NULL.  Workspace: mdn_chunk_bwd_chunked_workspace_bytes(p), 1024-byte aligned.
 */
size_t mdn_chunk_bwd_chunked_workspace_bytes(const mdn_params* p);

mdn_status mdn_chunk_bwd_chunked(const mdn_params* p,
                                 const void* q, const void* k, const void* v,
                                 const float* beta, const float* log_alpha, const float* log_mu, const float* eta,
                                 const float* initial_S, const float* initial_M,
                                 const int32_t* cu_seqlens,
                                 const void* d_o, const float* d_final_S, const float* d_final_M,
                                 float* dq, float* dk, float* dv,
                                 float* dbeta, float* dlog_alpha, float* dlog_mu, float* deta,
                                 float* d_initial_S, float* d_initial_M,
                                 void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The same backward for a caller that kept what the forward produced (the usual save-for-backward trade): steps 2
 * and 3 of mdn_chunk_bwd_chunked on the workspace and the chunk states of an mdn_chunk_fwd_keep_states call with the
 * same p and inputs, both untouched since.  Saves the second intra-chunk pass and the state-only forward; the price
 * is keeping that workspace and mdn_chunk_states_bytes(p) alive between the two calls.  Other arguments and the
 * results as mdn_chunk_bwd_chunked; workspace: mdn_chunk_bwd_saved_workspace_bytes(p), 1024-byte aligned.
 */
size_t mdn_chunk_bwd_saved_workspace_bytes(const mdn_params* p);

mdn_status mdn_chunk_bwd_saved(const mdn_params* p,
                               const void* q, const void* k, const void* v,
                               const float* beta, const float* log_alpha, const float* log_mu, const float* eta,
                               const int32_t* cu_seqlens,
                               void* fwd_workspace, size_t fwd_workspace_bytes, const void* chunk_states,
                               const void* d_o, const float* d_final_S, const float* d_final_M,
                               float* dq, float* dk, float* dv,
                               float* dbeta, float* dlog_alpha, float* dlog_mu, float* deta,
                               float* d_initial_S, float* d_initial_M,
                               void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Backward of mdn_chunk_fwd (Section 3.1: the training pass differentiates the same recurrence; like the paper's
 * kernels this keeps no per-token states and rebuilds them from per-chunk checkpoints):
 * given d_o = dL/do ([B,T,H,dv], o_dtype) and optionally dL/d(final_S), dL/d(final_M) ([N,H,dk,dv] float32, NULL =
 * zero), writes the float32 gradients
 *     dq, dk [B,T,H,dk];  dv [B,T,H,dv];  dbeta, dlog_alpha, dlog_mu, deta [B,T,H] (deta may be NULL);
 *     d_initial_S, d_initial_M [N,H,dk,dv] (either may be NULL).
 * q, k, v, the gates, the initial states, cu_seqlens, p: exactly the forward call's.  The pass recomputes the
 * forward itself, token by token in float32 (any dk, dv in {64, 128}; p->path and p->segments are ignored), so it
 * does not need the forward's outputs.  Workspace: mdn_chunk_bwd_workspace_bytes(p) bytes, 256-byte aligned,
 * scratch.  Same ownership, stream and error rules as mdn_chunk_fwd.  dv and the initial states' gradients are
 * bit-reproducible; dq, dk and the gate gradients sum over value columns through shared-memory floating-point
 * atomics, so their last bits can differ from run to run.
 */
size_t mdn_chunk_bwd_workspace_bytes(const mdn_params* p);

mdn_status mdn_chunk_bwd(const mdn_params* p,
                         const void* q, const void* k, const void* v,
                         const float* beta, const float* log_alpha, const float* log_mu, const float* eta,
                         const float* initial_S, const float* initial_M,
                         const int32_t* cu_seqlens,
                         const void* d_o, const float* d_final_S, const float* d_final_M,
                         float* dq, float* dk, float* dv,
                         float* dbeta, float* dlog_alpha, float* dlog_mu, float* deta,
                         float* d_initial_S, float* d_initial_M,
                         void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Stage entry points (the same kernels mdn_chunk_fwd launches, exposed so that each
 * stage can be checked on its own).  Both write into `workspace` using the layout
 * mdn_workspace_layout describes; mdn_intra_chunk expects mdn_coeff_scan's output there.
 *
 * mdn_coeff_scan (a0 + a1, Eq. 10): for every chunk slot s and head h, twelve float32
 * vectors of length 64 at  coef + ((s*H + h)*MDN_NUM_COEF + i)*64 :
 *   i=0 abar_r   1 b_r   2 alpha_r*b_{r-1}   3 gamma_{last,r}*eta_r   4 (mubar_last/mubar_r)*eta_r
 *   5 mubar_r    6 1/|k_r|   7 1/|q_r - d k_r|   (both 1 unless the fused q/k norm is on; then 2, 3 and 4
 *   also carry the factor 1/|k_r|)   8 alpha_r  9 beta_r   10 mu_r   11 eta_r
 * Positions past the end of a short chunk hold exact no-ops (alpha = mu = 1, beta = eta = 0).
 *
 * mdn_intra_chunk (a2, Eq. 15 and the mask of Eq. 12): per (s, h) the 64x64 row-major
 * matrices T and W, as float32 (SIMT path) or bfloat16 (tensor path; W as a bf16 hi part and a bf16 lo part of
 * the residual, W = hi + lo).  Inside mdn_chunk_fwd the plain tensor-path forward has the same kernel write W as
 * float32 into the same 16 KB per matrix (its chain kernel reads W as a tf32 operand); T is bfloat16 there too.
 */
#define MDN_NUM_COEF 12

typedef struct {
  int32_t num_slots;        /* chunk slots: B*ceil(T/64), or an upper bound T/64 + num_seqs when packed */
  int32_t mat_dtype;        /* mdn_dtype of the T and W matrices                                         */
  uint64_t off_status;      /* int32[4]: [0] 0 = ok, else first device-side error code                   */
  uint64_t off_chunk_off;   /* int32[num_seqs+1]: first chunk slot of each sequence (packed only)        */
  uint64_t off_slot_map;    /* int32[num_slots][4]: seq, first token, valid tokens n, local chunk index  */
  uint64_t off_coef;        /* float32[num_slots][H][MDN_NUM_COEF][64]                                   */
  uint64_t off_T;           /* [num_slots][H][64][64]                                                    */
  uint64_t off_W;           /* [num_slots][H][64][64]  (tensor path: bf16 hi part, lo part follows; or fp32) */
  uint64_t total_bytes;
  uint64_t off_seg;         /* segment states, Psi and Phi matrices of the parallel scan (fp32)          */
  int32_t segments;         /* segments per sequence the call will use (1 = plain serial chain)          */
  int32_t reserved;
} mdn_ws_layout;

mdn_status mdn_workspace_layout(const mdn_params* p, mdn_ws_layout* out /* host */);

mdn_status mdn_coeff_scan(const mdn_params* p,
                          const float* beta, const float* log_alpha, const float* log_mu,
                          const float* eta, const int32_t* cu_seqlens,
                          void* workspace, size_t workspace_bytes, void* cuda_stream);

mdn_status mdn_intra_chunk(const mdn_params* p, const void* q, const void* k,
                           const int32_t* cu_seqlens,
                           void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Copies the workspace status word to the host (synchronises the stream).  Returns MDN_OK,
 * MDN_ERR_INVALID_ARG (cu_seqlens rejected by the device-side check) or
 * MDN_ERR_DEVICE_TIMEOUT. */
mdn_status mdn_read_status(const mdn_params* p, const void* workspace, void* cuda_stream);

/* Static string for a status code (host pointer, never NULL). */
const char* mdn_status_string(mdn_status s);

/*
 * Optional timing hooks for the stages of mdn_chunk_fwd.  `events` is a HOST array of
 * MDN_NUM_STAGE_EVENTS created cudaEvent_t handles (copied by this call).  While set, every
 * mdn_chunk_fwd on this host thread records, on its stream: events[0] before its first kernel,
 * [1] after the chunk map + coefficient scan, [2] after the intra-chunk stage, [3] after the
 * chain kernel (inter-chunk propagation + output).  NULL clears the hooks.
 */
#define MDN_NUM_STAGE_EVENTS 4
mdn_status mdn_set_stage_events(void* const* events /* host */, int32_t n);

/* Text of the CUDA runtime error behind the last MDN_ERR_CUDA returned on this host thread by the
 * intra-chunk or chain launches (static string, host pointer). */
const char* mdn_last_cuda_error_string(void);

/* Number of kernels the last mdn_* call on this host thread enqueued. */
int32_t mdn_last_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* MDN_H_ */
