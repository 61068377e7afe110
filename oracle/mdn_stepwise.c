/*
 * TEST INFRASTRUCTURE, NOT THE PRODUCT.  CPU oracle for the MDN forward.
 *
 * A plain, slow, fp64 evaluation of the stepwise-momentum delta-rule recurrence,
 * token by token, exactly as Section 3.1 states it (Eq. 5-6 with the correction
 * value v~_t = v_t - S_{t-1}^T p_t, p_t = alpha_t k_t):
 *
 *     v~_t = v_t - alpha_t * S_{t-1}^T k_t
 *     M_t  = mu_t * M_{t-1} - eta_t * k_t v~_t^T
 *     S_t  = alpha_t * S_{t-1} - beta_t * M_t          (uses the NEW M_t)
 *     o_t  = scale * S_t^T q_t                          (uses the NEW S_t)
 *
 * with alpha_t = exp(log_alpha_t), mu_t = exp(log_mu_t); S, M in R^{dk x dv}.
 * "scale" multiplies q (scale = 1 gives the bare o_t = S_t^T q_t of Section 3.1;
 * the appendix code defaults to dk^-0.5).  Every sequence starts from the given
 * initial (S, M) or from zeros; state never crosses a sequence boundary.
 *
 * Inputs are float32 arrays holding the already rounded storage values (bf16 or
 * fp32 are both exact in float32); all arithmetic here is double.  Columns of
 * S, M, o are independent, so the work is split over (chain, column block) with
 * OpenMP; nothing else is blocked, fused or reordered.
 *
 * Nothing in the CUDA path includes, links or calls this file, and this file
 * uses nothing of the CUDA path.  Pinned by tests/test_oracle_pins.py.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define COLS_PER_TASK 16

int mdn_oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/*
 * Token axis: q,k [tokens,H,dk]; v,o [tokens,H,dv]; gates [tokens,H].
 * Sequence n covers tokens seq_start[n] .. seq_start[n]+seq_len[n]-1.
 * chains: optional list of chain ids (n*H + h) to evaluate; NULL = all N*H.
 * S0/M0/S_fin/M_fin: [N,H,dk,dv]; S0,M0 float32 (NULL = zeros); outputs double
 * (NULL = not wanted).  eta NULL = 1.  Only the selected chains' outputs are
 * written.  Returns 0, or -1 on allocation failure / bad arguments.
 */
int mdn_oracle_stepwise(int64_t num_seqs, const int64_t* seq_start, const int64_t* seq_len,
                        int H, int dk, int dv,
                        const float* q, const float* k, const float* v,
                        const float* beta, const float* log_alpha, const float* log_mu,
                        const float* eta, double scale,
                        const float* S0, const float* M0,
                        const int32_t* chains, int64_t n_chains,
                        double* o, double* S_fin, double* M_fin) {
  if (num_seqs <= 0 || H <= 0 || dk <= 0 || dv <= 0 || !q || !k || !v || !beta ||
      !log_alpha || !log_mu || !o)
    return -1;
  const int64_t total_chains = chains ? n_chains : num_seqs * (int64_t)H;
  const int col_blocks = (dv + COLS_PER_TASK - 1) / COLS_PER_TASK;
  const int64_t n_tasks = total_chains * col_blocks;
  int failed = 0;

#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t task = 0; task < n_tasks; ++task) {
    const int64_t ci = task / col_blocks;
    const int cb = (int)(task % col_blocks);
    const int64_t chain = chains ? (int64_t)chains[ci] : ci;
    const int64_t n = chain / H;
    const int h = (int)(chain % H);
    const int j0 = cb * COLS_PER_TASK;
    const int j1 = (j0 + COLS_PER_TASK < dv) ? j0 + COLS_PER_TASK : dv;
    const int nc = j1 - j0;

    /* column-major slices: S[j][d], M[j][d] for j in [j0,j1) */
    double* S = (double*)malloc(sizeof(double) * (size_t)nc * dk);
    double* M = (double*)malloc(sizeof(double) * (size_t)nc * dk);
    if (!S || !M) {
      free(S); free(M);
#pragma omp atomic write
      failed = 1;
      continue;
    }
    const size_t st_off = ((size_t)n * H + h) * (size_t)dk * dv;
    for (int j = 0; j < nc; ++j)
      for (int d = 0; d < dk; ++d) {
        S[(size_t)j * dk + d] = S0 ? (double)S0[st_off + (size_t)d * dv + (j0 + j)] : 0.0;
        M[(size_t)j * dk + d] = M0 ? (double)M0[st_off + (size_t)d * dv + (j0 + j)] : 0.0;
      }

    for (int64_t t = seq_start[n]; t < seq_start[n] + seq_len[n]; ++t) {
      const size_t g = (size_t)t * H + h;
      const double alpha = exp((double)log_alpha[g]);
      const double mu = exp((double)log_mu[g]);
      const double bt = (double)beta[g];
      const double et = eta ? (double)eta[g] : 1.0;
      const float* kt = k + g * dk;
      const float* qt = q + g * dk;
      const float* vt = v + g * dv;
      double* ot = o + g * dv;
      for (int j = 0; j < nc; ++j) {
        double* Sj = S + (size_t)j * dk;
        double* Mj = M + (size_t)j * dk;
        double pred = 0.0;                       /* (S_{t-1}^T k_t)_j */
        for (int d = 0; d < dk; ++d) pred += Sj[d] * (double)kt[d];
        const double vtil = (double)vt[j0 + j] - alpha * pred;
        double acc = 0.0;
        for (int d = 0; d < dk; ++d) {
          const double m_new = mu * Mj[d] - et * (double)kt[d] * vtil;
          const double s_new = alpha * Sj[d] - bt * m_new;
          Mj[d] = m_new;
          Sj[d] = s_new;
          acc += s_new * (double)qt[d];          /* (S_t^T q_t)_j */
        }
        ot[j0 + j] = scale * acc;
      }
    }

    for (int j = 0; j < nc; ++j)
      for (int d = 0; d < dk; ++d) {
        if (S_fin) S_fin[st_off + (size_t)d * dv + (j0 + j)] = S[(size_t)j * dk + d];
        if (M_fin) M_fin[st_off + (size_t)d * dv + (j0 + j)] = M[(size_t)j * dk + d];
      }
    free(S);
    free(M);
  }
  return failed ? -1 : 0;
}
