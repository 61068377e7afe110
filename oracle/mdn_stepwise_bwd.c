/*
 * TEST INFRASTRUCTURE, NOT THE PRODUCT.  CPU oracle for the MDN backward.
 *
 * Reverse-mode differentiation of the stepwise recurrence of Section 3.1 (Eq. 5-6), token by token, in fp64:
 *
 *     v~_t = v_t - alpha_t S_{t-1}^T k_t      M_t = mu_t M_{t-1} - eta_t k_t v~_t^T
 *     S_t  = alpha_t S_{t-1} - beta_t M_t     o_t = scale S_t^T q_t
 *
 * Given the loss gradients dO (and optionally dS_T, dM_T of the final states), walking t = T-1 .. 0 with the
 * adjoints GS, GM of the states AFTER token t:
 *
 *     GS   += scale q_t dO_t^T                    dq_t    = scale S_t dO_t
 *     dbeta_t = -<GS, M_t>                        GM     += -beta_t GS
 *     a     = GM v~_t                             deta_t  = -k_t . a          dk_t  = -eta_t a
 *     dv~   = -eta_t GM^T k_t                     dv_t    = dv~
 *     dalpha_t = <GS, S_{t-1}> - dv~ . (S_{t-1}^T k_t)                         dk_t -= alpha_t S_{t-1} dv~
 *     dmu_t = <GM, M_{t-1}>
 *     GS  <- alpha_t (GS - k_t dv~^T)             GM  <- mu_t GM
 *
 * and d log_alpha = alpha dalpha, d log_mu = mu dmu (the library's gates are the logarithms).  The states the
 * formulas need are recomputed from checkpoints kept every CK tokens; nothing else is blocked, fused or reordered.
 * One OpenMP task per (sequence, head) chain.  The paper trains with the chunkwise algorithm's backward (Section
 * 3.1, "materialise V~, reconstruct the states"); its result is the gradient of the same function, which is what
 * this file evaluates.  Pinned by central finite differences of the forward oracle (tests/test_oracle_bwd_pins.py).
 *
 * Nothing in the CUDA path includes, links or calls this file, and this file uses nothing of the CUDA path.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define CK 64

/* one forward token on full matrices S, M [dk][dv] (row-major); returns v~ in vt[dv] and S_{t-1}^T k in pred[dv] */
static void step_forward(int dk, int dv, double* S, double* M, const float* k, const float* v, double alpha, double mu,
                         double beta, double eta, double* vt, double* pred) {
  for (int j = 0; j < dv; ++j) pred[j] = 0.0;
  for (int d = 0; d < dk; ++d)
    for (int j = 0; j < dv; ++j) pred[j] += S[(size_t)d * dv + j] * (double)k[d];
  for (int j = 0; j < dv; ++j) vt[j] = (double)v[j] - alpha * pred[j];
  for (int d = 0; d < dk; ++d)
    for (int j = 0; j < dv; ++j) {
      const double m_new = mu * M[(size_t)d * dv + j] - eta * (double)k[d] * vt[j];
      M[(size_t)d * dv + j] = m_new;
      S[(size_t)d * dv + j] = alpha * S[(size_t)d * dv + j] - beta * m_new;
    }
}

/*
 * Layout as in mdn_oracle_stepwise.  d_o: [tokens,H,dv] float32; dSf, dMf: [N,H,dk,dv] float32 or NULL (zeros).
 * Outputs (double, only the selected chains' entries are written): dq, dk [tokens,H,dk]; dv [tokens,H,dv];
 * dbeta, dlog_alpha, dlog_mu, deta [tokens,H] (deta may be NULL); dS0, dM0 [N,H,dk,dv] (may be NULL).
 */
int mdn_oracle_stepwise_bwd(int64_t num_seqs, const int64_t* seq_start, const int64_t* seq_len, int H, int dk, int dv,
                            const float* q, const float* k, const float* v, const float* beta,
                            const float* log_alpha, const float* log_mu, const float* eta, double scale,
                            const float* S0, const float* M0, const int32_t* chains, int64_t n_chains,
                            const float* d_o, const float* dSf, const float* dMf, double* dq, double* dk_out,
                            double* dv_out, double* dbeta, double* dlog_alpha, double* dlog_mu, double* deta,
                            double* dS0, double* dM0) {
  if (num_seqs <= 0 || H <= 0 || dk <= 0 || dv <= 0 || !q || !k || !v || !beta || !log_alpha || !log_mu || !d_o ||
      !dq || !dk_out || !dv_out || !dbeta || !dlog_alpha || !dlog_mu)
    return -1;
  const int64_t total = chains ? n_chains : num_seqs * (int64_t)H;
  const size_t mat = (size_t)dk * dv;
  int failed = 0;

#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t ci = 0; ci < total; ++ci) {
    const int64_t chain = chains ? (int64_t)chains[ci] : ci;
    const int64_t n = chain / H;
    const int h = (int)(chain % H);
    const int64_t t0 = seq_start[n], len = seq_len[n];
    const int64_t nck = (len + CK - 1) / CK;
    const size_t st_off = ((size_t)n * H + h) * mat;
    double* ckS = (double*)malloc(sizeof(double) * mat * (size_t)(nck > 0 ? nck : 1));
    double* ckM = (double*)malloc(sizeof(double) * mat * (size_t)(nck > 0 ? nck : 1));
    double* prevS = (double*)malloc(sizeof(double) * mat * CK);   /* S_{t-1} for the tokens of one segment */
    double* prevM = (double*)malloc(sizeof(double) * mat * CK);
    double* S = (double*)malloc(sizeof(double) * mat);
    double* M = (double*)malloc(sizeof(double) * mat);
    double* GS = (double*)malloc(sizeof(double) * mat);
    double* GM = (double*)malloc(sizeof(double) * mat);
    double* vec = (double*)malloc(sizeof(double) * (size_t)(4 * dv + 2 * dk));
    if (!ckS || !ckM || !prevS || !prevM || !S || !M || !GS || !GM || !vec) {
#pragma omp atomic write
      failed = 1;
    } else {
      double* vt = vec; double* pred = vec + dv; double* dvt = vec + 2 * dv; double* dO = vec + 3 * dv;
      double* a = vec + 4 * dv; double* e = a + dk;
      for (size_t i = 0; i < mat; ++i) {
        S[i] = S0 ? (double)S0[st_off + i] : 0.0;
        M[i] = M0 ? (double)M0[st_off + i] : 0.0;
        GS[i] = dSf ? (double)dSf[st_off + i] : 0.0;
        GM[i] = dMf ? (double)dMf[st_off + i] : 0.0;
      }
      /* forward: keep the state at the start of every segment */
      for (int64_t c = 0; c < nck; ++c) {
        memcpy(ckS + (size_t)c * mat, S, sizeof(double) * mat);
        memcpy(ckM + (size_t)c * mat, M, sizeof(double) * mat);
        const int64_t tb = c * CK, te = (tb + CK < len) ? tb + CK : len;
        for (int64_t t = tb; t < te; ++t) {
          const size_t g = (size_t)(t0 + t) * H + h;
          step_forward(dk, dv, S, M, k + g * dk, v + g * dv, exp((double)log_alpha[g]), exp((double)log_mu[g]),
                       (double)beta[g], eta ? (double)eta[g] : 1.0, vt, pred);
        }
      }
      /* backward, segment by segment */
      for (int64_t c = nck - 1; c >= 0; --c) {
        const int64_t tb = c * CK, te = (tb + CK < len) ? tb + CK : len;
        memcpy(S, ckS + (size_t)c * mat, sizeof(double) * mat);
        memcpy(M, ckM + (size_t)c * mat, sizeof(double) * mat);
        for (int64_t t = tb; t < te; ++t) {
          memcpy(prevS + (size_t)(t - tb) * mat, S, sizeof(double) * mat);
          memcpy(prevM + (size_t)(t - tb) * mat, M, sizeof(double) * mat);
          const size_t g = (size_t)(t0 + t) * H + h;
          step_forward(dk, dv, S, M, k + g * dk, v + g * dv, exp((double)log_alpha[g]), exp((double)log_mu[g]),
                       (double)beta[g], eta ? (double)eta[g] : 1.0, vt, pred);
        }
        for (int64_t t = te - 1; t >= tb; --t) {
          const size_t g = (size_t)(t0 + t) * H + h;
          const double alpha = exp((double)log_alpha[g]), mu = exp((double)log_mu[g]);
          const double bt = (double)beta[g], et = eta ? (double)eta[g] : 1.0;
          const float* kt = k + g * dk;
          const float* qt = q + g * dk;
          const double* Sp = prevS + (size_t)(t - tb) * mat;   /* S_{t-1} */
          const double* Mp = prevM + (size_t)(t - tb) * mat;   /* M_{t-1} */
          /* recompute v~_t, pred, M_t, S_t from the stored previous state */
          for (int j = 0; j < dv; ++j) pred[j] = 0.0;
          for (int d = 0; d < dk; ++d)
            for (int j = 0; j < dv; ++j) pred[j] += Sp[(size_t)d * dv + j] * (double)kt[d];
          for (int j = 0; j < dv; ++j) {
            vt[j] = (double)v[g * dv + j] - alpha * pred[j];
            dO[j] = (double)d_o[g * dv + j];
          }
          double d_beta = 0.0, d_alpha = 0.0, d_mu = 0.0, d_eta = 0.0;
          for (int d = 0; d < dk; ++d) {
            double dq_d = 0.0;
            for (int j = 0; j < dv; ++j) {
              const size_t i = (size_t)d * dv + j;
              const double m_t = mu * Mp[i] - et * (double)kt[d] * vt[j];
              const double s_t = alpha * Sp[i] - bt * m_t;
              GS[i] += scale * (double)qt[d] * dO[j];        /* o_t = scale S_t^T q_t */
              dq_d += s_t * dO[j];
              d_beta -= GS[i] * m_t;                        /* S_t = alpha S_{t-1} - beta M_t */
              GM[i] -= bt * GS[i];
            }
            dq[g * dk + d] = scale * dq_d;
          }
          for (int j = 0; j < dv; ++j) dvt[j] = 0.0;
          for (int d = 0; d < dk; ++d) {
            double a_d = 0.0;
            for (int j = 0; j < dv; ++j) {
              const size_t i = (size_t)d * dv + j;
              a_d += GM[i] * vt[j];                          /* M_t = mu M_{t-1} - eta k v~^T */
              dvt[j] -= et * GM[i] * (double)kt[d];
              d_mu += GM[i] * Mp[i];
            }
            a[d] = a_d;
            d_eta -= (double)kt[d] * a_d;
          }
          for (int d = 0; d < dk; ++d) {
            double e_d = 0.0;
            for (int j = 0; j < dv; ++j) {
              const size_t i = (size_t)d * dv + j;
              e_d += Sp[i] * dvt[j];                         /* v~ = v - alpha S_{t-1}^T k */
              d_alpha += GS[i] * Sp[i];
            }
            e[d] = e_d;
            dk_out[g * dk + d] = -et * a[d] - alpha * e_d;
          }
          for (int j = 0; j < dv; ++j) {
            d_alpha -= dvt[j] * pred[j];
            dv_out[g * dv + j] = dvt[j];
          }
          dbeta[g] = d_beta;
          dlog_alpha[g] = alpha * d_alpha;
          dlog_mu[g] = mu * d_mu;
          if (deta) deta[g] = d_eta;
          for (int d = 0; d < dk; ++d)
            for (int j = 0; j < dv; ++j) {
              const size_t i = (size_t)d * dv + j;
              GS[i] = alpha * (GS[i] - (double)kt[d] * dvt[j]);
              GM[i] = mu * GM[i];
            }
        }
      }
      for (size_t i = 0; i < mat; ++i) {
        if (dS0) dS0[st_off + i] = GS[i];
        if (dM0) dM0[st_off + i] = GM[i];
      }
    }
    free(ckS); free(ckM); free(prevS); free(prevM); free(S); free(M); free(GS); free(GM); free(vec);
  }
  return failed ? -1 : 0;
}
