/*
 * CPU oracle for one routed MoE decode layer whose expert matrices are stored as a
 * vector-quantised part plus a shared-basis low-rank part.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is deliberately plain and slow: it
 * rebuilds every selected expert's dense matrices in fp64 and multiplies them out.  It shares
 * no code with the CUDA library and is called only by the tests, the smoke check and the
 * CPU-baseline timing of the benchmark.
 *
 * Conventions.  bf16 values arrive as uint16 bit patterns and are widened exactly to double.
 * All arithmetic is fp64 with no intermediate rounding.  A projection is stored transposed
 * with respect to the paper's W_e in R^{in x out}: row o of the stored matrix is column o of
 * W_e, so "W_e^T h" (Eq. 1) is a plain row-times-vector product here.
 *
 *   paper symbol            here
 *   B (code book, K x d)    codebook[K][d]
 *   J_e  (in/d x out)       idx[e][out][in/d]      (one index per length-d block of a column)
 *   D    (in x r)           basis[r][in]  = D^T    (shared by the experts of a layer)
 *   C_e  (r x out)          factor[e][out][r] = C_e^T
 *
 * Pinned by tests/test_oracle_pins.py (paper-printed storage rates and sizes, brute force in
 * the paper's own index order, closed forms, library routines).  Float outputs on the large
 * synthetic layers have no paper value to compare with: "parity unpinned" beyond those pins.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_PROJ_VQLR = 0, ORACLE_PROJ_DENSE = 1 };
enum { ORACLE_ACT_SILU = 0, ORACLE_ACT_GELU_TANH = 1,
       ORACLE_ACT_RELU2_UP_ONLY = 2 /* no gate projection: p = max(W_up x, 0)^2 (Section 5.7) */ };

typedef struct {
  int32_t kind;
  int32_t idx_bytes;          /* 1 or 2; 12: indices of 12 bits packed two to three bytes */
  const uint16_t* codebook;   /* [K][d] bf16 */
  const void* idx;            /* [E+S][out][in/d] */
  const uint16_t* basis;      /* [r][in] bf16 or NULL */
  const uint16_t* factor;     /* [E+S][out][r] bf16 or NULL */
  const uint16_t* dense;      /* [E+S][out][in] bf16, kind == DENSE */
} oracle_proj;

typedef struct {
  int32_t H, I, E, k, S, d, K, r;
  int32_t renorm_topk;        /* 1: affinities are a softmax over the k selected logits */
  int32_t act;                /* expert activation phi: ORACLE_ACT_SILU or ORACLE_ACT_GELU_TANH */
  const uint16_t* router_w;   /* [E][H] bf16 */
  const float* router_bias;   /* [E] or NULL */
  oracle_proj gate, up, down;
} oracle_layer;

static double bf16_to_double(uint16_t v) {
  uint32_t u = (uint32_t)v << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

int oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void oracle_set_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}

/* Router scores (Section 2.1): logit[t][e] = <router_w[e], x[t]> + bias[e]. */
void oracle_router_logits(const oracle_layer* L, const uint16_t* x, int T, double* logits) {
  for (int t = 0; t < T; ++t)
    for (int e = 0; e < L->E; ++e) {
      double s = 0.0;
      for (int j = 0; j < L->H; ++j)
        s += bf16_to_double(L->router_w[(size_t)e * L->H + j]) *
             bf16_to_double(x[(size_t)t * L->H + j]);
      if (L->router_bias) s += (double)L->router_bias[e];
      logits[(size_t)t * L->E + e] = s;
    }
}

/* Selection of k experts and their routing affinities a_e (Section 2.1).  Experts are ranked
 * by (logit descending, id ascending); slot s holds the s-th ranked expert.  With renorm the
 * affinities are the softmax over the k selected logits, otherwise the softmax over all E. */
void oracle_topk_affinity(const double* logits, int T, int E, int k, int renorm,
                          int32_t* ids, double* w) {
  char* taken = (char*)malloc((size_t)E);
  for (int t = 0; t < T; ++t) {
    const double* l = logits + (size_t)t * E;
    memset(taken, 0, (size_t)E);
    for (int s = 0; s < k; ++s) {
      int best = -1;
      for (int e = 0; e < E; ++e) {
        if (taken[e]) continue;
        if (best < 0 || l[e] > l[best]) best = e;   /* strict '>' keeps the lower id on ties */
      }
      taken[best] = 1;
      ids[(size_t)t * k + s] = best;
    }
    double lmax = l[ids[(size_t)t * k]];
    double denom = 0.0;
    if (renorm) {
      for (int s = 0; s < k; ++s) denom += exp(l[ids[(size_t)t * k + s]] - lmax);
    } else {
      for (int e = 0; e < E; ++e) denom += exp(l[e] - lmax);
    }
    for (int s = 0; s < k; ++s) w[(size_t)t * k + s] = exp(l[ids[(size_t)t * k + s]] - lmax) / denom;
  }
  free(taken);
}

/* Grouping of the T*k (token, slot) pairs by expert so that each activated expert's payload
 * is used once per layer (Section 5.6, batch scaling).  Pairs of one expert keep ascending
 * token order. */
void oracle_group_by_expert(const int32_t* ids, int T, int k, int E, int32_t* counts,
                            int32_t* offsets, int32_t* pair_token, int32_t* pair_slot) {
  int n = 0;
  for (int e = 0; e < E; ++e) {
    offsets[e] = n;
    counts[e] = 0;
    for (int t = 0; t < T; ++t)
      for (int s = 0; s < k; ++s)
        if (ids[(size_t)t * k + s] == e) {
          pair_token[n] = t;
          pair_slot[n] = s;
          ++n;
          ++counts[e];
        }
  }
  offsets[E] = n;
}

/* Index number `pos` of a map.  The deployed index width b_J(K) grows only when K crosses an
 * encoding boundary (Appendix "Exact engine-work counts"): one byte up to K = 256, two bytes
 * beyond, or -- the packed encoding for 256 < K <= 4096 -- twelve bits, two indices to three
 * bytes, little end first: index 2q sits in byte 3q and the low half of byte 3q+1, index 2q+1 in
 * the high half of byte 3q+1 and byte 3q+2. */
uint32_t oracle_read_index(const void* idx, int idx_bytes, size_t pos) {
  if (idx_bytes == 1) return (uint32_t)((const uint8_t*)idx)[pos];
  if (idx_bytes == 2) return (uint32_t)((const uint16_t*)idx)[pos];
  const uint8_t* b = (const uint8_t*)idx + (pos >> 1) * 3;
  return (pos & 1) ? ((uint32_t)b[1] >> 4) | ((uint32_t)b[2] << 4)
                   : (uint32_t)b[0] | (((uint32_t)b[1] & 0xfu) << 8);
}

static uint32_t read_index(const oracle_proj* P, size_t pos) {
  return oracle_read_index(P->idx, P->idx_bytes, pos);
}

/* Dense reconstruction of one projection of expert e (Eq. 1, transposed):
 *   W[o][b*d + j] = codebook[ idx[e][o][b] ][j] + sum_rho factor[e][o][rho] * basis[rho][b*d+j]
 * or the stored bf16 matrix for a projection that is kept uncompressed (Section 3.1, the down
 * projection).  Returns 0, or 1 when an index is >= K. */
int oracle_reconstruct(const oracle_proj* P, int e, int out_dim, int in_dim, int d, int K,
                       int r, double* W) {
  int bad = 0;
  if (P->kind == ORACLE_PROJ_DENSE) {
#pragma omp parallel for schedule(static)
    for (int o = 0; o < out_dim; ++o)
      for (int j = 0; j < in_dim; ++j)
        W[(size_t)o * in_dim + j] =
            bf16_to_double(P->dense[((size_t)e * out_dim + o) * in_dim + j]);
    return 0;
  }
  const int nb = in_dim / d;
#pragma omp parallel for schedule(static) reduction(| : bad)
  for (int o = 0; o < out_dim; ++o) {
    double* row = W + (size_t)o * in_dim;
    for (int b = 0; b < nb; ++b) {
      uint32_t c = read_index(P, ((size_t)e * out_dim + o) * nb + b);
      if (c >= (uint32_t)K) { bad |= 1; c = 0; }
      for (int j = 0; j < d; ++j) row[b * d + j] = bf16_to_double(P->codebook[(size_t)c * d + j]);
    }
    if (r > 0 && P->basis && P->factor)
      for (int rho = 0; rho < r; ++rho) {
        double a = bf16_to_double(P->factor[((size_t)e * out_dim + o) * r + rho]);
        const uint16_t* brow = P->basis + (size_t)rho * in_dim;
        for (int j = 0; j < in_dim; ++j) row[j] += a * bf16_to_double(brow[j]);
      }
  }
  return bad;
}

/* y = W v for a row-major [out][in] matrix. */
void oracle_matvec(const double* W, const double* v, int out_dim, int in_dim, double* y) {
#pragma omp parallel for schedule(static)
  for (int o = 0; o < out_dim; ++o) {
    double s = 0.0;
    const double* row = W + (size_t)o * in_dim;
    for (int j = 0; j < in_dim; ++j) s += row[j] * v[j];
    y[o] = s;
  }
}

/* The expert activation phi of Section 2.1, which depends on the model:
 * SiLU, phi(v) = v / (1 + exp(-v)) (SwiGLU experts), or the tanh form of GELU,
 * phi(v) = v/2 (1 + tanh(sqrt(2/pi) (v + 0.044715 v^3))) (GeGLU experts). */
double oracle_activation(double v, int act) {
  if (act == ORACLE_ACT_GELU_TANH)
    return 0.5 * v * (1.0 + tanh(sqrt(2.0 / 3.14159265358979323846) * (v + 0.044715 * v * v * v)));
  return v / (1.0 + exp(-v));
}

/* One expert on one token (Section 2.1): g = Wg x, u = Wu x, p = phi(g) * u, y = Wd p.
 * Wd has n_out rows (H, or fewer when rows are sampled). */
void oracle_gated_expert(const double* Wg, const double* Wu, const double* Wd, const double* x,
                         int H, int I, int n_out, int act, double* g, double* u, double* p, double* y) {
  if (act == ORACLE_ACT_RELU2_UP_ONLY) {      /* experts without a gate: p = relu(u)^2, Wg is not read */
    oracle_matvec(Wu, x, I, H, u);
    for (int i = 0; i < I; ++i) { g[i] = 0.0; p[i] = u[i] > 0.0 ? u[i] * u[i] : 0.0; }
    oracle_matvec(Wd, p, n_out, I, y);
    return;
  }
  oracle_matvec(Wg, x, I, H, g);
  oracle_matvec(Wu, x, I, H, u);
  for (int i = 0; i < I; ++i) p[i] = oracle_activation(g[i], act) * u[i];
  oracle_matvec(Wd, p, n_out, I, y);
}

/* The SwiGLU case, phi = SiLU. */
void oracle_swiglu_expert(const double* Wg, const double* Wu, const double* Wd, const double* x,
                          int H, int I, int n_out, double* g, double* u, double* p, double* y) {
  oracle_gated_expert(Wg, Wu, Wd, x, H, I, n_out, ORACLE_ACT_SILU, g, u, p, y);
}

/* The whole layer.  Outputs (each may be NULL except out):
 *   out[T][n_out] f64; logits[T][E]; ids/w[T][k]; counts[E]; offsets[E+1];
 *   pair_token/slot[T*k]; y_pair[T][k+S][n_out] per-slot expert outputs before the weighted
 *   sum (shared experts in slots k..k+S-1).
 *   down_rows: when n_down_rows > 0 only those rows of the down projection are computed and
 *   n_out = n_down_rows (used to sample outputs of layers whose full result is too slow to
 *   compute); otherwise n_out = H.
 * Returns 0, 1 on an index >= K, 2 on allocation failure. */
int oracle_decode_layer(const oracle_layer* L, const uint16_t* x, int T, double* out,
                        double* logits_out, int32_t* ids_out, double* w_out, int32_t* counts_out,
                        int32_t* offsets_out, int32_t* pair_token_out, int32_t* pair_slot_out,
                        double* y_pair_out, const int32_t* down_rows, int n_down_rows) {
  const int H = L->H, I = L->I, E = L->E, k = L->k, S = L->S;
  const int n_out = n_down_rows > 0 ? n_down_rows : H;
  int rc = 0;
  double* logits = (double*)malloc(sizeof(double) * (size_t)T * E);
  int32_t* ids = (int32_t*)malloc(sizeof(int32_t) * (size_t)T * k);
  double* w = (double*)malloc(sizeof(double) * (size_t)T * k);
  int32_t* counts = (int32_t*)malloc(sizeof(int32_t) * (size_t)E);
  int32_t* offsets = (int32_t*)malloc(sizeof(int32_t) * (size_t)(E + 1));
  int32_t* pair_token = (int32_t*)malloc(sizeof(int32_t) * (size_t)T * k);
  int32_t* pair_slot = (int32_t*)malloc(sizeof(int32_t) * (size_t)T * k);
  double* Wg = (double*)malloc(sizeof(double) * (size_t)I * H);
  double* Wu = (double*)malloc(sizeof(double) * (size_t)I * H);
  double* Wd_full = (double*)malloc(sizeof(double) * (size_t)H * I);
  double* Wd = (double*)malloc(sizeof(double) * (size_t)n_out * I);
  double* xd = (double*)malloc(sizeof(double) * (size_t)H);
  double* g = (double*)malloc(sizeof(double) * (size_t)I);
  double* u = (double*)malloc(sizeof(double) * (size_t)I);
  double* p = (double*)malloc(sizeof(double) * (size_t)I);
  double* y_pair = (double*)calloc((size_t)T * (k + S) * n_out, sizeof(double));
  if (!logits || !ids || !w || !counts || !offsets || !pair_token || !pair_slot || !Wg || !Wu ||
      !Wd_full || !Wd || !xd || !g || !u || !p || !y_pair) {
    rc = 2;
    goto done;
  }

  oracle_router_logits(L, x, T, logits);
  oracle_topk_affinity(logits, T, E, k, L->renorm_topk, ids, w);
  oracle_group_by_expert(ids, T, k, E, counts, offsets, pair_token, pair_slot);

  /* every routed expert that received at least one pair, then the always-on shared experts:
   * rebuild its three dense matrices once and run each of its tokens through it */
  for (int e = 0; e < E + S; ++e) {
    const int shared = e >= E;
    const int n_pairs = shared ? T : counts[e];
    if (n_pairs == 0) continue;
    if (L->act != ORACLE_ACT_RELU2_UP_ONLY) rc |= oracle_reconstruct(&L->gate, e, I, H, L->d, L->K, L->r, Wg);
    rc |= oracle_reconstruct(&L->up, e, I, H, L->d, L->K, L->r, Wu);
    rc |= oracle_reconstruct(&L->down, e, H, I, L->d, L->K, L->r, Wd_full);
    for (int q = 0; q < n_out; ++q) {
      const int row = n_down_rows > 0 ? down_rows[q] : q;
      memcpy(Wd + (size_t)q * I, Wd_full + (size_t)row * I, sizeof(double) * (size_t)I);
    }
    for (int q = 0; q < n_pairs; ++q) {
      const int t = shared ? q : pair_token[offsets[e] + q];
      const int slot = shared ? k + (e - E) : pair_slot[offsets[e] + q];
      for (int j = 0; j < H; ++j) xd[j] = bf16_to_double(x[(size_t)t * H + j]);
      oracle_gated_expert(Wg, Wu, Wd, xd, H, I, n_out, L->act, g, u, p,
                          y_pair + ((size_t)t * (k + S) + slot) * n_out);
    }
  }
  /* weighted sum in slot order (Section 2.1: scale each selected expert's output by its
   * affinity and sum); shared experts enter with weight 1 */
  for (int t = 0; t < T; ++t)
    for (int j = 0; j < n_out; ++j) {
      double acc = 0.0;
      for (int s = 0; s < k + S; ++s) {
        const double a = s < k ? w[(size_t)t * k + s] : 1.0;
        acc += a * y_pair[((size_t)t * (k + S) + s) * n_out + j];
      }
      out[(size_t)t * n_out + j] = acc;
    }

  if (logits_out) memcpy(logits_out, logits, sizeof(double) * (size_t)T * E);
  if (ids_out) memcpy(ids_out, ids, sizeof(int32_t) * (size_t)T * k);
  if (w_out) memcpy(w_out, w, sizeof(double) * (size_t)T * k);
  if (counts_out) memcpy(counts_out, counts, sizeof(int32_t) * (size_t)E);
  if (offsets_out) memcpy(offsets_out, offsets, sizeof(int32_t) * (size_t)(E + 1));
  if (pair_token_out) memcpy(pair_token_out, pair_token, sizeof(int32_t) * (size_t)T * k);
  if (pair_slot_out) memcpy(pair_slot_out, pair_slot, sizeof(int32_t) * (size_t)T * k);
  if (y_pair_out) memcpy(y_pair_out, y_pair, sizeof(double) * (size_t)T * (k + S) * n_out);
done:
  free(logits); free(ids); free(w); free(counts); free(offsets); free(pair_token);
  free(pair_slot); free(Wg); free(Wu); free(Wd_full); free(Wd); free(xd); free(g); free(u);
  free(p); free(y_pair);
  return rc;
}

/* ------------------------------------------------------------------------------------------
 * The paper's own way to evaluate the VQ term (Section 4.2, "reuse of shared projections"):
 * first the projection code book  Tp[b][c] = <x_b, codebook[c]>  for every length-d block x_b
 * of the input, once per token; then each output is a sum of selected entries plus the
 * low-rank term,  o[i] = sum_b Tp[b][ idx[e][i][b] ] + sum_rho factor[e][i][rho] * z[rho]
 * with z = basis * x computed once per token ("joint accumulation").  Algebraically equal to
 * row i of the reconstructed matrix times x.
 * ---------------------------------------------------------------------------------------- */
void oracle_projection_codebook(const uint16_t* codebook, const double* x, int in_dim, int d,
                                int K, double* Tp /* [in/d][K] */) {
  const int nb = in_dim / d;
  for (int b = 0; b < nb; ++b)
    for (int c = 0; c < K; ++c) {
      double s = 0.0;
      for (int j = 0; j < d; ++j) s += x[b * d + j] * bf16_to_double(codebook[(size_t)c * d + j]);
      Tp[(size_t)b * K + c] = s;
    }
}

void oracle_basis_projection(const uint16_t* basis, const double* x, int in_dim, int r,
                             double* z) {
  for (int rho = 0; rho < r; ++rho) {
    double s = 0.0;
    for (int j = 0; j < in_dim; ++j) s += bf16_to_double(basis[(size_t)rho * in_dim + j]) * x[j];
    z[rho] = s;
  }
}

void oracle_project_shared(const oracle_proj* P, int e, int out_dim, int in_dim, int d, int K,
                           int r, const double* x, double* o) {
  const int nb = in_dim / d;
  double* Tp = (double*)malloc(sizeof(double) * (size_t)nb * K);
  double* z = (double*)calloc((size_t)(r > 0 ? r : 1), sizeof(double));
  oracle_projection_codebook(P->codebook, x, in_dim, d, K, Tp);
  if (r > 0 && P->basis) oracle_basis_projection(P->basis, x, in_dim, r, z);
  for (int i = 0; i < out_dim; ++i) {
    double s = 0.0;
    for (int b = 0; b < nb; ++b)
      s += Tp[(size_t)b * K + read_index(P, ((size_t)e * out_dim + i) * nb + b)];
    if (r > 0 && P->basis && P->factor)
      for (int rho = 0; rho < r; ++rho)
        s += bf16_to_double(P->factor[((size_t)e * out_dim + i) * r + rho]) * z[rho];
    o[i] = s;
  }
  free(Tp);
  free(z);
}

/* ------------------------------------------------------------------------------------------
 * Accounting.
 * ---------------------------------------------------------------------------------------- */
/* Storage rate in bits per original weight of one projection (Appendix "Exact rate
 * accounting"):  log2(K)/d + b_C r/H + (b_B K d + b_D H r)/(E H I), where the index term is
 * the deployed index width b_J over d. */
double oracle_storage_bits_per_weight(int d, int K, int r, int H, int I, int E, int b_J,
                                      int b_C, int b_B, int b_D) {
  (void)K;
  return (double)b_J / d + (double)b_C * r / H +
         ((double)b_B * K * d + (double)b_D * H * r) / ((double)E * H * I);
}

/* Leading-order decode work for one projection (Appendix "Exact engine-work counts"):
 *   out[0] shared code-book-projection MACs  H K      out[1] shared basis MACs   H r
 *   out[2] shared load bits of the code book 16 K d   out[3] shared load bits of D  16 H r
 *   out[4] private index bits  (H I / d) b_J          out[5] private coefficient bits 16 I r
 *   out[6] private selections  H I / d                out[7] private VQ adds  H I / d
 *   out[8] private low-rank MACs  I r */
void oracle_work_counts(int H, int I, int d, int K, int r, int b_J, double* out) {
  out[0] = (double)H * K;
  out[1] = (double)H * r;
  out[2] = 16.0 * K * d;
  out[3] = 16.0 * H * r;
  out[4] = (double)H * I / d * b_J;
  out[5] = 16.0 * I * r;
  out[6] = (double)H * I / d;
  out[7] = (double)H * I / d;
  out[8] = (double)I * r;
}
