/*
 * CodeNet CPU oracle -- TEST INFRASTRUCTURE ONLY (see codenet_oracle.h).
 *
 * Plain loops over the node grid, double accumulation, no tiling, no fusion.  Each function
 * names the passage of the paper it follows.
 */
#include "codenet_oracle.h"

#include <float.h>
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------------------------------ */
/* helpers                                                                                    */
/* ------------------------------------------------------------------------------------------ */

static int g_threads = 1;

void orc_set_threads(int n) {
  g_threads = n < 1 ? 1 : n;
#ifdef _OPENMP
  omp_set_num_threads(g_threads);
#else
  g_threads = 1;
#endif
}
int orc_get_threads(void) { return g_threads; }

/* bfloat16 storage emulation: round-to-nearest-even on the upper 16 bits of a float. */
static float round_bf16(float x) {
  uint32_t u;
  memcpy(&u, &x, 4);
  u += 0x7FFFu + ((u >> 16) & 1u);
  u &= 0xFFFF0000u;
  memcpy(&x, &u, 4);
  return x;
}

struct orc_layer {
  orc_desc_t d;
  int b_r, b_c, M, Nn, T, ns, Tc, nsc, n_out_p, n_in_p;
  double* P_row; /* m x r_row */
  double* P_col; /* n x r_col */
  float** blk;   /* M*Nn pointers, NULL where no node exists (corner) */
  float** u;     /* per stored block: ns x b_c inner checksum rows */
  float** v;     /* per stored block: nsc x b_r inner checksum columns */
  float** ck_blk; /* the last checkpoint (same shapes), NULL until one is taken */
  float** ck_u;
  float** ck_v;
  orc_small_faults_t small;  /* soft errors in the small steps; all probabilities zero: none */
  int have_small;
  uint32_t small_iteration;  /* iteration of the call in progress (orc_forward / orc_backward_update set it) */
};

static float store_w(const orc_layer_t* L, double x) {
  float f = (float)x;
  return L->d.store_bf16 ? round_bf16(f) : f;
}

static int has_node(const orc_layer_t* L, int i, int j) {
  return i >= 0 && j >= 0 && i < L->M && j < L->Nn && (i < L->d.m || j < L->d.n);
}

/* Generator entries: G_r[a, i] (m x M) and G_c[b, j] (n x Nn), systematic: [I | P]. */
static double g_row(const orc_layer_t* L, int a, int i) {
  if (i < L->d.m) return a == i ? 1.0 : 0.0;
  return L->P_row[a * L->d.r_row + (i - L->d.m)];
}
static double g_col(const orc_layer_t* L, int b, int j) {
  if (j < L->d.n) return b == j ? 1.0 : 0.0;
  return L->P_col[b * L->d.r_col + (j - L->d.n)];
}

/* ------------------------------------------------------------------------------------------ */
/* counter-based random numbers (Philox4x32-10, Salmon et al.) and the soft-error noise       */
/* ------------------------------------------------------------------------------------------ */

void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    uint64_t p0 = (uint64_t)0xD2511F53u * c0;
    uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
    uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    uint32_t n1 = (uint32_t)p1;
    uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    uint32_t n3 = (uint32_t)p0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Additive continuous-valued noise on an erroneous node's output (Error Model 2).  Twelve
 * 16-bit uniforms are summed (Irwin-Hall, unit variance after scaling); everything is integer
 * until the final float products, so any implementation reproduces the same bits. */
float orc_noise(uint32_t seed, uint32_t layer, uint32_t phase, uint32_t iteration,
                uint32_t node_id, uint32_t element, float sigma) {
  uint32_t key[2] = {seed, (layer << 8) | phase};
  uint32_t c1[4] = {iteration, node_id, element, 1u};
  uint32_t c2[4] = {iteration, node_id, element, 2u};
  uint32_t a[4], b[4];
  orc_philox4x32_10(c1, key, a);
  orc_philox4x32_10(c2, key, b);
  int32_t sum = 0;
  for (int w = 0; w < 4; ++w) sum += (int32_t)(a[w] & 0xFFFFu) + (int32_t)(a[w] >> 16);
  for (int w = 0; w < 2; ++w) sum += (int32_t)(b[w] & 0xFFFFu) + (int32_t)(b[w] >> 16);
  int32_t v = sum - 393210; /* 12 * 32767.5 */
  float unit = (float)v * (1.0f / 65536.0f);
  return sigma * unit;
}

int orc_node_hit(const orc_fault_t* f, uint32_t phase, uint32_t iteration, uint32_t node_id,
                 uint32_t active_index, uint32_t n_active) {
  if (!f || f->mode == ORC_FAULT_NONE) return 0;
  uint32_t key[2] = {f->seed, (f->layer << 8) | phase};
  uint32_t out[4];
  if (f->mode == ORC_FAULT_BERNOULLI) {
    uint32_t c[4] = {iteration, node_id, 0u, 0u};
    orc_philox4x32_10(c, key, out);
    return out[0] < f->p_q32;
  }
  if (f->mode == ORC_FAULT_EXACTLY_ONE) {
    uint32_t c[4] = {iteration, 0xFFFFFFFFu, 0u, 0u};
    orc_philox4x32_10(c, key, out);
    return (out[0] % n_active) == active_index;
  }
  return 0;
}

int orc_small_hit(const orc_small_faults_t* plan, uint32_t phase, uint32_t iteration, uint32_t unit) {
  if (!plan) return 0;
  const uint32_t p = phase == ORC_PHASE_ENCODE ? plan->p_encode_q32 : phase == ORC_PHASE_INPUT ? plan->p_input_q32
                   : phase == ORC_PHASE_CHECK ? plan->p_check_q32 : plan->p_decode_q32;
  if (p == 0) return 0;
  uint32_t key[2] = {plan->seed, (plan->layer << 8) | phase};
  uint32_t c[4] = {iteration, unit, 0u, 0u}, out[4];
  orc_philox4x32_10(c, key, out);
  return out[0] < p;
}

void orc_layer_set_small_faults(orc_layer_t* L, const orc_small_faults_t* plan) {
  L->have_small = plan != NULL;
  if (plan) L->small = *plan;
}

/* ------------------------------------------------------------------------------------------ */
/* initial encoding (Claim 1): W~ = (G_r^T (x) I) W (G_c (x) I), corner blocks not computed    */
/* ------------------------------------------------------------------------------------------ */

static void recompute_checksums(orc_layer_t* L, int i, int j) {
  const float* w = L->blk[i * L->Nn + j];
  float* u = L->u[i * L->Nn + j];
  float* v = L->v[i * L->Nn + j];
  for (int s = 0; s < L->ns; ++s)
    for (int c = 0; c < L->b_c; ++c) {
      double acc = 0.0;
      for (int r = s * L->T; r < (s + 1) * L->T; ++r) acc += (double)w[r * L->b_c + c];
      u[s * L->b_c + c] = (float)acc;
    }
  for (int s = 0; s < L->nsc; ++s)
    for (int r = 0; r < L->b_r; ++r) {
      double acc = 0.0;
      for (int c = s * L->Tc; c < (s + 1) * L->Tc; ++c) acc += (double)w[r * L->b_c + c];
      v[s * L->b_r + r] = (float)acc;
    }
}

orc_layer_t* orc_layer_create(const orc_desc_t* d, const float* W) {
  if (!d || !W || d->m < 1 || d->n < 1 || d->r_row < 0 || d->r_col < 0) return NULL;
  if (d->m + d->r_row > 64 || d->n + d->r_col > 64) return NULL;
  orc_layer_t* L = (orc_layer_t*)calloc(1, sizeof(*L));
  L->d = *d;
  L->b_r = (d->n_out + d->m - 1) / d->m;
  L->b_c = (d->n_in + d->n - 1) / d->n;
  L->n_out_p = L->b_r * d->m;
  L->n_in_p = L->b_c * d->n;
  L->M = d->m + d->r_row;
  L->Nn = d->n + d->r_col;
  L->T = d->check_rows > 0 ? d->check_rows : L->b_r;
  if (L->b_r % L->T != 0) { free(L); return NULL; }
  L->ns = L->b_r / L->T;
  L->Tc = d->check_cols > 0 ? d->check_cols : L->b_c;
  if (L->b_c % L->Tc != 0) { free(L); return NULL; }
  L->nsc = L->b_c / L->Tc;
  L->P_row = (double*)calloc((size_t)d->m * (d->r_row > 0 ? d->r_row : 1), sizeof(double));
  L->P_col = (double*)calloc((size_t)d->n * (d->r_col > 0 ? d->r_col : 1), sizeof(double));
  for (int k = 0; k < d->m * d->r_row; ++k) L->P_row[k] = d->P_row ? (double)d->P_row[k] : 1.0;
  for (int k = 0; k < d->n * d->r_col; ++k) L->P_col[k] = d->P_col ? (double)d->P_col[k] : 1.0;
  L->d.P_row = NULL;
  L->d.P_col = NULL;
  L->blk = (float**)calloc((size_t)L->M * L->Nn, sizeof(float*));
  L->u = (float**)calloc((size_t)L->M * L->Nn, sizeof(float*));
  L->v = (float**)calloc((size_t)L->M * L->Nn, sizeof(float*));
  const size_t bsz = (size_t)L->b_r * L->b_c;
#pragma omp parallel for collapse(2) schedule(dynamic)
  for (int i = 0; i < L->M; ++i)
    for (int j = 0; j < L->Nn; ++j) {
      if (!has_node(L, i, j)) continue;
      float* w = (float*)malloc(bsz * sizeof(float));
      L->blk[i * L->Nn + j] = w;
      L->u[i * L->Nn + j] = (float*)malloc((size_t)L->ns * L->b_c * sizeof(float));
      L->v[i * L->Nn + j] = (float*)malloc((size_t)L->nsc * L->b_r * sizeof(float));
      for (int r = 0; r < L->b_r; ++r)
        for (int c = 0; c < L->b_c; ++c) {
          double acc = 0.0;
          for (int a = 0; a < d->m; ++a) {
            double ga = g_row(L, a, i);
            if (ga == 0.0) continue;
            for (int b = 0; b < d->n; ++b) {
              double gb = g_col(L, b, j);
              if (gb == 0.0) continue;
              int gr = a * L->b_r + r, gc = b * L->b_c + c;
              double wv = (gr < d->n_out && gc < d->n_in) ? (double)W[(size_t)gr * d->n_in + gc] : 0.0;
              acc += ga * gb * wv;
            }
          }
          w[(size_t)r * L->b_c + c] = store_w(L, acc);
        }
      recompute_checksums(L, i, j);
    }
  return L;
}

void orc_layer_free(orc_layer_t* L) {
  if (!L) return;
  for (int k = 0; k < L->M * L->Nn; ++k) {
    free(L->blk[k]); free(L->u[k]); free(L->v[k]);
    if (L->ck_blk) { free(L->ck_blk[k]); free(L->ck_u[k]); free(L->ck_v[k]); }
  }
  free(L->ck_blk); free(L->ck_u); free(L->ck_v);
  free(L->blk); free(L->u); free(L->v); free(L->P_row); free(L->P_col); free(L);
}

/* Checkpoint of everything the layer stores between iterations (Section "Decentralized implementation":
 * an uncorrectable pattern restores the weight matrices from the last checkpoint; Theorem 2, assumptions
 * (ii) and (iv)): the coded blocks and their inner checksums, copied as they are. */
int orc_checkpoint_save(orc_layer_t* L) {
  const int nb = L->M * L->Nn;
  if (!L->ck_blk) {
    L->ck_blk = (float**)calloc((size_t)nb, sizeof(float*));
    L->ck_u = (float**)calloc((size_t)nb, sizeof(float*));
    L->ck_v = (float**)calloc((size_t)nb, sizeof(float*));
    if (!L->ck_blk || !L->ck_u || !L->ck_v) return -2;
    for (int k = 0; k < nb; ++k) {
      if (!L->blk[k]) continue;
      L->ck_blk[k] = (float*)malloc((size_t)L->b_r * L->b_c * sizeof(float));
      L->ck_u[k] = (float*)malloc((size_t)L->ns * L->b_c * sizeof(float));
      L->ck_v[k] = (float*)malloc((size_t)L->nsc * L->b_r * sizeof(float));
      if (!L->ck_blk[k] || !L->ck_u[k] || !L->ck_v[k]) return -2;
    }
  }
  for (int k = 0; k < nb; ++k) {
    if (!L->blk[k]) continue;
    memcpy(L->ck_blk[k], L->blk[k], (size_t)L->b_r * L->b_c * sizeof(float));
    memcpy(L->ck_u[k], L->u[k], (size_t)L->ns * L->b_c * sizeof(float));
    memcpy(L->ck_v[k], L->v[k], (size_t)L->nsc * L->b_r * sizeof(float));
  }
  return 0;
}

int orc_checkpoint_restore(orc_layer_t* L) {
  if (!L->ck_blk) return -1; /* none taken */
  for (int k = 0; k < L->M * L->Nn; ++k) {
    if (!L->blk[k]) continue;
    memcpy(L->blk[k], L->ck_blk[k], (size_t)L->b_r * L->b_c * sizeof(float));
    memcpy(L->u[k], L->ck_u[k], (size_t)L->ns * L->b_c * sizeof(float));
    memcpy(L->v[k], L->ck_v[k], (size_t)L->nsc * L->b_r * sizeof(float));
  }
  return 0;
}

void orc_layer_dims(const orc_layer_t* L, int32_t dims[10]) {
  dims[0] = L->b_r; dims[1] = L->b_c; dims[2] = L->M; dims[3] = L->Nn;
  dims[4] = L->T; dims[5] = L->ns; dims[6] = L->n_out_p; dims[7] = L->n_in_p;
  dims[8] = L->Tc; dims[9] = L->nsc;
}

int orc_get_block(const orc_layer_t* L, int i, int j, float* out) {
  if (!has_node(L, i, j)) return -1;
  memcpy(out, L->blk[i * L->Nn + j], (size_t)L->b_r * L->b_c * sizeof(float));
  return 0;
}
int orc_get_u(const orc_layer_t* L, int i, int j, float* out) {
  if (!has_node(L, i, j)) return -1;
  memcpy(out, L->u[i * L->Nn + j], (size_t)L->ns * L->b_c * sizeof(float));
  return 0;
}
int orc_get_v(const orc_layer_t* L, int i, int j, float* out) {
  if (!has_node(L, i, j)) return -1;
  memcpy(out, L->v[i * L->Nn + j], (size_t)L->nsc * L->b_r * sizeof(float));
  return 0;
}
int orc_set_block(orc_layer_t* L, int i, int j, const float* in) {
  if (!has_node(L, i, j)) return -1;
  memcpy(L->blk[i * L->Nn + j], in, (size_t)L->b_r * L->b_c * sizeof(float));
  return 0;
}

/* ------------------------------------------------------------------------------------------ */
/* faults in the stored blocks, and regeneration of a block from its code                      */
/* (Section "Experimental Results": a sparse matrix added to a node's stored sub-matrix;        */
/*  feedforward stage, "regenerate" step: the sub-matrix of an erroneous node is rebuilt from   */
/*  the sub-matrices of the other nodes of its grid column / row)                               */
/* ------------------------------------------------------------------------------------------ */

/* Adds a sparse random matrix to the stored block (i, j): element e = row * b_c + col changes
 * when word 0 of Philox(counter = (iteration, node, e, 3), key = (seed, layer << 8 | 2)) is below
 * density_q32; the value added is amplitude * u with u uniform on [-1, 1) from the upper 24 bits
 * of word 1.  Returns the number of elements changed, or -1 if the block does not exist. */
long orc_corrupt_block(orc_layer_t* L, int i, int j, uint32_t seed, uint32_t layer, uint32_t iteration,
                       uint32_t density_q32, float amplitude) {
  if (!has_node(L, i, j)) return -1;
  const uint32_t key[2] = {seed, (layer << 8) | 2u};
  const uint32_t node_id = (uint32_t)(i * L->Nn + j);
  float* w = L->blk[i * L->Nn + j];
  long changed = 0;
  for (uint32_t e = 0; e < (uint32_t)(L->b_r * L->b_c); ++e) {
    uint32_t c[4] = {iteration, node_id, e, 3u}, out[4];
    orc_philox4x32_10(c, key, out);
    if (out[0] >= density_q32) continue;
    volatile float unit = (float)(out[1] >> 8) * (1.0f / 8388608.0f) - 1.0f; /* exact */
    volatile float add = amplitude * unit;
    volatile float sum = w[e] + add;
    w[e] = L->d.store_bf16 ? round_bf16(sum) : sum;
    ++changed;
  }
  return changed;
}

/* Rebuilds the stored block (i, j) from the other blocks of its block-column (along = 0: the M
 * blocks of block-column j are a G_r codeword, element by element) or of its block-row
 * (along = 1: the Nn blocks of block-row i are a G_c codeword).  A data block is solved from
 * the lowest-indexed parity whose generator entry is not zero; a parity block is re-encoded.
 * Returns 0, -1 if the block does not exist, -2 if that direction has no redundancy for it. */
int orc_regenerate_block(orc_layer_t* L, int i, int j, int along) {
  if (!has_node(L, i, j)) return -1;
  const int kd = along == 0 ? L->d.m : L->d.n;          /* data positions of the codeword */
  const int r = along == 0 ? L->d.r_row : L->d.r_col;   /* parities */
  const int pos = along == 0 ? i : j;                   /* position of the block in it */
  const double* P = along == 0 ? L->P_row : L->P_col;   /* kd x r */
  /* the codeword exists only where the other coordinate is a data index (no corner blocks) */
  if (r < 1 || (along == 0 ? j >= L->d.n : i >= L->d.m)) return -2;
  double coef[128];
  int use[128], n_use = 0;
  if (pos >= kd) {                                      /* parity block: sum_k P[k, pos - kd] * block_k */
    for (int k = 0; k < kd; ++k) { use[n_use] = k; coef[n_use++] = P[k * r + (pos - kd)]; }
  } else {
    int q = -1;
    for (int t = 0; t < r && q < 0; ++t)
      if (P[pos * r + t] != 0.0) q = t;
    if (q < 0) return -2;
    const double inv = 1.0 / P[pos * r + q];            /* block = (parity_q - sum_{k != pos} P[k,q] block_k) / P[pos,q] */
    for (int k = 0; k < kd; ++k)
      if (k != pos) { use[n_use] = k; coef[n_use++] = -P[k * r + q] * inv; }
    use[n_use] = kd + q; coef[n_use++] = inv;
  }
  float* dst = L->blk[i * L->Nn + j];
  const size_t n_el = (size_t)L->b_r * L->b_c;
  for (size_t e = 0; e < n_el; ++e) {
    double acc = 0.0;
    for (int t = 0; t < n_use; ++t) {
      const float* src = along == 0 ? L->blk[use[t] * L->Nn + j] : L->blk[i * L->Nn + use[t]];
      acc += coef[t] * (double)src[e];
    }
    dst[e] = store_w(L, acc);
  }
  /* everything the node stored is generated again, its inner checksums included */
  recompute_checksums(L, i, j);
  return 0;
}

/* ------------------------------------------------------------------------------------------ */
/* additional encoding of the vectors (feedforward Step 4, backpropagation Step 4)             */
/* ------------------------------------------------------------------------------------------ */

/* x~ = (G_c^T (x) I) x : Xt[b][j*b_c + c] for j < Nn; zero padding beyond n_in. */
void orc_encode_x(const orc_layer_t* L, const float* X, int B, float* Xt) {
  const int n = L->d.n, bc = L->b_c;
  for (int b = 0; b < B; ++b)
    for (int j = 0; j < L->Nn; ++j)
      for (int c = 0; c < bc; ++c) {
        double acc = 0.0;
        for (int q = 0; q < n; ++q) {
          int gc = q * bc + c;
          double xv = gc < L->d.n_in ? (double)X[(size_t)b * L->d.n_in + gc] : 0.0;
          acc += g_col(L, q, j) * xv;
        }
        Xt[(size_t)b * L->Nn * bc + j * bc + c] = (float)acc;
      }
}

/* delta~^T = delta^T (G_r (x) I) : Dt[b][i*b_r + r] for i < M; zero padding beyond n_out. */
void orc_encode_delta(const orc_layer_t* L, const float* Delta, int B, float* Dt) {
  const int m = L->d.m, br = L->b_r;
  for (int b = 0; b < B; ++b)
    for (int i = 0; i < L->M; ++i)
      for (int r = 0; r < br; ++r) {
        double acc = 0.0;
        for (int a = 0; a < m; ++a) {
          int gr = a * br + r;
          double dv = gr < L->d.n_out ? (double)Delta[(size_t)b * L->d.n_out + gr] : 0.0;
          acc += g_row(L, a, i) * dv;
        }
        Dt[(size_t)b * L->M * br + i * br + r] = (float)acc;
      }
}

/* ------------------------------------------------------------------------------------------ */
/* node products: step O1 on nodes (i < M, j < n), step O2 on nodes (i < m, j < Nn)            */
/* ------------------------------------------------------------------------------------------ */

void orc_forward_products(const orc_layer_t* L, const float* X, int B, float* Y) {
  const int br = L->b_r, bc = L->b_c, M = L->M, n = L->d.n;
  float* Xt = (float*)malloc((size_t)B * L->Nn * bc * sizeof(float));
  orc_encode_x(L, X, B, Xt);
#pragma omp parallel for collapse(2) schedule(dynamic)
  for (int j = 0; j < n; ++j)
    for (int i = 0; i < M; ++i) {
      const float* w = L->blk[i * L->Nn + j];
      float* y = Y + ((size_t)(j * M + i) * br) * B;
      for (int r = 0; r < br; ++r)
        for (int b = 0; b < B; ++b) {
          const float* x = Xt + (size_t)b * L->Nn * bc + j * bc;
          double acc = 0.0;
          for (int c = 0; c < bc; ++c) acc += (double)w[(size_t)r * bc + c] * (double)x[c];
          y[(size_t)r * B + b] = (float)acc;
        }
    }
  free(Xt);
}

void orc_backward_products(const orc_layer_t* L, const float* Delta, int B, float* Z) {
  const int br = L->b_r, bc = L->b_c, Nn = L->Nn, m = L->d.m;
  float* Dt = (float*)malloc((size_t)B * L->M * br * sizeof(float));
  orc_encode_delta(L, Delta, B, Dt);
#pragma omp parallel for collapse(2) schedule(dynamic)
  for (int i = 0; i < m; ++i)
    for (int j = 0; j < Nn; ++j) {
      const float* w = L->blk[i * Nn + j];
      float* z = Z + ((size_t)(i * Nn + j) * bc) * B;
      double* acc = (double*)calloc((size_t)bc * B, sizeof(double));
      for (int r = 0; r < br; ++r)
        for (int b = 0; b < B; ++b) {
          double dv = (double)Dt[(size_t)b * L->M * br + i * br + r];
          for (int c = 0; c < bc; ++c) acc[(size_t)c * B + b] += (double)w[(size_t)r * bc + c] * dv;
        }
      for (size_t e = 0; e < (size_t)bc * B; ++e) z[e] = (float)acc[e];
      free(acc);
    }
  free(Dt);
}

/* ------------------------------------------------------------------------------------------ */
/* soft-error injection into node outputs                                                     */
/* ------------------------------------------------------------------------------------------ */

static void phase_geometry(const orc_layer_t* L, int phase, int* n_cw, int* K, int* kd, int* r,
                           int* len, const double** P) {
  if (phase == ORC_PHASE_FWD) {
    *n_cw = L->d.n; *K = L->M; *kd = L->d.m; *r = L->d.r_row; *len = L->b_r; *P = L->P_row;
  } else {
    *n_cw = L->d.m; *K = L->Nn; *kd = L->d.n; *r = L->d.r_col; *len = L->b_c; *P = L->P_col;
  }
}

void orc_inject(const orc_layer_t* L, int phase, const orc_fault_t* f, uint32_t iteration,
                float* Y, int B, uint64_t injected[64]) {
  int n_cw, K, kd, r, len; const double* P;
  phase_geometry(L, phase, &n_cw, &K, &kd, &r, &len, &P);
  for (int c = 0; c < 64; ++c) injected[c] = 0;
  if (!f || f->mode == ORC_FAULT_NONE) return;
  const uint32_t n_active = (uint32_t)(n_cw * K);
  for (int cw = 0; cw < n_cw; ++cw)
    for (int k = 0; k < K; ++k) {
      int i = phase == ORC_PHASE_FWD ? k : cw;
      int j = phase == ORC_PHASE_FWD ? cw : k;
      uint32_t node_id = (uint32_t)(i * L->Nn + j);
      uint32_t active_index = phase == ORC_PHASE_FWD ? (uint32_t)(i * L->d.n + j) : (uint32_t)(i * L->Nn + j);
      if (!orc_node_hit(f, (uint32_t)phase, iteration, node_id, active_index, n_active)) continue;
      injected[cw] |= (uint64_t)1 << k;
      float* y = Y + ((size_t)(cw * K + k) * len) * B;
      for (uint32_t e = 0; e < (uint32_t)(len * B); ++e)
        y[e] = y[e] + orc_noise(f->seed, f->layer, (uint32_t)phase, iteration, node_id, e, f->sigma);
    }
}

/* ------------------------------------------------------------------------------------------ */
/* detection, location, erasure decoding ("General Error-Detection Method", "Decoding          */
/* Algorithm")                                                                                */
/* ------------------------------------------------------------------------------------------ */

/* Inverse of a small s x s matrix by Gaussian elimination with partial pivoting.  Returns 0 if
 * a pivot vanishes. */
static int invert_small(int s, const double* A, double* inv) {
  double a[8 * 16];
  if (s > 8) return 0;
  for (int r = 0; r < s; ++r)
    for (int c = 0; c < s; ++c) {
      a[r * 2 * s + c] = A[r * s + c];
      a[r * 2 * s + s + c] = r == c ? 1.0 : 0.0;
    }
  for (int p = 0; p < s; ++p) {
    int best = p;
    for (int r = p + 1; r < s; ++r)
      if (fabs(a[r * 2 * s + p]) > fabs(a[best * 2 * s + p])) best = r;
    if (a[best * 2 * s + p] == 0.0) return 0;
    if (best != p)
      for (int c = 0; c < 2 * s; ++c) {
        double t = a[p * 2 * s + c]; a[p * 2 * s + c] = a[best * 2 * s + c]; a[best * 2 * s + c] = t;
      }
    double piv = a[p * 2 * s + p];
    for (int c = 0; c < 2 * s; ++c) a[p * 2 * s + c] /= piv;
    for (int r = 0; r < s; ++r) {
      if (r == p) continue;
      double fct = a[r * 2 * s + p];
      if (fct == 0.0) continue;
      for (int c = 0; c < 2 * s; ++c) a[r * 2 * s + c] -= fct * a[p * 2 * s + c];
    }
  }
  for (int r = 0; r < s; ++r)
    for (int c = 0; c < s; ++c) inv[r * s + c] = a[r * 2 * s + s + c];
  return 1;
}

/* Conditioning of the erasure decoding of one direction's code (Section "Some Notations": any a of the b columns
 * of the generator are independent; "Decoding Algorithm": located outputs are solved from the remaining ones).
 * Every erasure sub-system is a square matrix A = P[F, Q]^T, F a set of s data indices, Q a set of s parity
 * indices, 1 <= s <= r.  out[0] = worst ||A||_inf ||A^-1||_inf, out[1] = worst ||A^-1||_inf, out[2] = worst
 * amplification of node-output errors into a decoded output,
 *   max_a sum_b |A^-1[a, b]| (1 + sum_{k not in F} |P[k, Q_b]|);
 * a singular sub-system gives infinity. */
static void conditioning_rec(const double* P, int kd, int r, int s, int* F, int nF, int startF, double* out) {
  if (nF < s) {
    for (int k = startF; k < kd; ++k) { F[nF] = k; conditioning_rec(P, kd, r, s, F, nF + 1, k + 1, out); }
    return;
  }
  /* every choice of s parities: bit masks with s bits */
  for (unsigned mask = 0; mask < (1u << r); ++mask) {
    int Q[8], nQ = 0;
    for (int q = 0; q < r; ++q) if ((mask >> q) & 1u) Q[nQ++] = q;
    if (nQ != s) continue;
    double A[64], Ai[64];
    for (int a = 0; a < s; ++a)
      for (int b = 0; b < s; ++b) A[a * s + b] = P[F[b] * r + Q[a]];
    if (!invert_small(s, A, Ai)) { out[0] = out[1] = out[2] = INFINITY; continue; }
    double nA = 0.0, nAi = 0.0, amp = 0.0;
    for (int a = 0; a < s; ++a) {
      double ra = 0.0, ri = 0.0, am = 0.0;
      for (int b = 0; b < s; ++b) {
        ra += fabs(A[a * s + b]);
        ri += fabs(Ai[a * s + b]);
        double w = 1.0;
        for (int k = 0; k < kd; ++k) {
          int inF = 0;
          for (int f = 0; f < s; ++f) if (F[f] == k) inF = 1;
          if (!inF) w += fabs(P[k * r + Q[b]]);
        }
        am += fabs(Ai[a * s + b]) * w;
      }
      if (ra > nA) nA = ra;
      if (ri > nAi) nAi = ri;
      if (am > amp) amp = am;
    }
    if (nA * nAi > out[0]) out[0] = nA * nAi;
    if (nAi > out[1]) out[1] = nAi;
    if (amp > out[2]) out[2] = amp;
  }
}

void orc_code_conditioning(const orc_layer_t* L, int phase, double out[3]) {
  int n_cw, K, kd, r, len; const double* P;
  phase_geometry(L, phase, &n_cw, &K, &kd, &r, &len, &P);
  out[0] = out[1] = out[2] = 0.0;
  int F[8];
  for (int s = 1; s <= r && s <= kd && s <= 8; ++s) conditioning_rec(P, kd, r, s, F, 0, 0, out);
}

/* Column k of the parity-check matrix H = [P^T | -I]  (r entries). */
static void h_column(const double* P, int kd, int r, int k, double* col) {
  for (int q = 0; q < r; ++q) col[q] = k < kd ? P[k * r + q] : (k - kd == q ? -1.0 : 0.0);
}

/* Syndrome-only location: smallest support (lexicographic order within a size) whose least-
 * squares fit leaves a residual below tau.  syn: r x n_el doubles.  Returns the support mask.
 * Largest size tried: r/2, the paper's t ("Decoding Algorithm": at most t non-zero blocks), or, with
 * `joint`, r - 1: the errors are whole sub-vectors (many elements, one support), every element's
 * syndrome lies in span(H_F) of the one true support F, and since any r columns of H are independent no
 * other support of up to r - 1 columns contains that span -- so the smallest support that fits every
 * element is F itself whenever |F| <= r - 1 and the error vectors are in general position.  (At most
 * three nodes: four parities is the most a layer takes.) */
static uint64_t syndrome_locate(const double* P, int kd, int r, int K, const double* syn,
                                size_t n_el, double tau, int joint) {
  int t = joint ? r - 1 : r / 2;
  const int cap = joint ? 3 : 2;
  if (t > cap) t = cap;
  double proj[8 * 8];
  for (int size = 1; size <= t && size <= K; ++size) {
    int idx[3] = {0, 1, 2};
    for (;;) {
      /* projector onto the orthogonal complement of span(H_F) */
      double HF[8 * 3], G[9], Ginv[9];
      for (int a = 0; a < size; ++a) {
        double col[8];
        h_column(P, kd, r, idx[a], col);
        for (int q = 0; q < r; ++q) HF[q * size + a] = col[q];
      }
      for (int a = 0; a < size; ++a)
        for (int b = 0; b < size; ++b) {
          double acc = 0.0;
          for (int q = 0; q < r; ++q) acc += HF[q * size + a] * HF[q * size + b];
          G[a * size + b] = acc;
        }
      if (invert_small(size, G, Ginv)) {
        for (int p = 0; p < r; ++p)
          for (int q = 0; q < r; ++q) {
            double acc = p == q ? 1.0 : 0.0;
            for (int a = 0; a < size; ++a)
              for (int b = 0; b < size; ++b) acc -= HF[p * size + a] * Ginv[a * size + b] * HF[q * size + b];
            proj[p * r + q] = acc;
          }
        double worst = 0.0;
        for (size_t e = 0; e < n_el; ++e)
          for (int p = 0; p < r; ++p) {
            double acc = 0.0;
            for (int q = 0; q < r; ++q) acc += proj[p * r + q] * syn[(size_t)q * n_el + e];
            if (fabs(acc) > worst) worst = fabs(acc);
          }
        if (worst <= tau) {
          uint64_t mask = 0;
          for (int a = 0; a < size; ++a) mask |= (uint64_t)1 << idx[a];
          return mask;
        }
      }
      /* next support in lexicographic order */
      if (size == 1) {
        if (++idx[0] >= K) break;
      } else if (size == 2) {
        if (++idx[1] >= K) {
          if (++idx[0] >= K - 1) break;
          idx[1] = idx[0] + 1;
        }
      } else {
        if (++idx[2] >= K) {
          if (++idx[1] >= K - 1) {
            if (++idx[0] >= K - 2) break;
            idx[1] = idx[0] + 1;
          }
          idx[2] = idx[1] + 1;
        }
      }
    }
  }
  return 0;
}

static int popcount64(uint64_t x) { int c = 0; while (x) { x &= x - 1; ++c; } return c; }

void orc_detect_decode(const orc_layer_t* L, int phase, float* Y, const float* V, int B,
                       const float* Yclean, const uint64_t* injected, orc_report_t* rep) {
  int n_cw, K, kd, r, len; const double* P;
  phase_geometry(L, phase, &n_cw, &K, &kd, &r, &len, &P);
  const size_t n_el = (size_t)len * B;
  const double tau_rel = (double)L->d.tau_rel, tau_abs = (double)L->d.tau_abs;
  /* rounding floor of the inner check: a sum of n outputs carries an error proportional to the
   * sum of their magnitudes, which the checksum-side scale misses when a checksum cancels */
  const double tau_floor = tau_rel / 512.0;
  memset(rep, 0, sizeof(*rep));
  rep->min_margin_hit = FLT_MAX;
  rep->max_margin_clean = 0.0f;
  if (injected) for (int c = 0; c < n_cw; ++c) rep->injected_mask[c] = injected[c];

  /* zero-padded copy of the vector the inner check needs */
  const int vlen = phase == ORC_PHASE_FWD ? L->n_in_p : L->n_out_p;
  const int vsrc = phase == ORC_PHASE_FWD ? L->d.n_in : L->d.n_out;
  double* Vp = (double*)calloc((size_t)B * vlen, sizeof(double));
  if (V)
    for (int b = 0; b < B; ++b)
      for (int c = 0; c < vsrc; ++c) Vp[(size_t)b * vlen + c] = (double)V[(size_t)b * vsrc + c];

  double* syn = (double*)malloc((size_t)(r > 0 ? r : 1) * n_el * sizeof(double));
  float* work = (float*)malloc((size_t)K * n_el * sizeof(float));
  double h = 0.0;
  for (int q = 0; q < r; ++q) {
    double acc = 1.0;
    for (int k = 0; k < kd; ++k) acc += fabs(P[k * r + q]);
    if (acc > h) h = acc;
  }

  for (int cw = 0; cw < n_cw; ++cw) {
    float* out = Y + (size_t)cw * K * n_el;
    const uint64_t inj = injected ? injected[cw] : 0;

    /* scale of the codeword: the (r+1)-th largest node norm, so that up to r corrupted
     * outputs cannot inflate the thresholds */
    double norms[64];
    for (int k = 0; k < K; ++k) {
      double mx = 0.0;
      for (size_t e = 0; e < n_el; ++e) { double a = fabs((double)out[(size_t)k * n_el + e]); if (a > mx) mx = a; }
      norms[k] = mx;
    }
    double sorted[64];
    memcpy(sorted, norms, sizeof(double) * K);
    for (int a = 0; a < K; ++a)
      for (int b = a + 1; b < K; ++b)
        if (sorted[b] > sorted[a]) { double t = sorted[a]; sorted[a] = sorted[b]; sorted[b] = t; }
    const double scale = sorted[r < K ? r : K - 1];
    const double tau_syn = tau_rel * h * scale + tau_abs;

    /* inner-checksum node check (Claim 1's encoding applied once more inside each block) */
    uint64_t flags = 0;
    if (L->d.locate_mode == ORC_LOCATE_NODECHECK && V) {
      for (int k = 0; k < K; ++k) {
        int i = phase == ORC_PHASE_FWD ? k : cw;
        int j = phase == ORC_PHASE_FWD ? cw : k;
        const float* o = out + (size_t)k * n_el;
        double worst = 0.0;
        if (phase == ORC_PHASE_FWD) {
          const float* u = L->u[i * L->Nn + j];
          for (int s = 0; s < L->ns; ++s)
            for (int b = 0; b < B; ++b) {
              double sum_y = 0.0, sum_abs = 0.0, ux = 0.0, uxabs = 0.0;
              for (int rr = s * L->T; rr < (s + 1) * L->T; ++rr) {
                sum_y += (double)o[(size_t)rr * B + b];
                sum_abs += fabs((double)o[(size_t)rr * B + b]);
              }
              for (int c = 0; c < L->b_c; ++c) {
                double uv = (double)u[s * L->b_c + c], xv = Vp[(size_t)b * vlen + j * L->b_c + c];
                ux += uv * xv;
                uxabs += fabs(uv) * fabs(xv);
              }
              double ratio = fabs(sum_y - ux) / (tau_rel * uxabs + tau_floor * sum_abs + tau_abs);
              if (ratio > worst) worst = ratio;
            }
        } else {
          const float* v = L->v[i * L->Nn + j];
          for (int s = 0; s < L->nsc; ++s)
            for (int b = 0; b < B; ++b) {
              double sum_z = 0.0, sum_abs = 0.0, vd = 0.0, vdabs = 0.0;
              for (int c = s * L->Tc; c < (s + 1) * L->Tc; ++c) {
                sum_z += (double)o[(size_t)c * B + b];
                sum_abs += fabs((double)o[(size_t)c * B + b]);
              }
              for (int rr = 0; rr < L->b_r; ++rr) {
                double vv = (double)v[s * L->b_r + rr], dv = Vp[(size_t)b * vlen + i * L->b_r + rr];
                vd += vv * dv;
                vdabs += fabs(vv) * fabs(dv);
              }
              double ratio = fabs(sum_z - vd) / (tau_rel * vdabs + tau_floor * sum_abs + tau_abs);
              if (ratio > worst) worst = ratio;
            }
        }
        if (worst > 1.0) flags |= (uint64_t)1 << k;
        if ((inj >> k) & 1) { if ((float)worst < rep->min_margin_hit) rep->min_margin_hit = (float)worst; }
        else if ((float)worst > rep->max_margin_clean) rep->max_margin_clean = (float)worst;
      }
    }

    /* syndrome  (H (x) I) out,  H = [P^T | -I] */
    double smax = 0.0;
    for (int q = 0; q < r; ++q)
      for (size_t e = 0; e < n_el; ++e) {
        double acc = -(double)out[(size_t)(kd + q) * n_el + e];
        for (int k = 0; k < kd; ++k) acc += P[k * r + q] * (double)out[(size_t)k * n_el + e];
        syn[(size_t)q * n_el + e] = acc;
        if (fabs(acc) > smax) smax = fabs(acc);
      }
    if (r > 0) {
      /* a hit codeword is detected by its node flags or by its syndrome, so the syndrome is the
       * margin of a hit only where no node check runs */
      float ratio = (float)(smax / tau_syn);
      if (inj) { if (L->d.locate_mode != ORC_LOCATE_NODECHECK && ratio < rep->min_margin_hit) rep->min_margin_hit = ratio; }
      else if (ratio > rep->max_margin_clean) rep->max_margin_clean = ratio;
    }
    const int detected = (r > 0 && smax > tau_syn) || flags != 0;
    /* Verification step of the error detection (Section "Decentralized Implementation", "Errors in Error-Detection
     * under Error Model 2"): the evaluation of the codeword's parity checks is made twice and compared.  A soft error
     * in one evaluation shifts its value by a noise sample; any difference means the nodes disagree, and the caller
     * has to restore the last checkpoint (the codeword is left as it is). */
    const uint32_t vunit = (uint32_t)(phase * 64 + cw);
    if (L->have_small && orc_small_hit(&L->small, ORC_PHASE_CHECK, L->small_iteration, vunit)) {
      const float shift = orc_noise(L->small.seed, L->small.layer, ORC_PHASE_CHECK, L->small_iteration, vunit, 0u, L->small.sigma);
      if (shift != 0.0f) {
        if (rep->status < ORC_DISAGREE) rep->status = ORC_DISAGREE;
        continue;
      }
    }
    if (!detected) continue;
    rep->detected_mask |= (uint64_t)1 << cw;
    rep->n_detected_cw++;

    uint64_t F = flags;
    int ok = 1;
    if (F == 0) {
      if (L->d.locate_mode != ORC_LOCATE_NONE && r >= 2)
        F = syndrome_locate(P, kd, r, K, syn, n_el, tau_syn, L->d.locate_mode == ORC_LOCATE_JOINT);
      if (F == 0) ok = 0;
    }
    rep->flagged_mask[cw] = F;
    rep->n_flagged_nodes += (uint32_t)popcount64(F);
    /* Verification step of the decoding ("Errors in decoding under Error Model 2"): the list of nodes found
     * erroneous is made twice and compared.  A soft error in one evaluation changes the membership of one node
     * (chosen by the generator); the lists then differ and the decoding is deemed erroneous. */
    if (L->have_small && orc_small_hit(&L->small, ORC_PHASE_DECODE, L->small_iteration, vunit)) {
      uint32_t key[2] = {L->small.seed, (L->small.layer << 8) | ORC_PHASE_DECODE};
      uint32_t c[4] = {L->small_iteration, vunit, 1u, 0u}, o[4];
      orc_philox4x32_10(c, key, o);
      const uint64_t F_other = F ^ ((uint64_t)1 << (o[0] % (uint32_t)K));
      if (F_other != F) {
        if (rep->status < ORC_DISAGREE) rep->status = ORC_DISAGREE;
        continue;
      }
    }
    if (ok && popcount64(F) > r) ok = 0;

    if (ok) {
      /* erasure decoding: flagged data outputs from the lowest-indexed unflagged parities */
      int Fd[8], nFd = 0, Q[8], nQ = 0;
      for (int k = 0; k < kd; ++k) if ((F >> k) & 1) Fd[nFd++] = k;
      for (int q = 0; q < r && nQ < nFd; ++q) if (!((F >> (kd + q)) & 1)) Q[nQ++] = q;
      if (nQ < nFd) ok = 0;
      double A[64], Ainv[64];
      if (ok && nFd > 0) {
        for (int a = 0; a < nFd; ++a)
          for (int b = 0; b < nFd; ++b) A[a * nFd + b] = P[Fd[b] * r + Q[a]];
        if (!invert_small(nFd, A, Ainv)) ok = 0;
      }
      if (ok) {
        memcpy(work, out, (size_t)K * n_el * sizeof(float));
        for (size_t e = 0; e < n_el && nFd > 0; ++e) {
          double rhs[8];
          for (int a = 0; a < nFd; ++a) {
            double acc = (double)out[(size_t)(kd + Q[a]) * n_el + e];
            for (int k = 0; k < kd; ++k)
              if (!((F >> k) & 1)) acc -= P[k * r + Q[a]] * (double)out[(size_t)k * n_el + e];
            rhs[a] = acc;
          }
          for (int a = 0; a < nFd; ++a) {
            double acc = 0.0;
            for (int b = 0; b < nFd; ++b) acc += Ainv[a * nFd + b] * rhs[b];
            work[(size_t)Fd[a] * n_el + e] = (float)acc;
          }
        }
        /* flagged parity outputs are discarded and re-encoded from the data outputs */
        for (int q = 0; q < r; ++q) {
          if (!((F >> (kd + q)) & 1)) continue;
          for (size_t e = 0; e < n_el; ++e) {
            double acc = 0.0;
            for (int k = 0; k < kd; ++k) acc += P[k * r + q] * (double)work[(size_t)k * n_el + e];
            work[(size_t)(kd + q) * n_el + e] = (float)acc;
          }
        }
        /* remaining unflagged, unused parities must agree with the corrected codeword */
        for (int q = 0; q < r && ok; ++q) {
          if ((F >> (kd + q)) & 1) continue;
          int used = 0;
          for (int a = 0; a < nQ; ++a) if (Q[a] == q) used = 1;
          if (used) continue;
          for (size_t e = 0; e < n_el; ++e) {
            double acc = -(double)work[(size_t)(kd + q) * n_el + e];
            for (int k = 0; k < kd; ++k) acc += P[k * r + q] * (double)work[(size_t)k * n_el + e];
            if (fabs(acc) > tau_syn) { ok = 0; break; }
          }
        }
      }
      if (ok) {
        memcpy(out, work, (size_t)K * n_el * sizeof(float));
        if (rep->status < ORC_CORRECTED) rep->status = ORC_CORRECTED;
      }
    }
    if (!ok) {
      /* uncorrectable: the paper restores a checkpoint; here the transient fault is undone by
       * taking the fault-free recomputation of this codeword's node outputs */
      rep->n_fallback_cw++;
      if (Yclean) {
        memcpy(out, Yclean + (size_t)cw * K * n_el, (size_t)K * n_el * sizeof(float));
        if (rep->status < ORC_FALLBACK) rep->status = ORC_FALLBACK;
      } else {
        if (rep->status < ORC_FAILED) rep->status = ORC_FAILED;
      }
    }
  }
  free(work); free(syn); free(Vp);
}

/* ------------------------------------------------------------------------------------------ */
/* per-layer calls                                                                            */
/* ------------------------------------------------------------------------------------------ */

void orc_forward(orc_layer_t* L, const float* X, int B, const orc_fault_t* f,
                 uint32_t iteration, float* S, orc_report_t* rep) {
  const int M = L->M, n = L->d.n, br = L->b_r;
  const size_t total = (size_t)n * M * br * B;
  float* Y = (float*)malloc(total * sizeof(float));
  float* Yc = (float*)malloc(total * sizeof(float));
  uint64_t inj[64];
  L->small_iteration = iteration;
  orc_forward_products(L, X, B, Y);
  memcpy(Yc, Y, total * sizeof(float));
  orc_inject(L, ORC_PHASE_FWD, f, iteration, Y, B, inj);
  if (L->have_small && L->small.p_input_q32) {
    /* a node whose own copy of x_j is off by a noise vector nu produces W~_ij (x_j + nu): its output is off by
     * W~_ij nu, like any other erroneous output (and it counts among the injected nodes) */
    const orc_small_faults_t* sf = &L->small;
    const int bc = L->b_c;
    double* nu = (double*)malloc((size_t)bc * B * sizeof(double));
    for (int j = 0; j < n; ++j)
      for (int i = 0; i < M; ++i) {
        const uint32_t node = (uint32_t)(i * L->Nn + j);
        if (!orc_small_hit(sf, ORC_PHASE_INPUT, iteration, node)) continue;
        inj[j] |= (uint64_t)1 << i;
        for (int e = 0; e < bc * B; ++e) nu[e] = (double)orc_noise(sf->seed, sf->layer, ORC_PHASE_INPUT, iteration, node, (uint32_t)e, sf->sigma);
        const float* w = L->blk[i * L->Nn + j];
        float* y = Y + ((size_t)(j * M + i) * br) * B;
        for (int r = 0; r < br; ++r)
          for (int b = 0; b < B; ++b) {
            double acc = 0.0;
            for (int c = 0; c < bc; ++c) acc += (double)w[(size_t)r * bc + c] * nu[(size_t)c * B + b];
            y[(size_t)r * B + b] = (float)((double)y[(size_t)r * B + b] + acc);
          }
      }
    free(nu);
  }
  orc_detect_decode(L, ORC_PHASE_FWD, Y, X, B, Yc, inj, rep);
  /* s_i = sum_j y_ij (the row All-Reduce of the decentralised algorithm) */
  for (int b = 0; b < B; ++b)
    for (int i = 0; i < L->d.m; ++i)
      for (int r = 0; r < br; ++r) {
        int g = i * br + r;
        if (g >= L->d.n_out) continue;
        double acc = 0.0;
        for (int j = 0; j < n; ++j) acc += (double)Y[((size_t)(j * M + i) * br + r) * B + b];
        S[(size_t)b * L->d.n_out + g] = (float)acc;
      }
  free(Y); free(Yc);
}

/* Coded rank-B update (step O3, the three update rules): every stored block adds
 * lr * delta~_i x~_j^T; the inner checksums follow the same rule so they stay valid. */
static void update_impl(orc_layer_t* L, const float* Delta, const float* X, int B, float lr, int small, uint32_t iteration);
void orc_update(orc_layer_t* L, const float* Delta, const float* X, int B, float lr) {
  update_impl(L, Delta, X, B, lr, 0, 0u);
}

static void update_impl(orc_layer_t* L, const float* Delta, const float* X, int B, float lr, int small, uint32_t iteration) {
  const int br = L->b_r, bc = L->b_c, M = L->M, Nn = L->Nn;
  float* Xt = (float*)malloc((size_t)B * Nn * bc * sizeof(float));
  float* Dt = (float*)malloc((size_t)B * M * br * sizeof(float));
  orc_encode_x(L, X, B, Xt);
  orc_encode_delta(L, Delta, B, Dt);
  if (small && L->have_small) {
    /* soft errors in the additional encoding: the whole encoded sub-vector of a hit parity index is off; the
     * update (blocks and inner checksums alike) takes the erroneous vector, so the stored parity blocks of that
     * block-column / block-row leave the code and the next products on them show it */
    const orc_small_faults_t* sf = &L->small;
    for (int j = L->d.n; j < Nn; ++j)
      if (orc_small_hit(sf, ORC_PHASE_ENCODE, iteration, (uint32_t)j))
        for (int c = 0; c < bc; ++c)
          for (int b = 0; b < B; ++b)
            Xt[(size_t)b * Nn * bc + j * bc + c] += orc_noise(sf->seed, sf->layer, ORC_PHASE_ENCODE, iteration, (uint32_t)j,
                                                            (uint32_t)(c * B + b), sf->sigma);
    for (int i = L->d.m; i < M; ++i)
      if (orc_small_hit(sf, ORC_PHASE_ENCODE, iteration, (uint32_t)(Nn + i)))
        for (int r = 0; r < br; ++r)
          for (int b = 0; b < B; ++b)
            Dt[(size_t)b * M * br + i * br + r] += orc_noise(sf->seed, sf->layer, ORC_PHASE_ENCODE, iteration, (uint32_t)(Nn + i),
                                                           (uint32_t)(r * B + b), sf->sigma);
  }
  const double eta = (double)lr;
#pragma omp parallel for collapse(2) schedule(dynamic)
  for (int i = 0; i < M; ++i)
    for (int j = 0; j < Nn; ++j) {
      if (!has_node(L, i, j)) continue;
      float* w = L->blk[i * Nn + j];
      float* u = L->u[i * Nn + j];
      float* v = L->v[i * Nn + j];
      for (int r = 0; r < br; ++r)
        for (int c = 0; c < bc; ++c) {
          double acc = 0.0;
          for (int b = 0; b < B; ++b)
            acc += (double)Dt[(size_t)b * M * br + i * br + r] * (double)Xt[(size_t)b * Nn * bc + j * bc + c];
          w[(size_t)r * bc + c] = store_w(L, (double)w[(size_t)r * bc + c] + eta * acc);
        }
      for (int s = 0; s < L->ns; ++s)
        for (int c = 0; c < bc; ++c) {
          double acc = 0.0;
          for (int b = 0; b < B; ++b) {
            double dsum = 0.0;
            for (int r = s * L->T; r < (s + 1) * L->T; ++r) dsum += (double)Dt[(size_t)b * M * br + i * br + r];
            acc += dsum * (double)Xt[(size_t)b * Nn * bc + j * bc + c];
          }
          u[s * bc + c] = (float)((double)u[s * bc + c] + eta * acc);
        }
      for (int s = 0; s < L->nsc; ++s)
        for (int r = 0; r < br; ++r) {
          double acc = 0.0;
          for (int b = 0; b < B; ++b) {
            double xsum = 0.0;
            for (int c = s * L->Tc; c < (s + 1) * L->Tc; ++c) xsum += (double)Xt[(size_t)b * Nn * bc + j * bc + c];
            acc += (double)Dt[(size_t)b * M * br + i * br + r] * xsum;
          }
          v[s * br + r] = (float)((double)v[s * br + r] + eta * acc);
        }
    }
  free(Xt); free(Dt);
}

void orc_backward_update(orc_layer_t* L, const float* Delta, const float* X, int B, float lr,
                         const orc_fault_t* f, uint32_t iteration, float* C, orc_report_t* rep) {
  const int Nn = L->Nn, m = L->d.m, bc = L->b_c;
  const size_t total = (size_t)m * Nn * bc * B;
  float* Z = (float*)malloc(total * sizeof(float));
  float* Zc = (float*)malloc(total * sizeof(float));
  uint64_t inj[64];
  L->small_iteration = iteration;
  orc_backward_products(L, Delta, B, Z); /* uses the weights of this iteration, before O3 */
  memcpy(Zc, Z, total * sizeof(float));
  orc_inject(L, ORC_PHASE_BWD, f, iteration, Z, B, inj);
  orc_detect_decode(L, ORC_PHASE_BWD, Z, Delta, B, Zc, inj, rep);
  /* c_j = sum_i z_ij (the column All-Reduce) */
  for (int b = 0; b < B; ++b)
    for (int j = 0; j < L->d.n; ++j)
      for (int c = 0; c < bc; ++c) {
        int g = j * bc + c;
        if (g >= L->d.n_in) continue;
        double acc = 0.0;
        for (int i = 0; i < m; ++i) acc += (double)Z[((size_t)(i * Nn + j) * bc + c) * B + b];
        C[(size_t)b * L->d.n_in + g] = (float)acc;
      }
  free(Z); free(Zc);
  update_impl(L, Delta, X, B, lr, 1, iteration);
}

void orc_decode_weights(const orc_layer_t* L, float* W_out) {
  for (int gr = 0; gr < L->d.n_out; ++gr)
    for (int gc = 0; gc < L->d.n_in; ++gc) {
      int i = gr / L->b_r, r = gr % L->b_r, j = gc / L->b_c, c = gc % L->b_c;
      W_out[(size_t)gr * L->d.n_in + gc] = L->blk[i * L->Nn + j][(size_t)r * L->b_c + c];
    }
}

/* Largest relative deviation of a stored parity block (and of the inner checksums) from the
 * re-encoding of the stored data blocks: zero up to rounding while the coded structure holds. */
double orc_check_invariance(const orc_layer_t* L) {
  const int br = L->b_r, bc = L->b_c, m = L->d.m, n = L->d.n;
  double worst = 0.0;
  for (int i = 0; i < L->M; ++i)
    for (int j = 0; j < L->Nn; ++j) {
      if (!has_node(L, i, j)) continue;
      const float* w = L->blk[i * L->Nn + j];
      if (i >= m || j >= n) {
        double dev = 0.0, ref = 0.0;
        for (int r = 0; r < br; ++r)
          for (int c = 0; c < bc; ++c) {
            double acc = 0.0;
            for (int a = 0; a < m; ++a)
              for (int b = 0; b < n; ++b) {
                double g = g_row(L, a, i) * g_col(L, b, j);
                if (g != 0.0) acc += g * (double)L->blk[a * L->Nn + b][(size_t)r * bc + c];
              }
            double d = fabs(acc - (double)w[(size_t)r * bc + c]);
            if (d > dev) dev = d;
            if (fabs(acc) > ref) ref = fabs(acc);
          }
        if (ref > 0.0 && dev / ref > worst) worst = dev / ref;
      }
      const float* u = L->u[i * L->Nn + j];
      const float* v = L->v[i * L->Nn + j];
      double dev = 0.0, ref = 0.0;
      for (int s = 0; s < L->ns; ++s)
        for (int c = 0; c < bc; ++c) {
          double acc = 0.0;
          for (int r = s * L->T; r < (s + 1) * L->T; ++r) acc += (double)w[(size_t)r * bc + c];
          double d = fabs(acc - (double)u[s * bc + c]);
          if (d > dev) dev = d;
          if (fabs(acc) > ref) ref = fabs(acc);
        }
      if (ref > 0.0 && dev / ref > worst) worst = dev / ref;
      dev = 0.0; ref = 0.0;
      for (int s = 0; s < L->nsc; ++s)
        for (int r = 0; r < br; ++r) {
          double acc = 0.0;
          for (int c = s * L->Tc; c < (s + 1) * L->Tc; ++c) acc += (double)w[(size_t)r * bc + c];
          double d = fabs(acc - (double)v[s * br + r]);
          if (d > dev) dev = d;
          if (fabs(acc) > ref) ref = fabs(acc);
        }
      if (ref > 0.0 && dev / ref > worst) worst = dev / ref;
    }
  return worst;
}

/* ------------------------------------------------------------------------------------------ */
/* whole-network step: feedforward (O1, C1) for l = 1..L, loss, backpropagation (O2, C2) and   */
/* update (O3) for l = L..1  (Algorithm 1 without the collectives)                             */
/* ------------------------------------------------------------------------------------------ */

struct orc_net {
  int L, activation, loss;
  orc_layer_t** layers;
};

orc_net_t* orc_net_create(orc_layer_t** layers, int L, int activation, int loss) {
  if (L < 1) return NULL;
  for (int l = 1; l < L; ++l)
    if (layers[l]->d.n_in != layers[l - 1]->d.n_out) return NULL;
  orc_net_t* net = (orc_net_t*)calloc(1, sizeof(*net));
  net->L = L; net->activation = activation; net->loss = loss;
  net->layers = (orc_layer_t**)malloc(sizeof(orc_layer_t*) * L);
  memcpy(net->layers, layers, sizeof(orc_layer_t*) * L);
  return net;
}
void orc_net_free(orc_net_t* net) { if (net) { free(net->layers); free(net); } }

void orc_step(orc_net_t* net, const float* X, const void* target, int B, float lr,
              const orc_fault_t* faults, uint32_t iteration, orc_report_t* reports,
              float* loss, float* out_last) {
  const int L = net->L;
  float** xs = (float**)calloc((size_t)L + 1, sizeof(float*));
  xs[0] = (float*)malloc((size_t)B * net->layers[0]->d.n_in * sizeof(float));
  memcpy(xs[0], X, (size_t)B * net->layers[0]->d.n_in * sizeof(float));
  float* S = NULL;
  for (int l = 0; l < L; ++l) {
    orc_layer_t* Ly = net->layers[l];
    const size_t cnt = (size_t)B * Ly->d.n_out;
    S = (float*)malloc(cnt * sizeof(float));
    orc_forward(Ly, xs[l], B, faults ? &faults[l] : NULL, iteration, S, &reports[2 * l]);
    if (l < L - 1) {
      /* step C1: x^{l+1} = f(s^l) */
      for (size_t e = 0; e < cnt; ++e)
        if (net->activation == ORC_ACT_RELU && S[e] < 0.0f) S[e] = 0.0f;
      xs[l + 1] = S;
    }
  }
  /* loss and the error vector of the last layer, delta^L = -d loss / d s^L */
  const int nL = net->layers[L - 1]->d.n_out;
  float* delta = (float*)malloc((size_t)B * nL * sizeof(float));
  double total = 0.0;
  if (net->loss == ORC_LOSS_MSE_MEAN) {
    const float* y = (const float*)target;
    const double scale = 1.0 / ((double)nL * B);
    for (size_t e = 0; e < (size_t)B * nL; ++e) {
      double d = (double)y[e] - (double)S[e];
      total += d * d * scale;
      delta[e] = (float)(2.0 * d * scale);
    }
  } else {
    const int32_t* lab = (const int32_t*)target;
    for (int b = 0; b < B; ++b) {
      double mx = -DBL_MAX, den = 0.0;
      for (int k = 0; k < nL; ++k) if ((double)S[(size_t)b * nL + k] > mx) mx = (double)S[(size_t)b * nL + k];
      for (int k = 0; k < nL; ++k) den += exp((double)S[(size_t)b * nL + k] - mx);
      for (int k = 0; k < nL; ++k) {
        double p = exp((double)S[(size_t)b * nL + k] - mx) / den;
        delta[(size_t)b * nL + k] = (float)(((k == lab[b] ? 1.0 : 0.0) - p) / B);
        if (k == lab[b]) total += -log(p) / B;
      }
    }
  }
  if (loss) *loss = (float)total;
  if (out_last) memcpy(out_last, S, (size_t)B * nL * sizeof(float));
  free(S);
  for (int l = L - 1; l >= 0; --l) {
    orc_layer_t* Ly = net->layers[l];
    float* C = (float*)malloc((size_t)B * Ly->d.n_in * sizeof(float));
    orc_backward_update(Ly, delta, xs[l], B, lr, faults ? &faults[l] : NULL, iteration, C, &reports[2 * l + 1]);
    /* step C2: delta^{l-1} = c^l (.) g(x^l), with g(f(u)) = f'(u) */
    if (l > 0)
      for (size_t e = 0; e < (size_t)B * Ly->d.n_in; ++e)
        if (net->activation == ORC_ACT_RELU && !(xs[l][e] > 0.0f)) C[e] = 0.0f;
    free(delta);
    delta = C;
  }
  free(delta);
  for (int l = 0; l < L; ++l) free(xs[l]);
  free(xs);
}
