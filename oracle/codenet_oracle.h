/*
 * CodeNet CPU oracle -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, obviously-correct CPU statement of the per-layer coded training step of
 * CodeNet (Dutta, Bai, Low, Grover).  It exists so that the CUDA library can be checked
 * against something written straight from the paper.  Only the test-suite, the smoke check
 * and the CPU-baseline leg of the benchmark may call it; the product never does.  It shares
 * no code, header, table or constant with the CUDA library.
 *
 * Arithmetic: every sum is accumulated in double; stored quantities (coded blocks, inner
 * checksums, vectors, node outputs) are rounded to their storage type (float, or bfloat16
 * emulated by round-to-nearest-even) at the point where a node would store them.
 *
 * Notation follows the paper (Section "Some Notations"): N_out = N_l, N_in = N_{l-1}, data
 * grid m x n, r_row parity block-rows, r_col parity block-columns, M = m + r_row,
 * Nn = n + r_col, block size b_r x b_c = N_out/m x N_in/n, generators G_r = [I_m | P_row],
 * G_c = [I_n | P_col], parity checks H = [P^T | -I].
 *
 * Parity status: values and the coding identities are pinned by the tests against the
 * paper's worked example and the plain products.  "parity unpinned" (fixed by this build's
 * reading, not by the paper): decision thresholds, tie-breaks in erasure decoding, the
 * inner-checksum node check, the fallback for uncorrectable codewords, loss scaling, padding.
 */
#ifndef CODENET_ORACLE_H
#define CODENET_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { ORC_LOCATE_NONE = 0, ORC_LOCATE_SYNDROME = 1, ORC_LOCATE_NODECHECK = 2,
       ORC_LOCATE_JOINT = 4 /* syndrome-only, supports of up to r - 1 nodes (vector errors); 3 is not used here */ };
enum { ORC_FAULT_NONE = 0, ORC_FAULT_BERNOULLI = 1, ORC_FAULT_EXACTLY_ONE = 2 };
enum { ORC_PHASE_FWD = 0, ORC_PHASE_BWD = 1 };
enum { ORC_CLEAN = 0, ORC_CORRECTED = 1, ORC_FALLBACK = 2, ORC_FAILED = 3,
       ORC_DISAGREE = 5 /* a verification step found two evaluations that differ: restore the last checkpoint */ };
enum { ORC_PHASE_ENCODE = 2, ORC_PHASE_INPUT = 3, ORC_PHASE_CHECK = 4, ORC_PHASE_DECODE = 5 };  /* small steps */
enum { ORC_ACT_IDENTITY = 0, ORC_ACT_RELU = 1 };
enum { ORC_LOSS_MSE_MEAN = 0, ORC_LOSS_SOFTMAX_CE = 1 };

typedef struct {
  int32_t n_out, n_in;      /* N_l, N_{l-1} (unpadded)                                   */
  int32_t m, n;             /* data grid                                                 */
  int32_t r_row, r_col;     /* parity block-rows / block-columns (0 = uncoded)           */
  int32_t store_bf16;       /* 0: coded blocks stored as float, 1: as bfloat16           */
  int32_t locate_mode;      /* ORC_LOCATE_*                                              */
  int32_t check_rows;       /* T, rows per inner-checksum slice (forward check); 0 = b_r  */
  int32_t check_cols;       /* Tc, columns per inner-checksum slice (backward check); 0 = b_c */
  float tau_rel, tau_abs;   /* decision thresholds                                       */
  const float* P_row;       /* m x r_row row-major, NULL = all ones                      */
  const float* P_col;       /* n x r_col row-major, NULL = all ones                      */
} orc_desc_t;

typedef struct {
  uint32_t seed, layer, mode, p_q32;
  float sigma;
} orc_fault_t;

/* Soft errors in the steps around the products (Error Model 2 in the additional encoding, in the generation of a
 * node's input sub-vector by the activation / post-multiplication step, in error detection and in decoding;
 * Section "Decentralized Implementation").  Unit u of phase ph is hit in an iteration when word 0 of
 * Philox(counter (iteration, u, 0, 0), key (seed, layer << 8 | ph)) is below the phase's p_q32; noise values come
 * from orc_noise with the same key.  Units: ENCODE: j for x~_j (j >= n), Nn + i for delta~_i (i >= m), drawn in the
 * backward call; INPUT: node i * Nn + j of the feedforward products (its own copy of x_j is off by a noise vector,
 * so its output is off by W~_ij times that vector); CHECK and DECODE: the codeword, per phase of the call. */
typedef struct {
  uint32_t seed, layer;
  uint32_t p_encode_q32, p_input_q32, p_check_q32, p_decode_q32;
  float sigma;
} orc_small_faults_t;

typedef struct {
  uint32_t status;
  uint32_t n_detected_cw, n_flagged_nodes, n_fallback_cw;
  uint64_t detected_mask;
  uint64_t flagged_mask[64];
  uint64_t injected_mask[64];
  float min_margin_hit, max_margin_clean;
} orc_report_t;

typedef struct orc_layer orc_layer_t;
typedef struct orc_net orc_net_t;

void orc_set_threads(int n);
int orc_get_threads(void);

/* Counter-based generator (Philox4x32, 10 rounds) and the derived noise sample. */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]);
float orc_noise(uint32_t seed, uint32_t layer, uint32_t phase, uint32_t iteration,
                uint32_t node_id, uint32_t element, float sigma);
int orc_node_hit(const orc_fault_t* f, uint32_t phase, uint32_t iteration, uint32_t node_id,
                 uint32_t active_index, uint32_t n_active);

/* Initial encoding (Claim 1).  W is n_out x n_in row-major float. */
orc_layer_t* orc_layer_create(const orc_desc_t* d, const float* W);
void orc_layer_free(orc_layer_t* L);
/* Checkpoint / roll-back of the stored state (coded blocks + inner checksums): 0, -1 = nothing saved, -2 = no memory */
int orc_checkpoint_save(orc_layer_t* L);
int orc_checkpoint_restore(orc_layer_t* L);
/* dims[0..9] = b_r, b_c, M, Nn, T, row slices, n_out_padded, n_in_padded, Tc, column slices */
void orc_layer_dims(const orc_layer_t* L, int32_t dims[10]);
int orc_get_block(const orc_layer_t* L, int i, int j, float* out /* b_r*b_c */);
int orc_get_u(const orc_layer_t* L, int i, int j, float* out /* n_slices*b_c */);
int orc_get_v(const orc_layer_t* L, int i, int j, float* out /* column slices * b_r */);
/* Overwrite one stored block (tests use this to model a corrupted stored sub-matrix). */
int orc_set_block(orc_layer_t* L, int i, int j, const float* in);

/* faults in the stored blocks (Section "Experimental Results") and regeneration of a block from
 * the code of its block-column (along = 0) or block-row (along = 1) (feedforward stage, the
 * "regenerate" step) */
long orc_corrupt_block(orc_layer_t* L, int i, int j, uint32_t seed, uint32_t layer, uint32_t iteration,
                       uint32_t density_q32, float amplitude);
int orc_regenerate_block(orc_layer_t* L, int i, int j, int along);

/* Additional encoding of vectors: Xt is (B, Nn*b_c), Dt is (B, M*b_r). */
void orc_encode_x(const orc_layer_t* L, const float* X, int B, float* Xt);
void orc_encode_delta(const orc_layer_t* L, const float* Delta, int B, float* Dt);

/* Un-reduced node outputs.  Y: [cw=j<n][node=i<M][row<b_r][B]; Z: [cw=i<m][node=j<Nn][col<b_c][B] */
void orc_forward_products(const orc_layer_t* L, const float* X, int B, float* Y);
void orc_backward_products(const orc_layer_t* L, const float* Delta, int B, float* Z);

/* Soft-error injection into node outputs (Error Model 2); fills injected[cw]. */
void orc_inject(const orc_layer_t* L, int phase, const orc_fault_t* f, uint32_t iteration,
                float* Y, int B, uint64_t injected[64]);

/* Detection, location, erasure decoding in place.  V = X (forward) or Delta (backward).
 * Yclean (may be NULL) supplies the fault-free outputs used when a codeword is uncorrectable. */
void orc_detect_decode(const orc_layer_t* L, int phase, float* Y, const float* V, int B,
                       const float* Yclean, const uint64_t* injected, orc_report_t* rep);

void orc_forward(orc_layer_t* L, const float* X, int B, const orc_fault_t* f,
                 uint32_t iteration, float* S, orc_report_t* rep);
void orc_update(orc_layer_t* L, const float* Delta, const float* X, int B, float lr);
void orc_backward_update(orc_layer_t* L, const float* Delta, const float* X, int B, float lr,
                         const orc_fault_t* f, uint32_t iteration, float* C, orc_report_t* rep);

void orc_decode_weights(const orc_layer_t* L, float* W_out /* n_out x n_in */);
/* Plan for soft errors in the small steps of every later call on this layer (copied; NULL: none). */
void orc_layer_set_small_faults(orc_layer_t* L, const orc_small_faults_t* plan);
/* Was unit `unit` of small-step phase `phase` hit in `iteration` under `plan`? */
int orc_small_hit(const orc_small_faults_t* plan, uint32_t phase, uint32_t iteration, uint32_t unit);
double orc_check_invariance(const orc_layer_t* L);
/* Conditioning of the erasure decoding of the code of one direction (phase 0: G_r, phase 1: G_c), over every square
 * sub-system of the parity part with at most r unknowns: out[0] worst ||A||_inf ||A^-1||_inf, out[1] worst
 * ||A^-1||_inf, out[2] worst amplification of node-output errors into a decoded output. */
void orc_code_conditioning(const orc_layer_t* L, int phase, double out[3]);

orc_net_t* orc_net_create(orc_layer_t** layers, int L, int activation, int loss);
void orc_net_free(orc_net_t* net);
/* target: float (B, n_L) for MSE, int32 labels (B) for softmax-CE.  faults: L entries or NULL.
 * reports: 2L entries (2l = forward of layer l, 2l+1 = backward of layer l).
 * out_last (may be NULL): (B, n_L) pre-loss output of the last layer. */
void orc_step(orc_net_t* net, const float* X, const void* target, int B, float lr,
              const orc_fault_t* faults, uint32_t iteration, orc_report_t* reports,
              float* loss, float* out_last);

#ifdef __cplusplus
}
#endif
#endif
