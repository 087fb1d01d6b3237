/*
 * libcodenet -- CodeNet's per-layer coded training step on one NVIDIA B200 (sm_100a).
 *
 * Method: Dutta, Bai, Low, Grover, "CodeNet: Training Large Scale Neural Networks in Presence
 * of Soft-Errors".  Each fully-connected layer's weight matrix W (N_out x N_in) is stored once
 * as a grid of coded blocks W~ = (G_r^T (x) I) W (G_c (x) I)  (Claim 1), one block per "node"
 * of the paper's (m + r_row) x (n + r_col) node grid, corner blocks absent.  The feedforward
 * product (step O1) runs on the (m + r_row) x n active blocks, the backpropagation product
 * (step O2) on the m x (n + r_col) active blocks, the rank-B update (step O3) on every stored
 * block with the encoded vectors, so W~ is never re-encoded.  Block outputs are checked with
 * the parity-check matrix H = [P^T | -I], erroneous outputs are located and erasure-decoded.
 *
 * Conventions for every entry point
 *  - Pointers named *_dev are DEVICE pointers on the current CUDA device; everything else is
 *    host memory.  Matrices are row-major.  Batched vectors are (B, length) row-major.
 *  - `stream` is a cudaStream_t passed as void*.  Calls enqueue work on it and return without
 *    synchronising, except codenet_encode_layer / codenet_net_create / the free functions,
 *    which allocate or release device memory and may synchronise.
 *  - Return value 0 = enqueued; negative = error (codenet_strerror).  A soft-error outcome is
 *    not an API error: it is written to the device-side report.
 *  - The caller owns inputs, outputs and reports and keeps them alive until the stream has
 *    passed the call.  The library owns the coded weights, inner checksums and workspace of a
 *    layer; calls on the same layer must be ordered on one stream (they share workspace).
 *  - There is no CPU fallback: without a CUDA device every compute entry point fails with
 *    CODENET_E_CUDA.
 */
#ifndef CODENET_H
#define CODENET_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct codenet_layer codenet_layer_t; /* opaque: coded weights + workspace of one layer */
typedef struct codenet_net codenet_net_t;     /* opaque: L layers + activation / loss           */
typedef void* codenet_stream_t;               /* a cudaStream_t                                 */

enum { CODENET_F32 = 0, CODENET_BF16 = 1 };                       /* storage of W~              */
enum { CODENET_MATH_FFMA = 0, CODENET_MATH_TF32 = 1, CODENET_MATH_BF16 = 2 };
enum { CODENET_LOCATE_NONE = 0, CODENET_LOCATE_SYNDROME = 1, CODENET_LOCATE_NODECHECK = 2,
       CODENET_LOCATE_OFF = 3, CODENET_LOCATE_JOINT = 4 };
enum { CODENET_FAULT_NONE = 0, CODENET_FAULT_BERNOULLI = 1, CODENET_FAULT_EXACTLY_ONE = 2 };
enum { CODENET_PHASE_FWD = 0, CODENET_PHASE_BWD = 1 };
enum { CODENET_CLEAN = 0, CODENET_CORRECTED = 1, CODENET_FALLBACK = 2, CODENET_FAILED = 3,
       CODENET_TIMEOUT = 4,
       CODENET_DISAGREE = 5 /* a verification step found two evaluations that differ: restore the last checkpoint */ };
enum { CODENET_PHASE_ENCODE = 2, CODENET_PHASE_INPUT = 3, CODENET_PHASE_CHECK = 4, CODENET_PHASE_DECODE = 5 };
enum { CODENET_ACT_IDENTITY = 0, CODENET_ACT_RELU = 1 };
enum { CODENET_LOSS_MSE_MEAN = 0, CODENET_LOSS_SOFTMAX_CE = 1 };

enum {
  CODENET_OK = 0,
  CODENET_E_BADARG = -1, /* NULL pointer, unknown enum value, batch out of range            */
  CODENET_E_SHAPE = -2,  /* grid / block sizes the library cannot lay out                    */
  CODENET_E_CUDA = -3,   /* a CUDA call failed (no device, launch error)                     */
  CODENET_E_NOMEM = -4,  /* device allocation failed                                         */
  CODENET_E_TOOBIG = -5  /* problem larger than the fixed scratch of codenet_matvec_noalloc  */
};

#define CODENET_MAX_NODES 64  /* nodes per codeword and codewords per phase                    */
#define CODENET_MAX_PARITY 4  /* r_row, r_col                                                  */

/* Layer description (paper notation, Section "Some Notations"). */
typedef struct {
  int32_t n_out, n_in;     /* N_l, N_{l-1}.  Padded internally to multiples of m and n.      */
  int32_t m, n;            /* data grid: W is split into m x n blocks                        */
  int32_t r_row, r_col;    /* parity block-rows / block-columns, 0..CODENET_MAX_PARITY        */
  int32_t dtype;           /* CODENET_F32 | CODENET_BF16: storage type of the coded blocks    */
  int32_t math;            /* CODENET_MATH_*: arithmetic of the products for batch >= 64;     */
                           /* smaller batches always use fp32 FFMA                            */
  int32_t batch_max;       /* largest B any later call will pass (sizes the workspace)        */
  int32_t locate_mode;     /* NONE: detect only; SYNDROME: locate from the parity checks      */
                           /* alone (needs r >= 2); NODECHECK: locate with the inner          */
                           /* checksums, fall back to SYNDROME when nothing is flagged;       */
                           /* OFF: no check at all (timing baseline for the cost of the       */
                           /* redundant blocks alone; injected errors pass through; the inner */
                           /* checksums are not maintained, and neither are they in a layer    */
                           /* without parity blocks that runs no node check);                  */
                           /* JOINT: as SYNDROME ("Decoding Algorithm", Appendix B: the       */
                           /* block-sparsest e with (H x I) e = syndrome), but supports of up */
                           /* to r - 1 nodes (at most 3) instead of t = r / 2: the errors are  */
                           /* whole sub-vectors, so the smallest support that fits every       */
                           /* element is the true one while it has at most r - 1 nodes and     */
                           /* the error vectors are in general position                       */
  int32_t check_rows;      /* T: rows per inner-checksum slice (forward check), divides        */
                           /* N_out/m; 0 = N_out/m                                            */
  int32_t check_cols;      /* Tc: columns per inner-checksum slice (backward check), divides   */
                           /* N_in/n; 0 = N_in/n                                              */
  const float* P_row;      /* host, m x r_row row-major: parity part of G_r = [I | P_row];    */
                           /* NULL = all ones.  Copied at encode time.                        */
  const float* P_col;      /* host, n x r_col row-major; NULL = all ones                      */
  float tau_rel, tau_abs;  /* decision thresholds: a statistic s counts as non-zero when      */
                           /* s > tau_rel * scale + tau_abs                                   */
} codenet_layer_desc_t;

/* Soft-error injection plan (Error Model 2 on the outputs of steps O1 / O2).  A node (i, j) is
 * hit in (iteration, layer, phase) when word 0 of Philox4x32-10(counter = (iteration,
 * i*(n+r_col)+j, 0, 0), key = (seed, layer<<8 | phase)) < p_q32 (BERNOULLI), or when it is the
 * one victim drawn for that phase (EXACTLY_ONE).  Every element e of a hit node's output gets
 * sigma * (sum of twelve 16-bit uniforms - 393210) / 65536 added (counters (.., e, 1), (.., e, 2)). */
typedef struct {
  uint32_t seed;
  uint32_t layer;
  uint32_t mode;                  /* CODENET_FAULT_*                                         */
  uint32_t p_q32;                 /* floor(p * 2^32)                                         */
  float sigma;                    /* noise standard deviation                                */
  const uint32_t* iteration_dev;  /* DEVICE counter read by the kernels (lets a captured     */
                                  /* CUDA graph be replayed); NULL = iteration 0             */
} codenet_fault_t;

/* Soft errors in the steps around the products (Section "Decentralized Implementation": under Error Model 2 the
 * additional encoding, the generation of a node's input sub-vector by the activation / post-multiplication step,
 * the error detection and the decoding can err as well).  Unit u of small-step phase ph is hit in an iteration when
 * word 0 of Philox4x32-10(counter = (iteration, u, 0, 0), key = (seed, layer << 8 | ph)) is below that phase's
 * p_q32; noise values are drawn like those of codenet_fault_t with the same key.
 *   CODENET_PHASE_ENCODE  drawn in the backward call: unit j for x~_j (j >= n), unit (n + r_col) + i for delta~_i
 *                         (i >= m).  The whole encoded sub-vector is off by noise; the update (blocks and inner
 *                         checksums alike) takes it as it is, so the stored parity blocks of that block-column /
 *                         block-row leave the code and the next products on them show it.
 *   CODENET_PHASE_INPUT   feedforward products: unit = node i * (n + r_col) + j.  The node's own copy of x_j is off
 *                         by a noise vector nu, so its output is off by W~_ij nu; it counts among the injected nodes
 *                         of the report.
 *   CODENET_PHASE_CHECK   unit = phase of the call * 64 + codeword: one of the two evaluations of the codeword's
 *                         parity checks is off by a noise value ("Errors in Error-Detection under Error Model 2").
 *   CODENET_PHASE_DECODE  same units, detected codewords only: one of the two lists of nodes found erroneous has
 *                         the membership of one node changed ("Errors in decoding under Error Model 2").
 * The two verification steps compare the evaluations; a difference makes the report's status CODENET_DISAGREE and
 * leaves the codeword as it is: the caller restores the last checkpoint (codenet_checkpoint_restore). */
typedef struct {
  uint32_t seed;
  uint32_t layer;
  uint32_t p_encode_q32, p_input_q32, p_check_q32, p_decode_q32;   /* floor(p * 2^32) per phase; 0 = never */
  float sigma;
  const uint32_t* iteration_dev;  /* DEVICE counter as in codenet_fault_t; NULL = iteration 0 */
} codenet_small_faults_t;

/* Written on the device by each call that checks outputs. */
typedef struct {
  uint32_t status;                /* worst outcome over codewords: CODENET_CLEAN ..          */
  uint32_t n_detected_cw;         /* codewords whose checks fired                            */
  uint32_t n_flagged_nodes;       /* nodes located as erroneous                              */
  uint32_t n_fallback_cw;         /* codewords that could not be corrected                   */
  uint64_t detected_mask;         /* bit c = codeword c detected                             */
  uint64_t flagged_mask[CODENET_MAX_NODES];  /* per codeword: bit k = node k located         */
  uint64_t injected_mask[CODENET_MAX_NODES]; /* per codeword: nodes the injection plan hit    */
  float min_margin_hit;           /* min over hit nodes/codewords of statistic / threshold   */
  float max_margin_clean;         /* max over clean nodes/codewords of statistic / threshold */
} codenet_report_t;

/* Initial encoding (Claim 1; Section "Pre-processing: Initial Encoding of weight matrices").
 * W_dev: n_out x n_in row-major, float (CODENET_F32) or bfloat16 (CODENET_BF16); read only
 * during this call.  Builds the coded block grid, the inner checksums and the workspace for
 * batches up to batch_max; *out receives the handle (release with codenet_free_layer).
 * Errors: BADARG (NULL, bad enum, batch_max < 1), SHAPE (m + r_row or n + r_col above
 * CODENET_MAX_NODES, parities above CODENET_MAX_PARITY, check_rows / check_cols not dividing
 * the block height / width), NOMEM, CUDA. */
int codenet_encode_layer(const codenet_layer_desc_t* desc, const void* W_dev,
                         codenet_stream_t stream, codenet_layer_t** out);

/* Feedforward stage of one layer (step O1 with its checks; Algorithm 1, feedforward loop):
 * node products W~_ij x_j on the (m + r_row) x n active blocks, soft-error injection per
 * `fault` (NULL = none), detection / location / erasure decoding of each block-column's
 * codeword, then s_i = sum_j y_ij.  X_dev: (B, n_in).  S_dev: (B, n_out) receives W x.
 * rep_dev (may be NULL) receives the report.  Errors: BADARG (B < 1 or > batch_max). */
int codenet_forward(codenet_layer_t* layer, const float* X_dev, int B, const codenet_fault_t* fault,
                    float* S_dev, codenet_report_t* rep_dev, codenet_stream_t stream);

/* Backpropagation product and update of one layer (steps O2 and O3; Algorithm 1, backpropagation
 * loop and update stage): node products delta_i^T W~_ij on the m x (n + r_col) active blocks
 * from the weights as they are before this call, injection, checks and decoding of each
 * block-row's codeword, c_j = sum_i z_ij, and the coded rank-B update
 * W~_ij += lr * delta~_i x~_j^T on every stored block (the three update rules), with the inner
 * checksums updated alongside.  Delta_dev: (B, n_out) holds -d loss / d s (already divided by
 * the batch size where the loss is a batch mean).  X_dev: (B, n_in), the layer's input of this
 * iteration.  C_dev: (B, n_in) receives W^T delta.  Errors: BADARG. */
int codenet_backward_update(codenet_layer_t* layer, const float* Delta_dev, const float* X_dev,
                            int B, float lr, const codenet_fault_t* fault, float* C_dev,
                            codenet_report_t* rep_dev, codenet_stream_t stream);

/* As codenet_backward_update, and in the same sweep over the coded blocks also takes the feedforward
 * node products of the NEXT iteration, W~_new x_next, from the values just updated (the update needs
 * no communication and the next step O1 reads exactly these blocks, so the two sweeps can be one).
 * X_next_dev: (B, n_in), the layer's input of the next iteration, already known (first layer of a
 * network, or a single layer), 16-byte aligned; NULL = plain codenet_backward_update.  The next
 * codenet_forward on this layer that is given the same pointer and B (contents unchanged) then skips its
 * own sweep; any other call discards the stored products.  Ignored (plain behaviour) for B > 8 and for
 * layouts whose column strips do not tile the block-columns (N_in/n not a multiple of 512 floats /
 * 1024 bfloat16). */
int codenet_backward_update_next(codenet_layer_t* layer, const float* Delta_dev, const float* X_dev,
                                 int B, float lr, const codenet_fault_t* fault, float* C_dev,
                                 codenet_report_t* rep_dev, const float* X_next_dev,
                                 codenet_stream_t stream);

/* As codenet_backward_update_next followed by codenet_forward(layer, X_next_dev, B, fault_next, S_next_dev,
 * rep_next_dev): the backpropagation product, checks and update of this iteration (Algorithm 1,
 * backpropagation loop and update stage) and the whole feedforward stage of the next one (Algorithm 1,
 * feedforward loop) on the blocks just updated.  The two checks decide on independent codewords (block-rows of
 * this iteration's products, block-columns of the next one's), so for batch 1 with the node check and at most
 * one parity per code they share one launch; otherwise the two calls are made one after the other: the results
 * are the same either way.  The forward stage belongs to the NEXT iteration: its fault plan's device counter is
 * read plus one (the counter is advanced only after this call), so fault_next may point at the same plan as
 * `fault`.  S_next_dev: (B, n_out) receives W_new x_next; rep_next_dev (may be NULL) its report.
 * Errors: BADARG (also X_next_dev or S_next_dev NULL). */
int codenet_backward_update_forward_next(codenet_layer_t* layer, const float* Delta_dev, const float* X_dev,
                                         int B, float lr, const codenet_fault_t* fault, float* C_dev,
                                         codenet_report_t* rep_dev, const float* X_next_dev,
                                         const codenet_fault_t* fault_next, float* S_next_dev,
                                         codenet_report_t* rep_next_dev, codenet_stream_t stream);

/* Fault in the stored weights, as in the paper's own experiment (Section "Experimental Results": a
 * sparse matrix is added to the sub-matrix a node stores).  Element e = row * (N_in/n) + col of coded
 * block (i, j) changes when word 0 of Philox4x32-10(counter = (iteration, i * (n + r_col) + j, e, 3),
 * key = (seed, fault_layer << 8 | 2)) is below density_q32 (= density * 2^32); the value added is
 * amplitude * u, u uniform on [-1, 1) from the upper 24 bits of word 1.  The inner checksums are left
 * as they are, so the next feedforward / backpropagation products locate the node (its outputs are
 * still corrected from the code) until the block is regenerated.  Errors: BADARG (no such block). */
int codenet_corrupt_block(codenet_layer_t* layer, int i, int j, uint32_t seed, uint32_t fault_layer,
                          uint32_t iteration, uint32_t density_q32, float amplitude, codenet_stream_t stream);

/* Regeneration of a stored block (feedforward stage, the "regenerate" step; Section "Update stage
 * on a single layer", last paragraph): block (i, j) is rebuilt from the other blocks of its
 * block-column (along = 0: the m + r_row blocks of a block-column j < n are a codeword of G_r,
 * element by element) or of its block-row (along = 1: the n + r_col blocks of a block-row i < m are a
 * codeword of G_c).  A parity block is re-encoded from the data blocks; a data block is solved from
 * the lowest-indexed parity block whose generator entry for it is not zero.  Sums in double, one
 * rounding to the storage type.  The blocks it reads must be intact.  Errors: BADARG (no such
 * block, along not 0 / 1), SHAPE (that direction holds no parity for the block: r_row = 0, r_col = 0,
 * a parity block-column asked along = 0, a parity block-row asked along = 1, or every generator entry
 * zero). */
int codenet_regenerate_block(codenet_layer_t* layer, int i, int j, int along, codenet_stream_t stream);

/* Checkpoint and roll-back of a layer's stored state (Section "Decentralized Implementation": when the
 * nodes disagree, or a pattern cannot be decoded, the weight matrices are restored from the last
 * checkpoint; Theorem 2, assumptions (ii) and (iv): a checkpoint every I_0 iterations at a cost
 * tau_cpt, a restore at a cost tau_b).  save copies the coded blocks and the inner checksums, as stored,
 * into device memory the layer owns (allocated by the first call: as many bytes again as the layer's
 * blocks and checksums; freed by codenet_free_layer); restore copies them back and drops feedforward
 * products taken ahead of time.  Both are asynchronous on `stream`.  The codes, thresholds and
 * workspaces are not part of a checkpoint.  Errors: BADARG (NULL layer; restore before any save),
 * NOMEM (save could not allocate), CUDA. */
int codenet_checkpoint_save(codenet_layer_t* layer, codenet_stream_t stream);
int codenet_checkpoint_restore(codenet_layer_t* layer, codenet_stream_t stream);

/* Plan for soft errors in the small steps of every later call on this layer (copied; NULL switches them off).  A plan
 * with p_input_q32 > 0 makes the layer allocate one more buffer of the size of its node outputs; this call may
 * therefore allocate and synchronise.  Errors: BADARG, NOMEM. */
int codenet_layer_set_small_faults(codenet_layer_t* layer, const codenet_small_faults_t* plan);

/* Stand-alone detection / location / erasure decoding ("General Error-Detection Method" and
 * "Decoding Algorithm", Appendix B) of un-reduced node outputs the caller supplies.
 * Y_dev: [codeword][node][len][B] floats -- forward: codeword = block-column j < n, node =
 * block-row i < m + r_row, len = N_out/m; backward: codeword = block-row i < m, node =
 * block-column j < n + r_col, len = N_in/n.  Corrected in place.  V_dev: the vector the inner
 * check needs, X (B, n_in) for CODENET_PHASE_FWD or Delta (B, n_out) for CODENET_PHASE_BWD.
 * No fault-free copy exists here, so an uncorrectable codeword is left as it is and reported
 * as CODENET_FAILED.  Errors: BADARG. */
int codenet_detect_decode(const codenet_layer_t* layer, int phase, float* Y_dev, const float* V_dev,
                          int B, codenet_report_t* rep_dev, codenet_stream_t stream);

/* A network of L coded layers (n_in of layer l+1 = n_out of layer l) for codenet_step.
 * `activation` is applied after every layer but the last (step C1), `loss` to the last
 * layer's output.  The layers stay owned by the caller and must outlive the net. */
int codenet_net_create(codenet_layer_t** layers, int L, int activation, int loss,
                       codenet_net_t** out);

/* One training iteration (Algorithm 1 without the collectives): feedforward l = 1..L with
 * x^{l+1} = f(s^l), loss and delta^L, then for l = L..1 codenet_backward_update followed by
 * delta^{l-1} = c^l (.) g(x^l)  (step C2).  X_dev: (B, n_in of layer 1).  target_dev: float
 * (B, n_L) for CODENET_LOSS_MSE_MEAN (mean over outputs and batch), int32 labels (B) for
 * CODENET_LOSS_SOFTMAX_CE (mean over the batch).  per_layer: host array of L fault plans or
 * NULL.  reps_dev: device array of 2L reports (2l = forward, 2l+1 = backward of layer l) or
 * NULL.  loss_dev: one float or NULL.  Errors: BADARG. */
int codenet_step(codenet_net_t* net, const float* X_dev, const void* target_dev, int B, float lr,
                 const codenet_fault_t* per_layer, codenet_report_t* reps_dev, float* loss_dev,
                 codenet_stream_t stream);

/* Announce the input of the NEXT codenet_step (device pointer, (B, n_in of layer 1)); the coming step
 * then uses codenet_backward_update_next on layer 1 (codenet_backward_update_forward_next where that
 * call shares a launch: the next step, given the announced pointer, then finds layer 1's forward stage done;
 * its sums and report appear where this interface says when that step ends).  One-shot: cleared by that step. */
int codenet_net_set_next_input(codenet_net_t* net, const float* X_next_dev);

/* Switch the use of announced next inputs on (the default) or off.  Off: codenet_net_set_next_input and the
 * successor inputs a recording knows are ignored, every step sweeps the weights for its own forward products (three
 * passes over the first layer's weights per iteration instead of two).  Results are the same either way.
 * Errors: BADARG. */
int codenet_net_set_lookahead(codenet_net_t* net, int on);

/* Give the network an iteration counter of its own (a device word, e.g. the one the fault plans read): every
 * codenet_step from now on ends by adding one to it, in its last kernel where that kernel can (so a step the caller
 * captures into a graph of their own draws a new fault pattern at every replay, like the recorded steps below).
 * NULL switches it off.  Errors: BADARG. */
int codenet_net_set_iteration_counter(codenet_net_t* net, uint32_t* counter_dev);

/* Record one codenet_step (same arguments; X_next_dev as in codenet_net_set_next_input, or NULL) into a
 * CUDA graph instead of running it, and keep the instantiated graph in the network; *graph_id names it.
 * Nothing is computed by this call.  `stream` must be a created stream, not the default stream
 * (CODENET_E_BADARG).  Run at least one plain codenet_step first (it sizes the launches).
 * Every pointer is baked into the graph: feed later steps by writing into the same buffers.  A recorded
 * step ends by adding 1 to every iteration counter its fault plans point to.  With X_next_dev the skipping of layer 1's product
 * sweep is decided while recording, from the network's state as if the recorded step had run: record
 * the graphs in the order they will be replayed (for two alternating input buffers: record the step that
 * follows the last plain step first, then the other one, then replay them alternately).
 * codenet_net_replay enqueues one recorded step. */
int codenet_net_capture_step(codenet_net_t* net, const float* X_dev, const void* target_dev, int B, float lr,
                             const codenet_fault_t* per_layer, codenet_report_t* reps_dev, float* loss_dev,
                             const float* X_next_dev, codenet_stream_t stream, int* graph_id);

/* Record n_steps consecutive codenet_step calls into ONE graph (a replay then runs them back to back, without
 * the pause between two graph launches): step s takes X_devs[s] and target_devs[s] (host arrays of device
 * pointers), announces X_devs[s + 1] as the next input (X_next_dev after the last step, or NULL), writes its
 * reports at reps_dev + s * reps_stride (in reports; 0: every step writes the same 2L reports) and its loss at
 * loss_dev + s * loss_stride.  Everything else as codenet_net_capture_step.  Errors: BADARG. */
int codenet_net_capture_steps(codenet_net_t* net, int n_steps, const float* const* X_devs,
                              const void* const* target_devs, int B, float lr,
                              const codenet_fault_t* per_layer, codenet_report_t* reps_dev, int reps_stride,
                              float* loss_dev, int loss_stride, const float* X_next_dev,
                              codenet_stream_t stream, int* graph_id);
int codenet_net_replay(codenet_net_t* net, int graph_id, codenet_stream_t stream);

/* Copy the last layer's pre-loss output of the most recent codenet_step into out_dev (B, n_L). */
int codenet_net_output(const codenet_net_t* net, float* out_dev, int B, codenet_stream_t stream);

/* Extract the m x n data blocks as a plain n_out x n_in matrix of the layer's dtype. */
int codenet_decode_weights(const codenet_layer_t* layer, void* W_dev_out, codenet_stream_t stream);

/* Largest relative deviation of a stored parity block or inner checksum from the re-encoding of
 * the stored data blocks (zero up to rounding while the update keeps the coded structure,
 * Section "Update stage on a single layer").  max_rel_dev: one float. */
int codenet_check_invariance(const codenet_layer_t* layer, float* max_rel_dev, codenet_stream_t stream);

/* Conditioning of the erasure decoding of one direction's code (Section "Some Notations": any a of the b columns of
 * a systematic MDS generator are independent; "Decoding Algorithm", Appendix B: located outputs are solved from the
 * others).  phase = CODENET_PHASE_FWD looks at G_r = [I | P_row], CODENET_PHASE_BWD at G_c.  Over every square
 * sub-system A = P[F, Q]^T of s <= r located data outputs F and s parities Q: out[0] = the worst
 * ||A||_inf ||A^-1||_inf, out[1] = the worst ||A^-1||_inf, out[2] = the worst factor by which errors of the node
 * outputs can grow in a decoded output, max_a sum_b |A^-1[a,b]| (1 + sum_{k not in F} |P[k, Q_b]|).  `out` is host
 * memory; nothing runs on the device.  A code without parity gives zeros; a singular sub-system gives infinity:
 * such a generator is not MDS (two all-ones parities, a zero entry), the patterns that need the singular system are
 * reported as uncorrectable when they occur, and a caller that wants every pattern of r located outputs decoded
 * draws another generator.  Errors: BADARG. */
int codenet_code_conditioning(const codenet_layer_t* layer, int phase, double out[3]);

/* Copy one stored coded block (i, j) out as b_r x b_c floats (diagnostics / tests).
 * Errors: BADARG when the grid has no node at (i, j). */
int codenet_get_block(const codenet_layer_t* layer, int i, int j, float* out_dev, codenet_stream_t stream);

/* Copy the inner checksums of block (i, j) out: u_out_dev gets (row slices) x b_c floats (column
 * sums of each slice of T rows), v_out_dev gets (column slices) x b_r floats (row sums of each
 * slice of Tc columns); either may be NULL. */
int codenet_get_checksums(const codenet_layer_t* layer, int i, int j, float* u_out_dev,
                          float* v_out_dev, codenet_stream_t stream);

/* dims[0..9] = b_r, b_c, m + r_row, n + r_col, T, row slices, padded n_out, padded n_in, Tc,
 * column slices */
int codenet_layer_dims(const codenet_layer_t* layer, int32_t dims[10]);

/* s = W x without any allocation (the paper has no counterpart; this exists for callers that cannot
 * allocate device memory when they call: latency-critical loops, where cudaMalloc's implicit
 * device synchronisation is not acceptable; processes in which a memory pool or another framework
 * has already claimed the whole device; code run under a no-allocation-after-start-up policy).  W_dev: rows x cols row-major fp32, 16-byte aligned, seen as n_blocks uncoded
 * block-columns (cols divisible by n_blocks, cols / n_blocks a multiple of 4, n_blocks <= 64); x_dev:
 * cols floats, 16-byte aligned; s_dev: rows floats.  The per-block-column products y_j = W_j x_j
 * (step O1 on an uncoded 1 x n_blocks grid) go to a scratch array of 2^20 floats (4 MiB) that is part
 * of the library image on every GPU until the process exits, then s = sum_j y_j.  Needs
 * rows * n_blocks <= 2^20, otherwise CODENET_E_TOOBIG and nothing is launched.  Calls cudaMalloc,
 * cudaFree or any allocating routine never.  The first call on each device looks up the array's device
 * address (cudaGetSymbolAddress) with that device current: make that first call outside any stream
 * capture.  All calls share the one array and it keeps the previous call's contents; each call
 * overwrites what it reads, so nothing needs clearing, but two calls that overlap on the GPU (different
 * streams) race on it.  Same result, bit for bit, as codenet_forward on a layer encoded with m = 1,
 * n = n_blocks, no parities and locate_mode OFF. */
int codenet_matvec_noalloc(const float* W_dev, int rows, int cols, int n_blocks, const float* x_dev,
                           float* s_dev, codenet_stream_t stream);

/* Bounded waits.  Every wait inside a kernel (a pipeline barrier of the tensor-core kernels) gives up after a time
 * limit: the kernel then sets a flag of the layer, releases what it holds and returns, and every report written for
 * the layer from then on carries CODENET_TIMEOUT instead of the outcome of its checks (the products of that launch
 * are not valid) until codenet_reset_timeout acknowledges it.  The paper has no counterpart (its nodes are
 * processes; a stuck one is found by the verification steps of Section "Decentralized Implementation").
 *   codenet_set_wait_limit       the limit in nanoseconds for all later launches on this device (0: the default,
 *                                about one second).
 *   codenet_withhold_tile_loads  diagnostic: while on, the forward product kernel for batches >= 64 issues none of
 *                                its tile loads, so the waits that depend on them run out after the limit.  Nothing
 *                                faults and nothing is left in flight; it exists so that the give-up path can be
 *                                exercised.
 *   codenet_reset_timeout        clears the layer's flag.
 * All three are asynchronous on `stream` and ordered with the launches on it.  Errors: BADARG, CUDA. */
int codenet_set_wait_limit(uint64_t nanoseconds, codenet_stream_t stream);
int codenet_withhold_tile_loads(int on, codenet_stream_t stream);
int codenet_reset_timeout(codenet_layer_t* layer, codenet_stream_t stream);

/* Kernels launched by this library since it was loaded (all streams). */
uint64_t codenet_launch_count(void);

/* Per-kernel device timing for benchmarks.  While enabled, the streaming kernels are
 * bracketed by CUDA events on the stream they are launched on (at most 4096 launches each are
 * kept).  codenet_profile_read synchronises the device and returns the summed duration and the
 * number of launches of `kernel` (CODENET_KERNEL_*) since codenet_profile_enable(1). */
enum { CODENET_KERNEL_FORWARD = 0,          /* forward node products (FFMA or tensor-core tiles)      */
       CODENET_KERNEL_BACKWARD_UPDATE = 1,  /* fused backward products + update (batch <= 8)          */
       CODENET_KERNEL_BACKWARD = 2,         /* backward node products alone (batch > 8)               */
       CODENET_KERNEL_UPDATE = 3,           /* rank-B update alone (batch > 8)                        */
       CODENET_KERNEL_REGENERATE = 4,       /* a stored block rebuilt from its code                   */
       CODENET_KERNEL_COUNT = 5 };
int codenet_profile_enable(int on);
int codenet_profile_read(int kernel, float* total_ms, uint64_t* launches);

void codenet_free_layer(codenet_layer_t* layer);
void codenet_free_net(codenet_net_t* net);
const char* codenet_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* CODENET_H */
