// Internal declarations shared by the translation units of libcodenet (CUDA, sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "../../include/codenet.h"

namespace codenet {

// Geometry and device pointers of one coded layer, passed by value to the kernels.
// Coded weights: one row-major matrix of (M*b_r) rows, row stride ld = Nn*ldb elements; block
// (i, j) occupies rows [i*b_r, (i+1)*b_r) and columns [j*ldb, j*ldb + b_c); columns b_c..ldb
// of every block are zero padding that keeps each block row 16-byte aligned.  The r_row x r_col
// corner (i >= m and j >= n) is allocated but never read or written.
struct Geom {
  int n_out, n_in, m, n, r_row, r_col;
  int M, Nn, b_r, b_c, ldb, ld, T, ns, Tc, nsc;
  int Mbr;  // M * b_r coded rows
  int dtype, locate_mode;
  float tau_rel, tau_abs;
  void* Wt;         // coded blocks, float or __nv_bfloat16
  float* U;         // inner checksum rows  [(i*Nn + j)*ns + s][ldb]
  float* V;         // inner checksum columns [(i*Nn + j)*nsc + s][b_r]
  const float* Pr;  // m x r_row
  const float* Pc;  // n x r_col
};

// Inner checksums are kept valid only where something can read them: not with the checks switched off, and not in
// a layer without any parity block that runs no node check.
__host__ __device__ inline bool keeps_checksums(const Geom& g) {
  return g.locate_mode != CODENET_LOCATE_OFF &&
         (g.r_row > 0 || g.r_col > 0 || g.locate_mode == CODENET_LOCATE_NODECHECK);
}

struct FaultDev {
  uint32_t seed, layer, mode, p_q32;
  float sigma;
  const uint32_t* iteration;
};

// Soft errors in the small steps (codenet_small_faults_t on the device side); on == 0: none.
struct SmallDev {
  uint32_t seed, layer, p_encode, p_input, p_check, p_decode;
  float sigma;
  const uint32_t* iteration;
  int on;
};

// Statistics gathered across CTAs by the check kernel (floats as ordered unsigned bit patterns,
// combined with atomicMax so the result does not depend on arrival order).
struct CheckStats {
  unsigned norm[CODENET_MAX_NODES * CODENET_MAX_NODES];   // [codeword][node] max |output|
  unsigned ratio[CODENET_MAX_NODES * CODENET_MAX_NODES];  // [codeword][node] inner-check statistic / threshold
  unsigned syn[CODENET_MAX_NODES];                        // [codeword] max |syndrome|
  unsigned resid[CODENET_MAX_NODES];                      // [codeword] max residual of the decoding plan
  unsigned need_fix;   // some codeword needs work (read by a fix kernel that follows)
  unsigned done_d;     // low half: codewords that have decided; high half: how many of them need work
};

// Per-codeword decision and erasure-decoding plan.
struct CwPlan {
  unsigned long long F, injected;  // located nodes; nodes the injection plan hit
  double ainv[CODENET_MAX_PARITY * CODENET_MAX_PARITY];
  int state;                       // 0 clean, 1 decode with this plan, 3 uncorrectable
  int detected, nfd;
  int fd[CODENET_MAX_PARITY], q[CODENET_MAX_PARITY];  // located data nodes; parities used to solve them
  unsigned spare;                  // parities left over to verify the result
  float tau, min_hit, max_clean;
};

// Workspace of a layer (device memory, sized for batch_max).
struct Workspace {
  float* Xt;      // (B, ld)    zero-padded x with the parity sub-vectors x~ appended per block
  float* Dt;      // (B, Mbr)   delta with the parity sub-vectors delta~
  float* dsum;    // [(i*ns + s)*B + b]  sum of delta~_i over the rows of slice s
  float* xsum;    // [(j*nsc + s)*B + b] sum of x~_j over the columns of slice s
  float* Y;       // clean un-reduced node outputs (forward) / z partials (backward)
  float* Yw;      // working copy [codeword][node][len][B]
  float* Yw2;     // the same for the forward part of a paired check (feedforward size), or NULL
  float* pair_sums;   // paired check: [unit][2] slice sums of the forward part between its phases, or NULL
  float* Ynext;   // feedforward partials of the next iteration [strip][coded row][b], or NULL
  void* tc_x;     // tensor-core operand copy of x: (B, n*ldb) in the multiplication type, or NULL
  void* tc_d;     // tensor-core operand copy of delta~: (B, M*b_r), or NULL
  void* tc_dT;    // transposed operand copies for the update: (M*b_r, B) and (ld, B), or NULL
  void* tc_xT;
  int* tc_flag;   // [0] set by a tensor-core kernel whose bounded wait ran out; [1] which statistics buffer the
                  // next check kernel works in (kept on the device, flipped by the kernel); [2] the same for the
                  // second pair of buffers, those of the forward part of a paired check
  float* chk;     // inner-check scratch for batches > 8 (check_scratch_floats), or NULL
  float* dY;      // output deviations W~_ij nu of nodes whose input copy is hit, [codeword][node][len][B], or NULL
  CheckStats* stats;  // two buffers used alternately; each check clears the other one (and two more for the
                      // forward part of a paired check)
  CwPlan* plan;       // one per codeword (and a second set for the forward part of a paired check)
  size_t y_elems, yw_elems;
};

}  // namespace codenet

// The opaque handle of the C interface.
struct codenet_layer {
  codenet_layer_desc_t desc;
  codenet::Geom g;
  codenet::Workspace ws;
  int batch_max;
  int bwd_rows;   // R: rows per tile of the fused backward+update kernel
  int bwd_rt;     // RT = ceil(b_r / R)
  int next_ok;               // the layout allows taking the next feedforward products in the update sweep
  const float* next_x;       // input those products were taken for (NULL: none pending)
  int next_B;
  int pair_ok;               // the buffers of the paired check exist
  const float* pair_x;       // input whose whole forward stage a paired check has already done (NULL: none)
  int pair_B;
  // set by codenet_step for the next check of this layer, cleared by it: the activation applied to the
  // forward sums (step C1) and the input whose derivative masks the backward sums (step C2)
  mutable int out_act;
  mutable const float* out_mask;
  // a recorded step's iteration counter: the backward check of the step's last layer advances it itself when
  // no other kernel of the step reads it afterwards (bump_done tells the recorder that it did)
  codenet::SmallDev small = {0, 0, 0, 0, 0, 0, 0.0f, nullptr, 0};   // soft errors in the small steps
  mutable int z_cleared = 0;        // the vector-encoding kernel has zeroed the backward outputs for the split sweep
  mutable int sweep_reverse = 0;    // direction of the next single-pass update sweep (alternates)
  mutable int operands_ready = 0;   // the vector-encoding kernel has written the tensor-core operand copies
  mutable uint32_t* bump_after = nullptr;
  mutable bool bump_done = false;
  std::vector<float> P_row_host, P_col_host;   // host copies of the parity parts of the generators
  // the last checkpoint of the stored state (coded blocks, inner checksums); NULL until one is taken
  void* ck_W = nullptr;
  float* ck_U = nullptr;
  float* ck_V = nullptr;
};

namespace codenet {
using codenet_layer_impl = ::codenet_layer;

extern unsigned long long g_launches;
inline void count_launch(int n = 1) { g_launches += (unsigned long long)n; }

// Optional event brackets around the streaming kernels (see codenet_profile_enable).
void profile_begin(int kernel, cudaStream_t st);
void profile_end(int kernel, cudaStream_t st);
struct ProfileScope {
  int k; cudaStream_t st;
  ProfileScope(int kernel, cudaStream_t s) : k(kernel), st(s) { profile_begin(k, st); }
  ~ProfileScope() { profile_end(k, st); }
};

// ---- launchers (kernels_stream.cu) ----------------------------------------------------------
cudaError_t launch_forward_products(const Geom& g, const float* x, int ldx, int B, float* Y,
                                    cudaStream_t st);
cudaError_t launch_forward_products_plain(const Geom& g, const float* x, int ldx, int B, float* Y,
                                          cudaStream_t st);   // never allocates (no profiling events)
// xnext != NULL: also produce the next iteration's feedforward partials ynext[strip][coded row][b]
struct LossFuse;
// enc_fuse != NULL: the launch also carries the additional encoding of the vectors (which then is not launched on its
// own): its CTAs write Xt, Dt, the slice sums, delta^L and the loss partials for the check that follows, and the sweep
// forms the delta~ / x~ entries it needs itself from the sums, the target and the raw input.
cudaError_t launch_backward_update_fused(const codenet_layer_impl& L, int B, float lr, float* zpart,
                                         const float* xnext, int ldxn, float* ynext, cudaStream_t st,
                                         const float* enc_X = nullptr, const float* enc_Delta = nullptr,
                                         const LossFuse* enc_fuse = nullptr);
// The 16-byte path of the vector encoding needs every length, offset and pointer to be a multiple of four floats.
inline bool encode_vec_ok(const Geom& g, const float* X, const float* Delta, const float* S, const float* target) {
  return g.b_c % 4 == 0 && g.b_r % 4 == 0 && g.Tc % 4 == 0 && g.T % 4 == 0 && g.n_in % 4 == 0 && g.n_out % 4 == 0 &&
         g.Mbr % 4 == 0 && (reinterpret_cast<uintptr_t>(X) & 15u) == 0 && (reinterpret_cast<uintptr_t>(Delta) & 15u) == 0 &&
         (reinterpret_cast<uintptr_t>(S) & 15u) == 0 && (reinterpret_cast<uintptr_t>(target) & 15u) == 0;
}
int backward_strip_elems(int dtype);  // columns per CTA of the fused backward kernel
cudaError_t launch_backward_products(const codenet_layer_impl& L, int B, float* Z, cudaStream_t st);
cudaError_t launch_update(const codenet_layer_impl& L, int B, float lr, cudaStream_t st);

// ---- launchers (kernels_tc.cu) --------------------------------------------------------------
bool tc_forward_supported(const Geom& g, int math, int B);
cudaError_t launch_tc_forward(const codenet_layer_impl& L, const float* X, int B, float* Y, cudaStream_t st);
bool tc_backward_supported(const Geom& g, int math, int B);
// needs ws.Dt (encoded delta) of this call; Z is [i][j][col][b]
cudaError_t launch_tc_backward(const codenet_layer_impl& L, int B, float* Z, cudaStream_t st);
bool tc_update_supported(const Geom& g, int math, int B);
// needs ws.Xt and ws.Dt (encoded vectors) of this call
cudaError_t launch_tc_update(const codenet_layer_impl& L, int B, float lr, cudaStream_t st);
// Steps O2 and O3 in one tensor-core sweep (bfloat16 blocks): Z receives the backward node products.
bool tc_backward_update_supported(const Geom& g, int math, int B);
cudaError_t launch_tc_backward_update(const codenet_layer_impl& L, int B, float lr, float* Z, cudaStream_t st);

// ---- launchers (kernels_check.cu) -----------------------------------------------------------
cudaError_t launch_encode_layer(const Geom& g, const void* W, cudaStream_t st);
// Mean-squared-error loss folded into the vector encoding of the last layer: delta^L = 2 (y - s) / (N B) is
// formed where the delta segments are read, stored to `delta`, and the loss is gathered from one partial
// per data segment (n_part = m * slices * B of them) by the last CTA to finish.
constexpr int LOSS_FUSE_PARTIALS = 8192;   // scratch for the partial sums of the folded loss
struct LossFuse {
  const float* S; const float* target; float* delta;
  float scale;            // 1 / (N B)
  float* partials; unsigned* counter; float* loss_out;
  int n_part;
  int defer;              // the partials are added up later in the step (by the paired check that ends it), not here
};
// emit: 0 = the fp32 vectors only; 1 = also their transposes (rows, B) for the fused TF32 kernel; 2 = also the
// bfloat16 copies the fused bf16 kernel reads (delta~ as a hi / lo pair, x~ rounded).  Sets L.operands_ready
// when the extra copies were written (the 16-byte path only).
// small != NULL: soft errors in the additional encoding (the parity sub-vectors of hit units get noise)
cudaError_t launch_encode_vectors(const codenet_layer_impl& L, const float* X, const float* Delta,
                                  int B, cudaStream_t st, const LossFuse* fuse = nullptr, int emit = 0,
                                  const SmallDev* small = nullptr, float* clear = nullptr, size_t clear_floats = 0);
// Does the fused tensor-core sweep share an item's row tiles out among two CTAs (which add into a cleared Z)?
bool tc_backward_update_splits(const codenet_layer_impl& L, int B);
// Output deviations of the feedforward nodes whose own input copy the plan hits, into L.ws.dY (zeroed first).
cudaError_t launch_input_faults(const codenet_layer_impl& L, int B, cudaStream_t st);
// Injection, detection, location, decoding plan and the final sums over codewords.
// src_kind: 0 = canonical [cw][node][len][B] in `src`; 1 = backward partials [i][rt][b][ld];
// 2 = feedforward partials [strip][coded row][b] with ldb / strip-width strips per block-column.
// Vraw: X (forward) or Delta (backward) as the caller passed it.  commit: write corrected codewords to Yw.
cudaError_t launch_check(const codenet_layer_impl& L, int phase, const float* src, int src_kind, float* Yw,
                         const float* Vraw, int B, const FaultDev* fault, int have_clean, int commit, float* out,
                         float lr, int update_checksums, codenet_report_t* rep, cudaStream_t st, uint32_t it_add = 0u);
// The backward check of this iteration (arguments as launch_check, phase BWD, partials of the fused sweep) and the
// forward check of the next one on the products the sweep took ahead (X_next, its fault plan read one iteration
// on, sums to S_next, report to rep_next) in one cooperative launch.  commit_*: staged sums / report of the previous
// pair to copy out on entry, or NULL.  The caller has checked pair_supported.
struct PairNext {
  const float* X_next;
  const FaultDev* fault;
  float* S_next;
  codenet_report_t* rep_next;
  const float* commit_S; float* commit_S_to; int commit_n;
  const codenet_report_t* commit_rep; codenet_report_t* commit_rep_to;
  const float* loss_partials; int loss_n; float* loss_out;   // a loss whose partial sums wait to be added up, or NULL
};
bool pair_supported(const codenet_layer_impl& L, int B);
bool pair_checks(const codenet_layer_impl& L);   // the pair is the cooperative check kernel (else: the two plain sums)
cudaError_t launch_check_pair(const codenet_layer_impl& L, const float* src, float* Yw, const float* Delta, int B,
                              const FaultDev* fault, float* out, float lr, codenet_report_t* rep,
                              const PairNext& nx, cudaStream_t st);
size_t check_scratch_floats(const Geom& g, int B);  // size of Workspace::chk for batches > 8
cudaError_t launch_sum_outputs(const Geom& g, int phase, int B, const float* Y, float* out, int out_act, codenet_report_t* rep,
                               cudaStream_t st);
cudaError_t launch_decode_weights(const Geom& g, void* W_out, cudaStream_t st);
cudaError_t launch_check_invariance(const Geom& g, float* out, cudaStream_t st);
cudaError_t launch_get_block(const Geom& g, int i, int j, float* out, cudaStream_t st);
cudaError_t launch_corrupt_block(const Geom& g, int i, int j, uint32_t seed, uint32_t layer, uint32_t iteration,
                                 uint32_t density_q32, float amplitude, cudaStream_t st);
// status_dev: set to 1 by the kernel when no parity of that direction involves the block
cudaError_t launch_regenerate_block(const Geom& g, int i, int j, int along, int* status_dev, cudaStream_t st);
// plain streaming copy of `bytes` bytes (both pointers 16-byte aligned), used by checkpoint save / restore
cudaError_t launch_copy_bytes(const void* src, void* dst, size_t bytes, cudaStream_t st);
cudaError_t launch_get_checksums(const Geom& g, int i, int j, float* u_out, float* v_out, cudaStream_t st);
cudaError_t launch_activation(float* x, size_t n, int act, cudaStream_t st);
// partials: 512 floats of scratch, counter: one zero-initialised word (both owned by the network)
cudaError_t launch_loss(const float* S, const void* target, int B, int n, int loss, float* delta,
                        float* loss_out, float* partials, unsigned* counter, cudaStream_t st);
cudaError_t launch_bump_counter(uint32_t* counter, cudaStream_t st);
cudaError_t launch_sum_loss_partials(const float* partials, int n, float* out, cudaStream_t st);
cudaError_t launch_mask_delta(float* C, const float* x, size_t n, int act, cudaStream_t st);

// ---- device helpers -------------------------------------------------------------------------
#ifdef __CUDACC__

__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              uint32_t k0, uint32_t k1, uint32_t out[4]) {
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Additive noise of element e of a hit node: twelve 16-bit uniforms, centred, scaled by
// sigma / 65536.  Integer until the last two float products.
__device__ __forceinline__ float soft_error_noise(uint32_t seed, uint32_t key1, uint32_t iteration,
                                                  uint32_t node_id, uint32_t e, float sigma) {
  uint32_t a[4], b[4];
  philox4x32_10(iteration, node_id, e, 1u, seed, key1, a);
  philox4x32_10(iteration, node_id, e, 2u, seed, key1, b);
  int sum = 0;
#pragma unroll
  for (int w = 0; w < 4; ++w) sum += (int)(a[w] & 0xFFFFu) + (int)(a[w] >> 16);
#pragma unroll
  for (int w = 0; w < 2; ++w) sum += (int)(b[w] & 0xFFFFu) + (int)(b[w] >> 16);
  const float unit = __fmul_rn((float)(sum - 393210), 1.0f / 65536.0f);
  return __fmul_rn(sigma, unit);
}

__device__ __forceinline__ bool node_is_hit(const FaultDev& f, uint32_t phase, uint32_t iteration,
                                            uint32_t node_id, uint32_t active_index, uint32_t n_active) {
  if (f.mode == CODENET_FAULT_NONE) return false;
  uint32_t o[4];
  const uint32_t key1 = (f.layer << 8) | phase;
  if (f.mode == CODENET_FAULT_BERNOULLI) {
    philox4x32_10(iteration, node_id, 0u, 0u, f.seed, key1, o);
    return o[0] < f.p_q32;
  }
  philox4x32_10(iteration, 0xFFFFFFFFu, 0u, 0u, f.seed, key1, o);
  return (o[0] % n_active) == active_index;
}

__device__ __forceinline__ bool small_is_hit(const SmallDev& sf, uint32_t phase, uint32_t iteration, uint32_t unit) {
  const uint32_t pq = phase == CODENET_PHASE_ENCODE ? sf.p_encode : phase == CODENET_PHASE_INPUT ? sf.p_input
                    : phase == CODENET_PHASE_CHECK ? sf.p_check : sf.p_decode;
  if (!sf.on || pq == 0u) return false;
  uint32_t o[4];
  philox4x32_10(iteration, unit, 0u, 0u, sf.seed, (sf.layer << 8) | phase, o);
  return o[0] < pq;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
  return v;
}

// 16-byte vector of storage elements -> floats (4 for float, 8 for bfloat16).
template <typename T> struct Vec16;
template <> struct Vec16<float> {
  static constexpr int N = 4;
  __device__ __forceinline__ static void load(const float* p, float (&v)[4]) {
    const float4 t = *reinterpret_cast<const float4*>(p);
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
  }
  __device__ __forceinline__ static void load_stream(const float* p, float (&v)[4]) {
    const float4 t = __ldcs(reinterpret_cast<const float4*>(p));
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
  }
  __device__ __forceinline__ static void store(float* p, const float (&v)[4]) {
    *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
  }
};
template <> struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ __forceinline__ static void unpack(const uint4& t, float (&v)[8]) {
    const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      v[2 * k] = __uint_as_float(w[k] << 16);
      v[2 * k + 1] = __uint_as_float(w[k] & 0xFFFF0000u);
    }
  }
  __device__ __forceinline__ static void load(const __nv_bfloat16* p, float (&v)[8]) {
    unpack(*reinterpret_cast<const uint4*>(p), v);
  }
  __device__ __forceinline__ static void load_stream(const __nv_bfloat16* p, float (&v)[8]) {
    unpack(__ldcs(reinterpret_cast<const uint4*>(p)), v);
  }
  __device__ __forceinline__ static void store(__nv_bfloat16* p, const float (&v)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * k], v[2 * k + 1]);
      w[k] = *reinterpret_cast<const uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
  }
};

__device__ __forceinline__ float load_elem(const void* base, int dtype, size_t idx) {
  return dtype == CODENET_BF16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(base)[idx])
                               : reinterpret_cast<const float*>(base)[idx];
}
__device__ __forceinline__ void store_elem(void* base, int dtype, size_t idx, float v) {
  if (dtype == CODENET_BF16) reinterpret_cast<__nv_bfloat16*>(base)[idx] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(base)[idx] = v;
}

#endif  // __CUDACC__

}  // namespace codenet
