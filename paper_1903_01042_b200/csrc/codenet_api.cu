// C interface of libcodenet: argument checks, layout planning, workspace, launch order.
#include "codenet_internal.cuh"

#include <algorithm>
#include <cmath>
#include <new>
#include <vector>

using namespace codenet;

struct codenet_net {
  int L, activation, loss, batch_max;
  std::vector<codenet_layer*> layers;
  std::vector<float*> xs;  // xs[l] = input of layer l for l >= 1 (library-owned)
  float* out_last;         // (B, n_L)
  const float* x_next;     // input of the next step, for layer 1's look-ahead products (one-shot)
  float* s_stage;          // one-layer networks: sums of the next step's forward stage, done ahead by a paired check
  codenet_report_t* rep_stage;   // its report, until the step it belongs to ends
  uint32_t* step_counter;  // device word every codenet_step advances when it ends (codenet_net_set_iteration_counter), or NULL
  int lookahead;           // 0: announced next inputs are ignored (every step runs its own forward sweep)
  float* delta[2];         // ping-pong error vectors, (B, widest layer)
  float* loss_partials;    // 512 partial sums + one counter word (loss kernel), then LOSS_FUSE_PARTIALS + a counter (loss folded into the vector encoding)
  std::vector<cudaGraphExec_t> graphs;  // captured steps (codenet_net_capture_step)
};

namespace {

inline size_t round_up(size_t a, size_t b) { return (a + b - 1) / b * b; }

template <typename T> cudaError_t dev_alloc(T** p, size_t count) {
  *p = nullptr;
  if (count == 0) count = 1;
  return cudaMalloc(reinterpret_cast<void**>(p), count * sizeof(T));
}

void free_layer_memory(codenet_layer* L) {
  cudaFree(L->g.Wt); cudaFree(L->g.U); cudaFree(L->g.V);
  cudaFree(L->ck_W); cudaFree(L->ck_U); cudaFree(L->ck_V);
  cudaFree(const_cast<float*>(L->g.Pr)); cudaFree(const_cast<float*>(L->g.Pc));
  cudaFree(L->ws.Xt); cudaFree(L->ws.Dt); cudaFree(L->ws.dsum); cudaFree(L->ws.xsum);
  cudaFree(L->ws.tc_x); cudaFree(L->ws.tc_d); cudaFree(L->ws.tc_dT); cudaFree(L->ws.tc_xT); cudaFree(L->ws.tc_flag); cudaFree(L->ws.chk);
  cudaFree(L->ws.Y); cudaFree(L->ws.Yw); cudaFree(L->ws.Yw2); cudaFree(L->ws.pair_sums); cudaFree(L->ws.Ynext); cudaFree(L->ws.stats); cudaFree(L->ws.plan);
  cudaFree(L->ws.dY);
}

int cuda_status(cudaError_t e) {
  if (e == cudaSuccess) return CODENET_OK;
  if (e == cudaErrorMemoryAllocation) return CODENET_E_NOMEM;
  return CODENET_E_CUDA;
}

bool fill_fault(const codenet_fault_t* f, FaultDev* out) {
  if (!f || f->mode == CODENET_FAULT_NONE) return false;
  out->seed = f->seed; out->layer = f->layer; out->mode = f->mode; out->p_q32 = f->p_q32;
  out->sigma = f->sigma; out->iteration = f->iteration_dev;
  return true;
}

struct ProfileState {
  bool on = false;
  std::vector<cudaEvent_t> ev[CODENET_KERNEL_COUNT];  // begin/end pairs
  size_t used[CODENET_KERNEL_COUNT] = {0, 0, 0, 0, 0};
} g_prof;
constexpr size_t kMaxProfiled = 4096;

#define CN_TRY(expr)                                 \
  do {                                               \
    cudaError_t e__ = (expr);                        \
    if (e__ != cudaSuccess) return cuda_status(e__); \
  } while (0)

}  // namespace

namespace codenet {
bool stream_is_capturing(cudaStream_t st) {
  cudaStreamCaptureStatus status = cudaStreamCaptureStatusNone;
  return cudaStreamIsCapturing(st, &status) == cudaSuccess && status != cudaStreamCaptureStatusNone;
}
void profile_begin(int kernel, cudaStream_t st) {
  if (!g_prof.on || g_prof.used[kernel] >= kMaxProfiled || stream_is_capturing(st)) return;
  std::vector<cudaEvent_t>& v = g_prof.ev[kernel];
  const size_t need = 2 * (g_prof.used[kernel] + 1);
  while (v.size() < need) {
    cudaEvent_t e;
    if (cudaEventCreate(&e) != cudaSuccess) return;
    v.push_back(e);
  }
  cudaEventRecord(v[2 * g_prof.used[kernel]], st);
}
void profile_end(int kernel, cudaStream_t st) {
  if (!g_prof.on || g_prof.used[kernel] >= kMaxProfiled || stream_is_capturing(st)) return;
  std::vector<cudaEvent_t>& v = g_prof.ev[kernel];
  if (v.size() < 2 * (g_prof.used[kernel] + 1)) return;
  cudaEventRecord(v[2 * g_prof.used[kernel] + 1], st);
  g_prof.used[kernel]++;
}
}  // namespace codenet

namespace {
// Inverse of an s x s matrix (s <= CODENET_MAX_PARITY) by elimination with partial pivoting; false when singular.
bool host_invert(int s, const double* A, double* inv) {
  double a[CODENET_MAX_PARITY][2 * CODENET_MAX_PARITY];
  for (int r = 0; r < s; ++r)
    for (int c = 0; c < s; ++c) { a[r][c] = A[r * s + c]; a[r][s + c] = r == c ? 1.0 : 0.0; }
  for (int pv = 0; pv < s; ++pv) {
    int best = pv;
    for (int r = pv + 1; r < s; ++r) if (std::fabs(a[r][pv]) > std::fabs(a[best][pv])) best = r;
    if (a[best][pv] == 0.0) return false;
    for (int c = 0; c < 2 * s; ++c) std::swap(a[pv][c], a[best][c]);
    const double piv = a[pv][pv];
    for (int c = 0; c < 2 * s; ++c) a[pv][c] /= piv;
    for (int r = 0; r < s; ++r) {
      if (r == pv) continue;
      const double f = a[r][pv];
      for (int c = 0; c < 2 * s; ++c) a[r][c] -= f * a[pv][c];
    }
  }
  for (int r = 0; r < s; ++r) for (int c = 0; c < s; ++c) inv[r * s + c] = a[r][s + c];
  return true;
}

// Worst figures over every erasure sub-system of the parity part P (k x r): see codenet_code_conditioning.
void code_conditioning(const std::vector<float>& P, int k, int r, double out[3]) {
  out[0] = out[1] = out[2] = 0.0;
  for (int s = 1; s <= r && s <= k; ++s) {
    std::vector<int> F(s);
    for (int a = 0; a < s; ++a) F[a] = a;
    for (;;) {
      for (unsigned mask = 0; mask < (1u << r); ++mask) {
        int Q[CODENET_MAX_PARITY], nq = 0;
        for (int q = 0; q < r; ++q) if ((mask >> q) & 1u) Q[nq++] = q;
        if (nq != s) continue;
        double A[CODENET_MAX_PARITY * CODENET_MAX_PARITY], Ai[CODENET_MAX_PARITY * CODENET_MAX_PARITY];
        for (int a = 0; a < s; ++a) for (int b = 0; b < s; ++b) A[a * s + b] = (double)P[(size_t)F[b] * r + Q[a]];
        if (!host_invert(s, A, Ai)) { out[0] = out[1] = out[2] = INFINITY; continue; }
        double w[CODENET_MAX_PARITY];
        for (int b = 0; b < s; ++b) {
          w[b] = 1.0;
          for (int kk = 0; kk < k; ++kk) {
            bool in_f = false;
            for (int f = 0; f < s; ++f) in_f = in_f || F[f] == kk;
            if (!in_f) w[b] += std::fabs((double)P[(size_t)kk * r + Q[b]]);
          }
        }
        double na = 0.0, ni = 0.0, amp = 0.0;
        for (int a = 0; a < s; ++a) {
          double ra = 0.0, ri = 0.0, am = 0.0;
          for (int b = 0; b < s; ++b) { ra += std::fabs(A[a * s + b]); ri += std::fabs(Ai[a * s + b]); am += std::fabs(Ai[a * s + b]) * w[b]; }
          na = std::max(na, ra); ni = std::max(ni, ri); amp = std::max(amp, am);
        }
        out[0] = std::max(out[0], na * ni); out[1] = std::max(out[1], ni); out[2] = std::max(out[2], amp);
      }
      // next combination of s data indices out of k
      int pos = s - 1;
      while (pos >= 0 && F[pos] == k - s + pos) --pos;
      if (pos < 0) break;
      ++F[pos];
      for (int a = pos + 1; a < s; ++a) F[a] = F[a - 1] + 1;
    }
  }
}
}  // namespace

extern "C" {

int codenet_code_conditioning(const codenet_layer_t* L, int phase, double out[3]) {
  if (!L || !out || (phase != CODENET_PHASE_FWD && phase != CODENET_PHASE_BWD)) return CODENET_E_BADARG;
  if (phase == CODENET_PHASE_FWD) code_conditioning(L->P_row_host, L->g.m, L->g.r_row, out);
  else code_conditioning(L->P_col_host, L->g.n, L->g.r_col, out);
  return CODENET_OK;
}

int codenet_profile_enable(int on) {
  g_prof.on = on != 0;
  if (on) for (int k = 0; k < CODENET_KERNEL_COUNT; ++k) g_prof.used[k] = 0;
  return CODENET_OK;
}

int codenet_profile_read(int kernel, float* total_ms, uint64_t* launches) {
  if (kernel < 0 || kernel >= CODENET_KERNEL_COUNT || !total_ms || !launches) return CODENET_E_BADARG;
  if (cudaDeviceSynchronize() != cudaSuccess) return CODENET_E_CUDA;
  float total = 0.0f;
  for (size_t k = 0; k < g_prof.used[kernel]; ++k) {
    float ms = 0.0f;
    if (cudaEventElapsedTime(&ms, g_prof.ev[kernel][2 * k], g_prof.ev[kernel][2 * k + 1]) != cudaSuccess)
      return CODENET_E_CUDA;
    total += ms;
  }
  *total_ms = total;
  *launches = g_prof.used[kernel];
  return CODENET_OK;
}

const char* codenet_strerror(int code) {
  switch (code) {
    case CODENET_OK: return "ok";
    case CODENET_E_BADARG: return "bad argument";
    case CODENET_E_SHAPE: return "unsupported grid or block shape";
    case CODENET_E_CUDA: return "CUDA call failed (is a CUDA device present?)";
    case CODENET_E_NOMEM: return "device allocation failed";
    case CODENET_E_TOOBIG: return "rows * n_blocks exceeds the 2^20-float scratch of codenet_matvec_noalloc";
    default: return "unknown error code";
  }
}

uint64_t codenet_launch_count(void) { return g_launches; }

int codenet_encode_layer(const codenet_layer_desc_t* d, const void* W_dev, codenet_stream_t stream,
                         codenet_layer_t** out) {
  if (!d || !W_dev || !out) return CODENET_E_BADARG;
  *out = nullptr;
  if (d->n_out < 1 || d->n_in < 1 || d->m < 1 || d->n < 1 || d->batch_max < 1) return CODENET_E_BADARG;
  if (d->dtype != CODENET_F32 && d->dtype != CODENET_BF16) return CODENET_E_BADARG;
  if (d->math < CODENET_MATH_FFMA || d->math > CODENET_MATH_BF16) return CODENET_E_BADARG;
  if (d->math == CODENET_MATH_TF32 && d->dtype != CODENET_F32) return CODENET_E_BADARG;
  if (d->math == CODENET_MATH_BF16 && d->dtype != CODENET_BF16) return CODENET_E_BADARG;
  if (d->locate_mode < CODENET_LOCATE_NONE || d->locate_mode > CODENET_LOCATE_JOINT) return CODENET_E_BADARG;
  if (d->r_row < 0 || d->r_col < 0 || d->r_row > CODENET_MAX_PARITY || d->r_col > CODENET_MAX_PARITY)
    return CODENET_E_SHAPE;
  if (d->m + d->r_row > CODENET_MAX_NODES || d->n + d->r_col > CODENET_MAX_NODES) return CODENET_E_SHAPE;
  if (d->m > d->n_out || d->n > d->n_in) return CODENET_E_SHAPE;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) return CODENET_E_CUDA;

  codenet_layer* L = new (std::nothrow) codenet_layer();
  if (!L) return CODENET_E_NOMEM;
  L->desc = *d;
  L->desc.P_row = nullptr;
  L->desc.P_col = nullptr;
  L->batch_max = d->batch_max;
  L->out_act = CODENET_ACT_IDENTITY;
  L->out_mask = nullptr;
  L->next_x = nullptr;
  L->next_B = 0;
  L->ws.Ynext = nullptr;
  L->ws.dY = nullptr;
  L->ws.tc_x = nullptr;
  L->ws.tc_d = nullptr;
  L->ws.tc_dT = nullptr;
  L->ws.tc_xT = nullptr;
  L->ws.tc_flag = nullptr;
  L->ws.chk = nullptr;
  Geom& g = L->g;
  g.n_out = d->n_out; g.n_in = d->n_in; g.m = d->m; g.n = d->n; g.r_row = d->r_row; g.r_col = d->r_col;
  g.M = d->m + d->r_row; g.Nn = d->n + d->r_col;
  g.b_r = (d->n_out + d->m - 1) / d->m;
  g.b_c = (d->n_in + d->n - 1) / d->n;
  const int vec = d->dtype == CODENET_BF16 ? 8 : 4;
  g.ldb = (int)round_up((size_t)g.b_c, (size_t)vec);
  g.ld = g.Nn * g.ldb;
  g.T = d->check_rows > 0 ? d->check_rows : g.b_r;
  if (g.b_r % g.T != 0) { delete L; return CODENET_E_SHAPE; }
  g.ns = g.b_r / g.T;
  g.Tc = d->check_cols > 0 ? d->check_cols : g.b_c;
  if (g.b_c % g.Tc != 0) { delete L; return CODENET_E_SHAPE; }
  g.nsc = g.b_c / g.Tc;
  g.Mbr = g.M * g.b_r;
  g.dtype = d->dtype; g.locate_mode = d->locate_mode; g.tau_rel = d->tau_rel; g.tau_abs = d->tau_abs;
  L->bwd_rows = g.b_r < 64 ? g.b_r : 64;
  L->bwd_rt = (g.b_r + L->bwd_rows - 1) / L->bwd_rows;

  const size_t esz = d->dtype == CODENET_BF16 ? 2 : 4;
  const size_t Bm = (size_t)d->batch_max;
  const size_t w_bytes = (size_t)g.Mbr * g.ld * esz;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  cudaError_t e = cudaSuccess;
  float *Pr = nullptr, *Pc = nullptr;
  Workspace& ws = L->ws;
  const size_t fwd_elems = (size_t)g.n * g.Mbr * Bm;
  const size_t bwd_canon = (size_t)g.m * g.Nn * g.b_c * Bm;
  const size_t bwd_part = (size_t)g.m * L->bwd_rt * (Bm < 8 ? Bm : 8) * g.ld;
  ws.y_elems = fwd_elems;
  if (Bm > 8 && bwd_canon > ws.y_elems) ws.y_elems = bwd_canon;
  if (bwd_part > ws.y_elems) ws.y_elems = bwd_part;
  ws.yw_elems = fwd_elems > bwd_canon ? fwd_elems : bwd_canon;
  do {
    if ((e = cudaMalloc(&g.Wt, w_bytes)) != cudaSuccess) break;
    if ((e = dev_alloc(&g.U, (size_t)g.M * g.Nn * g.ns * g.ldb)) != cudaSuccess) break;
    if ((e = dev_alloc(&g.V, (size_t)g.M * g.Nn * g.nsc * g.b_r)) != cudaSuccess) break;
    if ((e = dev_alloc(&Pr, (size_t)g.m * (g.r_row > 0 ? g.r_row : 1))) != cudaSuccess) break;
    if ((e = dev_alloc(&Pc, (size_t)g.n * (g.r_col > 0 ? g.r_col : 1))) != cudaSuccess) break;
    g.Pr = Pr; g.Pc = Pc;
    if ((e = dev_alloc(&ws.Xt, Bm * g.ld)) != cudaSuccess) break;
    if ((e = dev_alloc(&ws.Dt, Bm * g.Mbr)) != cudaSuccess) break;
    if ((e = dev_alloc(&ws.dsum, (size_t)g.M * g.ns * Bm)) != cudaSuccess) break;
    if ((e = dev_alloc(&ws.xsum, (size_t)g.Nn * g.nsc * Bm)) != cudaSuccess) break;
    if ((e = dev_alloc(&ws.Y, ws.y_elems)) != cudaSuccess) break;
    if ((e = dev_alloc(&ws.Yw, ws.yw_elems)) != cudaSuccess) break;
    if ((e = dev_alloc(&ws.tc_flag, (size_t)4)) != cudaSuccess) break;
    if ((e = cudaMemsetAsync(ws.tc_flag, 0, 4 * sizeof(int), st)) != cudaSuccess) break;
    if (Bm > 8) {
      if ((e = dev_alloc(&ws.chk, check_scratch_floats(g, (int)Bm))) != cudaSuccess) break;
    }
    if (d->math != CODENET_MATH_FFMA && Bm >= 64) {
      // fp32 copy, or a bfloat16 hi/lo pair: 4 bytes per element either way
      if ((e = cudaMalloc(&ws.tc_x, Bm * (size_t)g.n * g.ldb * 4)) != cudaSuccess) break;
      if ((e = cudaMalloc(&ws.tc_d, Bm * (size_t)g.Mbr * 4)) != cudaSuccess) break;
      if ((e = cudaMalloc(&ws.tc_dT, Bm * (size_t)g.Mbr * 4)) != cudaSuccess) break;
      if ((e = cudaMalloc(&ws.tc_xT, Bm * (size_t)g.ld * 4)) != cudaSuccess) break;
    }
    // the update sweep can also take the next feedforward products when its column strips tile the
    // block-columns exactly and x needs no padding
    L->next_ok = (g.ldb % backward_strip_elems(g.dtype) == 0) && g.ldb == g.b_c && g.n * g.b_c == g.n_in;
    const size_t Bs = Bm < 8 ? Bm : 8;   // the streaming path serves batches up to 8
    if (L->next_ok) {
      const size_t strips = (size_t)g.n * g.ldb / backward_strip_elems(g.dtype);
      if ((e = dev_alloc(&ws.Ynext, strips * g.Mbr * Bs)) != cudaSuccess) break;
      // a second working copy and the hand-over scratch for the forward part of a paired check (batch 1)
      if ((e = dev_alloc(&ws.Yw2, (size_t)g.n * g.Mbr)) != cudaSuccess) break;
      if ((e = dev_alloc(&ws.pair_sums, (size_t)2 * g.n * g.M * g.ns)) != cudaSuccess) break;
      L->pair_ok = 1;
    }
    if ((e = dev_alloc(&ws.stats, (size_t)4)) != cudaSuccess) break;
    if ((e = dev_alloc(&ws.plan, (size_t)2 * CODENET_MAX_NODES)) != cudaSuccess) break;
    std::vector<float> pr((size_t)g.m * (g.r_row > 0 ? g.r_row : 1), 1.0f);
    std::vector<float> pc((size_t)g.n * (g.r_col > 0 ? g.r_col : 1), 1.0f);
    if (d->P_row) for (int k = 0; k < g.m * g.r_row; ++k) pr[k] = d->P_row[k];
    if (d->P_col) for (int k = 0; k < g.n * g.r_col; ++k) pc[k] = d->P_col[k];
    L->P_row_host = pr;
    L->P_col_host = pc;
    if ((e = cudaMemcpy(Pr, pr.data(), pr.size() * sizeof(float), cudaMemcpyHostToDevice)) != cudaSuccess) break;
    if ((e = cudaMemcpy(Pc, pc.data(), pc.size() * sizeof(float), cudaMemcpyHostToDevice)) != cudaSuccess) break;
    if ((e = cudaMemsetAsync(g.Wt, 0, w_bytes, st)) != cudaSuccess) break;
    if ((e = cudaMemsetAsync(ws.stats, 0, sizeof(CheckStats) * 4, st)) != cudaSuccess) break;
    if ((e = cudaMemsetAsync(ws.plan, 0, sizeof(CwPlan) * 2 * CODENET_MAX_NODES, st)) != cudaSuccess) break;
    if ((e = launch_encode_layer(g, W_dev, st)) != cudaSuccess) break;
  } while (0);
  if (e != cudaSuccess) {
    free_layer_memory(L);
    delete L;
    return cuda_status(e);
  }
  *out = L;
  return CODENET_OK;
}

void codenet_free_layer(codenet_layer_t* L) {
  if (!L) return;
  cudaDeviceSynchronize();
  free_layer_memory(L);
  delete L;
}

int codenet_layer_dims(const codenet_layer_t* L, int32_t dims[10]) {
  if (!L || !dims) return CODENET_E_BADARG;
  const Geom& g = L->g;
  dims[0] = g.b_r; dims[1] = g.b_c; dims[2] = g.M; dims[3] = g.Nn; dims[4] = g.T; dims[5] = g.ns;
  dims[6] = g.m * g.b_r; dims[7] = g.n * g.b_c; dims[8] = g.Tc; dims[9] = g.nsc;
  return CODENET_OK;
}

// it_add: added to the fault plan's device counter (1 when the call stands for the next iteration's forward stage)
static int forward_impl(codenet_layer_t* L, const float* X_dev, int B, const codenet_fault_t* fault,
                        float* S_dev, codenet_report_t* rep_dev, codenet_stream_t stream, uint32_t it_add);

int codenet_forward(codenet_layer_t* L, const float* X_dev, int B, const codenet_fault_t* fault,
                    float* S_dev, codenet_report_t* rep_dev, codenet_stream_t stream) {
  return forward_impl(L, X_dev, B, fault, S_dev, rep_dev, stream, 0u);
}

static int forward_impl(codenet_layer_t* L, const float* X_dev, int B, const codenet_fault_t* fault,
                        float* S_dev, codenet_report_t* rep_dev, codenet_stream_t stream, uint32_t it_add) {
  if (!L || !X_dev || !S_dev || B < 1 || B > L->batch_max) return CODENET_E_BADARG;
  L->pair_x = nullptr;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const Geom& g = L->g;
  // x can be read in place when no padding separates its sub-vectors
  const bool direct = g.ldb == g.b_c && g.n * g.b_c == g.n_in &&
                      (reinterpret_cast<uintptr_t>(X_dev) & 15u) == 0 && (g.n_in % 4) == 0;
  const float* x = X_dev;
  int ldx = g.n_in;
  FaultDev fd;
  const bool inject = fill_fault(fault, &fd);
  // products already taken from the updated weights by the previous update sweep?
  const bool have_next = L->next_x != nullptr && L->next_x == X_dev && L->next_B == B;
  L->next_x = nullptr;
  if (have_next) {
    CN_TRY(launch_input_faults(*L, B, st));
    CN_TRY(launch_check(*L, CODENET_PHASE_FWD, L->ws.Ynext, 2, L->ws.Yw, X_dev, B, inject ? &fd : nullptr, 1, 0,
                        S_dev, 0.0f, 0, rep_dev, st, it_add));
    return CODENET_OK;
  }
  if (!direct) {
    CN_TRY(launch_encode_vectors(*L, X_dev, nullptr, B, st));
    x = L->ws.Xt;
    ldx = g.ld;
  }
  if (tc_forward_supported(g, L->desc.math, B)) CN_TRY(launch_tc_forward(*L, X_dev, B, L->ws.Y, st));
  else CN_TRY(launch_forward_products(g, x, ldx, B, L->ws.Y, st));
  const bool checks = inject || L->small.on ||
                      (g.locate_mode != CODENET_LOCATE_OFF && (g.r_row > 0 || g.locate_mode == CODENET_LOCATE_NODECHECK));
  if (checks) CN_TRY(launch_input_faults(*L, B, st));
  if (checks)
    CN_TRY(launch_check(*L, CODENET_PHASE_FWD, L->ws.Y, 0, L->ws.Yw, X_dev, B, inject ? &fd : nullptr, 1, 0, S_dev,
                        0.0f, 0, rep_dev, st, it_add));
  else {
    const int act = L->out_act;
    L->out_act = CODENET_ACT_IDENTITY;
    CN_TRY(launch_sum_outputs(g, CODENET_PHASE_FWD, B, L->ws.Y, S_dev, act, rep_dev, st));
  }
  return CODENET_OK;
}

int codenet_backward_update(codenet_layer_t* L, const float* Delta_dev, const float* X_dev, int B,
                            float lr, const codenet_fault_t* fault, float* C_dev,
                            codenet_report_t* rep_dev, codenet_stream_t stream) {
  return codenet_backward_update_next(L, Delta_dev, X_dev, B, lr, fault, C_dev, rep_dev, nullptr, stream);
}

// fuse != NULL: delta^L is formed from the last layer's sums and the target while the vectors are encoded
// (Delta_dev receives it), see LossFuse.
// pair != NULL: the forward stage of the next iteration (input X_next_dev) is wanted as well; where the layer allows
// it (pair_supported, products taken ahead by the sweep) its check shares a launch with the backward check and
// *paired is set, otherwise the caller runs it.
struct PairWish {
  const codenet_fault_t* fault_next;
  float* S_next;
  codenet_report_t* rep_next;
  const float* commit_S; float* commit_S_to; int commit_n;
  const codenet_report_t* commit_rep; codenet_report_t* commit_rep_to;
  const float* loss_partials; int loss_n; float* loss_out;
};
static int backward_update_impl(codenet_layer_t* L, const float* Delta_dev, const float* X_dev, int B,
                                float lr, const codenet_fault_t* fault, float* C_dev,
                                codenet_report_t* rep_dev, const float* X_next_dev, codenet_stream_t stream,
                                const LossFuse* fuse, const PairWish* pair = nullptr, bool* paired = nullptr);
static bool lookahead_ok(const codenet_layer_t* L, const float* X_next_dev, int B) {
  return X_next_dev != nullptr && B <= 8 && L->next_ok && (reinterpret_cast<uintptr_t>(X_next_dev) & 15u) == 0 &&
         (L->g.n_in % 4) == 0;
}

int codenet_backward_update_next(codenet_layer_t* L, const float* Delta_dev, const float* X_dev, int B,
                                 float lr, const codenet_fault_t* fault, float* C_dev,
                                 codenet_report_t* rep_dev, const float* X_next_dev, codenet_stream_t stream) {
  return backward_update_impl(L, Delta_dev, X_dev, B, lr, fault, C_dev, rep_dev, X_next_dev, stream, nullptr);
}

int codenet_backward_update_forward_next(codenet_layer_t* L, const float* Delta_dev, const float* X_dev, int B,
                                         float lr, const codenet_fault_t* fault, float* C_dev,
                                         codenet_report_t* rep_dev, const float* X_next_dev,
                                         const codenet_fault_t* fault_next, float* S_next_dev,
                                         codenet_report_t* rep_next_dev, codenet_stream_t stream) {
  if (!X_next_dev || !S_next_dev) return CODENET_E_BADARG;
  PairWish w;
  memset(&w, 0, sizeof(w));
  w.fault_next = fault_next; w.S_next = S_next_dev; w.rep_next = rep_next_dev;
  bool paired = false;
  const int rc = backward_update_impl(L, Delta_dev, X_dev, B, lr, fault, C_dev, rep_dev, X_next_dev, stream, nullptr,
                                      &w, &paired);
  if (rc != CODENET_OK || paired) return rc;
  return forward_impl(L, X_next_dev, B, fault_next, S_next_dev, rep_next_dev, stream, 1u);
}

static int backward_update_impl(codenet_layer_t* L, const float* Delta_dev, const float* X_dev, int B,
                                float lr, const codenet_fault_t* fault, float* C_dev,
                                codenet_report_t* rep_dev, const float* X_next_dev, codenet_stream_t stream,
                                const LossFuse* fuse, const PairWish* pair, bool* paired) {
  if (!L || !Delta_dev || !X_dev || B < 1 || B > L->batch_max) return CODENET_E_BADARG;
  if (paired) *paired = false;
  L->pair_x = nullptr;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const Geom& g = L->g;
  // the operand copies of the fused tensor-core kernel ride on the vector encoding
  const int emit = (B > 8 && tc_backward_update_supported(g, L->desc.math, B)) ? (g.dtype == CODENET_F32 ? 1 : 2) : 0;
  // (a fused tensor-core sweep that shares items out among CTAs adds into Z: the encoding kernel clears it on its way)
  const bool clear_z = emit != 0 && tc_backward_update_splits(*L, B);
  const bool next = B <= 8 && lookahead_ok(L, X_next_dev, B);
  // The step of a one-layer network with the loss folded into the encoding, a look-ahead sweep and a paired check
  // behind it: the encoding rides on the sweep's launch instead of standing between the previous check and the sweep.
  FaultDev fd, fdn;
  const bool inject = fill_fault(fault, &fd);
  const bool inject_next = pair != nullptr && fill_fault(pair->fault_next, &fdn);
  // (a layer that checks nothing can share a launch for its two sums only while nothing is to be injected)
  const bool can_pair = pair != nullptr && next && C_dev != nullptr && pair->S_next != nullptr && pair_supported(*L, B) &&
                        (pair_checks(*L) || (!inject && !inject_next));
  const bool ride = can_pair && fuse != nullptr && fuse->defer && !L->small.on;
  if (!ride)
    CN_TRY(launch_encode_vectors(*L, X_dev, Delta_dev, B, st, fuse, emit, L->small.on ? &L->small : nullptr,
                                 clear_z ? L->ws.Y : nullptr, clear_z ? (size_t)g.m * g.Nn * g.b_c * B : 0));
  int src_kind;
  if (B <= 8) {
    CN_TRY(launch_backward_update_fused(*L, B, lr, L->ws.Y, next ? X_next_dev : nullptr, g.n_in, L->ws.Ynext, st,
                                        ride ? X_dev : nullptr, ride ? Delta_dev : nullptr, ride ? fuse : nullptr));
    L->next_x = next ? X_next_dev : nullptr;
    L->next_B = B;
    src_kind = 1;
  } else {
    if (tc_backward_update_supported(g, L->desc.math, B)) {
      CN_TRY(launch_tc_backward_update(*L, B, lr, L->ws.Y, st));   // one sweep for both steps
    } else {
      if (tc_backward_supported(g, L->desc.math, B)) CN_TRY(launch_tc_backward(*L, B, L->ws.Y, st));
      else CN_TRY(launch_backward_products(*L, B, L->ws.Y, st));
      if (tc_update_supported(g, L->desc.math, B)) CN_TRY(launch_tc_update(*L, B, lr, st));
      else CN_TRY(launch_update(*L, B, lr, st));
    }
    src_kind = 0;
  }
  if (can_pair) {
    PairNext nx;
    nx.X_next = X_next_dev; nx.fault = inject_next ? &fdn : nullptr; nx.S_next = pair->S_next; nx.rep_next = pair->rep_next;
    nx.commit_S = pair->commit_S; nx.commit_S_to = pair->commit_S_to; nx.commit_n = pair->commit_n;
    nx.commit_rep = pair->commit_rep; nx.commit_rep_to = pair->commit_rep_to;
    nx.loss_partials = pair->loss_partials; nx.loss_n = pair->loss_n; nx.loss_out = pair->loss_out;
    CN_TRY(launch_check_pair(*L, L->ws.Y, L->ws.Yw, Delta_dev, B, inject ? &fd : nullptr, C_dev, lr, rep_dev, nx, st));
    L->next_x = nullptr;         // the products taken ahead are used up
    L->pair_x = X_next_dev;
    L->pair_B = B;
    if (paired) *paired = true;
    return CODENET_OK;
  }
  CN_TRY(launch_check(*L, CODENET_PHASE_BWD, L->ws.Y, src_kind, L->ws.Yw, Delta_dev, B, inject ? &fd : nullptr, 1, 0,
                      C_dev, lr, 1, rep_dev, st));
  return CODENET_OK;
}

int codenet_corrupt_block(codenet_layer_t* L, int i, int j, uint32_t seed, uint32_t fault_layer,
                          uint32_t iteration, uint32_t density_q32, float amplitude, codenet_stream_t stream) {
  if (!L) return CODENET_E_BADARG;
  const Geom& g = L->g;
  if (i < 0 || j < 0 || i >= g.M || j >= g.Nn || (i >= g.m && j >= g.n)) return CODENET_E_BADARG;
  CN_TRY(launch_corrupt_block(g, i, j, seed, fault_layer, iteration, density_q32, amplitude,
                              reinterpret_cast<cudaStream_t>(stream)));
  L->next_x = nullptr;   // products taken ahead from the blocks as they were no longer describe them
  L->pair_x = nullptr;
  return CODENET_OK;
}

int codenet_regenerate_block(codenet_layer_t* L, int i, int j, int along, codenet_stream_t stream) {
  if (!L || (along != 0 && along != 1)) return CODENET_E_BADARG;
  const Geom& g = L->g;
  if (i < 0 || j < 0 || i >= g.M || j >= g.Nn || (i >= g.m && j >= g.n)) return CODENET_E_BADARG;
  // the codeword exists only where the other coordinate is a data index (no corner blocks)
  if (along == 0 ? (g.r_row < 1 || j >= g.n) : (g.r_col < 1 || i >= g.m)) return CODENET_E_SHAPE;
  // a data block needs a parity whose generator entry for it is not zero: the host copy of P decides
  const int kd = along == 0 ? g.m : g.n, r = along == 0 ? g.r_row : g.r_col, pos = along == 0 ? i : j;
  if (pos < kd) {
    const std::vector<float>& P = along == 0 ? L->P_row_host : L->P_col_host;
    bool any = false;
    for (int t = 0; t < r; ++t) any = any || P[(size_t)pos * r + t] != 0.0f;
    if (!any) return CODENET_E_SHAPE;
  }
  CN_TRY(launch_regenerate_block(g, i, j, along, nullptr, reinterpret_cast<cudaStream_t>(stream)));
  L->next_x = nullptr;
  L->pair_x = nullptr;
  return CODENET_OK;
}

int codenet_layer_set_small_faults(codenet_layer_t* L, const codenet_small_faults_t* plan) {
  if (!L) return CODENET_E_BADARG;
  if (plan == nullptr) { L->small.on = 0; return CODENET_OK; }
  if (plan->p_input_q32 != 0u && L->ws.dY == nullptr) {
    // the deviations of the nodes with an erroneous input copy need a buffer of the size of the node outputs
    const size_t elems = (size_t)L->g.n * L->g.Mbr * (size_t)L->batch_max;
    if (cudaMalloc(reinterpret_cast<void**>(&L->ws.dY), elems * sizeof(float)) != cudaSuccess) {
      cudaGetLastError();
      L->ws.dY = nullptr;
      return CODENET_E_NOMEM;
    }
  }
  L->small.seed = plan->seed; L->small.layer = plan->layer;
  L->small.p_encode = plan->p_encode_q32; L->small.p_input = plan->p_input_q32;
  L->small.p_check = plan->p_check_q32; L->small.p_decode = plan->p_decode_q32;
  L->small.sigma = plan->sigma; L->small.iteration = plan->iteration_dev;
  L->small.on = 1;
  return CODENET_OK;
}

int codenet_detect_decode(const codenet_layer_t* Lc, int phase, float* Y_dev, const float* V_dev, int B,
                          codenet_report_t* rep_dev, codenet_stream_t stream) {
  if (!Lc || !Y_dev || !V_dev || B < 1 || B > Lc->batch_max) return CODENET_E_BADARG;
  if (phase != CODENET_PHASE_FWD && phase != CODENET_PHASE_BWD) return CODENET_E_BADARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const codenet_layer& L = *Lc;  // the workspace behind the handle is scratch, not layer state
  CN_TRY(launch_check(L, phase, Y_dev, 0, Y_dev, V_dev, B, nullptr, 0, 1, nullptr, 0.0f, 0, rep_dev, st));
  return CODENET_OK;
}

// sizes of the three stored arrays in bytes
static void stored_bytes(const Geom& g, size_t* w, size_t* u, size_t* v) {
  *w = (size_t)g.Mbr * g.ld * (g.dtype == CODENET_BF16 ? 2 : 4);
  *u = (size_t)g.M * g.Nn * g.ns * g.ldb * sizeof(float);
  *v = (size_t)g.M * g.Nn * g.nsc * g.b_r * sizeof(float);
}

int codenet_checkpoint_save(codenet_layer_t* L, codenet_stream_t stream) {
  if (!L) return CODENET_E_BADARG;
  size_t wb, ub, vb;
  stored_bytes(L->g, &wb, &ub, &vb);
  if (!L->ck_W) {
    void* w = nullptr; float *u = nullptr, *v = nullptr;
    cudaError_t e = cudaMalloc(&w, wb ? wb : 16);
    if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&u), ub ? ub : 16);
    if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&v), vb ? vb : 16);
    if (e != cudaSuccess) { cudaFree(w); cudaFree(u); cudaFree(v); cudaGetLastError(); return CODENET_E_NOMEM; }
    L->ck_W = w; L->ck_U = u; L->ck_V = v;
  }
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  CN_TRY(launch_copy_bytes(L->g.Wt, L->ck_W, wb, st));
  CN_TRY(launch_copy_bytes(L->g.U, L->ck_U, ub, st));
  CN_TRY(launch_copy_bytes(L->g.V, L->ck_V, vb, st));
  return CODENET_OK;
}

int codenet_checkpoint_restore(codenet_layer_t* L, codenet_stream_t stream) {
  if (!L) return CODENET_E_BADARG;
  if (!L->ck_W) return CODENET_E_BADARG;   // no checkpoint has been taken
  size_t wb, ub, vb;
  stored_bytes(L->g, &wb, &ub, &vb);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  CN_TRY(launch_copy_bytes(L->ck_W, L->g.Wt, wb, st));
  CN_TRY(launch_copy_bytes(L->ck_U, L->g.U, ub, st));
  CN_TRY(launch_copy_bytes(L->ck_V, L->g.V, vb, st));
  L->next_x = nullptr;   // products taken ahead from the blocks as they were no longer describe them
  L->pair_x = nullptr;
  return CODENET_OK;
}

int codenet_decode_weights(const codenet_layer_t* L, void* W_dev_out, codenet_stream_t stream) {
  if (!L || !W_dev_out) return CODENET_E_BADARG;
  CN_TRY(launch_decode_weights(L->g, W_dev_out, reinterpret_cast<cudaStream_t>(stream)));
  return CODENET_OK;
}

int codenet_check_invariance(const codenet_layer_t* L, float* max_rel_dev, codenet_stream_t stream) {
  if (!L || !max_rel_dev) return CODENET_E_BADARG;
  CN_TRY(launch_check_invariance(L->g, max_rel_dev, reinterpret_cast<cudaStream_t>(stream)));
  return CODENET_OK;
}

int codenet_get_block(const codenet_layer_t* L, int i, int j, float* out_dev, codenet_stream_t stream) {
  if (!L || !out_dev) return CODENET_E_BADARG;
  const Geom& g = L->g;
  if (i < 0 || j < 0 || i >= g.M || j >= g.Nn || (i >= g.m && j >= g.n)) return CODENET_E_BADARG;
  CN_TRY(launch_get_block(g, i, j, out_dev, reinterpret_cast<cudaStream_t>(stream)));
  return CODENET_OK;
}

int codenet_get_checksums(const codenet_layer_t* L, int i, int j, float* u_out_dev, float* v_out_dev,
                          codenet_stream_t stream) {
  if (!L) return CODENET_E_BADARG;
  const Geom& g = L->g;
  if (i < 0 || j < 0 || i >= g.M || j >= g.Nn || (i >= g.m && j >= g.n)) return CODENET_E_BADARG;
  CN_TRY(launch_get_checksums(g, i, j, u_out_dev, v_out_dev, reinterpret_cast<cudaStream_t>(stream)));
  return CODENET_OK;
}

int codenet_net_create(codenet_layer_t** layers, int L, int activation, int loss, codenet_net_t** out) {
  if (!layers || !out || L < 1) return CODENET_E_BADARG;
  *out = nullptr;
  if (activation != CODENET_ACT_IDENTITY && activation != CODENET_ACT_RELU) return CODENET_E_BADARG;
  if (loss != CODENET_LOSS_MSE_MEAN && loss != CODENET_LOSS_SOFTMAX_CE) return CODENET_E_BADARG;
  int bmax = 1 << 30, widest = 0;
  for (int l = 0; l < L; ++l) {
    if (!layers[l]) return CODENET_E_BADARG;
    if (l > 0 && layers[l]->g.n_in != layers[l - 1]->g.n_out) return CODENET_E_SHAPE;
    if (layers[l]->batch_max < bmax) bmax = layers[l]->batch_max;
    if (layers[l]->g.n_in > widest) widest = layers[l]->g.n_in;
    if (layers[l]->g.n_out > widest) widest = layers[l]->g.n_out;
  }
  codenet_net* net = new (std::nothrow) codenet_net();
  if (!net) return CODENET_E_NOMEM;
  net->L = L; net->activation = activation; net->loss = loss; net->batch_max = bmax;
  net->layers.assign(layers, layers + L);
  net->xs.assign(L, nullptr);
  net->out_last = nullptr;
  net->s_stage = nullptr;
  net->rep_stage = nullptr;
  net->step_counter = nullptr;
  net->lookahead = 1;
  net->x_next = nullptr;
  net->delta[0] = net->delta[1] = nullptr;
  net->loss_partials = nullptr;
  cudaError_t e = cudaSuccess;
  for (int l = 1; l < L && e == cudaSuccess; ++l) e = dev_alloc(&net->xs[l], (size_t)bmax * layers[l]->g.n_in);
  if (e == cudaSuccess) e = dev_alloc(&net->out_last, (size_t)bmax * layers[L - 1]->g.n_out);
  if (e == cudaSuccess && L == 1) e = dev_alloc(&net->s_stage, (size_t)bmax * layers[0]->g.n_out);
  if (e == cudaSuccess) e = dev_alloc(&net->rep_stage, (size_t)1);
  if (e == cudaSuccess) e = dev_alloc(&net->delta[0], (size_t)bmax * widest);
  if (e == cudaSuccess) e = dev_alloc(&net->delta[1], (size_t)bmax * widest);
  if (e == cudaSuccess) e = dev_alloc(&net->loss_partials, (size_t)513 + LOSS_FUSE_PARTIALS + 1);
  if (e == cudaSuccess) e = cudaMemset(net->loss_partials, 0, (513 + LOSS_FUSE_PARTIALS + 1) * sizeof(float));
  if (e != cudaSuccess) {
    codenet_free_net(net);
    return cuda_status(e);
  }
  *out = net;
  return CODENET_OK;
}

void codenet_free_net(codenet_net_t* net) {
  if (!net) return;
  cudaDeviceSynchronize();
  for (cudaGraphExec_t ge : net->graphs) cudaGraphExecDestroy(ge);
  for (float* p : net->xs) cudaFree(p);
  cudaFree(net->out_last);
  cudaFree(net->s_stage);
  cudaFree(net->rep_stage);
  cudaFree(net->delta[0]);
  cudaFree(net->delta[1]);
  cudaFree(net->loss_partials);
  delete net;
}

int codenet_net_output(const codenet_net_t* net, float* out_dev, int B, codenet_stream_t stream) {
  if (!net || !out_dev || B < 1 || B > net->batch_max) return CODENET_E_BADARG;
  const size_t bytes = (size_t)B * net->layers[net->L - 1]->g.n_out * sizeof(float);
  CN_TRY(cudaMemcpyAsync(out_dev, net->out_last, bytes, cudaMemcpyDeviceToDevice, reinterpret_cast<cudaStream_t>(stream)));
  return CODENET_OK;
}

int codenet_step(codenet_net_t* net, const float* X_dev, const void* target_dev, int B, float lr,
                 const codenet_fault_t* per_layer, codenet_report_t* reps_dev, float* loss_dev,
                 codenet_stream_t stream) {
  if (!net || !X_dev || !target_dev || B < 1 || B > net->batch_max) return CODENET_E_BADARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const int L = net->L;
  if (!net->lookahead) net->x_next = nullptr;
  // The first layer's forward stage may have been done by the previous step (its check shared a launch with that
  // step's last backward check): its sums are in place (in the staging buffer for a one-layer network), its report
  // is staged.  And this step may end the same way for the next input.
  codenet_layer* L0 = net->layers[0];
  const bool paired_in = L0->pair_x != nullptr && L0->pair_x == X_dev && L0->pair_B == B;
  const bool pair_out = lookahead_ok(L0, net->x_next, B) && pair_supported(*L0, B);
  const float* out_cur = net->out_last;   // where this step's last sums are while the step runs
  PairWish wish;
  memset(&wish, 0, sizeof(wish));
  if (paired_in) {
    codenet_report_t* rep0 = reps_dev ? &reps_dev[0] : nullptr;
    if (pair_out) {
      // the paired check at the end of this step copies them out before it reuses the staging buffers
      if (L == 1) { out_cur = net->s_stage; wish.commit_S = net->s_stage; wish.commit_S_to = net->out_last; wish.commit_n = B * L0->g.n_out; }
      if (rep0) { wish.commit_rep = net->rep_stage; wish.commit_rep_to = rep0; }
    } else {
      if (L == 1) CN_TRY(cudaMemcpyAsync(net->out_last, net->s_stage, (size_t)B * L0->g.n_out * sizeof(float), cudaMemcpyDeviceToDevice, st));
      if (rep0) CN_TRY(cudaMemcpyAsync(rep0, net->rep_stage, sizeof(codenet_report_t), cudaMemcpyDeviceToDevice, st));
    }
  }
  // feedforward: step O1 with its checks, then step C1
  for (int l = paired_in ? 1 : 0; l < L; ++l) {
    const float* x = l == 0 ? X_dev : net->xs[l];
    float* S = l < L - 1 ? net->xs[l + 1] : net->out_last;
    // step C1 rides on the sums: x^{l+1} = f(s^l) is what the check writes
    net->layers[l]->out_act = l < L - 1 ? net->activation : CODENET_ACT_IDENTITY;
    int rc = codenet_forward(net->layers[l], x, B, per_layer ? &per_layer[l] : nullptr, S,
                             reps_dev ? &reps_dev[2 * l] : nullptr, stream);
    if (rc != CODENET_OK) return rc;
  }
  // the mean-squared-error loss rides on the vector encoding of the last layer's backward stage (one
  // kernel fewer); other losses, large batches, or more partial sums than the scratch holds, take the loss kernel
  LossFuse fuse;
  fuse.defer = 0;
  const Geom& gl = net->layers[L - 1]->g;
  const int n_part = gl.m * gl.ns * B;
  // (small batches only: with many batch entries the parity segments would form delta m times over)
  const bool fused_loss = net->loss == CODENET_LOSS_MSE_MEAN && n_part <= LOSS_FUSE_PARTIALS && B <= 8;
  if (fused_loss) {
    fuse.S = out_cur; fuse.target = reinterpret_cast<const float*>(target_dev); fuse.delta = net->delta[0];
    fuse.scale = 1.0f / ((float)gl.n_out * (float)B);
    fuse.partials = net->loss_partials + 513; fuse.counter = reinterpret_cast<unsigned*>(net->loss_partials + 513 + LOSS_FUSE_PARTIALS);
    fuse.loss_out = loss_dev; fuse.n_part = n_part;
    // a step that ends with a paired check lets that kernel add the loss partials up: the vector encoding sits
    // between two sweeps and should not wait for its last CTA
    fuse.defer = (pair_out && loss_dev != nullptr) ? 1 : 0;
    if (fuse.defer) { wish.loss_partials = fuse.partials; wish.loss_n = n_part; wish.loss_out = loss_dev; }
  } else {
    CN_TRY(launch_loss(out_cur, target_dev, B, gl.n_out, net->loss, net->delta[0], loss_dev,
                       net->loss_partials, reinterpret_cast<unsigned*>(net->loss_partials + 512), st));
  }
  // a step counter of the network's own: the step's last check kernel advances it where it can (a recording sets
  // bump_after itself and then this stays out of the way)
  const bool own_bump = net->step_counter != nullptr && L0->bump_after == nullptr;
  if (own_bump) { L0->bump_after = net->step_counter; L0->bump_done = false; }
  // backpropagation: step O2 with its checks fused with the update O3, then step C2
  int cur = 0;
  for (int l = L - 1; l >= 0; --l) {
    const float* x = l == 0 ? X_dev : net->xs[l];
    // step C2 rides on the sums: delta^{l-1} = c^l (.) g(x^l)
    net->layers[l]->out_mask = (l > 0 && net->activation == CODENET_ACT_RELU) ? x : nullptr;
    const bool wish_pair = l == 0 && pair_out;
    if (wish_pair) {
      // the forward stage of the next step, first layer: sums to where that step's second layer (or its loss) reads
      // them, the activation between the layers applied as they are written
      wish.fault_next = per_layer ? &per_layer[0] : nullptr;
      wish.S_next = L == 1 ? net->s_stage : net->xs[1];
      wish.rep_next = net->rep_stage;
      L0->out_act = L > 1 ? net->activation : CODENET_ACT_IDENTITY;
    }
    bool paired = false;
    int rc = backward_update_impl(net->layers[l], net->delta[cur], x, B, lr,
                                  per_layer ? &per_layer[l] : nullptr, net->delta[cur ^ 1],
                                  reps_dev ? &reps_dev[2 * l + 1] : nullptr,
                                  l == 0 ? net->x_next : nullptr, stream, (l == L - 1 && fused_loss) ? &fuse : nullptr,
                                  wish_pair ? &wish : nullptr, &paired);
    if (rc != CODENET_OK) return rc;
    if (wish_pair && !paired) {
      L0->out_act = CODENET_ACT_IDENTITY;
      // (no pair after all: what was staged for this step goes out by plain copies)
      if (wish.commit_S) CN_TRY(cudaMemcpyAsync(wish.commit_S_to, wish.commit_S, (size_t)wish.commit_n * sizeof(float), cudaMemcpyDeviceToDevice, st));
      if (wish.commit_rep) CN_TRY(cudaMemcpyAsync(wish.commit_rep_to, wish.commit_rep, sizeof(codenet_report_t), cudaMemcpyDeviceToDevice, st));
      if (wish.loss_partials) CN_TRY(launch_sum_loss_partials(wish.loss_partials, wish.loss_n, wish.loss_out, st));
    }
    cur ^= 1;
  }
  net->x_next = nullptr;
  if (own_bump) {
    const bool bumped = L0->bump_done;
    L0->bump_after = nullptr;
    L0->bump_done = false;
    if (!bumped) CN_TRY(launch_bump_counter(net->step_counter, st));
  }
  return CODENET_OK;
}

int codenet_net_set_lookahead(codenet_net_t* net, int on) {
  if (!net) return CODENET_E_BADARG;
  net->lookahead = on ? 1 : 0;
  if (!on) net->x_next = nullptr;
  return CODENET_OK;
}

int codenet_net_set_iteration_counter(codenet_net_t* net, uint32_t* counter_dev) {
  if (!net) return CODENET_E_BADARG;
  net->step_counter = counter_dev;
  return CODENET_OK;
}

int codenet_net_capture_step(codenet_net_t* net, const float* X_dev, const void* target_dev, int B, float lr,
                             const codenet_fault_t* per_layer, codenet_report_t* reps_dev, float* loss_dev,
                             const float* X_next_dev, codenet_stream_t stream, int* graph_id) {
  return codenet_net_capture_steps(net, 1, &X_dev, &target_dev, B, lr, per_layer, reps_dev, 0, loss_dev, 0, X_next_dev,
                                   stream, graph_id);
}

int codenet_net_capture_steps(codenet_net_t* net, int n_steps, const float* const* X_devs,
                              const void* const* target_devs, int B, float lr, const codenet_fault_t* per_layer,
                              codenet_report_t* reps_dev, int reps_stride, float* loss_dev, int loss_stride,
                              const float* X_next_dev, codenet_stream_t stream, int* graph_id) {
  if (!net || !graph_id || n_steps < 1 || !X_devs || !target_devs || reps_stride < 0 || loss_stride < 0)
    return CODENET_E_BADARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (st == nullptr || stream_is_capturing(st)) return CODENET_E_BADARG;  // the default stream cannot record
  CN_TRY(cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal));
  // a recorded step ends by advancing each iteration counter its fault plans read (once per counter).  With one
  // counter for the whole network the step's last kernel, the backward check of the first layer, can do it
  // itself; otherwise one-thread kernels follow.
  const uint32_t* only = nullptr;
  bool single = per_layer != nullptr;
  for (int l = 0; l < net->L && single; ++l) {
    const uint32_t* ctr = per_layer[l].iteration_dev;
    if (ctr == nullptr) continue;
    if (only == nullptr) only = ctr;
    else if (only != ctr) single = false;
  }
  const codenet_layer_impl* first = net->layers[0];
  int rc = CODENET_OK;
  for (int s = 0; s < n_steps && rc == CODENET_OK; ++s) {
    net->x_next = s + 1 < n_steps ? X_devs[s + 1] : X_next_dev;
    first->bump_after = (single && only != nullptr) ? const_cast<uint32_t*>(only) : nullptr;
    first->bump_done = false;
    rc = codenet_step(net, X_devs[s], target_devs[s], B, lr, per_layer,
                      reps_dev ? reps_dev + (size_t)s * reps_stride : nullptr,
                      loss_dev ? loss_dev + (size_t)s * loss_stride : nullptr, stream);
    const bool bumped = first->bump_done;
    first->bump_after = nullptr;
    first->bump_done = false;
    if (rc == CODENET_OK && per_layer && !bumped) {
      for (int l = 0; l < net->L && rc == CODENET_OK; ++l) {
        const uint32_t* ctr = per_layer[l].iteration_dev;
        bool seen = ctr == nullptr;
        for (int k = 0; k < l && !seen; ++k) seen = per_layer[k].iteration_dev == ctr;
        if (!seen && launch_bump_counter(const_cast<uint32_t*>(ctr), st) != cudaSuccess) rc = CODENET_E_CUDA;
      }
    }
  }
  cudaGraph_t graph = nullptr;
  const cudaError_t e = cudaStreamEndCapture(st, &graph);
  if (rc != CODENET_OK) { if (graph) cudaGraphDestroy(graph); return rc; }
  if (e != cudaSuccess || !graph) return CODENET_E_CUDA;
  cudaGraphExec_t exec = nullptr;
  const cudaError_t e2 = cudaGraphInstantiate(&exec, graph, 0);
  cudaGraphDestroy(graph);
  if (e2 != cudaSuccess) return cuda_status(e2);
  // the device-side copy of the graph is made now, not by the first replay
  if (cudaGraphUpload(exec, st) != cudaSuccess) { cudaGraphExecDestroy(exec); return CODENET_E_CUDA; }
  net->graphs.push_back(exec);
  *graph_id = (int)net->graphs.size() - 1;
  return CODENET_OK;
}

int codenet_net_replay(codenet_net_t* net, int graph_id, codenet_stream_t stream) {
  if (!net || graph_id < 0 || graph_id >= (int)net->graphs.size()) return CODENET_E_BADARG;
  CN_TRY(cudaGraphLaunch(net->graphs[graph_id], reinterpret_cast<cudaStream_t>(stream)));
  return CODENET_OK;
}

int codenet_net_set_next_input(codenet_net_t* net, const float* X_next_dev) {
  if (!net) return CODENET_E_BADARG;
  net->x_next = X_next_dev;
  return CODENET_OK;
}

}  // extern "C"
