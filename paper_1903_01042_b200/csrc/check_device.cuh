// Device helpers shared by the kernels that check node outputs: the cooperative check / fix kernels and
// the last-arriver tail of the fused backward + update sweep.  Included inside namespace codenet { namespace {
// of each translation unit that uses them.
#pragma once

constexpr int CK_THREADS = 256;
constexpr int CK_WARPS = CK_THREADS / 32;
constexpr int MAXR = CODENET_MAX_PARITY;
constexpr int MAXN = CODENET_MAX_NODES;
constexpr int BIG_WC = 8;     // large batches: 16-byte accesses in flight per lane
constexpr int BIG_SR = 64;    // large batches: rows per work item of the statistics pass
constexpr int BIG_DC = 128;   // large batches: dot-product entries per work item
constexpr int BIG_TR = 16;    // large batches: positions per tile of the syndrome / sums pass
constexpr int BIG_KD = 16;    // large batches: most data nodes per codeword the one-pass sums handle

struct CheckParams {
  Geom g;
  int phase, B, src_kind, have_clean, RT, commit, update_checksums, spb;  // spb: strips per block-column
  float lr;
  FaultDev fault;
  const float* src;    // clean node outputs: canonical, or backward partials [i][rt][b][ld]
  float* Yw;           // working copy [codeword][node][len][B]
  const float* Vraw;   // X (B, n_in) for the forward check, Delta (B, n_out) for the backward check
  float* out;          // S (B, n_out) / C (B, n_in) or NULL
  const float* Xt; const float* Dt; const float* dsum; const float* xsum;
  CheckStats* st; CheckStats* st_next;   // set by the kernel from st_base and *parity
  CheckStats* st_base;     // two statistics buffers used alternately: a check works in one and clears the other
  int* parity;             // device word: which buffer the next check kernel uses (flipped by the kernel itself, so
                           // eager calls and replayed graphs can follow one another in any order)
  CwPlan* plan;
  codenet_report_t* rep;
  const int* tc_flag;  // non-zero: a tensor-core kernel of this layer gave up on a bounded wait
  float* chk;          // large batches: [unit][b][partials] of slice sum / magnitudes and checksum dot / scale
  int lazy;                // large-batch path: node outputs stay where the product kernel wrote them, only
                           // hit nodes get a working copy (set by the host together with the instantiation)
  int inline_fix;          // small batches, at most one parity, sums wanted: the CTAs that decided the codewords stay
                           // until the last one has and, if some codeword needs work, recompute the sums of the
                           // located / fallen-back nodes together: no fix kernel follows
  int tail_fix;            // large batches, or two and more parities: every CTA stays until the last codeword has
                           // decided and, if some codeword needs work, the whole grid does what the fix kernel would
  int out_act;             // forward sums: activation applied as they are written (step C1), or identity
  const float* out_mask;   // backward sums: zeroed where this input is not positive (step C2), or NULL
  uint32_t* bump;          // iteration counter of the fault plans to advance when the kernel ends, or NULL
  SmallDev small;          // soft errors in the small steps (input copies, the two verification steps); on == 0: none
  const float* dY;         // output deviations of the nodes whose input copy is hit [codeword][node][len][B], or NULL
  // --- paired launch (the backward check of one iteration and the forward check of the next in one kernel) ---
  uint32_t it_add;         // added to the fault plan's counter: 1 for the look-ahead forward check, whose
                           // iteration starts only when the counter has been advanced
  int pair;                // 0: a check of its own; 1: the backward part of a pair; 2: the forward part
  float* pair_sums;        // forward part: [unit][2] slice sum and magnitude sum, from phase U to phase X
  const float* commit_S; float* commit_S_to; int commit_n;   // forward part, on entry: sums and report of the
  const codenet_report_t* commit_rep; codenet_report_t* commit_rep_to;   // previous pair go where the caller reads them
  const float* loss_partials; int loss_n; float* loss_out;   // forward part: partial sums of this step's loss to add up
};

struct PhaseGeom {
  int n_cw, K, kd, r, len, nsl, slen;
  size_t n_el;
  const float* P;
};

__device__ __forceinline__ PhaseGeom phase_geom(const Geom& g, int phase, int B) {
  PhaseGeom q;
  if (phase == CODENET_PHASE_FWD) {
    q.n_cw = g.n; q.K = g.M; q.kd = g.m; q.r = g.r_row; q.len = g.b_r; q.nsl = g.ns; q.slen = g.T; q.P = g.Pr;
  } else {
    q.n_cw = g.m; q.K = g.Nn; q.kd = g.n; q.r = g.r_col; q.len = g.b_c; q.nsl = g.nsc; q.slen = g.Tc; q.P = g.Pc;
  }
  q.n_el = (size_t)q.len * B;
  return q;
}

// A sum on its way out: s -> f(s) for the feedforward sums, c -> c * [x > 0] for the backpropagated ones.
__device__ __forceinline__ float finish_out(const CheckParams& p, float acc, size_t idx) {
  if (p.out_act == CODENET_ACT_RELU && acc < 0.0f) acc = 0.0f;
  if (p.out_mask != nullptr && !(p.out_mask[idx] > 0.0f)) acc = 0.0f;
  return acc;
}

// The noise of one element of a hit node, as a real call: hit nodes are rare, and every inlined copy of the
// generator is a few kilobytes of instructions that the clean path would have to fetch past.
__device__ __noinline__ float hit_noise(uint32_t seed, uint32_t key1, uint32_t iteration, uint32_t node_id, uint32_t e,
                                        float sigma) {
  return soft_error_noise(seed, key1, iteration, node_id, e, sigma);
}

__device__ __forceinline__ float clean_value(const CheckParams& p, const PhaseGeom& q, int cw, int k, size_t e) {
  if (p.src_kind == 0) return p.src[((size_t)cw * q.K + k) * q.n_el + e];
  if (p.src_kind == 2) {  // feedforward partials of the column strips of block-column cw, fixed order
    float v = 0.0f;
    for (int s = 0; s < p.spb; ++s) v += p.src[((size_t)(cw * p.spb + s) * p.g.Mbr) * p.B + (size_t)k * q.n_el + e];
    return v;
  }
  const int pos = (int)(e / p.B), b = (int)(e % p.B);
  const float* s0 = p.src + ((size_t)cw * p.RT * p.B + b) * p.g.ld + (size_t)k * p.g.ldb + pos;
  const size_t step = (size_t)p.B * p.g.ld;
  // fixed summation order (row tiles in increasing order), loads issued sixteen at a time
  float v = 0.0f;
  int rt = 0;
  for (; rt + 16 <= p.RT; rt += 16) {
    float a[16];
#pragma unroll
    for (int w = 0; w < 16; ++w) a[w] = s0[(size_t)(rt + w) * step];
#pragma unroll
    for (int w = 0; w < 16; ++w) v += a[w];
  }
  for (; rt + 4 <= p.RT; rt += 4) {
    const float a0 = s0[(size_t)rt * step], a1 = s0[(size_t)(rt + 1) * step];
    const float a2 = s0[(size_t)(rt + 2) * step], a3 = s0[(size_t)(rt + 3) * step];
    v = (((v + a0) + a1) + a2) + a3;
  }
  for (; rt < p.RT; ++rt) v += s0[(size_t)rt * step];
  return v;
}

// clean_value for four elements of one node at a time: the same sums in the same order, with the partials of
// all four (eight rows of partials per round) in flight together.  Elements that are not wanted repeat e[0].
__device__ __forceinline__ void clean_value4(const CheckParams& p, const PhaseGeom& q, int cw, int k,
                                             const size_t (&e)[4], float (&v)[4]) {
  if (p.src_kind == 0) {
#pragma unroll
    for (int u = 0; u < 4; ++u) v[u] = p.src[((size_t)cw * q.K + k) * q.n_el + e[u]];
    return;
  }
  const float* s0[4];
  size_t step;
  int np;
  if (p.src_kind == 2) {
#pragma unroll
    for (int u = 0; u < 4; ++u) s0[u] = p.src + ((size_t)cw * p.spb * p.g.Mbr) * p.B + (size_t)k * q.n_el + e[u];
    step = (size_t)p.g.Mbr * p.B;
    np = p.spb;
  } else {
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int pos = (int)(e[u] / p.B), b = (int)(e[u] % p.B);
      s0[u] = p.src + ((size_t)cw * p.RT * p.B + b) * p.g.ld + (size_t)k * p.g.ldb + pos;
    }
    step = (size_t)p.B * p.g.ld;
    np = p.RT;
  }
#pragma unroll
  for (int u = 0; u < 4; ++u) v[u] = 0.0f;
  int r = 0;
  for (; r + 8 <= np; r += 8) {
    float a[4][8];
#pragma unroll
    for (int w = 0; w < 8; ++w)
#pragma unroll
      for (int u = 0; u < 4; ++u) a[u][w] = s0[u][(size_t)(r + w) * step];
#pragma unroll
    for (int w = 0; w < 8; ++w)
#pragma unroll
      for (int u = 0; u < 4; ++u) v[u] += a[u][w];
  }
  if (r < np) {   // the last, partial round: its loads together as well
    float a[4][8];
#pragma unroll
    for (int w = 0; w < 8; ++w)
#pragma unroll
      for (int u = 0; u < 4; ++u) a[u][w] = s0[u][(size_t)min(r + w, np - 1) * step];
#pragma unroll
    for (int w = 0; w < 8; ++w)
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (r + w < np) v[u] += a[u][w];
  }
}

__device__ __forceinline__ uint32_t node_id_of(const Geom& g, int phase, int cw, int k) {
  const int i = phase == CODENET_PHASE_FWD ? k : cw, j = phase == CODENET_PHASE_FWD ? cw : k;
  return (uint32_t)(i * g.Nn + j);
}

// Which nodes of every codeword are erroneous, into shared memory: s_inj = the nodes whose output the injection
// plan hits or (feedforward) whose own input copy the small-step plan hits; s_out / s_in (may be NULL) tell the two
// kinds apart for the code that builds the working copy.
__device__ void build_hit_masks(const CheckParams& p, const PhaseGeom& q, unsigned long long* s_inj,
                                unsigned long long* s_out = nullptr, unsigned long long* s_in = nullptr) {
  for (int t = threadIdx.x; t < MAXN; t += blockDim.x) {
    s_inj[t] = 0ull;
    if (s_out) s_out[t] = 0ull;
    if (s_in) s_in[t] = 0ull;
  }
  __syncthreads();
  const bool fwd = p.phase == CODENET_PHASE_FWD;
  const bool inputs = fwd && p.small.on && p.small.p_input != 0u && p.dY != nullptr;
  if (p.fault.mode != CODENET_FAULT_NONE || inputs) {
    const uint32_t it = (p.fault.iteration ? *p.fault.iteration : 0u) + p.it_add;
    const uint32_t its = p.small.iteration ? *p.small.iteration : 0u;
    const uint32_t n_active = (uint32_t)(q.n_cw * q.K);
    for (int t = threadIdx.x; t < q.n_cw * q.K; t += blockDim.x) {
      const int cw = t / q.K, k = t % q.K;
      const int i = fwd ? k : cw, j = fwd ? cw : k;
      const uint32_t node_id = (uint32_t)(i * p.g.Nn + j);
      const uint32_t active = fwd ? (uint32_t)(i * p.g.n + j) : node_id;
      if (p.fault.mode != CODENET_FAULT_NONE && node_is_hit(p.fault, (uint32_t)p.phase, it, node_id, active, n_active)) {
        atomicOr(&s_inj[cw], 1ull << k);
        if (s_out) atomicOr(&s_out[cw], 1ull << k);
      }
      if (inputs && small_is_hit(p.small, CODENET_PHASE_INPUT, its, node_id)) {
        atomicOr(&s_inj[cw], 1ull << k);
        if (s_in) atomicOr(&s_in[cw], 1ull << k);
      }
    }
  }
  __syncthreads();
}

// The value of element e of a node output as the checks see it: the product, plus the noise of an erroneous output,
// plus the deviation an erroneous input copy causes (in that order, each one rounding).
__device__ __forceinline__ float with_faults(const CheckParams& p, float v, bool out_hit, bool in_hit, uint32_t key1,
                                             uint32_t it, uint32_t node_id, size_t node_base, size_t e) {
  if (out_hit) v = __fadd_rn(v, hit_noise(p.fault.seed, key1, it, node_id, (uint32_t)e, p.fault.sigma));
  if (in_hit) v = __fadd_rn(v, p.dY[node_base + e]);
  return v;
}

__device__ __forceinline__ float block_max256(float v, float* red) {
  v = warp_max(v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float m = 0.0f;
#pragma unroll
  for (int w = 0; w < CK_WARPS; ++w) m = fmaxf(m, red[w]);
  return m;
}

// Inverse of an s x s matrix (s <= 4), Gaussian elimination with partial pivoting, in double.
__device__ bool invert_small(int s, const double* A, double* inv) {
  double a[MAXR][2 * MAXR];
  for (int r = 0; r < s; ++r)
    for (int c = 0; c < s; ++c) {
      a[r][c] = A[r * s + c];
      a[r][s + c] = r == c ? 1.0 : 0.0;
    }
  for (int pv = 0; pv < s; ++pv) {
    int best = pv;
    for (int r = pv + 1; r < s; ++r)
      if (fabs(a[r][pv]) > fabs(a[best][pv])) best = r;
    if (a[best][pv] == 0.0) return false;
    if (best != pv)
      for (int c = 0; c < 2 * s; ++c) {
        const double t = a[pv][c]; a[pv][c] = a[best][c]; a[best][c] = t;
      }
    const double piv = a[pv][pv];
    for (int c = 0; c < 2 * s; ++c) a[pv][c] /= piv;
    for (int r = 0; r < s; ++r) {
      if (r == pv) continue;
      const double f = a[r][pv];
      if (f == 0.0) continue;
      for (int c = 0; c < 2 * s; ++c) a[r][c] -= f * a[pv][c];
    }
  }
  for (int r = 0; r < s; ++r)
    for (int c = 0; c < s; ++c) inv[r * s + c] = a[r][s + c];
  return true;
}

// The outputs of one codeword as the checks see them.  Small batches copy every node output into the
// working copy; large batches copy only the nodes the injection plan hits (the others are read where
// the product kernel left them), so `own` says which nodes live in the working copy.
struct CwView {
  const float* yw;          // working copy of the codeword
  const float* ys;          // clean source of the codeword (same layout)
  unsigned long long own;   // bit k: node k is read from the working copy
  __device__ __forceinline__ float at(const PhaseGeom& q, int k, size_t e) const {
    return (((own >> k) & 1ull) ? yw : ys)[(size_t)k * q.n_el + e];
  }
  // four consecutive elements (e a multiple of four; large batches: the buffers are 16-byte aligned)
  __device__ __forceinline__ float4 at4(const PhaseGeom& q, int k, size_t e) const {
    return *reinterpret_cast<const float4*>((((own >> k) & 1ull) ? yw : ys) + (size_t)k * q.n_el + e);
  }
};

__device__ __forceinline__ bool lazy_copy(const CheckParams& p) {
  return p.lazy != 0;   // decided on the host: large batch, node outputs read in place, 16-byte aligned buffers
}

__device__ __forceinline__ CwView cw_view(const CheckParams& p, const PhaseGeom& q, const unsigned long long* s_inj,
                                          int cw) {
  CwView v;
  v.yw = p.Yw + (size_t)cw * q.K * q.n_el;
  if (lazy_copy(p)) { v.ys = p.src + (size_t)cw * q.K * q.n_el; v.own = s_inj[cw]; }
  else { v.ys = v.yw; v.own = ~0ull; }
  return v;
}

// Syndrome of one element: syn[q] = sum_k P[k,q] out_k - out_{kd+q}.
__device__ __forceinline__ void syndrome_at(const CwView& yw, const PhaseGeom& q, const float* sP, size_t e,
                                            float (&syn)[MAXR]) {
#pragma unroll
  for (int t = 0; t < MAXR; ++t) syn[t] = t < q.r ? -yw.at(q, q.kd + t, e) : 0.0f;
  for (int k = 0; k < q.kd; ++k) {
    const float o = yw.at(q, k, e);
#pragma unroll
    for (int t = 0; t < MAXR; ++t)
      if (t < q.r) syn[t] = fmaf(sP[k * q.r + t], o, syn[t]);
  }
}

// Erasure decoding of one element under a plan: the located data outputs are solved from the
// lowest-indexed unlocated parities; par[] receives every parity re-encoded from the result.
__device__ __forceinline__ void decode_at(const CwView& yw, const PhaseGeom& q, const float* sP, const CwPlan& pl,
                                          size_t e, float (&fix)[MAXR], double (&par)[MAXR]) {
  // the plan's fields once, into registers (the plan sits in global memory and is the same for every element)
  const unsigned long long F = pl.F;
  const int nfd = pl.nfd;
  int qa[MAXR], fda[MAXR];
#pragma unroll
  for (int a = 0; a < MAXR; ++a) { qa[a] = a < nfd ? pl.q[a] : 0; fda[a] = a < nfd ? pl.fd[a] : 0; }
  double rhs[MAXR];
#pragma unroll
  for (int a = 0; a < MAXR; ++a) rhs[a] = a < nfd ? (double)yw.at(q, q.kd + qa[a], e) : 0.0;
#pragma unroll
  for (int t = 0; t < MAXR; ++t) par[t] = 0.0;
  // node outputs eight at a time (independent loads, in flight together), used in node order
  for (int k0 = 0; k0 < q.kd; k0 += 8) {
    float o8[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) o8[u] = yw.at(q, min(k0 + u, q.kd - 1), e);
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int k = k0 + u;
      if (k >= q.kd || ((F >> k) & 1ull)) continue;
      const double o = (double)o8[u];
#pragma unroll
      for (int a = 0; a < MAXR; ++a)
        if (a < nfd) rhs[a] -= (double)sP[k * q.r + qa[a]] * o;
#pragma unroll
      for (int t = 0; t < MAXR; ++t)
        if (t < q.r) par[t] += (double)sP[k * q.r + t] * o;
    }
  }
#pragma unroll
  for (int a = 0; a < MAXR; ++a) {
    double acc = 0.0;
#pragma unroll
    for (int b = 0; b < MAXR; ++b)
      if (a < nfd && b < nfd) acc += pl.ainv[a * nfd + b] * rhs[b];
    fix[a] = (float)acc;
  }
#pragma unroll
  for (int a = 0; a < MAXR; ++a)
    if (a < nfd) {
#pragma unroll
      for (int t = 0; t < MAXR; ++t)
        if (t < q.r) par[t] += (double)sP[fda[a] * q.r + t] * (double)fix[a];
    }
}

// decode_at for a plan with ONE located data node and at most two parities, four consecutive elements at a time
// (large batches): per element the same operations in the same order, with 16-byte loads and a quarter of the
// instructions.  PAR: also re-encode the parities (for the verification on a spare one).
template <bool PAR>
__device__ __forceinline__ void decode1_at4(const CwView& yw, const PhaseGeom& q, const float* sP, const CwPlan& pl,
                                            size_t e, float (&fix)[4], double (&par)[2][4]) {
  const unsigned long long F = pl.F;
  const int qa = pl.q[0], fd = pl.fd[0];
  const float4 r4 = yw.at4(q, q.kd + qa, e);
  double rhs[4] = {(double)r4.x, (double)r4.y, (double)r4.z, (double)r4.w};
#pragma unroll
  for (int t = 0; t < 2; ++t)
#pragma unroll
    for (int c = 0; c < 4; ++c) par[t][c] = 0.0;
#pragma unroll 1
  for (int k0 = 0; k0 < q.kd; k0 += 8) {
    float4 o8[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) o8[u] = yw.at4(q, min(k0 + u, q.kd - 1), e);
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int k = k0 + u;
      if (k >= q.kd || ((F >> k) & 1ull)) continue;
      const double o[4] = {(double)o8[u].x, (double)o8[u].y, (double)o8[u].z, (double)o8[u].w};
      const double pq = (double)sP[k * q.r + qa];
#pragma unroll
      for (int c = 0; c < 4; ++c) rhs[c] -= pq * o[c];
      if (PAR) {
#pragma unroll
        for (int t = 0; t < 2; ++t)
          if (t < q.r) {
            const double pt = (double)sP[k * q.r + t];
#pragma unroll
            for (int c = 0; c < 4; ++c) par[t][c] += pt * o[c];
          }
      }
    }
  }
  const double ainv = pl.ainv[0];
#pragma unroll
  for (int c = 0; c < 4; ++c) fix[c] = (float)(ainv * rhs[c]);
  if (PAR) {
#pragma unroll
    for (int t = 0; t < 2; ++t)
      if (t < q.r) {
        const double pt = (double)sP[fd * q.r + t];
#pragma unroll
        for (int c = 0; c < 4; ++c) par[t][c] += pt * (double)fix[c];
      }
  }
}

// Report from the per-codeword plans; called by every thread of one CTA (>= 64 threads).
// s_a / s_b: two shared float arrays of MAXN entries used as scratch.
__device__ void write_report(const CheckParams& p, int n_cw, const unsigned* final_state, float* s_a, float* s_b) {
  __shared__ unsigned s_cnt[4];
  __shared__ unsigned long long s_dmask;
  codenet_report_t* rep = p.rep;
  const int cw = threadIdx.x;
  if (cw < 4) s_cnt[cw] = 0u;
  if (cw == 0) s_dmask = 0ull;
  __syncthreads();
  if (cw < MAXN) {
    float mn = FLT_MAX, mx = 0.0f;
    if (cw < n_cw) {
      const volatile CwPlan& pl = p.plan[cw];  // written by other CTAs of this grid
      const int state = final_state ? (int)final_state[cw] : pl.state;
      uint32_t outcome = CODENET_CLEAN;
      if (state == 1) outcome = CODENET_CORRECTED;
      else if (state == 3) outcome = p.have_clean ? CODENET_FALLBACK : CODENET_FAILED;
      else if (state == 4) outcome = CODENET_DISAGREE;
      const unsigned long long F = pl.F;
      rep->flagged_mask[cw] = pl.detected ? F : 0ull;
      rep->injected_mask[cw] = pl.injected;
      if (pl.detected) {
        atomicOr(&s_dmask, 1ull << cw);
        atomicAdd(&s_cnt[0], 1u);
        atomicAdd(&s_cnt[1], (unsigned)__popcll(F));
      }
      if (state == 3) atomicAdd(&s_cnt[2], 1u);
      atomicMax(&s_cnt[3], outcome);
      mn = pl.min_hit;
      mx = pl.max_clean;
    } else {
      rep->flagged_mask[cw] = 0;
      rep->injected_mask[cw] = 0;
    }
    s_a[cw] = mn;
    s_b[cw] = mx;
  }
  __syncthreads();
  if (cw == 0) {
    float mn = FLT_MAX, mx = 0.0f;
    for (int k = 0; k < MAXN; ++k) { mn = fminf(mn, s_a[k]); mx = fmaxf(mx, s_b[k]); }
    rep->status = (p.tc_flag && *p.tc_flag) ? (uint32_t)CODENET_TIMEOUT : s_cnt[3];
    rep->n_detected_cw = s_cnt[0];
    rep->n_flagged_nodes = s_cnt[1];
    rep->n_fallback_cw = s_cnt[2];
    rep->detected_mask = s_dmask;
    rep->min_margin_hit = mn;
    rep->max_margin_clean = mx;
  }
  __syncthreads();
}

// Sum over codewords of the data-node outputs: s_i = sum_j y_ij (forward), c_j = sum_i z_ij (backward).
__device__ __forceinline__ void output_index(const Geom& g, bool fwd, int gidx, int* node, int* pos) {
  const int len = fwd ? g.b_r : g.b_c;
  *node = gidx / len;
  *pos = gidx % len;
}


// Value of data node `node` of codeword `cw` at element e after decoding / fallback (plans: a copy in shared memory).
__device__ __forceinline__ float final_value(const CheckParams& p, const PhaseGeom& q, const float* sP,
                                             const unsigned long long* s_inj, const unsigned* s_final,
                                             const CwPlan* plans, int cw, int node, size_t e) {
  const CwView yw = cw_view(p, q, s_inj, cw);
  const int state = (int)s_final[cw];
  if (state == 0 || state == 4) return yw.at(q, node, e);   // (4: the verification steps disagreed: left as it is)
  if (state == 1) {
    const CwPlan& pl = plans[cw];
    if (!((pl.F >> node) & 1ull)) return yw.at(q, node, e);
    if (pl.nfd == 1) {
      // One located data node, the usual case, in few instructions (this code runs once in a while, so what it costs
      // is the fetching of its instructions): the same operations in the same order as the general decoding below.
      const unsigned long long F = pl.F;
      const int qa = pl.q[0];
      double rhs = (double)yw.at(q, q.kd + qa, e);
#pragma unroll 1
      for (int k0 = 0; k0 < q.kd; k0 += 8) {
        float o8[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) o8[u] = yw.at(q, min(k0 + u, q.kd - 1), e);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int k = k0 + u;
          if (k >= q.kd || ((F >> k) & 1ull)) continue;
          rhs -= (double)sP[k * q.r + qa] * (double)o8[u];
        }
      }
      return (float)(pl.ainv[0] * rhs);
    }
    float fix[MAXR];
    double par[MAXR];
    decode_at(yw, q, sP, pl, e, fix, par);
    float v = 0.0f;
#pragma unroll
    for (int a = 0; a < MAXR; ++a)
      if (a < pl.nfd && pl.fd[a] == node) v = fix[a];
    return v;
  }
  // uncorrectable: the fault-free recomputation, when there is one
  if (p.have_clean && ((s_inj[cw] >> node) & 1ull)) return clean_value(p, q, cw, node, e);
  return yw.at(q, node, e);
}

// Sum over the codewords of one output (data node `node`, element e) with final values, in codeword order.  The values
// of the codewords whose plan does not touch the node (the many) are plain loads, sixteen at a time so that they are in
// flight together; the loads of a touched codeword's decoding follow them at once (the plan sits in shared memory, so
// nothing they need is still on its way).  s_touch[c] holds the nodes codeword c's final plan replaces (decoded or
// fault-free).
__device__ __forceinline__ float sum_final_values(const CheckParams& p, const PhaseGeom& q, const float* sP,
                                                  const unsigned long long* s_inj, const unsigned* s_final,
                                                  const unsigned long long* s_touch, const CwPlan* plans, int node,
                                                  size_t e) {
  float acc = 0.0f;
  for (int c0 = 0; c0 < q.n_cw; c0 += 16) {
    float v[16];
    if (!lazy_copy(p)) {
      // every node output sits in the working copy: one base and one stride (few instructions: see final_value)
      const float* base = p.Yw + (size_t)node * q.n_el + e;
      const size_t stride = (size_t)q.K * q.n_el;
#pragma unroll
      for (int u = 0; u < 16; ++u) v[u] = base[(size_t)min(c0 + u, q.n_cw - 1) * stride];
    } else {
#pragma unroll
      for (int u = 0; u < 16; ++u) {
        const int c = min(c0 + u, q.n_cw - 1);
        v[u] = cw_view(p, q, s_inj, c).at(q, node, e);
      }
    }
#pragma unroll 1
    for (int c = c0; c < min(c0 + 16, q.n_cw); ++c) {
      if (!((s_touch[c] >> node) & 1ull)) continue;
      const float d = final_value(p, q, sP, s_inj, s_final, plans, c, node, e);
#pragma unroll
      for (int u = 0; u < 16; ++u) v[u] = (c0 + u == c) ? d : v[u];
    }
#pragma unroll
    for (int u = 0; u < 16; ++u)
      if (c0 + u < q.n_cw) acc += v[u];
  }
  return acc;
}

// sum_final_values for four consecutive elements of a large batch (e a multiple of four): 16-byte loads, eight
// codewords in flight; a touched codeword whose plan has one located data node is decoded four elements at a time,
// any other one element by element.  Per element the additions run in codeword order, as above.
__device__ __forceinline__ void sum_final_values4(const CheckParams& p, const PhaseGeom& q, const float* sP,
                                                  const unsigned long long* s_inj, const unsigned* s_final,
                                                  const unsigned long long* s_touch, const CwPlan* plans, int node,
                                                  size_t e, float (&acc)[4]) {
#pragma unroll
  for (int c = 0; c < 4; ++c) acc[c] = 0.0f;
  for (int c0 = 0; c0 < q.n_cw; c0 += 8) {
    float4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) v[u] = cw_view(p, q, s_inj, min(c0 + u, q.n_cw - 1)).at4(q, node, e);
#pragma unroll 1
    for (int cw = c0; cw < min(c0 + 8, q.n_cw); ++cw) {
      if (!((s_touch[cw] >> node) & 1ull)) continue;
      float d[4];
      const CwPlan& pl = plans[cw];
      if (s_final[cw] == 1u && pl.nfd == 1 && pl.fd[0] == node) {
        double par[2][4];
        decode1_at4<false>(cw_view(p, q, s_inj, cw), q, sP, pl, e, d, par);
      } else {
#pragma unroll 1
        for (int c = 0; c < 4; ++c) d[c] = final_value(p, q, sP, s_inj, s_final, plans, cw, node, e + c);
      }
#pragma unroll
      for (int u = 0; u < 8; ++u)
        if (c0 + u == cw) v[u] = make_float4(d[0], d[1], d[2], d[3]);
    }
#pragma unroll
    for (int u = 0; u < 8; ++u)
      if (c0 + u < q.n_cw) { acc[0] += v[u].x; acc[1] += v[u].y; acc[2] += v[u].z; acc[3] += v[u].w; }
  }
}
