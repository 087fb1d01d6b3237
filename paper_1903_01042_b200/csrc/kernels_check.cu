// Around the streaming kernels: initial encoding (Claim 1), additional encoding of the vectors,
// accessors, and the small element-wise steps (activation, loss, step C2).
#include "codenet_internal.cuh"

#include <float.h>

namespace codenet {
namespace {

// -------------------------------------------------------------------------------------------
// Initial encoding: W~_ij = sum_a G_r[a,i] W_aj (parity rows), sum_b G_c[b,j] W_ib (parity
// columns); data blocks are copies.  One thread per stored element (padding columns get 0).
// -------------------------------------------------------------------------------------------
__global__ void encode_layer_kernel(Geom g, const void* __restrict__ W) {
  const size_t total = (size_t)g.Mbr * g.ld;
  for (size_t idx = blockIdx.x * (size_t)blockDim.x + threadIdx.x; idx < total;
       idx += (size_t)gridDim.x * blockDim.x) {
    const int gr = (int)(idx / g.ld), gc = (int)(idx % g.ld);
    const int i = gr / g.b_r, r = gr % g.b_r, j = gc / g.ldb, c = gc % g.ldb;
    if (i >= g.m && j >= g.n) continue;
    // one-off, so the sums are taken in double: the stored parity blocks are then the correctly
    // rounded combinations (in bfloat16 a single rounding the other way is 2^-8 of the element)
    double acc = 0.0;
    if (c < g.b_c) {
      if (i < g.m && j < g.n) {
        const int wr = i * g.b_r + r, wc = j * g.b_c + c;
        if (wr < g.n_out && wc < g.n_in) acc = (double)load_elem(W, g.dtype, (size_t)wr * g.n_in + wc);
      } else if (i >= g.m) {
        const int wc = j * g.b_c + c;
        for (int a = 0; a < g.m; ++a) {
          const int wr = a * g.b_r + r;
          if (wr < g.n_out && wc < g.n_in)
            acc += (double)g.Pr[a * g.r_row + (i - g.m)] * (double)load_elem(W, g.dtype, (size_t)wr * g.n_in + wc);
        }
      } else {
        const int wr = i * g.b_r + r;
        for (int b = 0; b < g.n; ++b) {
          const int wc = b * g.b_c + c;
          if (wr < g.n_out && wc < g.n_in)
            acc += (double)g.Pc[b * g.r_col + (j - g.n)] * (double)load_elem(W, g.dtype, (size_t)wr * g.n_in + wc);
        }
      }
    }
    store_elem(g.Wt, g.dtype, idx, (float)acc);
  }
}

// Inner checksums of the stored blocks: u = column sums per slice of T rows, v = row sums.
// only_blk >= 0: the checksums of that block alone (regeneration), otherwise of every block (initial encoding).
__global__ void checksum_kernel(Geom g, int only_blk) {
  const size_t nu = (size_t)g.M * g.Nn * g.ns * g.ldb;
  const size_t nv = (size_t)g.M * g.Nn * g.nsc * g.b_r;
  const size_t per_u = (size_t)g.ns * g.ldb, per_v = (size_t)g.nsc * g.b_r;
  const size_t count = only_blk >= 0 ? per_u + per_v : nu + nv;
  for (size_t it = blockIdx.x * (size_t)blockDim.x + threadIdx.x; it < count; it += (size_t)gridDim.x * blockDim.x) {
    // position in the full index space (all u entries, then all v entries)
    const size_t idx = only_blk < 0 ? it
                       : (it < per_u ? (size_t)only_blk * per_u + it : nu + (size_t)only_blk * per_v + (it - per_u));
    if (idx < nu) {
      const int c = (int)(idx % g.ldb);
      const size_t t = idx / g.ldb;
      const int s = (int)(t % g.ns), blk = (int)(t / g.ns);
      const int i = blk / g.Nn, j = blk % g.Nn;
      double acc = 0.0;
      if (!(i >= g.m && j >= g.n) && c < g.b_c)
        for (int rr = 0; rr < g.T; ++rr)
          acc += (double)load_elem(g.Wt, g.dtype, ((size_t)i * g.b_r + s * g.T + rr) * g.ld + (size_t)j * g.ldb + c);
      g.U[idx] = (float)acc;
    } else {
      const size_t t = idx - nu;
      const int rr = (int)(t % g.b_r);
      const size_t t2 = t / g.b_r;
      const int s = (int)(t2 % g.nsc), blk = (int)(t2 / g.nsc);
      const int i = blk / g.Nn, j = blk % g.Nn;
      double acc = 0.0;
      if (!(i >= g.m && j >= g.n))
        for (int c = s * g.Tc; c < (s + 1) * g.Tc; ++c)
          acc += (double)load_elem(g.Wt, g.dtype, ((size_t)i * g.b_r + rr) * g.ld + (size_t)j * g.ldb + c);
      g.V[t] = (float)acc;
    }
  }
}

// -------------------------------------------------------------------------------------------
// Additional encoding of the vectors (Step 4 of the feedforward / backpropagation stages):
// x~_j = sum_b G_c[b,j] x_b, delta~_i = sum_a G_r[a,i] delta_a, plus the sums the inner
// checksums need.  One CTA per segment: (x, j, b) of length ldb or (delta, i, slice, b) of length T.
// -------------------------------------------------------------------------------------------
#include "encode_device.cuh"

// One CTA per segment: (x, j, b) of length ldb or (delta, i, slice, b) of length T.
__global__ void __launch_bounds__(128) encode_vectors_kernel(Geom g, EncodeArgs ea) {
  encode_vectors_body(g, ea, blockIdx.x, gridDim.x);
}

// -------------------------------------------------------------------------------------------
// small utilities
// -------------------------------------------------------------------------------------------
__global__ void decode_weights_kernel(Geom g, void* __restrict__ out) {
  const size_t total = (size_t)g.n_out * g.n_in;
  for (size_t idx = blockIdx.x * (size_t)blockDim.x + threadIdx.x; idx < total;
       idx += (size_t)gridDim.x * blockDim.x) {
    const int wr = (int)(idx / g.n_in), wc = (int)(idx % g.n_in);
    const int j = wc / g.b_c, c = wc % g.b_c;
    store_elem(out, g.dtype, idx, load_elem(g.Wt, g.dtype, (size_t)wr * g.ld + (size_t)j * g.ldb + c));
  }
}

__global__ void get_block_kernel(Geom g, int i, int j, float* __restrict__ out) {
  const size_t total = (size_t)g.b_r * g.b_c;
  for (size_t idx = blockIdx.x * (size_t)blockDim.x + threadIdx.x; idx < total;
       idx += (size_t)gridDim.x * blockDim.x) {
    const int rr = (int)(idx / g.b_c), c = (int)(idx % g.b_c);
    out[idx] = load_elem(g.Wt, g.dtype, ((size_t)i * g.b_r + rr) * g.ld + (size_t)j * g.ldb + c);
  }
}

// -------------------------------------------------------------------------------------------
// Faults in the stored blocks (Section "Experimental Results": a sparse matrix added to a node's
// stored sub-matrix) and regeneration of a block from the code of its block-column or block-row
// (the "regenerate" step of the feedforward stage).
// -------------------------------------------------------------------------------------------

// Element e = row * b_c + col of block (i, j) changes when word 0 of Philox(counter = (iteration,
// node, e, 3), key = (seed, layer << 8 | 2)) is below density_q32; amplitude * u is added, u uniform
// on [-1, 1) from the upper 24 bits of word 1.  Integer until the last product and sum, each a single
// rounding, so that every implementation of this rule changes the same elements by the same bits.
__global__ void corrupt_block_kernel(Geom g, int i, int j, uint32_t seed, uint32_t layer, uint32_t iteration,
                                     uint32_t density_q32, float amplitude) {
  const size_t total = (size_t)g.b_r * g.b_c;
  const uint32_t node_id = (uint32_t)(i * g.Nn + j), key1 = (layer << 8) | 2u;
  for (size_t idx = blockIdx.x * (size_t)blockDim.x + threadIdx.x; idx < total;
       idx += (size_t)gridDim.x * blockDim.x) {
    uint32_t o[4];
    philox4x32_10(iteration, node_id, (uint32_t)idx, 3u, seed, key1, o);
    if (o[0] >= density_q32) continue;
    const int rr = (int)(idx / g.b_c), c = (int)(idx % g.b_c);
    const size_t at = ((size_t)i * g.b_r + rr) * g.ld + (size_t)j * g.ldb + c;
    const float unit = __fsub_rn(__fmul_rn((float)(o[1] >> 8), 1.0f / 8388608.0f), 1.0f);
    store_elem(g.Wt, g.dtype, at, __fadd_rn(load_elem(g.Wt, g.dtype, at), __fmul_rn(amplitude, unit)));
  }
}

// Block (i, j) as the code combination of the other blocks of its block-column (along = 0, code G_r)
// or block-row (along = 1, code G_c): a parity block is re-encoded, a data block is solved from the
// lowest-indexed parity whose generator entry is not zero.  One 16-byte group per thread and step,
// every source read once, sums in double in source order, one rounding to the storage type.
template <typename T>
__global__ void __launch_bounds__(256) regenerate_block_kernel(Geom g, int i, int j, int along, int* status) {
  constexpr int VEC = Vec16<T>::N;
  __shared__ double s_coef[CODENET_MAX_NODES];
  __shared__ int s_use[CODENET_MAX_NODES], s_n;
  const int kd = along == 0 ? g.m : g.n, r = along == 0 ? g.r_row : g.r_col, pos = along == 0 ? i : j;
  const float* P = along == 0 ? g.Pr : g.Pc;
  if (threadIdx.x == 0) {
    int n_use = 0;
    if (pos >= kd) {
      for (int k = 0; k < kd; ++k) { s_use[n_use] = k; s_coef[n_use++] = (double)P[k * r + (pos - kd)]; }
    } else {
      int q = -1;
      for (int t = 0; t < r && q < 0; ++t)
        if (P[pos * r + t] != 0.0f) q = t;
      if (q >= 0) {
        const double inv = 1.0 / (double)P[pos * r + q];
        for (int k = 0; k < kd; ++k)
          if (k != pos) { s_use[n_use] = k; s_coef[n_use++] = __dmul_rn(-(double)P[k * r + q], inv); }
        s_use[n_use] = kd + q; s_coef[n_use++] = inv;
      } else if (blockIdx.x == 0 && status != nullptr) {
        *status = 1;   // no parity of this direction involves the block
      }
    }
    s_n = n_use;
  }
  __syncthreads();
  const int n_use = s_n;
  if (n_use == 0) return;
  T* W = reinterpret_cast<T*>(g.Wt);
  const int groups = g.ldb / VEC;                         // the padding columns are rebuilt too (zeros)
  const size_t total = (size_t)g.b_r * groups;
  for (size_t idx = blockIdx.x * (size_t)blockDim.x + threadIdx.x; idx < total;
       idx += (size_t)gridDim.x * blockDim.x) {
    const int rr = (int)(idx / groups), cg = (int)(idx % groups);
    double acc[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) acc[v] = 0.0;
    for (int t0 = 0; t0 < n_use; t0 += 4) {   // four sources in flight, added in source order
      float f[4][VEC];
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const int t = min(t0 + w, n_use - 1);
        const int bi = along == 0 ? s_use[t] : i, bj = along == 0 ? j : s_use[t];
        Vec16<T>::load(W + ((size_t)bi * g.b_r + rr) * g.ld + (size_t)bj * g.ldb + (size_t)cg * VEC, f[w]);
      }
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        if (t0 + w >= n_use) continue;
        const double c = s_coef[t0 + w];
#pragma unroll
        for (int v = 0; v < VEC; ++v) acc[v] = __dadd_rn(acc[v], __dmul_rn(c, (double)f[w][v]));
      }
    }
    float o[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) o[v] = (float)acc[v];
    Vec16<T>::store(W + ((size_t)i * g.b_r + rr) * g.ld + (size_t)j * g.ldb + (size_t)cg * VEC, o);
  }
}

// scratch[0] = max |stored - re-encoded| style ratios are formed per block: one CTA per stored
// block computes dev and ref maxima, then an atomicMax on the ratio bits.
__global__ void __launch_bounds__(256) invariance_kernel(Geom g, unsigned* __restrict__ out_bits) {
  __shared__ float red_dev[8], red_ref[8];
  const int blk = blockIdx.x;
  const int i = blk / g.Nn, j = blk % g.Nn;
  if (i >= g.m && j >= g.n) return;
  for (int what = 0; what < (keeps_checksums(g) ? 3 : 1); ++what) {   // checksums only where they are kept valid
    float dev = 0.0f, ref = 0.0f;
    if (what == 0) {
      if (i < g.m && j < g.n) continue;
      for (int idx = threadIdx.x; idx < g.b_r * g.b_c; idx += blockDim.x) {
        const int rr = idx / g.b_c, c = idx % g.b_c;
        double acc = 0.0;
        if (i >= g.m)
          for (int a = 0; a < g.m; ++a)
            acc += (double)g.Pr[a * g.r_row + (i - g.m)] *
                   (double)load_elem(g.Wt, g.dtype, ((size_t)a * g.b_r + rr) * g.ld + (size_t)j * g.ldb + c);
        else
          for (int b = 0; b < g.n; ++b)
            acc += (double)g.Pc[b * g.r_col + (j - g.n)] *
                   (double)load_elem(g.Wt, g.dtype, ((size_t)i * g.b_r + rr) * g.ld + (size_t)b * g.ldb + c);
        const float st = load_elem(g.Wt, g.dtype, ((size_t)i * g.b_r + rr) * g.ld + (size_t)j * g.ldb + c);
        dev = fmaxf(dev, (float)fabs(acc - (double)st));
        ref = fmaxf(ref, (float)fabs(acc));
      }
    } else if (what == 1) {
      for (int idx = threadIdx.x; idx < g.ns * g.b_c; idx += blockDim.x) {
        const int s = idx / g.b_c, c = idx % g.b_c;
        double acc = 0.0;
        for (int rr = 0; rr < g.T; ++rr)
          acc += (double)load_elem(g.Wt, g.dtype, ((size_t)i * g.b_r + s * g.T + rr) * g.ld + (size_t)j * g.ldb + c);
        dev = fmaxf(dev, (float)fabs(acc - (double)g.U[((size_t)blk * g.ns + s) * g.ldb + c]));
        ref = fmaxf(ref, (float)fabs(acc));
      }
    } else {
      for (int idx = threadIdx.x; idx < g.nsc * g.b_r; idx += blockDim.x) {
        const int s = idx / g.b_r, rr = idx % g.b_r;
        double acc = 0.0;
        for (int c = s * g.Tc; c < (s + 1) * g.Tc; ++c)
          acc += (double)load_elem(g.Wt, g.dtype, ((size_t)i * g.b_r + rr) * g.ld + (size_t)j * g.ldb + c);
        dev = fmaxf(dev, (float)fabs(acc - (double)g.V[((size_t)blk * g.nsc + s) * g.b_r + rr]));
        ref = fmaxf(ref, (float)fabs(acc));
      }
    }
    dev = warp_max(dev); ref = warp_max(ref);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) { red_dev[threadIdx.x >> 5] = dev; red_ref[threadIdx.x >> 5] = ref; }
    __syncthreads();
    if (threadIdx.x == 0) {
      float d = 0.0f, rf = 0.0f;
      for (int w = 0; w < 8; ++w) { d = fmaxf(d, red_dev[w]); rf = fmaxf(rf, red_ref[w]); }
      if (rf > 0.0f) atomicMax(out_bits, __float_as_uint(d / rf));
    }
  }
}

__global__ void activation_kernel(float* __restrict__ x, size_t n, int act) {
  for (size_t idx = blockIdx.x * (size_t)blockDim.x + threadIdx.x; idx < n; idx += (size_t)gridDim.x * blockDim.x)
    if (act == CODENET_ACT_RELU && x[idx] < 0.0f) x[idx] = 0.0f;
}

// Step C2: delta^{l-1} = c^l (.) g(x^l); for ReLU g(x) = [x > 0].
__global__ void mask_delta_kernel(float* __restrict__ C, const float* __restrict__ x, size_t n, int act) {
  for (size_t idx = blockIdx.x * (size_t)blockDim.x + threadIdx.x; idx < n; idx += (size_t)gridDim.x * blockDim.x)
    if (act == CODENET_ACT_RELU && !(x[idx] > 0.0f)) C[idx] = 0.0f;
}

// Loss and delta^L = -d loss / d s^L.  The squared-error loss is spread over CTAs; every CTA leaves
// one partial sum, and the last one to finish adds them up in index order (same result every run).
constexpr int LOSS_THREADS = 256;
constexpr int LOSS_MAX_BLOCKS = 512;
__global__ void __launch_bounds__(LOSS_THREADS)
loss_kernel(const float* __restrict__ S, const void* __restrict__ target, int B, int n, int loss,
            float* __restrict__ delta, float* __restrict__ loss_out, float* __restrict__ partials,
            unsigned* __restrict__ counter) {
  __shared__ float red[LOSS_THREADS / 32];
  __shared__ int s_last;
  float part = 0.0f;
  if (loss == CODENET_LOSS_MSE_MEAN) {
    const float* y = reinterpret_cast<const float*>(target);
    const float scale = 1.0f / ((float)n * (float)B);
    const size_t total = (size_t)B * n;
    if ((total & 3) == 0 && ((reinterpret_cast<uintptr_t>(y) | reinterpret_cast<uintptr_t>(S) |
                              reinterpret_cast<uintptr_t>(delta)) & 15) == 0) {
      // four entries per thread and step, four steps in flight
#pragma unroll 4
      for (size_t q = blockIdx.x * (size_t)LOSS_THREADS + threadIdx.x; q < total / 4; q += (size_t)gridDim.x * LOSS_THREADS) {
        const float4 yv = reinterpret_cast<const float4*>(y)[q], sv = reinterpret_cast<const float4*>(S)[q];
        const float d0 = yv.x - sv.x, d1 = yv.y - sv.y, d2 = yv.z - sv.z, d3 = yv.w - sv.w;
        part = fmaf(d0 * d0, scale, part); part = fmaf(d1 * d1, scale, part);
        part = fmaf(d2 * d2, scale, part); part = fmaf(d3 * d3, scale, part);
        reinterpret_cast<float4*>(delta)[q] = make_float4(2.0f * d0 * scale, 2.0f * d1 * scale, 2.0f * d2 * scale, 2.0f * d3 * scale);
      }
    } else {
#pragma unroll 4
      for (size_t e = blockIdx.x * (size_t)LOSS_THREADS + threadIdx.x; e < total; e += (size_t)gridDim.x * LOSS_THREADS) {
        const float d = y[e] - S[e];
        part = fmaf(d * d, scale, part);
        delta[e] = 2.0f * d * scale;
      }
    }
  } else {
    const int* lab = reinterpret_cast<const int*>(target);
    for (int b = blockIdx.x * LOSS_THREADS + threadIdx.x; b < B; b += gridDim.x * LOSS_THREADS) {
      const float* s = S + (size_t)b * n;
      float mx = -FLT_MAX, den = 0.0f;
      for (int k = 0; k < n; ++k) mx = fmaxf(mx, s[k]);
      for (int k = 0; k < n; ++k) den += expf(s[k] - mx);
      for (int k = 0; k < n; ++k) {
        const float pk = expf(s[k] - mx) / den;
        delta[(size_t)b * n + k] = ((k == lab[b] ? 1.0f : 0.0f) - pk) / (float)B;
        if (k == lab[b]) part += -logf(pk) / (float)B;
      }
    }
  }
  part = warp_sum(part);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = part;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.0f;
    for (int w = 0; w < LOSS_THREADS / 32; ++w) t += red[w];
    partials[blockIdx.x] = t;
    __threadfence();
    s_last = atomicAdd(counter, 1u) == gridDim.x - 1 ? 1 : 0;
  }
  __syncthreads();
  if (s_last) {
    // the last CTA to finish adds the partials: every thread takes two of them (at most 512 CTAs), then a
    // fixed tree over the warp and over the eight warps -- the same order every run
    __threadfence();
    float t = 0.0f;
    if (threadIdx.x < gridDim.x) t = __ldcg(&partials[threadIdx.x]);
    if (threadIdx.x + LOSS_THREADS < gridDim.x) t += __ldcg(&partials[threadIdx.x + LOSS_THREADS]);
    t = warp_sum(t);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = t;
    __syncthreads();
    if (threadIdx.x == 0) {
      float tot = 0.0f;
      for (int w = 0; w < LOSS_THREADS / 32; ++w) tot += red[w];
      if (loss_out) *loss_out = tot;
      *counter = 0u;  // ready for the next call
    }
  }
}

inline int grid_for(size_t n, int threads) {
  size_t b = (n + threads - 1) / threads;
  if (b > 148 * 16) b = 148 * 16;
  if (b < 1) b = 1;
  return (int)b;
}

}  // namespace

cudaError_t launch_encode_layer(const Geom& g, const void* W, cudaStream_t st) {
  encode_layer_kernel<<<grid_for((size_t)g.Mbr * g.ld, 256), 256, 0, st>>>(g, W);
  const size_t nchk = (size_t)g.M * g.Nn * ((size_t)g.ns * g.ldb + (size_t)g.nsc * g.b_r);
  checksum_kernel<<<grid_for(nchk, 128), 128, 0, st>>>(g, -1);
  count_launch(2);
  return cudaGetLastError();
}

cudaError_t launch_encode_vectors(const codenet_layer_impl& L, const float* X, const float* Delta,
                                  int B, cudaStream_t st, const LossFuse* fuse, int emit, const SmallDev* small,
                                  float* clear, size_t clear_floats) {
  const Geom& g = L.g;
  const int nseg = (X ? g.Nn * g.nsc * B : 0) + (Delta ? g.M * g.ns * B : 0);
  if (nseg == 0) return cudaSuccess;
  LossFuse lf;
  if (fuse) lf = *fuse;
  else { lf.S = nullptr; lf.target = nullptr; lf.delta = nullptr; lf.scale = 0.0f; lf.partials = nullptr; lf.counter = nullptr; lf.loss_out = nullptr; lf.n_part = 0; lf.defer = 0; }
  const bool vec_ok = encode_vec_ok(g, X, Delta, lf.S, lf.target);
  EmitOperands em;
  em.xT = nullptr; em.dT = nullptr; em.xb = nullptr; em.dpair = nullptr; em.dcount = (size_t)B * g.Mbr;
  em.clear = nullptr; em.clear_n16 = 0;
  if (clear != nullptr && (reinterpret_cast<uintptr_t>(clear) & 15u) == 0 && clear_floats % 4 == 0) {
    em.clear = reinterpret_cast<float4*>(clear); em.clear_n16 = clear_floats / 4;
    L.z_cleared = 1;
  }
  L.operands_ready = 0;
  // (the bfloat16 copies move 8 bytes per four entries: padded widths that are multiples of four make them aligned)
  if (emit != 0 && vec_ok && X && Delta && g.ldb % 4 == 0 && g.ld % 4 == 0) {
    if (emit == 1) { em.xT = reinterpret_cast<float*>(L.ws.tc_xT); em.dT = reinterpret_cast<float*>(L.ws.tc_dT); }
    else { em.xb = reinterpret_cast<__nv_bfloat16*>(L.ws.tc_xT); em.dpair = reinterpret_cast<__nv_bfloat16*>(L.ws.tc_d); }
    L.operands_ready = (em.xT || em.xb) ? 1 : 0;
  }
  SmallDev sf = {0, 0, 0, 0, 0, 0, 0.0f, nullptr, 0};
  if (small != nullptr) sf = *small;
  EncodeArgs ea;
  ea.X = X; ea.Delta = Delta; ea.B = B; ea.Xt = L.ws.Xt; ea.Dt = L.ws.Dt; ea.dsum = L.ws.dsum; ea.xsum = L.ws.xsum;
  ea.vec_ok = vec_ok ? 1 : 0; ea.lf = lf; ea.em = em; ea.sf = sf;
  encode_vectors_kernel<<<nseg, 128, 0, st>>>(g, ea);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_decode_weights(const Geom& g, void* W_out, cudaStream_t st) {
  decode_weights_kernel<<<grid_for((size_t)g.n_out * g.n_in, 256), 256, 0, st>>>(g, W_out);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_check_invariance(const Geom& g, float* out, cudaStream_t st) {
  cudaError_t e = cudaMemsetAsync(out, 0, sizeof(float), st);
  if (e != cudaSuccess) return e;
  invariance_kernel<<<g.M * g.Nn, 256, 0, st>>>(g, reinterpret_cast<unsigned*>(out));
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_get_block(const Geom& g, int i, int j, float* out, cudaStream_t st) {
  get_block_kernel<<<grid_for((size_t)g.b_r * g.b_c, 256), 256, 0, st>>>(g, i, j, out);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_get_checksums(const Geom& g, int i, int j, float* u_out, float* v_out, cudaStream_t st) {
  const size_t blk = (size_t)i * g.Nn + j;
  cudaError_t e = cudaSuccess;
  if (u_out)
    e = cudaMemcpy2DAsync(u_out, (size_t)g.b_c * sizeof(float), g.U + blk * g.ns * g.ldb, (size_t)g.ldb * sizeof(float),
                          (size_t)g.b_c * sizeof(float), (size_t)g.ns, cudaMemcpyDeviceToDevice, st);
  if (e == cudaSuccess && v_out)
    e = cudaMemcpyAsync(v_out, g.V + blk * g.nsc * g.b_r, (size_t)g.nsc * g.b_r * sizeof(float),
                        cudaMemcpyDeviceToDevice, st);
  return e;
}

cudaError_t launch_corrupt_block(const Geom& g, int i, int j, uint32_t seed, uint32_t layer, uint32_t iteration,
                                 uint32_t density_q32, float amplitude, cudaStream_t st) {
  corrupt_block_kernel<<<grid_for((size_t)g.b_r * g.b_c, 256), 256, 0, st>>>(g, i, j, seed, layer, iteration,
                                                                               density_q32, amplitude);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_regenerate_block(const Geom& g, int i, int j, int along, int* status_dev, cudaStream_t st) {
  const int vec = g.dtype == CODENET_BF16 ? 8 : 4;
  const size_t groups = (size_t)g.b_r * (g.ldb / vec);
  size_t blocks = (groups + 255) / 256;
  if (blocks > 148 * 8) blocks = 148 * 8;
  if (blocks < 1) blocks = 1;
  ProfileScope scope(CODENET_KERNEL_REGENERATE, st);
  if (g.dtype == CODENET_BF16) regenerate_block_kernel<__nv_bfloat16><<<(int)blocks, 256, 0, st>>>(g, i, j, along, status_dev);
  else regenerate_block_kernel<float><<<(int)blocks, 256, 0, st>>>(g, i, j, along, status_dev);
  // everything the node stored is generated again: its inner checksums follow from the rebuilt block
  checksum_kernel<<<grid_for((size_t)g.ns * g.ldb + (size_t)g.nsc * g.b_r, 128), 128, 0, st>>>(g, i * g.Nn + j);
  count_launch(2);
  return cudaGetLastError();
}

// Streaming copy for checkpoints: 16 bytes per thread and step, eight steps in flight; the last bytes (a
// size that is not a multiple of 16) go word by word.
__global__ void __launch_bounds__(256) copy_bytes_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst,
                                                         size_t n16, size_t bytes) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
  for (; i + 7 * stride < n16; i += 8 * stride) {
    uint4 a[8];
#pragma unroll
    for (int w = 0; w < 8; ++w) a[w] = __ldcs(src + i + w * stride);   // streamed: read once, written once
#pragma unroll
    for (int w = 0; w < 8; ++w) __stcs(dst + i + w * stride, a[w]);
  }
  for (; i < n16; i += stride) dst[i] = src[i];
  if (blockIdx.x == 0) {
    const unsigned char* s8 = reinterpret_cast<const unsigned char*>(src);
    unsigned char* d8 = reinterpret_cast<unsigned char*>(dst);
    for (size_t t = n16 * 16 + threadIdx.x; t < bytes; t += blockDim.x) d8[t] = s8[t];
  }
}

cudaError_t launch_copy_bytes(const void* src, void* dst, size_t bytes, cudaStream_t st) {
  const size_t n16 = bytes / 16;
  size_t blocks = (n16 + 8 * 256 - 1) / (8 * 256);
  if (blocks > 148 * 8) blocks = 148 * 8;
  if (blocks < 1) blocks = 1;
  copy_bytes_kernel<<<(int)blocks, 256, 0, st>>>(reinterpret_cast<const uint4*>(src), reinterpret_cast<uint4*>(dst), n16, bytes);
  count_launch();
  return cudaGetLastError();
}

__global__ void bump_counter_kernel(uint32_t* counter) { *counter += 1u; }

// The loss from its partial sums, in the order the vector-encoding kernel uses when it adds them up itself.
__global__ void __launch_bounds__(128) sum_loss_partials_kernel(const float* __restrict__ partials, int n, float* out) {
  __shared__ float red[4];
  float t = 0.0f;
  for (int idx = threadIdx.x; idx < n; idx += 128) t += partials[idx];
  t = warp_sum(t);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = t;
  __syncthreads();
  if (threadIdx.x == 0) *out = red[0] + red[1] + red[2] + red[3];
}

cudaError_t launch_sum_loss_partials(const float* partials, int n, float* out, cudaStream_t st) {
  sum_loss_partials_kernel<<<1, 128, 0, st>>>(partials, n, out);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_bump_counter(uint32_t* counter, cudaStream_t st) {
  bump_counter_kernel<<<1, 1, 0, st>>>(counter);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_activation(float* x, size_t n, int act, cudaStream_t st) {
  if (act == CODENET_ACT_IDENTITY) return cudaSuccess;
  activation_kernel<<<grid_for(n, 256), 256, 0, st>>>(x, n, act);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_mask_delta(float* C, const float* x, size_t n, int act, cudaStream_t st) {
  if (act == CODENET_ACT_IDENTITY) return cudaSuccess;
  mask_delta_kernel<<<grid_for(n, 256), 256, 0, st>>>(C, x, n, act);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_loss(const float* S, const void* target, int B, int n, int loss, float* delta,
                        float* loss_out, float* partials, unsigned* counter, cudaStream_t st) {
  const size_t work = loss == CODENET_LOSS_MSE_MEAN ? (size_t)B * n : (size_t)B;
  size_t blocks = (work + (size_t)LOSS_THREADS * 4 - 1) / ((size_t)LOSS_THREADS * 4);
  if (blocks > LOSS_MAX_BLOCKS) blocks = LOSS_MAX_BLOCKS;
  if (blocks < 1) blocks = 1;
  loss_kernel<<<(int)blocks, LOSS_THREADS, 0, st>>>(S, target, B, n, loss, delta, loss_out, partials, counter);
  count_launch();
  return cudaGetLastError();
}

}  // namespace codenet
