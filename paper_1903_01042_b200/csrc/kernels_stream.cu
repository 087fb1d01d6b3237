// Streaming kernels over the coded weights: node products of step O1 (feedforward), and the
// fused node products of step O2 (backpropagation) + coded rank-B update of step O3.
// HBM-bound for small batches: every coded block is read once per pass with 16-byte loads,
// the backward pass writes each block back in the same sweep.
#include "codenet_internal.cuh"

#include <string.h>

namespace codenet {

unsigned long long g_launches = 0;

namespace {

template <typename T> struct Raw16 {
  static constexpr int N = Vec16<T>::N;
  // Every coded block is touched once per pass: evict-first loads and stores measured fastest.
  __device__ __forceinline__ static uint4 load_stream(const T* p) {
    return __ldcs(reinterpret_cast<const uint4*>(p));
  }
  // The same with an L2 eviction policy chosen at run time (createpolicy): evict-first for tiles that will not be
  // touched again before they leave L2, evict-last for the tail of a sweep that the next sweep starts on.
  __device__ __forceinline__ static uint4 load_policy(const T* p, uint64_t pol) {
    uint4 v;
    asm volatile("ld.global.L1::no_allocate.L2::cache_hint.v4.u32 {%0, %1, %2, %3}, [%4], %5;"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p), "l"(pol));
    return v;
  }
  __device__ __forceinline__ static void store_policy(T* p, const uint4& v, uint64_t pol) {
    asm volatile("st.global.L2::cache_hint.v4.u32 [%0], {%1, %2, %3, %4}, %5;"
                 :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "l"(pol) : "memory");
  }
  __device__ __forceinline__ static void unpack(const uint4& t, float (&v)[N]);
  __device__ __forceinline__ static uint4 pack(const float (&v)[N]);
};
__device__ __forceinline__ uint64_t l2_policy(bool keep) {
  uint64_t pol;
  if (keep) asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(pol));
  else asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
template <> __device__ __forceinline__ void Raw16<float>::unpack(const uint4& t, float (&v)[4]) {
  v[0] = __uint_as_float(t.x); v[1] = __uint_as_float(t.y);
  v[2] = __uint_as_float(t.z); v[3] = __uint_as_float(t.w);
}
template <> __device__ __forceinline__ uint4 Raw16<float>::pack(const float (&v)[4]) {
  return make_uint4(__float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]), __float_as_uint(v[3]));
}
template <> __device__ __forceinline__ void Raw16<__nv_bfloat16>::unpack(const uint4& t, float (&v)[8]) {
  Vec16<__nv_bfloat16>::unpack(t, v);
}
template <> __device__ __forceinline__ uint4 Raw16<__nv_bfloat16>::pack(const float (&v)[8]) {
  uint32_t w[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * k], v[2 * k + 1]);
    w[k] = *reinterpret_cast<const uint32_t*>(&h);
  }
  return make_uint4(w[0], w[1], w[2], w[3]);
}

template <int N> __device__ __forceinline__ void load_x(const float* p, float (&v)[N]) {
#pragma unroll
  for (int q = 0; q < N / 4; ++q) {
    const float4 t = __ldg(reinterpret_cast<const float4*>(p) + q);
    v[4 * q] = t.x; v[4 * q + 1] = t.y; v[4 * q + 2] = t.z; v[4 * q + 3] = t.w;
  }
}

#include "encode_device.cuh"

// -------------------------------------------------------------------------------------------
// Step O1: y_ij = W~_ij x_j for every active node (i < M, j < n).  One warp owns RW coded rows
// of one block-column; Y is [j][coded row][b], i.e. [codeword][node][row][b].
// -------------------------------------------------------------------------------------------
constexpr int FWD_WARPS = 8;

template <typename T, int BT, int FWD_RW, int FWD_UNR>
__global__ void __launch_bounds__(FWD_WARPS * 32)
forward_products_kernel(Geom g, const float* __restrict__ x, int ldx, int B, float* __restrict__ Y) {
  constexpr int VEC = Raw16<T>::N;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gr0 = (blockIdx.x * FWD_WARPS + warp) * FWD_RW;
  if (gr0 >= g.Mbr) return;
  const int j = blockIdx.y;
  const int b0 = blockIdx.z * BT;
  const T* W = reinterpret_cast<const T*>(g.Wt);
  const T* rowp[FWD_RW];
#pragma unroll
  for (int rw = 0; rw < FWD_RW; ++rw) {
    const int gr = min(gr0 + rw, g.Mbr - 1);
    rowp[rw] = W + (size_t)gr * g.ld + (size_t)j * g.ldb;
  }
  const float* xp[BT];
#pragma unroll
  for (int b = 0; b < BT; ++b) xp[b] = x + (size_t)min(b0 + b, B - 1) * ldx + (size_t)j * g.ldb;

  float acc[FWD_RW][BT];
#pragma unroll
  for (int rw = 0; rw < FWD_RW; ++rw)
#pragma unroll
    for (int b = 0; b < BT; ++b) acc[rw][b] = 0.0f;

#pragma unroll FWD_UNR
  for (int c = lane * VEC; c < g.ldb; c += 32 * VEC) {
    uint4 raw[FWD_RW];
#pragma unroll
    for (int rw = 0; rw < FWD_RW; ++rw) raw[rw] = Raw16<T>::load_stream(rowp[rw] + c);
    float xv[BT][VEC];
#pragma unroll
    for (int b = 0; b < BT; ++b) load_x<VEC>(xp[b] + c, xv[b]);
#pragma unroll
    for (int rw = 0; rw < FWD_RW; ++rw) {
      float wv[VEC];
      Raw16<T>::unpack(raw[rw], wv);
#pragma unroll
      for (int b = 0; b < BT; ++b)
#pragma unroll
        for (int k = 0; k < VEC; ++k) acc[rw][b] = fmaf(wv[k], xv[b][k], acc[rw][b]);
    }
  }
#pragma unroll
  for (int rw = 0; rw < FWD_RW; ++rw)
#pragma unroll
    for (int b = 0; b < BT; ++b) {
      const float s = warp_sum(acc[rw][b]);
      if (lane == 0 && gr0 + rw < g.Mbr && b0 + b < B)
        Y[((size_t)j * g.Mbr + gr0 + rw) * B + b0 + b] = s;
    }
}

// -------------------------------------------------------------------------------------------
// Steps O2 + O3 fused (batch <= 8).  A CTA owns R rows of block-row i and 128 16-byte column
// groups; each thread walks its column group down the rows: the old value feeds the column
// partial of z = W~^T delta, then the updated value W~ + lr * delta~ x~^T is written back.
// Parity block-rows (i >= m) are update-only.  zpart is [i][rt][b][ld].
//
// NEXT = true additionally takes the feedforward products of the NEXT iteration from the values just
// updated (y = W~_new x_next on the block-columns j < n), so that iteration's own sweep over the
// coded weights is not needed: per row a warp-shuffle sum of each thread's partial dot product,
// summed over the CTA's four warps in fixed order, one partial per (column strip, coded row, b) in
// ynext[strip][coded row][b].  Only used when every strip lies inside one block-column.
// -------------------------------------------------------------------------------------------
constexpr int BU_THREADS = 128;
constexpr int BU_UNROLL = 8;

template <typename T, int BT, bool NEXT>
__global__ void __launch_bounds__(BU_THREADS)
backward_update_kernel(Geom g, const float* __restrict__ Xt, const float* __restrict__ Dt, int B,
                       float lr, int R, int RT, float* __restrict__ zpart,
                       const float* __restrict__ xnext, int ldxn, float* __restrict__ ynext, int reverse, int keep_from,
                       int n_enc, EncodeArgs ea) {
  constexpr int VEC = Raw16<T>::N;
  extern __shared__ float sdelta[];  // [rows of the tile][BT], then (NEXT) [rows][4 warps][BT]
  // Tiles are walked column strip by column strip: the parity block-columns first, then the data
  // block-columns from the last to the first, rows top to bottom inside a strip.  The feedforward
  // pass walks the data block-columns first to last, so each pass starts on what the previous one
  // touched last and finds part of it still in L2.  When this sweep is the only pass of an iteration (it takes
  // the next feedforward products as well) every other launch walks the tiles in the opposite order (reverse),
  // for the same reason: the last tiles of one sweep, updated and still in L2, are the first of the next.
  // n_enc > 0: the first n_enc CTAs of the launch do the additional encoding of the vectors (the stand-alone
  // kernel's code) for the check that follows, and the sweep CTAs form the delta~ and x~ entries they need
  // themselves, from the last layer's sums, the target and the raw input, with that code's arithmetic: the
  // encoding no longer stands between the check of one iteration and the sweep of the next.
  if (n_enc > 0 && (int)blockIdx.x < n_enc) {
    encode_vectors_body(g, ea, (int)blockIdx.x, n_enc);
    return;
  }
  const int cta = (int)blockIdx.x - n_enc, n_sweep = (int)gridDim.x - n_enc;
  const int n_rowtiles = g.M * RT;
  const int bx = reverse ? n_sweep - 1 - cta : cta;
  const uint64_t pol = l2_policy(cta >= keep_from);   // the last CTAs' tiles stay for the next sweep
  uint64_t pol_keep;   // the partial sums the check kernel reads next
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
  const int strip_order = bx / n_rowtiles, rowtile = bx % n_rowtiles;
  const int n_strips = n_sweep / n_rowtiles;
  const int data_strips = (g.n * g.ldb) / (BU_THREADS * VEC);  // strips wholly inside the data columns
  int strip;
  if (strip_order < n_strips - data_strips) strip = data_strips + strip_order;
  else strip = n_strips - 1 - strip_order;
  const int i = rowtile / RT, rt = rowtile % RT;
  const int r0 = rt * R;
  const int nrows = min(R, g.b_r - r0);
  for (int idx = threadIdx.x; idx < nrows * BT; idx += BU_THREADS) {
    const int rr = idx / BT, b = idx % BT;
    float d = 0.0f;
    if (b < B && n_enc == 0) {
      d = Dt[(size_t)b * g.Mbr + (size_t)i * g.b_r + r0 + rr];
    } else if (b < B) {
      // delta^L = 2 (y - s) / (N B) of the mean-squared-error loss, or the parity combination of it
      const float* fy = ea.lf.target + (size_t)b * g.n_out;
      const float* fs = ea.lf.S + (size_t)b * g.n_out;
      const int e = r0 + rr;
      if (i < g.m) {
        const int gi = i * g.b_r + e;
        if (gi < g.n_out) d = 2.0f * (fy[gi] - fs[gi]) * ea.lf.scale;
      } else {
        for (int q = 0; q < g.m; ++q) {
          const int gi = q * g.b_r + e;
          if (gi >= g.n_out) break;
          d = fmaf(g.Pr[q * g.r_row + (i - g.m)], 2.0f * (fy[gi] - fs[gi]) * ea.lf.scale, d);
        }
      }
    }
    sdelta[idx] = d;
  }
  __syncthreads();
  const int gc0 = (strip * BU_THREADS + threadIdx.x) * VEC;
  if (gc0 >= g.ld) return;
  const int j = gc0 / g.ldb;
  if (i >= g.m && j >= g.n) return;  // no node in the corner (with NEXT: the whole CTA leaves here)
  const bool fwd_active = NEXT && j < g.n;
  float* sy = sdelta + R * BT;
  float xn[NEXT ? BT : 1][VEC];
  if (NEXT) {
#pragma unroll
    for (int b = 0; b < BT; ++b) {
      if (fwd_active && b < B) load_x<VEC>(xnext + (size_t)b * ldxn + gc0, xn[b]);
      else {
#pragma unroll
        for (int k = 0; k < VEC; ++k) xn[b][k] = 0.0f;
      }
    }
  }

  float xs[BT][VEC];  // lr * x~
#pragma unroll
  for (int b = 0; b < BT; ++b) {
    if (b < B) {
      if (n_enc == 0) {
        load_x<VEC>(Xt + (size_t)b * g.ld + gc0, xs[b]);
      } else if (j < g.n) {
        load_x<VEC>(ea.X + (size_t)b * g.n_in + gc0, xs[b]);      // (no padding between the sub-vectors here)
      } else {
        // x~ of a parity block-column: the combination of the data sub-vectors, in their order
#pragma unroll
        for (int k = 0; k < VEC; ++k) xs[b][k] = 0.0f;
        const int e = gc0 - j * g.ldb;
        for (int q = 0; q < g.n; ++q) {
          float t[VEC];
          load_x<VEC>(ea.X + (size_t)b * g.n_in + (size_t)q * g.b_c + e, t);
          const float c = g.Pc[q * g.r_col + (j - g.n)];
#pragma unroll
          for (int k = 0; k < VEC; ++k) xs[b][k] = fmaf(c, t[k], xs[b][k]);
        }
      }
#pragma unroll
      for (int k = 0; k < VEC; ++k) xs[b][k] *= lr;
    } else {
#pragma unroll
      for (int k = 0; k < VEC; ++k) xs[b][k] = 0.0f;
    }
  }
  float z[BT][VEC];
#pragma unroll
  for (int b = 0; b < BT; ++b)
#pragma unroll
    for (int k = 0; k < VEC; ++k) z[b][k] = 0.0f;

  T* wp = reinterpret_cast<T*>(g.Wt) + ((size_t)i * g.b_r + r0) * g.ld + gc0;
  // sums of eight rows' partial dot products across the warp in 9 shuffles instead of 40: each step halves
  // the number of rows a lane still carries; lanes (4r .. 4r+3) end up with the sum of row r
  auto reduce_rows = [&](const float (&yp)[NEXT && BT <= 2 ? BU_UNROLL : 1][NEXT && BT <= 2 ? BT : 1], int base) {
    if (!(NEXT && BT <= 2)) return;
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int b = 0; b < (BT <= 2 ? BT : 1); ++b) {
      float v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = yp[NEXT && BT <= 2 ? u : 0][b];
#pragma unroll
      for (int i2 = 0; i2 < 4; ++i2) {
        const float send = (lane & 16) ? v[i2] : v[i2 + 4];
        const float keep = (lane & 16) ? v[i2 + 4] : v[i2];
        v[i2] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 16);
      }
#pragma unroll
      for (int i2 = 0; i2 < 2; ++i2) {
        const float send = (lane & 8) ? v[i2] : v[i2 + 2];
        const float keep = (lane & 8) ? v[i2 + 2] : v[i2];
        v[i2] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 8);
      }
      {
        const float send = (lane & 4) ? v[0] : v[1];
        const float keep = (lane & 4) ? v[1] : v[0];
        v[0] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 4);
      }
      v[0] += __shfl_xor_sync(0xFFFFFFFFu, v[0], 2);
      v[0] += __shfl_xor_sync(0xFFFFFFFFu, v[0], 1);
      const int u = lane >> 2;
      if ((lane & 3) == 0 && base + u < nrows) sy[((base + u) * 4 + (threadIdx.x >> 5)) * BT + b] = v[0];
    }
  };
  float ypart[NEXT && BT <= 2 ? BU_UNROLL : 1][NEXT && BT <= 2 ? BT : 1];  // per-row partial dot products
  float yprev[NEXT && BT <= 2 ? BU_UNROLL : 1][NEXT && BT <= 2 ? BT : 1];  // ... of the previous eight rows
  for (int rr0 = 0; rr0 < nrows; rr0 += BU_UNROLL) {
    uint4 raw[BU_UNROLL];
#pragma unroll
    for (int u = 0; u < BU_UNROLL; ++u)
      if (rr0 + u < nrows) raw[u] = Raw16<T>::load_policy(wp + (size_t)(rr0 + u) * g.ld, pol);
    // the previous rows' partials are summed across the warp while these loads are in flight
    if (NEXT && BT <= 2 && fwd_active && rr0 > 0) reduce_rows(yprev, rr0 - BU_UNROLL);
#pragma unroll
    for (int u = 0; u < BU_UNROLL; ++u) {
      if (rr0 + u < nrows) {
        float wold[VEC], wv[VEC];
        Raw16<T>::unpack(raw[u], wold);
#pragma unroll
        for (int k = 0; k < VEC; ++k) wv[k] = wold[k];
#pragma unroll
        for (int b = 0; b < BT; ++b) {
          const float d = sdelta[(rr0 + u) * BT + b];
#pragma unroll
          for (int k = 0; k < VEC; ++k) {
            z[b][k] = fmaf(d, wold[k], z[b][k]);  // the product uses this iteration's weights
            wv[k] = fmaf(d, xs[b][k], wv[k]);
          }
        }
        const uint4 packed = Raw16<T>::pack(wv);
        Raw16<T>::store_policy(wp + (size_t)(rr0 + u) * g.ld, packed, pol);
        if (NEXT && fwd_active) {  // warp-uniform: a warp's columns lie in one block-column
          float wr[VEC];
          Raw16<T>::unpack(packed, wr);  // the stored (rounded) values are what the next pass would read
#pragma unroll
          for (int b = 0; b < BT; ++b) {
            float yp = 0.0f;
#pragma unroll
            for (int k = 0; k < VEC; ++k) yp = fmaf(wr[k], xn[b][k], yp);
            if (BT <= 2) {
              ypart[u][b] = yp;
            } else {
              yp = warp_sum(yp);
              if ((threadIdx.x & 31) == 0) sy[((rr0 + u) * 4 + (threadIdx.x >> 5)) * BT + b] = yp;
            }
          }
        }
      } else if (NEXT && BT <= 2) {
#pragma unroll
        for (int b = 0; b < BT; ++b) ypart[u][b] = 0.0f;
      }
    }
    if (NEXT && BT <= 2) {
#pragma unroll
      for (int u = 0; u < BU_UNROLL; ++u)
#pragma unroll
        for (int b = 0; b < BT; ++b) yprev[u][b] = ypart[u][b];
    }
  }
  if (NEXT && BT <= 2 && fwd_active && nrows > 0) reduce_rows(yprev, ((nrows - 1) / BU_UNROLL) * BU_UNROLL);
  if (NEXT && fwd_active) {
    __syncthreads();
    for (int idx = threadIdx.x; idx < nrows * BT; idx += BU_THREADS) {
      const int rr = idx / BT, b = idx % BT;
      if (b >= B) continue;
      const float* q = sy + (rr * 4) * BT + b;
      const float v = ((q[0] + q[BT]) + q[2 * BT]) + q[3 * BT];
      float* yp = &ynext[((size_t)strip * g.Mbr + (size_t)i * g.b_r + r0 + rr) * B + b];
      asm volatile("st.global.L2::cache_hint.f32 [%0], %1, %2;" :: "l"(yp), "f"(v), "l"(pol_keep) : "memory");
    }
  }
  if (i < g.m) {
#pragma unroll
    for (int b = 0; b < BT; ++b)
      if (b < B) {
        float* zp = zpart + (((size_t)i * RT + rt) * B + b) * g.ld + gc0;
#pragma unroll
        for (int q = 0; q < VEC / 4; ++q)
          asm volatile("st.global.L2::cache_hint.v4.f32 [%0], {%1, %2, %3, %4}, %5;"
                       :: "l"(zp + 4 * q), "f"(z[b][4 * q]), "f"(z[b][4 * q + 1]), "f"(z[b][4 * q + 2]), "f"(z[b][4 * q + 3]), "l"(pol_keep) : "memory");
      }
  }
}

// -------------------------------------------------------------------------------------------
// Step O2 alone for larger batches without tensor-core tiles: z_ij = W~_ij^T delta_i for the
// active nodes (i < m, j < Nn), batch entries in chunks of BT.  Z is [i][j][col][b].
// -------------------------------------------------------------------------------------------
template <typename T, int BT>
__global__ void __launch_bounds__(BU_THREADS)
backward_products_kernel(Geom g, const float* __restrict__ Dt, int B, float* __restrict__ Z) {
  constexpr int VEC = Raw16<T>::N;
  const int gc0 = (blockIdx.x * BU_THREADS + threadIdx.x) * VEC;
  if (gc0 >= g.ld) return;
  const int i = blockIdx.y, b0 = blockIdx.z * BT;
  const int j = gc0 / g.ldb, c0 = gc0 - j * g.ldb;
  float z[BT][VEC];
#pragma unroll
  for (int b = 0; b < BT; ++b)
#pragma unroll
    for (int k = 0; k < VEC; ++k) z[b][k] = 0.0f;
  const T* wp = reinterpret_cast<const T*>(g.Wt) + (size_t)i * g.b_r * g.ld + gc0;
  const float* dp[BT];
#pragma unroll
  for (int b = 0; b < BT; ++b) dp[b] = Dt + (size_t)min(b0 + b, B - 1) * g.Mbr + (size_t)i * g.b_r;
#pragma unroll 4
  for (int rr = 0; rr < g.b_r; ++rr) {
    float wv[VEC];
    Raw16<T>::unpack(*reinterpret_cast<const uint4*>(wp + (size_t)rr * g.ld), wv);
#pragma unroll
    for (int b = 0; b < BT; ++b) {
      const float d = __ldg(dp[b] + rr);
#pragma unroll
      for (int k = 0; k < VEC; ++k) z[b][k] = fmaf(d, wv[k], z[b][k]);
    }
  }
#pragma unroll
  for (int k = 0; k < VEC; ++k) {
    if (c0 + k >= g.b_c) continue;
#pragma unroll
    for (int b = 0; b < BT; ++b)
      if (b0 + b < B) Z[(((size_t)i * g.Nn + j) * g.b_c + c0 + k) * B + b0 + b] = z[b][k];
  }
}

// -------------------------------------------------------------------------------------------
// Step O3 alone for larger batches without tensor-core tiles: W~ += lr * Dt^T Xt on every stored
// block, one rounding per element.  CTA tile 32 rows x (32 * VEC) columns, batch staged through
// shared memory in chunks of 32.
// -------------------------------------------------------------------------------------------
constexpr int UPD_KC = 32;

template <typename T>
__global__ void __launch_bounds__(128)
update_kernel(Geom g, const float* __restrict__ Xt, const float* __restrict__ Dt, int B, float lr) {
  constexpr int VEC = Raw16<T>::N;
  constexpr int TC = 32 * VEC;
  __shared__ __align__(16) float sd[UPD_KC][32];
  __shared__ __align__(16) float sx[UPD_KC][TC];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int gr_tile = blockIdx.y * 32, gc_tile = blockIdx.x * TC;
  float acc[8][VEC];
#pragma unroll
  for (int a = 0; a < 8; ++a)
#pragma unroll
    for (int k = 0; k < VEC; ++k) acc[a][k] = 0.0f;
  for (int bb = 0; bb < B; bb += UPD_KC) {
    for (int idx = threadIdx.x; idx < UPD_KC * 32; idx += 128) {
      const int b = idx / 32, rr = idx % 32;
      const int gr = gr_tile + rr;
      sd[b][rr] = (bb + b < B && gr < g.Mbr) ? Dt[(size_t)(bb + b) * g.Mbr + gr] : 0.0f;
    }
    for (int idx = threadIdx.x; idx < UPD_KC * TC; idx += 128) {
      const int b = idx / TC, cc = idx % TC;
      const int gc = gc_tile + cc;
      sx[b][cc] = (bb + b < B && gc < g.ld) ? Xt[(size_t)(bb + b) * g.ld + gc] : 0.0f;
    }
    __syncthreads();
#pragma unroll 4
    for (int b = 0; b < UPD_KC; ++b) {
      float dv[8], xv[VEC];
#pragma unroll
      for (int a = 0; a < 8; ++a) dv[a] = sd[b][ty * 8 + a];
#pragma unroll
      for (int k = 0; k < VEC; ++k) xv[k] = sx[b][tx * VEC + k];
#pragma unroll
      for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int k = 0; k < VEC; ++k) acc[a][k] = fmaf(dv[a], xv[k], acc[a][k]);
    }
    __syncthreads();
  }
  const int gc0 = gc_tile + tx * VEC;
  if (gc0 >= g.ld) return;
  const int j = gc0 / g.ldb;
#pragma unroll
  for (int a = 0; a < 8; ++a) {
    const int gr = gr_tile + ty * 8 + a;
    if (gr >= g.Mbr) continue;
    const int i = gr / g.b_r;
    if (i >= g.m && j >= g.n) continue;
    T* p = reinterpret_cast<T*>(g.Wt) + (size_t)gr * g.ld + gc0;
    float wv[VEC];
    Raw16<T>::unpack(*reinterpret_cast<const uint4*>(p), wv);
#pragma unroll
    for (int k = 0; k < VEC; ++k) wv[k] = fmaf(lr, acc[a][k], wv[k]);
    *reinterpret_cast<uint4*>(p) = Raw16<T>::pack(wv);
  }
}

template <typename T, int RW, int UNR>
cudaError_t forward_launch(const Geom& g, const float* x, int ldx, int B, float* Y, cudaStream_t st) {
  const int bt = B >= 8 ? 8 : (B >= 4 ? 4 : (B >= 2 ? 2 : 1));
  dim3 grid((g.Mbr + FWD_WARPS * RW - 1) / (FWD_WARPS * RW), g.n, (B + bt - 1) / bt);
  dim3 block(FWD_WARPS * 32);
  switch (bt) {
    case 1: forward_products_kernel<T, 1, RW, UNR><<<grid, block, 0, st>>>(g, x, ldx, B, Y); break;
    case 2: forward_products_kernel<T, 2, RW, UNR><<<grid, block, 0, st>>>(g, x, ldx, B, Y); break;
    case 4: forward_products_kernel<T, 4, RW, UNR><<<grid, block, 0, st>>>(g, x, ldx, B, Y); break;
    default: forward_products_kernel<T, 8, RW, UNR><<<grid, block, 0, st>>>(g, x, ldx, B, Y); break;
  }
  count_launch();
  return cudaGetLastError();
}

template <typename T>
cudaError_t forward_dispatch(const Geom& g, const float* x, int ldx, int B, float* Y, cudaStream_t st) {
  // two rows per warp, four 16-byte loads per row in flight: fastest of the shapes tried on a B200
  return forward_launch<T, 2, 4>(g, x, ldx, B, Y, st);
}

template <typename T, bool NEXT>
cudaError_t backward_fused_launch(const codenet_layer_impl& L, int B, float lr, float* zpart, const float* xnext,
                                  int ldxn, float* ynext, cudaStream_t st, const float* enc_X, const float* enc_Delta,
                                  const LossFuse* enc_fuse) {
  constexpr int VEC = Raw16<T>::N;
  const Geom& g = L.g;
  const int bt = B > 4 ? 8 : (B > 2 ? 4 : (B > 1 ? 2 : 1));
  dim3 grid(((g.ld / VEC + BU_THREADS - 1) / BU_THREADS) * (g.M * L.bwd_rt));
  // the additional encoding rides on this launch (its CTAs come first): see the kernel
  EncodeArgs ea;
  memset(&ea, 0, sizeof(ea));
  int n_enc = 0;
  if (enc_fuse != nullptr) {
    ea.X = enc_X; ea.Delta = enc_Delta; ea.B = B; ea.Xt = L.ws.Xt; ea.Dt = L.ws.Dt; ea.dsum = L.ws.dsum; ea.xsum = L.ws.xsum;
    ea.lf = *enc_fuse;
    ea.em.dcount = (size_t)B * g.Mbr;
    ea.vec_ok = encode_vec_ok(g, enc_X, enc_Delta, enc_fuse->S, enc_fuse->target) ? 1 : 0;
    n_enc = (g.Nn * g.nsc + g.M * g.ns) * B;
  }
  const int n_sweep = (int)grid.x;
  grid.x += n_enc;
  const size_t smem = (size_t)L.bwd_rows * bt * sizeof(float) * (NEXT ? 5 : 1);
  const float* Xt = L.ws.Xt;
  const float* Dt = L.ws.Dt;
  int reverse = 0;
  int keep_from = n_sweep;   // no tile is kept
  if (NEXT) {
    reverse = L.sweep_reverse; L.sweep_reverse ^= 1;
    // the last 48 MB of a sweep stay at normal priority (measured on a B200 against 0, 96 and 160 MB: larger tails
    // make the sweep itself faster and the step slower, they crowd out what the kernels between two sweeps read)
    const size_t keep_bytes = (size_t)48 << 20;
    const size_t cta_bytes = (size_t)L.bwd_rows * BU_THREADS * 16;
    const size_t keep_ctas = keep_bytes / cta_bytes;
    keep_from = keep_ctas >= (size_t)n_sweep ? 0 : (int)(n_sweep - keep_ctas);
  }
  switch (bt) {
    case 1: backward_update_kernel<T, 1, NEXT><<<grid, BU_THREADS, smem, st>>>(g, Xt, Dt, B, lr, L.bwd_rows, L.bwd_rt, zpart, xnext, ldxn, ynext, reverse, keep_from, n_enc, ea); break;
    case 2: backward_update_kernel<T, 2, NEXT><<<grid, BU_THREADS, smem, st>>>(g, Xt, Dt, B, lr, L.bwd_rows, L.bwd_rt, zpart, xnext, ldxn, ynext, reverse, keep_from, n_enc, ea); break;
    case 4: backward_update_kernel<T, 4, NEXT><<<grid, BU_THREADS, smem, st>>>(g, Xt, Dt, B, lr, L.bwd_rows, L.bwd_rt, zpart, xnext, ldxn, ynext, reverse, keep_from, n_enc, ea); break;
    default: backward_update_kernel<T, 8, NEXT><<<grid, BU_THREADS, smem, st>>>(g, Xt, Dt, B, lr, L.bwd_rows, L.bwd_rt, zpart, xnext, ldxn, ynext, reverse, keep_from, n_enc, ea); break;
  }
  count_launch();
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_forward_products(const Geom& g, const float* x, int ldx, int B, float* Y, cudaStream_t st) {
  ProfileScope scope(CODENET_KERNEL_FORWARD, st);
  return launch_forward_products_plain(g, x, ldx, B, Y, st);
}

// the same launch without the optional event bracket (which creates events, i.e. allocates, when profiling is on)
cudaError_t launch_forward_products_plain(const Geom& g, const float* x, int ldx, int B, float* Y, cudaStream_t st) {
  return g.dtype == CODENET_BF16 ? forward_dispatch<__nv_bfloat16>(g, x, ldx, B, Y, st)
                                 : forward_dispatch<float>(g, x, ldx, B, Y, st);
}

cudaError_t launch_backward_update_fused(const codenet_layer_impl& L, int B, float lr, float* zpart,
                                         const float* xnext, int ldxn, float* ynext, cudaStream_t st,
                                         const float* enc_X, const float* enc_Delta, const LossFuse* enc_fuse) {
  ProfileScope scope(CODENET_KERNEL_BACKWARD_UPDATE, st);
  const bool bf16 = L.g.dtype == CODENET_BF16;
  if (xnext)
    return bf16 ? backward_fused_launch<__nv_bfloat16, true>(L, B, lr, zpart, xnext, ldxn, ynext, st, enc_X, enc_Delta, enc_fuse)
                : backward_fused_launch<float, true>(L, B, lr, zpart, xnext, ldxn, ynext, st, enc_X, enc_Delta, enc_fuse);
  return bf16 ? backward_fused_launch<__nv_bfloat16, false>(L, B, lr, zpart, nullptr, 0, nullptr, st, nullptr, nullptr, nullptr)
              : backward_fused_launch<float, false>(L, B, lr, zpart, nullptr, 0, nullptr, st, nullptr, nullptr, nullptr);
}

int backward_strip_elems(int dtype) { return BU_THREADS * (dtype == CODENET_BF16 ? 8 : 4); }

cudaError_t launch_backward_products(const codenet_layer_impl& L, int B, float* Z, cudaStream_t st) {
  ProfileScope scope(CODENET_KERNEL_BACKWARD, st);
  const Geom& g = L.g;
  const int vec = g.dtype == CODENET_BF16 ? 8 : 4;
  dim3 grid((g.ld / vec + BU_THREADS - 1) / BU_THREADS, g.m, (B + 7) / 8);
  if (g.dtype == CODENET_BF16)
    backward_products_kernel<__nv_bfloat16, 8><<<grid, BU_THREADS, 0, st>>>(g, L.ws.Dt, B, Z);
  else
    backward_products_kernel<float, 8><<<grid, BU_THREADS, 0, st>>>(g, L.ws.Dt, B, Z);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_update(const codenet_layer_impl& L, int B, float lr, cudaStream_t st) {
  ProfileScope scope(CODENET_KERNEL_UPDATE, st);
  const Geom& g = L.g;
  const int vec = g.dtype == CODENET_BF16 ? 8 : 4;
  dim3 grid((g.ld + 32 * vec - 1) / (32 * vec), (g.Mbr + 31) / 32);
  if (g.dtype == CODENET_BF16)
    update_kernel<__nv_bfloat16><<<grid, 128, 0, st>>>(g, L.ws.Xt, L.ws.Dt, B, lr);
  else
    update_kernel<float><<<grid, 128, 0, st>>>(g, L.ws.Xt, L.ws.Dt, B, lr);
  count_launch();
  return cudaGetLastError();
}

}  // namespace codenet
