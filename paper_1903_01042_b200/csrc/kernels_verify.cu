// Parity-check verification of the block outputs ("General Error-Detection Method" and
// "Decoding Algorithm" of the paper's Appendix B), soft-error injection, and the final row /
// column sums:
//
//   check_kernel:  U  every (codeword, node, slice) unit: working copy of the node output
//                     (+ injected noise), node norm, inner-checksum statistic
//                  X  syndrome maxima, the sums s_i / c_j assuming no error, inner-checksum update
//                  D  one CTA per codeword: thresholds, detection, location, erasure-decoding plan, its part
//                     of the report; then, only if some codeword needs work (the CTAs concerned wait for that
//                     word), the fix below inside the same launch
//   check_pair_kernel: the backward check of one iteration and the forward check of the next, side by side
//   fix (fix_body; fix_kernel for the stand-alone detect / decode call):
//                  V  verifies each decoding plan against the spare parities (codes with two and more
//                     parities: a grid barrier)
//                  F  recomputes the sums of the data nodes a final plan touches with corrected /
//                     fault-free values, rewrites the report
//
// Both kernels are several hundred kilobytes of instructions, most of them on paths a fault-free call
// never takes.  What a call does execute runs once or twice per warp, so instruction fetch is part of
// every phase's latency: rarely used arithmetic (the noise generator) is a real call, and work that a
// warp runs once is kept to few instructions rather than unrolled.
//
// Phases are separated by cooperative-groups grid barriers (cooperative launch: every CTA is
// resident, so the barrier cannot wait on a CTA that never runs).
#include "codenet_internal.cuh"

#include <cooperative_groups.h>
#include <float.h>
#include <string.h>

namespace cg = cooperative_groups;

namespace codenet {
namespace {

#include "check_device.cuh"


// Sums over the 32 lanes of 32 values per lane (v[a][b], index a * 8 + b) with 31 shuffles: at every
// step a lane keeps the half of its values whose index bit matches its lane bit and hands the other
// half to its partner.  Lane l returns the total of value l.
__device__ __forceinline__ float warp_sum32(float (&v2)[4][8]) {
  const int lane = threadIdx.x & 31;
  float v[32];
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = v2[i >> 3][i & 7];
#pragma unroll
  for (int h = 16; h >= 1; h >>= 1) {
    const bool up = lane & h;
#pragma unroll
    for (int i = 0; i < h; ++i) {
      const float keep = up ? v[i + h] : v[i], send = up ? v[i] : v[i + h];
      v[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, h);
    }
  }
  return v[0];
}

// Large batches, phase U: statistics of every node output.  A warp takes one (codeword, node, slice),
// BIG_SR rows of it and 32 batch entries: node norm and the slice sums of the inner check.  Only nodes the
// injection plan hits get noise and a working copy; the others stay where the product kernel wrote them.
__device__ __forceinline__ void big_phase_u(const CheckParams& p, const PhaseGeom& q,
                                            const unsigned long long* s_inj, const unsigned long long* s_out,
                                            const unsigned long long* s_in, uint32_t it, uint32_t key1,
                                            bool node_check, int nrch, int NS) {
  const Geom& g = p.g;
  const int B = p.B, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // 16-byte accesses: a warp covers 32 batch entries (four per lane, eight lanes) and four rows per access;
  // the four lanes that hold the same batch entries add up at the end.  B is a multiple of 32 and the
  // buffers are 16-byte aligned (checked before the launch).
  constexpr int lpr = 8, rpl = 4;
  const int wgroups = B / 32;
  const int lr = lane / lpr, lb = (lane % lpr) * 4;
  const int n_items = q.n_cw * q.K * q.nsl * nrch * wgroups;
  for (int item = blockIdx.x * CK_WARPS + warp; item < n_items; item += gridDim.x * CK_WARPS) {
    const int gq = item % wgroups;
    int rest = item / wgroups;
    const int k = rest % q.K; rest /= q.K;
    const int cw = rest % q.n_cw; rest /= q.n_cw;
    const int rc = rest % nrch, s = rest / nrch;
    const int b = gq * 32 + lb;
    const int t_begin = rc * BIG_SR, t_end = min(t_begin + BIG_SR, q.slen);
    const bool hit = (s_inj[cw] >> k) & 1ull, h_out = (s_out[cw] >> k) & 1ull, h_in = (s_in[cw] >> k) & 1ull;
    const size_t nb = ((size_t)cw * q.K + k) * q.n_el;
    const float* src = p.src + nb;
    float* yw = p.Yw + nb;
    const uint32_t node_id = node_id_of(g, p.phase, cw, k);
    float mx = 0.0f, so[4] = {0.0f, 0.0f, 0.0f, 0.0f}, sa[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    for (int t0 = t_begin; t0 < t_end; t0 += BIG_WC * rpl) {
      float4 v[BIG_WC];
#pragma unroll
      for (int w = 0; w < BIG_WC; ++w) {
        const int t = min(t0 + w * rpl + lr, t_end - 1);
        v[w] = *reinterpret_cast<const float4*>(src + ((size_t)s * q.slen + t) * B + b);
      }
      if (hit) {
#pragma unroll
        for (int w = 0; w < BIG_WC; ++w) {
          const int t = t0 + w * rpl + lr;
          if (t >= t_end) continue;
          const size_t e = ((size_t)s * q.slen + t) * B + b;
          v[w].x = with_faults(p, v[w].x, h_out, h_in, key1, it, node_id, nb, e);
          v[w].y = with_faults(p, v[w].y, h_out, h_in, key1, it, node_id, nb, e + 1);
          v[w].z = with_faults(p, v[w].z, h_out, h_in, key1, it, node_id, nb, e + 2);
          v[w].w = with_faults(p, v[w].w, h_out, h_in, key1, it, node_id, nb, e + 3);
          *reinterpret_cast<float4*>(yw + e) = v[w];
        }
      }
#pragma unroll
      for (int w = 0; w < BIG_WC; ++w)
        if (t0 + w * rpl + lr < t_end) {
          const float a0 = fabsf(v[w].x), a1 = fabsf(v[w].y), a2 = fabsf(v[w].z), a3 = fabsf(v[w].w);
          mx = fmaxf(mx, fmaxf(fmaxf(a0, a1), fmaxf(a2, a3)));
          so[0] += v[w].x; so[1] += v[w].y; so[2] += v[w].z; so[3] += v[w].w;
          sa[0] += a0; sa[1] += a1; sa[2] += a2; sa[3] += a3;
        }
    }
    mx = warp_max(mx);
    if (lane == 0) atomicMax(&p.st->norm[cw * MAXN + k], __float_as_uint(mx));
    if (node_check) {
#pragma unroll
      for (int h = lpr; h < 32; h <<= 1) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          so[c] += __shfl_xor_sync(0xFFFFFFFFu, so[c], h);
          sa[c] += __shfl_xor_sync(0xFFFFFFFFu, sa[c], h);
        }
      }
      if (lr == 0) {
        const size_t unit = ((size_t)cw * q.K + k) * q.nsl + s;
        *reinterpret_cast<float4*>(p.chk + (unit * NS + 2 * rc) * B + b) = make_float4(so[0], so[1], so[2], so[3]);
        *reinterpret_cast<float4*>(p.chk + (unit * NS + 2 * rc + 1) * B + b) = make_float4(sa[0], sa[1], sa[2], sa[3]);
      }
    }
  }
}

// Large batches, phase X: syndrome maxima and the sums s_i / c_j in ONE pass over the node outputs.
// A CTA takes 16 positions x 32 batch entries; a thread owns one (position, b) and walks every
// codeword and node: the syndrome of that element per codeword, and the running sum over codewords
// for each of the (at most KD) data nodes.  The sums leave through shared memory so that the
// (B, n_out) result is written along the output index.
template <int KD, int R>
__device__ __forceinline__ void big_phase_x(const CheckParams& p, const PhaseGeom& q, const float* sP,
                                            const unsigned long long* s_inj, unsigned* s_syn,
                                            float (*s_tile)[BIG_TR][33], bool check_off) {
  const Geom& g = p.g;
  const bool fwd = p.phase == CODENET_PHASE_FWD;
  const int B = p.B, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nout = fwd ? g.n_out : g.n_in;
  constexpr int tr = BIG_TR;   // (8-position tiles on small layers were tried: no faster there, slower on large ones)
  const int tiles_b = B / 32, tiles_p = (q.len + tr - 1) / tr;
  const bool want_syn = q.r > 0 && !check_off;
  for (int tile = blockIdx.x; tile < tiles_p * tiles_b; tile += gridDim.x) {
    const int pos0 = (tile / tiles_b) * tr, b0 = (tile % tiles_b) * 32;
#pragma unroll 1
    for (int rr = 0; rr < tr / CK_WARPS; ++rr) {
      const int row = warp + rr * CK_WARPS;
      const int pos = min(pos0 + row, q.len - 1);   // rows past the end repeat the last one; never stored
      const size_t e = (size_t)pos * B + b0 + lane;
      float acc[KD];
#pragma unroll
      for (int k = 0; k < KD; ++k) acc[k] = 0.0f;
      for (int cw0 = 0; cw0 < q.n_cw; cw0 += 2) {
        // every load of two codewords first (clamped indices instead of branches, so that all of them
        // are in flight together), then the arithmetic
        float par[2][R], o[2][KD];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int cw = min(cw0 + h, q.n_cw - 1);
          const unsigned long long own = s_inj[cw];
          const size_t cb = (size_t)cw * q.K * q.n_el + e;
#pragma unroll
          for (int t = 0; t < R; ++t) {
            const int k = q.kd + min(t, max(q.r - 1, 0));
            par[h][t] = q.r > 0 ? (((own >> k) & 1ull) ? p.Yw : p.src)[cb + (size_t)k * q.n_el] : 0.0f;
          }
#pragma unroll
          for (int k = 0; k < KD; ++k) {
            const int kc = min(k, q.kd - 1);
            o[h][k] = (((own >> kc) & 1ull) ? p.Yw : p.src)[cb + (size_t)kc * q.n_el];
          }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (cw0 + h >= q.n_cw) continue;
          float syn[R];
#pragma unroll
          for (int t = 0; t < R; ++t) syn[t] = t < q.r ? -par[h][t] : 0.0f;
#pragma unroll
          for (int k = 0; k < KD; ++k) {
            if (k < q.kd) {
              acc[k] += o[h][k];
#pragma unroll
              for (int t = 0; t < R; ++t)
                if (t < q.r) syn[t] = fmaf(sP[k * q.r + t], o[h][k], syn[t]);
            }
          }
          if (want_syn) {
            float m = 0.0f;
#pragma unroll
            for (int t = 0; t < R; ++t) m = fmaxf(m, fabsf(syn[t]));
            m = warp_max(m);
            if (lane == 0 && m > 0.0f) atomicMax(&s_syn[cw0 + h], __float_as_uint(m));
          }
        }
      }
#pragma unroll
      for (int k = 0; k < KD; ++k) s_tile[k][row][lane] = acc[k];
    }
    __syncthreads();
    if (p.out) {
      // runs of `tr` positions along the output index: segment = (data node, batch entry)
      const int segs = 32 / tr, sub = lane / tr, rp = lane % tr;
      for (int seg = warp * segs + sub; seg < q.kd * 32; seg += CK_WARPS * segs) {
        const int k = seg >> 5, bb = seg & 31;
        const int pos = pos0 + rp, gidx = k * q.len + pos;
        if (pos < q.len && gidx < nout) {
          const size_t oi = (size_t)(b0 + bb) * nout + gidx;
          p.out[oi] = finish_out(p, s_tile[k][rp][bb], oi);
        }
      }
    }
    __syncthreads();
  }
  if (want_syn) {
    __syncthreads();
    for (int cw = threadIdx.x; cw < q.n_cw; cw += CK_THREADS)
      if (s_syn[cw]) atomicMax(&p.st->syn[cw], s_syn[cw]);
  }
}

// The same pass for codewords of at most eight data nodes, with 16-byte accesses: a CTA takes 32 positions x
// 32 batch entries, a warp four positions (eight lanes x four batch entries each), a thread walks the
// codewords, NCW at a time, with all of their nodes' loads in flight (two codewords where a codeword has
// at most four data nodes: short codewords alone leave too few loads in flight).  The sums leave in runs of
// 32 positions.
template <int KD, int R, int NCW>
__device__ __forceinline__ void big_phase_x_wide(const CheckParams& p, const PhaseGeom& q, const float* sP,
                                                 const unsigned long long* s_inj, unsigned* s_syn,
                                                 float (*s_tile)[32][33], bool check_off) {
  constexpr int TW = 32;
  const Geom& g = p.g;
  const bool fwd = p.phase == CODENET_PHASE_FWD;
  const int B = p.B, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nout = fwd ? g.n_out : g.n_in;
  const int tiles_p = (q.len + TW - 1) / TW, tiles_b = B / 32;
  const bool want_syn = q.r > 0 && !check_off;
  const int row = warp * 4 + (lane >> 3), lb = (lane & 7) * 4;
  for (int tile = blockIdx.x; tile < tiles_p * tiles_b; tile += gridDim.x) {
    const int pos0 = (tile / tiles_b) * TW, b0 = (tile % tiles_b) * 32;
    const int pos = min(pos0 + row, q.len - 1);   // rows past the end repeat the last one; never stored
    const size_t e = (size_t)pos * B + b0 + lb;
    float acc[KD][4];
#pragma unroll
    for (int k = 0; k < KD; ++k)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[k][c] = 0.0f;
#pragma unroll 1
    for (int cw0 = 0; cw0 < q.n_cw; cw0 += NCW) {
      float4 par[NCW][R], o[NCW][KD];
#pragma unroll
      for (int h = 0; h < NCW; ++h) {
        const int cw = min(cw0 + h, q.n_cw - 1);
        const unsigned long long own = s_inj[cw];
        const size_t cb = (size_t)cw * q.K * q.n_el + e;
#pragma unroll
        for (int t = 0; t < R; ++t) {
          const int k = q.kd + min(t, max(q.r - 1, 0));
          par[h][t] = q.r > 0
                          ? *reinterpret_cast<const float4*>((((own >> k) & 1ull) ? p.Yw : p.src) + cb + (size_t)k * q.n_el)
                          : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        }
#pragma unroll
        for (int k = 0; k < KD; ++k) {
          const int kc = min(k, q.kd - 1);
          o[h][k] = *reinterpret_cast<const float4*>((((own >> kc) & 1ull) ? p.Yw : p.src) + cb + (size_t)kc * q.n_el);
        }
      }
#pragma unroll
      for (int h = 0; h < NCW; ++h) {
        if (cw0 + h >= q.n_cw) continue;
        float syn[R][4];
#pragma unroll
        for (int t = 0; t < R; ++t) {
          const bool on = t < q.r;
          syn[t][0] = on ? -par[h][t].x : 0.0f; syn[t][1] = on ? -par[h][t].y : 0.0f;
          syn[t][2] = on ? -par[h][t].z : 0.0f; syn[t][3] = on ? -par[h][t].w : 0.0f;
        }
#pragma unroll
        for (int k = 0; k < KD; ++k) {
          if (k < q.kd) {
            const float v[4] = {o[h][k].x, o[h][k].y, o[h][k].z, o[h][k].w};
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[k][c] += v[c];
#pragma unroll
            for (int t = 0; t < R; ++t)
              if (t < q.r) {
                const float pk = sP[k * q.r + t];
#pragma unroll
                for (int c = 0; c < 4; ++c) syn[t][c] = fmaf(pk, v[c], syn[t][c]);
              }
          }
        }
        if (want_syn) {
          float m = 0.0f;
#pragma unroll
          for (int t = 0; t < R; ++t)
#pragma unroll
            for (int c = 0; c < 4; ++c) m = fmaxf(m, fabsf(syn[t][c]));
          m = warp_max(m);
          if (lane == 0 && m > 0.0f) atomicMax(&s_syn[cw0 + h], __float_as_uint(m));
        }
      }
    }
#pragma unroll
    for (int k = 0; k < KD; ++k)
#pragma unroll
      for (int c = 0; c < 4; ++c) s_tile[k][row][lb + c] = acc[k][c];
    __syncthreads();
    if (p.out) {
      // 128-byte runs along the output index: segment = (data node, batch entry), lanes along the positions
      for (int seg = warp; seg < q.kd * 32; seg += CK_WARPS) {
        const int k = seg >> 5, bb = seg & 31;
        const int ps = pos0 + lane, gidx = k * q.len + ps;
        if (ps < q.len && gidx < nout) {
          const size_t oi = (size_t)(b0 + bb) * nout + gidx;
          p.out[oi] = finish_out(p, s_tile[k][lane][bb], oi);
        }
      }
    }
    __syncthreads();
  }
  if (want_syn) {
    __syncthreads();
    for (int cw = threadIdx.x; cw < q.n_cw; cw += CK_THREADS)
      if (s_syn[cw]) atomicMax(&p.st->syn[cw], s_syn[cw]);
  }
}

// Inner-checksum upkeep for small batches, same rule as the blocks: u += lr (1^T delta~_i) x~_j^T,
// v += lr delta~_i (x~_j^T 1).  One warp per checksum vector, lanes along it; vectors [vec_begin, vec_end) of the
// list (all u vectors, then all v vectors), handed out from the last warp of the part backwards; warps below
// first_warp of every CTA take none (they have other work in the same phase).
__device__ __forceinline__ void update_checksum_vectors(const CheckParams& p, const unsigned bid, const unsigned gdim,
                                                        int vec_begin, int vec_end, int first_warp) {
  const Geom& g = p.g;
  const int B = p.B, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (warp < first_warp) return;
  const int wpc = CK_WARPS - first_warp;
  const int gw = (gdim - 1 - bid) * wpc + (CK_WARPS - 1 - warp), nw = gdim * wpc;
  const int n_uvec = g.M * g.Nn * g.ns;
  for (int vec = vec_begin + gw; vec < vec_end; vec += nw) {
    const bool is_u = vec < n_uvec;
    const int v2 = is_u ? vec : vec - n_uvec, nsl = is_u ? g.ns : g.nsc;
    const int s = v2 % nsl, blk = v2 / nsl;
    const int i = blk / g.Nn, j = blk % g.Nn;
    if (i >= g.m && j >= g.n) continue;
    const int len = is_u ? g.b_c : g.b_r;
    float* tgt = is_u ? g.U + (size_t)v2 * g.ldb : g.V + (size_t)v2 * g.b_r;
    // entry e gets lr * sum_b coef[b] * rows[b][e]
    const float* rows = is_u ? p.Xt + (size_t)j * g.ldb : p.Dt + (size_t)i * g.b_r;
    const size_t rstride = is_u ? (size_t)g.ld : (size_t)g.Mbr;
    const float* coef = is_u ? p.dsum + ((size_t)i * g.ns + s) * B : p.xsum + ((size_t)j * g.nsc + s) * B;
    if ((len & 3) == 0 && (rstride & 3) == 0 &&
        ((reinterpret_cast<uintptr_t>(tgt) | reinterpret_cast<uintptr_t>(rows)) & 15) == 0) {
      // 16-byte accesses, eight per lane and round: a 1024-entry vector is one round
      for (int c0 = 4 * lane; c0 < len; c0 += 128 * 8) {
        float4 acc[8], old[8];
#pragma unroll
        for (int w = 0; w < 8; ++w) {
          const int c = c0 + 128 * w;
          old[w] = c < len ? *reinterpret_cast<const float4*>(tgt + c) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
          acc[w] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        }
        for (int b = 0; b < B; ++b) {
          const float d = coef[b];
#pragma unroll
          for (int w = 0; w < 8; ++w) {
            const int c = c0 + 128 * w;
            if (c < len) {
              const float4 x = *reinterpret_cast<const float4*>(rows + (size_t)b * rstride + c);
              acc[w].x = fmaf(d, x.x, acc[w].x); acc[w].y = fmaf(d, x.y, acc[w].y);
              acc[w].z = fmaf(d, x.z, acc[w].z); acc[w].w = fmaf(d, x.w, acc[w].w);
            }
          }
        }
#pragma unroll
        for (int w = 0; w < 8; ++w) {
          const int c = c0 + 128 * w;
          if (c < len)
            *reinterpret_cast<float4*>(tgt + c) =
                make_float4(fmaf(p.lr, acc[w].x, old[w].x), fmaf(p.lr, acc[w].y, old[w].y),
                            fmaf(p.lr, acc[w].z, old[w].z), fmaf(p.lr, acc[w].w, old[w].w));
        }
      }
      continue;
    }
    for (int c0 = lane; c0 < len; c0 += 32 * 8) {
      float acc[8], old[8];
#pragma unroll
      for (int w = 0; w < 8; ++w) {  // loads first, so that eight are in flight per lane
        const int c = c0 + 32 * w;
        old[w] = c < len ? tgt[c] : 0.0f;
        acc[w] = 0.0f;
      }
      for (int b = 0; b < B; ++b) {
        const float d = coef[b];
#pragma unroll
        for (int w = 0; w < 8; ++w) {
          const int c = c0 + 32 * w;
          if (c < len) acc[w] = fmaf(d, rows[(size_t)b * rstride + c], acc[w]);
        }
      }
#pragma unroll
      for (int w = 0; w < 8; ++w) {
        const int c = c0 + 32 * w;
        if (c < len) tgt[c] = fmaf(p.lr, acc[w], old[w]);
      }
    }
  }
}

// Checksum side of the inner check at batch 1: dot = a . w and dabs = |a| . |w| over lim entries, lanes along the index
// (each lane's part; the caller adds the lanes up).
__device__ __forceinline__ void checksum_dot(const float* a, const float* w, int lim, int lane, float& dot, float& dabs) {
  if ((lim & 3) == 0 && ((reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(w)) & 15) == 0) {
    // 16-byte loads: a 1024-entry product is one round of sixteen loads per lane
#pragma unroll 8
    for (int c = 4 * lane; c < lim; c += 128) {
      const float4 av = *reinterpret_cast<const float4*>(a + c), wv = *reinterpret_cast<const float4*>(w + c);
      dot = fmaf(av.x, wv.x, dot); dabs = fmaf(fabsf(av.x), fabsf(wv.x), dabs);
      dot = fmaf(av.y, wv.y, dot); dabs = fmaf(fabsf(av.y), fabsf(wv.y), dabs);
      dot = fmaf(av.z, wv.z, dot); dabs = fmaf(fabsf(av.z), fabsf(wv.z), dabs);
      dot = fmaf(av.w, wv.w, dot); dabs = fmaf(fabsf(av.w), fabsf(wv.w), dabs);
    }
  } else {
#pragma unroll 16
    for (int c = lane; c < lim; c += 32) {
      const float av = a[c], wv = w[c];
      dot = fmaf(av, wv, dot);
      dabs = fmaf(fabsf(av), fabsf(wv), dabs);
    }
  }
}

template <bool SPARE>
__device__ __forceinline__ void fix_body(CheckParams& p, const PhaseGeom& q, const float* sP, const unsigned long long* s_inj,
                                         CwPlan* s_plan, const unsigned bid, const unsigned gdim);

// PAIR: the body runs as one part of a paired launch (p.pair says which); bid / gdim are the CTA's index and the
// number of CTAs within its part.  Both parts pass the same two grid barriers.
template <bool BIG, bool PAIR>
__device__ __forceinline__ void check_body(CheckParams& p, const unsigned bid, const unsigned gdim) {
  cg::grid_group grid = cg::this_grid();
  const bool pair_bwd = PAIR && p.pair == 1, pair_fwd = PAIR && p.pair == 2;
  // which statistics buffer this call works in: read by every CTA before the first grid barrier, flipped by
  // CTA 0 after the second
  const int st_par = __ldcg(p.parity) & 1;
  p.st = p.st_base + st_par;
  p.st_next = p.st_base + (st_par ^ 1);
  const Geom& g = p.g;
  const bool fwd = p.phase == CODENET_PHASE_FWD;
  const PhaseGeom q = phase_geom(g, p.phase, p.B);
  const int B = p.B;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const bool check_off = g.locate_mode == CODENET_LOCATE_OFF;
  const bool node_check = g.locate_mode == CODENET_LOCATE_NODECHECK;
  constexpr bool big_batch = BIG;  // the host launches this instantiation exactly when lazy_copy(p) holds

  __shared__ float sP[MAXN * MAXR];
  __shared__ unsigned long long s_inj[MAXN], s_out[MAXN], s_in[MAXN];
  __shared__ unsigned s_syn[MAXN];
  __shared__ float red[CK_WARPS];
  __shared__ float s_proj[MAXR * MAXR];
  __shared__ int s_state, s_cand_ok, s_accept, s_verify;
  __shared__ unsigned long long s_F;
  __shared__ float s_tau, s_scale, s_smax, s_h;
  __shared__ float s_nrm[MAXN], s_rat[MAXN];
  // one buffer, two tenants that never overlap in time: the tiles of the large-batch sums pass, and the plans of the fix
  constexpr size_t kSumsBytes = sizeof(float) * BIG_KD * BIG_TR * 33, kPlanBytes = sizeof(CwPlan) * MAXN;
  __shared__ __align__(16) unsigned char s_scratch[BIG ? (kSumsBytes > kPlanBytes ? kSumsBytes : kPlanBytes) : kPlanBytes];

  for (int t = tid; t < q.kd * q.r; t += CK_THREADS) sP[t] = q.P[t];
  for (int t = tid; t < MAXN; t += CK_THREADS) s_syn[t] = 0u;
  build_hit_masks(p, q, s_inj, s_out, s_in);
  if (tid == 0) {
    // h = max_t (1 + sum_k |P[k, t]|), the code's part of the syndrome threshold (read in phase D)
    float h = 0.0f;
    for (int t = 0; t < q.r; ++t) {
      float acc = 1.0f;
      for (int k = 0; k < q.kd; ++k) acc += fabsf(sP[k * q.r + t]);
      h = fmaxf(h, acc);
    }
    s_h = h;
  }
  const uint32_t it = (p.fault.iteration ? *p.fault.iteration : 0u) + p.it_add;
  const uint32_t key1 = (p.fault.layer << 8) | (uint32_t)p.phase;

  // ------------------------------------------------------------------------------------------
  // phase U: one warp per (codeword, node, slice): working copy, node norm, inner-checksum ratio
  // ------------------------------------------------------------------------------------------
  {
    const int n_units = q.n_cw * q.K * q.nsl;
    const size_t SL = (size_t)q.slen * B;
    const float floor_c = g.tau_rel * (1.0f / 512.0f);
    const bool by_bgroup = big_batch;
    const int nrch = (q.slen + BIG_SR - 1) / BIG_SR;                        // row chunks of a slice
    const int dlen = fwd ? g.b_c : g.b_r;                                   // length of the checksum dot
    const int ncch = (dlen + BIG_DC - 1) / BIG_DC;                          // chunks of it
    const int NS = 2 * nrch + 2 * ncch;                                     // scratch floats per (unit, b)
    if (by_bgroup) {
      big_phase_u(p, q, s_inj, s_out, s_in, it, key1, node_check, nrch, NS);
    }
    // units go round the CTAs first and then round the warps, so that a few hundred of them spread over
    // all SMs instead of filling the first CTAs
    for (int unit = bid + gdim * warp; unit < (by_bgroup ? 0 : n_units); unit += gdim * CK_WARPS) {
      const int s = unit % q.nsl, ck = unit / q.nsl;
      const int k = ck % q.K, cw = ck / q.K;
      const bool hit = (s_inj[cw] >> k) & 1ull, h_out = (s_out[cw] >> k) & 1ull, h_in = (s_in[cw] >> k) & 1ull;
      const uint32_t node_id = node_id_of(g, p.phase, cw, k);
      const size_t nb = ((size_t)cw * q.K + k) * q.n_el;
      float* yw = p.Yw + nb;
      const size_t e0 = (size_t)s * SL;
      const bool copy = !(p.src_kind == 0 && p.src == p.Yw && !hit);
      float mx = 0.0f;
      if (B == 1 && node_check) {
        // batch 1: the checksum side of the inner check first (its loads do not wait for the working copy),
        // then the working copy with the slice sums taken from the values in registers
        const int i1 = fwd ? k : cw, j1 = fwd ? cw : k;
        const int blk1 = i1 * g.Nn + j1;
        const float* a = fwd ? g.U + ((size_t)blk1 * g.ns + s) * g.ldb : g.V + ((size_t)blk1 * g.nsc + s) * g.b_r;
        const float* w = fwd ? p.Vraw + (size_t)j1 * g.b_c : p.Vraw + (size_t)i1 * g.b_r;
        const int lim = fwd ? min(g.b_c, g.n_in - j1 * g.b_c) : min(g.b_r, g.n_out - i1 * g.b_r);
        float dot = 0.0f, dabs = 0.0f, sum_o = 0.0f, sum_abs = 0.0f;
        // (the forward part of a pair takes the checksum side after the barrier: the backward part is updating u)
        if (!pair_fwd) checksum_dot(a, w, lim, lane, dot, dabs);
        // four elements per lane and round, their partials loaded together (clean_value4): a round is a few
        // round trips to memory instead of one per element and sixteen partials
        for (size_t t0 = 0; t0 < SL; t0 += 128) {
          float v[4];
          size_t e4[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const size_t t = t0 + lane + 32 * u;
            e4[u] = e0 + (t < SL ? t : t0 + lane);   // (lanes past the end have no element at all: skipped below)
          }
          if (t0 + lane < SL) {
            if (copy) {
              clean_value4(p, q, cw, k, e4, v);
            } else {
#pragma unroll
              for (int u = 0; u < 4; ++u) v[u] = yw[e4[u]];
            }
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const size_t t = t0 + lane + 32 * u;
            if (t >= SL) continue;
            const size_t e = e0 + t;
            if (copy) {
              if (hit) v[u] = with_faults(p, v[u], h_out, h_in, key1, it, node_id, nb, e);
              yw[e] = v[u];
            }
            mx = fmaxf(mx, fabsf(v[u]));
            sum_o += v[u];
            sum_abs += fabsf(v[u]);
          }
        }
        mx = warp_max(mx);
        if (lane == 0) atomicMax(&p.st->norm[cw * MAXN + k], __float_as_uint(mx));
        sum_o = warp_sum(sum_o); sum_abs = warp_sum(sum_abs);
        if (pair_fwd) {
          if (lane == 0) { p.pair_sums[2 * unit] = sum_o; p.pair_sums[2 * unit + 1] = sum_abs; }
          continue;
        }
        dot = warp_sum(dot); dabs = warp_sum(dabs);
        const float ratio = fabsf(sum_o - dot) / (g.tau_rel * dabs + floor_c * sum_abs + g.tau_abs);
        if (lane == 0) atomicMax(&p.st->ratio[cw * MAXN + k], __float_as_uint(ratio));
        continue;
      }
#pragma unroll 4
      for (size_t t = lane; t < SL; t += 32) {
        const size_t e = e0 + t;
        float v;
        if (copy) {
          v = clean_value(p, q, cw, k, e);
          if (hit) v = with_faults(p, v, h_out, h_in, key1, it, node_id, nb, e);
          yw[e] = v;
        } else {
          v = yw[e];
        }
        mx = fmaxf(mx, fabsf(v));
      }
      mx = warp_max(mx);
      if (lane == 0) atomicMax(&p.st->norm[cw * MAXN + k], __float_as_uint(mx));
      if (!node_check) continue;
      __syncwarp();
      const int i = fwd ? k : cw, j = fwd ? cw : k;
      const int blk = i * g.Nn + j;
      float worst = 0.0f;
      for (int b = 0; b < B; ++b) {
        float sum_o = 0.0f, sum_abs = 0.0f, dot = 0.0f, dabs = 0.0f;
#pragma unroll 4
        for (int t = lane; t < q.slen; t += 32) {
          const float o = yw[e0 + (size_t)t * B + b];
          sum_o += o;
          sum_abs += fabsf(o);
        }
        if (fwd) {
          const float* u = g.U + ((size_t)blk * g.ns + s) * g.ldb;
          const float* x = p.Vraw + (size_t)b * g.n_in + (size_t)j * g.b_c;
          const int cmax = min(g.b_c, g.n_in - j * g.b_c);
#pragma unroll 16
          for (int c = lane; c < cmax; c += 32) {
            const float uv = u[c], xv = x[c];
            dot = fmaf(uv, xv, dot);
            dabs = fmaf(fabsf(uv), fabsf(xv), dabs);
          }
        } else {
          const float* v = g.V + ((size_t)blk * g.nsc + s) * g.b_r;
          const float* d = p.Vraw + (size_t)b * g.n_out + (size_t)i * g.b_r;
          const int rmax = min(g.b_r, g.n_out - i * g.b_r);
#pragma unroll 16
          for (int rr = lane; rr < rmax; rr += 32) {
            const float vv = v[rr], dv = d[rr];
            dot = fmaf(vv, dv, dot);
            dabs = fmaf(fabsf(vv), fabsf(dv), dabs);
          }
        }
        sum_o = warp_sum(sum_o); sum_abs = warp_sum(sum_abs); dot = warp_sum(dot); dabs = warp_sum(dabs);
        // checksum-side scale plus a rounding floor proportional to the magnitudes summed
        worst = fmaxf(worst, fabsf(sum_o - dot) / (g.tau_rel * dabs + floor_c * sum_abs + g.tau_abs));
      }
      if (lane == 0) atomicMax(&p.st->ratio[cw * MAXN + k], __float_as_uint(worst));
    }
    if (big_batch && node_check) {
      // checksum side of the inner check, u.x or v.delta: a warp takes four units of one codeword (they
      // share the vector operand) and eight batch entries, lanes along the dot-product index
      const int per_cw = q.K * q.nsl, ugroups = (per_cw + 3) / 4, chunks = (B + 7) / 8;
      const int n_items = q.n_cw * ugroups * chunks * ncch;
      // handed out from the last warp of the grid backwards: the statistics items above fill the grid from
      // the front, so on small layers the two kinds of work run side by side
      for (int item = (gdim - 1 - bid) * CK_WARPS + (CK_WARPS - 1 - warp); item < n_items;
           item += gdim * CK_WARPS) {
        const int cc = item % ncch, it3 = item / ncch;
        const int cw = it3 / (ugroups * chunks), rem = it3 % (ugroups * chunks);
        const int u0 = (rem / chunks) * 4, b0 = (rem % chunks) * 8;
        const float* a[4];
        int n_valid = 0;
#pragma unroll
        for (int uu = 0; uu < 4; ++uu) {
          const int local = min(u0 + uu, per_cw - 1);
          if (u0 + uu < per_cw) n_valid = uu + 1;
          const int s = local % q.nsl, k = local / q.nsl;
          const int i = fwd ? k : cw, j = fwd ? cw : k;
          const int blk = i * g.Nn + j;
          a[uu] = fwd ? g.U + ((size_t)blk * g.ns + s) * g.ldb : g.V + ((size_t)blk * g.nsc + s) * g.b_r;
        }
        const int len = fwd ? min(g.b_c, g.n_in - cw * g.b_c) : min(g.b_r, g.n_out - cw * g.b_r);
        const int c_begin = cc * BIG_DC, c_end = min(c_begin + BIG_DC, len);
        const size_t ldv = fwd ? (size_t)g.n_in : (size_t)g.n_out;
        const float* v0 = p.Vraw + (fwd ? (size_t)cw * g.b_c : (size_t)cw * g.b_r);
        float dot[4][8], dabs[4][8];
#pragma unroll
        for (int uu = 0; uu < 4; ++uu)
#pragma unroll
          for (int bb = 0; bb < 8; ++bb) { dot[uu][bb] = 0.0f; dabs[uu][bb] = 0.0f; }
#pragma unroll 2
        for (int c = c_begin + lane; c < c_end; c += 32) {
          float av[4], xv[8];
#pragma unroll
          for (int uu = 0; uu < 4; ++uu) av[uu] = a[uu][c];
#pragma unroll
          for (int bb = 0; bb < 8; ++bb) xv[bb] = v0[(size_t)min(b0 + bb, B - 1) * ldv + c];
#pragma unroll
          for (int uu = 0; uu < 4; ++uu)
#pragma unroll
            for (int bb = 0; bb < 8; ++bb) {
              dot[uu][bb] = fmaf(av[uu], xv[bb], dot[uu][bb]);
              dabs[uu][bb] = fmaf(fabsf(av[uu]), fabsf(xv[bb]), dabs[uu][bb]);
            }
        }
        // lane l ends up with the totals of pair (unit l / 8, batch entry l % 8)
        const float d = warp_sum32(dot), da = warp_sum32(dabs);
        const int uu = lane >> 3, bb = lane & 7;
        if (uu < n_valid && b0 + bb < B) {
          const size_t unit = (size_t)cw * per_cw + u0 + uu;
          p.chk[(unit * NS + 2 * nrch + 2 * cc) * B + b0 + bb] = d;
          p.chk[(unit * NS + 2 * nrch + 2 * cc + 1) * B + b0 + bb] = da;
        }
      }
    }
  }
  if (pair_bwd && p.update_checksums) {
    // the u vectors get this iteration's update before the barrier: the forward part, whose products come from
    // the updated blocks, reads them after it (nothing in a backward check reads u)
    // (warps that had no unit above: the units went round the CTAs first, so these are the same in every CTA)
    const int unit_warps = (q.n_cw * q.K * q.nsl + (int)gdim - 1) / (int)gdim;
    update_checksum_vectors(p, bid, gdim, 0, g.M * g.Nn * g.ns, unit_warps < CK_WARPS ? unit_warps : 0);
  }
  if (pair_fwd) {
    // what the forward part of the previous pair left in the staging buffers (sums and report of the iteration
    // that is ending) goes where the caller reads it, before this part overwrites them behind the barrier
    if (p.commit_S != nullptr)
      for (int idx = (int)bid * CK_THREADS + tid; idx < p.commit_n; idx += (int)gdim * CK_THREADS)
        p.commit_S_to[idx] = p.commit_S[idx];
    if (p.loss_partials != nullptr && bid == (gdim > 1 ? gdim - 2 : 0)) {
      // this step's loss, left as partial sums by the vector encoding: added up in that kernel's own order
      // (128 threads stride the list, lanes, then the four warps)
      float t = 0.0f;
      if (tid < 128)
        for (int idx = tid; idx < p.loss_n; idx += 128) t += __ldcg(&p.loss_partials[idx]);
      t = warp_sum(t);
      if (lane == 0) red[warp] = t;
      __syncthreads();
      if (tid == 0) *p.loss_out = red[0] + red[1] + red[2] + red[3];
      __syncthreads();
    }
    if (p.commit_rep != nullptr && bid == gdim - 1) {
      const uint32_t* from = reinterpret_cast<const uint32_t*>(p.commit_rep);
      uint32_t* to = reinterpret_cast<uint32_t*>(p.commit_rep_to);
      for (int t = tid; t < (int)(sizeof(codenet_report_t) / sizeof(uint32_t)); t += CK_THREADS) to[t] = from[t];
    }
  }
  grid.sync();

  // ------------------------------------------------------------------------------------------
  // phase X: syndrome maxima; sums assuming no error; inner-checksum update; reset of the
  // statistics buffer of the next call
  // ------------------------------------------------------------------------------------------
  const size_t gstride = (size_t)gdim * CK_THREADS;
  const size_t g0 = bid * (size_t)CK_THREADS + tid;
  if (pair_fwd) {
    // checksum side of the inner check, u . x, with the u vectors as the backward part has just updated them;
    // the slice sums wait in pair_sums.  Same units, same warps, same arithmetic as a check of its own.
    const int n_units = q.n_cw * q.K * q.nsl;
    const float floor_c = g.tau_rel * (1.0f / 512.0f);
    for (int unit = bid + gdim * warp; unit < n_units; unit += gdim * CK_WARPS) {
      const int s = unit % q.nsl, ck = unit / q.nsl;
      const int k = ck % q.K, cw = ck / q.K;
      const int blk1 = k * g.Nn + cw;
      const float* a = g.U + ((size_t)blk1 * g.ns + s) * g.ldb;
      const float* w = p.Vraw + (size_t)cw * g.b_c;
      const int lim = min(g.b_c, g.n_in - cw * g.b_c);
      float dot = 0.0f, dabs = 0.0f;
      checksum_dot(a, w, lim, lane, dot, dabs);
      dot = warp_sum(dot); dabs = warp_sum(dabs);
      const float sum_o = p.pair_sums[2 * unit], sum_abs = p.pair_sums[2 * unit + 1];
      const float ratio = fabsf(sum_o - dot) / (g.tau_rel * dabs + floor_c * sum_abs + g.tau_abs);
      if (lane == 0) atomicMax(&p.st->ratio[cw * MAXN + k], __float_as_uint(ratio));
    }
  }
  if (big_batch && node_check) {
    const float floor_c = g.tau_rel * (1.0f / 512.0f);
    const size_t total = (size_t)q.n_cw * q.K * q.nsl * B;
    const int nrch = (q.slen + BIG_SR - 1) / BIG_SR;
    const int ncch = ((fwd ? g.b_c : g.b_r) + BIG_DC - 1) / BIG_DC;
    const int NS = 2 * nrch + 2 * ncch;
    // the ratios start behind the CTAs that take the sum tiles below, the checksum update comes from the
    // far end of the grid: three independent pieces of work, side by side on small layers
    const int sum_tiles = ((q.len + BIG_TR - 1) / BIG_TR) * (B / 32);
    const int rot = sum_tiles % (int)gdim;
    const size_t g0r = (size_t)((bid + gdim - rot) % gdim) * CK_THREADS + tid;
    for (size_t idx = g0r; idx < total; idx += gstride) {
      // partial sums in index order: the same result every run
      const float* c = p.chk + (idx / B) * NS * B + idx % B;   // [unit][partial][b]
      float so = 0.0f, sa = 0.0f, d = 0.0f, da = 0.0f;
      for (int r0 = 0; r0 < nrch; r0 += 8) {  // eight partials of each kind in flight, added in order
        float t0[8], t1[8];
#pragma unroll
        for (int w = 0; w < 8; ++w) {
          const int r = min(r0 + w, nrch - 1);
          t0[w] = c[(size_t)(2 * r) * B];
          t1[w] = c[(size_t)(2 * r + 1) * B];
        }
#pragma unroll
        for (int w = 0; w < 8; ++w)
          if (r0 + w < nrch) { so += t0[w]; sa += t1[w]; }
      }
      for (int r0 = 0; r0 < ncch; r0 += 8) {
        float t0[8], t1[8];
#pragma unroll
        for (int w = 0; w < 8; ++w) {
          const int r = min(r0 + w, ncch - 1);
          t0[w] = c[(size_t)(2 * nrch + 2 * r) * B];
          t1[w] = c[(size_t)(2 * nrch + 2 * r + 1) * B];
        }
#pragma unroll
        for (int w = 0; w < 8; ++w)
          if (r0 + w < ncch) { d += t0[w]; da += t1[w]; }
      }
      float ratio = fabsf(so - d) / (g.tau_rel * da + floor_c * sa + g.tau_abs);
      // the 32 lanes of a warp hold 32 batch entries of one unit (B is a multiple of 32): one atomic per warp
      ratio = warp_max(ratio);
      const int ck = (int)(idx / B) / q.nsl;
      if (lane == 0) atomicMax(&p.st->ratio[(ck / q.K) * MAXN + ck % q.K], __float_as_uint(ratio));
    }
  }
  const bool one_pass = big_batch && q.kd <= BIG_KD;   // syndrome and sums together (large batches)
  // small batches: the syndrome pass starts at CTA 0, the sums right behind its CTAs, the checksum update at
  // the far end of the grid, so that the three pieces run side by side instead of one after the other in the
  // first CTAs
  const size_t syn_total = (q.r > 0 && !check_off && !one_pass) ? (size_t)q.n_cw * q.n_el : 0;
  const unsigned syn_ctas = (unsigned)(((syn_total + CK_THREADS - 1) / CK_THREADS) % gdim);
  const size_t g0s = (size_t)((bid + gdim - syn_ctas) % gdim) * CK_THREADS + tid;
  if (q.r > 0 && !check_off && !one_pass) {
    const size_t total = (size_t)q.n_cw * q.n_el;
    for (size_t idx = g0; idx < total; idx += gstride) {
      const int cw = (int)(idx / q.n_el);
      const size_t e = idx % q.n_el;
      float syn[MAXR];
      syndrome_at(cw_view(p, q, s_inj, cw), q, sP, e, syn);
      float m = 0.0f;
#pragma unroll
      for (int t = 0; t < MAXR; ++t) m = fmaxf(m, fabsf(syn[t]));
      atomicMax(&s_syn[cw], __float_as_uint(m));
    }
    __syncthreads();
    for (int cw = tid; cw < q.n_cw; cw += CK_THREADS)
      if (s_syn[cw]) atomicMax(&p.st->syn[cw], s_syn[cw]);
  }
  if (big_batch && one_pass) {
    float (*s_sums)[BIG_TR][33] = reinterpret_cast<float (*)[BIG_TR][33]>(s_scratch);   // [BIG_KD][BIG_TR][33]
    if (q.kd <= 8) {
      float (*s_wide)[32][33] = reinterpret_cast<float (*)[32][33]>(&s_sums[0][0][0]);   // [8][32][33]: the same bytes
      if (q.kd <= 4 && q.r <= 2) big_phase_x_wide<4, 2, 2>(p, q, sP, s_inj, s_syn, s_wide, check_off);
      else if (q.r <= 2) big_phase_x_wide<8, 2, 1>(p, q, sP, s_inj, s_syn, s_wide, check_off);
      else big_phase_x_wide<8, MAXR, 1>(p, q, sP, s_inj, s_syn, s_wide, check_off);
    } else {
      if (q.r <= 2) big_phase_x<BIG_KD, 2>(p, q, sP, s_inj, s_syn, s_sums, check_off);
      else big_phase_x<BIG_KD, MAXR>(p, q, sP, s_inj, s_syn, s_sums, check_off);
    }
  }
  if (p.out && big_batch && !one_pass) {
    // tiles of 32 outputs x 32 batch entries: rows of the node outputs are read along b, the sums leave
    // through shared memory along the output index, so both sides are whole 128-byte accesses
    __shared__ float s_tile[32][33];
    const int nout = fwd ? g.n_out : g.n_in;
    const int tiles_o = (nout + 31) / 32, tiles_b = B / 32;
    for (int tile = bid; tile < tiles_o * tiles_b; tile += gdim) {
      const int o0 = (tile / tiles_b) * 32, b0 = (tile % tiles_b) * 32;
#pragma unroll
      for (int rr = 0; rr < 32 / CK_WARPS; ++rr) {
        const int r = warp + rr * CK_WARPS, gidx = o0 + r;
        float acc = 0.0f;
        if (gidx < nout) {
          int node, pos;
          output_index(g, fwd, gidx, &node, &pos);
          const size_t e = (size_t)pos * B + b0 + lane;
#pragma unroll 8
          for (int cw = 0; cw < q.n_cw; ++cw) {
            const float* base = ((s_inj[cw] >> node) & 1ull) ? p.Yw : p.src;
            acc += base[((size_t)cw * q.K + node) * q.n_el + e];
          }
        }
        s_tile[r][lane] = acc;
      }
      __syncthreads();
#pragma unroll
      for (int rr = 0; rr < 32 / CK_WARPS; ++rr) {
        const int bb = warp + rr * CK_WARPS;
        if (o0 + lane < nout) {
          const size_t oi = (size_t)(b0 + bb) * nout + o0 + lane;
          p.out[oi] = finish_out(p, s_tile[lane][bb], oi);
        }
      }
      __syncthreads();
    }
  }
  if (p.out && !big_batch) {
    const int nout = fwd ? g.n_out : g.n_in;
    for (size_t idx = g0s; idx < (size_t)nout * B; idx += gstride) {
      const int b = (int)(idx % B), gidx = (int)(idx / B);
      int node, pos;
      output_index(g, fwd, gidx, &node, &pos);
      float acc = 0.0f;
#pragma unroll 8
      for (int cw = 0; cw < q.n_cw; ++cw) acc += p.Yw[(((size_t)cw * q.K + node) * q.len + pos) * B + b];
      p.out[(size_t)b * nout + gidx] = finish_out(p, acc, (size_t)b * nout + gidx);
    }
  }
  if (p.update_checksums && !big_batch) {
    // (in a pair the u vectors were updated before the first barrier: the forward part reads them after it)
    const int n_uvec = g.M * g.Nn * g.ns, n_vvec = g.M * g.Nn * g.nsc;
    update_checksum_vectors(p, bid, gdim, pair_bwd ? n_uvec : 0, n_uvec + n_vvec, 0);
  }
  if (p.update_checksums && big_batch && B >= 128) {
    // batches of 128 and more: u_ij += lr sum_b (1^T delta~_i)[b] x~_j[b][:] and
    // v_ij += lr sum_b (x~_j^T 1)[b] delta~_i[b][:], with the row loads shared between blocks (a batch this long
    // makes one warp per vector, below, a chain of eight and more dependent rounds of loads).  The rows
    // x~_j[b][:] serve every block of block column j (delta~_i[b][:] every block of block row i):
    // a warp takes 32 entries of the rows of one j (or i), up to eight partner blocks and one slice; eight
    // lanes cover the entries, four per lane, and the four lane groups take a quarter of the batch each, added
    // up in a fixed order at the end.
    const int gw = (gdim - 1 - bid) * CK_WARPS + (CK_WARPS - 1 - warp), nw = gdim * CK_WARPS;
    const int uspans = (g.b_c + 31) / 32, vspans = (g.b_r + 31) / 32;
    const int ugr = (g.M + 7) / 8, vgr = (g.Nn + 7) / 8;                      // partner groups
    const int ugs = (g.M + ugr - 1) / ugr, vgs = (g.Nn + vgr - 1) / vgr;      // partners per group, evened out
    const int n_uitems = g.Nn * g.ns * ugr * uspans, n_vitems = g.M * g.nsc * vgr * vspans;
    const int eq = lane & 7, bg = lane >> 3;
    for (int item = gw; item < n_uitems + n_vitems; item += nw) {
      const bool is_u = item >= n_vitems;
      const int it2 = is_u ? item - n_vitems : item;
      const int spans = is_u ? uspans : vspans, nsl = is_u ? g.ns : g.nsc;
      const int ngr = is_u ? ugr : vgr, gs = is_u ? ugs : vgs, P = is_u ? g.M : g.Nn;
      const int e = (it2 % spans) * 32 + 4 * eq;
      int rest = it2 / spans;
      const int grp = rest % ngr; rest /= ngr;
      const int sv = rest % nsl, o = rest / nsl;               // o: block column j (u) or block row i (v)
      const int q0 = grp * gs, nq = min(gs, P - q0);           // partners: block rows i (u) or block columns j (v)
      const int vlen = is_u ? g.b_c : g.b_r;
      const float* row = is_u ? p.Xt + (size_t)o * g.ldb : p.Dt + (size_t)o * g.b_r;
      const size_t rstride = is_u ? (size_t)g.ld : (size_t)g.Mbr;
      const float* coef = (is_u ? p.dsum : p.xsum) + ((size_t)q0 * nsl + sv) * B;
      const size_t cstride = (size_t)nsl * B;
      const bool vec = e + 3 < vlen && (rstride & 3) == 0 && (reinterpret_cast<uintptr_t>(row + e) & 15) == 0;
      int ee[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) ee[c] = min(e + c, vlen - 1);
      float acc[8][4];
#pragma unroll
      for (int qq = 0; qq < 8; ++qq)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[qq][c] = 0.0f;
      // lane group bg walks the batch entries [bg * B/4, (bg + 1) * B/4) in order, eight rows in flight; the
      // eight coefficients of a partner for those rows are two 16-byte loads (B is a multiple of 32 here)
      const int bq = bg * (B / 4);
      for (int t0 = 0; t0 < B / 4; t0 += 8) {
        float4 rv[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const float* r = row + (size_t)(bq + t0 + u) * rstride;
          if (vec) rv[u] = *reinterpret_cast<const float4*>(r + e);
          else rv[u] = make_float4(r[ee[0]], r[ee[1]], r[ee[2]], r[ee[3]]);
        }
#pragma unroll
        for (int qq = 0; qq < 8; ++qq) {
          const float4* cb = reinterpret_cast<const float4*>(coef + (size_t)min(qq, nq - 1) * cstride + bq + t0);
          const float4 c0 = cb[0], c1 = cb[1];
          const float cf[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            acc[qq][0] = fmaf(cf[u], rv[u].x, acc[qq][0]);
            acc[qq][1] = fmaf(cf[u], rv[u].y, acc[qq][1]);
            acc[qq][2] = fmaf(cf[u], rv[u].z, acc[qq][2]);
            acc[qq][3] = fmaf(cf[u], rv[u].w, acc[qq][3]);
          }
        }
      }
#pragma unroll
      for (int qq = 0; qq < 8; ++qq)
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          acc[qq][c] += __shfl_xor_sync(0xFFFFFFFFu, acc[qq][c], 8);
          acc[qq][c] += __shfl_xor_sync(0xFFFFFFFFu, acc[qq][c], 16);
        }
      if (bg == 0) {
        // every old value first, then every store: one round trip to memory instead of one per partner
        float* vp[8];
        float old[8][4];
#pragma unroll
        for (int qq = 0; qq < 8; ++qq) {
          const int i = is_u ? q0 + qq : o, j = is_u ? o : q0 + qq;
          vp[qq] = nullptr;
          if (qq < nq && !(i >= g.m && j >= g.n)) {
            const int blk = i * g.Nn + j;
            vp[qq] = is_u ? g.U + ((size_t)blk * g.ns + sv) * g.ldb : g.V + ((size_t)blk * g.nsc + sv) * g.b_r;
          }
#pragma unroll
          for (int c = 0; c < 4; ++c) old[qq][c] = (vp[qq] != nullptr && e + c < vlen) ? vp[qq][e + c] : 0.0f;
        }
#pragma unroll
        for (int qq = 0; qq < 8; ++qq)
#pragma unroll
          for (int c = 0; c < 4; ++c)
            if (vp[qq] != nullptr && e + c < vlen) vp[qq][e + c] = fmaf(p.lr, acc[qq][c], old[qq][c]);
      }
    }
  }
  if (p.update_checksums && big_batch && B < 128) {
    // batches under 128: a warp takes 32 entries of one checksum vector (one per lane) and walks the batch in
    // index order, 32 batch entries in flight: one or two rounds of loads per item, and few instructions,
    // which counts on small layers where every warp runs this once
    const int gw = (gdim - 1 - bid) * CK_WARPS + (CK_WARPS - 1 - warp), nw = gdim * CK_WARPS;
    const int ucols = (g.b_c + 31) / 32, vrows = (g.b_r + 31) / 32;
    const int n_blk = g.M * g.Nn;
    const int n_uitems = n_blk * g.ns * ucols, n_vitems = n_blk * g.nsc * vrows;
    for (int item = gw; item < n_uitems + n_vitems; item += nw) {
      const bool is_u = item < n_uitems;
      const int it2 = is_u ? item : item - n_uitems;
      const int spans = is_u ? ucols : vrows, nsl = is_u ? g.ns : g.nsc;
      const int blk = it2 / (nsl * spans), rem = it2 % (nsl * spans);
      const int sv = rem / spans, e = (rem % spans) * 32 + lane;
      const int i = blk / g.Nn, j = blk % g.Nn;
      if (i >= g.m && j >= g.n) continue;
      const int vlen = is_u ? g.b_c : g.b_r;            // entries of a checksum vector
      float* v = is_u ? g.U + ((size_t)blk * g.ns + sv) * g.ldb : g.V + ((size_t)blk * g.nsc + sv) * g.b_r;
      // entry e gets lr * sum_b coef[b] * row[b][e]
      const float* coef = is_u ? p.dsum + ((size_t)i * g.ns + sv) * B : p.xsum + ((size_t)j * g.nsc + sv) * B;
      const float* row = (is_u ? p.Xt + (size_t)j * g.ldb : p.Dt + (size_t)i * g.b_r) + min(e, vlen - 1);
      const size_t rstride = is_u ? (size_t)g.ld : (size_t)g.Mbr;
      const float old = e < vlen ? v[e] : 0.0f;
      float acc = 0.0f;
      for (int bq = 0; bq < B; bq += 32) {   // B is a multiple of 32 here
        float cf[32], rv[32];
#pragma unroll
        for (int u = 0; u < 32; ++u) {
          cf[u] = coef[bq + u];
          rv[u] = row[(size_t)(bq + u) * rstride];
        }
#pragma unroll
        for (int u = 0; u < 32; ++u) acc = fmaf(cf[u], rv[u], acc);
      }
      if (e < vlen) v[e] = fmaf(p.lr, acc, old);
    }
  }
  {
    unsigned* z = reinterpret_cast<unsigned*>(p.st_next);
    for (size_t idx = g0; idx < sizeof(CheckStats) / sizeof(unsigned); idx += gstride) z[idx] = 0u;
  }
  if (p.rep != nullptr && bid == gdim - 1) {
    // the report starts empty; every codeword's CTA adds its part in phase D (counts, masks, extremes:
    // all order-independent), so no CTA has to come last and gather
    codenet_report_t* r = p.rep;
    if (tid == 0) {
      r->status = (p.tc_flag && *p.tc_flag) ? (uint32_t)CODENET_TIMEOUT : (uint32_t)CODENET_CLEAN;
      r->n_detected_cw = 0u; r->n_flagged_nodes = 0u; r->n_fallback_cw = 0u;
      r->detected_mask = 0ull;
      r->min_margin_hit = FLT_MAX;
      r->max_margin_clean = 0.0f;
    }
    for (int c = q.n_cw + tid; c < MAXN; c += CK_THREADS) { r->flagged_mask[c] = 0ull; r->injected_mask[c] = 0ull; }
  }
  grid.sync();
  if (bid == 0 && tid == 0) *p.parity = st_par ^ 1;

  // ------------------------------------------------------------------------------------------
  // phase D: one CTA per codeword decides
  // ------------------------------------------------------------------------------------------
  for (int cw = bid; cw < q.n_cw; cw += gdim) {
    const CwView yw = cw_view(p, q, s_inj, cw);
    const unsigned long long injected = s_inj[cw];
    float cw_min_hit = FLT_MAX, cw_max_clean = 0.0f;
    __syncthreads();
    if (tid < q.K) {
      s_nrm[tid] = __uint_as_float(__ldcg(&p.st->norm[cw * MAXN + tid]));
      s_rat[tid] = __uint_as_float(__ldcg(&p.st->ratio[cw * MAXN + tid]));
    }
    if (tid == MAXN) s_smax = __uint_as_float(__ldcg(&p.st->syn[cw]));
    __syncthreads();
    // scale: the (r+1)-th largest node norm, so that up to r corrupted outputs cannot inflate it.  Every
    // node's thread counts the norms that come before its own in decreasing order (ties by index); the
    // one with exactly r before it holds the scale.
    if (tid < q.K) {
      const float mine = s_nrm[tid];
      int before = 0;
      for (int k = 0; k < q.K; ++k) {
        const float o = s_nrm[k];
        before += (o > mine || (o == mine && k < tid)) ? 1 : 0;
      }
      if (before == (q.r < q.K ? q.r : q.K - 1)) s_scale = mine;
    }
    __syncthreads();
    if (tid == 0) {
      const float scale = s_scale;
      const float tau = g.tau_rel * s_h * scale + g.tau_abs;
      s_tau = tau;
        const float smax = s_smax;
      unsigned long long flags = 0;
      if (node_check)
        for (int k = 0; k < q.K; ++k) {
          const float ratio = s_rat[k];
          if (ratio > 1.0f) flags |= 1ull << k;
          if ((injected >> k) & 1ull) cw_min_hit = fminf(cw_min_hit, ratio);
          else cw_max_clean = fmaxf(cw_max_clean, ratio);
        }
      if (q.r > 0 && !check_off) {
        // a hit codeword is detected by its node flags or by its syndrome, so the syndrome is the
        // margin of a hit only where no node check runs
        const float ratio = smax / tau;
        if (injected) { if (!node_check) cw_min_hit = fminf(cw_min_hit, ratio); }
        else cw_max_clean = fmaxf(cw_max_clean, ratio);
      }
      const bool detected = !check_off && ((q.r > 0 && smax > tau) || flags != 0);
      s_F = flags;
      if (!detected) s_state = 0;
      else if (flags != 0) s_state = 1;
      else if (g.locate_mode != CODENET_LOCATE_NONE && q.r >= 2) s_state = 2;
      else s_state = 3;
      // Verification step of the error detection ("Errors in Error-Detection under Error Model 2"): the evaluation
      // of the codeword's parity checks is made twice and compared.  A soft error in one evaluation shifts its
      // value by a noise sample; any difference means the evaluations disagree: the codeword is left as it is and
      // the caller restores the last checkpoint.
      s_verify = 0;
      if (p.small.on) {
        const uint32_t its = p.small.iteration ? *p.small.iteration : 0u;
        const uint32_t vunit = (uint32_t)(p.phase * 64 + cw);
        if (small_is_hit(p.small, CODENET_PHASE_CHECK, its, vunit) &&
            hit_noise(p.small.seed, (p.small.layer << 8) | (uint32_t)CODENET_PHASE_CHECK, its, vunit, 0u, p.small.sigma) != 0.0f)
          s_verify = 1;
      }
      }
    __syncthreads();
    const bool disagree_check = s_verify != 0;
    int state = disagree_check ? 4 : s_state;  // block-uniform copy
    const bool detected = state != 0 && !disagree_check;

    // location from the syndrome alone: smallest support (<= r/2 nodes, lexicographic order) whose
    // least-squares fit leaves a residual below tau
    if (state == 2) {
      // largest support tried: the paper's t = r / 2, or r - 1 in the joint mode (whole sub-vectors in error:
      // the smallest support that fits every element is the true one while it has at most r - 1 nodes)
      const bool joint = g.locate_mode == CODENET_LOCATE_JOINT;
      const int tmax = min(joint ? min(q.r - 1, 3) : min(q.r / 2, 2), q.K);
      int found = 0;
      for (int size = 1; size <= tmax && !found; ++size) {
        int i0 = 0, i1 = 1, i2 = 2;
        for (;;) {
          if (tid == 0) {
            double HF[MAXR][3], G[9], Ginv[9];
            const int idx[3] = {i0, i1, i2};
            for (int a = 0; a < size; ++a)
              for (int t = 0; t < q.r; ++t)
                HF[t][a] = idx[a] < q.kd ? (double)sP[idx[a] * q.r + t] : (idx[a] - q.kd == t ? -1.0 : 0.0);
            for (int a = 0; a < size; ++a)
              for (int b = 0; b < size; ++b) {
                double acc = 0.0;
                for (int t = 0; t < q.r; ++t) acc += HF[t][a] * HF[t][b];
                G[a * size + b] = acc;
              }
            s_cand_ok = invert_small(size, G, Ginv) ? 1 : 0;
            if (s_cand_ok)
              for (int a = 0; a < q.r; ++a)
                for (int b = 0; b < q.r; ++b) {
                  double acc = a == b ? 1.0 : 0.0;
                  for (int c = 0; c < size; ++c)
                    for (int d = 0; d < size; ++d) acc -= HF[a][c] * Ginv[c * size + d] * HF[b][d];
                  s_proj[a * q.r + b] = (float)acc;
                }
          }
          __syncthreads();
          float worst = 0.0f;
          if (s_cand_ok) {
            for (size_t e = tid; e < q.n_el; e += CK_THREADS) {
              float syn[MAXR];
              syndrome_at(yw, q, sP, e, syn);
              for (int a = 0; a < q.r; ++a) {
                float acc = 0.0f;
#pragma unroll
                for (int t = 0; t < MAXR; ++t)
                  if (t < q.r) acc = fmaf(s_proj[a * q.r + t], syn[t], acc);
                worst = fmaxf(worst, fabsf(acc));
              }
            }
          }
          worst = block_max256(worst, red);
          if (tid == 0) {
            s_accept = (s_cand_ok && worst <= s_tau) ? 1 : 0;
            if (s_accept) {
              s_F = 1ull << i0;
              if (size >= 2) s_F |= 1ull << i1;
              if (size == 3) s_F |= 1ull << i2;
            }
          }
          __syncthreads();
          if (s_accept) { found = 1; break; }
          if (size == 1) {
            if (++i0 >= q.K) break;
          } else if (size == 2) {
            if (++i1 >= q.K) {
              if (++i0 >= q.K - 1) break;
              i1 = i0 + 1;
            }
          } else {
            if (++i2 >= q.K) {
              if (++i1 >= q.K - 1) {
                if (++i0 >= q.K - 2) break;
                i1 = i0 + 1;
              }
              i2 = i1 + 1;
            }
          }
        }
      }
      state = found ? 1 : 3;
    }

    if (tid == 0) {
      CwPlan& pl = p.plan[cw];
      const unsigned long long F = s_F;
      pl.F = F;
      pl.injected = injected;
      pl.detected = detected ? 1 : 0;
      pl.tau = s_tau;
      pl.min_hit = cw_min_hit;
      pl.max_clean = cw_max_clean;
      pl.nfd = 0;
      pl.spare = 0;
      if (detected && p.small.on) {
        // Verification step of the decoding ("Errors in decoding under Error Model 2"): the list of nodes found
        // erroneous is made twice and compared.  A soft error in one evaluation changes the membership of one node
        // (chosen by the generator): the lists differ and the decoding is deemed erroneous.
        const uint32_t its = p.small.iteration ? *p.small.iteration : 0u;
        const uint32_t vunit = (uint32_t)(p.phase * 64 + cw);
        if (small_is_hit(p.small, CODENET_PHASE_DECODE, its, vunit)) {
          uint32_t o[4];
          philox4x32_10(its, vunit, 1u, 0u, p.small.seed, (p.small.layer << 8) | (uint32_t)CODENET_PHASE_DECODE, o);
          const unsigned long long F_other = F ^ (1ull << (o[0] % (uint32_t)q.K));
          if (F_other != F) state = 4;
        }
      }
      if (state == 1) {
        int nfd = 0, nq = 0, ok = 1;
        if (__popcll(F) > q.r) ok = 0;
        if (ok) {
          for (int k = 0; k < q.kd; ++k) if ((F >> k) & 1ull) pl.fd[nfd++] = k;
          for (int t = 0; t < q.r && nq < nfd; ++t) if (!((F >> (q.kd + t)) & 1ull)) pl.q[nq++] = t;
          if (nq < nfd) ok = 0;
        }
        if (ok && nfd == 1) {
          // one located data node, the usual case: the 1 x 1 system as the general elimination would solve it
          const double a00 = (double)sP[pl.fd[0] * q.r + pl.q[0]];
          if (a00 == 0.0) ok = 0;
          else pl.ainv[0] = 1.0 / a00;
        } else if (ok && nfd > 0) {
          double A[MAXR * MAXR];
          for (int a = 0; a < nfd; ++a)
            for (int b = 0; b < nfd; ++b) A[a * nfd + b] = (double)sP[pl.fd[b] * q.r + pl.q[a]];
          if (!invert_small(nfd, A, pl.ainv)) ok = 0;
        }
        if (ok) {
          pl.nfd = nfd;
          // parities that are neither located nor used must agree with the corrected codeword
          for (int t = 0; t < q.r; ++t) {
            bool used = false;
            for (int a = 0; a < nfd; ++a) used |= pl.q[a] == t;
            if (!used && !((F >> (q.kd + t)) & 1ull)) pl.spare |= 1u << t;
          }
        } else {
          state = 3;
        }
      }
      pl.state = state;
      if (p.inline_fix || p.tail_fix) {
        // one counter tells the waiting CTAs both things: how many codewords have decided (low half) and how many of
        // them need work (high half)
        __threadfence();
        atomicAdd(&p.st->done_d, 1u + (state != 0 ? 0x10000u : 0u));
      } else if (state != 0) {
        atomicOr(&p.st->need_fix, 1u);   // read by the fix kernel that follows
      }
      // the report after the counter: the CTAs that wait for the counter read the plans, not the report, and the fence
      // in front of it then has the plan's stores alone to wait for
      if (p.rep != nullptr) {
        codenet_report_t* r = p.rep;
        r->flagged_mask[cw] = detected ? F : 0ull;
        r->injected_mask[cw] = injected;
        if (detected) {
          atomicAdd(&r->n_detected_cw, 1u);
          atomicAdd(&r->n_flagged_nodes, (unsigned)__popcll(F));
          atomicOr(reinterpret_cast<unsigned long long*>(&r->detected_mask), 1ull << cw);
        }
        if (state == 3) atomicAdd(&r->n_fallback_cw, 1u);
        const uint32_t outcome = state == 1 ? (uint32_t)CODENET_CORRECTED
                               : state == 3 ? (uint32_t)(p.have_clean ? CODENET_FALLBACK : CODENET_FAILED)
                               : state == 4 ? (uint32_t)CODENET_DISAGREE
                                            : (uint32_t)CODENET_CLEAN;
        // (a wait that ran out in a tensor-core kernel outranks every outcome: the status was set to TIMEOUT above)
        if (outcome != CODENET_CLEAN && !(p.tc_flag && *p.tc_flag)) atomicMax(&r->status, outcome);
        atomicMin(reinterpret_cast<unsigned*>(&r->min_margin_hit), __float_as_uint(cw_min_hit));
        atomicMax(reinterpret_cast<unsigned*>(&r->max_margin_clean), __float_as_uint(cw_max_clean));
      }
    }
    __syncthreads();
  }
  // No fix kernel follows a check whose sums are wanted.  The CTAs that take part stay until the counter says that
  // every codeword has decided (a bounded wait, about a microsecond) and, if it also says that some codeword needs
  // work, do the fix kernel's work together (`fix_body`, the same code).  Small batches with at most one parity (no plan has a spare parity to be verified against, so the
  // plans are final): the CTAs that decided the codewords, which end at about the same time anyway.  Large batches, or
  // two and more parities: the whole (co-resident) grid; with spare parities that includes their verification pass
  // and its grid barrier, which every CTA then takes.
  const bool whole_grid = !PAIR && p.tail_fix;
  const unsigned n_fix = whole_grid ? gdim : min((unsigned)q.n_cw, gdim);
  if ((whole_grid || p.inline_fix) && bid < n_fix) {
    __shared__ unsigned s_go;
    if (tid == 0) {
      unsigned v = 0u, go = 0u;
      for (unsigned spin = 0; spin < (1u << 22); ++spin) {
        v = *reinterpret_cast<volatile unsigned*>(&p.st->done_d);
        if ((v & 0xFFFFu) >= (unsigned)q.n_cw) { go = (v >> 16) != 0u ? 2u : 1u; break; }
        __nanosleep(64);
      }
      if (go == 0u) atomicExch(const_cast<int*>(p.tc_flag), 1);   // gave up: reported as TIMEOUT by the next check
      __threadfence();
      s_go = go;
    }
    __syncthreads();
    if (s_go == 2u) {
      CwPlan* s_plan = reinterpret_cast<CwPlan*>(s_scratch);   // (the sums pass is long over)
      if (whole_grid && q.r >= 2) fix_body<true>(p, q, sP, s_inj, s_plan, bid, n_fix);
      else fix_body<false>(p, q, sP, s_inj, s_plan, bid, n_fix);
    }
  }
  // every CTA read the counter before the first grid barrier
  if (p.bump != nullptr && bid == 0 && tid == 0) *p.bump += 1u;
}

template <bool BIG>
__global__ void __launch_bounds__(CK_THREADS, 2) check_kernel(CheckParams p) {
  check_body<BIG, false>(p, blockIdx.x, gridDim.x);
}

// The backward check of one iteration and the forward check of the next (on the products the update sweep took
// ahead) in one cooperative launch: CTAs [0, n_first) are the backward part, the rest the forward part, each part
// with its own statistics buffers, plans, working copy and report.  Small batches only (B = 1, node check, at most
// one parity per code), where a check is a chain of short latency-bound phases and two of them side by side take
// little longer than one.
struct PairParams {
  CheckParams v[2];
  int n_first;
};

__global__ void __launch_bounds__(CK_THREADS, 2) check_pair_kernel(const __grid_constant__ PairParams pp) {
  const int part = blockIdx.x >= (unsigned)pp.n_first ? 1 : 0;
  CheckParams p = pp.v[part];
  check_body<false, true>(p, part ? blockIdx.x - pp.n_first : blockIdx.x, part ? gridDim.x - pp.n_first : pp.n_first);
}

// SPARE: some plan may have a spare parity to be verified on (two and more parities in the phase's code);
// that pass needs a grid barrier, so only this instantiation is a cooperative launch.
// s_plan: room for MAXN plans in shared memory.
template <bool SPARE>
__device__ __forceinline__ void fix_body(CheckParams& p, const PhaseGeom& q, const float* sP, const unsigned long long* s_inj,
                                         CwPlan* s_plan, const unsigned bid, const unsigned gdim) {
  const Geom& g = p.g;
  const bool fwd = p.phase == CODENET_PHASE_FWD;
  const int B = p.B;
  const int tid = threadIdx.x;
  __shared__ unsigned s_res[MAXN];
  __shared__ unsigned s_final[MAXN];
  for (int t = tid; t < MAXN; t += CK_THREADS) s_res[t] = 0u;
  // the plans, once per CTA, into shared memory: every element's decoding reads them, and from global memory each
  // field would be one more round trip in front of the loads that depend on it
  {
    const uint32_t* from = reinterpret_cast<const uint32_t*>(p.plan);
    uint32_t* to = reinterpret_cast<uint32_t*>(s_plan);
    const int words = q.n_cw * (int)(sizeof(CwPlan) / sizeof(uint32_t));
    for (int w = tid; w < words; w += CK_THREADS) to[w] = __ldcg(from + w);
  }
  __syncthreads();
  const size_t gstride = (size_t)gdim * CK_THREADS;
  const size_t g0 = bid * (size_t)CK_THREADS + tid;

  // phase V: residual of every decoding plan on its spare parities
  if (SPARE) {
    cg::grid_group grid = cg::this_grid();
    // only the codewords whose plan has a spare parity are walked (the others, nearly all, cost one test each)
    for (int cw = 0; cw < q.n_cw; ++cw) {
      const CwPlan& pl = s_plan[cw];
      if (pl.state != 1 || pl.spare == 0u) continue;
      const CwView yw = cw_view(p, q, s_inj, cw);
      float resid = 0.0f;
      if (lazy_copy(p) && pl.nfd == 1 && q.r <= 2) {
        // large batches, one located data node: four batch entries per thread and round
        for (unsigned e = (unsigned)g0 * 4u; e < (unsigned)q.n_el; e += (unsigned)gstride * 4u) {
          float fix[4];
          double par[2][4];
          decode1_at4<true>(yw, q, sP, pl, e, fix, par);
#pragma unroll
          for (int t = 0; t < 2; ++t)
            if (t < q.r && ((pl.spare >> t) & 1u)) {
              const float4 o = yw.at4(q, q.kd + t, e);
              resid = fmaxf(resid, fmaxf(fmaxf(fabsf((float)(par[t][0] - (double)o.x)), fabsf((float)(par[t][1] - (double)o.y))),
                                         fmaxf(fabsf((float)(par[t][2] - (double)o.z)), fabsf((float)(par[t][3] - (double)o.w)))));
            }
        }
      } else {
        for (unsigned e = (unsigned)g0; e < (unsigned)q.n_el; e += (unsigned)gstride) {
          float fix[MAXR];
          double par[MAXR];
          decode_at(yw, q, sP, pl, e, fix, par);
#pragma unroll
          for (int t = 0; t < MAXR; ++t)
            if (t < q.r && ((pl.spare >> t) & 1u))
              resid = fmaxf(resid, fabsf((float)(par[t] - (double)yw.at(q, q.kd + t, e))));
        }
      }
      resid = warp_max(resid);
      if ((tid & 31) == 0 && resid > 0.0f) atomicMax(&s_res[cw], __float_as_uint(resid));
    }
    __syncthreads();
    for (int cw = tid; cw < q.n_cw; cw += CK_THREADS)
      if (s_res[cw]) atomicMax(&p.st->resid[cw], s_res[cw]);
    grid.sync();
  }
  for (int cw = tid; cw < MAXN; cw += CK_THREADS) {
    unsigned st = 0u;
    if (cw < q.n_cw) {
      const CwPlan& pl = s_plan[cw];
      st = (unsigned)pl.state;
      if (SPARE && st == 1u && pl.spare != 0u && __uint_as_float(__ldcg(&p.st->resid[cw])) > pl.tau) st = 3u;
    }
    s_final[cw] = st;
  }
  __syncthreads();

  // phase F: sums with the corrected / fault-free values.  Only data nodes that some codeword's final
  // plan touches change (a located parity output, or a failed codeword without a fault-free copy, leaves
  // every sum as the check kernel wrote it), so only their outputs are recomputed.
  if (p.out) {
    __shared__ unsigned long long s_nodes, s_touch[MAXN];
    if (tid == 0) s_nodes = 0ull;
    for (int c = tid; c < MAXN; c += CK_THREADS) s_touch[c] = 0ull;
    __syncthreads();
    if (tid < q.n_cw) {
      const unsigned long long data = q.kd >= 64 ? ~0ull : ((1ull << q.kd) - 1ull);
      unsigned long long mask = 0ull;
      if (s_final[tid] == 1u) mask = s_plan[tid].F & data;
      else if (s_final[tid] == 3u && p.have_clean) mask = s_inj[tid] & data;
      s_touch[tid] = mask;
      if (mask) atomicOr(&s_nodes, mask);
    }
    __syncthreads();
    const unsigned long long nodes = s_nodes;
    const int nout = fwd ? g.n_out : g.n_in;
    const size_t per_node = (size_t)q.len * B;
    for (int node = 0; node < q.kd; ++node) {
      if (!((nodes >> node) & 1ull)) continue;
      if (lazy_copy(p)) {
        // large batches (B a multiple of 32): four batch entries of one position per thread and round
        for (unsigned idx = (unsigned)g0 * 4u; idx < (unsigned)per_node; idx += (unsigned)gstride * 4u) {
          const int b = (int)(idx % (unsigned)B), pos = (int)(idx / (unsigned)B);
          const int gidx = node * q.len + pos;
          if (gidx >= nout) continue;
          float acc[4];
          sum_final_values4(p, q, sP, s_inj, s_final, s_touch, s_plan, node, idx, acc);
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const size_t oi = (size_t)(b + c) * nout + gidx;
            p.out[oi] = finish_out(p, acc[c], oi);
          }
        }
        continue;
      }
      // (32-bit index arithmetic: a node output has fewer than 2^32 elements, and 64-bit division is a long routine)
      for (unsigned idx = (unsigned)g0; idx < (unsigned)per_node; idx += (unsigned)gstride) {
        const int b = B == 1 ? 0 : (int)(idx % (unsigned)B), pos = B == 1 ? (int)idx : (int)(idx / (unsigned)B);
        const int gidx = node * q.len + pos;
        if (gidx >= nout) continue;
        const float acc = sum_final_values(p, q, sP, s_inj, s_final, s_touch, s_plan, node, idx);
        p.out[(size_t)b * nout + gidx] = finish_out(p, acc, (size_t)b * nout + gidx);
      }
    }
  }
  if (p.commit) {
    // write the corrected codewords back (located data outputs solved, located parities re-encoded)
    const size_t total = (size_t)q.n_cw * q.n_el;
    for (size_t idx = g0; idx < total; idx += gstride) {
      const int cw = (int)(idx / q.n_el);
      const size_t e = idx % q.n_el;
      float* yw = p.Yw + (size_t)cw * q.K * q.n_el;
      if (s_final[cw] == 1u) {
        const CwPlan& pl = s_plan[cw];
        float fix[MAXR];
        double par[MAXR];
        decode_at(cw_view(p, q, s_inj, cw), q, sP, pl, e, fix, par);
#pragma unroll
        for (int a = 0; a < MAXR; ++a)
          if (a < pl.nfd) yw[(size_t)pl.fd[a] * q.n_el + e] = fix[a];
#pragma unroll
        for (int t = 0; t < MAXR; ++t)
          if (t < q.r && ((pl.F >> (q.kd + t)) & 1ull)) yw[(size_t)(q.kd + t) * q.n_el + e] = (float)par[t];
      } else if (s_final[cw] == 3u && p.have_clean) {
        for (int k = 0; k < q.K; ++k)
          if ((s_inj[cw] >> k) & 1ull) yw[(size_t)k * q.n_el + e] = clean_value(p, q, cw, k, e);
      }
    }
  }
  // (without spare parities the plans are final as the check kernel's decision phase reported them)
  if (SPARE && p.rep && bid == 0) {
    __shared__ float s_a[MAXN], s_b[MAXN];
    write_report(p, q.n_cw, s_final, s_a, s_b);
  }
}

template <bool SPARE>
__global__ void __launch_bounds__(CK_THREADS) fix_kernel(CheckParams p) {
  p.st = p.st_base + ((__ldcg(p.parity) & 1) ^ 1);   // the buffer the check kernel before this one worked in
  if (p.st->need_fix == 0u) return;  // the usual case: every codeword passed its checks
  const PhaseGeom q = phase_geom(p.g, p.phase, p.B);
  __shared__ float sP[MAXN * MAXR];
  __shared__ unsigned long long s_inj[MAXN];
  for (int t = threadIdx.x; t < q.kd * q.r; t += CK_THREADS) sP[t] = q.P[t];
  build_hit_masks(p, q, s_inj);
  __shared__ CwPlan s_plan[MAXN];
  fix_body<SPARE>(p, q, sP, s_inj, s_plan, blockIdx.x, gridDim.x);
}

// Soft errors in a node's own copy of its input sub-vector (the copy the activation / post-multiplication step
// generated for it): the node multiplies W~_ij (x_j + nu), so its output is off by W~_ij nu.  One CTA per
// (feedforward node, slab of 32 columns): a hit node's slab of nu goes to shared memory, every row's partial product
// is added into dY (zeroed before the launch; the order of the additions is not fixed: the node is located and its
// output discarded, only the size of the deviation matters).
__global__ void __launch_bounds__(256) input_fault_kernel(Geom g, SmallDev sf, int B, float* __restrict__ dY) {
  extern __shared__ float s_nu[];   // [32 columns][B]
  const int node = blockIdx.x, j = node / g.M, i = node % g.M;   // codeword (block-column) j, node (block-row) i
  const uint32_t its = sf.iteration ? *sf.iteration : 0u;
  const uint32_t node_id = (uint32_t)(i * g.Nn + j);
  if (!small_is_hit(sf, CODENET_PHASE_INPUT, its, node_id)) return;
  const int c0 = blockIdx.y * 32, nc = min(32, g.b_c - c0);
  const uint32_t key1 = (sf.layer << 8) | (uint32_t)CODENET_PHASE_INPUT;
  for (int t = threadIdx.x; t < nc * B; t += blockDim.x)
    s_nu[t] = soft_error_noise(sf.seed, key1, its, node_id, (uint32_t)((c0 + t / B) * B + t % B), sf.sigma);
  __syncthreads();
  float* out = dY + ((size_t)j * g.M + i) * ((size_t)g.b_r * B);
  for (int t = threadIdx.x; t < g.b_r * B; t += blockDim.x) {
    const int r = t / B, b = t % B;
    float acc = 0.0f;
    for (int c = 0; c < nc; ++c)
      acc = fmaf(load_elem(g.Wt, g.dtype, ((size_t)i * g.b_r + r) * g.ld + (size_t)j * g.ldb + c0 + c), s_nu[c * B + b], acc);
    atomicAdd(out + t, acc);
  }
}

// Plain sums of the data-node outputs for calls that check nothing (no code, or the checks switched off, and no
// injection): s_i = sum_j y_ij / c_j = sum_i z_ij straight from the node outputs or their partial sums, in the same
// fixed order as the checked path, an empty report.  No barrier, no working copy, no inner-checksum update.
// bid / gdim: the CTA's index and the number of CTAs within its part (a launch of its own: the whole grid).
__device__ __forceinline__ void sum_body(const CheckParams& p, const unsigned bid, const unsigned gdim) {
  const Geom& g = p.g;
  const bool fwd = p.phase == CODENET_PHASE_FWD;
  const PhaseGeom q = phase_geom(g, p.phase, p.B);
  const int B = p.B;
  const int nout = fwd ? g.n_out : g.n_in;
  for (size_t idx = bid * (size_t)CK_THREADS + threadIdx.x; idx < (size_t)nout * B; idx += (size_t)gdim * CK_THREADS) {
    const int b = (int)(idx % B), gidx = (int)(idx / B);
    int node, pos;
    output_index(g, fwd, gidx, &node, &pos);
    float acc = 0.0f;
    for (int cw = 0; cw < q.n_cw; ++cw) acc += clean_value(p, q, cw, node, (size_t)pos * B + b);
    const size_t oi = (size_t)b * nout + gidx;
    // (paired form: what the previous pair staged at this index goes out first, by the thread that overwrites it)
    if (p.commit_S != nullptr && oi < (size_t)p.commit_n) p.commit_S_to[oi] = p.commit_S[oi];
    p.out[oi] = finish_out(p, acc, oi);
  }
  codenet_report_t* rep = p.rep;
  if (bid == 0) {
    if (p.commit_rep != nullptr) {
      const uint32_t* from = reinterpret_cast<const uint32_t*>(p.commit_rep);
      uint32_t* to = reinterpret_cast<uint32_t*>(p.commit_rep_to);
      for (int t = threadIdx.x; t < (int)(sizeof(codenet_report_t) / sizeof(uint32_t)); t += CK_THREADS) to[t] = from[t];
      __syncthreads();
    }
    if (rep) {
      if (threadIdx.x == 0) {
        rep->status = (p.tc_flag && *p.tc_flag) ? (uint32_t)CODENET_TIMEOUT : (uint32_t)CODENET_CLEAN;
        rep->n_detected_cw = 0; rep->n_flagged_nodes = 0; rep->n_fallback_cw = 0;
        rep->detected_mask = 0; rep->min_margin_hit = FLT_MAX; rep->max_margin_clean = 0.0f;
      }
      for (int cw = threadIdx.x; cw < MAXN; cw += CK_THREADS) { rep->flagged_mask[cw] = 0; rep->injected_mask[cw] = 0; }
    }
  }
  if (p.loss_partials != nullptr && bid == gdim - 1) {
    // the step's loss from the partial sums the vector encoding left (its own order: see check_body)
    __shared__ float red[CK_WARPS];
    float t = 0.0f;
    if (threadIdx.x < 128)
      for (int idx = threadIdx.x; idx < p.loss_n; idx += 128) t += __ldcg(&p.loss_partials[idx]);
    t = warp_sum(t);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = t;
    __syncthreads();
    if (threadIdx.x == 0) *p.loss_out = red[0] + red[1] + red[2] + red[3];
  }
  if (p.bump != nullptr && bid == 0 && threadIdx.x == 0) *p.bump += 1u;
}

__global__ void __launch_bounds__(CK_THREADS) sum_outputs_kernel(CheckParams p) {
  sum_body(p, blockIdx.x, gridDim.x);
}

// The sums of one iteration's backward stage and of the next iteration's forward stage in one plain launch, for
// layers that check nothing: the counterpart of check_pair_kernel (same staging of the next iteration's sums and
// report, same loss hand-over), without a barrier: every output is written by one thread.
__global__ void __launch_bounds__(CK_THREADS) sum_pair_kernel(const __grid_constant__ PairParams pp) {
  const int part = blockIdx.x >= (unsigned)pp.n_first ? 1 : 0;
  const CheckParams& p = pp.v[part];
  sum_body(p, part ? blockIdx.x - pp.n_first : blockIdx.x, part ? gridDim.x - pp.n_first : pp.n_first);
}

int g_coop_blocks_check = 0, g_coop_blocks_fix = 0, g_coop_blocks_check_max = 0;

cudaError_t coop_grid_limits() {
  if (g_coop_blocks_check > 0) return cudaSuccess;
  int dev = 0, sms = 0, occ_c = 0, occ_b = 0, occ_f = 0, coop = 0;
  cudaError_t e;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev)) != cudaSuccess) return e;
  if (!coop) return cudaErrorNotSupported;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ_c, check_kernel<false>, CK_THREADS, 0)) != cudaSuccess) return e;
  if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ_b, check_kernel<true>, CK_THREADS, 0)) != cudaSuccess) return e;
  if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ_f, fix_kernel<true>, CK_THREADS, 0)) != cudaSuccess) return e;
  if (occ_c < 1 || occ_b < 1 || occ_f < 1) return cudaErrorLaunchOutOfResources;
  g_coop_blocks_check = sms * occ_c;
  g_coop_blocks_check_max = sms * occ_b;
  g_coop_blocks_fix = sms * occ_f;
  // two CTAs per SM are enough to hide latency and keep the grid barriers short
  if (g_coop_blocks_check > 2 * sms) g_coop_blocks_check = 2 * sms;
  if (g_coop_blocks_fix > 2 * sms) g_coop_blocks_fix = 2 * sms;
  return cudaSuccess;
}

}  // namespace

size_t check_scratch_floats(const Geom& g, int B) {
  size_t worst = 0;
  for (int phase = 0; phase < 2; ++phase) {
    const bool fwd = phase == CODENET_PHASE_FWD;
    const size_t units = fwd ? (size_t)g.n * g.M * g.ns : (size_t)g.m * g.Nn * g.nsc;
    const int slen = fwd ? g.T : g.Tc, dlen = fwd ? g.b_c : g.b_r;
    const size_t ns = 2 * (size_t)((slen + BIG_SR - 1) / BIG_SR) + 2 * (size_t)((dlen + BIG_DC - 1) / BIG_DC);
    if (units * B * ns > worst) worst = units * B * ns;
  }
  return worst;
}

namespace {
// Everything of CheckParams that does not depend on how the kernel is launched.
void fill_check_params(const codenet_layer_impl& L, int phase, const float* src, int src_kind, float* Yw,
                       const float* Vraw, int B, const FaultDev* fault, int have_clean, int commit, float* out,
                       float lr, int update_checksums, codenet_report_t* rep, CheckParams& p) {
  p.g = L.g; p.phase = phase; p.B = B; p.src_kind = src_kind; p.have_clean = have_clean; p.RT = L.bwd_rt;
  p.commit = commit; p.update_checksums = update_checksums; p.lr = lr;
  p.spb = L.g.ldb / backward_strip_elems(L.g.dtype);
  if (fault) p.fault = *fault;
  else { p.fault.seed = 0; p.fault.layer = 0; p.fault.mode = CODENET_FAULT_NONE; p.fault.p_q32 = 0; p.fault.sigma = 0.0f; p.fault.iteration = nullptr; }
  p.src = src; p.Yw = Yw; p.Vraw = Vraw; p.out = out;
  p.Xt = L.ws.Xt; p.Dt = L.ws.Dt; p.dsum = L.ws.dsum; p.xsum = L.ws.xsum;
  p.st = nullptr; p.st_next = nullptr; p.st_base = L.ws.stats; p.parity = L.ws.tc_flag + 1;
  p.plan = L.ws.plan; p.rep = rep; p.tc_flag = L.ws.tc_flag; p.chk = L.ws.chk;
  p.small = L.small; p.dY = L.ws.dY;
  p.out_act = phase == CODENET_PHASE_FWD ? L.out_act : CODENET_ACT_IDENTITY;
  p.out_mask = phase == CODENET_PHASE_BWD ? L.out_mask : nullptr;
  if (phase == CODENET_PHASE_FWD) L.out_act = CODENET_ACT_IDENTITY; else L.out_mask = nullptr;
  p.lazy = 0; p.inline_fix = 0; p.tail_fix = 0; p.bump = nullptr;
  p.it_add = 0u; p.pair = 0; p.pair_sums = nullptr;
  p.commit_S = nullptr; p.commit_S_to = nullptr; p.commit_n = 0; p.commit_rep = nullptr; p.commit_rep_to = nullptr;
  p.loss_partials = nullptr; p.loss_n = 0; p.loss_out = nullptr;
}
}  // namespace

// Both checks of a layer decide something (node check, at most one parity per code: the cooperative pair) ...
bool pair_checks(const codenet_layer_impl& L) {
  const Geom& g = L.g;
  return g.locate_mode == CODENET_LOCATE_NODECHECK && g.r_row <= 1 && g.r_col <= 1 && keeps_checksums(g);
}
// ... or neither does anything but sum (checks switched off, or no code and no node check: the plain pair, which
// cannot inject faults).
static bool pair_sums_only(const codenet_layer_impl& L) {
  const Geom& g = L.g;
  return (g.locate_mode == CODENET_LOCATE_OFF ||
          (g.r_row == 0 && g.r_col == 0 && g.locate_mode != CODENET_LOCATE_NODECHECK)) && !keeps_checksums(g);
}
bool pair_supported(const codenet_layer_impl& L, int B) {
  return L.pair_ok && B == 1 && !L.small.on && (pair_checks(L) || pair_sums_only(L));
}

cudaError_t launch_check_pair(const codenet_layer_impl& L, const float* src, float* Yw, const float* Delta, int B,
                              const FaultDev* fault, float* out, float lr, codenet_report_t* rep,
                              const PairNext& nx, cudaStream_t st) {
  cudaError_t e = coop_grid_limits();
  if (e != cudaSuccess) return e;
  const Geom& g = L.g;
  PairParams pp;
  memset(&pp, 0, sizeof(pp));
  CheckParams& pb = pp.v[0];
  CheckParams& pf = pp.v[1];
  // (the forward part first: it takes the layer's pending activation, as the forward call it stands for would)
  fill_check_params(L, CODENET_PHASE_FWD, L.ws.Ynext, 2, L.ws.Yw2, nx.X_next, B, nx.fault, 1, 0, nx.S_next, 0.0f, 0,
                    nx.rep_next, pf);
  fill_check_params(L, CODENET_PHASE_BWD, src, 1, Yw, Delta, B, fault, 1, 0, out, lr, 1, rep, pb);
  pb.pair = 1; pb.inline_fix = 1;
  pf.pair = 2; pf.inline_fix = 1; pf.it_add = 1u;
  pf.st_base = L.ws.stats + 2; pf.parity = L.ws.tc_flag + 2; pf.plan = L.ws.plan + CODENET_MAX_NODES;
  pf.pair_sums = L.ws.pair_sums;
  pf.commit_S = nx.commit_S; pf.commit_S_to = nx.commit_S_to; pf.commit_n = nx.commit_n;
  pf.commit_rep = nx.commit_rep; pf.commit_rep_to = nx.commit_rep_to;
  pf.loss_partials = nx.loss_partials; pf.loss_n = nx.loss_n; pf.loss_out = nx.loss_out;
  if (L.bump_after != nullptr) { pb.bump = L.bump_after; L.bump_done = true; }
  if (!pair_checks(L)) {
    // nothing to inject and nothing to decide (the caller has made sure of the first): the two sums, one plain launch
    size_t nb = ((size_t)g.n_in * B + CK_THREADS - 1) / CK_THREADS, nf = ((size_t)g.n_out * B + CK_THREADS - 1) / CK_THREADS;
    if (nb > 148 * 4) nb = 148 * 4;
    if (nf > 148 * 4) nf = 148 * 4;
    if (nb < 1) nb = 1;
    if (nf < 2) nf = 2;
    pp.n_first = (int)nb;
    sum_pair_kernel<<<(unsigned)(nb + nf), CK_THREADS, 0, st>>>(pp);
    count_launch();
    return cudaGetLastError();
  }
  // forward part: one warp per unit and one thread per element; backward part: the same and a warp per checksum
  // vector, within what is left of the co-resident limit
  const size_t cap = (size_t)g_coop_blocks_check;
  size_t nf = ((size_t)g.n * g.M * g.ns + CK_WARPS - 1) / CK_WARPS;
  const size_t f_el = ((size_t)g.n * g.b_r * B + CK_THREADS - 1) / CK_THREADS;
  if (f_el > nf) nf = f_el;
  if (nf > cap / 2) nf = cap / 2;
  size_t nb = ((size_t)g.m * g.Nn * g.nsc + CK_WARPS - 1) / CK_WARPS;
  const size_t b_el = ((size_t)g.m * g.b_c * B + CK_THREADS - 1) / CK_THREADS;
  if (b_el > nb) nb = b_el;
  const size_t chk = ((size_t)g.M * g.Nn * ((size_t)g.ns * g.ldb + (size_t)g.nsc * g.b_r) + CK_THREADS - 1) / CK_THREADS;
  if (chk > nb) nb = chk;
  if (nb > cap - nf) nb = cap - nf;
  if (nf < 1 || nb < 1) return cudaErrorLaunchOutOfResources;
  pp.n_first = (int)nb;
  void* args[] = {&pp};
  e = cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(check_pair_kernel), dim3((unsigned)(nb + nf)),
                                  dim3(CK_THREADS), args, 0, st);
  if (e != cudaSuccess) return e;
  count_launch();
  return cudaSuccess;
}

cudaError_t launch_check(const codenet_layer_impl& L, int phase, const float* src, int src_kind, float* Yw,
                         const float* Vraw, int B, const FaultDev* fault, int have_clean, int commit, float* out,
                         float lr, int update_checksums, codenet_report_t* rep, cudaStream_t st, uint32_t it_add) {
  cudaError_t e = coop_grid_limits();
  if (e != cudaSuccess) return e;
  CheckParams p;
  fill_check_params(L, phase, src, src_kind, Yw, Vraw, B, fault, have_clean, commit, out, lr, update_checksums, rep, p);
  p.it_add = it_add;

  const Geom& g = L.g;
  const bool fwd = phase == CODENET_PHASE_FWD;
  const bool phase_unchecked = g.locate_mode == CODENET_LOCATE_OFF ||
                               ((fwd ? g.r_row : g.r_col) == 0 && g.locate_mode != CODENET_LOCATE_NODECHECK);
  if (fault == nullptr && !L.small.on && out != nullptr && have_clean && !commit && phase_unchecked &&
      (!update_checksums || !keeps_checksums(g))) {
    // nothing to inject and nothing to decide: the sums alone, one plain launch (the inner checksums are left
    // alone where nothing can read them: keeps_checksums)
    p.bump = nullptr;
    if (L.bump_after != nullptr && !fwd) { p.bump = L.bump_after; L.bump_done = true; }
    const size_t n = (size_t)(fwd ? g.n_out : g.n_in) * B;
    size_t blocks = (n + CK_THREADS - 1) / CK_THREADS;
    if (blocks > 148 * 8) blocks = 148 * 8;
    sum_outputs_kernel<<<(int)(blocks < 1 ? 1 : blocks), CK_THREADS, 0, st>>>(p);
    count_launch();
    return cudaGetLastError();
  }
  const int n_cw = fwd ? g.n : g.m, K = fwd ? g.M : g.Nn, nsl = fwd ? g.ns : g.nsc;
  const size_t n_el = (size_t)(fwd ? g.b_r : g.b_c) * B;
  // enough CTAs for one warp per unit and one thread per element, within the co-resident limit
  size_t want = ((size_t)n_cw * K * nsl + CK_WARPS - 1) / CK_WARPS;
  const size_t by_el = ((size_t)n_cw * n_el + CK_THREADS - 1) / CK_THREADS;
  if (by_el > want) want = by_el;
  if (B > 8) {
    const size_t items = ((size_t)n_cw * K * nsl * ((B + 7) / 8) + CK_WARPS - 1) / CK_WARPS;  // >= units * B/32
    if (items > want) want = items;
  }
  if (update_checksums) {
    const size_t chk = ((size_t)g.M * g.Nn * ((size_t)g.ns * g.ldb + (size_t)g.nsc * g.b_r) + CK_THREADS - 1) / CK_THREADS;
    if (chk > want) want = chk;
  }
  if (want < (size_t)n_cw) want = (size_t)n_cw;
  // large batches have long phases and many equal work items: use every co-resident CTA so that the
  // items spread evenly; small batches keep the grid (and its barriers) small
  const bool aligned16 = ((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(Yw) |
                           reinterpret_cast<uintptr_t>(p.chk)) & 15) == 0;   // the statistics pass moves 16 bytes per lane
  const bool big = B > 8 && B % 32 == 0 && p.chk != nullptr && src_kind == 0 && aligned16;
  // small batches with at most one parity: no decoding plan has a spare parity to verify, the sums of the
  // few nodes a plan touches are cheap, so the check kernel finishes them itself and no fix kernel follows
  p.lazy = big ? 1 : 0;
  p.bump = nullptr;
  p.inline_fix = (!big && B <= 8 && (fwd ? g.r_row : g.r_col) <= 1 && !commit && out != nullptr) ? 1 : 0;
  // large batches, or two and more parities: the grid waits for the last decision and fixes together (check_body)
  p.tail_fix = ((big || (fwd ? g.r_row : g.r_col) >= 2) && !p.inline_fix && !commit && out != nullptr) ? 1 : 0;
  const size_t cap = big ? (size_t)g_coop_blocks_check_max : (size_t)g_coop_blocks_check;
  int grid_c = (int)(want < cap ? want : cap);
  int grid_f = (int)(by_el < (size_t)g_coop_blocks_fix ? (by_el < 1 ? 1 : by_el) : (size_t)g_coop_blocks_fix);
  if (L.bump_after != nullptr && !fwd && (p.inline_fix || p.tail_fix)) {   // (with a fix kernel behind, the counter is still read)
    p.bump = L.bump_after;
    L.bump_done = true;
  }
  void* args[] = {&p};
  e = cudaLaunchCooperativeKernel(big ? reinterpret_cast<const void*>(check_kernel<true>)
                                      : reinterpret_cast<const void*>(check_kernel<false>),
                                  dim3(grid_c), dim3(CK_THREADS), args, 0, st);
  if (e != cudaSuccess) return e;
  count_launch();
  if (p.inline_fix || p.tail_fix) return cudaSuccess;   // the check kernel has done what the fix kernel would do
  if ((fwd ? g.r_row : g.r_col) >= 2) {
    e = cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(fix_kernel<true>), dim3(grid_f), dim3(CK_THREADS), args, 0, st);
  } else {
    // at most one parity: no plan has a spare one, no barrier inside, a plain launch
    fix_kernel<false><<<grid_f, CK_THREADS, 0, st>>>(p);
    e = cudaGetLastError();
  }
  count_launch();
  return e;
}

cudaError_t launch_input_faults(const codenet_layer_impl& L, int B, cudaStream_t st) {
  const Geom& g = L.g;
  if (!L.small.on || L.small.p_input == 0u || L.ws.dY == nullptr) return cudaSuccess;
  cudaError_t e = cudaMemsetAsync(L.ws.dY, 0, (size_t)g.n * g.Mbr * B * sizeof(float), st);
  if (e != cudaSuccess) return e;
  dim3 grid(g.n * g.M, (g.b_c + 31) / 32);
  input_fault_kernel<<<grid, 256, (size_t)32 * B * sizeof(float), st>>>(g, L.small, B, L.ws.dY);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_sum_outputs(const Geom& g, int phase, int B, const float* Y, float* out, int out_act,
                               codenet_report_t* rep, cudaStream_t st) {
  CheckParams p;
  memset(&p, 0, sizeof(p));
  p.g = g; p.phase = phase; p.B = B; p.src = Y; p.src_kind = 0; p.out = out; p.rep = rep; p.out_act = out_act;
  const size_t n = (size_t)(phase == CODENET_PHASE_FWD ? g.n_out : g.n_in) * B;
  size_t blocks = (n + CK_THREADS - 1) / CK_THREADS;
  if (blocks > 148 * 8) blocks = 148 * 8;
  if (blocks < 1) blocks = 1;
  sum_outputs_kernel<<<(int)blocks, CK_THREADS, 0, st>>>(p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace codenet

