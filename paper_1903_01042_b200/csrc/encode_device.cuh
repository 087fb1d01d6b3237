// Additional encoding of the vectors (Step 4 of the feedforward / backpropagation stages) as a device function, so
// that the stand-alone kernel and the update sweep that carries the encoding along (kernels_stream.cu) run the same
// code.  Included inside namespace codenet { namespace { of the including file.

// Operand copies for the fused tensor-core kernel, written with the vectors themselves (16-byte path only):
// TF32: the transposes xT (ld, B) and dT (Mbr, B); bf16: x~ rounded to bfloat16 (B, ld) and delta~ as a
// hi / lo pair (hi at the vector's index, lo `dcount` elements further).
struct EmitOperands {
  float* xT; float* dT;
  __nv_bfloat16* xb; __nv_bfloat16* dpair;
  size_t dcount;
  float4* clear; size_t clear_n16;   // a buffer to fill with zeros on the way (16-byte units), or NULL
};

// Everything the encoding needs besides the layer's geometry.
struct EncodeArgs {
  const float* X; const float* Delta; int B;
  float* Xt; float* Dt; float* dsum; float* xsum;
  int vec_ok;
  LossFuse lf; EmitOperands em; SmallDev sf;
};

// cta / n_cta: index of this CTA among the encoding CTAs and their number (128 threads each).
__device__ __forceinline__ void encode_vectors_body(const Geom& g, const EncodeArgs& ea, const int cta, const int n_cta) {
  const float* __restrict__ X = ea.X; const float* __restrict__ Delta = ea.Delta;
  const int B = ea.B, vec_ok = ea.vec_ok;
  float* __restrict__ Xt = ea.Xt; float* __restrict__ Dt = ea.Dt; float* __restrict__ dsum = ea.dsum; float* __restrict__ xsum = ea.xsum;
  const LossFuse& lf = ea.lf; const EmitOperands& em = ea.em; const SmallDev& sf = ea.sf;
  __shared__ float red[4];
  __shared__ int s_last, s_enc_hit;
  if (em.clear != nullptr)
    for (size_t c = cta * (size_t)blockDim.x + threadIdx.x; c < em.clear_n16; c += (size_t)n_cta * blockDim.x)
      em.clear[c] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
  const int nxseg = X ? g.Nn * g.nsc * B : 0;
  int seg = cta;
  float part = 0.0f, loss_part = 0.0f;
  float* sum_out;
  // one segment per CTA.  src: the raw vector of batch entry b; kd data sub-vectors of length len (padded
  // length ldl in the encoded vector), P the parity part of the generator, k the coded index, [e0, e1) the
  // entries of the segment; entries past len (alignment padding) are written as zeros.
  const float* src; float* dst; const float* P;
  int kd, r, k, len, n_src, e0, e1;
  // lf.S != NULL: the delta segments take delta^L = 2 (y - s) / (N B) straight from the last layer's sums and
  // the target (mean-squared-error loss), the data segments also store it and gather the loss
  const float *fy = nullptr, *fs = nullptr;
  float* fd = nullptr;
  int loss_id = -1;
  float* tr = nullptr;              // transposed copy: entry e of this segment goes to tr[e * B]
  __nv_bfloat16* b16 = nullptr;     // bfloat16 copy of the segment (+ lo part lo_off further, if not 0)
  size_t lo_off = 0;
  if (seg < nxseg) {
    const int b = seg % B, js = seg / B;
    const int j = js / g.nsc, sl = js % g.nsc;
    src = X + (size_t)b * g.n_in; dst = Xt + (size_t)b * g.ld + (size_t)j * g.ldb; P = g.Pc;
    kd = g.n; r = g.r_col; k = j; len = g.b_c; n_src = g.n_in;
    e0 = sl * g.Tc; e1 = sl == g.nsc - 1 ? g.ldb : (sl + 1) * g.Tc;   // the last slice also clears the padding
    sum_out = xsum + (size_t)js * B + b;
    if (em.xT) tr = em.xT + (size_t)j * g.ldb * B + b;
    if (em.xb) b16 = em.xb + (size_t)b * g.ld + (size_t)j * g.ldb;
  } else {
    seg -= nxseg;
    const int b = seg % B, is = seg / B;
    const int i = is / g.ns, sl = is % g.ns;
    src = Delta + (size_t)b * g.n_out; dst = Dt + (size_t)b * g.Mbr + (size_t)i * g.b_r; P = g.Pr;
    kd = g.m; r = g.r_row; k = i; len = g.b_r; n_src = g.n_out;
    e0 = sl * g.T; e1 = (sl + 1) * g.T;
    sum_out = dsum + (size_t)is * B + b;
    if (em.dT) tr = em.dT + (size_t)i * g.b_r * B + b;
    if (em.dpair) { b16 = em.dpair + (size_t)b * g.Mbr + (size_t)i * g.b_r; lo_off = em.dcount; }
    if (lf.S != nullptr) {
      fy = lf.target + (size_t)b * g.n_out; fs = lf.S + (size_t)b * g.n_out; fd = lf.delta + (size_t)b * g.n_out;
      if (i < g.m) loss_id = (i * g.ns + sl) * B + b;
    }
  }
  // soft error in the additional encoding: the whole parity sub-vector of a hit unit is off by noise
  const int seg_b = (cta < nxseg ? cta : cta - nxseg) % B;
  const uint32_t enc_unit = cta < nxseg ? (uint32_t)k : (uint32_t)(g.Nn + k);
  const uint32_t enc_it = sf.iteration ? *sf.iteration : 0u;
  if (threadIdx.x == 0) s_enc_hit = (k >= kd && small_is_hit(sf, CODENET_PHASE_ENCODE, enc_it, enc_unit)) ? 1 : 0;
  __syncthreads();
  const bool enc_hit = s_enc_hit != 0;
  const uint32_t enc_key = (sf.layer << 8) | (uint32_t)CODENET_PHASE_ENCODE;
  const float scale = lf.scale;
  if (vec_ok) {
    // four entries per thread and step: lengths, offsets and pointers are multiples of four floats
    auto load4 = [&](int gi, bool store) {
      if (fy == nullptr) return *reinterpret_cast<const float4*>(src + gi);
      const float4 y = *reinterpret_cast<const float4*>(fy + gi), sv = *reinterpret_cast<const float4*>(fs + gi);
      const float d0 = y.x - sv.x, d1 = y.y - sv.y, d2 = y.z - sv.z, d3 = y.w - sv.w;
      const float4 d = make_float4(2.0f * d0 * scale, 2.0f * d1 * scale, 2.0f * d2 * scale, 2.0f * d3 * scale);
      if (store) {
        *reinterpret_cast<float4*>(fd + gi) = d;
        loss_part = fmaf(d0 * d0, scale, loss_part); loss_part = fmaf(d1 * d1, scale, loss_part);
        loss_part = fmaf(d2 * d2, scale, loss_part); loss_part = fmaf(d3 * d3, scale, loss_part);
      }
      return d;
    };
    for (int e = e0 + 4 * threadIdx.x; e < e1; e += 4 * blockDim.x) {
      float4 v = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
      if (e < len) {
        if (k < kd) {
          if (k * len + e < n_src) v = load4(k * len + e, true);
        } else {
          for (int q = 0; q < kd; ++q) {
            if (q * len + e >= n_src) break;
            const float c = P[q * r + (k - kd)];
            const float4 t = load4(q * len + e, false);
            v.x = fmaf(c, t.x, v.x); v.y = fmaf(c, t.y, v.y); v.z = fmaf(c, t.z, v.z); v.w = fmaf(c, t.w, v.w);
          }
        }
      }
      if (enc_hit && e < len) {
        v.x = __fadd_rn(v.x, soft_error_noise(sf.seed, enc_key, enc_it, enc_unit, (uint32_t)(e * B + seg_b), sf.sigma));
        v.y = __fadd_rn(v.y, soft_error_noise(sf.seed, enc_key, enc_it, enc_unit, (uint32_t)((e + 1) * B + seg_b), sf.sigma));
        v.z = __fadd_rn(v.z, soft_error_noise(sf.seed, enc_key, enc_it, enc_unit, (uint32_t)((e + 2) * B + seg_b), sf.sigma));
        v.w = __fadd_rn(v.w, soft_error_noise(sf.seed, enc_key, enc_it, enc_unit, (uint32_t)((e + 3) * B + seg_b), sf.sigma));
      }
      *reinterpret_cast<float4*>(dst + e) = v;
      if (tr) {
        float* t = tr + (size_t)e * B;
        t[0] = v.x; t[B] = v.y; t[2 * (size_t)B] = v.z; t[3 * (size_t)B] = v.w;
      }
      if (b16) {
        const __nv_bfloat16 h0 = __float2bfloat16_rn(v.x), h1 = __float2bfloat16_rn(v.y);
        const __nv_bfloat16 h2 = __float2bfloat16_rn(v.z), h3 = __float2bfloat16_rn(v.w);
        __nv_bfloat162 hi[2] = {__nv_bfloat162(h0, h1), __nv_bfloat162(h2, h3)};
        *reinterpret_cast<uint2*>(b16 + e) = *reinterpret_cast<uint2*>(hi);
        if (lo_off) {
          __nv_bfloat162 lo[2] = {__nv_bfloat162(__float2bfloat16_rn(v.x - __bfloat162float(h0)),
                                                 __float2bfloat16_rn(v.y - __bfloat162float(h1))),
                                  __nv_bfloat162(__float2bfloat16_rn(v.z - __bfloat162float(h2)),
                                                 __float2bfloat16_rn(v.w - __bfloat162float(h3)))};
          *reinterpret_cast<uint2*>(b16 + lo_off + e) = *reinterpret_cast<uint2*>(lo);
        }
      }
      part += (v.x + v.y) + (v.z + v.w);
    }
  } else {
    auto load1 = [&](int gi, bool store) {
      if (fy == nullptr) return src[gi];
      const float d0 = fy[gi] - fs[gi];
      const float d = 2.0f * d0 * scale;
      if (store) { fd[gi] = d; loss_part = fmaf(d0 * d0, scale, loss_part); }
      return d;
    };
    for (int e = e0 + threadIdx.x; e < e1; e += blockDim.x) {
      float v = 0.0f;
      if (e < len) {
        if (k < kd) {
          const int gi = k * len + e;
          v = gi < n_src ? load1(gi, true) : 0.0f;
        } else {
          for (int q = 0; q < kd; ++q) {
            const int gi = q * len + e;
            if (gi < n_src) v = fmaf(P[q * r + (k - kd)], load1(gi, false), v);
          }
        }
      }
      if (enc_hit && e < len) v = __fadd_rn(v, soft_error_noise(sf.seed, enc_key, enc_it, enc_unit, (uint32_t)(e * B + seg_b), sf.sigma));
      dst[e] = v;
      part += v;
    }
  }
  part = warp_sum(part);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = part;
  __syncthreads();
  if (threadIdx.x == 0) *sum_out = red[0] + red[1] + red[2] + red[3];
  if (lf.S == nullptr) return;
  // the loss: one partial per data segment of delta, added by the last CTA to finish in a fixed order
  loss_part = warp_sum(loss_part);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = loss_part;
  __syncthreads();
  if (lf.defer) {   // a later kernel of the step adds the partials up, in the order used below
    if (threadIdx.x == 0 && loss_id >= 0) lf.partials[loss_id] = red[0] + red[1] + red[2] + red[3];
    return;
  }
  if (threadIdx.x == 0) {
    if (loss_id >= 0) lf.partials[loss_id] = red[0] + red[1] + red[2] + red[3];
    __threadfence();
    s_last = atomicAdd(lf.counter, 1u) == (unsigned)n_cta - 1 ? 1 : 0;
  }
  __syncthreads();
  if (s_last) {
    __threadfence();
    float t = 0.0f;
    for (int idx = threadIdx.x; idx < lf.n_part; idx += blockDim.x) t += __ldcg(&lf.partials[idx]);
    t = warp_sum(t);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = t;
    __syncthreads();
    if (threadIdx.x == 0) {
      if (lf.loss_out) *lf.loss_out = red[0] + red[1] + red[2] + red[3];
      *lf.counter = 0u;
    }
  }
}

