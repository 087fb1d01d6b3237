// Tensor-core tiles for batches >= 64 (sm_100a): tcgen05.mma with accumulators in tensor memory,
// operands staged in shared memory by TMA (cp.async.bulk.tensor, every CTA loading its own tiles), an mbarrier ring
// between a producer warp, an MMA warp and four epilogue warps.
//
// Forward node products (step O1):  Y[j][coded row][b] = sum_c W~[coded row][j*ldb + c] X[b][j*ldb + c]
// is, per block-column j, a (M*b_r) x b_c by b_c x B product: tile M = 128 coded rows, N = B, K = b_c.
// Both operands are K-major (W~ is row-major, X is (B, columns) row-major), 128-byte swizzled.
// A CTA owns MT row tiles so that each staged X slice is used MT times.  With bfloat16 blocks X is
// staged as a bfloat16 pair x = hi + lo (two instructions per K step into the same accumulator):
// rounding x to one bfloat16 alone would cost 2^-9 per element, about 2e-3 of the output.
//
// Backward node products (step O2):  Z[i][j][col][b] = sum_row W~[i*b_r + row][col] Delta[b][i*b_r + row]
// uses the same pipeline with tile M = 128 columns of W~, N = B, K = the b_r rows of block-row i.  Here
// the W~ tile is the M-major operand (its rows are K): TMA brings it as 128-byte column chunks of KT
// rows, and the descriptor says "MN-major" (chunks KT*128 bytes apart, 8-row groups 1024 bytes apart).
//
// Every wait on an mbarrier is bounded; a wait that runs out sets a device flag, and the kernel
// still releases its tensor memory and returns.
#include "codenet_internal.cuh"

#include <cuda.h>

namespace codenet {
namespace {

constexpr int TC_THREADS = 192;          // warp 0: TMA producer, warp 1: MMA issuer, warps 2..5: epilogue
constexpr int TC_TILE_M = 128;
constexpr int TC_KBYTES = 128;           // one 128-byte swizzle atom of K per stage
constexpr uint32_t TC_SPIN_LIMIT = 1u << 24;
// How long a stuck wait keeps trying before it gives up (codenet_set_wait_limit; about a second unless set), and a
// diagnostic switch: the producer warp of the forward product kernel issues no tile loads at all, so that the waits
// that depend on them run out (codenet_withhold_tile_loads: exercises the give-up path without any fault).
__constant__ unsigned long long c_wait_ns = 1000000000ull;
__constant__ int c_withhold_loads = 0;

// ---- PTX wrappers -----------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Bounded wait: returns false if the phase did not complete within about a second.  The limit is in
// time, not in polls: one try_wait may itself suspend the thread for a while, so a poll count says
// little about how long a stuck pipeline keeps the kernel alive.
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  const uint32_t addr = smem_u32(bar);
  unsigned long long t0 = 0;
  for (uint32_t spin = 0; spin < TC_SPIN_LIMIT; ++spin) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(addr), "r"(parity) : "memory");
    if (done) return true;
    if ((spin & 1023u) == 1023u) {
      const unsigned long long now = global_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > c_wait_ns) return false;
    }
  }
  return false;
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y) : "memory");
}
// The same with an L2 eviction policy (createpolicy): the coded weights stream through once per kernel, evict-first
// keeps them from pushing out what is read again and again (the operand tiles, the node outputs the check kernel reads
// next, and the instructions of the kernels that follow, which live in the same cache).
__device__ __forceinline__ uint64_t l2_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void tma_load_2d_hint(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y), "l"(pol) : "memory");
}
// Tile from shared memory back to global memory (bulk group of the issuing thread), same policy.
__device__ __forceinline__ void tma_store_2d_hint(const CUtensorMap* map, int x, int y, const void* src, uint64_t pol) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group.L2::cache_hint [%0, {%2, %3}], [%1], %4;"
               ::"l"(map), "r"(smem_u32(src)), "r"(x), "r"(y), "l"(pol) : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// the stores committed so far have read their shared-memory source (it may be overwritten)
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// ... and have been written to global memory
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// writes to shared memory by this thread become visible to the TMA engine
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t* slot, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
template <bool TF32>
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  if (TF32)
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
  else
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory operand descriptor: K-major tile, rows of 128 bytes, 128-byte swizzle, 8-row groups
// 1024 bytes apart (stride byte offset); the leading byte offset is unused for this layout.
__device__ __forceinline__ uint64_t smem_desc_k128(const void* tile) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_u32(tile) & 0x3FFFFu) >> 4);   // start address
  d |= (uint64_t)1 << 16;                              // leading byte offset (ignored), 16 bytes
  d |= (uint64_t)(1024 >> 4) << 32;                    // stride byte offset
  d |= (uint64_t)1 << 46;                              // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                              // 128-byte swizzle
  return d;
}

// The same for an MN-major tile stored as 128-byte chunks along M (or N), each chunk holding all K
// rows of the stage: chunks `chunk_bytes` apart (leading byte offset).  16-bit elements: plain
// 128-byte swizzle, 8-row K groups 1024 bytes apart.  32-bit elements: the 128-byte swizzle with 32-byte
// atoms (the TMA map must use the same mode), 4-row K groups 512 bytes apart -- the only combination
// that multiplied correctly on a B200 (the plain 128-byte swizzle reads nothing for tf32 here).
template <bool TF32>
__device__ __forceinline__ uint64_t smem_desc_mn128(const void* tile, uint32_t chunk_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_u32(tile) & 0x3FFFFu) >> 4);
  d |= (uint64_t)((chunk_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((TF32 ? 512 : 1024) >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)(TF32 ? 1 : 2) << 61;
  return d;
}

// Instruction descriptor: fp32 accumulator; A K-major or M-major, B K-major.
__host__ __device__ constexpr uint32_t instr_desc(bool tf32, int M, int N, bool a_mn_major = false,
                                                  bool b_mn_major = false) {
  const uint32_t fmt = tf32 ? 2u : 1u;  // kind::tf32: TF32; kind::f16: BF16
  return (1u << 4) | (fmt << 7) | (fmt << 10) | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16) |
         ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

struct TcFwdParams {
  Geom g;
  int B, ksteps;      // ksteps: 128-byte K slices per block-column
  float* Y;
  int* flag;          // set to 1 when a bounded wait runs out
};

template <bool TF32, int MT, int SPLIT, int STAGES, bool BWD>
__global__ void __launch_bounds__(TC_THREADS, 1)
tc_products_kernel(const __grid_constant__ CUtensorMap mapW, const __grid_constant__ CUtensorMap mapX, TcFwdParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const int N = p.B;
  const uint32_t a_tile = TC_TILE_M * TC_KBYTES, a_bytes = MT * a_tile;
  const uint32_t b_tile = (uint32_t)N * TC_KBYTES, b_bytes = SPLIT * b_tile;
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* sA = base;                          // [STAGES][MT][128 rows][128 bytes]
  uint8_t* sB = base + (size_t)STAGES * a_bytes;  // [STAGES][SPLIT][N rows][128 bytes]
  __shared__ uint64_t full[STAGES], empty[STAGES], accum_full;
  __shared__ uint32_t tmem_slot;
  __shared__ int s_fail;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row0 = blockIdx.x * (MT * TC_TILE_M), j = blockIdx.y;  // BWD: row0 is a column origin, j a block-row
  constexpr int elems_per_kstep = TC_KBYTES / (TF32 ? 4 : 2);  // K elements per stage = elements per 128-byte chunk
  constexpr int CH = TC_TILE_M / elems_per_kstep;                 // BWD: 128-byte column chunks per tile
  constexpr uint32_t chunk_bytes = elems_per_kstep * TC_KBYTES;   // BWD: KT rows of 128 bytes
  uint32_t ncols = 32;
  while (ncols < (uint32_t)(MT * N)) ncols <<= 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(&accum_full, 1);
    s_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(&tmem_slot, ncols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_slot;

  if (warp == 0 && lane == 0) {
    // ---- TMA producer ----
    const uint64_t w_pol = l2_evict_first();
    for (int k = 0; k < (c_withhold_loads ? 0 : p.ksteps); ++k) {
      const int s = k % STAGES;
      if (k >= STAGES && !mbar_wait(&empty[s], ((k / STAGES) - 1) & 1)) { s_fail = 1; break; }
      mbar_expect_tx(&full[s], a_bytes + b_bytes);
      if (!BWD) {
        const int x = j * p.g.ldb + k * elems_per_kstep;
#pragma unroll
        for (int t = 0; t < MT; ++t) tma_load_2d_hint(sA + (size_t)s * a_bytes + t * a_tile, &mapW, x, row0 + t * TC_TILE_M, &full[s], w_pol);
#pragma unroll
        for (int h = 0; h < SPLIT; ++h) tma_load_2d(sB + (size_t)s * b_bytes + h * b_tile, &mapX, x, h * N, &full[s]);
      } else {
        const int y = j * p.g.b_r + k * elems_per_kstep;  // first of the KT coded rows of this stage
#pragma unroll
        for (int t = 0; t < MT; ++t)
#pragma unroll
          for (int ch = 0; ch < CH; ++ch)
            tma_load_2d_hint(sA + (size_t)s * a_bytes + t * a_tile + ch * chunk_bytes, &mapW,
                             row0 + t * TC_TILE_M + ch * elems_per_kstep, y, &full[s], w_pol);
#pragma unroll
        for (int h = 0; h < SPLIT; ++h) tma_load_2d(sB + (size_t)s * b_bytes + h * b_tile, &mapX, y, h * N, &full[s]);
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ---- MMA issuer ----
    const uint32_t idesc = instr_desc(TF32, TC_TILE_M, N, BWD);
    bool ok = true;
    for (int k = 0; k < p.ksteps && ok; ++k) {
      const int s = k % STAGES;
      if (!mbar_wait(&full[s], (k / STAGES) & 1)) { s_fail = 1; ok = false; break; }
      tc_fence_after();
#pragma unroll
      for (int t = 0; t < MT; ++t) {
        const uint64_t da = BWD ? smem_desc_mn128<TF32>(sA + (size_t)s * a_bytes + t * a_tile, chunk_bytes)
                                : smem_desc_k128(sA + (size_t)s * a_bytes + t * a_tile);
        // K advance per instruction: 32 bytes inside a K-major row, or 16 / 8 rows of an MN-major tile
        constexpr uint64_t a_step = BWD ? (uint64_t)((TF32 ? 8 : 16) * TC_KBYTES >> 4) : 2;
#pragma unroll
        for (int h = 0; h < SPLIT; ++h) {
          const uint64_t db = smem_desc_k128(sB + (size_t)s * b_bytes + h * b_tile);
#pragma unroll
          for (int kk = 0; kk < TC_KBYTES / 32; ++kk)  // one instruction consumes 32 bytes of K
            tc_mma<TF32>(tmem + (uint32_t)(t * N), da + (uint64_t)kk * a_step, db + (uint64_t)(kk * 2), idesc,
                         (k > 0 || kk > 0 || h > 0) ? 1u : 0u);
        }
      }
      tc_commit(&empty[s]);   // the stage is free once these instructions have read it
    }
    tc_commit(&accum_full);   // arrives when every instruction issued above has completed
  } else if (warp >= 2) {
    // ---- epilogue: tensor memory -> registers -> Y ----
    bool ok = mbar_wait(&accum_full, 0);
    if (!ok) s_fail = 1;
    tc_fence_after();
    if (*reinterpret_cast<volatile int*>(&s_fail)) ok = false;   // the multiplication gave up: nothing to read back
    const int quad = warp & 3;                   // the lane quadrant this warp may read
    if (ok) {
      for (int tc = 0; tc < MT * N; tc += 32) {
        const int t = tc / N, c0 = tc % N;
        const int gr = row0 + t * TC_TILE_M + quad * 32 + lane;
        uint32_t r[32];
        tmem_ld32(tmem + ((uint32_t)(quad * 32) << 16) + (uint32_t)tc, r);
        bool valid;
        size_t off;
        if (!BWD) {
          valid = gr < p.g.Mbr;
          off = ((size_t)j * p.g.Mbr + gr) * p.B + c0;
        } else {  // gr is a coded column: node = its block-column, position inside the block
          const int node = gr / p.g.ldb, c = gr % p.g.ldb;
          valid = gr < p.g.ld && c < p.g.b_c;
          off = (((size_t)j * p.g.Nn + node) * p.g.b_c + c) * p.B + c0;
        }
        if (valid) {
          float4* dst = reinterpret_cast<float4*>(p.Y + off);
#pragma unroll
          for (int q = 0; q < 8; ++q)
            dst[q] = make_float4(__uint_as_float(r[4 * q]), __uint_as_float(r[4 * q + 1]),
                                 __uint_as_float(r[4 * q + 2]), __uint_as_float(r[4 * q + 3]));
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && s_fail) atomicExch(p.flag, 1);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, ncols);
  }
}

// X (B, n_in) fp32 -> padded operand (B, n*ldb), zero where a block is padded: fp32 as it is, or a
// bfloat16 pair hi (rows 0..B-1) and lo = x - hi (rows B..2B-1).
template <typename T>
__global__ void tc_prep_x_kernel(Geom g, const float* __restrict__ X, int B, T* __restrict__ out) {
  const size_t ldo = (size_t)g.n * g.ldb;
  for (size_t idx = blockIdx.x * (size_t)blockDim.x + threadIdx.x; idx < (size_t)B * ldo;
       idx += (size_t)gridDim.x * blockDim.x) {
    const int b = (int)(idx / ldo), gc = (int)(idx % ldo);
    const int j = gc / g.ldb, c = gc % g.ldb;
    const int src = j * g.b_c + c;
    const float v = (c < g.b_c && src < g.n_in) ? X[(size_t)b * g.n_in + src] : 0.0f;
    if (sizeof(T) == 4) {
      out[idx] = (T)v;
    } else {
      const T hi = (T)v;
      out[idx] = hi;
      out[idx + (size_t)B * ldo] = (T)(v - (float)hi);
    }
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// 2-D K-major tensor map: `rows` rows of `cols` elements (row stride ld elements), box = 128 bytes x box_rows.
bool make_map(CUtensorMap* map, const void* base, bool fp32, size_t rows, size_t cols, size_t ld, int box_rows,
              bool atom32 = false) {
  if (box_rows > 256) return false;
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const size_t esz = fp32 ? 4 : 2;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)(ld * esz)};
  cuuint32_t box[2] = {(cuuint32_t)(TC_KBYTES / esz), (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, fp32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
            const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            atom32 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool tc_forward_supported(const Geom& g, int math, int B) {
  if (math == CODENET_MATH_FFMA) return false;
  const bool tf32 = g.dtype == CODENET_F32;
  if (tf32 != (math == CODENET_MATH_TF32)) return false;  // TF32 tiles read fp32 blocks, BF16 tiles bf16 blocks
  const int kelems = TC_KBYTES / (tf32 ? 4 : 2);
  return B >= 64 && B <= 128 && B % 32 == 0 && g.ldb % kelems == 0 && g.Mbr >= TC_TILE_M && encode_tiled_fn() != nullptr;
}

cudaError_t launch_tc_forward(const codenet_layer_impl& L, const float* X, int B, float* Y, cudaStream_t st) {
  const Geom& g = L.g;
  const bool tf32 = g.dtype == CODENET_F32;
  const size_t ldo = (size_t)g.n * g.ldb;
  // operand X in the multiplication type, padded like the blocks; fp32 inputs whose sub-vectors are not
  // padded apart are read where they are (TF32 takes the fp32 bits as they come)
  const bool in_place = tf32 && g.ldb == g.b_c && (size_t)g.n * g.b_c == (size_t)g.n_in &&
                        (reinterpret_cast<uintptr_t>(X) & 15u) == 0;
  if (!in_place) {
    const int pgrid = (int)(((size_t)B * ldo + 255) / 256 < 148 * 8 ? ((size_t)B * ldo + 255) / 256 : 148 * 8);
    if (tf32) tc_prep_x_kernel<float><<<pgrid, 256, 0, st>>>(g, X, B, reinterpret_cast<float*>(L.ws.tc_x));
    else tc_prep_x_kernel<__nv_bfloat16><<<pgrid, 256, 0, st>>>(g, X, B, reinterpret_cast<__nv_bfloat16*>(L.ws.tc_x));
    count_launch();
  }
  CUtensorMap mapW, mapX;
  if (!make_map(&mapW, g.Wt, tf32, (size_t)g.Mbr, (size_t)g.ld, (size_t)g.ld, TC_TILE_M)) return cudaErrorInvalidValue;
  if (!make_map(&mapX, in_place ? static_cast<const void*>(X) : L.ws.tc_x, tf32, (size_t)(tf32 ? B : 2 * B), ldo, ldo, B))
    return cudaErrorInvalidValue;
  TcFwdParams p;
  p.g = g; p.B = B; p.ksteps = g.ldb / (TC_KBYTES / (tf32 ? 4 : 2)); p.Y = Y; p.flag = L.ws.tc_flag;
  cudaError_t e;
  ProfileScope scope(CODENET_KERNEL_FORWARD, st);
  if (tf32) {
    int sms = 148, dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    constexpr int SPLIT = 1, STAGES = 4;
    const long ctas2 = (long)((g.Mbr + 2 * TC_TILE_M - 1) / (2 * TC_TILE_M)) * g.n;
    if (ctas2 * 4 < (long)sms * 3) {
      // two row tiles per CTA would leave a quarter of the SMs and more without one (configuration 5: 80 CTAs):
      // one tile per CTA, two CTAs fit an SM
      constexpr int MT = 1;
      const size_t smem = (size_t)STAGES * (MT * TC_TILE_M + SPLIT * B) * TC_KBYTES + 1024;
      dim3 grid((g.Mbr + MT * TC_TILE_M - 1) / (MT * TC_TILE_M), g.n);
      e = cudaFuncSetAttribute(tc_products_kernel<true, MT, SPLIT, STAGES, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
      tc_products_kernel<true, MT, SPLIT, STAGES, false><<<grid, TC_THREADS, smem, st>>>(mapW, mapX, p);
    } else {
      constexpr int MT = 2;
      const size_t smem = (size_t)STAGES * (MT * TC_TILE_M + SPLIT * B) * TC_KBYTES + 1024;
      dim3 grid((g.Mbr + MT * TC_TILE_M - 1) / (MT * TC_TILE_M), g.n);
      e = cudaFuncSetAttribute(tc_products_kernel<true, MT, SPLIT, STAGES, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
      tc_products_kernel<true, MT, SPLIT, STAGES, false><<<grid, TC_THREADS, smem, st>>>(mapW, mapX, p);
    }
  } else {
    // Two or three 128-row tiles per CTA.  The kernel sits at the bandwidth between L2 and the SM (the hi + lo
    // operand tiles of a K step are as many bytes as two weight tiles), so what a K step moves per weight tile
    // and how evenly the CTAs fill the SMs decide: estimated time = waves x bytes per K step of one CTA.
    constexpr int SPLIT = 2;
    int sms = 148, dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    auto cost = [&](int mt) {
      const long ctas = (long)((g.Mbr + mt * TC_TILE_M - 1) / (mt * TC_TILE_M)) * g.n;
      return ((ctas + sms - 1) / sms) * (long)(mt * TC_TILE_M + SPLIT * B);
    };
    if (cost(3) < cost(2)) {
      constexpr int MT = 3, STAGES = 2;
      const size_t smem = (size_t)STAGES * (MT * TC_TILE_M + SPLIT * B) * TC_KBYTES + 1024;
      dim3 grid((g.Mbr + MT * TC_TILE_M - 1) / (MT * TC_TILE_M), g.n);
      e = cudaFuncSetAttribute(tc_products_kernel<false, MT, SPLIT, STAGES, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
      tc_products_kernel<false, MT, SPLIT, STAGES, false><<<grid, TC_THREADS, smem, st>>>(mapW, mapX, p);
    } else {
      constexpr int MT = 2, STAGES = 3;
      const size_t smem = (size_t)STAGES * (MT * TC_TILE_M + SPLIT * B) * TC_KBYTES + 1024;
      dim3 grid((g.Mbr + MT * TC_TILE_M - 1) / (MT * TC_TILE_M), g.n);
      e = cudaFuncSetAttribute(tc_products_kernel<false, MT, SPLIT, STAGES, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
      tc_products_kernel<false, MT, SPLIT, STAGES, false><<<grid, TC_THREADS, smem, st>>>(mapW, mapX, p);
    }
  }
  count_launch();
  return cudaGetLastError();
}

// Delta~ (B, M*b_r) fp32 (already encoded) -> operand in the multiplication type: fp32, or a bfloat16
// pair hi (rows 0..B-1), lo (rows B..2B-1).
template <typename T>
__global__ void tc_prep_d_kernel(const float* __restrict__ Dt, size_t count, T* __restrict__ out) {
  for (size_t idx = blockIdx.x * (size_t)blockDim.x + threadIdx.x; idx < count; idx += (size_t)gridDim.x * blockDim.x) {
    const float v = Dt[idx];
    if (sizeof(T) == 4) {
      out[idx] = (T)v;
    } else {
      const T hi = (T)v;
      out[idx] = hi;
      out[idx + count] = (T)(v - (float)hi);
    }
  }
}

bool tc_backward_supported(const Geom& g, int math, int B) {
  if (!tc_forward_supported(g, math, B)) return false;
  const int kt = TC_KBYTES / (g.dtype == CODENET_F32 ? 4 : 2);
  return g.b_r % kt == 0 && g.ld >= TC_TILE_M;
}

cudaError_t launch_tc_backward(const codenet_layer_impl& L, int B, float* Z, cudaStream_t st) {
  const Geom& g = L.g;
  const bool tf32 = g.dtype == CODENET_F32;
  const size_t count = (size_t)B * g.Mbr;
  const int pgrid = (int)((count + 255) / 256 < 148 * 8 ? (count + 255) / 256 : 148 * 8);
  if (tf32) tc_prep_d_kernel<float><<<pgrid, 256, 0, st>>>(L.ws.Dt, count, reinterpret_cast<float*>(L.ws.tc_d));
  else tc_prep_d_kernel<__nv_bfloat16><<<pgrid, 256, 0, st>>>(L.ws.Dt, count, reinterpret_cast<__nv_bfloat16*>(L.ws.tc_d));
  count_launch();
  const int kt = TC_KBYTES / (tf32 ? 4 : 2);
  CUtensorMap mapW, mapD;
  if (!make_map(&mapW, g.Wt, tf32, (size_t)g.Mbr, (size_t)g.ld, (size_t)g.ld, kt, tf32)) return cudaErrorInvalidValue;
  if (!make_map(&mapD, L.ws.tc_d, tf32, (size_t)(tf32 ? B : 2 * B), (size_t)g.Mbr, (size_t)g.Mbr, B)) return cudaErrorInvalidValue;
  TcFwdParams p;
  p.g = g; p.B = B; p.ksteps = g.b_r / kt; p.Y = Z; p.flag = L.ws.tc_flag;
  cudaError_t e;
  ProfileScope scope(CODENET_KERNEL_BACKWARD, st);
  if (tf32) {
    constexpr int MT = 2, SPLIT = 1, STAGES = 4;
    const size_t smem = (size_t)STAGES * (MT * TC_TILE_M + SPLIT * B) * TC_KBYTES + 1024;
    dim3 grid((g.ld + MT * TC_TILE_M - 1) / (MT * TC_TILE_M), g.m);
    e = cudaFuncSetAttribute(tc_products_kernel<true, MT, SPLIT, STAGES, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    tc_products_kernel<true, MT, SPLIT, STAGES, true><<<grid, TC_THREADS, smem, st>>>(mapW, mapD, p);
  } else {
    constexpr int MT = 2, SPLIT = 2, STAGES = 3;
    const size_t smem = (size_t)STAGES * (MT * TC_TILE_M + SPLIT * B) * TC_KBYTES + 1024;
    dim3 grid((g.ld + MT * TC_TILE_M - 1) / (MT * TC_TILE_M), g.m);
    e = cudaFuncSetAttribute(tc_products_kernel<false, MT, SPLIT, STAGES, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    tc_products_kernel<false, MT, SPLIT, STAGES, true><<<grid, TC_THREADS, smem, st>>>(mapW, mapD, p);
  }
  count_launch();
  return cudaGetLastError();
}

// -------------------------------------------------------------------------------------------
// Coded rank-B update (step O3) on tensor cores:  W~[row][col] += lr * sum_b Dt[b][row] Xt[b][col].
// Tile M = 128 coded rows, N = 128 columns, K = B; both operands are small K-major copies
// (rows x B and columns x B) in the multiplication type.  A CTA keeps its row tile's operand in
// shared memory and walks a run of column tiles; the accumulator alternates between two tensor-
// memory buffers so that the epilogue of one column tile (read W~, add, write back: the HBM-bound
// part) overlaps the multiplication of the next.
// -------------------------------------------------------------------------------------------
struct TcUpdParams {
  Geom g;
  int B, ksteps, tiles_per_cta;
  float lr;
  int* flag;
};

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

constexpr int TCU_THREADS = 64 + 256;  // producer warp, MMA warp, eight epilogue warps

template <bool TF32, int KS>
__global__ void __launch_bounds__(TCU_THREADS, 1)
tc_update_kernel(const __grid_constant__ CUtensorMap mapD, const __grid_constant__ CUtensorMap mapX, TcUpdParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  constexpr uint32_t tile_bytes = KS * TC_TILE_M * TC_KBYTES;  // one operand tile: KS chunks of 128 rows x 128 bytes
  constexpr int elems = TC_KBYTES / (TF32 ? 4 : 2);
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* sA = base;                 // delta~ operand of this row tile
  uint8_t* sB = base + tile_bytes;    // [2] x~ operand of a column tile
  float* sAcc = reinterpret_cast<float*>(base + 3 * tile_bytes);  // accumulator tile, 128 x 132 floats
  __shared__ uint64_t a_full, b_full[2], b_empty[2], acc_full[2], acc_empty[2];
  __shared__ int s_ok[8];
  __shared__ uint32_t tmem_slot;
  __shared__ int s_fail;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row0 = blockIdx.x * TC_TILE_M;
  const int i_blk = row0 / p.g.b_r;                      // tiles never straddle block-rows
  const int ct0 = blockIdx.y * p.tiles_per_cta;
  const int n_ct_all = p.g.ld / TC_TILE_M;
  const int ct1 = min(ct0 + p.tiles_per_cta, n_ct_all);

  if (threadIdx.x == 0) {
    mbar_init(&a_full, 1);
    for (int s = 0; s < 2; ++s) { mbar_init(&b_full[s], 1); mbar_init(&b_empty[s], 1); mbar_init(&acc_full[s], 1); mbar_init(&acc_empty[s], 8); }
    s_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(&tmem_slot, 256);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_slot;

  // a column tile is skipped when the grid has no node there (parity rows x parity columns)
  auto skipped = [&](int ct) { return i_blk >= p.g.m && (ct * TC_TILE_M) / p.g.ldb >= p.g.n; };

  if (warp == 0 && lane == 0) {
    mbar_expect_tx(&a_full, tile_bytes);
#pragma unroll
    for (int k = 0; k < KS; ++k) tma_load_2d(sA + k * (TC_TILE_M * TC_KBYTES), &mapD, k * elems, row0, &a_full);
    int n = 0;
    for (int ct = ct0; ct < ct1; ++ct) {
      if (skipped(ct)) continue;
      const int s = n & 1;
      if (n >= 2 && !mbar_wait(&b_empty[s], ((n >> 1) - 1) & 1)) { s_fail = 1; break; }
      mbar_expect_tx(&b_full[s], tile_bytes);
#pragma unroll
      for (int k = 0; k < KS; ++k)
        tma_load_2d(sB + s * tile_bytes + k * (TC_TILE_M * TC_KBYTES), &mapX, k * elems, ct * TC_TILE_M, &b_full[s]);
      ++n;
    }
  } else if (warp == 1 && lane == 0) {
    const uint32_t idesc = instr_desc(TF32, TC_TILE_M, TC_TILE_M);
    bool ok = mbar_wait(&a_full, 0);
    if (!ok) s_fail = 1;
    int n = 0;
    for (int ct = ct0; ct < ct1 && ok; ++ct) {
      if (skipped(ct)) continue;
      const int s = n & 1;
      if (!mbar_wait(&b_full[s], (n >> 1) & 1)) { s_fail = 1; break; }
      if (n >= 2 && !mbar_wait(&acc_empty[s], ((n >> 1) - 1) & 1)) { s_fail = 1; break; }
      tc_fence_after();
#pragma unroll
      for (int k = 0; k < KS; ++k) {
        const uint64_t da = smem_desc_k128(sA + k * (TC_TILE_M * TC_KBYTES));
        const uint64_t db = smem_desc_k128(sB + s * tile_bytes + k * (TC_TILE_M * TC_KBYTES));
#pragma unroll
        for (int kk = 0; kk < TC_KBYTES / 32; ++kk)
          tc_mma<TF32>(tmem + (uint32_t)(s * TC_TILE_M), da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc,
                       (k > 0 || kk > 0) ? 1u : 0u);
      }
      tc_commit(&b_empty[s]);
      tc_commit(&acc_full[s]);
      ++n;
    }
  } else if (warp >= 2) {
    const int quad = warp & 3;
    int n = 0;
    for (int ct = ct0; ct < ct1; ++ct) {
      if (skipped(ct)) continue;
      const int s = n & 1;
      // the eight epilogue warps leave together or not at all: they meet at named barriers below
      const bool got = mbar_wait(&acc_full[s], (n >> 1) & 1);
      if (lane == 0) s_ok[warp - 2] = got ? 1 : 0;
      asm volatile("bar.sync 1, 256;" ::: "memory");
      bool all_ok = true;
#pragma unroll
      for (int w = 0; w < 8; ++w) all_ok = all_ok && s_ok[w];
      if (!all_ok) { s_fail = 1; break; }
      tc_fence_after();
      // accumulator tile -> shared memory (row stride 132 floats: 16-byte aligned, conflict-free):
      // warp w reads its lane quadrant (w & 3) and one half of the columns
      const int half = (warp - 2) >> 2;
#pragma unroll 1
      for (int c0 = half * 64; c0 < half * 64 + 64; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(tmem + ((uint32_t)(quad * 32) << 16) + (uint32_t)(s * TC_TILE_M + c0), r);
        float4* dstrow = reinterpret_cast<float4*>(sAcc + (quad * 32 + lane) * 132 + c0);
#pragma unroll
        for (int q = 0; q < 8; ++q)
          dstrow[q] = make_float4(__uint_as_float(r[4 * q]), __uint_as_float(r[4 * q + 1]),
                                  __uint_as_float(r[4 * q + 2]), __uint_as_float(r[4 * q + 3]));
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[s]);   // the tensor-memory buffer can be refilled already
      asm volatile("bar.sync 1, 256;" ::: "memory");
      // ... then the warps walk whole rows with 16-byte accesses, eight in flight per lane: coalesced
      // read-modify-write of W~ (fp32: a warp per row; bfloat16: half a warp per row)
      const int ew = warp - 2;
      if (TF32) {
#pragma unroll 1
        for (int rr0 = ew; rr0 < TC_TILE_M; rr0 += 64) {
          float4 wv[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const int rr = rr0 + 8 * u;
            const float* wrow = reinterpret_cast<const float*>(p.g.Wt) + (size_t)min(row0 + rr, p.g.Mbr - 1) * p.g.ld +
                                (size_t)ct * TC_TILE_M + 4 * lane;
            wv[u] = __ldcs(reinterpret_cast<const float4*>(wrow));
          }
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const int rr = rr0 + 8 * u;
            if (row0 + rr >= p.g.Mbr) continue;
            const float4 a4 = *reinterpret_cast<const float4*>(sAcc + rr * 132 + 4 * lane);
            float4 o;
            o.x = fmaf(p.lr, a4.x, wv[u].x); o.y = fmaf(p.lr, a4.y, wv[u].y);
            o.z = fmaf(p.lr, a4.z, wv[u].z); o.w = fmaf(p.lr, a4.w, wv[u].w);
            float* wrow = reinterpret_cast<float*>(p.g.Wt) + (size_t)(row0 + rr) * p.g.ld + (size_t)ct * TC_TILE_M + 4 * lane;
            __stcs(reinterpret_cast<float4*>(wrow), o);
          }
        }
      } else {
        const int sub = lane >> 4, l16 = lane & 15;   // two rows per warp instruction
#pragma unroll 1
        for (int rr0 = 2 * ew + sub; rr0 < TC_TILE_M; rr0 += 128) {
          uint4 wv[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const int rr = rr0 + 16 * u;
            const __nv_bfloat16* wrow = reinterpret_cast<const __nv_bfloat16*>(p.g.Wt) +
                                        (size_t)min(row0 + rr, p.g.Mbr - 1) * p.g.ld + (size_t)ct * TC_TILE_M + 8 * l16;
            wv[u] = __ldcs(reinterpret_cast<const uint4*>(wrow));
          }
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const int rr = rr0 + 16 * u;
            if (row0 + rr >= p.g.Mbr) continue;
            const float4 a0 = *reinterpret_cast<const float4*>(sAcc + rr * 132 + 8 * l16);
            const float4 a1 = *reinterpret_cast<const float4*>(sAcc + rr * 132 + 8 * l16 + 4);
            float f[8];
            Vec16<__nv_bfloat16>::unpack(wv[u], f);
            f[0] = fmaf(p.lr, a0.x, f[0]); f[1] = fmaf(p.lr, a0.y, f[1]); f[2] = fmaf(p.lr, a0.z, f[2]); f[3] = fmaf(p.lr, a0.w, f[3]);
            f[4] = fmaf(p.lr, a1.x, f[4]); f[5] = fmaf(p.lr, a1.y, f[5]); f[6] = fmaf(p.lr, a1.z, f[6]); f[7] = fmaf(p.lr, a1.w, f[7]);
            uint32_t w[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * k], f[2 * k + 1]);
              w[k] = *reinterpret_cast<const uint32_t*>(&h);
            }
            __nv_bfloat16* wrow = reinterpret_cast<__nv_bfloat16*>(p.g.Wt) + (size_t)(row0 + rr) * p.g.ld +
                                  (size_t)ct * TC_TILE_M + 8 * l16;
            __stcs(reinterpret_cast<uint4*>(wrow), make_uint4(w[0], w[1], w[2], w[3]));
          }
        }
      }
      asm volatile("bar.sync 1, 256;" ::: "memory");
      ++n;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && s_fail) atomicExch(p.flag, 1);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 256);
  }
}

// Transposed operand copies for the update: src is (B, len) fp32, dst is (len, B) in T.
template <typename T>
__global__ void tc_transpose_kernel(const float* __restrict__ src, int B, int len, T* __restrict__ dst) {
  __shared__ float tile[32][33];
  const int x0 = blockIdx.x * 32, b0 = blockIdx.y * 32;
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int b = b0 + r, x = x0 + threadIdx.x;
    tile[r][threadIdx.x] = (b < B && x < len) ? src[(size_t)b * len + x] : 0.0f;
  }
  __syncthreads();
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int x = x0 + r, b = b0 + threadIdx.x;
    if (x < len && b < B) dst[(size_t)x * B + b] = (T)tile[threadIdx.x][r];
  }
}

bool tc_update_supported(const Geom& g, int math, int B) {
  if (!tc_forward_supported(g, math, B)) return false;
  const bool tf32 = g.dtype == CODENET_F32;
  const int ks = B * (tf32 ? 4 : 2) / TC_KBYTES;
  // three operand tiles of ks chunks and the 128 x 132 accumulator tile must fit one SM's shared memory
  // (ks = 4, i.e. fp32 blocks at batch 128, does not: that case keeps the FFMA update)
  const size_t smem = (size_t)3 * ks * TC_TILE_M * TC_KBYTES + (size_t)TC_TILE_M * 132 * sizeof(float) + 1024;
  return g.b_r % TC_TILE_M == 0 && g.ldb % TC_TILE_M == 0 && (ks == 1 || ks == 2 || ks == 4) && smem <= 227 * 1024;
}

template <bool TF32, int KS>
cudaError_t tc_update_launch(const CUtensorMap& mapD, const CUtensorMap& mapX, const TcUpdParams& p, dim3 grid, cudaStream_t st) {
  const size_t smem = (size_t)3 * KS * TC_TILE_M * TC_KBYTES + (size_t)TC_TILE_M * 132 * sizeof(float) + 1024;
  cudaError_t e = cudaFuncSetAttribute(tc_update_kernel<TF32, KS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  tc_update_kernel<TF32, KS><<<grid, TCU_THREADS, smem, st>>>(mapD, mapX, p);
  return cudaGetLastError();
}

cudaError_t launch_tc_update(const codenet_layer_impl& L, int B, float lr, cudaStream_t st) {
  const Geom& g = L.g;
  const bool tf32 = g.dtype == CODENET_F32;
  dim3 tb(32, 8);
  dim3 gd((g.Mbr + 31) / 32, (B + 31) / 32), gx((g.ld + 31) / 32, (B + 31) / 32);
  if (tf32) {
    tc_transpose_kernel<float><<<gd, tb, 0, st>>>(L.ws.Dt, B, g.Mbr, reinterpret_cast<float*>(L.ws.tc_dT));
    tc_transpose_kernel<float><<<gx, tb, 0, st>>>(L.ws.Xt, B, g.ld, reinterpret_cast<float*>(L.ws.tc_xT));
  } else {
    tc_transpose_kernel<__nv_bfloat16><<<gd, tb, 0, st>>>(L.ws.Dt, B, g.Mbr, reinterpret_cast<__nv_bfloat16*>(L.ws.tc_dT));
    tc_transpose_kernel<__nv_bfloat16><<<gx, tb, 0, st>>>(L.ws.Xt, B, g.ld, reinterpret_cast<__nv_bfloat16*>(L.ws.tc_xT));
  }
  count_launch(2);
  CUtensorMap mapD, mapX;
  if (!make_map(&mapD, L.ws.tc_dT, tf32, (size_t)g.Mbr, (size_t)B, (size_t)B, TC_TILE_M)) return cudaErrorInvalidValue;
  if (!make_map(&mapX, L.ws.tc_xT, tf32, (size_t)g.ld, (size_t)B, (size_t)B, TC_TILE_M)) return cudaErrorInvalidValue;
  TcUpdParams p;
  p.g = g; p.B = B; p.lr = lr; p.flag = L.ws.tc_flag;
  p.ksteps = B * (tf32 ? 4 : 2) / TC_KBYTES;
  const int n_ct = g.ld / TC_TILE_M;
  p.tiles_per_cta = n_ct < 20 ? n_ct : 20;
  dim3 grid(g.Mbr / TC_TILE_M, (n_ct + p.tiles_per_cta - 1) / p.tiles_per_cta);
  cudaError_t e;
  ProfileScope scope(CODENET_KERNEL_UPDATE, st);
  if (tf32) {
    if (p.ksteps == 1) e = tc_update_launch<true, 1>(mapD, mapX, p, grid, st);
    else if (p.ksteps == 2) e = tc_update_launch<true, 2>(mapD, mapX, p, grid, st);
    else e = tc_update_launch<true, 4>(mapD, mapX, p, grid, st);
  } else {
    if (p.ksteps == 1) e = tc_update_launch<false, 1>(mapD, mapX, p, grid, st);
    else if (p.ksteps == 2) e = tc_update_launch<false, 2>(mapD, mapX, p, grid, st);
    else e = tc_update_launch<false, 4>(mapD, mapX, p, grid, st);
  }
  count_launch();
  return e;
}


// -------------------------------------------------------------------------------------------
// Steps O2 and O3 in one sweep on tensor cores (bfloat16 blocks): every stored tile of W~ crosses
// HBM once in each direction.  A CTA owns (block-row i, 128 columns) and walks the 128-row tiles of
// the block-row.  Per tile: TMA brings the 128 x 128 tile into shared memory; one instruction group
// forms the update tile  D_u = delta~^T x~  (K = batch), another adds the tile's part of
// Z = W~^T delta (K = the tile's rows, from the values before the update, delta as a hi + lo pair)
// into an accumulator that lives for the whole block-row; the epilogue warps add lr * D_u to the
// tile where it sits in shared memory and TMA stores it back.  The operands need no transposed
// copies: delta~ (B, rows) row-major is the M-major A operand of the update and the K-major B
// operand of the backward product, x~ (B, columns) is the N-major B operand of the update.
// -------------------------------------------------------------------------------------------
namespace {

struct TcFusedParams {
  Geom g;
  int B, n_rt, n_items;   // row tiles per block-row; work items (block-row, column tile)
  int zsplit;             // an item's row tiles are shared out among this many CTAs (1 or 2); with 2 each adds its part
                          // of Z into a buffer cleared before the launch (two addends: the sum does not depend on the order)
  float lr;
  float* Z;               // [block-row][block-column][position][b], or NULL
  int* flag;
};

constexpr int TCF_THREADS = 64 + 256 + 32;   // producer warp, MMA warp, eight epilogue warps, store warp
// bfloat16: 128 x 128 tile = two 64-column chunks (32 KB), three stages; the delta~ tile (B, 128 rows) serves
// both products (M-major A of the update, K-major B of the backward product), three slots, hi and lo take
// one each.  fp32 / TF32: four 32-column chunks (64 KB), two stages.  A 32-bit M-major operand needs the
// 32-byte-atom swizzle and a K-major one the plain 128-byte swizzle (describing a K-major operand over
// 32-byte-atom data raises a misaligned-address fault), so one tile cannot serve both products: a slot
// holds two copies, delta~^T (128 rows, B) K-major for the update and delta~ (B, 128 rows) K-major for the
// backward product, and x~ comes as the transposed copy (128 columns, B).  One slot is enough: a 64 KB
// tile takes longer to stream than the small operand tiles take to arrive from L2.
// Work items are whole (block-row, column tile) pairs handed out round-robin, so that the CTAs of a wave
// stream neighbouring column tiles of the same rows together.  Cutting the last, incomplete wave into equal
// runs of tiles (an item's Z then built by several CTAs in a fixed order through a flag) was built and
// measured: no gain for configuration 5 (65.6 us against 63.7 us in the same build; runs of four tiles do
// not amortise the pipeline fill) and 2 % for configuration 4, for a per-tile bookkeeping cost that the
// epilogue warps, which sit on the critical path, paid on every tile: not kept.
// One column tile per work item.  Two (sharing the delta~ tiles; the tensor memory is just enough for
// 2 x D_u + 2 x Z) were tried for bfloat16: 459 us against 357 us for configuration 4, because two tiles per
// row step leave the three-stage W~ ring one tile of look-ahead, and shared memory has no room for a fourth
// stage beside two x~ tiles.
template <bool TF32> struct TcfCfg {
  static constexpr int EPC = TC_KBYTES / (TF32 ? 4 : 2);      // elements per 128-byte chunk row
  static constexpr int NCH = TC_TILE_M / EPC;                 // chunks per 128 elements
  static constexpr int KI = TF32 ? 8 : 16;                    // K per instruction
  static constexpr int WST = TF32 ? 2 : 3;
  static constexpr int DST = TF32 ? 1 : 3;
  static constexpr uint32_t WCHUNK = TC_TILE_M * TC_KBYTES;   // 128 rows x 128 bytes
  static constexpr uint32_t WTILE = NCH * WCHUNK;
  static constexpr int PARTS = TF32 ? 1 : 2;                  // delta operand: one TF32 copy, or bfloat16 hi + lo
};

template <bool TF32>
__global__ void __launch_bounds__(TCF_THREADS, 1)
tc_backward_update_kernel(const __grid_constant__ CUtensorMap mapW, const __grid_constant__ CUtensorMap mapD,
                          const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapDu,
                          TcFusedParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const int B = p.B;
  using Cfg = TcfCfg<TF32>;
  constexpr int TCF_WST = Cfg::WST, TCF_DST = Cfg::DST, NCH = Cfg::NCH, EPC = Cfg::EPC, KI = Cfg::KI;
  constexpr uint32_t TCF_WTILE = Cfg::WTILE, WCHUNK = Cfg::WCHUNK;
  const uint32_t vchunk = (uint32_t)B * TC_KBYTES;   // one chunk of a vector tile: B rows x 128 bytes
  const uint32_t vtile = NCH * vchunk;                // = 128 x B elements, whichever way round
  const uint32_t dslot = TF32 ? 2 * vtile : vtile;    // TF32: [delta~^T for the update][delta~ for the backward product]
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* sW = base;                                  // [TCF_WST][NCH chunks][128 rows][128 bytes]
  uint8_t* sX = sW + (size_t)TCF_WST * TCF_WTILE;      // [NCH chunks][B][128 bytes]: x~ of the item's columns
  uint8_t* sD = sX + vtile;                            // [TCF_DST] slots of delta~ tiles of a row tile
  __shared__ uint64_t w_full[TCF_WST], w_empty[TCF_WST], w_read[TCF_WST], d_full[TCF_DST], d_empty[TCF_DST];
  __shared__ uint64_t x_full, x_empty, acc_full[2], acc_empty[2], z_full, z_empty, w_done[TCF_WST];
  __shared__ uint32_t tmem_slot;
  __shared__ int s_fail;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_ct = p.g.ld / TC_TILE_M;

  if (threadIdx.x == 0) {
    for (int s = 0; s < TCF_WST; ++s) {
      mbar_init(&w_full[s], 1); mbar_init(&w_empty[s], 1); mbar_init(&w_read[s], 1); mbar_init(&w_done[s], 8);
    }
    for (int s = 0; s < TCF_DST; ++s) { mbar_init(&d_full[s], 1); mbar_init(&d_empty[s], 1); }
    mbar_init(&x_full, 1); mbar_init(&x_empty, 1); mbar_init(&z_full, 1); mbar_init(&z_empty, 8);
    for (int s = 0; s < 2; ++s) { mbar_init(&acc_full[s], 1); mbar_init(&acc_empty[s], 8); }
    s_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(&tmem_slot, 512);   // D_u twice (2 x 128 columns) and Z (B <= 128 columns)
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_slot;
  const uint32_t tmem_z = tmem + 256;

  // item -> (block-row, column tile); tiles of the absent corner (parity row x parity column) are not items
  const int n_units = p.n_items * p.zsplit, rt_per = p.n_rt / p.zsplit;
  auto item_of = [&](int unit, int* i_blk, int* ct, int* rt0) {
    const int item = unit / p.zsplit;
    *rt0 = (unit % p.zsplit) * rt_per;
    const int data_items = p.g.m * n_ct;
    if (item < data_items) { *i_blk = item / n_ct; *ct = item % n_ct; }
    else {
      const int per_row = p.g.n * (p.g.ldb / TC_TILE_M);
      *i_blk = p.g.m + (item - data_items) / per_row;
      *ct = (item - data_items) % per_row;
    }
  };

  if (warp == 0 && lane == 0) {
    // ---- TMA producer ----
    const uint64_t w_pol = l2_evict_first();
    uint32_t wn = 0, dn = 0, xn = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < n_units && ok; item += gridDim.x, ++xn) {
      int i_blk, ct, rt0;
      item_of(item, &i_blk, &ct, &rt0);
      const bool need_z = i_blk < p.g.m && p.Z != nullptr;
      for (int rt = rt0; rt < rt0 + rt_per && ok; ++rt, ++wn) {
        const int row0 = i_blk * p.g.b_r + rt * TC_TILE_M;
        const uint32_t s = wn % TCF_WST;
        if (wn >= TCF_WST && !mbar_wait(&w_empty[s], ((wn / TCF_WST) - 1) & 1)) { ok = false; break; }
        mbar_expect_tx(&w_full[s], TCF_WTILE);
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch)
          tma_load_2d_hint(sW + (size_t)s * TCF_WTILE + ch * WCHUNK, &mapW, ct * TC_TILE_M + ch * EPC, row0, &w_full[s], w_pol);
        for (int part = 0; part < (need_z ? Cfg::PARTS : 1); ++part, ++dn) {   // delta~ (hi, then lo)
          const uint32_t ds = dn % TCF_DST;
          if (dn >= TCF_DST && !mbar_wait(&d_empty[ds], ((dn / TCF_DST) - 1) & 1)) { ok = false; break; }
          uint8_t* slot = sD + (size_t)ds * dslot;
          if (TF32) {
            mbar_expect_tx(&d_full[ds], need_z ? 2 * vtile : vtile);
            for (int ch = 0; ch < B / EPC; ++ch)       // delta~^T: 128 rows x B, chunks of 32 batch entries
              tma_load_2d(slot + ch * WCHUNK, &mapDu, ch * EPC, row0, &d_full[ds]);
            if (need_z)
#pragma unroll
              for (int ch = 0; ch < NCH; ++ch)
                tma_load_2d(slot + vtile + ch * vchunk, &mapD, row0 + ch * EPC, 0, &d_full[ds]);
          } else {
            mbar_expect_tx(&d_full[ds], vtile);
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch)
              tma_load_2d(slot + ch * vchunk, &mapD, row0 + ch * EPC, part * B, &d_full[ds]);
          }
        }
        if (rt == rt0 && ok) {   // x~ of this item's columns, after the first tile so that it never delays it
          if (xn >= 1 && !mbar_wait(&x_empty, (xn - 1) & 1)) { ok = false; break; }
          mbar_expect_tx(&x_full, vtile);
          if (TF32) {
            for (int ch = 0; ch < B / EPC; ++ch) tma_load_2d(sX + ch * WCHUNK, &mapX, ch * EPC, ct * TC_TILE_M, &x_full);
          } else {
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) tma_load_2d(sX + ch * vchunk, &mapX, ct * TC_TILE_M + ch * EPC, 0, &x_full);
          }
        }
      }
    }
    if (!ok) s_fail = 1;
  } else if (warp == 1 && lane == 0) {
    // ---- MMA issuer ----
    const uint32_t idesc_u = instr_desc(TF32, TC_TILE_M, TC_TILE_M, !TF32, !TF32);
    const uint32_t idesc_z = instr_desc(TF32, TC_TILE_M, B, true, false);
    constexpr uint64_t kstep_mn = (uint64_t)(KI * TC_KBYTES) >> 4;   // KI K rows of an MN-major tile
    uint32_t wn = 0, dn = 0, xn = 0, zn = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < n_units && ok; item += gridDim.x, ++xn) {
      int i_blk, ct, rt0;
      item_of(item, &i_blk, &ct, &rt0);
      const bool need_z = i_blk < p.g.m && p.Z != nullptr;
      for (int rt = rt0; rt < rt0 + rt_per && ok; ++rt, ++wn) {
        const uint32_t s = wn % TCF_WST, u = wn & 1;
        if (!mbar_wait(&w_full[s], (wn / TCF_WST) & 1)) { ok = false; break; }
        uint32_t ds = dn % TCF_DST;
        if (!mbar_wait(&d_full[ds], (dn / TCF_DST) & 1)) { ok = false; break; }
        if (rt == rt0 && !mbar_wait(&x_full, xn & 1)) { ok = false; break; }
        if (wn >= 2 && !mbar_wait(&acc_empty[u], ((wn >> 1) - 1) & 1)) { ok = false; break; }
        if (rt == rt0 && need_z && zn >= 1 && !mbar_wait(&z_empty, (zn - 1) & 1)) { ok = false; break; }
        tc_fence_after();
        const uint8_t* wt = sW + (size_t)s * TCF_WTILE;
        const uint8_t* dt = sD + (size_t)ds * dslot;
        constexpr int KPC = EPC / KI;   // instructions per 128-byte chunk of K
        // update tile: D_u[row][col] = sum_b delta~[b][row] x~[b][col]
        {
          if (TF32) {
            for (int kk = 0; kk < B / KI; ++kk) {
              const uint64_t da = smem_desc_k128(dt + (kk / KPC) * WCHUNK) + (uint64_t)((kk % KPC) * 2);
              const uint64_t db = smem_desc_k128(sX + (kk / KPC) * WCHUNK) + (uint64_t)((kk % KPC) * 2);
              tc_mma<TF32>(tmem + u * TC_TILE_M, da, db, idesc_u, kk > 0 ? 1u : 0u);
            }
          } else {
            const uint64_t da = smem_desc_mn128<TF32>(dt, vchunk), db = smem_desc_mn128<TF32>(sX, vchunk);
            for (int kk = 0; kk < B / KI; ++kk)
              tc_mma<TF32>(tmem + u * TC_TILE_M, da + (uint64_t)kk * kstep_mn, db + (uint64_t)kk * kstep_mn, idesc_u, kk > 0 ? 1u : 0u);
          }
        }
        tc_commit(&acc_full[u]);
        if (need_z) {
          // Z[col][b] += sum_row W~[row][col] delta[b][row], hi part then lo part of delta
          const uint64_t da = smem_desc_mn128<TF32>(wt, WCHUNK);
          for (int part = 0; part < Cfg::PARTS; ++part) {
            if (part == 1) {
              tc_commit(&d_empty[ds]);
              ++dn;
              ds = dn % TCF_DST;
              if (!mbar_wait(&d_full[ds], (dn / TCF_DST) & 1)) { ok = false; break; }
              tc_fence_after();
              dt = sD + (size_t)ds * dslot;
            }
            const uint8_t* dz = TF32 ? dt + vtile : dt;   // the K-major delta~ tile
#pragma unroll
            for (int kk = 0; kk < TC_TILE_M / KI; ++kk) {
              const uint64_t db = smem_desc_k128(dz + (kk / KPC) * vchunk) + (uint64_t)((kk % KPC) * 2);
              tc_mma<TF32>(tmem_z, da + (uint64_t)kk * kstep_mn, db, idesc_z, (rt > rt0 || part > 0 || kk > 0) ? 1u : 0u);
            }
          }
          if (!ok) break;
        }
        tc_commit(&d_empty[ds]);
        ++dn;
        tc_commit(&w_read[s]);    // the tile may be rewritten once these instructions have read it
      }
      if (!ok) break;
      tc_commit(&x_empty);
      if (need_z) { tc_commit(&z_full); ++zn; }
    }
    if (!ok) s_fail = 1;
  } else if (warp >= 2 && warp < 10) {
    // ---- epilogue warps: update of the tile where it sits in shared memory; Z at the end of a
    // block-row.  The warps run independently (no barrier among them): each hands its part of a tile
    // to the store warp through w_done, and a warp whose bounded wait runs out simply leaves.
    const int ew = warp - 2, quad = warp & 3, half = ew >> 2;
    const int row = quad * 32 + lane;             // tile row (update) or tile column (Z) of this thread
    uint32_t wn = 0, zn = 0;
    bool alive = true;
    for (int item = blockIdx.x; item < n_units && alive; item += gridDim.x) {
      int i_blk, ct, rt0;
      item_of(item, &i_blk, &ct, &rt0);
      const bool need_z = i_blk < p.g.m && p.Z != nullptr;
      for (int rt = rt0; rt < rt0 + rt_per; ++rt, ++wn) {
        const uint32_t s = wn % TCF_WST, u = wn & 1;
        if (!mbar_wait(&acc_full[u], (wn >> 1) & 1) || !mbar_wait(&w_read[s], (wn / TCF_WST) & 1)) { alive = false; break; }
        tc_fence_after();
        uint8_t* wt = sW + (size_t)s * TCF_WTILE + row * TC_KBYTES;
#pragma unroll 1
        for (int c0 = half * 64; c0 < half * 64 + 64; c0 += 32) {   // this warp's 64 columns of the tile
          uint32_t r[32];
          tmem_ld32(tmem + ((uint32_t)(quad * 32) << 16) + (uint32_t)(u * TC_TILE_M + c0), r);
          if (TF32) {
            // 32 columns = one 128-byte chunk row; its 32-byte atoms sit at atom ^ (row % 4)
            uint8_t* wrow = wt + (c0 / 32) * WCHUNK;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              float4* cell = reinterpret_cast<float4*>(wrow + ((((q >> 1) ^ (row & 3)) << 5) | ((q & 1) << 4)));
              float4 w4 = *cell;
              w4.x = fmaf(p.lr, __uint_as_float(r[4 * q]), w4.x); w4.y = fmaf(p.lr, __uint_as_float(r[4 * q + 1]), w4.y);
              w4.z = fmaf(p.lr, __uint_as_float(r[4 * q + 2]), w4.z); w4.w = fmaf(p.lr, __uint_as_float(r[4 * q + 3]), w4.w);
              *cell = w4;
            }
          } else {
            // 32 columns = half a chunk row; 16-byte unit u16 of the row sits at u16 ^ (row % 8)
            uint8_t* wrow = wt + (c0 / 64) * WCHUNK;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              uint4* cell = reinterpret_cast<uint4*>(wrow + (((((c0 & 63) >> 3) + q) ^ (row & 7)) << 4));
              float f[8];
              Vec16<__nv_bfloat16>::unpack(*cell, f);
              uint32_t w[4];
#pragma unroll
              for (int kq = 0; kq < 4; ++kq) {
                const float a = fmaf(p.lr, __uint_as_float(r[8 * q + 2 * kq]), f[2 * kq]);
                const float b = fmaf(p.lr, __uint_as_float(r[8 * q + 2 * kq + 1]), f[2 * kq + 1]);
                const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
                w[kq] = *reinterpret_cast<const uint32_t*>(&h);
              }
              *cell = make_uint4(w[0], w[1], w[2], w[3]);
            }
          }
        }
        tc_fence_before();
        fence_async_smem();
        __syncwarp();
        if (lane == 0) { mbar_arrive(&acc_empty[u]); mbar_arrive(&w_done[s]); }
      }
      if (!alive) break;
      if (need_z) {
        if (!mbar_wait(&z_full, zn & 1)) { alive = false; break; }
        tc_fence_after();
        const int gr = ct * TC_TILE_M + row;                 // coded column of this thread
        const int node = gr / p.g.ldb, c = gr % p.g.ldb;
        const bool valid = c < p.g.b_c;
        float* zrow = p.Z + (((size_t)i_blk * p.g.Nn + node) * p.g.b_c + c) * B;
        for (int b0 = half * (B / 2); b0 < (half + 1) * (B / 2); b0 += 32) {
          uint32_t r[32];
          tmem_ld32(tmem_z + ((uint32_t)(quad * 32) << 16) + (uint32_t)b0, r);
          if (valid && p.zsplit == 1) {
            float4* dst = reinterpret_cast<float4*>(zrow + b0);
#pragma unroll
            for (int q = 0; q < 8; ++q)
              dst[q] = make_float4(__uint_as_float(r[4 * q]), __uint_as_float(r[4 * q + 1]),
                                   __uint_as_float(r[4 * q + 2]), __uint_as_float(r[4 * q + 3]));
          } else if (valid) {
#pragma unroll
            for (int q = 0; q < 8; ++q)
              asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};"
                           :: "l"(zrow + b0 + 4 * q), "f"(__uint_as_float(r[4 * q])), "f"(__uint_as_float(r[4 * q + 1])),
                              "f"(__uint_as_float(r[4 * q + 2])), "f"(__uint_as_float(r[4 * q + 3])) : "memory");
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&z_empty);
        ++zn;
      }
    }
    if (!alive) s_fail = 1;
  } else if (warp == 10 && lane == 0) {
    // ---- store warp: a tile every epilogue warp has finished goes back to global memory ----
    const uint64_t w_pol = l2_evict_first();
    uint32_t wn = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < n_units && ok; item += gridDim.x) {
      int i_blk, ct, rt0;
      item_of(item, &i_blk, &ct, &rt0);
      for (int rt = rt0; rt < rt0 + rt_per; ++rt, ++wn) {
        const uint32_t s = wn % TCF_WST;
        if (!mbar_wait(&w_done[s], (wn / TCF_WST) & 1)) { ok = false; break; }
        const int row0 = i_blk * p.g.b_r + rt * TC_TILE_M;
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch)
          tma_store_2d_hint(&mapW, ct * TC_TILE_M + ch * EPC, row0, sW + (size_t)s * TCF_WTILE + ch * WCHUNK, w_pol);
        tma_store_commit();
        tma_store_wait_read();
        mbar_arrive(&w_empty[s]);
      }
    }
    tma_store_wait_all();
    if (!ok) s_fail = 1;
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && s_fail) atomicExch(p.flag, 1);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// fp32 (B, len) -> bfloat16, same shape
__global__ void tc_to_bf16_kernel(const float* __restrict__ src, size_t count, __nv_bfloat16* __restrict__ dst) {
  for (size_t idx = blockIdx.x * (size_t)blockDim.x + threadIdx.x; idx < count; idx += (size_t)gridDim.x * blockDim.x)
    dst[idx] = __float2bfloat16_rn(src[idx]);
}

// Both operands of the fused bfloat16 kernel in one pass: delta~ (dcount floats) -> hi / lo pair, x~ (xcount
// floats) -> bfloat16.  Four values per thread and step (the counts are multiples of four: B x padded widths).
__global__ void tc_prep_pair_kernel(const float* __restrict__ Dt, size_t dcount, __nv_bfloat16* __restrict__ dpair,
                                    const float* __restrict__ Xt, size_t xcount, __nv_bfloat16* __restrict__ xb) {
  const size_t nd4 = dcount / 4, nx4 = xcount / 4;
  for (size_t q = blockIdx.x * (size_t)blockDim.x + threadIdx.x; q < nd4 + nx4; q += (size_t)gridDim.x * blockDim.x) {
    if (q < nd4) {
      const float4 v = reinterpret_cast<const float4*>(Dt)[q];
      const __nv_bfloat16 h0 = __float2bfloat16_rn(v.x), h1 = __float2bfloat16_rn(v.y);
      const __nv_bfloat16 h2 = __float2bfloat16_rn(v.z), h3 = __float2bfloat16_rn(v.w);
      __nv_bfloat162 hi[2] = {__nv_bfloat162(h0, h1), __nv_bfloat162(h2, h3)};
      __nv_bfloat162 lo[2] = {__nv_bfloat162(__float2bfloat16_rn(v.x - __bfloat162float(h0)),
                                             __float2bfloat16_rn(v.y - __bfloat162float(h1))),
                              __nv_bfloat162(__float2bfloat16_rn(v.z - __bfloat162float(h2)),
                                             __float2bfloat16_rn(v.w - __bfloat162float(h3)))};
      reinterpret_cast<uint2*>(dpair)[q] = *reinterpret_cast<uint2*>(hi);
      reinterpret_cast<uint2*>(dpair + dcount)[q] = *reinterpret_cast<uint2*>(lo);
    } else {
      const float4 v = reinterpret_cast<const float4*>(Xt)[q - nd4];
      __nv_bfloat162 o[2] = {__nv_bfloat162(__float2bfloat16_rn(v.x), __float2bfloat16_rn(v.y)),
                             __nv_bfloat162(__float2bfloat16_rn(v.z), __float2bfloat16_rn(v.w))};
      reinterpret_cast<uint2*>(xb)[q - nd4] = *reinterpret_cast<uint2*>(o);
    }
  }
}

// Both transposed fp32 operand copies of the fused TF32 kernel in one launch: blockIdx.z = 0 takes delta~
// (B, len_d) -> (len_d, B), 1 takes x~ (B, len_x) -> (len_x, B).
__global__ void tc_transpose_pair_kernel(const float* __restrict__ Dt, int len_d, float* __restrict__ dT,
                                         const float* __restrict__ Xt, int len_x, float* __restrict__ xT, int B) {
  __shared__ float tile[32][33];
  const float* src = blockIdx.z == 0 ? Dt : Xt;
  float* dst = blockIdx.z == 0 ? dT : xT;
  const int len = blockIdx.z == 0 ? len_d : len_x;
  const int x0 = blockIdx.x * 32, b0 = blockIdx.y * 32;
  if (x0 >= len) return;
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int b = b0 + r, x = x0 + threadIdx.x;
    tile[r][threadIdx.x] = (b < B && x < len) ? src[(size_t)b * len + x] : 0.0f;
  }
  __syncthreads();
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int x = x0 + r, b = b0 + threadIdx.x;
    if (x < len && b < B) dst[(size_t)x * B + b] = tile[threadIdx.x][r];
  }
}

}  // namespace

static size_t tcf_smem_bytes(bool tf32, int B) {
  const size_t wtile = (size_t)TC_TILE_M * TC_TILE_M * (tf32 ? 4 : 2), vtile = (size_t)B * TC_TILE_M * (tf32 ? 4 : 2);
  return (tf32 ? 2 : 3) * wtile + (1 + (tf32 ? 2 : 3)) * vtile + 1024;   // W~ ring, x~ tile, delta~ slots
}

bool tc_backward_update_supported(const Geom& g, int math, int B) {
  const bool tf32 = g.dtype == CODENET_F32;
  if (!tc_backward_supported(g, math, B) || !tc_update_supported(g, math, B)) return false;
  // Z is read back in two halves of whole 32-column groups; the tiles must fit one SM's shared memory
  return B % 64 == 0 && B <= 128 && tcf_smem_bytes(tf32, B) <= 227 * 1024;
}

// One CTA per SM walks whole items; when the items do not fill the last round of CTAs (configuration 5: 192 items on
// 148 SMs, two rounds for 1.3 rounds' worth of work) halves of items even the rounds out.  Taken only where it saves
// a fifth of the rounds: the halves add into Z, which costs a clearing pass over it.
bool tc_backward_update_splits(const codenet_layer_impl& L, int B) {
  const Geom& g = L.g;
  if (!tc_backward_update_supported(g, L.desc.math, B)) return false;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int n_rt = g.b_r / TC_TILE_M;
  const long n_items = (long)g.m * (g.ld / TC_TILE_M) + (long)g.r_row * g.n * (g.ldb / TC_TILE_M);
  if (n_rt % 2 != 0) return false;
  const long whole = (n_items + sms - 1) / sms * 2, halves = (2 * n_items + sms - 1) / sms;
  return halves * 5 <= whole * 4;
}

cudaError_t launch_tc_backward_update(const codenet_layer_impl& L, int B, float lr, float* Z, cudaStream_t st) {
  const Geom& g = L.g;
  const bool tf32 = g.dtype == CODENET_F32;
  const void* dptr = L.ws.Dt;
  const void* xptr = L.ws.Xt;
  const bool ready = L.operands_ready != 0;   // the vector-encoding kernel wrote the copies below itself
  L.operands_ready = 0;
  if (!tf32) {
    // operands: delta~ as a bfloat16 pair (hi rows 0..B-1, lo rows B..2B-1), x~ as one bfloat16 copy;
    // TF32 reads the fp32 vectors where they are
    const size_t dcount = (size_t)B * g.Mbr, xcount = (size_t)B * g.ld;
    if (ready) {
    } else if (dcount % 4 == 0 && xcount % 4 == 0) {
      const size_t quads = (dcount + xcount) / 4;
      const int pgrid = (int)((quads + 255) / 256 < 148 * 8 ? (quads + 255) / 256 : 148 * 8);
      tc_prep_pair_kernel<<<pgrid, 256, 0, st>>>(L.ws.Dt, dcount, reinterpret_cast<__nv_bfloat16*>(L.ws.tc_d), L.ws.Xt, xcount,
                                                 reinterpret_cast<__nv_bfloat16*>(L.ws.tc_xT));
      count_launch();
    } else {
      const int dgrid = (int)((dcount + 255) / 256 < 148 * 8 ? (dcount + 255) / 256 : 148 * 8);
      const int xgrid = (int)((xcount + 255) / 256 < 148 * 8 ? (xcount + 255) / 256 : 148 * 8);
      tc_prep_d_kernel<__nv_bfloat16><<<dgrid, 256, 0, st>>>(L.ws.Dt, dcount, reinterpret_cast<__nv_bfloat16*>(L.ws.tc_d));
      tc_to_bf16_kernel<<<xgrid, 256, 0, st>>>(L.ws.Xt, xcount, reinterpret_cast<__nv_bfloat16*>(L.ws.tc_xT));
      count_launch(2);
    }
    dptr = L.ws.tc_d;
    xptr = L.ws.tc_xT;
  }
  CUtensorMap mapW, mapD, mapX, mapDu;
  if (!make_map(&mapW, g.Wt, tf32, (size_t)g.Mbr, (size_t)g.ld, (size_t)g.ld, TC_TILE_M, tf32)) return cudaErrorInvalidValue;
  if (!make_map(&mapD, dptr, tf32, (size_t)(tf32 ? B : 2 * B), (size_t)g.Mbr, (size_t)g.Mbr, B)) return cudaErrorInvalidValue;
  if (tf32) {
    // transposed fp32 copies (rows, B) and (columns, B): K-major operands of the update
    dim3 tb(32, 8);
    const int lmax = g.Mbr > g.ld ? g.Mbr : g.ld;
    dim3 gp((lmax + 31) / 32, (B + 31) / 32, 2);
    if (!ready) {
      tc_transpose_pair_kernel<<<gp, tb, 0, st>>>(L.ws.Dt, g.Mbr, reinterpret_cast<float*>(L.ws.tc_dT), L.ws.Xt, g.ld,
                                                 reinterpret_cast<float*>(L.ws.tc_xT), B);
      count_launch();
    }
    if (!make_map(&mapDu, L.ws.tc_dT, true, (size_t)g.Mbr, (size_t)B, (size_t)B, TC_TILE_M)) return cudaErrorInvalidValue;
    if (!make_map(&mapX, L.ws.tc_xT, true, (size_t)g.ld, (size_t)B, (size_t)B, TC_TILE_M)) return cudaErrorInvalidValue;
  } else {
    if (!make_map(&mapX, xptr, false, (size_t)B, (size_t)g.ld, (size_t)g.ld, B)) return cudaErrorInvalidValue;
    mapDu = mapD;   // not used: the shared tile serves both products
  }
  TcFusedParams p;
  p.g = g; p.B = B; p.lr = lr; p.Z = Z; p.flag = L.ws.tc_flag;
  p.n_rt = g.b_r / TC_TILE_M;
  p.n_items = g.m * (g.ld / TC_TILE_M) + g.r_row * g.n * (g.ldb / TC_TILE_M);
  const size_t smem = tcf_smem_bytes(tf32, B);
  cudaError_t e = tf32 ? cudaFuncSetAttribute(tc_backward_update_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)
                       : cudaFuncSetAttribute(tc_backward_update_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  p.zsplit = (Z != nullptr && tc_backward_update_splits(L, B)) ? 2 : 1;
  const bool cleared = L.z_cleared != 0;   // (by the vector-encoding kernel, on its way)
  L.z_cleared = 0;
  if (p.zsplit == 2 && !cleared) {
    e = cudaMemsetAsync(Z, 0, (size_t)g.m * g.Nn * g.b_c * B * sizeof(float), st);
    if (e != cudaSuccess) return e;
  }
  const int units = p.n_items * p.zsplit;
  const int grid = units < sms ? units : sms;
  ProfileScope scope(CODENET_KERNEL_BACKWARD_UPDATE, st);
  if (tf32) tc_backward_update_kernel<true><<<grid, TCF_THREADS, smem, st>>>(mapW, mapD, mapX, mapDu, p);
  else tc_backward_update_kernel<false><<<grid, TCF_THREADS, smem, st>>>(mapW, mapD, mapX, mapDu, p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace codenet

// ---- bounded waits: limit, diagnostic switch, acknowledgement -------------------------------------------------
extern "C" {

int codenet_set_wait_limit(uint64_t nanoseconds, codenet_stream_t stream) {
  const unsigned long long v = nanoseconds ? (unsigned long long)nanoseconds : 1000000000ull;
  return cudaMemcpyToSymbolAsync(codenet::c_wait_ns, &v, sizeof(v), 0, cudaMemcpyHostToDevice,
                                 reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess ? CODENET_OK : CODENET_E_CUDA;
}

int codenet_withhold_tile_loads(int on, codenet_stream_t stream) {
  const int v = on ? 1 : 0;
  return cudaMemcpyToSymbolAsync(codenet::c_withhold_loads, &v, sizeof(v), 0, cudaMemcpyHostToDevice,
                                 reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess ? CODENET_OK : CODENET_E_CUDA;
}

int codenet_reset_timeout(codenet_layer_t* layer, codenet_stream_t stream) {
  if (!layer) return CODENET_E_BADARG;
  return cudaMemsetAsync(layer->ws.tc_flag, 0, sizeof(int), reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess
             ? CODENET_OK : CODENET_E_CUDA;
}

}  // extern "C"
