// An entry point for callers that must not allocate device memory.
#include "codenet_internal.cuh"

using namespace codenet;

namespace {

// Scratch for the un-reduced per-block-column products of codenet_matvec_noalloc: 4 MiB that every
// GPU holding this library keeps until the process exits.
constexpr size_t kNoallocMaxFloats = (size_t)1 << 20;
static __device__ __align__(256) float g_noalloc_scratch[kNoallocMaxFloats];

// In host code the array's name is only a stand-in; the device address has to be asked for, once
// per device, with that device current.
constexpr int kMaxDevices = 64;
float* g_scratch_ptr[kMaxDevices] = {nullptr};

int scratch_for_current_device(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return CODENET_E_CUDA;
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return CODENET_E_CUDA;
    g_scratch_ptr[dev] = static_cast<float*>(p);
  }
  *out = g_scratch_ptr[dev];
  return CODENET_OK;
}

}  // namespace

extern "C" int codenet_matvec_noalloc(const float* W_dev, int rows, int cols, int n_blocks, const float* x_dev,
                                      float* s_dev, codenet_stream_t stream) {
  if (!W_dev || !x_dev || !s_dev || rows < 1 || cols < 1 || n_blocks < 1) return CODENET_E_BADARG;
  if (n_blocks > CODENET_MAX_NODES || cols % n_blocks != 0 || (cols / n_blocks) % 4 != 0) return CODENET_E_SHAPE;
  if ((reinterpret_cast<uintptr_t>(W_dev) & 15u) || (reinterpret_cast<uintptr_t>(x_dev) & 15u)) return CODENET_E_BADARG;
  if ((size_t)rows * (size_t)n_blocks > kNoallocMaxFloats) return CODENET_E_TOOBIG;
  float* scratch = nullptr;
  const int rc = scratch_for_current_device(&scratch);
  if (rc != CODENET_OK) return rc;

  // the caller's matrix seen as one block-row of n_blocks uncoded blocks
  Geom g = {};
  g.n_out = rows; g.n_in = cols; g.m = 1; g.n = n_blocks; g.r_row = 0; g.r_col = 0;
  g.M = 1; g.Nn = n_blocks; g.b_r = rows; g.b_c = cols / n_blocks; g.ldb = g.b_c; g.ld = cols;
  g.T = rows; g.ns = 1; g.Tc = g.b_c; g.nsc = 1; g.Mbr = rows;
  g.dtype = CODENET_F32; g.locate_mode = CODENET_LOCATE_OFF; g.tau_rel = 0.0f; g.tau_abs = 0.0f;
  g.Wt = const_cast<float*>(W_dev);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  // every scratch element read by the sum is written by the product kernel of this same call,
  // so nothing has to start at zero
  if (launch_forward_products_plain(g, x_dev, cols, 1, scratch, st) != cudaSuccess) return CODENET_E_CUDA;
  if (launch_sum_outputs(g, CODENET_PHASE_FWD, 1, scratch, s_dev, CODENET_ACT_IDENTITY, nullptr, st) != cudaSuccess) return CODENET_E_CUDA;
  return CODENET_OK;
}
