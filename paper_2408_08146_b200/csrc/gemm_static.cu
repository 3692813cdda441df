// koala_gemm_bf16_static: the stand-alone weight-streaming GEMM for callers that must not allocate.
//
// The split-K partial sums of the tensor-core GEMM normally live in a scratch buffer that the
// caller allocates.  Some callers cannot do that: code running inside a real-time serving loop
// whose memory pool is fixed at start-up, plug-ins handed only input and output buffers by a host
// framework that owns all device memory, or code running while the process is near its memory
// limit, where a cudaMalloc could fail or stall every stream of the device.  For them the scratch
// is a fixed array in the library's own device image.
#include "../../include/koala.h"
#include "common.cuh"

#include <mutex>

namespace {

// 8 MiB of fp32 partial sums; every device that loads the library holds this until the process exits.
constexpr size_t STATIC_SCRATCH_FLOATS = (size_t)2 * 1024 * 1024;
static __device__ __align__(256) float g_static_scratch[STATIC_SCRATCH_FLOATS];

constexpr int MAX_DEVICES = 64;
constexpr int MAX_STATIC_SPLIT = 8;
float *g_scratch_ptr[MAX_DEVICES] = {nullptr};   // device address of the array, per device
std::mutex g_scratch_mu;

}  // namespace

extern "C" {
#pragma GCC visibility push(default)

size_t koala_gemm_static_scratch_bytes(void) { return STATIC_SCRATCH_FLOATS * sizeof(float); }

int koala_gemm_bf16_static(const void *X, const void *X_lo, const void *W, float *Y, int ldy, int M,
                           int N_out, int K_in, int split_k, void *cuda_stream, int *device_status) {
  using namespace koala;
  if (!X || !W || !Y || M < 1 || N_out < 1 || K_in < 1 || ldy < N_out) return KOALA_E_INVALID;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return KOALA_E_CUDA;
  if (dev < 0 || dev >= MAX_DEVICES) return KOALA_E_UNSUPPORTED;
  if (split_k < 0 || split_k > MAX_STATIC_SPLIT) return KOALA_E_INVALID;
  float *scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_scratch_mu);
    if (g_scratch_ptr[dev] == nullptr) {
      // The array's name is only a host-side handle; kernels need its address on the current device.
      // (With lazy module loading this look-up is also what gives the array its device memory.)
      float *p = nullptr;
      if (cudaGetSymbolAddress((void **)&p, g_static_scratch) != cudaSuccess || p == nullptr) return KOALA_E_CUDA;
      g_scratch_ptr[dev] = p;
    }
    scratch = g_scratch_ptr[dev];
  }
  char err[160];
  if (tc_init_driver(err, sizeof(err)) != 0) return KOALA_E_CUDA;   // prepares this device once
  GemmMats m{{W, nullptr, nullptr}, {N_out, 0, 0}, 1};
  if (!tc_supported(m, K_in)) return KOALA_E_UNSUPPORTED;
  const size_t stride = (size_t)M * N_out;
  int split = split_k;
  if (split == 0) {
    // automatic: the factor the GEMM would choose, lowered until its partial sums fit in the array
    // (a caller that cannot allocate has no other entry point to fall back to)
    split = tc_default_split((N_out + 127) / 128, K_in / 64, M);
    if (split > MAX_STATIC_SPLIT) split = MAX_STATIC_SPLIT;
    const size_t fit = STATIC_SCRATCH_FLOATS / stride;
    if ((size_t)split > fit) split = fit < 1 ? 1 : (int)fit;
  }
  if (split > K_in / 64) split = K_in / 64;
  Launch L{(cudaStream_t)cuda_stream, false};
  Operand Xo{const_cast<void *>(X), const_cast<void *>(X_lo)};
  const int rows_alloc = koala_gemm_x_rows(M, X_lo != nullptr);
  if (split == 1)
    return gemm_tc(L, Xo, rows_alloc, m, K_in, M, Y, ldy, 1, 0, device_status, 1, nullptr) == cudaSuccess ? KOALA_OK
                                                                                              : KOALA_E_CUDA;
  if ((size_t)split * stride > STATIC_SCRATCH_FLOATS) return KOALA_E_CAPACITY;   // an explicit factor that does not fit
  // every partial element that is read below is written by exactly one CTA of this launch, so the
  // previous call's contents need no clearing
  SplitIn s;
  if (gemm_tc(L, Xo, rows_alloc, m, K_in, M, scratch, N_out, split, stride, device_status, split, &s) != cudaSuccess)
    return KOALA_E_CUDA;
  return reduce_splits(L, s, Y, ldy, M, N_out) == cudaSuccess ? KOALA_OK : KOALA_E_CUDA;
}

#pragma GCC visibility pop
}
