// CUDA-core matrix multiply: Y[R][N] = X[R][K] * W[N][K]^T with fp32 accumulation, for any
// shape and for fp32 or bf16 operands.  Used for the fp32 configuration (strict fp32, no TF32),
// for shapes the tensor-core path does not take, and as the A/B reference of that path.
#include "common.cuh"

namespace koala {
namespace {

constexpr int FPW = 4;       // output features per warp
constexpr int ROWS = 16;     // X rows per block
constexpr int KC = 512;      // K elements staged per step
constexpr int WARPS = 8;

template <typename T>
__global__ void __launch_bounds__(WARPS * 32)
gemm_simt_kernel(const T *X, const T *Xlo, int R, int K_in, const T *__restrict__ W0,
                 const T *__restrict__ W1, const T *__restrict__ W2, int n0, int n1, int n2,
                 float *__restrict__ Y, int ldy) {
  __shared__ float xs[ROWS][KC + 1];
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int r0 = blockIdx.y * ROWS;
  const int ntot = n0 + n1 + n2;
  const T *wrow[FPW];
  int col[FPW];
#pragma unroll
  for (int f = 0; f < FPW; ++f) {
    int g = (blockIdx.x * WARPS + w) * FPW + f;
    col[f] = g;
    if (g >= ntot) g = ntot - 1;
    const T *base = W0;
    if (g >= n0 + n1) { base = W2; g -= n0 + n1; }
    else if (g >= n0) { base = W1; g -= n0; }
    wrow[f] = base + (size_t)g * K_in;
  }
  float acc[FPW][ROWS];
#pragma unroll
  for (int f = 0; f < FPW; ++f)
#pragma unroll
    for (int r = 0; r < ROWS; ++r) acc[f][r] = 0.f;

  for (int k0 = 0; k0 < K_in; k0 += KC) {
    __syncthreads();
    for (int e = threadIdx.x; e < ROWS * KC; e += WARPS * 32) {
      const int r = e / KC, k = e % KC;
      float v = 0.f;
      if (r0 + r < R && k0 + k < K_in) {
        const size_t idx = (size_t)(r0 + r) * K_in + k0 + k;
        v = to_f(X[idx]);
        if (Xlo != nullptr) v += to_f(Xlo[idx]);
      }
      xs[r][k] = v;
    }
    __syncthreads();
    const int kend = min(KC, K_in - k0);
    for (int k = lane; k < kend; k += 32) {
      float wv[FPW];
#pragma unroll
      for (int f = 0; f < FPW; ++f) wv[f] = to_f(wrow[f][k0 + k]);
#pragma unroll
      for (int r = 0; r < ROWS; ++r) {
        const float xv = xs[r][k];
#pragma unroll
        for (int f = 0; f < FPW; ++f) acc[f][r] = fmaf(wv[f], xv, acc[f][r]);
      }
    }
  }
#pragma unroll
  for (int f = 0; f < FPW; ++f)
#pragma unroll
    for (int r = 0; r < ROWS; ++r) {
      const float v = warp_sum(acc[f][r]);
      if (lane == 0 && col[f] < ntot && r0 + r < R) Y[(size_t)(r0 + r) * ldy + col[f]] = v;
    }
}

}  // namespace

cudaError_t gemm_simt(Launch L, int dtype, Operand X, GemmMats m, int K_in, int R, float *Y,
                      int ldy) {
  const int n0 = m.n_out[0], n1 = m.n > 1 ? m.n_out[1] : 0, n2 = m.n > 2 ? m.n_out[2] : 0;
  const int ntot = n0 + n1 + n2;
  dim3 grid((ntot + WARPS * FPW - 1) / (WARPS * FPW), (R + ROWS - 1) / ROWS);
  if (dtype == 0)
    return launch_k(gemm_simt_kernel<float>, grid, dim3(WARPS * 32), 0, L.st, L.pdl, (const float *)X.hi,
                    (const float *)X.lo, R, K_in, (const float *)m.W[0], (const float *)(m.n > 1 ? m.W[1] : m.W[0]),
                    (const float *)(m.n > 2 ? m.W[2] : m.W[0]), n0, n1, n2, Y, ldy);
  return launch_k(gemm_simt_kernel<bf16>, grid, dim3(WARPS * 32), 0, L.st, L.pdl, (const bf16 *)X.hi,
                  (const bf16 *)X.lo, R, K_in, (const bf16 *)m.W[0], (const bf16 *)(m.n > 1 ? m.W[1] : m.W[0]),
                  (const bf16 *)(m.n > 2 ? m.W[2] : m.W[0]), n0, n1, n2, Y, ldy);
}

}  // namespace koala
