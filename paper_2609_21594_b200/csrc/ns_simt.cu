// Plain CUDA-core batched product kernel for the Newton-Schulz iteration (Eq. 1).
// It serves the fp32 precision mode (every product in true fp32: TF32 operands are not
// accurate enough for a 1e-4 match to fp64) and shapes the tensor-core engine does not take.
//   C[k] = gamma_k * (beta * D[k] + alpha * P[k] Q[k]^T + diag * I)   (nn = 0:  A = X X^T,  P = aI + bA + c A A^T)
//   C[k] = gamma_k * (beta * D[k] + alpha * P[k] Q[k])                (nn = 1:  X' = P X)
#include "internal.h"

namespace muon {
namespace {

constexpr int BM = 64, BN = 64, BK = 16;

template <typename T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ T cvt(float v);
template <> __device__ __forceinline__ float cvt<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 cvt<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

template <typename T, bool NN>
__global__ void __launch_bounds__(256) gemm_simt_kernel(GemmArgs a, int tiles_m, int tiles_n) {
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];
  const int per = tiles_m * tiles_n;
  const int mat = blockIdx.x / per;
  const int t = blockIdx.x - mat * per;
  const int m0 = (t / tiles_n) * BM, n0 = (t % tiles_n) * BN;
  const T* __restrict__ P = static_cast<const T*>(a.p) + size_t(mat) * a.stride_p;
  const T* __restrict__ Q = static_cast<const T*>(a.q) + size_t(mat) * a.stride_q;
  const T* __restrict__ D = a.d ? static_cast<const T*>(a.d) + size_t(mat) * a.stride_c : nullptr;
  T* __restrict__ C = static_cast<T*>(a.c) + size_t(mat) * a.stride_c;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (int k0 = 0; k0 < a.kdim; k0 += BK) {
    {  // P tile: 64 rows x 16 k
      const int i = tid >> 2, kk = (tid & 3) * 4;
      const int r = m0 + i;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int k = k0 + kk + e;
        As[kk + e][i] = (r < a.m && k < a.kdim) ? ldf<T>(P + size_t(r) * a.ldp + k) : 0.f;
      }
    }
    if (!NN) {  // Q tile: 64 rows (n) x 16 k
      const int j = tid >> 2, kk = (tid & 3) * 4;
      const int r = n0 + j;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int k = k0 + kk + e;
        Bs[kk + e][j] = (r < a.n && k < a.kdim) ? ldf<T>(Q + size_t(r) * a.ldq + k) : 0.f;
      }
    } else {    // Q tile: 16 k x 64 cols
      const int kk = tid >> 4, j = (tid & 15) * 4;
      const int k = k0 + kk;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int c = n0 + j + e;
        Bs[kk][j + e] = (k < a.kdim && c < a.n) ? ldf<T>(Q + size_t(k) * a.ldq + c) : 0.f;
      }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      float av[4], bv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) av[i] = As[k][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) bv[j] = Bs[k][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
  float gamma = 1.f;
  if (a.gamma_mode) {
    const float r = a.rnorm[mat];
    gamma = a.gamma_mode == 1 ? r : r * r;
  }
  float alpha = a.alpha, beta = a.beta, diag = a.diag;
  if (a.coef) {
    const float* co = a.coef + size_t(mat) * size_t(a.coef_stride);
    if (a.coef_a >= 0) alpha = co[a.coef_a];
    if (a.coef_b >= 0) beta = co[a.coef_b];
    if (a.coef_d >= 0) diag = co[a.coef_d];
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = m0 + ty * 4 + i;
    if (r >= a.m) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = n0 + tx * 4 + j;
      if (c >= a.n) continue;
      const size_t off = size_t(r) * a.ldc + c;
      float v = alpha * acc[i][j];
      if (D) v += beta * ldf<T>(D + off);
      if (r == c) v += diag;
      C[off] = cvt<T>(gamma * v);
    }
  }
}

}  // namespace

int launch_gemm_simt(const GemmArgs& a, int ns_precision, cudaStream_t st) {
  if (a.batch == 0 || a.m == 0 || a.n == 0) return 0;
  const int tiles_m = (a.m + BM - 1) / BM, tiles_n = (a.n + BN - 1) / BN;
  const int64_t blocks = int64_t(tiles_m) * tiles_n * a.batch;
  if (blocks > 0x7fffffffLL) return MUON_ERR_UNSUPPORTED;
  const unsigned g = unsigned(blocks);
  if (ns_precision == MUON_NS_FP32) {
    if (a.nn) gemm_simt_kernel<float, true><<<g, 256, 0, st>>>(a, tiles_m, tiles_n);
    else gemm_simt_kernel<float, false><<<g, 256, 0, st>>>(a, tiles_m, tiles_n);
  } else {
    if (a.nn) gemm_simt_kernel<__nv_bfloat16, true><<<g, 256, 0, st>>>(a, tiles_m, tiles_n);
    else gemm_simt_kernel<__nv_bfloat16, false><<<g, 256, 0, st>>>(a, tiles_m, tiles_n);
  }
  return cudaGetLastError() == cudaSuccess ? 1 : MUON_ERR_CUDA;
}

}  // namespace muon
