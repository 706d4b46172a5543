// Plain CUDA-core GEMM with arbitrary operand strides and fp32 accumulation.  It serves
// (a) every contraction of the fp32 configuration, where tensor cores (tf32/bf16) would not
// meet a 1e-5 tolerance, and (b) bf16 shapes the tensor-core kernel does not take (tiny or
// misaligned problems such as the 2-class head).
//
//   C[m,n] = sum_k A(m,k) * B(k,n) (+ bias[n]) (+ residual[m,n], fp32 residual stream),
//   A(m,k) = a[m*sam + k*sak],  B(k,n) = b[k*sbk + n*sbn].
#pragma once
#include "common.cuh"

namespace hift {

template <typename TIN, typename TOUT>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(int M, int N, int K, const TIN* __restrict__ a, int64_t sam, int64_t sak,
                 const TIN* __restrict__ b, int64_t sbk, int64_t sbn, TOUT* __restrict__ c,
                 int64_t ldc, const TIN* __restrict__ bias, const float* __restrict__ residual,
                 int64_t ldr) {
  constexpr int BM = 64, BN = 64, BK = 16;
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];
  const int tid = threadIdx.x;
  const int tx = tid % 16, ty = tid / 16;            // 16 x 16 threads, 4 x 4 outputs each
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  const bool a_k_fast = (sak == 1);
  const bool b_n_fast = (sbn == 1);
  for (int k0 = 0; k0 < K; k0 += BK) {
#pragma unroll
    for (int it = 0; it < (BM * BK) / 256; ++it) {
      const int idx = it * 256 + tid;
      int mm, kk;
      if (a_k_fast) { kk = idx % BK; mm = idx / BK; } else { mm = idx % BM; kk = idx / BM; }
      const int gm = m0 + mm, gk = k0 + kk;
      As[kk][mm] = (gm < M && gk < K) ? to_f(a[(int64_t)gm * sam + (int64_t)gk * sak]) : 0.f;
    }
#pragma unroll
    for (int it = 0; it < (BN * BK) / 256; ++it) {
      const int idx = it * 256 + tid;
      int nn, kk;
      if (b_n_fast) { nn = idx % BN; kk = idx / BN; } else { kk = idx % BK; nn = idx / BK; }
      const int gn = n0 + nn, gk = k0 + kk;
      Bs[kk][nn] = (gn < N && gk < K) ? to_f(b[(int64_t)gk * sbk + (int64_t)gn * sbn]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float av[4], bv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) av[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) bv[j] = Bs[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int gm = m0 + ty * 4 + i;
    if (gm >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int gn = n0 + tx * 4 + j;
      if (gn >= N) continue;
      float v = acc[i][j];
      if (bias) v += to_f(bias[gn]);
      if (residual) v += residual[(int64_t)gm * ldr + gn];
      c[(int64_t)gm * ldc + gn] = from_f<TOUT>(v);
    }
  }
}

// The same contraction for products with few outputs and a long k (the 2-class head: 16 x 2 outputs over k = 768):
// one warp per output element, lanes strided over k, a fixed shuffle tree at the end.  The tiled kernel above would
// run such a product in one block, k-step by k-step.
template <typename TIN, typename TOUT>
__global__ void __launch_bounds__(256)
gemm_few_outputs_kernel(int M, int N, int K, const TIN* __restrict__ a, int64_t sam, int64_t sak,
                        const TIN* __restrict__ b, int64_t sbk, int64_t sbn, TOUT* __restrict__ c,
                        int64_t ldc, const TIN* __restrict__ bias, const float* __restrict__ residual,
                        int64_t ldr) {
  const int lane = threadIdx.x & 31;
  const int64_t out = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (out >= (int64_t)M * N) return;
  const int m = (int)(out / N), n = (int)(out % N);
  const TIN* ap = a + (int64_t)m * sam;
  const TIN* bp = b + (int64_t)n * sbn;
  float acc = 0.f;
  for (int k = lane; k < K; k += 32) acc = fmaf(to_f(ap[(int64_t)k * sak]), to_f(bp[(int64_t)k * sbk]), acc);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) {
    if (bias) acc += to_f(bias[n]);
    if (residual) acc += residual[(int64_t)m * ldr + n];
    c[(int64_t)m * ldc + n] = from_f<TOUT>(acc);
  }
}

}  // namespace hift
