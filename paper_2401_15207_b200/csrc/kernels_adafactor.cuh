// Adafactor (Shazeer & Stern 2018, Algorithms 4-5: factored second moment, update clipping,
// relative step size and parameter scaling, no momentum) for one parameter tensor, in the variant
// where eps1 is a lower clamp on the estimate (as torch.optim.Adafactor has it), not an addend to g^2.
//   w     = tau^-0.8                 (1 - beta2_t)
//   rho   = min(lr, 1/sqrt(tau)),  alpha = max(eps2, RMS(theta)) * rho
//   theta <- theta * (1 - lr * wd)
//   matrix [n,m]: R <- lerp(R, rowmean(g^2), w); C <- lerp(C, colmean(g^2), w); V_ij = R_i C_j / max(mean(R), eps1)
//   vector      : V <- lerp(V, g^2, w)
//   U = g / max(sqrt(V), eps1);  theta <- theta - alpha / max(1, RMS(U)/d) * U
// State per matrix is n + m floats instead of n*m: this is why the paper lists Adafactor with
// sub-megabyte optimizer-state traffic.  All reductions have a fixed order.
// `gate` (device int, may be null): when non-zero, every kernel that would write state or
// parameters returns at once (the training step failed; nothing may change).
#pragma once
#include "common.cuh"

namespace hift {

struct AfScalars { float w, rho, eps1, eps2, d, decay; };

// per row i: R_i <- lerp(R_i, mean_j g_ij^2, w);  row_tsq[i] = sum_j theta_ij^2
__global__ void af_row_kernel(const float* __restrict__ g, const float* __restrict__ theta,
                              float* __restrict__ R, float* __restrict__ row_tsq, int cols, float w,
                              const int* __restrict__ gate) {
  if (gate != nullptr && *gate != 0) return;
  __shared__ float red[33];
  const int64_t row = blockIdx.x;
  float a = 0.f, b = 0.f;
  for (int c = threadIdx.x; c < cols; c += blockDim.x) {
    const float x = g[row * cols + c], t = theta[row * cols + c];
    a += x * x;
    b += t * t;
  }
  a = block_sum(a, red);
  b = block_sum(b, red);
  if (threadIdx.x == 0) {
    const float m = a / cols;
    R[row] = R[row] + w * (m - R[row]);
    row_tsq[row] = b;
  }
}
// column sums of g^2 over a slab of rows: partial[chunk][col]; grid (ceil(cols/32), n_chunks), block 32 x 8
__global__ void af_col_stage1_kernel(const float* __restrict__ g, float* __restrict__ partial, int64_t rows, int cols) {
  __shared__ float sh[8][33];
  const int col = blockIdx.x * 32 + threadIdx.x;
  const int nch = gridDim.y;
  const int64_t per = (rows + nch - 1) / nch;
  const int64_t r0 = (int64_t)blockIdx.y * per;
  const int64_t r1 = r0 + per < rows ? r0 + per : rows;
  float a = 0.f;
  if (col < cols)
    for (int64_t r = r0 + threadIdx.y; r < r1; r += 8) { const float x = g[r * cols + col]; a += x * x; }
  sh[threadIdx.y][threadIdx.x] = a;
  __syncthreads();
  if (threadIdx.y == 0 && col < cols) {
    float t = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) t += sh[i][threadIdx.x];
    partial[(size_t)blockIdx.y * cols + col] = t;
  }
}
__global__ void af_col_stage2_kernel(const float* __restrict__ partial, int nch, int cols, int64_t rows,
                                     float* __restrict__ Cv, float w, const int* __restrict__ gate) {
  if (gate != nullptr && *gate != 0) return;
  const int col = blockIdx.x * blockDim.x + threadIdx.x;
  if (col >= cols) return;
  float t = 0.f;
  for (int c = 0; c < nch; ++c) t += partial[(size_t)c * cols + col];
  const float m = t / (float)rows;
  Cv[col] = Cv[col] + w * (m - Cv[col]);
}
// single block: scal[0] = max(mean(R), eps1); scal[1] = alpha
__global__ void af_scalars_kernel(const float* __restrict__ R, const float* __restrict__ row_tsq, int rows,
                                  double numel, float* __restrict__ scal, AfScalars h) {
  __shared__ float red[33];
  float a = 0.f, b = 0.f;
  for (int i = threadIdx.x; i < rows; i += blockDim.x) { a += R[i]; b += row_tsq[i]; }
  a = block_sum(a, red);
  b = block_sum(b, red);
  if (threadIdx.x == 0) {
    scal[0] = fmaxf(a / rows, h.eps1);
    scal[1] = fmaxf(h.eps2, sqrtf((float)((double)b / numel))) * h.rho;
  }
}
// per row: row_usq[i] = sum_j U_ij^2
__global__ void af_usq_kernel(const float* __restrict__ g, const float* __restrict__ R, const float* __restrict__ Cv,
                              const float* __restrict__ scal, float* __restrict__ row_usq, int cols, float eps1) {
  __shared__ float red[33];
  const int64_t row = blockIdx.x;
  const float ri = R[row] / scal[0];
  float a = 0.f;
  for (int c = threadIdx.x; c < cols; c += blockDim.x) {
    const float u = g[row * cols + c] * (1.0f / fmaxf(sqrtf(ri * Cv[c]), eps1));
    a += u * u;
  }
  a = block_sum(a, red);
  if (threadIdx.x == 0) row_usq[row] = a;
}
// single block: scal[2] = alpha / max(1, RMS(U)/d)
__global__ void af_step_kernel(const float* __restrict__ row_usq, int rows, double numel, float* __restrict__ scal, float d) {
  __shared__ float red[33];
  float a = 0.f;
  for (int i = threadIdx.x; i < rows; i += blockDim.x) a += row_usq[i];
  a = block_sum(a, red);
  if (threadIdx.x == 0) scal[2] = scal[1] / fmaxf(1.0f, sqrtf((float)((double)a / numel)) / d);
}
template <bool HAS_BF16>
__global__ void af_apply_kernel(bf16* __restrict__ param, float* __restrict__ theta, const float* __restrict__ g,
                                const float* __restrict__ R, const float* __restrict__ Cv, const float* __restrict__ scal,
                                int64_t rows, int cols, float eps1, float decay, const int* __restrict__ gate) {
  if (gate != nullptr && *gate != 0) return;
  const size_t n = (size_t)rows * cols;
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  const float m0 = scal[0], step = scal[2];
  for (; i < n; i += stride) {
    const size_t r = i / cols, c = i % cols;
    const float u = g[i] * (1.0f / fmaxf(sqrtf(R[r] / m0 * Cv[c]), eps1));
    const float t = theta[i] * decay - step * u;
    theta[i] = t;
    if (HAS_BF16) param[i] = __float2bfloat16_rn(t);
  }
}
// vectors (one block): V <- lerp(V, g^2, w); scal[1] = alpha; scal[2] = alpha / max(1, RMS(U)/d)
__global__ void af_vector_kernel(const float* __restrict__ g, const float* __restrict__ theta, float* __restrict__ V,
                                 int n, float* __restrict__ scal, AfScalars h, const int* __restrict__ gate) {
  if (gate != nullptr && *gate != 0) return;
  __shared__ float red[33];
  float a = 0.f, b = 0.f;
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    const float x = g[i];
    const float v = V[i] + h.w * (x * x - V[i]);
    V[i] = v;
    const float u = x * (1.0f / fmaxf(sqrtf(v), h.eps1));
    a += u * u;
    b += theta[i] * theta[i];
  }
  a = block_sum(a, red);
  b = block_sum(b, red);
  if (threadIdx.x == 0) {
    const float alpha = fmaxf(h.eps2, sqrtf(b / n)) * h.rho;
    scal[1] = alpha;
    scal[2] = alpha / fmaxf(1.0f, sqrtf(a / n) / h.d);
  }
}
template <bool HAS_BF16>
__global__ void af_vector_apply_kernel(bf16* __restrict__ param, float* __restrict__ theta, const float* __restrict__ g,
                                       const float* __restrict__ V, const float* __restrict__ scal, int n,
                                       float eps1, float decay, const int* __restrict__ gate) {
  if (gate != nullptr && *gate != 0) return;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const float u = g[i] * (1.0f / fmaxf(sqrtf(V[i]), eps1));
  const float t = theta[i] * decay - scal[2] * u;
  theta[i] = t;
  if (HAS_BF16) param[i] = __float2bfloat16_rn(t);
}

// state floats a tensor needs: n + m for a matrix, numel for a vector (rows == 1)
inline size_t af_state_floats(int64_t rows, int64_t cols) { return rows == 1 ? (size_t)cols : (size_t)(rows + cols); }
inline size_t af_scratch_floats(int64_t rows, int64_t cols) { return (size_t)(2 * rows) + 64 * (size_t)cols + 8; }

// Launches the update of one tensor.  state: R[rows] | C[cols] (matrix) or V[cols] (vector).
// scratch: at least af_scratch_floats(rows, cols) floats.  Returns the number of kernels launched.
inline int launch_adafactor_tensor(cudaStream_t st, int64_t rows, int64_t cols, void* param_bf16, float* master,
                                   const float* grad, float* state, float* scratch, double lr, double eps1, double wd,
                                   int64_t tau, const int* gate = nullptr) {
  AfScalars h;
  h.w = (float)pow((double)tau, -0.8);
  h.rho = (float)fmin(lr, 1.0 / sqrt((double)tau));
  h.eps1 = (float)eps1; h.eps2 = 1e-3f; h.d = 1.0f;
  h.decay = (float)(1.0 - lr * wd);
  const float e1sq = (float)eps1;     // the clamp is applied after the square root: eps1^2 would underflow in fp32
  if (rows == 1) {
    float* scal = scratch;
    af_vector_kernel<<<1, 256, 0, st>>>(grad, master, state, (int)cols, scal, h, gate);
    const int grid = (int)((cols + 255) / 256);
    if (param_bf16) af_vector_apply_kernel<true><<<grid, 256, 0, st>>>((bf16*)param_bf16, master, grad, state, scal, (int)cols, e1sq, h.decay, gate);
    else af_vector_apply_kernel<false><<<grid, 256, 0, st>>>(nullptr, master, grad, state, scal, (int)cols, e1sq, h.decay, gate);
    return 2;
  }
  float* R = state;
  float* Cv = state + rows;
  float* row_tsq = scratch;
  float* row_usq = scratch + rows;
  float* partial = scratch + 2 * rows;
  float* scal = partial + 64 * (size_t)cols;
  const double numel = (double)rows * (double)cols;
  af_row_kernel<<<(unsigned)rows, 256, 0, st>>>(grad, master, R, row_tsq, (int)cols, h.w, gate);
  int nch = (int)((rows + 31) / 32);
  if (nch > 64) nch = 64;
  if (nch < 1) nch = 1;
  af_col_stage1_kernel<<<dim3((unsigned)((cols + 31) / 32), nch), dim3(32, 8), 0, st>>>(grad, partial, rows, (int)cols);
  af_col_stage2_kernel<<<(unsigned)((cols + 127) / 128), 128, 0, st>>>(partial, nch, (int)cols, rows, Cv, h.w, gate);
  af_scalars_kernel<<<1, 1024, 0, st>>>(R, row_tsq, (int)rows, numel, scal, h);
  af_usq_kernel<<<(unsigned)rows, 256, 0, st>>>(grad, R, Cv, scal, row_usq, (int)cols, e1sq);
  af_step_kernel<<<1, 1024, 0, st>>>(row_usq, (int)rows, numel, scal, h.d);
  size_t n = (size_t)rows * cols;
  size_t g = (n + 255) / 256;
  if (g > 148 * 16) g = 148 * 16;
  if (param_bf16) af_apply_kernel<true><<<(unsigned)g, 256, 0, st>>>((bf16*)param_bf16, master, grad, R, Cv, scal, rows, (int)cols, e1sq, h.decay, gate);
  else af_apply_kernel<false><<<(unsigned)g, 256, 0, st>>>(nullptr, master, grad, R, Cv, scal, rows, (int)cols, e1sq, h.decay, gate);
  return 7;
}

}  // namespace hift
