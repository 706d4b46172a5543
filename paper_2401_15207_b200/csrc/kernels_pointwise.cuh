// Bandwidth-bound kernels of the training step: embedding, LayerNorm/RMSNorm, GELU/SwiGLU,
// RoPE, softmax cross-entropy, column reductions (bias and gain gradients), the fused
// group-local optimizer, and small utilities.  All reductions have a fixed order.
//
// The residual stream and its gradient are fp32 in every configuration; P / T below is the
// parameter and GEMM-operand type (bf16 or fp32).
#pragma once
#include "common.cuh"
#include "dropout_rng.cuh"

namespace hift {

// ------------------------------------------------------------------ utilities
template <typename T>
__global__ void cast_from_f32_kernel(const float* __restrict__ src, T* __restrict__ dst, size_t n) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (; i < n; i += stride) dst[i] = from_f<T>(src[i]);
}
template <typename T>
__global__ void cast_to_f32_kernel(const T* __restrict__ src, float* __restrict__ dst, size_t n) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (; i < n; i += stride) dst[i] = to_f(src[i]);
}

// Counter-based synthetic weights: element i of stream `seed` is a Box-Muller normal built
// from the two 32-bit halves of a SplitMix64-style finaliser of (seed, i).
__device__ __forceinline__ uint64_t mix64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
template <typename T>
__global__ void init_tensor_kernel(T* __restrict__ param, float* __restrict__ master, size_t n,
                                   int kind, float stdv, uint64_t seed) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (; i < n; i += stride) {
    float v;
    if (kind == 0) {
      uint64_t h = mix64(seed + 0x9E3779B97F4A7C15ull * (uint64_t)(i + 1));
      float u1 = ((uint32_t)(h >> 32) + 1.0f) * (1.0f / 4294967808.0f);
      float u2 = (uint32_t)h * (1.0f / 4294967296.0f);
      v = stdv * sqrtf(-2.0f * logf(u1)) * cospif(2.0f * u2);
    } else {
      v = kind == 1 ? 1.0f : 0.0f;
    }
    if (master) master[i] = v;
    param[i] = from_f<T>(v);
  }
}

// ------------------------------------------------------------------ embedding
// x[t,:] = tok[id[t],:] (+ pos[t mod S,:]), written to the fp32 residual stream.
// One block per token row.  An id outside [0, vocab) is clamped (never gathered out of
// bounds) and reported through *bad.
template <typename T>
__global__ void embed_fwd_kernel(const int32_t* __restrict__ ids, const T* __restrict__ tok,
                                 const T* __restrict__ pos, float* __restrict__ x, int S, int d,
                                 int vocab, int* __restrict__ bad) {
  const int t = blockIdx.x;
  int id = ids[t];
  if (id < 0 || id >= vocab) {
    if (threadIdx.x == 0) *bad = 1;
    id = id < 0 ? 0 : vocab - 1;
  }
  const T* tr = tok + (size_t)id * d;
  const T* pr = pos ? pos + (size_t)(t % S) * d : nullptr;
  float* xr = x + (size_t)t * d;
  for (int c = threadIdx.x * 8; c < d; c += blockDim.x * 8) {
    float a[8];
    load8(tr + c, a);
    if (pr) {
      float b[8];
      load8(pr + c, b);
#pragma unroll
      for (int i = 0; i < 8; ++i) a[i] += b[i];
    }
    store8(xr + c, a);
  }
}

// Gradients live in one flat buffer of fp32 or (hift_opt_cfg.grad_bf16) bf16 elements; the small producers
// take the buffer as void* plus the element type.
__device__ __forceinline__ float grad_load(const void* g, size_t i, int bf) {
  return bf ? __bfloat162float(reinterpret_cast<const bf16*>(g)[i]) : reinterpret_cast<const float*>(g)[i];
}
__device__ __forceinline__ void grad_store(void* g, size_t i, float v, int bf) {
  if (bf) reinterpret_cast<bf16*>(g)[i] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(g)[i] = v;
}
// grad_tok[id,:] += sum over positions t with ids[t] == id of dx[t,:], occurrences added in
// increasing t.  Block t does the work for id = ids[t] only if t is the first occurrence, so
// every gradient row has one writer and a fixed summation order (no atomics).  The positions of
// the id are collected in order into a list of kEmbedOccCap entries; a full list is summed into
// the gradient row and emptied, so the number of positions is not bounded by shared memory.
constexpr int kEmbedOccCap = 2048;
__global__ void embed_bwd_tok_kernel(const int32_t* __restrict__ ids, const float* __restrict__ dx,
                                     void* __restrict__ grad_tok, int gbf, int Ttot, int d, int vocab) {
  __shared__ int occ[kEmbedOccCap];                  // positions of this id, in order
  __shared__ int n_occ;
  __shared__ int warp_cnt[32];
  const int t0 = blockIdx.x;
  const int id = ids[t0];
  if (id < 0 || id >= vocab) return;                 // reported by the forward pass
  int found = 0;
  for (int t = threadIdx.x; t < t0; t += blockDim.x) found |= (ids[t] == id);
  if (__syncthreads_or(found)) return;
  if (threadIdx.x == 0) n_occ = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
  const size_t row = (size_t)id * d;
  auto drain = [&](int n) {                          // gradient row += the listed positions, in order
    for (int c = threadIdx.x; c < d; c += blockDim.x) {
      float acc = 0.f;
      for (int i = 0; i < n; ++i) acc += dx[(size_t)occ[i] * d + c];
      grad_store(grad_tok, row + c, grad_load(grad_tok, row + c, gbf) + acc, gbf);   // on top of a tied head's share
    }
  };
  // ordered compaction, one blockDim-sized chunk at a time
  for (int base = t0; base < Ttot; base += blockDim.x) {
    if (n_occ + (int)blockDim.x > kEmbedOccCap) {    // uniform: n_occ is read after a barrier
      drain(n_occ);
      __syncthreads();
      if (threadIdx.x == 0) n_occ = 0;
      __syncthreads();
    }
    const int t = base + threadIdx.x;
    const int hit = (t < Ttot) && (ids[t] == id);
    const unsigned bal = __ballot_sync(0xffffffffu, hit);
    if (lane == 0) warp_cnt[w] = __popc(bal);
    __syncthreads();
    int off = n_occ;
    for (int i = 0; i < w; ++i) off += warp_cnt[i];
    if (hit) occ[off + __popc(bal & ((1u << lane) - 1u))] = t;
    __syncthreads();
    if (threadIdx.x == 0) {
      int tot = 0;
      for (int i = 0; i < nw; ++i) tot += warp_cnt[i];
      n_occ += tot;
    }
    __syncthreads();
  }
  drain(n_occ);
}

// grad_pos[s,:] = sum over batch rows b of dx[b*S+s,:]
__global__ void embed_bwd_pos_kernel(const float* __restrict__ dx, void* __restrict__ grad_pos, int gbf,
                                     int B, int S, int d) {
  const int s = blockIdx.x;
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    float acc = 0.f;
    for (int b = 0; b < B; ++b) acc += dx[((size_t)b * S + s) * d + c];
    grad_store(grad_pos, (size_t)s * d + c, acc, gbf);
  }
}

// ------------------------------------------------------------------ norms
// KIND 0: LayerNorm y = (x-mean)*rstd*g + b; KIND 1: RMSNorm y = x*rstd*g.
// stats[row] = mean (0 for RMSNorm), stats[rows+row] = rstd.  cols % 8 == 0.
// y_a (type P) feeds the next GEMM; y_r (fp32, optional) continues the residual stream.
template <typename P, int KIND>
__global__ void norm_fwd_kernel(const float* __restrict__ x, const P* __restrict__ gain,
                                const P* __restrict__ bias, P* __restrict__ y_a,
                                float* __restrict__ y_r, float* __restrict__ stats, int64_t rows,
                                int cols, float eps) {
  pdl_launch_next();
  pdl_wait_prior();
  __shared__ float red[33];
  const int64_t row = blockIdx.x;
  const float* xr = x + row * cols;
  float mean = 0.f;
  if (KIND == 0) {
    float s = 0.f;
    for (int c = threadIdx.x * 8; c < cols; c += blockDim.x * 8) {
      float v[8];
      load8(xr + c, v);
#pragma unroll
      for (int i = 0; i < 8; ++i) s += v[i];
    }
    mean = block_sum(s, red) / cols;
  }
  float q = 0.f;
  for (int c = threadIdx.x * 8; c < cols; c += blockDim.x * 8) {
    float v[8];
    load8(xr + c, v);
#pragma unroll
    for (int i = 0; i < 8; ++i) q += (v[i] - mean) * (v[i] - mean);
  }
  const float var = block_sum(q, red) / cols;
  const float rstd = 1.0f / sqrtf(var + eps);
  if (threadIdx.x == 0) {
    stats[row] = mean;
    stats[rows + row] = rstd;
  }
  for (int c = threadIdx.x * 8; c < cols; c += blockDim.x * 8) {
    float v[8], g[8];
    load8(xr + c, v);
    load8(gain + c, g);
    if (KIND == 0) {
      float b[8];
      load8(bias + c, b);
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = (v[i] - mean) * rstd * g[i] + b[i];
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = v[i] * rstd * g[i];
    }
    store8(y_a + row * cols + c, v);
    if (y_r) store8(y_r + row * cols + c, v);
  }
}

// The same with the row held in registers: every thread loads its NC chunks of 8 once (cols <= 8 * NC * blockDim.x) and the
// two reductions and the output run from registers; per-thread and block summation orders are those of the kernel above,
// so the results are the same bits.
template <typename P, int KIND, int NC>
__global__ void norm_fwd_reg_kernel(const float* __restrict__ x, const P* __restrict__ gain,
                                    const P* __restrict__ bias, P* __restrict__ y_a,
                                    float* __restrict__ y_r, float* __restrict__ stats, int64_t rows,
                                    int cols, float eps) {
  pdl_launch_next();
  pdl_wait_prior();
  __shared__ float red[33];
  const int64_t row = blockIdx.x;
  const float* xr = x + row * cols;
  float v[NC][8];
#pragma unroll
  for (int k = 0; k < NC; ++k) {
    const int c = (threadIdx.x + k * blockDim.x) * 8;
    if (c < cols) load8(xr + c, v[k]);
    else {
#pragma unroll
      for (int i = 0; i < 8; ++i) v[k][i] = 0.f;
    }
  }
  float mean = 0.f;
  if (KIND == 0) {
    float s = 0.f;
#pragma unroll
    for (int k = 0; k < NC; ++k) {
      if ((threadIdx.x + k * blockDim.x) * 8 < cols) {
#pragma unroll
        for (int i = 0; i < 8; ++i) s += v[k][i];
      }
    }
    mean = block_sum(s, red) / cols;
  }
  float q = 0.f;
#pragma unroll
  for (int k = 0; k < NC; ++k) {
    if ((threadIdx.x + k * blockDim.x) * 8 < cols) {
#pragma unroll
      for (int i = 0; i < 8; ++i) q += (v[k][i] - mean) * (v[k][i] - mean);
    }
  }
  const float var = block_sum(q, red) / cols;
  const float rstd = 1.0f / sqrtf(var + eps);
  if (threadIdx.x == 0) {
    stats[row] = mean;
    stats[rows + row] = rstd;
  }
#pragma unroll
  for (int k = 0; k < NC; ++k) {
    const int c = (threadIdx.x + k * blockDim.x) * 8;
    if (c >= cols) continue;
    float g[8];
    load8(gain + c, g);
    if (KIND == 0) {
      float b[8];
      load8(bias + c, b);
#pragma unroll
      for (int i = 0; i < 8; ++i) v[k][i] = (v[k][i] - mean) * rstd * g[i] + b[i];
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) v[k][i] = v[k][i] * rstd * g[i];
    }
    store8(y_a + row * cols + c, v[k]);
    if (y_r) store8(y_r + row * cols + c, v[k]);
  }
}

// dx = norm_bwd(dy; x, stats, gain) (+ add).  One block per row.  dy is either a GEMM
// output (type P) or a residual-stream gradient (fp32).  dx_r: fp32 stream gradient;
// dx_a (optional): the same values rounded once to the GEMM-operand type.
template <typename DY, typename P, int KIND>
__global__ void norm_bwd_dx_kernel(const DY* __restrict__ dy, const float* __restrict__ x,
                                   const float* __restrict__ stats, const P* __restrict__ gain,
                                   const float* __restrict__ add, float* __restrict__ dx_r,
                                   P* __restrict__ dx_a, int64_t rows, int cols) {
  pdl_launch_next();
  pdl_wait_prior();
  __shared__ float red[33];
  const int64_t row = blockIdx.x;
  const float mean = stats[row], rstd = stats[rows + row];
  const DY* dyr = dy + row * cols;
  const float* xr = x + row * cols;
  float s1 = 0.f, s2 = 0.f;
  for (int c = threadIdx.x * 8; c < cols; c += blockDim.x * 8) {
    float a[8], v[8], g[8];
    load8(dyr + c, a);
    load8(xr + c, v);
    load8(gain + c, g);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float dxh = a[i] * g[i];
      if (KIND == 0) {
        s1 += dxh;
        s2 += dxh * (v[i] - mean) * rstd;
      } else {
        s2 += dxh * v[i];
      }
    }
  }
  if (KIND == 0) s1 = block_sum(s1, red) / cols;
  s2 = block_sum(s2, red) / cols;
  const float* ar = add ? add + row * cols : nullptr;
  for (int c = threadIdx.x * 8; c < cols; c += blockDim.x * 8) {
    float a[8], v[8], g[8], o[8];
    load8(dyr + c, a);
    load8(xr + c, v);
    load8(gain + c, g);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float dxh = a[i] * g[i];
      if (KIND == 0) {
        const float xh = (v[i] - mean) * rstd;
        o[i] = rstd * (dxh - s1 - xh * s2);
      } else {
        o[i] = rstd * dxh - v[i] * rstd * rstd * rstd * s2;
      }
    }
    if (ar) {
      float r[8];
      load8(ar + c, r);
#pragma unroll
      for (int i = 0; i < 8; ++i) o[i] += r[i];
    }
    if (dx_r) store8(dx_r + row * cols + c, o);
    if (dx_a) store8(dx_a + row * cols + c, o);
  }
}

// ------------------------------------------------------------------ column reductions
// Stage 1: partial[chunk][col] over a slab of rows.  MODE 0: sum dy (bias gradient).
// MODE 1: LayerNorm: p0 = sum dy*xhat, p1 = sum dy.  MODE 2: RMSNorm: p0 = sum dy*x*rstd.
// Block = 32 x 8 threads over 32 columns; grid = (ceil(cols/32), n_chunks).
// partial layout: [2][n_chunks][cols].  x is the fp32 residual stream.  With fp32 dy the
// sums run in double: these sums cancel heavily and the fp32 configuration is held to 1e-5.
constexpr int kColChunks = 64;
template <typename T> struct ColAcc { typedef float type; };
template <> struct ColAcc<float> { typedef double type; };
template <typename DY, int MODE>
__global__ void colreduce_stage1_kernel(const DY* __restrict__ dy, int64_t ld,
                                        const float* __restrict__ x, const float* __restrict__ stats,
                                        float* __restrict__ partial, int64_t rows, int cols) {
  typedef typename ColAcc<DY>::type acc_t;
  __shared__ acc_t sh0[8][33], sh1[8][33];
  const int col = blockIdx.x * 32 + threadIdx.x;
  const int nch = gridDim.y;
  const int64_t per = (rows + nch - 1) / nch;
  const int64_t r0 = (int64_t)blockIdx.y * per;
  const int64_t r1 = r0 + per < rows ? r0 + per : rows;
  acc_t a0 = 0, a1 = 0;
  if (col < cols) {
    for (int64_t r = r0 + threadIdx.y; r < r1; r += 8) {
      const float g = to_f(dy[r * ld + col]);
      if (MODE == 0) {
        a0 += g;
      } else if (MODE == 1) {
        const float xh = (x[r * cols + col] - stats[r]) * stats[rows + r];
        a0 += (acc_t)g * xh;
        a1 += g;
      } else {
        a0 += (acc_t)g * (x[r * cols + col] * stats[rows + r]);
      }
    }
  }
  sh0[threadIdx.y][threadIdx.x] = a0;
  sh1[threadIdx.y][threadIdx.x] = a1;
  __syncthreads();
  if (threadIdx.y == 0 && col < cols) {
    acc_t t0 = 0, t1 = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      t0 += sh0[i][threadIdx.x];
      t1 += sh1[i][threadIdx.x];
    }
    partial[((size_t)0 * nch + blockIdx.y) * cols + col] = (float)t0;
    if (MODE == 1) partial[((size_t)1 * nch + blockIdx.y) * cols + col] = (float)t1;
  }
}
// Stage 2: out0[col] = sum_chunk partial[0][chunk][col] (and out1 likewise from plane 1).
__global__ void colreduce_stage2_kernel(const float* __restrict__ partial, int nch, int cols,
                                        void* __restrict__ out0, void* __restrict__ out1, int gbf) {
  const int col = blockIdx.x * blockDim.x + threadIdx.x;
  if (col >= cols) return;
  double t0 = 0.0, t1 = 0.0;
  for (int c = 0; c < nch; ++c) {
    t0 += partial[((size_t)c) * cols + col];
    if (out1) t1 += partial[((size_t)nch + c) * cols + col];
  }
  grad_store(out0, col, (float)t0, gbf);
  if (out1) grad_store(out1, col, (float)t1, gbf);
}

// ------------------------------------------------------------------ activations
__device__ __forceinline__ float gelu_f(float a) {
  return 0.5f * a * (1.0f + erff(a * 0.70710678118654752440f));
}
__device__ __forceinline__ float gelu_grad_f(float a) {
  const float cdf = 0.5f * (1.0f + erff(a * 0.70710678118654752440f));
  const float pdf = expf(-0.5f * a * a) * 0.39894228040143267794f;
  return cdf + a * pdf;
}
template <typename T>
__global__ void gelu_fwd_kernel(const T* __restrict__ a, T* __restrict__ u, size_t n8) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (; i < n8; i += stride) {
    float v[8];
    load8(a + i * 8, v);
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = gelu_f(v[j]);
    store8(u + i * 8, v);
  }
}
// du <- du * gelu'(a), in place
template <typename T>
__global__ void gelu_bwd_kernel(T* __restrict__ du, const T* __restrict__ a, size_t n8) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (; i < n8; i += stride) {
    float v[8], g[8];
    load8(a + i * 8, v);
    load8(du + i * 8, g);
#pragma unroll
    for (int j = 0; j < 8; ++j) g[j] *= gelu_grad_f(v[j]);
    store8(du + i * 8, g);
  }
}
// s[t,j] = silu(gu[t,j]) * gu[t,f+j];  f % 8 == 0
template <typename T>
__global__ void swiglu_fwd_kernel(const T* __restrict__ gu, T* __restrict__ s, int64_t rows, int f) {
  const size_t f8 = f / 8, n8 = (size_t)rows * f8;
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (; i < n8; i += stride) {
    const size_t r = i / f8, c = (i % f8) * 8;
    float g[8], u[8];
    load8(gu + r * 2 * f + c, g);
    load8(gu + r * 2 * f + f + c, u);
#pragma unroll
    for (int j = 0; j < 8; ++j) g[j] = g[j] / (1.0f + expf(-g[j])) * u[j];
    store8(s + r * f + c, g);
  }
}
// dgu[t,j] = ds*up*sig*(1+g(1-sig)); dgu[t,f+j] = ds*g*sig
template <typename T>
__global__ void swiglu_bwd_kernel(const T* __restrict__ ds, const T* __restrict__ gu,
                                  T* __restrict__ dgu, int64_t rows, int f) {
  const size_t f8 = f / 8, n8 = (size_t)rows * f8;
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (; i < n8; i += stride) {
    const size_t r = i / f8, c = (i % f8) * 8;
    float g[8], u[8], d[8], o0[8], o1[8];
    load8(gu + r * 2 * f + c, g);
    load8(gu + r * 2 * f + f + c, u);
    load8(ds + r * f + c, d);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float sig = 1.0f / (1.0f + expf(-g[j]));
      o0[j] = d[j] * u[j] * sig * (1.0f + g[j] * (1.0f - sig));
      o1[j] = d[j] * g[j] * sig;
    }
    store8(dgu + r * 2 * f + c, o0);
    store8(dgu + r * 2 * f + f + c, o1);
  }
}

// ------------------------------------------------------------------ RoPE
// In place on the q and k column blocks of qkv[T,3d]: pair (j, j+half) of every head rotated
// by angle(pos, j) (sign = +1) or its inverse (sign = -1).  cs: [S, half] cos | [S, half] sin.
// One thread rotates 8 consecutive pairs of q and of k (16-byte accesses); half % 8 == 0.
template <typename T>
__global__ void rope_kernel(T* __restrict__ qkv, const float* __restrict__ cs, int64_t Ttot, int S,
                            int H, int dh, float sign) {
  pdl_launch_next();
  pdl_wait_prior();
  const int half = dh / 2, hc = half / 8;
  const size_t n = (size_t)Ttot * H * hc;
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  const int d = H * dh;
  for (; i < n; i += stride) {
    const int j = (int)(i % hc) * 8;
    const int h = (int)((i / hc) % H);
    const size_t t = i / ((size_t)hc * H);
    const int pos = (int)(t % S);
    float c[8], sn[8];
    load8(cs + (size_t)pos * half + j, c);
    load8(cs + (size_t)S * half + (size_t)pos * half + j, sn);
#pragma unroll
    for (int part = 0; part < 2; ++part) {          // q then k
      T* p = qkv + t * 3 * d + (size_t)part * d + (size_t)h * dh + j;
      float x1[8], x2[8], y1[8], y2[8];
      load8(p, x1);
      load8(p + half, x2);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float s = sign * sn[e];
        y1[e] = x1[e] * c[e] - x2[e] * s;
        y2[e] = x1[e] * s + x2[e] * c[e];
      }
      store8(p, y1);
      store8(p + half, y2);
    }
  }
}

// ------------------------------------------------------------------ softmax cross-entropy
// nvalid[0] = number of labels >= 0  (single block)
__global__ void count_valid_kernel(const int32_t* __restrict__ labels, int64_t n, int* nvalid) {
  __shared__ float red[33];
  float c = 0.f;
  for (int64_t i = threadIdx.x; i < n; i += blockDim.x) c += labels[i] >= 0 ? 1.f : 0.f;
  c = block_sum(c, red);
  if (threadIdx.x == 0) nvalid[0] = (int)(c + 0.5f);
}
// One block per row.  rowloss[row] = lse - logit[label] (0 if ignored); logits overwritten by
// (softmax - onehot)/nvalid, zeros for ignored rows and padding columns.  A label >= vocab sets
// *bad = 1 and the row is treated as ignored.
template <typename T>
__global__ void cross_entropy_kernel(T* __restrict__ logits, const int32_t* __restrict__ labels,
                                     float* __restrict__ rowloss, const int* __restrict__ nvalid,
                                     int* __restrict__ bad, int64_t vocab, int64_t ld) {
  __shared__ float red[33];
  const int64_t row = blockIdx.x;
  T* lr = logits + row * ld;
  int label = labels[row];
  if (label >= vocab) {
    if (threadIdx.x == 0) *bad = 1;
    label = -1;
  }
  if (label < 0) {
    for (int64_t c = threadIdx.x; c < ld; c += blockDim.x) lr[c] = from_f<T>(0.f);
    if (threadIdx.x == 0) rowloss[row] = 0.f;
    return;
  }
  float mx = -INFINITY;
  for (int64_t c = threadIdx.x; c < vocab; c += blockDim.x) mx = fmaxf(mx, to_f(lr[c]));
  mx = block_max(mx, red);
  float se = 0.f;
  for (int64_t c = threadIdx.x; c < vocab; c += blockDim.x) se += expf(to_f(lr[c]) - mx);
  se = block_sum(se, red);
  const float lse = mx + logf(se);
  const float inv_n = 1.0f / (float)nvalid[0];
  if (threadIdx.x == 0) rowloss[row] = lse - to_f(lr[label]);
  __syncthreads();
  for (int64_t c = threadIdx.x; c < ld; c += blockDim.x) {
    float g = 0.f;
    if (c < vocab) {
      g = expf(to_f(lr[c]) - lse);
      if (c == label) g -= 1.0f;
      g *= inv_n;
    }
    lr[c] = from_f<T>(g);
  }
}
// The same with 16-byte accesses and one pass for the maximum and the sum (online softmax per thread, combined across the
// block): the row is read once from HBM, a second time from L2 for the gradient, and written once.  Needs ld to be a
// multiple of the vector width (8 bf16 / 4 fp32) and a 16-byte aligned base.
__device__ __forceinline__ float ce_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
template <typename T> struct CeVec;
template <> struct CeVec<float> {
  static constexpr int V = 4;
  __device__ static void load(const float* p, float (&x)[4]) { const float4 v = *reinterpret_cast<const float4*>(p); x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w; }
  __device__ static void store(float* p, const float (&x)[4]) { *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]); }
};
template <> struct CeVec<bf16> {
  static constexpr int V = 8;
  __device__ static void load(const bf16* p, float (&x)[8]) {
    const uint4 v = *reinterpret_cast<const uint4*>(p);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) { const float2 f = __bfloat1622float2(h[i]); x[2 * i] = f.x; x[2 * i + 1] = f.y; }
  }
  __device__ static void store(bf16* p, const float (&x)[8]) {
    uint4 v;
    __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);
    *reinterpret_cast<uint4*>(p) = v;
  }
};
template <typename T>
__global__ void cross_entropy_vec_kernel(T* __restrict__ logits, const int32_t* __restrict__ labels,
                                         float* __restrict__ rowloss, const int* __restrict__ nvalid,
                                         int* __restrict__ bad, int64_t vocab, int64_t ld) {
  constexpr int V = CeVec<T>::V;
  constexpr float kL2E = 1.4426950408889634f, kLn2 = 0.6931471805599453f;
  __shared__ float red[33];
  const int64_t row = blockIdx.x, nch = ld / V;
  T* lr = logits + row * ld;
  int label = labels[row];
  if (label >= vocab) {
    if (threadIdx.x == 0) *bad = 1;
    label = -1;
  }
  float x[V];
  if (label < 0) {
#pragma unroll
    for (int i = 0; i < V; ++i) x[i] = 0.f;
    for (int64_t ch = threadIdx.x; ch < nch; ch += blockDim.x) CeVec<T>::store(lr + ch * V, x);
    if (threadIdx.x == 0) rowloss[row] = 0.f;
    return;
  }
  // running maximum m and sum s of 2^(x log2 e - m) over this thread's chunks (all in log2 units).  (Two chunks per
  // trip, to have two loads in flight, ran 17 % slower.)
  float m = -INFINITY, sacc = 0.f;
  for (int64_t ch = threadIdx.x; ch < nch; ch += blockDim.x) {
    CeVec<T>::load(lr + ch * V, x);
    float cm = -INFINITY;
#pragma unroll
    for (int i = 0; i < V; ++i) {
      x[i] = ch * V + i < vocab ? x[i] * kL2E : -INFINITY;          // padding columns take no part
      cm = fmaxf(cm, x[i]);
    }
    if (cm > m) { sacc *= ce_ex2(m - cm); m = cm; }                 // m = -inf: sacc is 0 and stays 0
    if (m > -INFINITY) {
#pragma unroll
      for (int i = 0; i < V; ++i) sacc += ce_ex2(x[i] - m);
    }
  }
  const float M = block_max(m, red);
  sacc = (m > -INFINITY) ? sacc * ce_ex2(m - M) : 0.f;
  const float S = block_sum(sacc, red);
  const float lse2 = M + log2f(S);                                  // log2 of the sum of exponentials
  const float inv_n = 1.0f / (float)nvalid[0];
  if (threadIdx.x == 0) rowloss[row] = lse2 * kLn2 - to_f(lr[label]);
  __syncthreads();                                                  // lr[label] is read before anyone overwrites it
  for (int64_t ch = threadIdx.x; ch < nch; ch += blockDim.x) {
    CeVec<T>::load(lr + ch * V, x);
#pragma unroll
    for (int i = 0; i < V; ++i) {
      const int64_t c = ch * V + i;
      float g = 0.f;
      if (c < vocab) {
        g = ce_ex2(fmaf(x[i], kL2E, -lse2));
        if (c == label) g -= 1.0f;
        g *= inv_n;
      }
      x[i] = g;
    }
    CeVec<T>::store(lr + ch * V, x);
  }
}
// loss = sum(rowloss)/nvalid  (single block, fixed order)
__global__ void loss_reduce_kernel(const float* __restrict__ rowloss, int64_t rows,
                                   const int* __restrict__ nvalid, float* __restrict__ loss) {
  __shared__ float red[33];
  float s = 0.f;
  for (int64_t i = threadIdx.x; i < rows; i += blockDim.x) s += rowloss[i];
  s = block_sum(s, red);
  if (threadIdx.x == 0) loss[0] = s / (float)nvalid[0];
}

// Copies the step's scalar words (loss, valid count, bad-input flag, and the tensor-core GEMM's
// timeout flag) into mapped pinned host memory with plain stores, so that the read-back never
// queues on a copy engine behind the multi-gigabyte optimizer-state transfers.
__global__ void publish_scalars_kernel(const float* __restrict__ src, const int* __restrict__ tc_error,
                                       volatile float* dst_mapped_host) {
  if (threadIdx.x < 3) dst_mapped_host[threadIdx.x] = src[threadIdx.x];
  if (threadIdx.x == 3) dst_mapped_host[3] = tc_error ? __int_as_float(*tc_error) : 0.f;
  if (threadIdx.x == 4) dst_mapped_host[4] = src[4];      // the gate word of the step's update
  __threadfence_system();
}

// ------------------------------------------------------------------ dropout
// The mask is a pure function of (seed, step, site, element): Philox4x32-10 (Salmon et al., SC'11) with the
// 64-bit seed as key and (element / 4 as two words, site, step) as counter gives four 32-bit words, one per
// element of an aligned group of four; an element is kept iff its word >= floor(p 2^32), kept values are
// scaled by 1 / (1 - p).  One thread draws one group of four.
__device__ __forceinline__ float4 drop_mult4(size_t i4, const DropArgs& a) {
  const uint4 w = philox4x32_10(make_uint4((uint32_t)i4, (uint32_t)(i4 >> 32), a.site, a.step), a.k0, a.k1);
  return make_float4(w.x >= a.thr ? a.scale : 0.f, w.y >= a.thr ? a.scale : 0.f, w.z >= a.thr ? a.scale : 0.f,
                     w.w >= a.thr ? a.scale : 0.f);
}
template <typename T>
__device__ __forceinline__ void store4_op(T* p, float4 v);
template <> __device__ __forceinline__ void store4_op<float>(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
template <> __device__ __forceinline__ void store4_op<bf16>(bf16* p, float4 v) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 pk;
  pk.x = *reinterpret_cast<uint32_t*>(&lo);
  pk.y = *reinterpret_cast<uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(p) = pk;
}
// out = res + mask * t   (t: the branch output in fp32; out, res: the residual stream)
__global__ void dropout_add_kernel(const float* __restrict__ t, const float* __restrict__ res, float* __restrict__ out,
                                   size_t n4, DropArgs a) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    const float4 m = drop_mult4(i, a);
    const float4 x = reinterpret_cast<const float4*>(t)[i], r = reinterpret_cast<const float4*>(res)[i];
    reinterpret_cast<float4*>(out)[i] = make_float4(r.x + m.x * x.x, r.y + m.y * x.y, r.z + m.z * x.z, r.w + m.w * x.w);
  }
}
// x *= mask in place on an fp32 tensor; the operand copy x_a (may be null) is rewritten from the masked value
template <typename T>
__global__ void dropout_inplace_kernel(float* __restrict__ x, T* __restrict__ x_a, size_t n4, DropArgs a) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    const float4 m = drop_mult4(i, a);
    float4 v = reinterpret_cast<float4*>(x)[i];
    v = make_float4(m.x * v.x, m.y * v.y, m.z * v.z, m.w * v.w);
    reinterpret_cast<float4*>(x)[i] = v;
    if (x_a != nullptr) store4_op<T>(x_a + 4 * i, v);
  }
}
// backward through a dropout site: masked copies of the stream gradient dx, in fp32 (mf, may be null) and as the
// GEMM operand (mop); dx itself is left alone (the residual path carries it on unmasked)
template <typename T>
__global__ void dropout_bwd_kernel(const float* __restrict__ dx, float* __restrict__ mf, T* __restrict__ mop, size_t n4, DropArgs a) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    const float4 m = drop_mult4(i, a);
    float4 v = reinterpret_cast<const float4*>(dx)[i];
    v = make_float4(m.x * v.x, m.y * v.y, m.z * v.z, m.w * v.w);
    if (mf != nullptr) reinterpret_cast<float4*>(mf)[i] = v;
    store4_op<T>(mop + 4 * i, v);
  }
}

// The step's gate word, read by every optimizer kernel before its first store: non-zero when the
// update must not happen.  src = the step's scalars ([0] loss, [2] bad-input flag); tc_error = the
// tensor-core kernels' time-out flag (may be null).  Codes: the time-out code (1 .. 9), 100 bad input,
// 101 non-finite loss; all positive, so that data-parallel ranks can share the word with a MAX reduction and
// every rank calls the update off when any rank's step failed.
__global__ void step_gate_kernel(const float* __restrict__ src, const int* __restrict__ tc_error, int* __restrict__ gate) {
  if (threadIdx.x != 0) return;
  int v = 0;
  const int tc = tc_error ? *tc_error : 0;
  const float loss = src[0];
  if (tc != 0) v = tc;
  else if (__float_as_int(src[2]) != 0) v = 100;
  else if (!(fabsf(loss) <= 3.402823466e38f)) v = 101;
  *gate = v;
}

// ------------------------------------------------------------------ fused group optimizer
// One streaming pass over the group's flat buffers: 128-bit loads/stores, 4 elements per
// thread per iteration.  KIND 0 AdamW, 1 AdaGrad, 2 SGD-momentum, 3 plain SGD (no state).  Scalars precomputed on the
// host in double: decay = 1 - lr*wd, omb1 = 1-beta1, omb2 = 1-beta2, c1 = 1/(1-beta1^tau),
// c2 = 1/(1-beta2^tau).  IEEE sqrt and division.
struct OptScalars {
  float lr, beta1, beta2, eps, decay, omb1, omb2, c1, c2, mu;
};
// Every operation is spelled with an explicit round-to-nearest intrinsic, so that no compiler
// choice (contraction into FMAs) can differ between the kernels that share this function: the
// paged and the resident form of the state must give the same bits.
template <int KIND>
__device__ __forceinline__ void opt_update(float& th, float g, float& s0, float& s1,
                                           const OptScalars& h) {
  if (KIND == 0) {
    th = __fmul_rn(th, h.decay);
    s0 = __fmaf_rn(h.beta1, s0, __fmul_rn(h.omb1, g));
    s1 = __fmaf_rn(h.beta2, s1, __fmul_rn(__fmul_rn(h.omb2, g), g));
    const float mhat = __fmul_rn(s0, h.c1);
    const float vhat = __fmul_rn(s1, h.c2);
    th = __fsub_rn(th, __fdiv_rn(__fmul_rn(h.lr, mhat), __fadd_rn(__fsqrt_rn(vhat), h.eps)));
  } else if (KIND == 1) {
    s0 = __fmaf_rn(g, g, s0);
    th = __fsub_rn(th, __fdiv_rn(__fmul_rn(h.lr, g), __fadd_rn(__fsqrt_rn(s0), h.eps)));
  } else if (KIND == 2) {
    s0 = __fmaf_rn(h.mu, s0, g);
    th = __fmaf_rn(-h.lr, s0, th);
  } else {
    th = __fmaf_rn(-h.lr, g, th);
  }
}
// four consecutive gradient elements (16-byte or 8-byte load, streaming)
template <typename GT> __device__ __forceinline__ float4 grad4(const GT* g, size_t i4);
template <> __device__ __forceinline__ float4 grad4<float>(const float* g, size_t i4) { return __ldcs(reinterpret_cast<const float4*>(g) + i4); }
template <> __device__ __forceinline__ float4 grad4<bf16>(const bf16* g, size_t i4) {
  const uint2 r = __ldcs(reinterpret_cast<const uint2*>(g) + i4);
  const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&r.x));
  const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&r.y));
  return make_float4(a.x, a.y, b.x, b.y);
}
template <int KIND, bool HAS_BF16, typename GT>
__global__ void __launch_bounds__(256)
fused_opt_kernel(bf16* __restrict__ param, float* __restrict__ master, const GT* __restrict__ grad,
                 float* __restrict__ s0, float* __restrict__ s1, size_t n, OptScalars h,
                 const int* __restrict__ gate) {
  if (gate != nullptr && *gate != 0) return;        // the step failed: every buffer keeps its bits
  const size_t n4 = n / 4;
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (; i < n4; i += stride) {
    float4 th = reinterpret_cast<const float4*>(master)[i];
    const float4 g = grad4<GT>(grad, i);
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    if (KIND != 3) a = reinterpret_cast<const float4*>(s0)[i];
    float4 b = make_float4(0.f, 0.f, 0.f, 0.f);
    if (KIND == 0) b = reinterpret_cast<const float4*>(s1)[i];
    opt_update<KIND>(th.x, g.x, a.x, b.x, h);
    opt_update<KIND>(th.y, g.y, a.y, b.y, h);
    opt_update<KIND>(th.z, g.z, a.z, b.z, h);
    opt_update<KIND>(th.w, g.w, a.w, b.w, h);
    reinterpret_cast<float4*>(master)[i] = th;
    if (KIND != 3) reinterpret_cast<float4*>(s0)[i] = a;
    if (KIND == 0) reinterpret_cast<float4*>(s1)[i] = b;
    if (HAS_BF16) {
      uint2 pk;
      __nv_bfloat162 lo = __floats2bfloat162_rn(th.x, th.y), hi = __floats2bfloat162_rn(th.z, th.w);
      pk.x = *reinterpret_cast<uint32_t*>(&lo);
      pk.y = *reinterpret_cast<uint32_t*>(&hi);
      reinterpret_cast<uint2*>(param)[i] = pk;
    }
  }
  // ragged tail (n not a multiple of 4)
  const size_t t = n4 * 4 + (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (t < n) {
    float th = master[t], a = (KIND != 3) ? s0[t] : 0.f, b = (KIND == 0) ? s1[t] : 0.f;
    opt_update<KIND>(th, to_f(grad[t]), a, b, h);
    master[t] = th;
    if (KIND != 3) s0[t] = a;
    if (KIND == 0) s1[t] = b;
    if (HAS_BF16) param[t] = __float2bfloat16_rn(th);
  }
}

// ------------------------------------------------------------------ fused optimizer, compact master
// With bf16 parameters the model copy p = round-to-nearest-even(master) already holds the upper
// half of every fp32 master value, up to the rounding carry.  The paged form of the master is
// therefore 16 + 1 bits per element instead of 32: lo = the low 16 bits of the fp32 pattern and
// carry = 1 where the rounding stepped the upper half up, so that
//     master bits = ((p - carry) << 16) | lo            (exact for every finite value and infinity)
// (the carry needs its own bit: a low half of 0x8000 rounds up or down depending on the parity of the
// upper half, and both cases leave the same p).  One thread owns 8 consecutive elements = one byte
// of carry bits, 16 bytes of p and of lo, 32 bytes of every fp32 plane.  Per element this pass reads
// 16.125 and writes 12.125 bytes with AdamW (20.25 in all with one state plane, 12.25 with none).
__device__ __forceinline__ void master_pack(uint32_t u, uint32_t& p, uint32_t& lo, uint32_t& carry) {
  lo = u & 0xFFFFu;
  if ((u & 0x7F800000u) == 0x7F800000u) {                  // infinity / NaN: no rounding
    p = u >> 16;
    if (lo && !(p & 0x7Fu)) p |= 0x40u;                    // keep a NaN a NaN in bf16
    carry = 0;
  } else {
    p = (u + 0x7FFFu + ((u >> 16) & 1u)) >> 16;            // round to nearest, ties to even
    carry = p - (u >> 16);
  }
}
__device__ __forceinline__ uint32_t master_unpack(uint32_t p, uint32_t lo, uint32_t carry) {
  return ((p - carry) << 16) | lo;
}
template <int KIND, typename GT>
__global__ void __launch_bounds__(256)
fused_opt_compact_kernel(uint16_t* __restrict__ param, uint16_t* __restrict__ lo16, uint8_t* __restrict__ carry8,
                         const GT* __restrict__ grad, float* __restrict__ s0, float* __restrict__ s1,
                         size_t n8, OptScalars h, const int* __restrict__ gate) {
  if (gate != nullptr && *gate != 0) return;        // the step failed: every buffer keeps its bits
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (; i < n8; i += stride) {
    const uint4 pw = reinterpret_cast<const uint4*>(param)[i];
    const uint4 lw = reinterpret_cast<const uint4*>(lo16)[i];
    const uint32_t cb = carry8[i];
    const uint32_t pws[4] = {pw.x, pw.y, pw.z, pw.w}, lws[4] = {lw.x, lw.y, lw.z, lw.w};
    float g[8], a[8], b[8], th[8];
    {
      const float4 g0 = grad4<GT>(grad, 2 * i), g1 = grad4<GT>(grad, 2 * i + 1);
      g[0] = g0.x; g[1] = g0.y; g[2] = g0.z; g[3] = g0.w; g[4] = g1.x; g[5] = g1.y; g[6] = g1.z; g[7] = g1.w;
    }
    if (KIND != 3) load8(s0 + 8 * i, a);
    if (KIND == 0) load8(s1 + 8 * i, b);
    uint32_t pout[4], lout[4], cout = 0;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const uint32_t sh = (e & 1) * 16;
      th[e] = __uint_as_float(master_unpack((pws[e >> 1] >> sh) & 0xFFFFu, (lws[e >> 1] >> sh) & 0xFFFFu, (cb >> e) & 1u));
      float aa = KIND != 3 ? a[e] : 0.f, bb = KIND == 0 ? b[e] : 0.f;
      opt_update<KIND>(th[e], g[e], aa, bb, h);
      a[e] = aa; b[e] = bb;
      uint32_t pe, le, ce;
      master_pack(__float_as_uint(th[e]), pe, le, ce);
      if (e & 1) { pout[e >> 1] |= pe << 16; lout[e >> 1] |= le << 16; }
      else { pout[e >> 1] = pe; lout[e >> 1] = le; }
      cout |= ce << e;
    }
    reinterpret_cast<uint4*>(param)[i] = make_uint4(pout[0], pout[1], pout[2], pout[3]);
    reinterpret_cast<uint4*>(lo16)[i] = make_uint4(lout[0], lout[1], lout[2], lout[3]);
    carry8[i] = (uint8_t)cout;
    if (KIND != 3) store8(s0 + 8 * i, a);
    if (KIND == 0) store8(s1 + 8 * i, b);
  }
}
// fp32 master values -> (lo, carry); the bf16 copy p is written by whoever produced the values
__global__ void master_pack_kernel(const float* __restrict__ master, uint16_t* __restrict__ lo16,
                                   uint8_t* __restrict__ carry8, size_t n8) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (; i < n8; i += stride) {
    float m[8];
    load8(master + 8 * i, m);
    uint32_t lout[4], cout = 0;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      uint32_t pe, le, ce;
      master_pack(__float_as_uint(m[e]), pe, le, ce);
      if (e & 1) lout[e >> 1] |= le << 16; else lout[e >> 1] = le;
      cout |= ce << e;
    }
    reinterpret_cast<uint4*>(lo16)[i] = make_uint4(lout[0], lout[1], lout[2], lout[3]);
    carry8[i] = (uint8_t)cout;
  }
}

}  // namespace hift
