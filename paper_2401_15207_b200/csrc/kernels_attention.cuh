// Multi-head attention, forward and backward, on CUDA cores with fp32 arithmetic:
//   o = softmax(q k^T / sqrt(d_h) + causal mask) v   per (batch, head),
// online softmax over key tiles (nothing of size S x S is stored), log-sum-exp saved for the
// backward pass, which recomputes the probabilities.  The backward pass is split in two
// kernels so that every output element has exactly one writer (no atomics, deterministic):
// one owns query rows (dq), one owns key rows (dk, dv).
//
// Layout: qkv[T, 3d] with column blocks q | k | v and head h at columns h*d_h .. (h+1)*d_h;
// o, do: [T, d]; lse, dsum: [B, H, S] fp32.
//
// Thread mapping: 4 threads ("parts") share one row; part p owns elements {4i + p} of the
// head vector, which keeps shared-memory reads conflict-free; dot products finish with two
// quad shuffles.
#pragma once
#include "common.cuh"
#include "dropout_rng.cuh"

namespace hift {

constexpr int kAttRows = 64;    // rows (queries or keys) per block
constexpr int kAttTile = 32;    // rows of the other operand staged in shared memory per step

__device__ __forceinline__ float quad_sum(float v) {
  v += __shfl_xor_sync(0xffffffffu, v, 1);
  v += __shfl_xor_sync(0xffffffffu, v, 2);
  return v;
}

template <typename T, int DH>
__device__ __forceinline__ void stage_rows(float (*dst)[DH], const T* __restrict__ base,
                                           int64_t row_stride, int row0, int nrows_valid) {
  // kAttTile rows of DH elements, coalesced along the row; rows past nrows_valid are zeroed
  for (int idx = threadIdx.x; idx < kAttTile * DH; idx += blockDim.x) {
    const int r = idx / DH, c = idx % DH;
    dst[r][c] = (r < nrows_valid) ? to_f(base[(int64_t)(row0 + r) * row_stride + c]) : 0.f;
  }
}

template <typename T, int DH>
__global__ void __launch_bounds__(256)
attention_fwd_kernel(const T* __restrict__ qkv, T* __restrict__ o, float* __restrict__ lse,
                     int S, int H, int causal, float scale, const int* __restrict__ lens, DropArgs da) {
  constexpr int E = DH / 4;
  __shared__ float Ks[kAttTile][DH];
  __shared__ float Vs[kAttTile][DH];
  const int b = blockIdx.z, h = blockIdx.y, q0 = blockIdx.x * kAttRows;
  const int klen = key_len_of(lens, b, S);
  const int d = H * DH;
  const int p = threadIdx.x & 3, r = threadIdx.x >> 2;
  const int qrow = q0 + r;
  const bool active = qrow < S;
  const T* qbase = qkv + (int64_t)b * S * 3 * d + (int64_t)h * DH;
  const T* kbase = qbase + d;
  const T* vbase = qbase + 2 * d;
  float q[E], acc[E];
#pragma unroll
  for (int i = 0; i < E; ++i) {
    q[i] = active ? to_f(qbase[(int64_t)qrow * 3 * d + 4 * i + p]) * scale : 0.f;
    acc[i] = 0.f;
  }
  float m = -INFINITY, l = 0.f;
  const int q_last = min(q0 + kAttRows, S) - 1;
  const int k_end = min(causal ? q_last + 1 : S, klen);
  // dropout on the probabilities (da.thr != 0): the sum l runs over all of them, the product with V over the kept
  // ones; 1 / (1 - p) goes into the final scaling.  Tiles start at multiples of 32, so a generator block (four keys)
  // never straddles two tiles.
  const bool drop = da.thr != 0u;
  uint4 dw = make_uint4(0u, 0u, 0u, 0u);
  for (int k0 = 0; k0 < k_end; k0 += kAttTile) {
    const int nk = min(kAttTile, S - k0);
    __syncthreads();
    stage_rows<T, DH>(Ks, kbase, 3 * d, k0, nk);
    stage_rows<T, DH>(Vs, vbase, 3 * d, k0, nk);
    __syncthreads();
    for (int j = 0; j < nk; ++j) {
      float s = 0.f;
#pragma unroll
      for (int i = 0; i < E; ++i) s = fmaf(q[i], Ks[j][4 * i + p], s);
      s = quad_sum(s);
      const int key = k0 + j;
      if (drop && (key & 3) == 0 && active) dw = attn_drop_words(da, b * H + h, S, qrow, key);
      if (active && key < klen && (!causal || key <= qrow)) {
        const float mn = fmaxf(m, s);
        const float corr = expf(m - mn);
        const float pj = expf(s - mn);
        l = l * corr + pj;
        const float pv = (drop && word_of(dw, key & 3) < da.thr) ? 0.f : pj;
#pragma unroll
        for (int i = 0; i < E; ++i) acc[i] = fmaf(pv, Vs[j][4 * i + p], acc[i] * corr);
        m = mn;
      }
    }
  }
  if (active) {
    const float inv = (drop ? da.scale : 1.0f) / l;
    T* orow = o + ((int64_t)b * S + qrow) * d + (int64_t)h * DH;
#pragma unroll
    for (int i = 0; i < E; ++i) orow[4 * i + p] = from_f<T>(acc[i] * inv);
    if (p == 0) lse[((int64_t)b * H + h) * S + qrow] = m + logf(l);
  }
}

// dq (query-row owner).  Also writes dsum[b,h,row] = sum_e do*o for the dk/dv kernel.
template <typename T, int DH>
__global__ void __launch_bounds__(256)
attention_bwd_dq_kernel(const T* __restrict__ qkv, const T* __restrict__ o,
                        const float* __restrict__ lse, const T* __restrict__ dout,
                        T* __restrict__ dqkv, float* __restrict__ dsum, int S, int H, int causal,
                        float scale, const int* __restrict__ lens, DropArgs da) {
  constexpr int E = DH / 4;
  __shared__ float Ks[kAttTile][DH];
  __shared__ float Vs[kAttTile][DH];
  const int b = blockIdx.z, h = blockIdx.y, q0 = blockIdx.x * kAttRows;
  const int klen = key_len_of(lens, b, S);
  const int d = H * DH;
  const int p = threadIdx.x & 3, r = threadIdx.x >> 2;
  const int qrow = q0 + r;
  const bool active = qrow < S;
  const T* qbase = qkv + (int64_t)b * S * 3 * d + (int64_t)h * DH;
  const T* kbase = qbase + d;
  const T* vbase = qbase + 2 * d;
  float q[E], go[E], dq[E];
  float D = 0.f, L = 0.f;
#pragma unroll
  for (int i = 0; i < E; ++i) {
    q[i] = 0.f; go[i] = 0.f; dq[i] = 0.f;
  }
  if (active) {
    const int64_t orow = ((int64_t)b * S + qrow) * d + (int64_t)h * DH;
#pragma unroll
    for (int i = 0; i < E; ++i) {
      q[i] = to_f(qbase[(int64_t)qrow * 3 * d + 4 * i + p]) * scale;
      go[i] = to_f(dout[orow + 4 * i + p]);
      D = fmaf(go[i], to_f(o[orow + 4 * i + p]), D);
    }
    L = lse[((int64_t)b * H + h) * S + qrow];
  }
  D = quad_sum(D);
  if (active && p == 0) dsum[((int64_t)b * H + h) * S + qrow] = D;
  const bool drop = da.thr != 0u;
  uint4 dw = make_uint4(0u, 0u, 0u, 0u);
  const int q_last = min(q0 + kAttRows, S) - 1;
  const int k_end = min(causal ? q_last + 1 : S, klen);
  for (int k0 = 0; k0 < k_end; k0 += kAttTile) {
    const int nk = min(kAttTile, S - k0);
    __syncthreads();
    stage_rows<T, DH>(Ks, kbase, 3 * d, k0, nk);
    stage_rows<T, DH>(Vs, vbase, 3 * d, k0, nk);
    __syncthreads();
    for (int j = 0; j < nk; ++j) {
      float s = 0.f, dp = 0.f;
#pragma unroll
      for (int i = 0; i < E; ++i) {
        s = fmaf(q[i], Ks[j][4 * i + p], s);
        dp = fmaf(go[i], Vs[j][4 * i + p], dp);
      }
      s = quad_sum(s);
      dp = quad_sum(dp);
      const int key = k0 + j;
      if (drop && (key & 3) == 0 && active) dw = attn_drop_words(da, b * H + h, S, qrow, key);
      if (active && key < klen && (!causal || key <= qrow)) {
        // with dropout the gradient reaches the probability through its mask: dp -> dp o mask / (1 - p)
        if (drop) dp = word_of(dw, key & 3) < da.thr ? 0.f : dp * da.scale;
        const float ds = expf(s - L) * (dp - D);
#pragma unroll
        for (int i = 0; i < E; ++i) dq[i] = fmaf(ds, Ks[j][4 * i + p], dq[i]);
      }
    }
  }
  if (active) {
    T* out = dqkv + ((int64_t)b * S + qrow) * 3 * d + (int64_t)h * DH;
#pragma unroll
    for (int i = 0; i < E; ++i) out[4 * i + p] = from_f<T>(dq[i] * scale);
  }
}

// dk, dv (key-row owner).  Needs dsum from the dq kernel.
template <typename T, int DH>
__global__ void __launch_bounds__(256)
attention_bwd_dkv_kernel(const T* __restrict__ qkv, const float* __restrict__ lse,
                         const T* __restrict__ dout, const float* __restrict__ dsum,
                         T* __restrict__ dqkv, int S, int H, int causal, float scale,
                         const int* __restrict__ lens, DropArgs da) {
  constexpr int E = DH / 4;
  __shared__ float Qs[kAttTile][DH];
  __shared__ float Gs[kAttTile][DH];
  __shared__ float Ls[kAttTile], Ds[kAttTile];
  const int b = blockIdx.z, h = blockIdx.y, kr0 = blockIdx.x * kAttRows;
  const int klen = key_len_of(lens, b, S);
  const int d = H * DH;
  const int p = threadIdx.x & 3, r = threadIdx.x >> 2;
  const int krow = kr0 + r;
  const bool active = krow < S;
  const T* qbase = qkv + (int64_t)b * S * 3 * d + (int64_t)h * DH;
  const T* kbase = qbase + d;
  const T* vbase = qbase + 2 * d;
  const T* gbase = dout + (int64_t)b * S * d + (int64_t)h * DH;
  float k[E], v[E], dk[E], dv[E];
#pragma unroll
  for (int i = 0; i < E; ++i) {
    k[i] = active ? to_f(kbase[(int64_t)krow * 3 * d + 4 * i + p]) : 0.f;
    v[i] = active ? to_f(vbase[(int64_t)krow * 3 * d + 4 * i + p]) : 0.f;
    dk[i] = 0.f; dv[i] = 0.f;
  }
  const int q_begin = causal ? (kr0 / kAttTile) * kAttTile : 0;
  for (int q0 = q_begin; q0 < S; q0 += kAttTile) {
    const int nq = min(kAttTile, S - q0);
    __syncthreads();
    stage_rows<T, DH>(Qs, qbase, 3 * d, q0, nq);
    stage_rows<T, DH>(Gs, gbase, d, q0, nq);
    if (threadIdx.x < kAttTile) {
      const bool ok = threadIdx.x < nq;
      Ls[threadIdx.x] = ok ? lse[((int64_t)b * H + h) * S + q0 + threadIdx.x] : 0.f;
      Ds[threadIdx.x] = ok ? dsum[((int64_t)b * H + h) * S + q0 + threadIdx.x] : 0.f;
    }
    __syncthreads();
    for (int j = 0; j < nq; ++j) {
      float s = 0.f, dp = 0.f;
#pragma unroll
      for (int i = 0; i < E; ++i) {
        s = fmaf(k[i], Qs[j][4 * i + p], s);
        dp = fmaf(v[i], Gs[j][4 * i + p], dp);
      }
      s = quad_sum(s);
      dp = quad_sum(dp);
      const int qrow = q0 + j;
      if (active && krow < klen && (!causal || krow <= qrow)) {
        const float pr = expf(s * scale - Ls[j]);
        // with dropout: dv takes the dropped probability, and dp comes back through the same mask
        float keep = 1.0f;
        if (da.thr != 0u) keep = word_of(attn_drop_words(da, b * H + h, S, qrow, krow & ~3), krow & 3) < da.thr ? 0.f : da.scale;
        const float ds = pr * (dp * keep - Ds[j]);
        const float pd = pr * keep;
#pragma unroll
        for (int i = 0; i < E; ++i) {
          dv[i] = fmaf(pd, Gs[j][4 * i + p], dv[i]);
          dk[i] = fmaf(ds, Qs[j][4 * i + p], dk[i]);
        }
      }
    }
  }
  if (active) {
    T* outk = dqkv + ((int64_t)b * S + krow) * 3 * d + d + (int64_t)h * DH;
    T* outv = outk + d;
#pragma unroll
    for (int i = 0; i < E; ++i) {
      outk[4 * i + p] = from_f<T>(dk[i] * scale);
      outv[4 * i + p] = from_f<T>(dv[i]);
    }
  }
}

}  // namespace hift
