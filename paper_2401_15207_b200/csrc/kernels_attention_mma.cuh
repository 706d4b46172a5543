// bf16 attention on the warp-level tensor-core path (mma.sync m16n8k16, fp32 accumulate), for
// head sizes 64 and 128.  Same mathematics and layout as kernels_attention.cuh:
//   forward:  o = softmax(q k^T / sqrt(d_h) + causal mask) v, online softmax over 64-key tiles, LSE saved
//   backward: probabilities recomputed from LSE; one kernel owns query rows (dq), one owns key
//             rows (dk, dv), so every output has one writer and the result is deterministic.
// qkv[T,3d] with column blocks q | k | v, head h at columns h*d_h; o, do: [T,d]; lse, dsum: [B,H,S].
//
// Shared-memory tiles are [rows][DH] bf16 with the 16-byte chunk index XOR-ed with (row & 7), so
// that ldmatrix (8 rows x 16 bytes) is bank-conflict free.
#pragma once
#include "common.cuh"

namespace hift {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t saddr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(saddr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], uint32_t saddr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(saddr));
}
__device__ __forceinline__ void mma16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// byte offset of element (r, col) in a swizzled [rows][DH] bf16 tile; col % 8 == 0
template <int DH>
__device__ __forceinline__ uint32_t swz(int r, int col) {
  return (uint32_t)((r * (DH / 8) + ((col >> 3) ^ (r & 7))) * 16);
}
// Stage ROWS rows of DH bf16 (row pitch `pitch` elements) starting at global row row0; rows at
// or beyond `rows_total` are zero-filled.  All 128 threads of the block take part.
template <int ROWS, int DH>
__device__ __forceinline__ void stage_tile(uint8_t* tile, const bf16* __restrict__ g, int64_t pitch,
                                           int row0, int rows_total) {
  constexpr int CH = DH / 8;
  for (int idx = threadIdx.x; idx < ROWS * CH; idx += blockDim.x) {
    const int r = idx / CH, c = idx % CH;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (row0 + r < rows_total) v = *reinterpret_cast<const uint4*>(g + (int64_t)(row0 + r) * pitch + c * 8);
    *reinterpret_cast<uint4*>(tile + swz<DH>(r, c * 8)) = v;
  }
}
// The same through cp.async (16 bytes per request, zero-filled past the end), so that the next
// tile streams in while the tensor cores work on the current one.
__device__ __forceinline__ void cp_async16(uint32_t saddr, const void* g, bool valid) {
  const int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(saddr), "l"(g), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
template <int ROWS, int DH>
__device__ __forceinline__ void stage_tile_async(uint32_t tile, const bf16* __restrict__ g, int64_t pitch,
                                                 int row0, int rows_total) {
  constexpr int CH = DH / 8;
  for (int idx = threadIdx.x; idx < ROWS * CH; idx += blockDim.x) {
    const int r = idx / CH, c = idx % CH;
    const bool ok = row0 + r < rows_total;
    const bf16* src = g + (int64_t)(ok ? row0 + r : 0) * pitch + c * 8;
    cp_async16(tile + swz<DH>(r, c * 8), src, ok);
  }
}

// A fragment (16 rows x 16 k) of a row-major tile at (r0, c0)
template <int DH>
__device__ __forceinline__ void load_a(uint32_t (&a)[4], uint32_t tile, int r0, int c0, int lane) {
  ldsm_x4(a, tile + swz<DH>(r0 + (lane & 7) + ((lane >> 3) & 1) * 8, c0 + (lane >> 4) * 8));
}
// B fragments for two adjacent n8 tiles where B(k, n) = X[n][k] (tile rows are n, k contiguous):
// r[0], r[1] = b0, b1 of tile n0; r[2], r[3] = b0, b1 of tile n0 + 8
template <int DH>
__device__ __forceinline__ void load_b_nk(uint32_t (&r)[4], uint32_t tile, int n0, int k0, int lane) {
  ldsm_x4(r, tile + swz<DH>(n0 + (lane & 7) + (lane >> 4) * 8, k0 + ((lane >> 3) & 1) * 8));
}
// B fragments for two adjacent n8 tiles where B(k, n) = X[k][n] (tile rows are k, n contiguous)
template <int DH>
__device__ __forceinline__ void load_b_kn(uint32_t (&r)[4], uint32_t tile, int k0, int n0, int lane) {
  ldsm_x4_t(r, tile + swz<DH>(k0 + (lane & 7) + ((lane >> 3) & 1) * 8, n0 + (lane >> 4) * 8));
}

// ------------------------------------------------------------------ forward
// dynamic shared memory: K[2], V[2] tiles of 64 x DH bf16
template <int DH>
constexpr int attn_fwd_smem_bytes() { return 4 * 64 * DH * 2; }

template <int DH>
__global__ void __launch_bounds__(128, 3)
attn_fwd_mma_kernel(const bf16* __restrict__ qkv, bf16* __restrict__ o, float* __restrict__ lse,
                    int S, int H, int causal, float scale, const int* __restrict__ lens) {
  constexpr int BQ = 64, BKV = 64, KS = DH / 16;
  constexpr int TB = BKV * DH * 2;                    // bytes of one K or V tile
  extern __shared__ __align__(128) uint8_t smem_att[];   // K[2] | V[2]; Q is staged through V[1] first
  uint8_t* sQ = smem_att + 3 * TB;
  const int b = blockIdx.z, h = blockIdx.y, q0 = blockIdx.x * BQ;
  const int d = H * DH;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const bf16* qb = qkv + (int64_t)b * S * 3 * d + (int64_t)h * DH;
  const bf16* kb = qb + d;
  const bf16* vb = qb + 2 * d;
  const uint32_t tQ = (uint32_t)__cvta_generic_to_shared(sQ);
  const uint32_t tKb = (uint32_t)__cvta_generic_to_shared(smem_att);
  const uint32_t tVb = tKb + 2 * TB;

  stage_tile<BQ, DH>(sQ, qb, 3 * d, q0, S);
  __syncthreads();
  uint32_t qa[KS][4];
#pragma unroll
  for (int ks = 0; ks < KS; ++ks) load_a<DH>(qa[ks], tQ, warp * 16, ks * 16, lane);
  __syncthreads();                                      // Q fragments are in registers: V[1] may be overwritten

  float oacc[DH / 8][4];
#pragma unroll
  for (int i = 0; i < DH / 8; ++i) { oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f; }
  float mrow[2] = {-INFINITY, -INFINITY}, lrow[2] = {0.f, 0.f};
  const float sl2 = scale * kLog2e;
  const int row_lo = q0 + warp * 16 + g;              // this thread's rows: row_lo, row_lo + 8
  const int klen = key_len_of(lens, b, S);             // keys at or after klen are padding
  const int k_end = min(causal ? min(S, q0 + BQ) : S, klen);

  stage_tile_async<BKV, DH>(tKb, kb, 3 * d, 0, S);
  stage_tile_async<BKV, DH>(tVb, vb, 3 * d, 0, S);
  cp_async_commit();
  int buf = 0;
  for (int k0 = 0; k0 < k_end; k0 += BKV, buf ^= 1) {
    if (k0 + BKV < k_end) {                            // the next tile streams in behind this one
      stage_tile_async<BKV, DH>(tKb + (buf ^ 1) * TB, kb, 3 * d, k0 + BKV, S);
      stage_tile_async<BKV, DH>(tVb + (buf ^ 1) * TB, vb, 3 * d, k0 + BKV, S);
      cp_async_commit();
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    const uint32_t tK = tKb + buf * TB, tV = tVb + buf * TB;
    float sacc[BKV / 8][4];
#pragma unroll
    for (int i = 0; i < BKV / 8; ++i) { sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f; }
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
      for (int np = 0; np < BKV / 16; ++np) {
        uint32_t bfr[4];
        load_b_nk<DH>(bfr, tK, np * 16, ks * 16, lane);
        mma16816(sacc[2 * np], qa[ks], bfr[0], bfr[1]);
        mma16816(sacc[2 * np + 1], qa[ks], bfr[2], bfr[3]);
      }
    }
    // scale, mask, running max
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int i = 0; i < BKV / 8; ++i) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int col = k0 + i * 8 + 2 * t + (e & 1);
        const int row = row_lo + (e >> 1) * 8;
        float v = sacc[i][e] * sl2;
        if (col >= klen || (causal && col > row)) v = -INFINITY;
        sacc[i][e] = v;
        mx[e >> 1] = fmaxf(mx[e >> 1], v);
      }
    }
    float corr[2], muse[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
      const float mnew = fmaxf(mrow[r], mx[r]);
      muse[r] = (mnew == -INFINITY) ? 0.f : mnew;       // a row with nothing visible yet
      corr[r] = exp2f(mrow[r] - muse[r]);                // exp2(-inf) = 0 on the first tile
      mrow[r] = mnew;
      lrow[r] *= corr[r];
    }
#pragma unroll
    for (int i = 0; i < BKV / 8; ++i) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float p = exp2f(sacc[i][e] - muse[e >> 1]);
        sacc[i][e] = p;
        lrow[e >> 1] += p;
      }
    }
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) {
      oacc[i][0] *= corr[0]; oacc[i][1] *= corr[0]; oacc[i][2] *= corr[1]; oacc[i][3] *= corr[1];
    }
    // O += P V
#pragma unroll
    for (int j = 0; j < BKV / 16; ++j) {
      uint32_t pa[4];
      pa[0] = pack_bf16(sacc[2 * j][0], sacc[2 * j][1]);
      pa[1] = pack_bf16(sacc[2 * j][2], sacc[2 * j][3]);
      pa[2] = pack_bf16(sacc[2 * j + 1][0], sacc[2 * j + 1][1]);
      pa[3] = pack_bf16(sacc[2 * j + 1][2], sacc[2 * j + 1][3]);
#pragma unroll
      for (int np = 0; np < DH / 16; ++np) {
        uint32_t bfr[4];
        load_b_kn<DH>(bfr, tV, j * 16, np * 16, lane);
        mma16816(oacc[2 * np], pa, bfr[0], bfr[1]);
        mma16816(oacc[2 * np + 1], pa, bfr[2], bfr[3]);
      }
    }
    __syncthreads();                                   // this buffer is refilled two iterations from now
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    lrow[r] += __shfl_xor_sync(0xffffffffu, lrow[r], 1);
    lrow[r] += __shfl_xor_sync(0xffffffffu, lrow[r], 2);
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int row = row_lo + r * 8;
    if (row >= S) continue;
    const float inv = 1.0f / lrow[r];
    bf16* orow = o + ((int64_t)b * S + row) * d + (int64_t)h * DH;
#pragma unroll
    for (int i = 0; i < DH / 8; ++i)
      *reinterpret_cast<uint32_t*>(orow + i * 8 + 2 * t) = pack_bf16(oacc[i][2 * r] * inv, oacc[i][2 * r + 1] * inv);
    if (t == 0) lse[((int64_t)b * H + h) * S + row] = (mrow[r] + log2f(lrow[r])) * kLn2;
  }
}

// ------------------------------------------------------------------ backward: dsum = rowsum(do * o)
// DH/8 consecutive lanes per (token, head) row, 16 bytes of o and of do per lane; the row sum is
// a shuffle reduction inside that lane group (fixed order).  dsum layout [B, H, S].
template <int DH>
__global__ void attn_dsum_kernel(const bf16* __restrict__ o, const bf16* __restrict__ dout,
                                 float* __restrict__ dsum, int B, int S, int H) {
  constexpr int LPR = DH / 8;                              // lanes per row: 8 or 16
  pdl_launch_next();
  pdl_wait_prior();
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t row = i / LPR;                             // (token, head)
  const int part = (int)(i % LPR);
  const int64_t nrows = (int64_t)B * S * H;
  float acc = 0.f;
  if (row < nrows) {
    float a[8], c[8];
    load8(o + row * DH + part * 8, a);
    load8(dout + row * DH + part * 8, c);
#pragma unroll
    for (int e = 0; e < 8; ++e) acc += a[e] * c[e];
  }
#pragma unroll
  for (int off = LPR / 2; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
  if (row < nrows && part == 0) {
    const int h = (int)(row % H);
    const int64_t tok = row / H;
    const int b = (int)(tok / S), sq = (int)(tok % S);
    dsum[((int64_t)b * H + h) * S + sq] = acc;
  }
}
inline void launch_attn_dsum(cudaStream_t st, const bf16* o, const bf16* dout, float* dsum, int B, int S, int H, int DH) {
  const int64_t threads = (int64_t)B * S * H * (DH / 8);
  const unsigned grid = (unsigned)((threads + 255) / 256);
  if (DH == 64) launch_pdl(attn_dsum_kernel<64>, dim3(grid), dim3(256), 0, st, o, dout, dsum, B, S, H);
  else launch_pdl(attn_dsum_kernel<128>, dim3(grid), dim3(256), 0, st, o, dout, dsum, B, S, H);
}

// ------------------------------------------------------------------ backward: dq (owner of query rows)
template <int DH>
__global__ void __launch_bounds__(128)
attn_bwd_dq_mma_kernel(const bf16* __restrict__ qkv, const float* __restrict__ lse,
                       const bf16* __restrict__ dout, const float* __restrict__ dsum,
                       bf16* __restrict__ dqkv, int S, int H, int causal, float scale,
                       const int* __restrict__ lens) {
  constexpr int BQ = 64, BKV = 32, KS = DH / 16;
  constexpr int TB = BKV * DH * 2;
  __shared__ __align__(128) uint8_t sX[BQ * DH * 2];       // q tile, then do tile (fragments are kept in registers)
  __shared__ __align__(128) uint8_t sK[2 * TB];            // double-buffered
  __shared__ __align__(128) uint8_t sV[2 * TB];
  const int b = blockIdx.z, h = blockIdx.y, q0 = blockIdx.x * BQ;
  const int d = H * DH;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const bf16* qb = qkv + (int64_t)b * S * 3 * d + (int64_t)h * DH;
  const bf16* kb = qb + d;
  const bf16* vb = qb + 2 * d;
  const bf16* gb = dout + (int64_t)b * S * d + (int64_t)h * DH;
  const uint32_t tX = (uint32_t)__cvta_generic_to_shared(sX);
  const uint32_t tKb = (uint32_t)__cvta_generic_to_shared(sK);
  const uint32_t tVb = (uint32_t)__cvta_generic_to_shared(sV);

  const int klen = key_len_of(lens, b, S);             // keys at or after klen are padding
  const int k_end = min(causal ? min(S, q0 + BQ) : S, klen);
  stage_tile_async<BKV, DH>(tKb, kb, 3 * d, 0, S);         // first K/V tile streams in behind the Q / dO staging
  stage_tile_async<BKV, DH>(tVb, vb, 3 * d, 0, S);
  cp_async_commit();

  uint32_t qa[KS][4], ga[KS][4];
  stage_tile<BQ, DH>(sX, qb, 3 * d, q0, S);
  __syncthreads();
#pragma unroll
  for (int ks = 0; ks < KS; ++ks) load_a<DH>(qa[ks], tX, warp * 16, ks * 16, lane);
  __syncthreads();
  stage_tile<BQ, DH>(sX, gb, d, q0, S);
  __syncthreads();
#pragma unroll
  for (int ks = 0; ks < KS; ++ks) load_a<DH>(ga[ks], tX, warp * 16, ks * 16, lane);

  const int row_lo = q0 + warp * 16 + g;
  float L2[2], Dr[2];
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int row = row_lo + r * 8;
    const bool ok = row < S;
    L2[r] = ok ? lse[((int64_t)b * H + h) * S + row] * kLog2e : 0.f;
    Dr[r] = ok ? dsum[((int64_t)b * H + h) * S + row] : 0.f;
  }
  float dq[DH / 8][4];
#pragma unroll
  for (int i = 0; i < DH / 8; ++i) { dq[i][0] = dq[i][1] = dq[i][2] = dq[i][3] = 0.f; }
  const float sl2 = scale * kLog2e;

  int buf = 0;
  for (int k0 = 0; k0 < k_end; k0 += BKV, buf ^= 1) {
    if (k0 + BKV < k_end) {
      stage_tile_async<BKV, DH>(tKb + (buf ^ 1) * TB, kb, 3 * d, k0 + BKV, S);
      stage_tile_async<BKV, DH>(tVb + (buf ^ 1) * TB, vb, 3 * d, k0 + BKV, S);
      cp_async_commit();
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    const uint32_t tK = tKb + buf * TB, tV = tVb + buf * TB;
    float sacc[BKV / 8][4], pacc[BKV / 8][4];
#pragma unroll
    for (int i = 0; i < BKV / 8; ++i) {
      sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f;
      pacc[i][0] = pacc[i][1] = pacc[i][2] = pacc[i][3] = 0.f;
    }
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
      for (int np = 0; np < BKV / 16; ++np) {
        uint32_t bfr[4];
        load_b_nk<DH>(bfr, tK, np * 16, ks * 16, lane);
        mma16816(sacc[2 * np], qa[ks], bfr[0], bfr[1]);
        mma16816(sacc[2 * np + 1], qa[ks], bfr[2], bfr[3]);
        load_b_nk<DH>(bfr, tV, np * 16, ks * 16, lane);
        mma16816(pacc[2 * np], ga[ks], bfr[0], bfr[1]);
        mma16816(pacc[2 * np + 1], ga[ks], bfr[2], bfr[3]);
      }
    }
    // dS = P * (dP - D), masked entries 0
#pragma unroll
    for (int i = 0; i < BKV / 8; ++i) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int col = k0 + i * 8 + 2 * t + (e & 1);
        const int row = row_lo + (e >> 1) * 8;
        float ds = 0.f;
        if (col < klen && row < S && !(causal && col > row)) {
          const float p = exp2f(sacc[i][e] * sl2 - L2[e >> 1]);
          ds = p * (pacc[i][e] - Dr[e >> 1]);
        }
        sacc[i][e] = ds;
      }
    }
    // dQ += dS K
#pragma unroll
    for (int j = 0; j < BKV / 16; ++j) {
      uint32_t pa[4];
      pa[0] = pack_bf16(sacc[2 * j][0], sacc[2 * j][1]);
      pa[1] = pack_bf16(sacc[2 * j][2], sacc[2 * j][3]);
      pa[2] = pack_bf16(sacc[2 * j + 1][0], sacc[2 * j + 1][1]);
      pa[3] = pack_bf16(sacc[2 * j + 1][2], sacc[2 * j + 1][3]);
#pragma unroll
      for (int np = 0; np < DH / 16; ++np) {
        uint32_t bfr[4];
        load_b_kn<DH>(bfr, tK, j * 16, np * 16, lane);
        mma16816(dq[2 * np], pa, bfr[0], bfr[1]);
        mma16816(dq[2 * np + 1], pa, bfr[2], bfr[3]);
      }
    }
    __syncthreads();                                   // this buffer is refilled two iterations from now
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int row = row_lo + r * 8;
    if (row >= S) continue;
    bf16* out = dqkv + ((int64_t)b * S + row) * 3 * d + (int64_t)h * DH;
#pragma unroll
    for (int i = 0; i < DH / 8; ++i)
      *reinterpret_cast<uint32_t*>(out + i * 8 + 2 * t) = pack_bf16(dq[i][2 * r] * scale, dq[i][2 * r + 1] * scale);
  }
}

// ------------------------------------------------------------------ backward: dk, dv (owner of key rows)
// dynamic shared memory: K tile [64][DH], V tile [64][DH], double-buffered Q and dO tiles [2][32][DH], L2[2][32], D[2][32]
template <int DH>
constexpr int attn_dkv_smem_bytes() { return (64 + 64 + 2 * 32 + 2 * 32) * DH * 2 + 4 * 32 * 4; }

template <int DH>
__global__ void __launch_bounds__(128)
attn_bwd_dkv_mma_kernel(const bf16* __restrict__ qkv, const float* __restrict__ lse,
                        const bf16* __restrict__ dout, const float* __restrict__ dsum,
                        bf16* __restrict__ dqkv, int S, int H, int causal, float scale,
                        const int* __restrict__ lens) {
  constexpr int BKV = 64, BQ = 32, KS = DH / 16;
  extern __shared__ __align__(128) uint8_t smem_dkv[];
  uint8_t* sK = smem_dkv;
  uint8_t* sV = sK + BKV * DH * 2;
  constexpr int TB = BQ * DH * 2;
  uint8_t* sQ = sV + BKV * DH * 2;
  uint8_t* sG = sQ + 2 * TB;
  float* sLb = reinterpret_cast<float*>(sG + 2 * TB);
  float* sDb = sLb + 2 * BQ;
  const int b = blockIdx.z, h = blockIdx.y, kr0 = blockIdx.x * BKV;
  const int d = H * DH;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const bf16* qb = qkv + (int64_t)b * S * 3 * d + (int64_t)h * DH;
  const bf16* kb = qb + d;
  const bf16* vb = qb + 2 * d;
  const bf16* gb = dout + (int64_t)b * S * d + (int64_t)h * DH;
  const uint32_t tK = (uint32_t)__cvta_generic_to_shared(sK);
  const uint32_t tV = (uint32_t)__cvta_generic_to_shared(sV);
  const uint32_t tQb = (uint32_t)__cvta_generic_to_shared(sQ);
  const uint32_t tGb = (uint32_t)__cvta_generic_to_shared(sG);

  stage_tile<BKV, DH>(sK, kb, 3 * d, kr0, S);
  stage_tile<BKV, DH>(sV, vb, 3 * d, kr0, S);

  float dk[DH / 8][4], dv[DH / 8][4];
#pragma unroll
  for (int i = 0; i < DH / 8; ++i) {
    dk[i][0] = dk[i][1] = dk[i][2] = dk[i][3] = 0.f;
    dv[i][0] = dv[i][1] = dv[i][2] = dv[i][3] = 0.f;
  }
  const float sl2 = scale * kLog2e;
  const int key_lo = kr0 + warp * 16 + g;             // this thread's key rows: key_lo, key_lo + 8
  const int q_begin = causal ? (kr0 / BQ) * BQ : 0;
  const int klen = key_len_of(lens, b, S);             // keys at or after klen are padding: dk = dv = 0

  // per query tile: Q and dO rows through cp.async, LSE and dsum with plain loads, all double-buffered
  auto prefetch = [&](int q0, int bf) {
    stage_tile_async<BQ, DH>(tQb + bf * TB, qb, 3 * d, q0, S);
    stage_tile_async<BQ, DH>(tGb + bf * TB, gb, d, q0, S);
    cp_async_commit();
    if (threadIdx.x < BQ) {
      const int row = q0 + threadIdx.x;
      const bool ok = row < S;
      sLb[bf * BQ + threadIdx.x] = ok ? lse[((int64_t)b * H + h) * S + row] * kLog2e : 0.f;
      sDb[bf * BQ + threadIdx.x] = ok ? dsum[((int64_t)b * H + h) * S + row] : 0.f;
    }
  };
  if (q_begin < S) prefetch(q_begin, 0);
  int buf = 0;
  for (int q0 = q_begin; q0 < S; q0 += BQ, buf ^= 1) {
    if (q0 + BQ < S) {
      prefetch(q0 + BQ, buf ^ 1);
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    const uint32_t tQ = tQb + buf * TB, tG = tGb + buf * TB;
    const float* sL = sLb + buf * BQ;
    const float* sD = sDb + buf * BQ;
    // S^T = K Q^T and dP^T = V dO^T, 16 keys x 32 queries per warp
    float sacc[BQ / 8][4], pacc[BQ / 8][4];
#pragma unroll
    for (int i = 0; i < BQ / 8; ++i) {
      sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f;
      pacc[i][0] = pacc[i][1] = pacc[i][2] = pacc[i][3] = 0.f;
    }
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      uint32_t ka[4], va[4];
      load_a<DH>(ka, tK, warp * 16, ks * 16, lane);
      load_a<DH>(va, tV, warp * 16, ks * 16, lane);
#pragma unroll
      for (int np = 0; np < BQ / 16; ++np) {
        uint32_t bfr[4];
        load_b_nk<DH>(bfr, tQ, np * 16, ks * 16, lane);
        mma16816(sacc[2 * np], ka, bfr[0], bfr[1]);
        mma16816(sacc[2 * np + 1], ka, bfr[2], bfr[3]);
        load_b_nk<DH>(bfr, tG, np * 16, ks * 16, lane);
        mma16816(pacc[2 * np], va, bfr[0], bfr[1]);
        mma16816(pacc[2 * np + 1], va, bfr[2], bfr[3]);
      }
    }
    // P^T and dS^T (masked entries 0); rows are keys, columns are queries
#pragma unroll
    for (int i = 0; i < BQ / 8; ++i) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int qc = i * 8 + 2 * t + (e & 1);
        const int qrow = q0 + qc;
        const int key = key_lo + (e >> 1) * 8;
        float p = 0.f, ds = 0.f;
        if (qrow < S && key < klen && !(causal && key > qrow)) {
          p = exp2f(sacc[i][e] * sl2 - sL[qc]);
          ds = p * (pacc[i][e] - sD[qc]);
        }
        sacc[i][e] = p;
        pacc[i][e] = ds;
      }
    }
    // dV += P^T dO ; dK += dS^T Q
#pragma unroll
    for (int j = 0; j < BQ / 16; ++j) {
      uint32_t pa[4], da[4];
      pa[0] = pack_bf16(sacc[2 * j][0], sacc[2 * j][1]);
      pa[1] = pack_bf16(sacc[2 * j][2], sacc[2 * j][3]);
      pa[2] = pack_bf16(sacc[2 * j + 1][0], sacc[2 * j + 1][1]);
      pa[3] = pack_bf16(sacc[2 * j + 1][2], sacc[2 * j + 1][3]);
      da[0] = pack_bf16(pacc[2 * j][0], pacc[2 * j][1]);
      da[1] = pack_bf16(pacc[2 * j][2], pacc[2 * j][3]);
      da[2] = pack_bf16(pacc[2 * j + 1][0], pacc[2 * j + 1][1]);
      da[3] = pack_bf16(pacc[2 * j + 1][2], pacc[2 * j + 1][3]);
#pragma unroll
      for (int np = 0; np < DH / 16; ++np) {
        uint32_t bfr[4];
        load_b_kn<DH>(bfr, tG, j * 16, np * 16, lane);
        mma16816(dv[2 * np], pa, bfr[0], bfr[1]);
        mma16816(dv[2 * np + 1], pa, bfr[2], bfr[3]);
        load_b_kn<DH>(bfr, tQ, j * 16, np * 16, lane);
        mma16816(dk[2 * np], da, bfr[0], bfr[1]);
        mma16816(dk[2 * np + 1], da, bfr[2], bfr[3]);
      }
    }
    __syncthreads();                                   // this buffer is refilled two iterations from now
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int key = key_lo + r * 8;
    if (key >= S) continue;
    bf16* outk = dqkv + ((int64_t)b * S + key) * 3 * d + d + (int64_t)h * DH;
    bf16* outv = outk + d;
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) {
      *reinterpret_cast<uint32_t*>(outk + i * 8 + 2 * t) = pack_bf16(dk[i][2 * r] * scale, dk[i][2 * r + 1] * scale);
      *reinterpret_cast<uint32_t*>(outv + i * 8 + 2 * t) = pack_bf16(dv[i][2 * r], dv[i][2 * r + 1]);
    }
  }
}

}  // namespace hift
