// Attention backward on tcgen05: all five products run on the tensor cores with their
// accumulators in tensor memory; probabilities are recomputed from the saved log-sum-exp.
// Included into gemm_tc.cu after attention_tc.cuh (shares its PTX wrappers and descriptors).
//
// Two launches of one kernel template, so that every output row has exactly one writer and a
// fixed summation order (no atomics):
//   MODE 0 (dK, dV): one CTA owns 128 keys (tensor-memory lanes) and streams the queries
//   MODE 1 (dQ)    : one CTA owns 128 queries and streams the keys
// "Fixed" tiles F0, F1 [128, d_h] are loaded once, "streamed" tiles X0, X1 [64, d_h] go through
// a 3-deep TMA ring:
//              F0   F1    X0   X1     tS = F0 X0^T     tP = F1 X1^T     accumulators
//   MODE 0     K    V     Q    dO     scores^T         (dO V^T)^T       dV += P^T dO,  dK += dS^T Q
//   MODE 1     Q    dO    K    V      scores           dO V^T           dQ += dS K
// With P = exp(scale * scores - lse) and dS = P o (dP - D), D = rowsum(dO o O) (computed by a
// separate small kernel).  dK and dQ are multiplied by `scale` when they are stored.
//
//   warp 0     : TMA producer
//   warp 1     : MMA issuer and tensor-memory owner
//   warps 2-17 : element-wise stage, thread = one tensor-memory lane (a key in MODE 0, a query in
//                MODE 1) x 16 of the 64 streamed columns: read tS and tP, form P and dS, write
//                them as bf16 into 128-byte-swizzled shared tiles (the A operands of the
//                accumulating products); at the end convert and store the accumulators.
// tS / tP and the P / dS tiles are double-buffered, so the tensor core works on step t+1's
// scores while the element-wise warps are busy with step t.
#pragma once

constexpr int kAbThreads = 576;
constexpr int kAbEwWarps = 16;
constexpr int kAbF = 128;      // rows of a fixed tile
constexpr int kAbX = 64;       // rows of a streamed tile
constexpr int kAbStages = 3;

template <int DH, int MODE> struct AttnBwdCfg {
  static constexpr int kFBytes = kAbF * DH * 2;
  static constexpr int kXBytes = kAbX * DH * 2;
  static constexpr int kPBytes = kAbF * kAbX * 2;                 // one P or dS tile
  static constexpr int kNP = MODE == 0 ? 2 : 1;                   // P and dS, or dS only
  static constexpr int kSmem = 2 * kFBytes + kAbStages * 2 * kXBytes + 2 * kNP * kPBytes + 1024 + 256;
};

__device__ __forceinline__ void tmem_ld16_nowait(uint32_t addr, uint32_t (&v)[16]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
               : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
               : "r"(addr));
}
// Waits for the loads above; the registers are named as in/out operands so that no use of them
// can be scheduled ahead of the wait.
__device__ __forceinline__ void tmem_ld_wait16(uint32_t (&v)[16]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]), "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15])
               :: "memory");
}
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <int DH, int MODE>
__global__ void __launch_bounds__(kAbThreads, 1)
attn_bwd_tc_kernel(const __grid_constant__ CUtensorMap map_f0, const __grid_constant__ CUtensorMap map_f1,
                   const __grid_constant__ CUtensorMap map_x0, const __grid_constant__ CUtensorMap map_x1,
                   int col_f0, int col_f1, int col_x0, int col_x1,      // column of head 0 in each tensor
                   const float* __restrict__ lse, const float* __restrict__ dsum,
                   __nv_bfloat16* __restrict__ dqkv, int S, int H, int causal, float scale) {
  typedef AttnBwdCfg<DH, MODE> Cfg;
  constexpr int SP = DH / 64;                            // 64-column swizzle spans per tile row
  constexpr int FSPAN = kAbF * 128, XSPAN = kAbX * 128;  // bytes of one span of a fixed / streamed tile
  constexpr int NP = Cfg::kNP;
  extern __shared__ uint8_t smem_raw[];
  const int b = blockIdx.z, h = blockIdx.y, f0 = blockIdx.x * kAbF;
  const int d = H * DH;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sF0 = base, sF1 = sF0 + Cfg::kFBytes;
  const uint32_t sX = sF1 + Cfg::kFBytes;                // stage s: X0 at sX + s*2*kXBytes, X1 right after it
  const uint32_t sP = sX + kAbStages * 2 * Cfg::kXBytes; // buffer u: dS at sP + u*NP*kPBytes, then P (MODE 0)
  const uint32_t bar = sP + 2 * NP * Cfg::kPBytes;
  const uint32_t f_full = bar;
  auto x_full = [&](int s) { return bar + 8u + 8u * s; };
  auto x_empty = [&](int s) { return bar + 32u + 8u * s; };
  auto s_full = [&](int u) { return bar + 56u + 8u * u; };
  auto s_free = [&](int u) { return bar + 72u + 8u * u; };
  auto p_ready = [&](int u) { return bar + 88u + 8u * u; };
  auto p_free = [&](int u) { return bar + 104u + 8u * u; };
  const uint32_t acc_done = bar + 120u, tmem_slot = bar + 128u;
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot_gen = reinterpret_cast<volatile uint32_t*>(gen + (tmem_slot - base));
  uint8_t* p_gen = gen + (sP - base);

  // streamed 64-row blocks this CTA visits: [x_lo, x_hi)
  const int nx_all = (S + kAbX - 1) / kAbX;
  int x_lo = 0, x_hi = nx_all;
  if (causal) {
    if (MODE == 0) x_lo = f0 / kAbX;                                   // queries at or after the first key
    else x_hi = min(nx_all, (f0 + kAbF) / kAbX);                       // keys up to the last query
  }
  const int nsteps = x_hi - x_lo;
  const bool poisoned = g_tc_error != 0;

  if (threadIdx.x == 0) {
    mbar_init(f_full, 1);
    for (int i = 0; i < kAbStages; ++i) { mbar_init(x_full(i), 1); mbar_init(x_empty(i), 1); }
    for (int i = 0; i < 2; ++i) {
      mbar_init(s_full(i), 1); mbar_init(s_free(i), kAbEwWarps);
      mbar_init(p_ready(i), kAbEwWarps); mbar_init(p_free(i), 1);
    }
    mbar_init(acc_done, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_gen;
  // tensor-memory columns: tS[u] at 64u, tP[u] at 128 + 64u, accumulators from 256
  const uint32_t tAcc0 = tmem_base + 256;                // dS-fed accumulator: dK (MODE 0) / dQ (MODE 1)
  const uint32_t tAcc1 = tmem_base + 256 + DH;           // P-fed accumulator: dV (MODE 0 only)

  const int row_g0 = b * S;

  if (warp == 0) {
    // ---------------- TMA producer
    if (lane == 0 && !poisoned) {
      mbar_expect_tx(f_full, 2 * Cfg::kFBytes);
#pragma unroll
      for (int sp = 0; sp < SP; ++sp) {
        tma_load_2d(sF0 + sp * FSPAN, &map_f0, f_full, col_f0 + h * DH + sp * 64, row_g0 + f0);
        tma_load_2d(sF1 + sp * FSPAN, &map_f1, f_full, col_f1 + h * DH + sp * 64, row_g0 + f0);
      }
      int st = 0;
      uint32_t ph = 0;
      for (int t = 0; t < nsteps; ++t) {
        if (!mbar_wait(x_empty(st), ph ^ 1)) { atomicCAS(&g_tc_error, 0, 7); break; }
        const uint32_t s0 = sX + st * 2 * Cfg::kXBytes, s1 = s0 + Cfg::kXBytes;
        const int xrow = row_g0 + (x_lo + t) * kAbX;
        mbar_expect_tx(x_full(st), 2 * Cfg::kXBytes);
#pragma unroll
        for (int sp = 0; sp < SP; ++sp) {
          tma_load_2d(s0 + sp * XSPAN, &map_x0, x_full(st), col_x0 + h * DH + sp * 64, xrow);
          tma_load_2d(s1 + sp * XSPAN, &map_x1, x_full(st), col_x1 + h * DH + sp * 64, xrow);
        }
        if (++st == kAbStages) { st = 0; ph ^= 1; }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer
    if (lane == 0 && !poisoned) {
      // tS / tP: A and B K-major, M 128 x N 64.  Accumulators: A K-major (P / dS), B N-major, N = DH.
      const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kAbX >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
      const uint32_t idesc_a = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(DH >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
      bool ok = mbar_wait(f_full, 0);
      if (!ok) atomicCAS(&g_tc_error, 0, 8);
      // scores and dP of step t into buffer t & 1
      auto issue_s = [&](int t) -> bool {
        const int u = t & 1, st = t % kAbStages;
        if (!mbar_wait(x_full(st), (uint32_t)((t / kAbStages) & 1))) { atomicCAS(&g_tc_error, 0, 8); return false; }
        if (!mbar_wait(s_free(u), (uint32_t)(((t >> 1) & 1) ^ 1))) { atomicCAS(&g_tc_error, 0, 8); return false; }
        tc_fence_after();
        const uint32_t s0 = sX + st * 2 * Cfg::kXBytes, s1 = s0 + Cfg::kXBytes;
        const uint32_t ts = tmem_base + (uint32_t)(u * kAbX), tp = tmem_base + 128u + (uint32_t)(u * kAbX);
#pragma unroll
        for (int kk = 0; kk < DH / 16; ++kk) {
          const uint32_t fo = (uint32_t)((kk / 4) * FSPAN + (kk % 4) * 32), xo = (uint32_t)((kk / 4) * XSPAN + (kk % 4) * 32);
          tc_mma(ts, desc_kmajor(sF0 + fo), desc_kmajor(s0 + xo), idesc_s, kk > 0 ? 1u : 0u);
        }
#pragma unroll
        for (int kk = 0; kk < DH / 16; ++kk) {
          const uint32_t fo = (uint32_t)((kk / 4) * FSPAN + (kk % 4) * 32), xo = (uint32_t)((kk / 4) * XSPAN + (kk % 4) * 32);
          tc_mma(tp, desc_kmajor(sF1 + fo), desc_kmajor(s1 + xo), idesc_s, kk > 0 ? 1u : 0u);
        }
        tc_commit(s_full(u));
        return true;
      };
      if (ok && nsteps > 0) ok = issue_s(0);
      if (ok && nsteps > 1) ok = issue_s(1);
      for (int t = 0; t < nsteps && ok; ++t) {
        const int u = t & 1, st = t % kAbStages;
        if (!mbar_wait(p_ready(u), (uint32_t)((t >> 1) & 1))) { atomicCAS(&g_tc_error, 0, 8); ok = false; break; }
        tc_fence_after();
        const uint32_t s0 = sX + st * 2 * Cfg::kXBytes, s1 = s0 + Cfg::kXBytes;
        const uint32_t sdS = sP + (uint32_t)(u * NP * Cfg::kPBytes), sPr = sdS + Cfg::kPBytes;
#pragma unroll
        for (int kk = 0; kk < kAbX / 16; ++kk)       // 16 streamed rows per MMA: 32 B along the A tile's row, 16 rows of B
          tc_mma(tAcc0, desc_kmajor(sdS + kk * 32), desc_nmajor(s0 + (uint32_t)(kk * 16 * 128), XSPAN), idesc_a,
                 (t > 0 || kk > 0) ? 1u : 0u);
        if (MODE == 0) {
#pragma unroll
          for (int kk = 0; kk < kAbX / 16; ++kk)
            tc_mma(tAcc1, desc_kmajor(sPr + kk * 32), desc_nmajor(s1 + (uint32_t)(kk * 16 * 128), XSPAN), idesc_a,
                   (t > 0 || kk > 0) ? 1u : 0u);
        }
        tc_commit(p_free(u));
        tc_commit(x_empty(st));
        if (t + 2 < nsteps) ok = issue_s(t + 2);
      }
      if (ok) tc_commit(acc_done);
    }
  } else {
    // ---------------- element-wise warps
    const int q = warp & 3;                               // tensor-memory lane quarter this warp may access
    const int part = (warp - 2) >> 2;                     // which 16 of the 64 streamed columns
    const int r = q * 32 + lane;                          // row of the fixed tile
    const int frow = f0 + r;                              // key (MODE 0) / query (MODE 1) index in the sequence
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    const float sl2 = scale * 1.4426950408889634f;
    const float* lse_bh = lse + ((int64_t)b * H + h) * S;
    const float* dsum_bh = dsum + ((int64_t)b * H + h) * S;
    float row_l2 = 0.f, row_d = 0.f;                      // MODE 1: this query's lse * log2(e) and D
    if (MODE == 1) {
      const int qi = min(frow, S - 1);
      row_l2 = lse_bh[qi] * 1.4426950408889634f;
      row_d = dsum_bh[qi];
    }
    bool ok = !poisoned;
    for (int t = 0; t < nsteps; ++t) {
      const int u = t & 1;
      const int xb0 = (x_lo + t) * kAbX;                  // first streamed index of this step's block
      const int x0 = xb0 + part * 16;                     // ... and of this thread's 16 columns
      // MODE 0: lanes 0-15 hold lse * log2(e) of columns x0 .. x0+15, lanes 16-31 their D
      float col_v = 0.f;
      if (MODE == 0) {
        const int qi = min(x0 + (lane & 15), S - 1);
        col_v = lane < 16 ? lse_bh[qi] * 1.4426950408889634f : dsum_bh[qi];
      }
      // masking is needed only where the block touches the diagonal or the end of the sequence
      const int k_hi = MODE == 0 ? f0 + kAbF - 1 : xb0 + kAbX - 1;      // largest key of the block
      const int q_lo = MODE == 0 ? xb0 : f0;                            // smallest query of the block
      const bool masked = (causal && k_hi > q_lo) || f0 + kAbF > S || xb0 + kAbX > S;
      bool ready = ok && mbar_wait(s_full(u), (uint32_t)((t >> 1) & 1));
      if (ok && !ready && lane == 0) atomicCAS(&g_tc_error, 0, 9);
      tc_fence_after();
      ok = __all_sync(0xffffffffu, ready && *(volatile int*)&g_tc_error == 0);
      if (!ok) break;
      uint32_t sv[16], pv[16];
      tmem_ld16_nowait(tmem_base + lane_off + (uint32_t)(u * kAbX + part * 16), sv);
      tmem_ld16_nowait(tmem_base + lane_off + 128u + (uint32_t)(u * kAbX + part * 16), pv);
      tmem_ld_wait16(sv);
      tmem_ld_wait16(pv);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(s_free(u));              // the tensor core may overwrite tS / tP [u]
      uint32_t pk_p[8], pk_ds[8];
#pragma unroll
      for (int i = 0; i < 16; i += 2) {
        float pp[2], dd[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const float l2 = MODE == 0 ? __shfl_sync(0xffffffffu, col_v, i + e) : row_l2;
          const float dv = MODE == 0 ? __shfl_sync(0xffffffffu, col_v, 16 + i + e) : row_d;
          float p = ex2_approx(fmaf(__uint_as_float(sv[i + e]), sl2, -l2));
          if (masked) {
            const int xi = x0 + i + e;
            const int key = MODE == 0 ? frow : xi, qry = MODE == 0 ? xi : frow;
            if (key >= S || qry >= S || (causal && key > qry)) p = 0.f;
          }
          pp[e] = p;
          dd[e] = p * (__uint_as_float(pv[i + e]) - dv);
        }
        __nv_bfloat162 hp = __floats2bfloat162_rn(pp[0], pp[1]), hd = __floats2bfloat162_rn(dd[0], dd[1]);
        pk_p[i >> 1] = *reinterpret_cast<uint32_t*>(&hp);
        pk_ds[i >> 1] = *reinterpret_cast<uint32_t*>(&hd);
      }
      // the products that read this buffer two steps ago must be done before it is overwritten
      ready = mbar_wait(p_free(u), (uint32_t)(((t >> 1) & 1) ^ 1));
      if (!ready && lane == 0) atomicCAS(&g_tc_error, 0, 9);
      ok = __all_sync(0xffffffffu, ready);
      if (!ok) break;
      // row r of a [128][64] bf16 tile = one 128-byte swizzle span; this thread owns 16-byte chunks 2*part, 2*part+1
      uint8_t* ds_row = p_gen + u * NP * Cfg::kPBytes + r * 128;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        const int chunk = part * 2 + c;
        const int off = (chunk ^ (r & 7)) << 4;
        *reinterpret_cast<uint4*>(ds_row + off) = make_uint4(pk_ds[4 * c], pk_ds[4 * c + 1], pk_ds[4 * c + 2], pk_ds[4 * c + 3]);
        if (MODE == 0)
          *reinterpret_cast<uint4*>(ds_row + Cfg::kPBytes + off) = make_uint4(pk_p[4 * c], pk_p[4 * c + 1], pk_p[4 * c + 2], pk_p[4 * c + 3]);
      }
      fence_async_smem();                                 // read next by the tensor core (async proxy)
      __syncwarp();
      if (lane == 0) mbar_arrive(p_ready(u));
    }
    // ---------------- accumulators -> global: this thread stores DH/4 columns of its row
    if (ok && nsteps > 0) {
      const bool ready = mbar_wait(acc_done, 0);
      if (!ready && lane == 0) atomicCAS(&g_tc_error, 0, 9);
      tc_fence_after();
      ok = __all_sync(0xffffffffu, ready && *(volatile int*)&g_tc_error == 0);
    }
    if (ok && nsteps > 0) {
      constexpr int CW = DH / 4;                          // 16 or 32
      __nv_bfloat16* orow = dqkv + ((int64_t)(row_g0 + frow)) * (3 * d) + (int64_t)h * DH + part * CW;
#pragma unroll 1
      for (int a = 0; a < (MODE == 0 ? 2 : 1); ++a) {
        // a = 0: dS-fed accumulator (dK -> column block d, or dQ -> column block 0), scaled; a = 1: dV -> block 2d
        const uint32_t tacc = (a == 0 ? tAcc0 : tAcc1) + lane_off + (uint32_t)(part * CW);
        __nv_bfloat16* dst = orow + (MODE == 0 ? (a == 0 ? d : 2 * d) : 0);
        const float mul = a == 0 ? scale : 1.0f;
        uint32_t v[CW];
        if constexpr (CW == 32) {
          tmem_ld32(tacc, v);
        } else {
          tmem_ld16_nowait(tacc, v);
          tmem_ld_wait16(v);
        }
        if (frow < S) {
#pragma unroll
          for (int i = 0; i < CW; i += 8) {
            uint4 pk;
            __nv_bfloat162* hp = reinterpret_cast<__nv_bfloat162*>(&pk);
#pragma unroll
            for (int e = 0; e < 4; ++e)
              hp[e] = __floats2bfloat162_rn(__uint_as_float(v[i + 2 * e]) * mul, __uint_as_float(v[i + 2 * e + 1]) * mul);
            *reinterpret_cast<uint4*>(dst + i) = pk;
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}
