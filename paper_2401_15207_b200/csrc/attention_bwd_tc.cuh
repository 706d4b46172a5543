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
//   warp 1     : issues the scores / dP products (one thread); owns the tensor memory
//   warp 2     : issues the accumulating products (one thread); two issuers, because these
//                products are small and one thread cannot issue them as fast as they execute
//   warps 3-18 : element-wise stage in two groups of eight that take alternate steps; thread = one
//                tensor-memory lane (a key in MODE 0, a query in MODE 1) x 32 of the 64 streamed
//                columns: read tS and tP, form P and dS, write them as bf16 into 128-byte-swizzled
//                shared tiles (the A operands of the accumulating products); at the end all sixteen
//                warps convert and store the accumulators.
// tS / tP are double-buffered, so the tensor core works on step t+1's scores while the
// element-wise warps are busy with step t.  The kernel is persistent: a CTA walks a list of
// (batch, head, 128-row block) items, heaviest first; with a second set of fixed tiles (d_h = 64) the
// next item's tiles are fetched and its first scores computed while the current item finishes.
#pragma once

constexpr int kAbThreads = 608;
constexpr int kAbEwWarps = 16;
constexpr int kAbF = 128;      // rows of a fixed tile
constexpr int kAbX = 64;       // rows of a streamed tile

// Shared-memory plan.  d_h = 128: one set of fixed tiles, a 3-deep ring of streamed tiles and two
// P / dS buffers fill the 227 KB; d_h = 64: everything is half the size, so a second set of fixed
// tiles lets the next item's first scores be computed while the current item finishes.
template <int DH, int MODE> struct AttnBwdCfg {
  static constexpr int kFBytes = kAbF * DH * 2;
  static constexpr int kXBytes = kAbX * DH * 2;
  static constexpr int kPBytes = kAbF * kAbX * 2;                 // one P or dS tile
  static constexpr int kNP = MODE == 0 ? 2 : 1;                   // P and dS, or dS only
  static constexpr int kNF = DH == 64 ? 2 : 1;                    // sets of fixed tiles
  static constexpr int kXS = 3;                                   // stages of the streamed ring
  static constexpr int kNPB = 2;                                  // P / dS buffers
  static constexpr int kSmem = kNF * 2 * kFBytes + kXS * 2 * kXBytes + kNPB * kNP * kPBytes + 1024 + 256;
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
// P and dS of 16 consecutive streamed columns of one fixed row, packed to bf16 pairs.
//   sv, pv   : scores and dP from tensor memory
//   MODE 0   : lane i of col_l2 / col_d holds lse * log2(e) / D of column lane_base + i (read by shuffle);
//   MODE 1   : row_l2 / row_d are this thread's own
//   MASKED   : the block touches the diagonal or the end of the sequence (decided per step, so the
//              common case carries no comparisons)
//   DROP     : dropout on the probabilities: with keep = 0 or 1 / (1 - p) per (query, key), the P that feeds dV is
//              P o keep and dS = P o (dP o keep - D).  MODE 1 draws one generator block per four of its keys; MODE 0
//              has one key and sixteen queries, so one block per element.
template <int MODE, bool MASKED, bool DROP>
__device__ __forceinline__ void ab_p_ds16(const uint32_t (&sv)[16], const uint32_t (&pv)[16], float col_l2, float col_d,
                                          int lane_base, float row_l2, float row_d, float sl2, int S, int klen, int causal,
                                          int frow, int x_first, uint32_t (&pk_p)[8], uint32_t (&pk_ds)[8],
                                          const DropArgs& da, int bh) {
  uint4 w4 = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
  for (int i = 0; i < 16; i += 2) {
    float pp[2], dd[2];
    if (DROP && MODE == 1 && (i & 3) == 0) w4 = attn_drop_words(da, bh, S, min(frow, S - 1), x_first + i);
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const float l2 = MODE == 0 ? __shfl_sync(0xffffffffu, col_l2, lane_base + i + e) : row_l2;
      const float dv = MODE == 0 ? __shfl_sync(0xffffffffu, col_d, lane_base + i + e) : row_d;
      float p = ex2_approx(fmaf(__uint_as_float(sv[i + e]), sl2, -l2));
      if (MASKED) {
        const int xi = x_first + i + e;
        const int key = MODE == 0 ? frow : xi, qry = MODE == 0 ? xi : frow;
        if (key >= klen || qry >= S || (causal && key > qry)) p = 0.f;
      }
      if (DROP) {
        uint32_t word;
        if (MODE == 1) word = word_of(w4, (i + e) & 3);
        else word = word_of(attn_drop_words(da, bh, S, min(x_first + i + e, S - 1), frow & ~3), frow & 3);
        const float keep = word < da.thr ? 0.f : da.scale;
        pp[e] = p * keep;
        dd[e] = p * (__uint_as_float(pv[i + e]) * keep - dv);
      } else {
        pp[e] = p;
        dd[e] = p * (__uint_as_float(pv[i + e]) - dv);
      }
    }
    __nv_bfloat162 hp = __floats2bfloat162_rn(pp[0], pp[1]), hd = __floats2bfloat162_rn(dd[0], dd[1]);
    pk_p[i >> 1] = *reinterpret_cast<uint32_t*>(&hp);
    pk_ds[i >> 1] = *reinterpret_cast<uint32_t*>(&hd);
  }
}

template <int DH, int MODE, bool DROP>
__global__ void __launch_bounds__(kAbThreads, 1)
attn_bwd_tc_kernel(const __grid_constant__ CUtensorMap map_f0, const __grid_constant__ CUtensorMap map_f1,
                   const __grid_constant__ CUtensorMap map_x0, const __grid_constant__ CUtensorMap map_x1,
                   int col_f0, int col_f1, int col_x0, int col_x1,      // column of head 0 in each tensor
                   const float* __restrict__ lse, const float* __restrict__ dsum,
                   __nv_bfloat16* __restrict__ dqkv, int B, int S, int H, int causal, float scale,
                   const int* __restrict__ lens, DropArgs da) {
  typedef AttnBwdCfg<DH, MODE> Cfg;
  constexpr int SP = DH / 64;                            // 64-column swizzle spans per tile row
  constexpr int FSPAN = kAbF * 128, XSPAN = kAbX * 128;  // bytes of one span of a fixed / streamed tile
  constexpr int NP = Cfg::kNP;
  extern __shared__ uint8_t smem_raw[];
  const int d = H * DH;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  constexpr int NF = Cfg::kNF, XS = Cfg::kXS, NPB = Cfg::kNPB;
  const uint32_t sF = base;                              // set i: F0 at sF + i*2*kFBytes, F1 right after it
  const uint32_t sX = sF + NF * 2 * Cfg::kFBytes;        // stage s: X0 at sX + s*2*kXBytes, X1 right after it
  const uint32_t sP = sX + XS * 2 * Cfg::kXBytes;        // buffer i: dS at sP + i*NP*kPBytes, then P (MODE 0)
  const uint32_t bar = sP + NPB * NP * Cfg::kPBytes;
  auto f_full = [&](int i) { return bar + 8u * i; };
  auto f_empty = [&](int i) { return bar + 16u + 8u * i; };
  auto x_full = [&](int i) { return bar + 32u + 8u * i; };          // up to 4 stages
  auto x_empty = [&](int i) { return bar + 64u + 8u * i; };
  auto s_full = [&](int u) { return bar + 96u + 8u * u; };
  auto s_free = [&](int u) { return bar + 112u + 8u * u; };
  auto p_ready = [&](int i) { return bar + 128u + 8u * i; };
  auto p_free = [&](int i) { return bar + 144u + 8u * i; };
  const uint32_t acc_done = bar + 160u, acc_free = bar + 168u, tmem_slot = bar + 176u;
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot_gen = reinterpret_cast<volatile uint32_t*>(gen + (tmem_slot - base));
  uint8_t* p_gen = gen + (sP - base);

  // Work items: (batch, head, block of 128 fixed rows), the blocks with the most streamed steps
  // first; this CTA takes items blockIdx.x, blockIdx.x + gridDim.x, ...  Every role below walks the
  // same list and counts the streamed steps it has passed (g), which fixes ring slots and phases.
  const int nfb = (S + kAbF - 1) / kAbF, nbh = B * H, nitems = nfb * nbh;
  const int nx_all = (S + kAbX - 1) / kAbX;
  struct Item { int b, h, f0, x_lo, nsteps; };
  auto item_of = [&](int idx) {
    Item it;
    const int rank = idx / nbh, bh = idx - rank * nbh;
    it.b = bh / H;
    it.h = bh - it.b * H;
    const int fb = (MODE == 1 && causal) ? nfb - 1 - rank : rank;
    it.f0 = fb * kAbF;
    int x_lo = 0, x_hi = nx_all;                         // streamed 64-row blocks visited: [x_lo, x_hi)
    if (causal) {
      if (MODE == 0) x_lo = it.f0 / kAbX;                // queries at or after the first key
      else x_hi = min(nx_all, (it.f0 + kAbF) / kAbX);    // keys up to the last query
    }
    it.x_lo = x_lo;
    it.nsteps = x_hi - x_lo;
    return it;
  };
  // The n-th item of this CTA.  The list is sorted by weight, so handing it out forwards on even rounds and backwards
  // on odd ones pairs a CTA's heavy items with light ones (plain round-robin gave the first CTAs the heaviest item of
  // every round: 10 key blocks against a mean of 8.65 at batch 4 x 512 x 32 heads, causal).
  auto item_at = [&](int n) {
    const int first = n * (int)gridDim.x;
    return (n & 1) ? first + (int)gridDim.x - 1 - (int)blockIdx.x : first + (int)blockIdx.x;
  };
  // one thread reads the time-out flag, after griddepcontrol.wait, and the CTA shares the answer: every role must take the same way
  volatile uint32_t* poison_gen = reinterpret_cast<volatile uint32_t*>(gen + (tmem_slot + 8u - base));

  if (threadIdx.x == 0) {
    for (int i = 0; i < NF; ++i) { mbar_init(f_full(i), 1); mbar_init(f_empty(i), 1); }      // freed by the score issuer: only its products read them
    for (int i = 0; i < XS; ++i) { mbar_init(x_full(i), 1); mbar_init(x_empty(i), 2); }
    for (int i = 0; i < 2; ++i) { mbar_init(s_full(i), 1); mbar_init(s_free(i), kAbEwWarps / 2); }   // one group of warps each
    for (int i = 0; i < NPB; ++i) { mbar_init(p_ready(i), kAbEwWarps / 2); mbar_init(p_free(i), 1); }
    mbar_init(acc_done, 1);
    mbar_init(acc_free, kAbEwWarps);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    pdl_wait();                                          // no global access before it, the flag included
    *poison_gen = g_tc_error != 0 ? 1u : 0u;
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_gen;
  const bool poisoned = *poison_gen != 0;
  pdl_trigger();
  pdl_wait();                                          // the set-up above may run under the predecessor's tail
  // tensor-memory columns: tS[u] at 64u, tP[u] at 128 + 64u, accumulators from 256
  const uint32_t tAcc0 = tmem_base + 256;                // dS-fed accumulator: dK (MODE 0) / dQ (MODE 1)
  const uint32_t tAcc1 = tmem_base + 256 + DH;           // P-fed accumulator: dV (MODE 0 only)

  if (warp == 0) {
    // ---------------- TMA producer
    if (lane == 0 && !poisoned) {
      int st = 0;
      uint32_t ph = 0;
      bool ok = true;
      int n = 0;
      for (int idx = item_at(n); idx < nitems && ok; idx = item_at(++n)) {
        const Item it = item_of(idx);
        const int row_g0 = it.b * S;
        // this set of fixed tiles is free once the last score product of the item that used it has completed (the
        // accumulating products read the streamed tiles and P / dS only), a step or two before that item ends
        const int fi = n % NF;
        if (!mbar_wait(f_empty(fi), (uint32_t)(((n / NF) & 1) ^ 1))) { atomicCAS(&g_tc_error, 0, 7); break; }
        const uint32_t sF0 = sF + fi * 2 * Cfg::kFBytes, sF1 = sF0 + Cfg::kFBytes;
        mbar_expect_tx(f_full(fi), 2 * Cfg::kFBytes);
#pragma unroll
        for (int sp = 0; sp < SP; ++sp) {
          tma_load_2d(sF0 + sp * FSPAN, &map_f0, f_full(fi), col_f0 + it.h * DH + sp * 64, row_g0 + it.f0);
          tma_load_2d(sF1 + sp * FSPAN, &map_f1, f_full(fi), col_f1 + it.h * DH + sp * 64, row_g0 + it.f0);
        }
        for (int t = 0; t < it.nsteps; ++t) {
          if (!mbar_wait(x_empty(st), ph ^ 1)) { atomicCAS(&g_tc_error, 0, 7); ok = false; break; }
          const uint32_t s0 = sX + st * 2 * Cfg::kXBytes, s1 = s0 + Cfg::kXBytes;
          const int xrow = row_g0 + (it.x_lo + t) * kAbX;
          mbar_expect_tx(x_full(st), 2 * Cfg::kXBytes);
#pragma unroll
          for (int sp = 0; sp < SP; ++sp) {
            tma_load_2d(s0 + sp * XSPAN, &map_x0, x_full(st), col_x0 + it.h * DH + sp * 64, xrow);
            tma_load_2d(s1 + sp * XSPAN, &map_x1, x_full(st), col_x1 + it.h * DH + sp * 64, xrow);
          }
          if (++st == XS) { st = 0; ph ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer 1: scores and dP of every step into tS / tP [g & 1]; runs ahead of
    //                  the element-wise warps as far as the two buffers (s_free) allow
    if (lane == 0 && !poisoned) {
      // A and B K-major, M 128 x N 64
      const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kAbX >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
      int n = 0, g = 0;
      bool ok = true;
      for (int idx = item_at(n); idx < nitems && ok; idx = item_at(++n)) {
        const Item it = item_of(idx);
        const int fi = n % NF;
        if (!mbar_wait(f_full(fi), (uint32_t)((n / NF) & 1))) { atomicCAS(&g_tc_error, 0, 8); break; }
        const uint64_t dF0 = desc_kmajor(sF + fi * 2 * Cfg::kFBytes), dF1 = desc_kmajor(sF + fi * 2 * Cfg::kFBytes + Cfg::kFBytes);
        for (int t = 0; t < it.nsteps; ++t, ++g) {
          const int u = g & 1, st = g % XS;
          if (!mbar_wait(x_full(st), (uint32_t)((g / XS) & 1)) || !mbar_wait(s_free(u), (uint32_t)(((g >> 1) & 1) ^ 1))) {
            atomicCAS(&g_tc_error, 0, 8); ok = false; break;
          }
          tc_fence_after();
          const uint64_t dX0 = desc_kmajor(sX + st * 2 * Cfg::kXBytes), dX1 = desc_kmajor(sX + st * 2 * Cfg::kXBytes + Cfg::kXBytes);
          const uint32_t ts = tmem_base + (uint32_t)(u * kAbX), tp = tmem_base + 128u + (uint32_t)(u * kAbX);
#pragma unroll
          for (int kk = 0; kk < DH / 16; ++kk) {         // descriptor addresses are in 16-byte units
            const uint64_t fo = (uint64_t)(((kk / 4) * FSPAN + (kk % 4) * 32) >> 4), xo = (uint64_t)(((kk / 4) * XSPAN + (kk % 4) * 32) >> 4);
            tc_mma(ts, dF0 + fo, dX0 + xo, idesc_s, kk > 0 ? 1u : 0u);
          }
#pragma unroll
          for (int kk = 0; kk < DH / 16; ++kk) {
            const uint64_t fo = (uint64_t)(((kk / 4) * FSPAN + (kk % 4) * 32) >> 4), xo = (uint64_t)(((kk / 4) * XSPAN + (kk % 4) * 32) >> 4);
            tc_mma(tp, dF1 + fo, dX1 + xo, idesc_s, kk > 0 ? 1u : 0u);
          }
          tc_commit(s_full(u));
          tc_commit(x_empty(st));                        // this thread's reads of the stage (the other issuer arrives too)
        }
        if (ok) tc_commit(f_empty(fi));
      }
    }
  } else if (warp == 2) {
    // ---------------- MMA issuer 2: the accumulating products, fed by the element-wise warps
    if (lane == 0 && !poisoned) {
      // A K-major (P / dS), B N-major (the streamed tile as it lies), M 128 x N d_h
      const uint32_t idesc_a = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(DH >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
      int n = 0, g = 0;
      bool ok = true;
      for (int idx = item_at(n); idx < nitems && ok; idx = item_at(++n)) {
        const Item it = item_of(idx);
        for (int t = 0; t < it.nsteps; ++t, ++g) {
          const int st = g % XS, pb = g % NPB;
          if (!mbar_wait(p_ready(pb), (uint32_t)((g / NPB) & 1)) || !mbar_wait(x_full(st), (uint32_t)((g / XS) & 1))) {
            atomicCAS(&g_tc_error, 0, 8); ok = false; break;
          }
          // the first product of an item overwrites the accumulators: the previous item's must have been read
          if (t == 0 && n > 0 && !mbar_wait(acc_free, (uint32_t)((n - 1) & 1))) { atomicCAS(&g_tc_error, 0, 8); ok = false; break; }
          tc_fence_after();
          const uint32_t s0 = sX + st * 2 * Cfg::kXBytes, s1 = s0 + Cfg::kXBytes;
          const uint64_t ddS = desc_kmajor(sP + (uint32_t)(pb * NP * Cfg::kPBytes)), dPr = desc_kmajor(sP + (uint32_t)(pb * NP * Cfg::kPBytes) + Cfg::kPBytes);
          const uint64_t dB0 = desc_nmajor(s0, XSPAN), dB1 = desc_nmajor(s1, XSPAN);
#pragma unroll
          for (int kk = 0; kk < kAbX / 16; ++kk)     // 16 streamed rows per MMA: 32 B along the A tile's row, 16 rows of B
            tc_mma(tAcc0, ddS + (uint64_t)(kk * 32 >> 4), dB0 + (uint64_t)(kk * 16 * 128 >> 4), idesc_a, (t > 0 || kk > 0) ? 1u : 0u);
          if (MODE == 0) {
#pragma unroll
            for (int kk = 0; kk < kAbX / 16; ++kk)
              tc_mma(tAcc1, dPr + (uint64_t)(kk * 32 >> 4), dB1 + (uint64_t)(kk * 16 * 128 >> 4), idesc_a, (t > 0 || kk > 0) ? 1u : 0u);
          }
          tc_commit(p_free(pb));
          tc_commit(x_empty(st));
        }
        if (ok) tc_commit(acc_done);
      }
    }
  } else {
    // ---------------- element-wise warps: two groups of eight; group e takes the steps with
    //                  (g & 1) == e, so one group's waits and stores overlap the other's arithmetic
    const int q = warp & 3;                               // tensor-memory lane quarter this warp may access
    const int part = (warp - 3) >> 2;                     // 0..3: which quarter of the accumulator columns (epilogue)
    const int grp = part >> 1;                            // which steps
    const int hc = part & 1;                              // which 32 of the 64 streamed columns
    const int r = q * 32 + lane;                          // row of the fixed tile
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    const float sl2 = scale * 1.4426950408889634f;
    const int u = grp, pb = grp;                          // this group's tS / tP buffer and P / dS buffer
    bool ok = !poisoned;
    int g0 = 0, n = 0;
    // What an item needs before its first step (its description, the key length of its batch entry, and the first lse /
    // D values: MODE 1 this query's, MODE 0 those of the first step's columns) is fetched while the previous item's last
    // products finish, so that no global load stands between two items.
    struct Pre { Item it; int klen; float a, b; };
    auto prepare = [&](int idx, int g0v) {
      Pre p;
      p.a = 0.f; p.b = 0.f;
      p.it = item_of(idx);
      p.klen = tc_key_len(lens, p.it.b, S);
      const float* lse_p = lse + ((int64_t)p.it.b * H + p.it.h) * S;
      const float* dsum_p = dsum + ((int64_t)p.it.b * H + p.it.h) * S;
      if (MODE == 1) {
        const int qi = min(p.it.f0 + r, S - 1);
        p.a = lse_p[qi] * 1.4426950408889634f;
        p.b = dsum_p[qi];
      } else {
        const int t1 = (g0v ^ grp) & 1;
        if (t1 < p.it.nsteps) {
          const int c = min((p.it.x_lo + t1) * kAbX + hc * 32 + lane, S - 1);
          p.a = lse_p[c];
          p.b = dsum_p[c];
        }
      }
      return p;
    };
    Pre cur;
    if (item_at(0) < nitems && ok) cur = prepare(item_at(0), 0);
    for (int idx = item_at(n); idx < nitems && ok; idx = item_at(++n)) {
      const Item it = cur.it;
      const int f0 = it.f0, row_g0 = it.b * S;
      const int frow = f0 + r;                            // key (MODE 0) / query (MODE 1) index in the sequence
      const int klen = cur.klen;                          // keys at or after klen are padding: P = dS = 0 there
      const float* lse_bh = lse + ((int64_t)it.b * H + it.h) * S;
      const float* dsum_bh = dsum + ((int64_t)it.b * H + it.h) * S;
      const float row_l2 = cur.a, row_d = cur.b;          // MODE 1: this query's lse * log2(e) and D
      // MODE 0: lane i holds lse and D of column x0 + i of this thread's 32 columns; the values of
      // the group's next step are fetched while this step is worked on
      const int t_first = (g0 ^ grp) & 1;                 // first step of this item with (g & 1) == grp
      auto col_index = [&](int t) { return min((it.x_lo + t) * kAbX + hc * 32 + lane, S - 1); };
      float lse_next = cur.a, d_next = cur.b;
      for (int t = t_first; t < it.nsteps; t += 2) {
        const int g = g0 + t;
        const uint32_t par = (uint32_t)((g >> 1) & 1);
        const int xb0 = (it.x_lo + t) * kAbX;             // first streamed index of this step's block
        const float lse_raw = lse_next, d_raw = d_next;
        if (MODE == 0 && t + 2 < it.nsteps) { lse_next = lse_bh[col_index(t + 2)]; d_next = dsum_bh[col_index(t + 2)]; }
        // masking is needed only where the block touches the diagonal or the end of the sequence
        const int k_hi = MODE == 0 ? f0 + kAbF - 1 : xb0 + kAbX - 1;      // largest key of the block
        const int q_lo = MODE == 0 ? xb0 : f0;                            // smallest query of the block
        const bool masked = (causal && k_hi > q_lo) || f0 + kAbF > S || xb0 + kAbX > S || k_hi >= klen;
        bool ready = mbar_wait(s_full(u), par);
        if (!ready && lane == 0) atomicCAS(&g_tc_error, 0, 9);
        tc_fence_after();
        ok = __all_sync(0xffffffffu, ready);
        if (!ok) break;
        // the products that read this group's P / dS buffer last must be done before it is overwritten
        ready = mbar_wait(p_free(pb), par ^ 1);
        if (!ready && lane == 0) atomicCAS(&g_tc_error, 0, 9);
        ok = __all_sync(0xffffffffu, ready);
        if (!ok) break;
        const float col_l2 = lse_raw * 1.4426950408889634f;
        // row r of a [128][64] bf16 tile = one 128-byte swizzle span; this thread owns 16-byte chunks 4*hc .. 4*hc+3
        uint8_t* ds_row = p_gen + pb * NP * Cfg::kPBytes + r * 128;
#pragma unroll 1
        for (int hf = 0; hf < 2; ++hf) {                  // 16 columns at a time
          const int cb = hc * 32 + hf * 16;               // first of them inside the 64-column block
          uint32_t sv[16], pv[16];
          tmem_ld16_nowait(tmem_base + lane_off + (uint32_t)(u * kAbX + cb), sv);
          tmem_ld16_nowait(tmem_base + lane_off + 128u + (uint32_t)(u * kAbX + cb), pv);
          tmem_ld_wait16(sv);
          tmem_ld_wait16(pv);
          if (hf == 1) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(s_free(u));        // the tensor core may overwrite tS / tP [u]
          }
          uint32_t pk_p[8], pk_ds[8];
          const int bh = it.b * H + it.h;
          if (DROP) {              // with dropout every step takes the instance with the mask tests
            ab_p_ds16<MODE, true, true>(sv, pv, col_l2, d_raw, hf * 16, row_l2, row_d, sl2, S, klen, causal, frow, xb0 + cb, pk_p, pk_ds, da, bh);
          } else if (masked) {
            ab_p_ds16<MODE, true, false>(sv, pv, col_l2, d_raw, hf * 16, row_l2, row_d, sl2, S, klen, causal, frow, xb0 + cb, pk_p, pk_ds, da, bh);
          } else {
            ab_p_ds16<MODE, false, false>(sv, pv, col_l2, d_raw, hf * 16, row_l2, row_d, sl2, S, klen, causal, frow, xb0 + cb, pk_p, pk_ds, da, bh);
          }
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            const int chunk = hc * 4 + hf * 2 + c;
            const int off = (chunk ^ (r & 7)) << 4;
            *reinterpret_cast<uint4*>(ds_row + off) = make_uint4(pk_ds[4 * c], pk_ds[4 * c + 1], pk_ds[4 * c + 2], pk_ds[4 * c + 3]);
            if (MODE == 0)
              *reinterpret_cast<uint4*>(ds_row + Cfg::kPBytes + off) = make_uint4(pk_p[4 * c], pk_p[4 * c + 1], pk_p[4 * c + 2], pk_p[4 * c + 3]);
          }
        }
        fence_async_smem();                               // read next by the tensor core (async proxy)
        __syncwarp();
        if (lane == 0) mbar_arrive(p_ready(pb));
      }
      if (!ok) break;
      g0 += it.nsteps;
      if (item_at(n + 1) < nitems) cur = prepare(item_at(n + 1), g0);     // `it` and its values above are copies
      // ---------------- accumulators -> global: this thread stores DH/4 columns of its row
      {
        const bool ready = mbar_wait(acc_done, (uint32_t)(n & 1));
        if (!ready && lane == 0) atomicCAS(&g_tc_error, 0, 9);
        tc_fence_after();
        ok = __all_sync(0xffffffffu, ready);              // a role that gave up leaves acc_done unset
        if (!ok) break;
      }
      constexpr int CW = DH / 4;                          // 16 or 32
      uint32_t v0[CW], v1[CW];
      if constexpr (CW == 32) {
        tmem_ld32_nowait(tAcc0 + lane_off + (uint32_t)(part * CW), v0);
        if (MODE == 0) tmem_ld32_nowait(tAcc1 + lane_off + (uint32_t)(part * CW), v1);
        tmem_ld_wait32(v0);
        if (MODE == 0) tmem_ld_wait32(v1);
      } else {
        tmem_ld16_nowait(tAcc0 + lane_off + (uint32_t)(part * CW), v0);
        if (MODE == 0) tmem_ld16_nowait(tAcc1 + lane_off + (uint32_t)(part * CW), v1);
        tmem_ld_wait16(v0);
        if (MODE == 0) tmem_ld_wait16(v1);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_free);               // the next item may overwrite the accumulators
      // dS-fed accumulator, scaled: dK -> column block d (MODE 0) or dQ -> column block 0 (MODE 1); dV -> block 2d.
      // A thread that stored its own row would put 16 bytes into each of 32 lines per instruction, and the store path
      // charges per line.  So the warp parks its 32 rows x CW columns in shared memory, in the 16-byte chunks of the
      // dS (and P) tile of its group that only this warp ever writes (rows r, chunks 4 hc ..): every product that read
      // them is finished (acc_done), and their next writer is this warp, after this block.  It then writes them back
      // with NSEG consecutive lanes on the NSEG segments of a row, 32 / NSEG rows per instruction.
      {
        constexpr int NSEG = CW / 8;                      // 16-byte segments per row: 4 (d_h 128) or 2 (d_h 64)
        constexpr int RPI = 32 / NSEG;                    // rows per store instruction
        uint8_t* tile0 = p_gen + pb * NP * Cfg::kPBytes;  // dS tile of this group; the P tile follows it (MODE 0)
        uint8_t* mine = tile0 + r * 128;
#pragma unroll
        for (int sgm = 0; sgm < NSEG; ++sgm) {
          uint4 pk;
          __nv_bfloat162* hp = reinterpret_cast<__nv_bfloat162*>(&pk);
#pragma unroll
          for (int e = 0; e < 4; ++e)
            hp[e] = __floats2bfloat162_rn(__uint_as_float(v0[8 * sgm + 2 * e]) * scale, __uint_as_float(v0[8 * sgm + 2 * e + 1]) * scale);
          *reinterpret_cast<uint4*>(mine + (((hc * 4 + sgm) ^ (r & 7)) << 4)) = pk;
          if (MODE == 0) {
#pragma unroll
            for (int e = 0; e < 4; ++e)
              hp[e] = __floats2bfloat162_rn(__uint_as_float(v1[8 * sgm + 2 * e]), __uint_as_float(v1[8 * sgm + 2 * e + 1]));
            *reinterpret_cast<uint4*>(mine + Cfg::kPBytes + (((hc * 4 + sgm) ^ (r & 7)) << 4)) = pk;
          }
        }
        __syncwarp();
        const int sgm = lane % NSEG;
        __nv_bfloat16* obase = dqkv + (int64_t)it.h * DH + part * CW + 8 * sgm;
#pragma unroll
        for (int i = 0; i < NSEG; ++i) {
          const int rr = q * 32 + i * RPI + lane / NSEG;  // row of the fixed tile
          const uint8_t* src = tile0 + rr * 128 + (((hc * 4 + sgm) ^ (rr & 7)) << 4);
          const uint4 a0 = *reinterpret_cast<const uint4*>(src);
          uint4 a1 = a0;
          if (MODE == 0) a1 = *reinterpret_cast<const uint4*>(src + Cfg::kPBytes);
          if (f0 + rr < S) {
            __nv_bfloat16* orow = obase + ((int64_t)(row_g0 + f0 + rr)) * (3 * d);
            *reinterpret_cast<uint4*>(orow + (MODE == 0 ? d : 0)) = a0;
            if (MODE == 0) *reinterpret_cast<uint4*>(orow + 2 * d) = a1;
          }
        }
        __syncwarp();
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
