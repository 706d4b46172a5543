// Attention forward on tcgen05: scores and the output accumulator live in tensor memory.
// Included into gemm_tc.cu (inside its unnamed namespace) so that it shares the PTX wrappers,
// the bounded mbarrier waits, the time-out flag and the tensor-map cache.
//
// Work item = one (batch, head) and 128 query rows; key blocks of 128.  The kernel is persistent:
// a CTA walks a list of items, those with the most key blocks first; the next item's Q tile and
// first scores are ready when an item ends (two Q buffers, two score buffers, two output
// accumulators), and an item's normalisation and store are put off until the softmax warps hold
// the next item's first exponentials, so that they never wait for the item's last P V product.
//   warp 0    : TMA producer (Q per item; K and V blocks through two 2-deep rings)
//   warp 1    : issues S_j = Q K_j^T   (M 128 x N 128, k = d_h)      -> TMEM columns [0,128) / [128,256); owns the tensor memory
//   warp 2    : issues O += P_j V_j    (M 128 x N d_h, k = 128 keys) -> TMEM columns [256,384) / [384,512) by item parity
//   warps 3-10: softmax, two threads per query row (= one tensor-memory lane; warps w and w + 4 share
//               a lane quarter and take 64 of the block's 128 columns each): read S_j, mask, running
//               max / sum, write P_j as bf16 into a 128-byte-swizzled shared tile (the A operand of
//               the second product), rescale their half of O's columns in tensor memory when the
//               reference maximum moved, and at the end normalise and store O and the log-sum-exp.
//               The two threads of a row agree on the block maximum (and at the end on the sum)
//               through a 1 KB exchange in shared memory and a named barrier of their two warps.
// Q and K are K-major operands (d_h contiguous), V is an N-major operand (B(k = key, n = e) =
// V[key][e]): all three are read straight out of qkv[T, 3d] by one tensor map, nothing is copied
// or transposed.  Rows of a tile that lie beyond this batch entry's sequence hold the next
// entry's (finite) values or TMA zero fill; their scores are masked, their probabilities are 0.
#pragma once

constexpr int kAttThreads = 352;
constexpr int kAttBQ = 128, kAttBK = 128;

template <int DH> struct AttnTcCfg {
  static constexpr int kSpans = DH / 64;                       // 64-column swizzle spans per row
  static constexpr int kTileBytes = 128 * DH * 2;              // one Q / K / V tile
  static constexpr int kPBytes = 128 * kAttBK * 2;             // P tile: 128 rows x 128 keys
  static constexpr int kSmem = 6 * kTileBytes + kPBytes + 1024 + 256 + 1024;      // Q x 2, K x 2, V x 2, P, row exchange
};

__device__ __forceinline__ void tmem_st32(uint32_t addr, const uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(addr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
        "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]),
        "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]),
        "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// descriptor of a K-major tile with rows of 64 elements (one span), 128-byte swizzle
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFF) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// descriptor of an N-major operand staged as [k rows][64] boxes that are `box_bytes` apart along N
__device__ __forceinline__ uint64_t desc_nmajor(uint32_t saddr, uint32_t box_bytes) {
  return (uint64_t)((saddr & 0x3FFFF) >> 4) | ((uint64_t)(box_bytes >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}

// A warp's 32 rows x 64 bf16 columns (lane = row) written as whole 128-byte lines: parked in 4 KB of shared memory
// (16-byte segments XOR-swizzled by row, conflict-free both ways) and written back with eight consecutive lanes on the
// eight segments of a row, four rows per instruction.  att_stage32 parks 32 of the lane's fp32 values (times `mul`) as
// segments seg0 .. seg0 + 3 of its row; att_flush64 writes the rows out, skipping rows at or beyond row_end.
__device__ __forceinline__ void att_stage32(const uint32_t (&v)[32], float mul, uint8_t* __restrict__ stage, int lane, int seg0) {
  uint8_t* mine = stage + lane * 128;
#pragma unroll
  for (int sg = 0; sg < 4; ++sg) {
    uint4 pk;
    __nv_bfloat162* hp = reinterpret_cast<__nv_bfloat162*>(&pk);
#pragma unroll
    for (int t = 0; t < 4; ++t)
      hp[t] = __floats2bfloat162_rn(__uint_as_float(v[8 * sg + 2 * t]) * mul, __uint_as_float(v[8 * sg + 2 * t + 1]) * mul);
    *reinterpret_cast<uint4*>(mine + (((seg0 + sg) ^ (lane & 7)) << 4)) = pk;
  }
}
__device__ __forceinline__ void att_flush64(const uint8_t* __restrict__ stage, __nv_bfloat16* __restrict__ dst, int64_t ld, int row,
                                            int lane, int row_end, int col) {
  __syncwarp();
  const int row_base = row - lane, sg = lane & 7;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int r = 4 * i + (lane >> 3);
    const uint4 v = *reinterpret_cast<const uint4*>(stage + r * 128 + ((sg ^ (r & 7)) << 4));
    if (row_base + r < row_end) *reinterpret_cast<uint4*>(dst + (int64_t)(row_base + r) * ld + col + 8 * sg) = v;
  }
  __syncwarp();
}

// Key padding: batch entry b attends to keys 0 .. lens[b]-1 only (clamped to [1, S]); null = all S keys.
__device__ __forceinline__ int tc_key_len(const int* __restrict__ lens, int b, int S) {
  return lens != nullptr ? max(1, min(lens[b], S)) : S;
}

// DROP: dropout on the probabilities (its own instance, so that the plain kernel carries none of the generator's code)
template <int DH, bool DROP>
__global__ void __launch_bounds__(kAttThreads, 1)
attn_fwd_tc_kernel(const __grid_constant__ CUtensorMap tmap_qkv, __nv_bfloat16* __restrict__ o,
                   float* __restrict__ lse, int B, int S, int H, int causal, float scale,
                   const int* __restrict__ lens, DropArgs da) {
  typedef AttnTcCfg<DH> Cfg;
  constexpr int SP = Cfg::kSpans;
  constexpr int SPAN_BYTES = 128 * 128;                 // 128 rows x 64 elements x 2 bytes
  extern __shared__ uint8_t smem_raw[];
  const int d = H * DH;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sQ = base;                             // two buffers (item parity)
  const uint32_t sK = sQ + 2 * Cfg::kTileBytes;         // two stages
  const uint32_t sV = sK + 2 * Cfg::kTileBytes;         // two stages
  const uint32_t sP = sV + 2 * Cfg::kTileBytes;
  const uint32_t bar = sP + Cfg::kPBytes;
  auto q_full = [&](int i) { return bar + 8u * i; };
  auto q_empty = [&](int i) { return bar + 16u + 8u * i; };
  auto k_full = [&](int i) { return bar + 32u + 8u * i; };
  auto k_empty = [&](int i) { return bar + 48u + 8u * i; };
  auto v_full = [&](int i) { return bar + 64u + 8u * i; };
  auto v_empty = [&](int i) { return bar + 80u + 8u * i; };
  auto s_full = [&](int i) { return bar + 96u + 8u * i; };
  auto s_free = [&](int i) { return bar + 112u + 8u * i; };
  auto o_done = [&](int i) { return bar + 128u + 8u * i; };
  auto o_free = [&](int i) { return bar + 144u + 8u * i; };
  const uint32_t p_ready = bar + 160u, p_free = bar + 168u, tmem_slot = bar + 176u;
  float* xch = reinterpret_cast<float*>(smem_raw + (bar + 256u - smem_u32(smem_raw)));       // [128 rows][2 halves]
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot_gen = reinterpret_cast<volatile uint32_t*>(gen + (tmem_slot - base));
  uint8_t* p_gen = gen + (sP - base);

  // work items, heaviest first; every role walks the same list and counts key blocks (g)
  const int nqb = (S + kAttBQ - 1) / kAttBQ, nbh = B * H, nitems = nqb * nbh;
  struct Item { int b, h, q0, nblk, klen; };
  // item indices stay far below 2^24, so a float reciprocal and one correction step divide exactly (an integer
  // division by a run-time value costs a few hundred cycles of the softmax warps at every item boundary)
  auto div_small = [](int x, int dv) {
    int qt = (int)((float)x * __frcp_rn((float)dv));
    if (qt * dv > x) --qt;
    else if ((qt + 1) * dv <= x) ++qt;
    return qt;
  };
  auto item_of = [&](int idx) {
    Item it;
    const int rank = div_small(idx, nbh), bh = idx - rank * nbh;
    it.b = div_small(bh, H);
    it.h = bh - it.b * H;
    it.q0 = (causal ? nqb - 1 - rank : rank) * kAttBQ;
    it.klen = tc_key_len(lens, it.b, S);                // keys at or after klen are padding
    const int kv_len = min(causal ? min(S, it.q0 + kAttBQ) : S, it.klen);
    it.nblk = (kv_len + kAttBK - 1) / kAttBK;
    return it;
  };
  // The n-th item of this CTA.  The list is sorted by weight, so handing it out forwards on even rounds and backwards
  // on odd ones pairs a CTA's heavy items with light ones (plain round-robin gave the first CTAs the heaviest item of
  // every round: 10 key blocks against a mean of 8.65 at batch 4 x 512 x 32 heads, causal).
  auto item_at = [&](int n) {
    const int first = n * (int)gridDim.x;
    return (n & 1) ? first + (int)gridDim.x - 1 - (int)blockIdx.x : first + (int)blockIdx.x;
  };
  // one thread reads the time-out flag and the CTA shares the answer: the softmax warps meet at named
  // barriers in pairs, so they must all take the same way
  volatile uint32_t* poison_gen = reinterpret_cast<volatile uint32_t*>(gen + (tmem_slot + 8u - base));

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(q_full(i), 1); mbar_init(q_empty(i), 1);
      mbar_init(k_full(i), 1); mbar_init(k_empty(i), 1);
      mbar_init(v_full(i), 1); mbar_init(v_empty(i), 1);
      mbar_init(s_full(i), 1); mbar_init(s_free(i), 8);
      mbar_init(o_done(i), 1); mbar_init(o_free(i), 8);
    }
    mbar_init(p_ready, 8);                              // one arrival per softmax warp
    mbar_init(p_free, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    pdl_wait();                                         // no global access before it, the flag included
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

  if (warp == 0) {
    // ---------------- TMA producer
    if (lane == 0 && !poisoned) {
      int g = 0, n = 0;
      bool ok = true;
      for (int idx = item_at(n); idx < nitems && ok; idx = item_at(++n)) {
        const Item it = item_of(idx);
        const int row_g0 = it.b * S;                    // first row of this batch entry in qkv
        const int colQ = it.h * DH, colK = d + it.h * DH, colV = 2 * d + it.h * DH;
        const int qi = n & 1;
        if (!mbar_wait(q_empty(qi), (uint32_t)(((n >> 1) & 1) ^ 1))) { atomicCAS(&g_tc_error, 0, 4); break; }
        mbar_expect_tx(q_full(qi), Cfg::kTileBytes);
#pragma unroll
        for (int sp = 0; sp < SP; ++sp) tma_load_2d(sQ + qi * Cfg::kTileBytes + sp * SPAN_BYTES, &tmap_qkv, q_full(qi), colQ + sp * 64, row_g0 + it.q0);
        for (int j = 0; j < it.nblk; ++j, ++g) {
          const int st = g & 1;
          const uint32_t ph = (uint32_t)((g >> 1) & 1);
          const int krow = row_g0 + j * kAttBK;
          if (!mbar_wait(k_empty(st), ph ^ 1)) { atomicCAS(&g_tc_error, 0, 4); ok = false; break; }
          mbar_expect_tx(k_full(st), Cfg::kTileBytes);
#pragma unroll
          for (int sp = 0; sp < SP; ++sp)
            tma_load_2d(sK + st * Cfg::kTileBytes + sp * SPAN_BYTES, &tmap_qkv, k_full(st), colK + sp * 64, krow);
          if (!mbar_wait(v_empty(st), ph ^ 1)) { atomicCAS(&g_tc_error, 0, 4); ok = false; break; }
          mbar_expect_tx(v_full(st), Cfg::kTileBytes);
#pragma unroll
          for (int sp = 0; sp < SP; ++sp)
            tma_load_2d(sV + st * Cfg::kTileBytes + sp * SPAN_BYTES, &tmap_qkv, v_full(st), colV + sp * 64, krow);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer 1: scores.  A = Q (K-major), B = K (K-major), N = 128; runs ahead of the
    //                  softmax warps as far as the two score buffers allow, into the next item too
    if (lane == 0 && !poisoned) {
      const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kAttBK >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
      int g = 0, n = 0;
      bool ok = true;
      for (int idx = item_at(n); idx < nitems && ok; idx = item_at(++n)) {
        const Item it = item_of(idx);
        const int qi = n & 1;
        if (!mbar_wait(q_full(qi), (uint32_t)((n >> 1) & 1))) { atomicCAS(&g_tc_error, 0, 5); break; }
        const uint64_t dQ = desc_kmajor(sQ + qi * Cfg::kTileBytes);
        for (int j = 0; j < it.nblk; ++j, ++g) {
          const int st = g & 1;
          const uint32_t ph = (uint32_t)((g >> 1) & 1);
          if (!mbar_wait(k_full(st), ph) || !mbar_wait(s_free(st), ph ^ 1)) { atomicCAS(&g_tc_error, 0, 5); ok = false; break; }
          tc_fence_after();
          const uint64_t dK = desc_kmajor(sK + st * Cfg::kTileBytes);
          const uint32_t ts = tmem_base + (uint32_t)(st * 128);
#pragma unroll
          for (int kk = 0; kk < DH / 16; ++kk) {
            const uint64_t off = (uint64_t)(((kk / 4) * SPAN_BYTES + (kk % 4) * 32) >> 4);
            tc_mma(ts, dQ + off, dK + off, idesc_s, kk > 0 ? 1u : 0u);
          }
          tc_commit(s_full(st));
          tc_commit(k_empty(st));
        }
        if (ok) tc_commit(q_empty(qi));
      }
    }
  } else if (warp == 2) {
    // ---------------- MMA issuer 2: O += P V.  A = P (K-major), B = V (N-major), N = DH
    if (lane == 0 && !poisoned) {
      const uint32_t idesc_o = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(DH >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
      int g = 0, n = 0;
      bool ok = true;
      for (int idx = item_at(n); idx < nitems && ok; idx = item_at(++n)) {
        const Item it = item_of(idx);
        const uint32_t tO = tmem_base + 256u + (uint32_t)((n & 1) * 128);
        for (int j = 0; j < it.nblk; ++j, ++g) {
          const int st = g & 1;
          if (!mbar_wait(p_ready, (uint32_t)(g & 1)) || !mbar_wait(v_full(st), (uint32_t)((g >> 1) & 1))) {
            atomicCAS(&g_tc_error, 0, 5); ok = false; break;
          }
          // the first product of an item overwrites its accumulator: the item two before must have been stored
          if (j == 0 && n >= 2 && !mbar_wait(o_free(n & 1), (uint32_t)(((n >> 1) - 1) & 1))) { atomicCAS(&g_tc_error, 0, 5); ok = false; break; }
          tc_fence_after();
          const uint64_t dP = desc_kmajor(sP), dV = desc_nmajor(sV + st * Cfg::kTileBytes, SPAN_BYTES);
#pragma unroll
          for (int kk = 0; kk < kAttBK / 16; ++kk) {
            // P: 128 keys = two 64-key spans, 32 bytes per 16 keys inside a span; V: 16 key rows of 128 bytes
            tc_mma(tO, dP + (uint64_t)(((kk / 4) * SPAN_BYTES + (kk % 4) * 32) >> 4), dV + (uint64_t)((kk * 16 * 128) >> 4), idesc_o,
                   (j > 0 || kk > 0) ? 1u : 0u);
          }
          tc_commit(p_free);
          tc_commit(v_empty(st));
        }
        if (ok) tc_commit(o_done(n & 1));
      }
    }
  } else {
    // ---------------- softmax and epilogue: two threads per query row (= tensor-memory lane)
    const int q = warp & 3;                             // lane quarter; warps w and w + 4 share it
    const int half = (warp - 3) >> 2;                   // which 64 of the block's 128 columns, which half of O's columns
    const int r = q * 32 + lane;                        // row inside the tile
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    const float sl2 = scale * 1.4426950408889634f;
    constexpr int HB = kAttBK / 2, OC = DH / 2;
    auto pair_sync = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(1 + q) : "memory"); };
    // a warp that gives up on a bounded wait must not leave its partner at the named barrier: it arrives (without
    // waiting) for every meeting the partner can still reach before its own next bounded wait ends it
    auto pair_release = [&]() {
#pragma unroll 1
      for (int i = 0; i < 4; ++i) asm volatile("bar.arrive %0, 64;" ::"r"(1 + q) : "memory");
    };
    bool ok = !poisoned;
    int g = 0, n = 0;
    // The normalisation and store of an item wait for its last P V product, so they are put off until this thread
    // has the exponentials of the next item's first block in registers: by then the product is long finished, and the
    // P tile (this warp's rows of it are the staging area of the stores) has not been written for the new item yet.
    int pend_n = -1, pend_row = 0, pend_end = 0, pend_col = 0;      // pend_n < 0: nothing put off
    float pend_inv = 0.f;
    // Whole-line stores: the warp parks each 32 x 32 chunk in shared memory and writes it back with consecutive
    // lanes on consecutive 16-byte segments of a row (its own 32 rows of its 64-key span of the P tile: 4 KB).
    auto finish_item = [&]() -> bool {
      const bool ready = mbar_wait(o_done(pend_n & 1), (uint32_t)((pend_n >> 1) & 1));
      if (!ready && lane == 0) atomicCAS(&g_tc_error, 0, 6);
      tc_fence_after();
      if (!__all_sync(0xffffffffu, ready)) return false;
      const uint32_t tOp = tmem_base + 256u + (uint32_t)((pend_n & 1) * 128);
      uint8_t* stage = p_gen + half * SPAN_BYTES + (q * 32) * 128;
      if constexpr (OC == 64) {
        uint32_t v[32];
        tmem_ld32(tOp + lane_off + (uint32_t)(half * OC), v);
        att_stage32(v, pend_inv, stage, lane, 0);
        tmem_ld32(tOp + lane_off + (uint32_t)(half * OC + 32), v);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(o_free(pend_n & 1));   // everything read: the accumulator may be reused
        att_stage32(v, pend_inv, stage, lane, 4);
        att_flush64(stage, o, (int64_t)d, pend_row, lane, pend_end, pend_col);
      } else {
        uint32_t v[32];
        tmem_ld32(tOp + lane_off + (uint32_t)(half * OC), v);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(o_free(pend_n & 1));
        float f[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) f[i] = __uint_as_float(v[i]) * pend_inv;
        // rows at or beyond the batch entry's sequence end are skipped
        epi_store32_lines<false>(f, stage, o, (int64_t)d, pend_row, lane, pend_end, pend_col, nullptr);
      }
      pend_n = -1;
      return true;
    };
    for (int idx = item_at(n); idx < nitems && ok; idx = item_at(++n)) {
      const Item it = item_of(idx);
      const int q0 = it.q0, qrow = q0 + r, row_g0 = it.b * S, klen = it.klen;
      const uint32_t tO = tmem_base + 256u + (uint32_t)((n & 1) * 128);
      float m = -INFINITY, l = 0.f;                     // m: the row's reference maximum (same in both threads); l: this half's sum
      for (int j = 0; j < it.nblk; ++j, ++g) {
        const int st = g & 1;
        bool ready = mbar_wait(s_full(st), (uint32_t)((g >> 1) & 1));
        if (!ready && lane == 0) atomicCAS(&g_tc_error, 0, 6);
        tc_fence_after();
        ok = __all_sync(0xffffffffu, ready);
        if (!ok) { pair_release(); break; }
        // this thread's 64 scores of the row (raw; the scale is folded into the exponent below)
        float sc[HB];
#pragma unroll
        for (int c0 = 0; c0 < HB; c0 += 32) {
          uint32_t v[32];
          tmem_ld32(tmem_base + lane_off + (uint32_t)(st * 128 + half * HB + c0), v);
#pragma unroll
          for (int i = 0; i < 32; ++i) sc[c0 + i] = __uint_as_float(v[i]);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(s_free(st));         // the tensor core may overwrite this score buffer
        // masking only where the block touches the diagonal or the end of the sequence (uniform per CTA)
        if ((causal && j * kAttBK + kAttBK - 1 > q0) || (j + 1) * kAttBK > klen) {
#pragma unroll
          for (int i = 0; i < HB; ++i) {
            const int key = j * kAttBK + half * HB + i;
            if (key >= klen || (causal && key > qrow)) sc[i] = -INFINITY;
          }
        }
        // four independent chains each for the maximum and the sum
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int i = 0; i < HB; i += 4) {
#pragma unroll
          for (int e = 0; e < 4; ++e) mx4[e] = fmaxf(mx4[e], sc[i + e]);
        }
        float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * sl2;     // in log2 units (scale > 0)
        // the row's block maximum = the larger of the two halves'
        xch[r * 2 + half] = mx;
        pair_sync();
        mx = fmaxf(mx, xch[r * 2 + (half ^ 1)]);
        pair_sync();
        // Lazy reference maximum: m moves (and O is rescaled) only when some row of the warp has grown by
        // more than 2^8 over it; until then probabilities up to 256 are summed against the old reference,
        // which changes nothing in the final O / l and lse = m + log2(l).  Both warps of a quarter see the
        // same m and mx per row, so they take the same decision.
        const bool grow = __any_sync(0xffffffffu, mx > m + 8.0f);
        float corr = 1.0f;
        if (grow) {
          const float mnew = fmaxf(m, mx);
          corr = (mnew == -INFINITY) ? 1.0f : ex2_approx(m - mnew);    // m = -inf: corr = 0, nothing accumulated yet
          m = mnew;
        }
        const float nmuse = (m == -INFINITY) ? 0.f : -m;
        float sum4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int i = 0; i < HB; i += 4) {
#pragma unroll
          for (int e = 0; e < 4; ++e) { sc[i + e] = ex2_approx(fmaf(sc[i + e], sl2, nmuse)); sum4[e] += sc[i + e]; }
        }
        l = l * corr + ((sum4[0] + sum4[1]) + (sum4[2] + sum4[3]));
        // dropout on the probabilities (uniform across the CTA): the sum above runs over all of them, the product with
        // V over the kept ones; 1 / (1 - p) goes into the final scaling.  One generator block per four keys.
        if (DROP) {
          const int bh = it.b * H + it.h, qd = min(qrow, S - 1), kfirst = j * kAttBK + half * HB;
#pragma unroll
          for (int i = 0; i < HB; i += 4) {
            const uint4 w = attn_drop_words(da, bh, S, qd, kfirst + i);
            if (w.x < da.thr) sc[i] = 0.f;
            if (w.y < da.thr) sc[i + 1] = 0.f;
            if (w.z < da.thr) sc[i + 2] = 0.f;
            if (w.w < da.thr) sc[i + 3] = 0.f;
          }
        }
        if (pend_n >= 0) {                              // the previous item's output (uniform across the CTA)
          ok = finish_item();
          if (!ok) { pair_release(); break; }
        }
        // the previous P V product must be finished before P is overwritten and O is rescaled
        ready = mbar_wait(p_free, (uint32_t)((g & 1) ^ 1));
        if (!ready && lane == 0) atomicCAS(&g_tc_error, 0, 6);
        tc_fence_after();
        ok = __all_sync(0xffffffffu, ready);
        if (!ok) { pair_release(); break; }
        // this half of the P row -> shared memory, bf16: one 64-key span of the K-major, 128-byte-swizzled tile
#pragma unroll
        for (int c = 0; c < HB / 8; ++c) {
          uint4 pk;
          __nv_bfloat162* hp = reinterpret_cast<__nv_bfloat162*>(&pk);
#pragma unroll
          for (int t = 0; t < 4; ++t) hp[t] = __floats2bfloat162_rn(sc[c * 8 + 2 * t], sc[c * 8 + 2 * t + 1]);
          *reinterpret_cast<uint4*>(p_gen + half * SPAN_BYTES + r * 128 + ((c ^ (r & 7)) << 4)) = pk;
        }
        if (j > 0 && grow) {                            // warp-uniform; this thread's half of O's columns
#pragma unroll 1
          for (int c0 = 0; c0 < OC; c0 += 32) {
            uint32_t v[32];
            tmem_ld32(tO + lane_off + (uint32_t)(half * OC + c0), v);
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * corr);
            tmem_st32(tO + lane_off + (uint32_t)(half * OC + c0), v);
          }
          tmem_st_wait();
        }
        fence_async_smem();                             // P is read by the tensor core (async proxy)
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(p_ready);
      }
      if (!ok) break;
      // the row's sum = the two halves' (both relative to the same m)
      xch[r * 2 + half] = l;
      pair_sync();
      const float ltot = l + xch[r * 2 + (half ^ 1)];
      pair_sync();
      if (half == 0 && qrow < S) lse[((int64_t)it.b * H + it.h) * S + qrow] = (m + log2f(ltot)) * 0.6931471805599453f;
      pend_n = n;
      pend_inv = (DROP ? da.scale : 1.0f) / ltot;
      pend_row = row_g0 + qrow;
      pend_end = row_g0 + S;
      pend_col = it.h * DH + half * OC;
    }
    if (ok && pend_n >= 0) finish_item();                      // the last item of this CTA
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}
