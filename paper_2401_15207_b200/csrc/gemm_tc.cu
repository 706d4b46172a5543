// bf16 GEMM on the Blackwell tensor cores: tcgen05.mma with the accumulator in tensor memory,
// operands staged in shared memory by TMA (no cluster multicast), an mbarrier ring between a
// one-thread TMA producer, a one-thread MMA issuer and four epilogue warps.  The kernel is
// persistent (one CTA per SM) with two accumulators, so epilogues overlap the next tile's MMAs.
//
//   C[m,n] = sum_k A(m,k) * B(k,n) (+ bias[n]) (+ residual[m,n])
//
// The three linear-layer products of the training step differ only in which operand dimension
// is contiguous in memory, and the tensor core takes both:
//   forward  y  = x w^T : A K-major  (x[m,k]),   B K-major  (w[n,k])
//   dX       dx = dy w  : A K-major  (dy[m,k']), B N-major  (w[k',n])
//   dW       dw = dy^T x: A M-major  (dy[k',m]), B N-major  (x[k',n])
// so no operand is ever transposed or copied.  "MN-major" tiles are loaded as 64-element-wide
// TMA boxes (one 128-byte swizzle span along M or N) and described to the MMA with the
// matching shared-memory descriptor (leading-dimension offset = distance between boxes).
//
// Every wait on an mbarrier is bounded: after about a second it records an error code in
// g_tc_error, and the kernel drains and releases its tensor memory normally.
#include "gemm_tc.h"

#include <cuda.h>
#include <cuda_bf16.h>
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>
#include <unordered_map>

namespace hift {

namespace {

constexpr int BM = 128;          // rows of the output tile = MMA M
constexpr int BK = 64;           // k elements per pipeline stage = one 128-byte swizzle span
constexpr int UMMA_K = 16;       // k elements per tcgen05.mma (bf16)
constexpr int kThreads = 192;    // warp 0: TMA, warp 1: MMA + tensor-memory owner, warps 2-5: epilogue
constexpr long long kWaitCycles = 4000000000ll;   // ~2 s at 2 GHz

__device__ int g_tc_error = 0;   // 0 ok; 1 producer, 2 MMA issuer, 3 epilogue gave up waiting

// Tile width BN is a run-time multiple of 32 in [64, 256] (MMA N), chosen per problem so that the
// grid fills whole rounds of SMs.  Shared memory per stage: A 128 x 64 bf16 (16 KB) plus B, which is
// BN x 64 bf16 when K-major and ceil(BN/64) boxes of 64 x 64 when N-major.
constexpr int kABytes = BM * BK * 2;
constexpr int kSmemBudget = 196608;                 // operand ring
constexpr int kStoreStage = 4096;                   // per epilogue warp: one 32 x 32 fp32 chunk on its way to global memory
constexpr int kSmemBytes = kSmemBudget + 1024 /*alignment slack*/ + 256 /*barriers*/ + 4 * kStoreStage;
constexpr int kMaxStages = 8;
constexpr int kAccStride = 256;                     // tensor-memory columns between the two accumulators
struct TileRt { int bn, b_bytes, stage_bytes, stages; };
inline TileRt make_tile(int bn, bool b_mn) {
  TileRt t;
  t.bn = bn;
  t.b_bytes = b_mn ? ((bn + 63) / 64) * (BK * 128) : bn * BK * 2;
  t.stage_bytes = kABytes + t.b_bytes;
  t.stages = kSmemBudget / t.stage_bytes;
  if (t.stages > kMaxStages) t.stages = kMaxStages;
  return t;
}

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok;
}
// Bounded wait: false if the phase did not complete within kWaitCycles.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (clock64() - t0 > kWaitCycles) return false;
  }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"((uint64_t)map), "r"(bar), "r"(x), "r"(y) : "memory");
}
// Programmatic dependent launch: a kernel launched with the stream-serialisation attribute may start while
// its predecessor in the stream is still draining; pdl_wait() returns once the predecessor has completed and
// its writes are visible, and nothing before it may touch global data.  pdl_trigger() lets the successor of
// this kernel be scheduled as soon as every CTA has passed it (or exited).
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t tmem_c, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_c), "l"(da), "l"(db), "r"(idesc), "r"(accum) : "memory");
}
// 32 consecutive accumulator columns of this thread's lane.  The load is asynchronous: its registers
// may be read only after tmem_ld_wait32, which names them as in/out operands so that no use can be
// scheduled ahead of the wait.  (The wait covers every load this thread has issued so far.)
__device__ __forceinline__ void tmem_ld32_nowait(uint32_t addr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(addr));
}
__device__ __forceinline__ void tmem_ld_wait32(uint32_t (&v)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),
                 "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15]),
                 "+r"(v[16]), "+r"(v[17]), "+r"(v[18]), "+r"(v[19]), "+r"(v[20]), "+r"(v[21]), "+r"(v[22]), "+r"(v[23]),
                 "+r"(v[24]), "+r"(v[25]), "+r"(v[26]), "+r"(v[27]), "+r"(v[28]), "+r"(v[29]), "+r"(v[30]), "+r"(v[31])
               :: "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t addr, uint32_t (&v)[32]) {
  tmem_ld32_nowait(addr, v);
  tmem_ld_wait32(v);
}

// Shared-memory matrix descriptor, 128-byte swizzle.  Fields in 16-byte units: start address
// bits [0,14), leading-dimension byte offset [16,30), stride-dimension byte offset [32,46),
// descriptor version 1 at [46,48), swizzle mode (2 = 128 B) at [61,64).
//   K-major tile  [rows][64]: 8-row groups are 1024 B apart (stride offset); leading offset unused.
//   MN-major tile [k][64] boxes: 8-k groups are 1024 B apart (stride offset); the next 64-wide box
//   along M/N is BK*128 B further (leading offset).
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, bool mn_major) {
  const uint64_t lbo = mn_major ? (uint64_t)((BK * 128) >> 4) : 1ull;
  const uint64_t sbo = 1024 >> 4;
  return (uint64_t)((saddr & 0x3FFFF) >> 4) | (lbo << 16) | (sbo << 32) | (1ull << 46) | (2ull << 61);
}

// ------------------------------------------------------------------ epilogue pieces
struct RopeArgs { const float* cs; int seq; int64_t cols; };   // head size 128; cs == nullptr: none

// 32 consecutive outputs of row m starting at column n: bias, residual, conversion, store.
// FULL: the caller knows that all 32 columns exist.
template <bool OUT_F32, bool FULL>
__device__ __forceinline__ void epi_store32(float (&f)[32], void* __restrict__ cptr, int64_t ldc, int m, int n, int N,
                                            const __nv_bfloat16* __restrict__ bias, const float* __restrict__ residual,
                                            int64_t ldr) {
  if (FULL || n + 32 <= N) {
    if (bias) {
#pragma unroll
      for (int j = 0; j < 32; j += 8) {
        const uint4 b4 = *reinterpret_cast<const uint4*>(bias + n + j);
        const __nv_bfloat162* hb = reinterpret_cast<const __nv_bfloat162*>(&b4);
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          const float2 bf = __bfloat1622float2(hb[t]);
          f[j + 2 * t] += bf.x; f[j + 2 * t + 1] += bf.y;
        }
      }
    }
    if (OUT_F32) {
      float* crow = reinterpret_cast<float*>(cptr) + (int64_t)m * ldc + n;
      if (residual) {
        const float* rrow = residual + (int64_t)m * ldr + n;
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
          const float4 r = *reinterpret_cast<const float4*>(rrow + j);
          f[j] += r.x; f[j + 1] += r.y; f[j + 2] += r.z; f[j + 3] += r.w;
        }
      }
#pragma unroll
      for (int j = 0; j < 32; j += 4)
        *reinterpret_cast<float4*>(crow + j) = make_float4(f[j], f[j + 1], f[j + 2], f[j + 3]);
    } else {
      __nv_bfloat16* crow = reinterpret_cast<__nv_bfloat16*>(cptr) + (int64_t)m * ldc + n;
#pragma unroll
      for (int j = 0; j < 32; j += 8) {
        uint4 o;
        __nv_bfloat162* ho = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
        for (int t = 0; t < 4; ++t) ho[t] = __floats2bfloat162_rn(f[j + 2 * t], f[j + 2 * t + 1]);
        *reinterpret_cast<uint4*>(crow + j) = o;
      }
    }
  } else if (!FULL) {
    for (int j = 0; j < 32 && n + j < N; ++j) {     // ragged right edge
      float x = f[j];
      if (bias) x += __bfloat162float(bias[n + j]);
      if (OUT_F32) {
        if (residual) x += residual[(int64_t)m * ldr + n + j];
        reinterpret_cast<float*>(cptr)[(int64_t)m * ldc + n + j] = x;
      } else {
        reinterpret_cast<__nv_bfloat16*>(cptr)[(int64_t)m * ldc + n + j] = __float2bfloat16_rn(x);
      }
    }
  }
}

// The same 32 x 32 chunk of a warp (lane = row), written as whole lines.  A thread that stores its own row puts
// 16 bytes into each of 32 different lines per instruction, and the store path charges per line touched, not per
// byte: on short-K products that was what a tile waited for.  Here the warp parks the chunk in its 4 KB of shared
// memory (16-byte segments XOR-swizzled so that neither side has bank conflicts) and writes it back with
// consecutive lanes on consecutive segments of a row: 8 rows x 64 bytes (bf16) or 4 rows x 128 bytes (fp32) per
// instruction.  Only for chunks whose 32 columns all exist; `m` is this lane's row, rows at or beyond M are skipped.
template <bool OUT_F32>
__device__ __forceinline__ void epi_store32_lines(float (&f)[32], uint8_t* __restrict__ stage, void* __restrict__ cptr, int64_t ldc,
                                                  int m, int lane, int M, int n, const __nv_bfloat16* __restrict__ bias) {
  if (bias) {
#pragma unroll
    for (int j = 0; j < 32; j += 8) {
      const uint4 b4 = *reinterpret_cast<const uint4*>(bias + n + j);
      const __nv_bfloat162* hb = reinterpret_cast<const __nv_bfloat162*>(&b4);
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const float2 bf = __bfloat1622float2(hb[t]);
        f[j + 2 * t] += bf.x; f[j + 2 * t + 1] += bf.y;
      }
    }
  }
  const int row_base = m - lane;
  if (OUT_F32) {
    uint8_t* mine = stage + lane * 128;
#pragma unroll
    for (int sg = 0; sg < 8; ++sg)
      *reinterpret_cast<float4*>(mine + ((sg ^ (lane & 7)) << 4)) = make_float4(f[4 * sg], f[4 * sg + 1], f[4 * sg + 2], f[4 * sg + 3]);
    __syncwarp();
    const int sg = lane & 7;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int r = 4 * i + (lane >> 3);
      const float4 v = *reinterpret_cast<const float4*>(stage + r * 128 + ((sg ^ (r & 7)) << 4));
      if (row_base + r < M) *reinterpret_cast<float4*>(reinterpret_cast<float*>(cptr) + (int64_t)(row_base + r) * ldc + n + 4 * sg) = v;
    }
  } else {
    uint8_t* mine = stage + lane * 64;
#pragma unroll
    for (int sg = 0; sg < 4; ++sg) {
      uint4 o;
      __nv_bfloat162* ho = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
      for (int t = 0; t < 4; ++t) ho[t] = __floats2bfloat162_rn(f[8 * sg + 2 * t], f[8 * sg + 2 * t + 1]);
      *reinterpret_cast<uint4*>(mine + ((sg ^ ((lane >> 1) & 3)) << 4)) = o;
    }
    __syncwarp();
    const int sg = lane & 3;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int r = 8 * i + (lane >> 2);
      const uint4 v = *reinterpret_cast<const uint4*>(stage + r * 64 + ((sg ^ ((r >> 1) & 3)) << 4));
      if (row_base + r < M)
        *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(cptr) + (int64_t)(row_base + r) * ldc + n + 8 * sg) = v;
    }
  }
  __syncwarp();                                        // the next chunk overwrites the staging rows
}

// The reverse trip for what an epilogue reads per row (saved pre-activations, the fp32 residual): the warp fetches
// the 32 x 32 chunk as whole lines (lane -> one 16-byte segment of a row; this can be issued a chunk ahead), and
// when the chunk is due it goes through the warp's shared memory so that every lane ends up with its own row.
// bf16: lane holds segment (lane & 3) of rows 8 i + (lane >> 2), i = 0..3; a chunk takes 2 KB of the staging area.
__device__ __forceinline__ void lines_fetch_bf16(uint4 (&t)[4], const __nv_bfloat16* __restrict__ base, int64_t ld, int row_base,
                                                 int lane, int M, int n) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = row_base + 8 * i + (lane >> 2);
    t[i] = r < M ? *reinterpret_cast<const uint4*>(base + (int64_t)r * ld + n + 8 * (lane & 3)) : make_uint4(0u, 0u, 0u, 0u);
  }
}
__device__ __forceinline__ void lines_park_bf16(const uint4 (&t)[4], uint8_t* __restrict__ stage, int lane) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = 8 * i + (lane >> 2);
    *reinterpret_cast<uint4*>(stage + r * 64 + (((lane & 3) ^ ((r >> 1) & 3)) << 4)) = t[i];
  }
}
__device__ __forceinline__ void lines_own_row_bf16(uint4 (&row)[4], const uint8_t* __restrict__ stage, int lane) {
#pragma unroll
  for (int sg = 0; sg < 4; ++sg) row[sg] = *reinterpret_cast<const uint4*>(stage + lane * 64 + ((sg ^ ((lane >> 1) & 3)) << 4));
}
// fp32: lane holds segment (lane & 7) of rows 4 i + (lane >> 3), i = 0..7; a chunk takes the whole 4 KB.
__device__ __forceinline__ void lines_fetch_f32(float4 (&t)[8], const float* __restrict__ base, int64_t ld, int row_base, int lane,
                                                int M, int n) {
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int r = row_base + 4 * i + (lane >> 3);
    t[i] = r < M ? *reinterpret_cast<const float4*>(base + (int64_t)r * ld + n + 4 * (lane & 7)) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
}
__device__ __forceinline__ void lines_to_own_row_f32(const float4 (&t)[8], float4 (&row)[8], uint8_t* __restrict__ stage, int lane) {
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int r = 4 * i + (lane >> 3);
    *reinterpret_cast<float4*>(stage + r * 128 + (((lane & 7) ^ (r & 7)) << 4)) = t[i];
  }
  __syncwarp();
#pragma unroll
  for (int sg = 0; sg < 8; ++sg) row[sg] = *reinterpret_cast<const float4*>(stage + lane * 128 + ((sg ^ (lane & 7)) << 4));
  __syncwarp();
}

// One row's share of an output tile: BN columns from tensor memory at taddr, starting at column n0.
// With a rotary embedding (tiles are then whole heads of 128 columns) the chunk at head-local
// column j < 64 is read together with its partner at j + 64, both get their bias, and the pair is
// rotated in fp32 before the single rounding of the store.
template <bool OUT_F32>
__device__ __forceinline__ void epi_row(uint32_t taddr, int BN, int m, int M, int n0, int N, void* __restrict__ cptr, int64_t ldc,
                                        const __nv_bfloat16* __restrict__ bias, const float* __restrict__ residual, int64_t ldr,
                                        const RopeArgs& rope, uint8_t* __restrict__ stage, int lane) {
  // (the tensor-memory loads are warp-collective: take this path only if every row of the warp exists)
  if (OUT_F32 && residual != nullptr && n0 + BN <= N && __all_sync(0xffffffffu, m < M)) {
    // Output into the residual stream: the residual chunk of the next 32 columns is fetched while
    // this chunk is read from tensor memory, added and stored, so that only the first load's latency
    // is exposed per tile.
    const int row_base = m - lane;
    float4 rn[8];                                    // the next chunk of the residual, fetched as whole lines
    lines_fetch_f32(rn, residual, ldr, row_base, lane, M, n0);
    // the accumulator chunk after this one is requested from tensor memory before this one is worked on
    uint32_t va[32], vb[32];
    auto chunk = [&](uint32_t (&v)[32], int c0) {
      float4 rc[8];
      lines_to_own_row_f32(rn, rc, stage, lane);
      if (c0 + 32 < BN) lines_fetch_f32(rn, residual, ldr, row_base, lane, M, n0 + c0 + 32);
      float f[32];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        f[4 * j] = __uint_as_float(v[4 * j]) + rc[j].x; f[4 * j + 1] = __uint_as_float(v[4 * j + 1]) + rc[j].y;
        f[4 * j + 2] = __uint_as_float(v[4 * j + 2]) + rc[j].z; f[4 * j + 3] = __uint_as_float(v[4 * j + 3]) + rc[j].w;
      }
      epi_store32_lines<OUT_F32>(f, stage, cptr, ldc, m, lane, M, n0 + c0, bias);
    };
    tmem_ld32_nowait(taddr, va);
#pragma unroll 1
    for (int c0 = 0; c0 < BN; c0 += 64) {
      tmem_ld_wait32(va);
      const bool second = c0 + 32 < BN;              // uniform across the warp
      if (second) tmem_ld32_nowait(taddr + c0 + 32, vb);
      chunk(va, c0);
      if (second) {
        tmem_ld_wait32(vb);
        if (c0 + 64 < BN) tmem_ld32_nowait(taddr + c0 + 64, va);
        chunk(vb, c0 + 32);
      }
    }
    return;
  }
  if (OUT_F32 || rope.cs == nullptr || n0 >= rope.cols) {
    // no rotation in this tile: bias / residual / conversion per 32-column chunk, the next chunk's
    // tensor-memory load in flight meanwhile
    const int span = min(BN, ((N - n0 + 31) >> 5) << 5);      // columns to visit, a multiple of 32, uniform across the warp
    uint32_t va[32], vb[32];
    auto chunk = [&](uint32_t (&v)[32], int c0) {
      if (residual == nullptr && n0 + c0 + 32 <= N) {    // uniform across the warp: every lane takes part
        float f[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) f[j] = __uint_as_float(v[j]);
        epi_store32_lines<OUT_F32>(f, stage, cptr, ldc, m, lane, M, n0 + c0, bias);
      } else if (m < M) {
        float f[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) f[j] = __uint_as_float(v[j]);
        epi_store32<OUT_F32, false>(f, cptr, ldc, m, n0 + c0, N, bias, residual, ldr);
      }
    };
    if (span > 0) tmem_ld32_nowait(taddr, va);
#pragma unroll 1
    for (int c0 = 0; c0 < span; c0 += 64) {
      tmem_ld_wait32(va);
      const bool second = c0 + 32 < span;
      if (second) tmem_ld32_nowait(taddr + c0 + 32, vb);
      chunk(va, c0);
      if (second) {
        tmem_ld_wait32(vb);
        if (c0 + 64 < span) tmem_ld32_nowait(taddr + c0 + 64, va);
        chunk(vb, c0 + 32);
      }
    }
    return;
  }
#pragma unroll 1
  for (int c0 = 0; c0 < BN; c0 += 32) {
    if (n0 + c0 >= N) break;                       // uniform across the warp
    const int n = n0 + c0;
    if (!OUT_F32 && rope.cs != nullptr && n < rope.cols) {
      if (c0 & 64) continue;                       // second halves go with their partners
      uint32_t v1[32], v2[32];
      tmem_ld32(taddr + c0, v1);
      tmem_ld32(taddr + c0 + 64, v2);
      {                                             // every lane: the stores below are warp-wide (rows beyond M are not written)
        float f1[32], f2[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) { f1[j] = __uint_as_float(v1[j]); f2[j] = __uint_as_float(v2[j]); }
        if (bias) {
#pragma unroll
          for (int j = 0; j < 32; ++j) { f1[j] += __bfloat162float(bias[n + j]); f2[j] += __bfloat162float(bias[n + 64 + j]); }
        }
        const float* cr = rope.cs + (int64_t)(m % rope.seq) * 64 + (c0 & 32);
        const float* sr = cr + (int64_t)rope.seq * 64;
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
          const float4 c4 = *reinterpret_cast<const float4*>(cr + j), s4 = *reinterpret_cast<const float4*>(sr + j);
          const float cc[4] = {c4.x, c4.y, c4.z, c4.w}, ss[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
          for (int t = 0; t < 4; ++t) {
            const float x1 = f1[j + t], x2 = f2[j + t];
            f1[j + t] = x1 * cc[t] - x2 * ss[t];
            f2[j + t] = x1 * ss[t] + x2 * cc[t];
          }
        }
        epi_store32_lines<OUT_F32>(f1, stage, cptr, ldc, m, lane, M, n, nullptr);
        epi_store32_lines<OUT_F32>(f2, stage, cptr, ldc, m, lane, M, n + 64, nullptr);
      }
    } else {
      uint32_t v[32];
      tmem_ld32(taddr + c0, v);
      if (m < M) {
        float f[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) f[j] = __uint_as_float(v[j]);
        epi_store32<OUT_F32, false>(f, cptr, ldc, m, n, N, bias, residual, ldr);
      }
    }
  }
}

// Logistic function for the epilogues whose result is rounded to bf16: hardware exp2 and reciprocal
// (a few ulp of fp32, against the 2^-9 of the store); exp(-g) = inf gives 0, exp(-g) = 0 gives 1.
__device__ __forceinline__ float sigmoid_tc(float g) { return __fdividef(1.0f, 1.0f + __expf(-g)); }

// Gate | up tile: accumulator columns [0, 128) are gate columns nb .. nb+127, columns [128, 256) the
// up columns of the same index.  Stores silu(gate) * up, and the two pre-activations themselves
// when the backward pass will need them (cptr != nullptr).
struct SwigluArgs { __nv_bfloat16* out; int half; };          // out == nullptr: none; half = f
__device__ __forceinline__ void epi_row_swiglu(uint32_t taddr, int m, int M, int nb, void* __restrict__ cptr, int64_t ldc,
                                               const __nv_bfloat16* __restrict__ bias, const SwigluArgs& sw,
                                               uint8_t* __restrict__ stage, int lane) {
#pragma unroll 1
  for (int c0 = 0; c0 < 128; c0 += 32) {
    uint32_t vg[32], vu[32];
    tmem_ld32(taddr + c0, vg);
    tmem_ld32(taddr + 128 + c0, vu);
    {                                               // every lane: the stores are warp-wide (rows beyond M are not written)
      float g[32], u[32];
#pragma unroll
      for (int j = 0; j < 32; ++j) { g[j] = __uint_as_float(vg[j]); u[j] = __uint_as_float(vu[j]); }
      if (bias) {
#pragma unroll
        for (int j = 0; j < 32; ++j) { g[j] += __bfloat162float(bias[nb + c0 + j]); u[j] += __bfloat162float(bias[sw.half + nb + c0 + j]); }
      }
      float sgl[32];
#pragma unroll
      for (int j = 0; j < 32; ++j) sgl[j] = g[j] * sigmoid_tc(g[j]) * u[j];
      if (cptr) {
        epi_store32_lines<false>(g, stage, cptr, ldc, m, lane, M, nb + c0, nullptr);
        epi_store32_lines<false>(u, stage, cptr, ldc, m, lane, M, sw.half + nb + c0, nullptr);
      }
      epi_store32_lines<false>(sgl, stage, sw.out, sw.half, m, lane, M, nb + c0, nullptr);
    }
  }
}

// Backward of the gated activation on a tile of ds = dy W_down (columns n0 .. of f): reads the saved
// gate / up pre-activations of the same columns (the next chunk's while this one is worked on) and
// stores d gate and d up into the [M, 2f] gradient of the gate | up projection.
struct SwigluBwdArgs { const __nv_bfloat16* gu; };            // gu == nullptr: none
__device__ __forceinline__ void epi_row_swiglu_bwd(uint32_t taddr, int BN, int m, int M, int n0, int N, void* __restrict__ cptr,
                                                   const SwigluBwdArgs& sb, uint8_t* __restrict__ stage, int lane) {
  const int row_base = m - lane;
  const int64_t ldg = 2 * (int64_t)N;
  uint4 gn[4], un[4];                              // the next chunk of gate and up, fetched as whole lines (zeros beyond M)
  if (n0 < N) {
    lines_fetch_bf16(gn, sb.gu, ldg, row_base, lane, M, n0);
    lines_fetch_bf16(un, sb.gu, ldg, row_base, lane, M, N + n0);
  }
#pragma unroll 1
  for (int c0 = 0; c0 < BN; c0 += 32) {
    if (n0 + c0 >= N) break;                       // uniform across the warp; N is a multiple of 32
    lines_park_bf16(gn, stage, lane);
    lines_park_bf16(un, stage + 2048, lane);
    __syncwarp();
    uint4 gc[4], uc[4];
    lines_own_row_bf16(gc, stage, lane);
    lines_own_row_bf16(uc, stage + 2048, lane);
    __syncwarp();
    if (c0 + 32 < BN && n0 + c0 + 32 < N) {
      lines_fetch_bf16(gn, sb.gu, ldg, row_base, lane, M, n0 + c0 + 32);
      lines_fetch_bf16(un, sb.gu, ldg, row_base, lane, M, N + n0 + c0 + 32);
    }
    uint32_t v[32];
    tmem_ld32(taddr + c0, v);
    float dg[32], du[32];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const __nv_bfloat162* hg = reinterpret_cast<const __nv_bfloat162*>(&gc[j]);
      const __nv_bfloat162* hu = reinterpret_cast<const __nv_bfloat162*>(&uc[j]);
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const float2 g2 = __bfloat1622float2(hg[t]), u2 = __bfloat1622float2(hu[t]);
        const float d0 = __uint_as_float(v[8 * j + 2 * t]), d1 = __uint_as_float(v[8 * j + 2 * t + 1]);
        const float s0 = sigmoid_tc(g2.x), s1 = sigmoid_tc(g2.y);
        dg[8 * j + 2 * t] = d0 * u2.x * s0 * (1.0f + g2.x * (1.0f - s0));
        dg[8 * j + 2 * t + 1] = d1 * u2.y * s1 * (1.0f + g2.y * (1.0f - s1));
        du[8 * j + 2 * t] = d0 * g2.x * s0;
        du[8 * j + 2 * t + 1] = d1 * g2.y * s1;
      }
    }
    epi_store32_lines<false>(dg, stage, cptr, 2 * (int64_t)N, m, lane, M, n0 + c0, nullptr);
    epi_store32_lines<false>(du, stage, cptr, 2 * (int64_t)N, m, lane, M, N + n0 + c0, nullptr);
  }
}

// GELU (exact) in the epilogue.  Forward: stores gelu(y) (and y itself when cptr != nullptr).  Backward: the
// dX product's output times gelu'(a), a = saved pre-activation of the same element, prefetched a chunk ahead.
struct GeluArgs { __nv_bfloat16* out; const __nv_bfloat16* bwd_a; };      // both nullptr: none
// Normal CDF and density for epilogues whose result is rounded to bf16: erfc(x) = P(t) exp(-x^2),
// t = 1 / (1 + p x), x >= 0, the five-term rational approximation 7.1.26 of Abramowitz & Stegun
// (absolute error 1.5e-7, evaluated here with the hardware exp2 and reciprocal); the negative side
// uses erfc directly, so the small tail values carry no cancellation.  exp(-x^2) = exp(-a^2 / 2)
// also gives the density.
__device__ __forceinline__ void normal_cdf_pdf_tc(float a, float& cdf, float& pdf) {
  const float x = fabsf(a) * 0.70710678118654752440f;
  const float t = __fdividef(1.0f, fmaf(0.3275911f, x, 1.0f));
  const float poly = t * fmaf(t, fmaf(t, fmaf(t, fmaf(t, 1.061405429f, -1.453152027f), 1.421413741f), -0.284496736f), 0.254829592f);
  const float e = __expf(-x * x);
  const float half_erfc = 0.5f * poly * e;
  cdf = a >= 0.0f ? 1.0f - half_erfc : half_erfc;
  pdf = e * 0.39894228040143267794f;
}
__device__ __forceinline__ float gelu_tc(float a) {
  float cdf, pdf;
  normal_cdf_pdf_tc(a, cdf, pdf);
  return a * cdf;
}
__device__ __forceinline__ float gelu_grad_tc(float a) {
  float cdf, pdf;
  normal_cdf_pdf_tc(a, cdf, pdf);
  return fmaf(a, pdf, cdf);
}
__device__ __forceinline__ void epi_row_gelu_fwd(uint32_t taddr, int BN, int m, int M, int n0, int N, void* __restrict__ cptr,
                                                 int64_t ldc, const __nv_bfloat16* __restrict__ bias, const GeluArgs& ge,
                                                 uint8_t* __restrict__ stage, int lane) {
#pragma unroll 1
  for (int c0 = 0; c0 < BN; c0 += 32) {
    if (n0 + c0 >= N) break;                       // uniform across the warp; N is a multiple of 32
    uint32_t v[32];
    tmem_ld32(taddr + c0, v);
    {                                               // every lane: the stores are warp-wide (rows beyond M are not written)
      const int n = n0 + c0;
      float f[32], u[32];
#pragma unroll
      for (int j = 0; j < 32; ++j) f[j] = __uint_as_float(v[j]);
      if (bias) {
#pragma unroll
        for (int j = 0; j < 32; ++j) f[j] += __bfloat162float(bias[n + j]);
      }
#pragma unroll
      for (int j = 0; j < 32; ++j) u[j] = gelu_tc(f[j]);
      if (cptr) epi_store32_lines<false>(f, stage, cptr, ldc, m, lane, M, n, nullptr);
      epi_store32_lines<false>(u, stage, ge.out, N, m, lane, M, n, nullptr);
    }
  }
}
__device__ __forceinline__ void epi_row_gelu_bwd(uint32_t taddr, int BN, int m, int M, int n0, int N, void* __restrict__ cptr,
                                                 int64_t ldc, const GeluArgs& ge, uint8_t* __restrict__ stage, int lane) {
  const int row_base = m - lane;
  uint4 an[4];                                     // the next chunk of the saved pre-activation, fetched as whole lines
  if (n0 < N) lines_fetch_bf16(an, ge.bwd_a, N, row_base, lane, M, n0);
#pragma unroll 1
  for (int c0 = 0; c0 < BN; c0 += 32) {
    if (n0 + c0 >= N) break;
    lines_park_bf16(an, stage, lane);
    __syncwarp();
    uint4 ac[4];
    lines_own_row_bf16(ac, stage, lane);
    __syncwarp();
    if (c0 + 32 < BN && n0 + c0 + 32 < N) lines_fetch_bf16(an, ge.bwd_a, N, row_base, lane, M, n0 + c0 + 32);
    uint32_t v[32];
    tmem_ld32(taddr + c0, v);
    {
      float f[32];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const __nv_bfloat162* ha = reinterpret_cast<const __nv_bfloat162*>(&ac[j]);
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          const float2 a2 = __bfloat1622float2(ha[t]);
          f[8 * j + 2 * t] = __uint_as_float(v[8 * j + 2 * t]) * gelu_grad_tc(a2.x);
          f[8 * j + 2 * t + 1] = __uint_as_float(v[8 * j + 2 * t + 1]) * gelu_grad_tc(a2.y);
        }
      }
      epi_store32_lines<false>(f, stage, cptr, ldc, m, lane, M, n0 + c0, nullptr);
    }
  }
}

// ------------------------------------------------------------------ kernel
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Persistent: one CTA per SM walks output tiles (m fastest, so CTAs running together share the
// same B tile through L2).  Two accumulators in tensor memory: while the epilogue warps drain
// tile i, the MMA thread already accumulates tile i+1.
template <bool A_MN, bool B_MN, bool OUT_F32>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
               int M, int N, int K, void* __restrict__ cptr, int64_t ldc,
               const __nv_bfloat16* __restrict__ bias, const float* __restrict__ residual, int64_t ldr,
               int tiles_m, int num_tiles, int n_fast, TileRt tc, RopeArgs rope, SwigluArgs swg, SwigluBwdArgs swb, GeluArgs ge) {
  // Tile walk.  CTAs that run together should share the LARGER operand's slab and leave the smaller operand to L2:
  // row tiles fastest (n_fast = 0) when A is the smaller operand, column tiles fastest (n_fast = tiles along N) when B is.
  auto tm_of = [&](int tile) { return n_fast ? tile / n_fast : tile % tiles_m; };
  auto tn_of = [&](int tile) { return n_fast ? tile % n_fast : tile / tiles_m; };
  const int BN = tc.bn, S = tc.stages;
  const uint32_t kStageBytes = (uint32_t)tc.stage_bytes;
  extern __shared__ uint8_t smem_raw[];

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;   // 1024-byte aligned tiles
  const uint32_t bar_base = base + S * kStageBytes;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (S + s); };
  auto acc_full = [&](int a) { return bar_base + 8u * (2 * S + a); };
  auto acc_empty = [&](int a) { return bar_base + 8u * (2 * S + 2 + a); };
  const uint32_t tmem_slot = bar_base + 8u * (2 * S + 4);
  uint8_t* smem_gen = smem_raw + (base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot_gen = reinterpret_cast<volatile uint32_t*>(smem_gen + S * kStageBytes + 8 * (2 * S + 4));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_kb = (K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(acc_full(a), 1); mbar_init(acc_empty(a), 4); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(2 * kAccStride) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_gen;
  pdl_trigger();
  pdl_wait();                                        // barriers and tensor memory were set up under the predecessor's tail
  // An earlier launch timed out: do nothing but release the tensor memory.  The flag is global memory, so
  // it is read after the wait above; every role takes its own reading, and if two of them ever disagreed
  // the bounded waits below would end the launch the same way.
  const bool poisoned = *(volatile int*)&g_tc_error != 0;

  if (warp == 0) {
    // ---------------- TMA producer (one thread)
    if (lane == 0 && !poisoned) {
      int s = 0;
      uint32_t ph = 0;                   // ring position and its phase, advanced without divisions
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        const int m0 = tm_of(tile) * BM, n0 = tn_of(tile) * BN;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(empty_bar(s), ph ^ 1)) { atomicCAS(&g_tc_error, 0, 1); ok = false; break; }
          const uint32_t sa = base + s * kStageBytes, sb = sa + kABytes;
          mbar_expect_tx(full_bar(s), kStageBytes);
          const int k0 = kb * BK;
          if (A_MN) {
#pragma unroll
            for (int j = 0; j < BM / 64; ++j) tma_load_2d(sa + j * (BK * 128), &tmap_a, full_bar(s), m0 + j * 64, k0);
          } else {
            tma_load_2d(sa, &tmap_a, full_bar(s), k0, m0);
          }
          if (B_MN) {
            for (int j = 0; j * 64 < BN; ++j) tma_load_2d(sb + j * (BK * 128), &tmap_b, full_bar(s), n0 + j * 64, k0);
          } else if (swg.out != nullptr) {
            // gate | up: 128 rows of the gate block and the 128 rows of the same index in the up block
            const int nb = tn_of(tile) * 128;
            tma_load_2d(sb, &tmap_b, full_bar(s), k0, nb);
            tma_load_2d(sb + 128 * 128, &tmap_b, full_bar(s), k0, swg.half + nb);
          } else {
            tma_load_2d(sb, &tmap_b, full_bar(s), k0, n0);
          }
          if (++s == S) { s = 0; ph ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (one thread)
    if (lane == 0 && !poisoned) {
      // instruction descriptor: D fp32 (bits 4-5 = 1), A and B bf16 (bits 7-9, 10-12 = 1),
      // A / B major-ness (bits 15, 16: 1 = MN-major), N/8 at bits 17-22, M/16 at bits 24-28
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((A_MN ? 1u : 0u) << 15) |
                             ((B_MN ? 1u : 0u) << 16) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
      int s = 0, lt = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++lt) {
        const int ab = lt & 1;
        const uint32_t aph = (lt >> 1) & 1;
        // the epilogue must have drained this accumulator (passes at once on its first use)
        if (!mbar_wait(acc_empty(ab), aph ^ 1)) { atomicCAS(&g_tc_error, 0, 2); ok = false; break; }
        tc_fence_after();
        const uint32_t tacc = tmem_base + (uint32_t)(ab * kAccStride);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(full_bar(s), ph)) { atomicCAS(&g_tc_error, 0, 2); ok = false; break; }
          tc_fence_after();
          const uint32_t sa = base + s * kStageBytes, sb = sa + kABytes;
          const uint64_t da = make_desc(sa, A_MN), db = make_desc(sb, B_MN);
#pragma unroll
          for (int kk = 0; kk < BK / UMMA_K; ++kk) {
            // advance along k inside the stage: 32 B within the swizzle span (K-major) or
            // 16 k-rows of 128 B (MN-major); descriptor addresses are in 16-byte units
            const uint64_t adv_a = A_MN ? (uint64_t)(kk * UMMA_K * 128 >> 4) : (uint64_t)(kk * UMMA_K * 2 >> 4);
            const uint64_t adv_b = B_MN ? (uint64_t)(kk * UMMA_K * 128 >> 4) : (uint64_t)(kk * UMMA_K * 2 >> 4);
            tc_mma(tacc, da + adv_a, db + adv_b, idesc, (kb > 0 || kk > 0) ? 1u : 0u);
          }
          tc_commit(empty_bar(s));       // frees the stage once these MMAs have read it
          if (++s == S) { s = 0; ph ^= 1; }
        }
        tc_commit(acc_full(ab));         // accumulator complete (or abandoned: g_tc_error tells the epilogue)
      }
    }
  } else {
    // ---------------- epilogue: warps 2..5 own tensor-memory lanes 32*(warp%4) .. +31
    const int q = warp & 3;
    uint8_t* stage = smem_gen + S * kStageBytes + 256 + (warp - 2) * kStoreStage;   // behind the barriers
    int lt = 0;
    for (int tile = blockIdx.x; tile < num_tiles && !poisoned; tile += gridDim.x, ++lt) {
      const int ab = lt & 1;
      const uint32_t aph = (lt >> 1) & 1;
      const bool ready = mbar_wait(acc_full(ab), aph);
      if (!ready && lane == 0) atomicCAS(&g_tc_error, 0, 3);
      tc_fence_after();
      // one decision for the whole warp: the tensor-memory loads below are warp-collective
      if (!__all_sync(0xffffffffu, ready && *(volatile int*)&g_tc_error == 0)) break;
      const int m0 = tm_of(tile) * BM, n0 = tn_of(tile) * BN;
      const int m = m0 + q * 32 + lane;
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(ab * kAccStride);
      if (!OUT_F32 && swg.out != nullptr) epi_row_swiglu(taddr, m, M, tn_of(tile) * 128, cptr, ldc, bias, swg, stage, lane);
      else if (!OUT_F32 && swb.gu != nullptr) epi_row_swiglu_bwd(taddr, BN, m, M, n0, N, cptr, swb, stage, lane);
      else if (!OUT_F32 && ge.out != nullptr) epi_row_gelu_fwd(taddr, BN, m, M, n0, N, cptr, ldc, bias, ge, stage, lane);
      else if (!OUT_F32 && ge.bwd_a != nullptr) epi_row_gelu_bwd(taddr, BN, m, M, n0, N, cptr, ldc, ge, stage, lane);
      else epi_row<OUT_F32>(taddr, BN, m, M, n0, N, cptr, ldc, bias, residual, ldr, rope, stage, lane);
      // hand the accumulator back to the MMA thread
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty(ab));
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2 * kAccStride) : "memory");
  }
}

// ------------------------------------------------------------------ CTA-pair kernel
// Two CTAs of a cluster share one 256 x 256 output tile: each stages its own 128 rows of A and
// its own 128 columns of B, and one thread of the pair's first CTA issues tcgen05.mma with
// cta_group::2 (M = 256), which reads both CTAs' shared memory and writes each CTA's half of
// the accumulator into that CTA's tensor memory.  Per CTA the operand traffic from L2 drops by a
// third (16 + 16 KB per stage instead of 16 + 32 KB) for the same flops.  No multicast load:
// every CTA fetches what it stages; only mbarrier signals cross the pair.
constexpr int kBN2 = 256;
constexpr int kB2Bytes = (kBN2 / 2) * BK * 2;          // this CTA's half of B
constexpr int kStage2Bytes = kABytes + kB2Bytes;       // 32 KB
constexpr int kStages2 = kSmemBudget / kStage2Bytes;   // 6

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load whose completion is counted on a barrier that may live in the peer CTA
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster_addr, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"((uint64_t)map), "r"(bar_cluster_addr), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {      // arrives on `bar` in both CTAs of the pair
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t tmem_c, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_c), "l"(da), "l"(db), "r"(idesc), "r"(accum) : "memory");
}

template <bool A_MN, bool B_MN, bool OUT_F32>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc2_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                int M, int N, int K, void* __restrict__ cptr, int64_t ldc,
                const __nv_bfloat16* __restrict__ bias, const float* __restrict__ residual, int64_t ldr,
                int tiles_m, int num_tiles, int n_fast, RopeArgs rope, SwigluArgs swg, SwigluBwdArgs swb, GeluArgs ge) {
  auto tm_of = [&](int tile) { return n_fast ? tile / n_fast : tile % tiles_m; };      // see gemm_tc_kernel
  auto tn_of = [&](int tile) { return n_fast ? tile % n_fast : tile / tiles_m; };
  constexpr int S = kStages2;
  constexpr int BN = kBN2;
  extern __shared__ uint8_t smem_raw[];
  // both CTAs of a pair read the same flag value only by luck, so decide nothing on it before the
  // pair has synchronised once; an early exit of one CTA alone would strand its peer
  const uint32_t rank = cluster_ctarank();
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar_base = base + S * kStage2Bytes;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (S + s); };
  auto acc_full = [&](int a) { return bar_base + 8u * (2 * S + a); };
  auto acc_empty = [&](int a) { return bar_base + 8u * (2 * S + 2 + a); };
  const uint32_t tmem_slot = bar_base + 8u * (2 * S + 4);
  uint8_t* smem_gen = smem_raw + (base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot_gen = reinterpret_cast<volatile uint32_t*>(smem_gen + S * kStage2Bytes + 8 * (2 * S + 4));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_kb = (K + BK - 1) / BK;
  const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(acc_full(a), 1); mbar_init(acc_empty(a), 8); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(2 * kAccStride) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  cluster_sync_all();                                  // barriers of both CTAs are initialised
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_gen;
  pdl_trigger();
  pdl_wait();                                          // set-up above overlaps the predecessor's tail
  const bool poisoned = *(volatile int*)&g_tc_error != 0;   // read after the pair sync; see the exit below

  if (warp == 0) {
    // ---------------- TMA producer (one thread per CTA): own rows of A, own columns of B;
    //                  completion is counted on the first CTA's barrier
    if (lane == 0 && !poisoned) {
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
        const int m0 = tm_of(tile) * (2 * BM) + (int)rank * BM;
        // this CTA's 128 columns of B; gate | up: the first CTA stages the gate rows, the second the up rows
        const int n0 = (!B_MN && swg.out != nullptr) ? tn_of(tile) * 128 + (int)rank * swg.half
                                                     : tn_of(tile) * BN + (int)rank * (BN / 2);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(empty_bar(s), ph ^ 1)) { atomicCAS(&g_tc_error, 0, 1); ok = false; break; }
          const uint32_t sa = base + s * kStage2Bytes, sb = sa + kABytes;
          const uint32_t fb = map_to_cta(full_bar(s), 0);
          if (rank == 0) mbar_expect_tx(full_bar(s), 2 * kStage2Bytes);
          const int k0 = kb * BK;
          if (A_MN) {
#pragma unroll
            for (int j = 0; j < BM / 64; ++j) tma_load_2d_pair(sa + j * (BK * 128), &tmap_a, fb, m0 + j * 64, k0);
          } else {
            tma_load_2d_pair(sa, &tmap_a, fb, k0, m0);
          }
          if (B_MN) {
#pragma unroll
            for (int j = 0; j < BN / 128; ++j) tma_load_2d_pair(sb + j * (BK * 128), &tmap_b, fb, n0 + j * 64, k0);
          } else {
            tma_load_2d_pair(sb, &tmap_b, fb, k0, n0);
          }
          if (++s == S) { s = 0; ph ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer: one thread of the pair's first CTA
    if (lane == 0 && rank == 0 && !poisoned) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((A_MN ? 1u : 0u) << 15) |
                             ((B_MN ? 1u : 0u) << 16) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((2 * BM) >> 4) << 24);
      int s = 0, lt = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int tile = pair; tile < num_tiles && ok; tile += num_pairs, ++lt) {
        const int ab = lt & 1;
        const uint32_t aph = (lt >> 1) & 1;
        if (!mbar_wait(acc_empty(ab), aph ^ 1)) { atomicCAS(&g_tc_error, 0, 2); ok = false; break; }
        tc_fence_after();
        const uint32_t tacc = tmem_base + (uint32_t)(ab * kAccStride);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(full_bar(s), ph)) { atomicCAS(&g_tc_error, 0, 2); ok = false; break; }
          tc_fence_after();
          const uint32_t sa = base + s * kStage2Bytes, sb = sa + kABytes;
          const uint64_t da = make_desc(sa, A_MN), db = make_desc(sb, B_MN);
#pragma unroll
          for (int kk = 0; kk < BK / UMMA_K; ++kk) {
            const uint64_t adv_a = A_MN ? (uint64_t)(kk * UMMA_K * 128 >> 4) : (uint64_t)(kk * UMMA_K * 2 >> 4);
            const uint64_t adv_b = B_MN ? (uint64_t)(kk * UMMA_K * 128 >> 4) : (uint64_t)(kk * UMMA_K * 2 >> 4);
            tc_mma_pair(tacc, da + adv_a, db + adv_b, idesc, (kb > 0 || kk > 0) ? 1u : 0u);
          }
          tc_commit_pair(empty_bar(s));      // frees the stage in both CTAs
          if (++s == S) { s = 0; ph ^= 1; }
        }
        tc_commit_pair(acc_full(ab));        // both CTAs' epilogues may drain their half
      }
    }
  } else {
    // ---------------- epilogue (both CTAs): tensor-memory lanes 32*(warp%4).. hold rows of this CTA's half
    const int q = warp & 3;
    uint8_t* stage = smem_gen + S * kStage2Bytes + 256 + (warp - 2) * kStoreStage;   // behind the barriers
    int lt = 0;
    for (int tile = pair; tile < num_tiles && !poisoned; tile += num_pairs, ++lt) {
      const int ab = lt & 1;
      const uint32_t aph = (lt >> 1) & 1;
      const bool ready = mbar_wait(acc_full(ab), aph);
      if (!ready && lane == 0) atomicCAS(&g_tc_error, 0, 3);
      tc_fence_after();
      if (!__all_sync(0xffffffffu, ready && *(volatile int*)&g_tc_error == 0)) break;
      const int m0 = tm_of(tile) * (2 * BM) + (int)rank * BM, n0 = tn_of(tile) * BN;
      const int m = m0 + q * 32 + lane;
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(ab * kAccStride);
      if (!OUT_F32 && swg.out != nullptr) epi_row_swiglu(taddr, m, M, tn_of(tile) * 128, cptr, ldc, bias, swg, stage, lane);
      else if (!OUT_F32 && swb.gu != nullptr) epi_row_swiglu_bwd(taddr, BN, m, M, n0, N, cptr, swb, stage, lane);
      else if (!OUT_F32 && ge.out != nullptr) epi_row_gelu_fwd(taddr, BN, m, M, n0, N, cptr, ldc, bias, ge, stage, lane);
      else if (!OUT_F32 && ge.bwd_a != nullptr) epi_row_gelu_bwd(taddr, BN, m, M, n0, N, cptr, ldc, ge, stage, lane);
      else epi_row<OUT_F32>(taddr, BN, m, M, n0, N, cptr, ldc, bias, residual, ldr, rope, stage, lane);
      // hand this CTA's half of the accumulator back: the MMA thread counts 8 warps (4 per CTA)
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_remote(map_to_cta(acc_empty(ab), 0));
    }
  }
  // nobody leaves while the peer may still signal this CTA's barriers or read its shared memory
  tc_fence_before();
  cluster_sync_all();
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2 * kAccStride) : "memory");
  }
}

#include "attention_tc.cuh"
#include "attention_bwd_tc.cuh"

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;
int g_num_sms = 148;
int g_init_state = -1;    // -1 not tried, 0 ok, 1 failed
std::mutex g_mu;
int g_pdl = 1;            // programmatic dependent launch of the GEMM kernels (switch 1 of gemm_tc_switch; 0: plain stream order)

struct MapKey {
  const void* p; uint64_t inner, outer, stride; uint32_t box_outer;
  bool operator==(const MapKey& o) const {
    return p == o.p && inner == o.inner && outer == o.outer && stride == o.stride && box_outer == o.box_outer;
  }
};
struct MapKeyHash {
  size_t operator()(const MapKey& k) const {
    size_t h = (size_t)k.p;
    h = h * 1000003u ^ k.inner; h = h * 1000003u ^ k.outer; h = h * 1000003u ^ k.stride; h = h * 1000003u ^ k.box_outer;
    return h;
  }
};
std::unordered_map<MapKey, CUtensorMap, MapKeyHash> g_maps;

// 2-D bf16 tensor [outer][inner] with row pitch `stride_elems`; box = 64 x box_outer, 128-byte swizzle.
bool get_map(const void* p, uint64_t inner, uint64_t outer, uint64_t stride_elems, uint32_t box_outer, CUtensorMap* out) {
  MapKey key{p, inner, outer, stride_elems, box_outer};
  std::lock_guard<std::mutex> lk(g_mu);
  auto it = g_maps.find(key);
  if (it != g_maps.end()) { *out = it->second; return true; }
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {stride_elems * 2};
  cuuint32_t box[2] = {64, box_outer};
  cuuint32_t estr[2] = {1, 1};
  CUtensorMap m;
  CUresult r = g_encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(p), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  if (g_maps.size() > 65536) g_maps.clear();
  g_maps[key] = m;
  *out = m;
  return true;
}

template <typename... KArgs, typename... Args>
cudaError_t launch_pdl_tc(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = g_pdl;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
template <bool A_MN, bool B_MN, bool OUT_F32>
cudaError_t set_smem_attr() {
  return cudaFuncSetAttribute(gemm_tc_kernel<A_MN, B_MN, OUT_F32>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              kSmemBytes);
}
template <bool A_MN, bool B_MN, bool OUT_F32>
cudaError_t launch_inst(cudaStream_t st, const GemmArgs& g, const CUtensorMap& ta, const CUtensorMap& tb, int bn) {
  const TileRt tc = make_tile(bn, B_MN);
  const int tiles_m = (g.M + BM - 1) / BM, tiles_n = g.swiglu_out ? g.N / 256 : (g.N + bn - 1) / bn;
  const int num_tiles = tiles_m * tiles_n;
  const int grid = num_tiles < g_num_sms ? num_tiles : g_num_sms;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = g_pdl;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, gemm_tc_kernel<A_MN, B_MN, OUT_F32>, ta, tb, g.M, g.N, g.K, g.c, g.ldc,
                            (const __nv_bfloat16*)g.bias, g.residual, g.ldr, tiles_m, num_tiles, g.M > g.N ? tiles_n : 0, tc,
                            RopeArgs{g.rope_cs, g.rope_seq, g.rope_cols}, SwigluArgs{(__nv_bfloat16*)g.swiglu_out, g.N / 2},
                            SwigluBwdArgs{(const __nv_bfloat16*)g.swiglu_bwd_gu},
                            GeluArgs{(__nv_bfloat16*)g.gelu_out, (const __nv_bfloat16*)g.gelu_bwd_a});
}

template <bool A_MN, bool B_MN, bool OUT_F32>
cudaError_t launch_pair(cudaStream_t st, const GemmArgs& g, const CUtensorMap& ta, const CUtensorMap& tb) {
  const int tiles_m = (g.M + 2 * BM - 1) / (2 * BM), tiles_n = (g.N + kBN2 - 1) / kBN2;
  const int num_tiles = tiles_m * tiles_n;
  int pairs = g_num_sms / 2;
  if (num_tiles < pairs) pairs = num_tiles;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(2 * pairs);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = g_pdl;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, gemm_tc2_kernel<A_MN, B_MN, OUT_F32>, ta, tb, g.M, g.N, g.K, g.c, g.ldc,
                            (const __nv_bfloat16*)g.bias, g.residual, g.ldr, tiles_m, num_tiles, g.M > g.N ? tiles_n : 0,
                            RopeArgs{g.rope_cs, g.rope_seq, g.rope_cols}, SwigluArgs{(__nv_bfloat16*)g.swiglu_out, g.N / 2},
                            SwigluBwdArgs{(const __nv_bfloat16*)g.swiglu_bwd_gu},
                            GeluArgs{(__nv_bfloat16*)g.gelu_out, (const __nv_bfloat16*)g.gelu_bwd_a});
}
template <bool A_MN, bool B_MN, bool OUT_F32>
cudaError_t set_smem_attr2() {
  return cudaFuncSetAttribute(gemm_tc2_kernel<A_MN, B_MN, OUT_F32>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
}
int g_attn_tc = 1;       // tcgen05 attention forward (switch 2; 0 falls back to the mma.sync kernel)
int g_attn_bwd_tc = 1;   // tcgen05 attention backward (switch 3; 0 falls back to the mma.sync kernels)
template <int DH, int MODE>
cudaError_t set_smem_attr_ab() {
  cudaError_t e = cudaFuncSetAttribute(attn_bwd_tc_kernel<DH, MODE, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       AttnBwdCfg<DH, MODE>::kSmem);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(attn_bwd_tc_kernel<DH, MODE, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              AttnBwdCfg<DH, MODE>::kSmem);
}
int g_pair_mode = 1;     // CTA-pair kernel for 256-wide tiles (switch 0; 0 falls back to one CTA per tile)

}  // namespace

int gemm_tc_switch(int which, int value) {
  int* sw[4] = {&g_pair_mode, &g_pdl, &g_attn_tc, &g_attn_bwd_tc};
  if (which < 0 || which > 3) return -1;
  const int old = *sw[which];
  if (value >= 0) *sw[which] = value;
  return old;
}
int pdl_switch_value() { return g_pdl; }

int gemm_tc_init() {
  std::lock_guard<std::mutex> lk(g_mu);
  if (g_init_state >= 0) return g_init_state;
  g_init_state = 1;
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return g_init_state;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess || major != 10) return g_init_state;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
      qres != cudaDriverEntryPointSuccess) {
    cudaGetLastError();
    return g_init_state;
  }
  g_encode = (EncodeTiledFn)fn;
  if (cudaDeviceGetAttribute(&g_num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || g_num_sms < 1) g_num_sms = 148;
  cudaError_t e = cudaSuccess;
  if (e == cudaSuccess) e = set_smem_attr<false, false, false>();
  if (e == cudaSuccess) e = set_smem_attr<false, false, true>();
  if (e == cudaSuccess) e = set_smem_attr<false, true, false>();
  if (e == cudaSuccess) e = set_smem_attr<false, true, true>();
  if (e == cudaSuccess) e = set_smem_attr<true, true, true>();
  if (e == cudaSuccess) e = set_smem_attr<true, true, false>();
  if (e == cudaSuccess) e = set_smem_attr2<false, false, false>();
  if (e == cudaSuccess) e = set_smem_attr2<false, false, true>();
  if (e == cudaSuccess) e = set_smem_attr2<false, true, false>();
  if (e == cudaSuccess) e = set_smem_attr2<false, true, true>();
  if (e == cudaSuccess) e = set_smem_attr2<true, true, true>();
  if (e == cudaSuccess) e = set_smem_attr2<true, true, false>();
  if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_fwd_tc_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnTcCfg<64>::kSmem);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_fwd_tc_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnTcCfg<128>::kSmem);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_fwd_tc_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnTcCfg<64>::kSmem);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_fwd_tc_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnTcCfg<128>::kSmem);
  if (e == cudaSuccess) e = set_smem_attr_ab<64, 0>();
  if (e == cudaSuccess) e = set_smem_attr_ab<64, 1>();
  if (e == cudaSuccess) e = set_smem_attr_ab<128, 0>();
  if (e == cudaSuccess) e = set_smem_attr_ab<128, 1>();
  if (e != cudaSuccess) { cudaGetLastError(); return g_init_state; }
  g_init_state = 0;
  return 0;
}

// 0: not eligible; 1: forward (A K-major, B K-major); 2: dX (A K-major, B N-major); 3: dW (A M-major, B N-major)
static int classify(const GemmArgs& g) {
  if (g_init_state != 0) return 0;
  if (g.M < 128 || g.N < 64 || g.K < 64) return 0;
  const bool a_k = g.sak == 1, a_m = g.sam == 1, b_k = g.sbk == 1, b_n = g.sbn == 1;
  int form = 0;
  if (a_k && b_k) form = 1; else if (a_k && b_n) form = 2; else if (a_m && b_n) form = 3; else return 0;
  const int64_t lda = a_k ? g.sam : g.sak, ldb = b_k ? g.sbn : g.sbk;
  if (lda % 8 || ldb % 8 || g.ldc % (g.out_f32 ? 4 : 8)) return 0;
  if (((uintptr_t)g.a | (uintptr_t)g.b | (uintptr_t)g.c) & 15) return 0;
  if (g.bias && ((uintptr_t)g.bias & 15)) return 0;
  if (g.residual && (!g.out_f32 || ((uintptr_t)g.residual & 15) || g.ldr % 4)) return 0;
  if (form == 3 && (g.bias || g.residual)) return 0;        // weight gradients: fp32 out, or bf16 out when gradients are kept in bf16
  // rotary embedding in the epilogue: forward form, bf16 output, whole heads of 128 columns per tile
  // gated activation in the epilogue: forward form, bf16 output, f a multiple of 128 (a tile = 128 gate + 128 up columns)
  if (g.swiglu_out && (form != 1 || g.out_f32 || g.residual || g.rope_cs || (g.N / 2) % 128 || g.N % 2 ||
                       (((uintptr_t)g.swiglu_out) & 15))) return 0;
  // backward of the gated activation in the epilogue: dX form, bf16 output of 2N columns
  if (g.swiglu_bwd_gu && (form != 2 || g.out_f32 || g.bias || g.residual || g.N % 32 || g.ldc != 2 * (int64_t)g.N ||
                          (((uintptr_t)g.swiglu_bwd_gu) & 15))) return 0;
  // GELU in the epilogue: forward form (gelu_out) or dX form (gelu_bwd_a), bf16 output, N a multiple of 32
  if (g.gelu_out && (form != 1 || g.out_f32 || g.residual || g.rope_cs || g.swiglu_out || g.N % 32 || (((uintptr_t)g.gelu_out) & 15))) return 0;
  if (g.gelu_bwd_a && (form != 2 || g.out_f32 || g.bias || g.residual || g.swiglu_bwd_gu || g.N % 32 || (((uintptr_t)g.gelu_bwd_a) & 15))) return 0;
  if (g.rope_cs && (form != 1 || g.out_f32 || g.rope_dh != 128 || g.rope_seq < 1 || g.rope_cols % 128 || g.N % 128 ||
                    g.rope_cols > g.N || (((uintptr_t)g.rope_cs) & 15))) return 0;
  return form;
}
bool gemm_tc_eligible(const GemmArgs& g) { return classify(g) != 0; }

cudaError_t gemm_tc_launch(cudaStream_t st, const GemmArgs& g) {
  const int form = classify(g);
  if (!form) return cudaErrorInvalidValue;
  // Tile choice.  Wide tiles keep the tensor pipe busiest (less operand traffic per flop), the CTA-pair
  // kernel (256 x 256 per pair) more so; but a grid that leaves most SMs idle in its last round loses
  // more.  Score = fraction of SM-rounds doing work x columns that exist x a per-tile efficiency
  // (measured: pair 1.0, one CTA at width w about 0.87 * (w / (w + 48)) / (256 / 304)).
  int bn = 256;
  bool use_pair = false;
  {
    const int tm = (g.M + BM - 1) / BM;
    double best = -1.0;
    const bool b_mn = form != 1;
    for (int cand = 256; cand >= 64; cand -= 32) {
      if (g.rope_cs && cand % 128) continue;                               // tiles must hold whole heads
      if (g.swiglu_out && cand != 256) continue;                           // 128 gate + 128 up columns
      const int tn = (g.N + cand - 1) / cand;
      const int tiles = tm * tn;
      const int rounds = (tiles + g_num_sms - 1) / g_num_sms;
      const double useful = (double)g.N / ((double)tn * cand);            // columns of the last tile that exist
      double tile_eff = 0.87 * ((double)cand / (cand + 48.0)) / (256.0 / 304.0);
      if (b_mn) tile_eff *= (double)cand / (double)(((cand + 63) / 64) * 64);   // N-major B is staged in whole 64-wide boxes
      const double score = (double)tiles / ((double)rounds * g_num_sms) * useful * tile_eff;
      if (score > best * 1.08) { best = score; bn = cand; }               // leave a wider tile only for a clear gain
    }
    if (g_pair_mode && g.M >= 256 && g.N >= 256) {
      const int pm = (g.M + 2 * BM - 1) / (2 * BM), pn = (g.N + kBN2 - 1) / kBN2;
      const int pairs = g_num_sms / 2, ptiles = pm * pn;
      const int rounds = (ptiles + pairs - 1) / pairs;
      const double useful = ((double)g.N / ((double)pn * kBN2)) * ((double)g.M / ((double)pm * 2 * BM));
      const double score = (double)ptiles / ((double)rounds * pairs) * useful;
      if (score >= best) use_pair = true;
    }
  }
  CUtensorMap ta, tb;
  bool ok;
  if (use_pair) {
    // CTA pair: each CTA stages 128 rows of A and 128 columns of B
    if (form == 3) ok = get_map(g.a, (uint64_t)g.M, (uint64_t)g.K, (uint64_t)g.sak, BK, &ta);
    else ok = get_map(g.a, (uint64_t)g.K, (uint64_t)g.M, (uint64_t)g.sam, BM, &ta);
    if (form == 1) ok = ok && get_map(g.b, (uint64_t)g.K, (uint64_t)g.N, (uint64_t)g.sbn, (uint32_t)(kBN2 / 2), &tb);
    else ok = ok && get_map(g.b, (uint64_t)g.N, (uint64_t)g.K, (uint64_t)g.sbk, BK, &tb);
    if (!ok) return cudaErrorInvalidValue;
    if (form == 1) return g.out_f32 ? launch_pair<false, false, true>(st, g, ta, tb) : launch_pair<false, false, false>(st, g, ta, tb);
    if (form == 2) return g.out_f32 ? launch_pair<false, true, true>(st, g, ta, tb) : launch_pair<false, true, false>(st, g, ta, tb);
    return g.out_f32 ? launch_pair<true, true, true>(st, g, ta, tb) : launch_pair<true, true, false>(st, g, ta, tb);
  }
  // K-major operand: tensor [rows = M or N][inner = K]; MN-major operand: tensor [rows = K][inner = M or N]
  if (form == 3) ok = get_map(g.a, (uint64_t)g.M, (uint64_t)g.K, (uint64_t)g.sak, BK, &ta);
  else ok = get_map(g.a, (uint64_t)g.K, (uint64_t)g.M, (uint64_t)g.sam, BM, &ta);
  if (form == 1) ok = ok && get_map(g.b, (uint64_t)g.K, (uint64_t)g.N, (uint64_t)g.sbn, (uint32_t)(g.swiglu_out ? 128 : bn), &tb);
  else ok = ok && get_map(g.b, (uint64_t)g.N, (uint64_t)g.K, (uint64_t)g.sbk, BK, &tb);
  if (!ok) return cudaErrorInvalidValue;
  if (form == 1) return g.out_f32 ? launch_inst<false, false, true>(st, g, ta, tb, bn)
                                  : launch_inst<false, false, false>(st, g, ta, tb, bn);
  if (form == 2) return g.out_f32 ? launch_inst<false, true, true>(st, g, ta, tb, bn)
                                  : launch_inst<false, true, false>(st, g, ta, tb, bn);
  return g.out_f32 ? launch_inst<true, true, true>(st, g, ta, tb, bn) : launch_inst<true, true, false>(st, g, ta, tb, bn);
}

const int* gemm_tc_error_device_ptr() {
  static const int* ptr = nullptr;
  if (!ptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_tc_error) == cudaSuccess) ptr = (const int*)p;
    else cudaGetLastError();
  }
  return ptr;
}

bool attn_tc_eligible(int dh, const void* qkv, int H) {
  // head sizes 64 and 128 (switch 2 off sends both to the warp-level kernel)
  return g_init_state == 0 && g_attn_tc && (dh == 128 || dh == 64) && (((uintptr_t)qkv) & 15) == 0 && ((3 * H * dh) % 8) == 0;
}
cudaError_t attn_tc_fwd_launch(cudaStream_t st, int B, int S, int H, int dh, int causal, const void* qkv, void* o, float* lse,
                               const int* lens, const DropArgs& da) {
  CUtensorMap tm;
  const uint64_t d3 = 3ull * H * dh;
  if (!get_map(qkv, d3, (uint64_t)B * S, d3, 128, &tm)) return cudaErrorInvalidValue;
  const int nitems = ((S + kAttBQ - 1) / kAttBQ) * H * B;
  const int grid = nitems < g_num_sms ? nitems : g_num_sms;          // persistent: one CTA per SM
  const float scale = 1.0f / sqrtf((float)dh);
#define HIFT_ATTN_FWD(D, DR) launch_pdl_tc(attn_fwd_tc_kernel<D, DR>, dim3(grid), dim3(kAttThreads), AttnTcCfg<D>::kSmem, st, tm, (__nv_bfloat16*)o, lse, B, S, H, causal, scale, lens, da)
  if (da.thr != 0u) return dh == 64 ? HIFT_ATTN_FWD(64, true) : HIFT_ATTN_FWD(128, true);
  return dh == 64 ? HIFT_ATTN_FWD(64, false) : HIFT_ATTN_FWD(128, false);
#undef HIFT_ATTN_FWD
}

bool attn_tc_bwd_eligible(int dh, int H, const void* qkv, const void* dout, const void* dqkv) {
  return g_init_state == 0 && g_attn_bwd_tc && (dh == 64 || dh == 128) && ((H * dh) % 8) == 0 &&
         ((((uintptr_t)qkv) | ((uintptr_t)dout) | ((uintptr_t)dqkv)) & 15) == 0;
}
template <int DH>
static cudaError_t attn_tc_bwd_inst(cudaStream_t st, int B, int S, int H, int causal, const void* qkv, const void* dout,
                                    const float* lse, const float* dsum, void* dqkv, const int* lens, const DropArgs& da) {
  const uint64_t d = (uint64_t)H * DH, d3 = 3 * d, rows = (uint64_t)B * S;
  CUtensorMap qkv_f, qkv_x, do_f, do_x;
  if (!get_map(qkv, d3, rows, d3, kAbF, &qkv_f) || !get_map(qkv, d3, rows, d3, kAbX, &qkv_x) ||
      !get_map(dout, d, rows, d, kAbF, &do_f) || !get_map(dout, d, rows, d, kAbX, &do_x))
    return cudaErrorInvalidValue;
  const int nitems = ((S + kAbF - 1) / kAbF) * H * B;
  const int grid = nitems < g_num_sms ? nitems : g_num_sms;       // persistent: one CTA per SM
  const float scale = 1.0f / sqrtf((float)DH);
  // dK, dV: fixed K, V; streamed Q, dO
#define HIFT_ATTN_BWD0(DR) launch_pdl_tc(attn_bwd_tc_kernel<DH, 0, DR>, dim3(grid), dim3(kAbThreads), AttnBwdCfg<DH, 0>::kSmem, st, \
      qkv_f, qkv_f, qkv_x, do_x, (int)d, (int)(2 * d), 0, 0, lse, dsum, (__nv_bfloat16*)dqkv, B, S, H, causal, scale, lens, da)
#define HIFT_ATTN_BWD1(DR) launch_pdl_tc(attn_bwd_tc_kernel<DH, 1, DR>, dim3(grid), dim3(kAbThreads), AttnBwdCfg<DH, 1>::kSmem, st, \
      qkv_f, do_f, qkv_x, qkv_x, 0, 0, (int)d, (int)(2 * d), lse, dsum, (__nv_bfloat16*)dqkv, B, S, H, causal, scale, lens, da)
  const bool drop = da.thr != 0u;
  cudaError_t e = drop ? HIFT_ATTN_BWD0(true) : HIFT_ATTN_BWD0(false);
  if (e != cudaSuccess) return e;
  // dQ: fixed Q, dO; streamed K, V
  return drop ? HIFT_ATTN_BWD1(true) : HIFT_ATTN_BWD1(false);
#undef HIFT_ATTN_BWD0
#undef HIFT_ATTN_BWD1
}
cudaError_t attn_tc_bwd_launch(cudaStream_t st, int B, int S, int H, int dh, int causal, const void* qkv, const void* dout,
                               const float* lse, const float* dsum, void* dqkv, const int* lens, const DropArgs& da) {
  if (dh == 64) return attn_tc_bwd_inst<64>(st, B, S, H, causal, qkv, dout, lse, dsum, dqkv, lens, da);
  return attn_tc_bwd_inst<128>(st, B, S, H, causal, qkv, dout, lse, dsum, dqkv, lens, da);
}

int gemm_tc_set_error(int v) {
  return cudaMemcpyToSymbol(g_tc_error, &v, sizeof(int)) == cudaSuccess ? 0 : -1;
}

int gemm_tc_poll_error() {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_tc_error, sizeof(int)) != cudaSuccess) return -1;
  return v;
}

}  // namespace hift
