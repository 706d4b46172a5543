// Host-side launch wrappers: pick the template instance for the dtype / head size and the
// grid.  Shared by the training-step engine and the single-kernel C entry points.
#pragma once
#include "gemm_args.h"
#include "gemm_tc.h"
#include "kernels_attention.cuh"
#include "kernels_attention_mma.cuh"
#include "kernels_gemm_simt.cuh"
#include "kernels_pointwise.cuh"

namespace hift {

inline int grid_for(size_t n, int block, int max_blocks = 148 * 16) {
  size_t g = (n + block - 1) / block;
  if (g < 1) g = 1;
  if (g > (size_t)max_blocks) g = max_blocks;
  return (int)g;
}
inline int norm_threads(int cols) {
  int t = ((cols / 8 + 31) / 32) * 32;
  if (t < 32) t = 32;
  if (t > 256) t = 256;
  return t;
}

// ---- GEMM (CUDA cores) ----------------------------------------------------------
inline void launch_gemm_simt(cudaStream_t st, int dtype, const GemmArgs& g) {
  if ((int64_t)g.M * g.N <= 1024 && g.K >= 256) {      // few outputs, long k: one warp per output
    const unsigned blocks = (unsigned)(((int64_t)g.M * g.N + 7) / 8);
#define HIFT_FEW(TI, TO, BIAS, RES, LDR)                                                                                  \
  gemm_few_outputs_kernel<TI, TO><<<blocks, 256, 0, st>>>(g.M, g.N, g.K, (const TI*)g.a, g.sam, g.sak, (const TI*)g.b, g.sbk, \
                                                          g.sbn, (TO*)g.c, g.ldc, (const TI*)BIAS, RES, LDR)
    if (dtype == 0) HIFT_FEW(float, float, g.bias, g.residual, g.ldr);
    else if (g.out_f32) HIFT_FEW(bf16, float, g.bias, g.residual, g.ldr);
    else HIFT_FEW(bf16, bf16, g.bias, nullptr, 0);
#undef HIFT_FEW
    return;
  }
  dim3 grid((g.N + 63) / 64, (g.M + 63) / 64);
  if (dtype == 0) {
    gemm_simt_kernel<float, float><<<grid, 256, 0, st>>>(
        g.M, g.N, g.K, (const float*)g.a, g.sam, g.sak, (const float*)g.b, g.sbk, g.sbn,
        (float*)g.c, g.ldc, (const float*)g.bias, g.residual, g.ldr);
  } else if (g.out_f32) {
    gemm_simt_kernel<bf16, float><<<grid, 256, 0, st>>>(
        g.M, g.N, g.K, (const bf16*)g.a, g.sam, g.sak, (const bf16*)g.b, g.sbk, g.sbn,
        (float*)g.c, g.ldc, (const bf16*)g.bias, g.residual, g.ldr);
  } else {
    gemm_simt_kernel<bf16, bf16><<<grid, 256, 0, st>>>(
        g.M, g.N, g.K, (const bf16*)g.a, g.sam, g.sak, (const bf16*)g.b, g.sbk, g.sbn,
        (bf16*)g.c, g.ldc, (const bf16*)g.bias, nullptr, 0);
  }
}

// ---- attention ------------------------------------------------------------------
inline bool attention_head_ok(int dh) { return dh == 8 || dh == 16 || dh == 32 || dh == 64 || dh == 128; }

template <typename T, int DH>
inline void attention_fwd_inst(cudaStream_t st, int B, int S, int H, int causal, const void* qkv,
                               void* o, float* lse, const int* lens, const DropArgs& da) {
  dim3 grid((S + kAttRows - 1) / kAttRows, H, B);
  attention_fwd_kernel<T, DH><<<grid, 256, 0, st>>>((const T*)qkv, (T*)o, lse, S, H, causal,
                                                    1.0f / sqrtf((float)DH), lens, da);
}
template <typename T, int DH>
inline void attention_bwd_inst(cudaStream_t st, int B, int S, int H, int causal, const void* qkv,
                               const void* o, const float* lse, const void* dout, void* dqkv,
                               float* dsum, const int* lens, const DropArgs& da) {
  dim3 grid((S + kAttRows - 1) / kAttRows, H, B);
  const float scale = 1.0f / sqrtf((float)DH);
  attention_bwd_dq_kernel<T, DH><<<grid, 256, 0, st>>>((const T*)qkv, (const T*)o, lse,
                                                       (const T*)dout, (T*)dqkv, dsum, S, H, causal, scale, lens, da);
  attention_bwd_dkv_kernel<T, DH><<<grid, 256, 0, st>>>((const T*)qkv, lse, (const T*)dout, dsum,
                                                        (T*)dqkv, S, H, causal, scale, lens, da);
}
#define HIFT_DH_SWITCH(dh, CALL)            \
  switch (dh) {                             \
    case 8: { CALL(8); break; }             \
    case 16: { CALL(16); break; }           \
    case 32: { CALL(32); break; }           \
    case 64: { CALL(64); break; }           \
    case 128: { CALL(128); break; }         \
    default: break;                         \
  }
// bf16 with head size 64 or 128 goes to the tensor-core kernels
inline bool attention_use_mma(int dtype, int dh) { return dtype == 1 && (dh == 64 || dh == 128); }
template <int DH>
inline void attention_mma_fwd(cudaStream_t st, int B, int S, int H, int causal, const void* qkv, void* o, float* lse,
                              const int* lens) {
  static bool attr_set = false;
  if (!attr_set) {
    cudaFuncSetAttribute(attn_fwd_mma_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn_fwd_smem_bytes<DH>());
    cudaFuncSetAttribute(attn_fwd_mma_kernel<DH>, cudaFuncAttributePreferredSharedMemoryCarveout, 100);   // three CTAs per SM
    attr_set = true;
  }
  dim3 grid((S + 63) / 64, H, B);
  attn_fwd_mma_kernel<DH><<<grid, 128, attn_fwd_smem_bytes<DH>(), st>>>((const bf16*)qkv, (bf16*)o, lse, S, H, causal,
                                                                       1.0f / sqrtf((float)DH), lens);
}
template <int DH>
inline void attention_mma_bwd(cudaStream_t st, int B, int S, int H, int causal, const void* qkv, const void* o,
                              const float* lse, const void* dout, void* dqkv, float* dsum, const int* lens) {
  static bool attr_set = false;
  if (!attr_set) {
    cudaFuncSetAttribute(attn_bwd_dkv_mma_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn_dkv_smem_bytes<DH>());
    cudaFuncSetAttribute(attn_bwd_dkv_mma_kernel<DH>, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
    cudaFuncSetAttribute(attn_bwd_dq_mma_kernel<DH>, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
    attr_set = true;
  }
  const float scale = 1.0f / sqrtf((float)DH);
  launch_attn_dsum(st, (const bf16*)o, (const bf16*)dout, dsum, B, S, H, DH);
  dim3 grid((S + 63) / 64, H, B);
  attn_bwd_dq_mma_kernel<DH><<<grid, 128, 0, st>>>((const bf16*)qkv, lse, (const bf16*)dout, dsum, (bf16*)dqkv, S, H, causal, scale, lens);
  attn_bwd_dkv_mma_kernel<DH><<<grid, 128, attn_dkv_smem_bytes<DH>(), st>>>((const bf16*)qkv, lse, (const bf16*)dout, dsum,
                                                                           (bf16*)dqkv, S, H, causal, scale, lens);
}
// `da` (thr != 0): dropout on the probabilities (dropout_rng.cuh).  The CUDA-core kernels take it for every type and
// head size, the tcgen05 kernels for theirs; the warp-level kernels do not, so a dropped bf16 launch they would have
// got (tcgen05 switched off, or operands that are not 16-byte aligned) goes to the CUDA-core kernels.
inline void launch_attention_fwd(cudaStream_t st, int dtype, int B, int S, int H, int dh, int causal,
                                 const void* qkv, void* o, float* lse, const int* lens = nullptr,
                                 const DropArgs& da = DropArgs{0u, 0u, 0u, 0u, 0u, 1.0f}) {
  if (attention_use_mma(dtype, dh) && gemm_tc_init() == 0 && attn_tc_eligible(dh, qkv, H)) {        // tcgen05 kernel
    attn_tc_fwd_launch(st, B, S, H, dh, causal, qkv, o, lse, lens, da);
    return;
  }
  if (attention_use_mma(dtype, dh) && da.thr == 0u) {
    if (dh == 64) attention_mma_fwd<64>(st, B, S, H, causal, qkv, o, lse, lens);
    else attention_mma_fwd<128>(st, B, S, H, causal, qkv, o, lse, lens);
    return;
  }
#define CALL_F(D)                                                              \
  if (dtype == 0) attention_fwd_inst<float, D>(st, B, S, H, causal, qkv, o, lse, lens, da); \
  else attention_fwd_inst<bf16, D>(st, B, S, H, causal, qkv, o, lse, lens, da)
  HIFT_DH_SWITCH(dh, CALL_F)
#undef CALL_F
}
inline void launch_attention_bwd(cudaStream_t st, int dtype, int B, int S, int H, int dh, int causal,
                                 const void* qkv, const void* o, const float* lse, const void* dout,
                                 void* dqkv, float* dsum, const int* lens = nullptr,
                                 const DropArgs& da = DropArgs{0u, 0u, 0u, 0u, 0u, 1.0f}) {
  if (attention_use_mma(dtype, dh) && gemm_tc_init() == 0 && attn_tc_bwd_eligible(dh, H, qkv, dout, dqkv) &&
      (((uintptr_t)o) & 15) == 0) {                                                                   // tcgen05 kernels
    launch_attn_dsum(st, (const bf16*)o, (const bf16*)dout, dsum, B, S, H, dh);
    attn_tc_bwd_launch(st, B, S, H, dh, causal, qkv, dout, lse, dsum, dqkv, lens, da);
    return;
  }
  if (attention_use_mma(dtype, dh) && da.thr == 0u) {
    if (dh == 64) attention_mma_bwd<64>(st, B, S, H, causal, qkv, o, lse, dout, dqkv, dsum, lens);
    else attention_mma_bwd<128>(st, B, S, H, causal, qkv, o, lse, dout, dqkv, dsum, lens);
    return;
  }
#define CALL_B(D)                                                                              \
  if (dtype == 0) attention_bwd_inst<float, D>(st, B, S, H, causal, qkv, o, lse, dout, dqkv, dsum, lens, da); \
  else attention_bwd_inst<bf16, D>(st, B, S, H, causal, qkv, o, lse, dout, dqkv, dsum, lens, da)
  HIFT_DH_SWITCH(dh, CALL_B)
#undef CALL_B
}

// ---- norms ----------------------------------------------------------------------
// dtype 0: parameters fp32; 1: parameters / GEMM operands bf16.  x and y_r are fp32.
inline void launch_norm_fwd(cudaStream_t st, int dtype, int kind, int64_t rows, int cols, float eps,
                            const float* x, const void* gain, const void* bias, void* y_a, float* y_r,
                            float* stats) {
  const int th = norm_threads(cols);
  const int nc = (cols / 8 + th - 1) / th;            // chunks of 8 per thread: rows up to 8192 wide stay in registers
#define NFR(P, K, NC) launch_pdl(norm_fwd_reg_kernel<P, K, NC>, dim3((unsigned)rows), dim3(th), 0, st, x, (const P*)gain, (const P*)bias, (P*)y_a, y_r, stats, rows, cols, eps)
#define NF(P, K)                                                                                                   \
  do {                                                                                                             \
    if (nc <= 1) NFR(P, K, 1); else if (nc == 2) NFR(P, K, 2); else if (nc <= 4) NFR(P, K, 4);                      \
    else launch_pdl(norm_fwd_kernel<P, K>, dim3((unsigned)rows), dim3(th), 0, st, x, (const P*)gain, (const P*)bias, (P*)y_a, y_r, stats, rows, cols, eps); \
  } while (0)
  if (dtype == 0) { if (kind == 0) NF(float, 0); else NF(float, 1); }
  else { if (kind == 0) NF(bf16, 0); else NF(bf16, 1); }
#undef NF
#undef NFR
}
// dy_f32: dy is an fp32 stream gradient (else it has the operand type)
inline void launch_norm_bwd_dx(cudaStream_t st, int dtype, int kind, bool dy_f32, int64_t rows, int cols,
                               const void* dy, const float* x, const float* stats, const void* gain,
                               const float* add, float* dx_r, void* dx_a) {
  const int th = norm_threads(cols);
#define NB(DY, P, K) launch_pdl(norm_bwd_dx_kernel<DY, P, K>, dim3((unsigned)rows), dim3(th), 0, st, (const DY*)dy, x, stats, (const P*)gain, add, dx_r, (P*)dx_a, rows, cols)
  if (dtype == 0) { if (kind == 0) NB(float, float, 0); else NB(float, float, 1); }
  else if (dy_f32) { if (kind == 0) NB(float, bf16, 0); else NB(float, bf16, 1); }
  else { if (kind == 0) NB(bf16, bf16, 0); else NB(bf16, bf16, 1); }
#undef NB
}
// mode 0: out0 = colsum(dy) ; 1: out0 = sum dy*xhat, out1 = sum dy ; 2: out0 = sum dy*x*rstd
// dy_bf16: dy has type bf16 (else fp32); x is fp32.
inline int colreduce_chunks(int64_t rows) {
  int c = (int)((rows + 31) / 32);
  if (c < 1) c = 1;
  if (c > kColChunks) c = kColChunks;
  return c;
}
inline void launch_colreduce(cudaStream_t st, bool dy_bf16, int mode, int64_t rows, int cols,
                             const void* dy, int64_t ld, const float* x, const float* stats,
                             float* partial, void* out0, void* out1, int out_bf16 = 0) {
  const int nch = colreduce_chunks(rows);
  dim3 grid((cols + 31) / 32, nch), block(32, 8);
#define CR(T, M) colreduce_stage1_kernel<T, M><<<grid, block, 0, st>>>((const T*)dy, ld, x, stats, partial, rows, cols)
  if (!dy_bf16) { if (mode == 0) CR(float, 0); else if (mode == 1) CR(float, 1); else CR(float, 2); }
  else { if (mode == 0) CR(bf16, 0); else if (mode == 1) CR(bf16, 1); else CR(bf16, 2); }
#undef CR
  colreduce_stage2_kernel<<<(cols + 127) / 128, 128, 0, st>>>(partial, nch, cols, out0,
                                                             mode == 1 ? out1 : nullptr, out_bf16);
}

// ---- cross-entropy --------------------------------------------------------------
inline void launch_cross_entropy(cudaStream_t st, int dtype, int64_t rows, int64_t vocab, int64_t ld,
                                 void* logits, const int32_t* labels, float* rowloss, int* nvalid,
                                 int* bad, float* loss) {
  count_valid_kernel<<<1, 256, 0, st>>>(labels, rows, nvalid);
  const int th = vocab >= 4096 ? 512 : (vocab >= 256 ? 128 : 32);
  const bool vec = (((uintptr_t)logits) & 15) == 0 && ld % (dtype == 0 ? 4 : 8) == 0;     // 16-byte rows
  if (dtype == 0) {
    if (vec) cross_entropy_vec_kernel<float><<<(unsigned)rows, th, 0, st>>>((float*)logits, labels, rowloss, nvalid, bad, vocab, ld);
    else cross_entropy_kernel<float><<<(unsigned)rows, th, 0, st>>>((float*)logits, labels, rowloss, nvalid, bad, vocab, ld);
  } else {
    if (vec) cross_entropy_vec_kernel<bf16><<<(unsigned)rows, th, 0, st>>>((bf16*)logits, labels, rowloss, nvalid, bad, vocab, ld);
    else cross_entropy_kernel<bf16><<<(unsigned)rows, th, 0, st>>>((bf16*)logits, labels, rowloss, nvalid, bad, vocab, ld);
  }
  loss_reduce_kernel<<<1, 256, 0, st>>>(rowloss, rows, nvalid, loss);
}

// ---- optimizer ------------------------------------------------------------------
inline OptScalars make_opt_scalars(int kind, double lr, double b1, double b2, double eps, double wd,
                                   double mu, int64_t tau) {
  OptScalars h;
  h.lr = (float)lr; h.beta1 = (float)b1; h.beta2 = (float)b2; h.eps = (float)eps;
  h.decay = (float)(1.0 - lr * wd);
  h.omb1 = (float)(1.0 - b1); h.omb2 = (float)(1.0 - b2);
  h.c1 = 1.f; h.c2 = 1.f;
  if (kind == 0) {
    h.c1 = (float)(1.0 / (1.0 - pow(b1, (double)tau)));
    h.c2 = (float)(1.0 / (1.0 - pow(b2, (double)tau)));
  }
  h.mu = (float)mu;
  return h;
}
// grad_bf16: the gradient buffer holds bf16 elements (else fp32)
inline void launch_fused_opt(cudaStream_t st, int kind, size_t n, void* param_bf16, float* master,
                             const void* grad, float* s0, float* s1, const OptScalars& h,
                             const int* gate = nullptr, bool grad_bf16 = false) {
  if (n == 0) return;
  const int block = 256;
  int grid = grid_for((n + 3) / 4, block, 148 * 8);
#define OPTG(K, GT)                                                                                    \
  if (param_bf16) fused_opt_kernel<K, true, GT><<<grid, block, 0, st>>>((bf16*)param_bf16, master, (const GT*)grad, s0, s1, n, h, gate); \
  else fused_opt_kernel<K, false, GT><<<grid, block, 0, st>>>(nullptr, master, (const GT*)grad, s0, s1, n, h, gate)
#define OPT(K) if (grad_bf16) { OPTG(K, bf16); } else { OPTG(K, float); }
  if (kind == 0) { OPT(0) } else if (kind == 1) { OPT(1) } else if (kind == 2) { OPT(2) } else { OPT(3) }
#undef OPT
#undef OPTG
}

// compact master (bf16 copy + low halves + carry bits); n must be a multiple of 8
inline void launch_fused_opt_compact(cudaStream_t st, int kind, size_t n, void* param_bf16, uint16_t* lo16, uint8_t* carry8,
                                     const void* grad, float* s0, float* s1, const OptScalars& h,
                                     const int* gate = nullptr, bool grad_bf16 = false) {
  if (n == 0) return;
  const size_t n8 = n / 8;
  const int grid = grid_for(n8, 256, 148 * 8);
#define OPTC(K)                                                                                                                              \
  if (grad_bf16) fused_opt_compact_kernel<K, bf16><<<grid, 256, 0, st>>>((uint16_t*)param_bf16, lo16, carry8, (const bf16*)grad, s0, s1, n8, h, gate); \
  else fused_opt_compact_kernel<K, float><<<grid, 256, 0, st>>>((uint16_t*)param_bf16, lo16, carry8, (const float*)grad, s0, s1, n8, h, gate)
  if (kind == 0) { OPTC(0); } else if (kind == 1) { OPTC(1); } else if (kind == 2) { OPTC(2); } else { OPTC(3); }
#undef OPTC
}

}  // namespace hift
