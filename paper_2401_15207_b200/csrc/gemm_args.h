// Operand description shared by the CUDA-core and the tensor-core GEMM launchers.
#pragma once
#include <stdint.h>

namespace hift {

//   C[m,n] = sum_k A(m,k) * B(k,n) (+ bias[n]) (+ residual[m,n]),
//   A(m,k) = a[m*sam + k*sak],  B(k,n) = b[k*sbk + n*sbn].
struct GemmArgs {
  int M, N, K;
  const void* a; int64_t sam, sak;
  const void* b; int64_t sbk, sbn;
  void* c; int64_t ldc;
  const void* bias;                    // operand type, [N]
  const float* residual; int64_t ldr;  // fp32 (the residual stream); only with out_f32
  bool out_f32;          // bf16 operands, fp32 output (weight gradients, residual stream)
  // Optional rotary embedding applied to the output before it is stored (the q and k column
  // blocks of a fused qkv projection): columns [0, rope_cols) are heads of rope_dh columns whose
  // pair (j, j + rope_dh/2) is rotated by the angle of (row mod rope_seq, j).  rope_cs: fp32
  // [rope_seq, rope_dh/2] cosines followed by [rope_seq, rope_dh/2] sines; nullptr = none.
  const float* rope_cs = nullptr;
  int rope_seq = 0, rope_dh = 0;
  int64_t rope_cols = 0;
  // Optional gated activation applied to the output (a fused gate | up projection, N = 2f): besides
  // (or, with c == nullptr, instead of) c[m, 0..2f), the epilogue stores
  //     swiglu_out[m, j] = silu(y[m, j]) * y[m, f + j],  j < f,   as bf16 with leading dimension f.
  void* swiglu_out = nullptr;
  // Optional backward of that activation applied to the output of the down projection's dX product
  // (y = ds[M, f], N = f): instead of ds the epilogue stores, into c[M, 2f] (ldc = 2f),
  //     c[m, j]     = ds * up * sig * (1 + gate * (1 - sig)),   sig = sigmoid(gate)
  //     c[m, f + j] = ds * gate * sig
  // with gate = swiglu_bwd_gu[m, j], up = swiglu_bwd_gu[m, f + j] (the saved pre-activations, bf16).
  const void* swiglu_bwd_gu = nullptr;
  // GELU (exact, erf) blocks: the same two fusions for the plain feed-forward.
  //   gelu_out (forward form): besides (or, with c == nullptr, instead of) the pre-activation y in c, the
  //   epilogue stores gelu_out[m, n] = gelu(y[m, n]) as bf16 with leading dimension N.
  //   gelu_bwd_a (dX form): the output is multiplied by gelu'(a[m, n]), a = the saved pre-activation (bf16, ld N).
  void* gelu_out = nullptr;
  const void* gelu_bwd_a = nullptr;
};

}  // namespace hift
