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
};

}  // namespace hift
