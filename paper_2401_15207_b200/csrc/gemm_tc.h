// Tensor-core (tcgen05 / TMEM / TMA) bf16 GEMM: host interface.
#pragma once
#include <cuda_runtime.h>

#include "dropout_rng.cuh"
#include "gemm_args.h"

namespace hift {

// Resolves the driver entry point used to encode TMA descriptors and opts the kernels into
// large dynamic shared memory.  0 on success; anything else means the tensor-core path is
// unavailable and gemm_tc_eligible() answers false.
int gemm_tc_init();
// True when the operands are bf16 in one of the three supported major-ness combinations,
// 16-byte aligned with 16-byte-multiple leading dimensions.
bool gemm_tc_eligible(const GemmArgs& g);
cudaError_t gemm_tc_launch(cudaStream_t st, const GemmArgs& g);
// Attention forward on tcgen05 (scores and output in tensor memory): bf16, head size 64 or 128.
// `lens` (device, [B], may be null): batch entry b attends to its first lens[b] keys only.
bool attn_tc_eligible(int dh, const void* qkv, int H);
// `da` (thr != 0): dropout on the probabilities (dropout_rng.cuh).
cudaError_t attn_tc_fwd_launch(cudaStream_t st, int B, int S, int H, int dh, int causal, const void* qkv, void* o, float* lse,
                               const int* lens, const DropArgs& da);
// Attention backward on tcgen05 (two launches: dK/dV, then dQ): bf16, head size 64 or 128.  `dsum` holds
// rowsum(dO o O) per (batch, head, query); qkv, dout and dqkv must be 16-byte aligned.
bool attn_tc_bwd_eligible(int dh, int H, const void* qkv, const void* dout, const void* dqkv);
cudaError_t attn_tc_bwd_launch(cudaStream_t st, int B, int S, int H, int dh, int causal, const void* qkv, const void* dout,
                               const float* lse, const float* dsum, void* dqkv, const int* lens, const DropArgs& da);
// Code-path switches for A/B timing and for tests (all 1 by default = the fast path): which = 0 CTA-pair
// GEMM tiles, 1 programmatic dependent launch, 2 tcgen05 attention forward, 3 tcgen05 attention backward.
// value >= 0 sets the switch; returns its previous value (-1: no such switch).  Process-wide; read at
// each launch.
int gemm_tc_switch(int which, int value);
// 0 if no tensor-core kernel has given up on a bounded wait since the library was loaded, else the
// code of the first one (1 producer, 2 MMA issuer, 3 epilogue); -1 if the flag cannot be read.
int gemm_tc_poll_error();
// Overwrites the flag (0 clears it).  While it is non-zero every tensor-core GEMM launch returns without
// computing, which is what a launch after a real time-out does.  0 on success.
int gemm_tc_set_error(int v);
// Device address of that flag (an int), or nullptr if it cannot be resolved.
const int* gemm_tc_error_device_ptr();

}  // namespace hift
