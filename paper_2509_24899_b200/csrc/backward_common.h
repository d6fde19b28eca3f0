// Shared by the two implementations of the gradient w.r.t. the feature-map weights (CUDA cores / tensor cores):
// the launch parameters and the entry points of the tensor-core kernels.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

struct BwParams {
  const __nv_bfloat16 *q, *k, *v, *wq, *wk, *y, *yhat;
  const float *aux, *S, *z;          // forward results: aux [BH][N][3], S [BH][F][D], z [BH][F]
  const __nv_bfloat16* Sb;           // S once more in bf16 (the forward pass's MMA operand)
  const int32_t* sm_rank;
  float *part_dS, *part_dz, *part_dW, *part_loss;     // per (bh, chunk)
  float *dS, *dz;                    // [BH][F][D], [BH][F]
  __nv_bfloat16* dSb;                // dS once more in bf16 (the key side's MMA operand)
  uint32_t* status;                  // device status word of the handle (bounded waits)
  float *dWq, *dWk, *loss;           // outputs: [H][F][D] each, one float (may be NULL)
  int B, H, N, P, n_s, stab_mode, chunks, chunk_tokens;
};


// Tensor-core kernels (d = F = 128): query side (partial dS, dz, dW_q, loss per token chunk) and key side
// (partial dW_k); chunk_tokens must be a multiple of 128.
cudaError_t as_bw_tensor_init();
cudaError_t as_bw_tensor_query(const BwParams& p, cudaStream_t st);
cudaError_t as_bw_tensor_key(const BwParams& p, cudaStream_t st);
