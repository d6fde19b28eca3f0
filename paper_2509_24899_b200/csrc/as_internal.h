// Internal declarations shared by the translation units of libas_hybrid_attn.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "as_hybrid_attn.h"

constexpr int AS_TILE = 128;            // tokens per tile in every kernel
constexpr int AS_MAX_PROFILE = 1024;    // event pairs kept between two profile reads

// Byte offsets of the workspace segments (all multiples of 256).
struct as_ws_layout {
  size_t ks = 0, vs = 0;                // compacted softmax K / V   [B*H, N_S, d] bf16
  size_t part_s = 0, part_z = 0;        // per-chunk partial state   [B*H, chunks, F, d] / [.., F] fp32
  size_t S = 0, z = 0;                  // final state               [B*H, F, d] / [B*H, F] fp32
  size_t Sb = 0;                        // S rounded to bf16         [B*H, F, d] (MMA operand of the Q pass)
  size_t h1k = 0;                       // first-layer activations of the keys [B*H, N, hidden] bf16 (two-layer feature map only)
  size_t total = 0;
  size_t stage_q = 0, stage_k = 0, stage_v = 0, stage_o = 0, total_host = 0;
};

// Everything a kernel launch needs, resolved to device pointers.
struct as_launch_args {
  const __nv_bfloat16 *q, *k, *v, *wq, *wk;
  const __nv_bfloat16 *wq2, *wk2;       // second feature-map layer [H, F, hidden] (NULL for a one-layer map)
  const __nv_bfloat16 *bq1, *bk1, *bq2, *bk2;   // biases [H, width of the layer's output] (each may be NULL)
  __nv_bfloat16* h1k;                   // relu(k W_k1^T + b_k1) [B*H, N, hidden] when the map has two layers
  int layers;                           // depth of the feature map's embedding network (1 or 2)
  int hid;                              // hidden width of a two-layer map (0 otherwise)
  __nv_bfloat16* out;
  float* aux;
  const __nv_bfloat16 *ks, *vs;         // softmax keys / values the Q pass reads (k, v themselves at R = 1)
  __nv_bfloat16 *ks_w, *vs_w;           // where the K pass writes the compacted rows (NULL at R = 1)
  float *part_s, *part_z, *S, *z;
  __nv_bfloat16* Sb;
  const int32_t* sm_rank;               // [N]: position in T_S, or -1 for a linear token
  uint32_t* status;                     // device status word
  uint32_t* counters;                   // [B*H*4][2], zero between launches: K-pass CTAs of a (batch, head, feature chunk)
                                        // that have stored their partial state / that have added their slice up
  int B, H, N, d, F, P;
  int n_s, n_l;
  int n_chunks, chunk_tiles;            // K-pass split of the token axis
  float scale;
  int stab_mode;
};

struct as_hybrid_attn_s {
  as_hybrid_attn_desc_t desc;
  int device = -1;
  int n_s = 0, n_l = 0;
  float scale = 0.f;
  std::vector<int32_t> idx_host;        // sorted T_S
  int32_t* d_sm_rank = nullptr;
  uint32_t* d_status = nullptr;
  uint32_t* d_counters = nullptr;       // arrival counters of the K pass (cf. as_launch_args::counters)
  int n_chunks = 1, chunk_tiles = 1;
  as_ws_layout ws;
  uint64_t launches = 0;
  // profiling
  bool profiling = false;
  std::vector<cudaEvent_t> ev;          // 2 * AS_MAX_PROFILE events, created on first enable
  std::vector<int> ev_class;
  int ev_used = 0;
  // forward_host: side streams for the copies in and out, created on its first call
  bool side_ready = false;
  cudaStream_t s_in = nullptr, s_out = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  std::vector<cudaEvent_t> ev_run;      // per run of heads: inputs landed, kernels done
};

// Kernel launchers.  Each returns the launch's cudaError_t.
cudaError_t as_simt_kpass(const as_launch_args& a, cudaStream_t st);
cudaError_t as_simt_qpass(const as_launch_args& a, cudaStream_t st);
cudaError_t as_reduce_state(const as_launch_args& a, cudaStream_t st);
// Sb = bf16(S) for a state that came from outside (the Q pass reads S as a bf16 operand).
cudaError_t as_round_state(const as_launch_args& a, cudaStream_t st);
cudaError_t as_tensor_kpass(const as_launch_args& a, cudaStream_t st);
cudaError_t as_tensor_qpass(const as_launch_args& a, cudaStream_t st);
// Query stage of layers without softmax tokens in its streaming form (one-layer map, F = d = 128, no bias, degree
// <= 2): whether it covers the launch, and the launch itself.  as_tensor_qpass dispatches to it.
bool as_tensor_qstream_handles(const as_launch_args& a);
cudaError_t as_tensor_qstream(const as_launch_args& a, cudaStream_t st);
// First layer of a two-layer feature map for the keys: h1k = relu(k W_k1^T + b_k1).
cudaError_t as_tensor_phi1(const as_launch_args& a, cudaStream_t st);
// One-time set-up of the tensor path on the current device (driver entry points, smem opt-in).
cudaError_t as_tensor_init();

// Test aid: a kernel whose bounded wait (the one every kernel here uses) runs out after `limit_cycles`.
cudaError_t as_tensor_expire_wait(uint32_t* status, long long limit_cycles, cudaStream_t st);

// Status bits written by kernels into as_launch_args::status.
constexpr uint32_t AS_DEV_TIMEOUT = 1u;
