// Gradient of the value-distillation loss L = sum |y - y_hat| ("Attention Distillation", value-distillation
// loss; Algorithm 1 updates the feature maps only) w.r.t. the feature-map weights W_q, W_k of one hybrid
// attention layer, in fp32 on CUDA cores: one-layer feature maps with F == d and no bias.  (With d = F = 128 on the tensor
// path the products run on the tensor cores instead, backward_tensor.cu; this file keeps the reductions, the layout
// of the partial results and the entry points.)
//
// With y_hat_i = num_i / den_i, num_i = N_i + lambda_i phi_q,i S, den_i = D_i + lambda_i phi_q,i . z (N_i, D_i: the
// softmax branch, independent of the weights) the chain rule gives, per (batch, head):
//     G_i = sign(y_hat_i - y_i),  g_i = G_i / den_i,  s_i = -(G_i . y_hat_i) / den_i
//     dL/dphi_q,i = lambda_i (S g_i + z s_i)         dL/dS = sum_i lambda_i phi_q,i^T g_i    dL/dz = sum_i lambda_i phi_q,i s_i
//     dL/dphi_k,j = (dL/dS) v_j + dL/dz  (linear tokens j)
//     dL/da = dL/dphi * p r^(p-1) [a > 0]            dL/dW_q = sum_i (dL/da_q,i)^T q_i       dL/dW_k = sum_j (dL/da_k,j)^T k_j
// The forward pass supplies y_hat, aux = (c_i, D_i, phi_q,i . z) and S, z (in its workspace).
//
// Three launches: the query side (per token chunk: partial dL/dS, dL/dz, dL/dW_q, loss), a fixed-order reduction,
// and the key side (partial dL/dW_k) with its reduction.  No float atomics: results are run-to-run identical.
#include <algorithm>

#include "as_internal.h"
#include "backward_common.h"

namespace {

constexpr int BW_THREADS = 512;
constexpr int BW_TOK = 16;            // tokens per step

__device__ __forceinline__ float bf2f(__nv_bfloat16 x) { return __bfloat162float(x); }

// phi = r^p and its slope p r^(p-1) for r = relu(a), p = 1 + (index of the feature's part)
__device__ __forceinline__ void poly(float a, int p, float& phi, float& slope) {
  const float r = fmaxf(a, 0.f);
  float rp1 = 1.f;                   // r^(p-1)
  for (int i = 1; i < p; ++i) rp1 *= r;
  phi = rp1 * r;
  slope = a > 0.f ? (float)p * rp1 : 0.f;
}

// Shared-memory layout of both kernels: two [F][D+1] matrices, a vector [F], and per-step token data.
template <int D>
struct BwSmem {
  static constexpr int F = D;
  static constexpr int MAT = F * (D + 1);
  static constexpr size_t FLOATS = 2 * MAT + F + 2 * BW_TOK * D + 2 * BW_TOK * F + 2 * BW_TOK;
  static constexpr size_t BYTES = FLOATS * sizeof(float);
};

// Query side.  One CTA per (token chunk, batch*head).
template <int D>
__global__ void __launch_bounds__(BW_THREADS, 1) bw_query_kernel(BwParams p) {
  constexpr int F = D;
  using SM = BwSmem<D>;
  extern __shared__ float smem[];
  float* sW = smem;                          // W_q   [F][D+1]
  float* sS = sW + SM::MAT;                  // S     [F][D+1]
  float* sz = sS + SM::MAT;                  // z     [F]
  float* sQ = sz + F;                        // q rows of the step      [TOK][D]
  float* sG = sQ + BW_TOK * D;               // g = G / den             [TOK][D]
  float* sPhi = sG + BW_TOK * D;             // lambda phi_q            [TOK][F]
  float* sU = sPhi + BW_TOK * F;             // dL/da_q                 [TOK][F]
  float* sSc = sU + BW_TOK * F;              // s_i, lambda_i           [2][TOK]
  __shared__ float sLoss[BW_THREADS / 32];

  const int bh = blockIdx.y, chunk = blockIdx.x, tid = threadIdx.x, h = bh % p.H;
  const int warp = tid / 32, lane = tid % 32;
  const int part_width = F / p.P;
  const __nv_bfloat16* W = p.wq + (size_t)h * F * D;
  const float* Sg = p.S + (size_t)bh * F * D;
  for (int i = tid; i < F * D; i += BW_THREADS) {
    sW[(i / D) * (D + 1) + (i % D)] = bf2f(W[i]);
    sS[(i / D) * (D + 1) + (i % D)] = Sg[i];
  }
  for (int i = tid; i < F; i += BW_THREADS) sz[i] = p.z[(size_t)bh * F + i];

  constexpr int TPR = BW_THREADS / F;        // threads per feature row of the accumulators
  constexpr int COLS = D / TPR;
  const int f_own = tid / TPR, c0 = (tid % TPR) * COLS;
  float accS[COLS], accW[COLS];
#pragma unroll
  for (int c = 0; c < COLS; ++c) { accS[c] = 0.f; accW[c] = 0.f; }
  float accz = 0.f, loss = 0.f;

  const int tok_begin = chunk * p.chunk_tokens;
  const int tok_end = min(p.N, tok_begin + p.chunk_tokens);
  const size_t row0 = (size_t)bh * p.N;
  __syncthreads();

  for (int t0 = tok_begin; t0 < tok_end; t0 += BW_TOK) {
    // one warp per token: q, g = sign(y_hat - y) / den, s = -(G . y_hat) / den, lambda
    if (warp < BW_TOK) {
      const int n = t0 + warp;
      const bool in = n < tok_end;
      float lam = 1.f, den = 1.f;
      if (in) {
        const float* ap = p.aux + (row0 + n) * 3;
        if (p.stab_mode == AS_STAB_EXACT && p.n_s > 0) lam = __expf(-ap[0]);
        den = ap[1] + lam * ap[2];
      }
      float sdot = 0.f;
      for (int dd = lane; dd < D; dd += 32) {
        float qv = 0.f, gv = 0.f;
        if (in) {
          const size_t o = (row0 + n) * D + dd;
          const float yh = bf2f(p.yhat[o]), yt = bf2f(p.y[o]);
          const float diff = yh - yt;
          const float G = diff > 0.f ? 1.f : (diff < 0.f ? -1.f : 0.f);
          qv = bf2f(p.q[o]);
          gv = G / den;
          sdot += G * yh;
          loss += fabsf(diff);
        }
        sQ[warp * D + dd] = qv;
        sG[warp * D + dd] = gv;
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) sdot += __shfl_xor_sync(0xffffffffu, sdot, off);
      if (lane == 0) { sSc[warp] = in ? -sdot / den : 0.f; sSc[BW_TOK + warp] = in ? lam : 0.f; }
    }
    __syncthreads();
    // per (token, feature): a = W_q[f] . q, phi, slope; U = lambda (S[f] . g + z[f] s) slope
    for (int i = tid; i < BW_TOK * F; i += BW_THREADS) {
      const int tt = i / F, f = i % F;
      float a = 0.f, u = 0.f;
#pragma unroll 8
      for (int dd = 0; dd < D; ++dd) {
        a = fmaf(sW[f * (D + 1) + dd], sQ[tt * D + dd], a);
        u = fmaf(sS[f * (D + 1) + dd], sG[tt * D + dd], u);
      }
      float phi, slope;
      poly(a, f / part_width + 1, phi, slope);
      const float lam = sSc[BW_TOK + tt];
      sPhi[i] = lam * phi;
      sU[i] = lam * (u + sz[f] * sSc[tt]) * slope;
    }
    __syncthreads();
#pragma unroll 4
    for (int tt = 0; tt < BW_TOK; ++tt) {
      const float ph = sPhi[tt * F + f_own], uu = sU[tt * F + f_own];
      if (c0 == 0) accz = fmaf(ph, sSc[tt], accz);
#pragma unroll
      for (int c = 0; c < COLS; ++c) {
        accS[c] = fmaf(ph, sG[tt * D + c0 + c], accS[c]);
        accW[c] = fmaf(uu, sQ[tt * D + c0 + c], accW[c]);
      }
    }
    __syncthreads();
  }
  const size_t slot = (size_t)bh * p.chunks + chunk;
  float* ps = p.part_dS + (slot * F + f_own) * D + c0;
  float* pw = p.part_dW + (slot * F + f_own) * D + c0;
#pragma unroll
  for (int c = 0; c < COLS; ++c) { ps[c] = accS[c]; pw[c] = accW[c]; }
  if (c0 == 0) p.part_dz[slot * F + f_own] = accz;
  // loss of the chunk: warp sums, then one thread adds the warps in order
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) loss += __shfl_xor_sync(0xffffffffu, loss, off);
  if (lane == 0) sLoss[warp] = loss;
  __syncthreads();
  if (tid == 0) {
    float l = 0.f;
    for (int w = 0; w < BW_THREADS / 32; ++w) l += sLoss[w];
    p.part_loss[slot] = l;
  }
}

// Key side.  One CTA per (token chunk, batch*head): partial dL/dW_k over the chunk's linear tokens.
template <int D>
__global__ void __launch_bounds__(BW_THREADS, 1) bw_key_kernel(BwParams p) {
  constexpr int F = D;
  using SM = BwSmem<D>;
  extern __shared__ float smem[];
  float* sW = smem;                          // W_k    [F][D+1]
  float* sdS = sW + SM::MAT;                 // dL/dS  [F][D+1]
  float* sdz = sdS + SM::MAT;                // dL/dz  [F]
  float* sK = sdz + F;                       // k rows [TOK][D]
  float* sV = sK + BW_TOK * D;               // v rows [TOK][D]
  float* sT = sV + BW_TOK * D;               // dL/da_k [TOK][F]
  __shared__ int sLin[BW_TOK];

  const int bh = blockIdx.y, chunk = blockIdx.x, tid = threadIdx.x, h = bh % p.H;
  const int part_width = F / p.P;
  const __nv_bfloat16* W = p.wk + (size_t)h * F * D;
  const float* dSg = p.dS + (size_t)bh * F * D;
  for (int i = tid; i < F * D; i += BW_THREADS) {
    sW[(i / D) * (D + 1) + (i % D)] = bf2f(W[i]);
    sdS[(i / D) * (D + 1) + (i % D)] = dSg[i];
  }
  for (int i = tid; i < F; i += BW_THREADS) sdz[i] = p.dz[(size_t)bh * F + i];

  constexpr int TPR = BW_THREADS / F;
  constexpr int COLS = D / TPR;
  const int f_own = tid / TPR, c0 = (tid % TPR) * COLS;
  float accW[COLS];
#pragma unroll
  for (int c = 0; c < COLS; ++c) accW[c] = 0.f;

  const int tok_begin = chunk * p.chunk_tokens;
  const int tok_end = min(p.N, tok_begin + p.chunk_tokens);
  const size_t row0 = (size_t)bh * p.N;
  __syncthreads();

  for (int t0 = tok_begin; t0 < tok_end; t0 += BW_TOK) {
    for (int i = tid; i < BW_TOK * D; i += BW_THREADS) {
      const int n = t0 + i / D;
      const bool in = n < tok_end;
      sK[i] = in ? bf2f(p.k[(row0 + n) * D + i % D]) : 0.f;
      sV[i] = in ? bf2f(p.v[(row0 + n) * D + i % D]) : 0.f;
    }
    if (tid < BW_TOK) sLin[tid] = (t0 + tid < tok_end) && p.sm_rank[t0 + tid] < 0;
    __syncthreads();
    for (int i = tid; i < BW_TOK * F; i += BW_THREADS) {
      const int tt = i / F, f = i % F;
      float a = 0.f, t = 0.f;
#pragma unroll 8
      for (int dd = 0; dd < D; ++dd) {
        a = fmaf(sW[f * (D + 1) + dd], sK[tt * D + dd], a);
        t = fmaf(sdS[f * (D + 1) + dd], sV[tt * D + dd], t);
      }
      float phi, slope;
      poly(a, f / part_width + 1, phi, slope);
      sT[i] = sLin[tt] ? (t + sdz[f]) * slope : 0.f;
    }
    __syncthreads();
#pragma unroll 4
    for (int tt = 0; tt < BW_TOK; ++tt) {
      const float tv = sT[tt * F + f_own];
#pragma unroll
      for (int c = 0; c < COLS; ++c) accW[c] = fmaf(tv, sK[tt * D + c0 + c], accW[c]);
    }
    __syncthreads();
  }
  const size_t slot = (size_t)bh * p.chunks + chunk;
  float* pw = p.part_dW + (slot * F + f_own) * D + c0;
#pragma unroll
  for (int c = 0; c < COLS; ++c) pw[c] = accW[c];
}

// Fixed-order sums.  stage 0 (after the query side): dS, dz per (batch, head); dW_q per head over batch and
// chunks; the loss.  stage 1 (after the key side): dW_k per head.
__global__ void bw_reduce_kernel(BwParams p, int D, int stage) {
  const int F = D;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;          // entry of an [F][D] matrix, then of an [F] vector
  const int bh = blockIdx.y;                                    // stage 0, blockIdx.z == 0: per (batch, head)
  if (stage == 0 && blockIdx.z == 0) {
    if (i < F * D) {
      const float* src = p.part_dS + (size_t)bh * p.chunks * F * D + i;
      float s = 0.f;
      int c = 0;
      for (; c + 4 <= p.chunks; c += 4) {                          // four loads in flight, added in chunk order
        float v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = __ldcg(src + (size_t)(c + j) * F * D);
#pragma unroll
        for (int j = 0; j < 4; ++j) s += v[j];
      }
      for (; c < p.chunks; ++c) s += __ldcg(src + (size_t)c * F * D);
      p.dS[(size_t)bh * F * D + i] = s;
      p.dSb[(size_t)bh * F * D + i] = __float2bfloat16_rn(s);      // the tensor-core key side's MMA operand
    } else if (i < F * D + F) {
      const int f = i - F * D;
      float s = 0.f;
      for (int c = 0; c < p.chunks; ++c) s += p.part_dz[((size_t)bh * p.chunks + c) * F + f];
      p.dz[(size_t)bh * F + f] = s;
    }
    return;
  }
  // blockIdx.z == 1, per head (blockIdx.y < H): sum over the batch, then over the chunks
  const int h = blockIdx.y;
  if (blockIdx.z != 1 || h >= p.H) return;
  float* out = stage == 0 ? p.dWq : p.dWk;
  if (i < F * D) {
    float s = 0.f;
    for (int b = 0; b < p.B; ++b) {
      const float* src = p.part_dW + (size_t)(b * p.H + h) * p.chunks * F * D + i;
      int c = 0;
      for (; c + 4 <= p.chunks; c += 4) {                          // four loads in flight, added in (batch, chunk) order
        float v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = __ldcg(src + (size_t)(c + j) * F * D);
#pragma unroll
        for (int j = 0; j < 4; ++j) s += v[j];
      }
      for (; c < p.chunks; ++c) s += __ldcg(src + (size_t)c * F * D);
    }
    out[(size_t)h * F * D + i] = s;
  }
  if (stage == 0 && h == 0 && i == 0 && p.loss != nullptr) {
    float l = 0.f;
    for (int s = 0; s < p.B * p.H * p.chunks; ++s) l += p.part_loss[s];
    *p.loss = l;
  }
}

size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

struct BwLayout { size_t part_dS, part_dz, part_dW, part_loss, dS, dz, dSb, total; int chunks, chunk_tokens; };

BwLayout bw_layout(const as_hybrid_attn_s* h) {
  const auto& d = h->desc;
  const size_t BH = (size_t)d.B * d.H, F = d.phi_dim, D = d.d;
  BwLayout L{};
  int sms = 148;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, h->device);
  // chunks of whole 128-token tiles (the tensor-core kernels work tile by tile; a multiple of BW_TOK as well)
  constexpr int STEP = 128;
  const int steps = (d.N + STEP - 1) / STEP;
  int chunks = std::max(1, std::min(steps, (int)(sms / BH)));
  L.chunk_tokens = (steps + chunks - 1) / chunks * STEP;
  L.chunks = (d.N + L.chunk_tokens - 1) / L.chunk_tokens;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += align256(bytes); return o; };
  L.part_dS = take(BH * L.chunks * F * D * 4);
  L.part_dz = take(BH * L.chunks * F * 4);
  L.part_dW = take(BH * L.chunks * F * D * 4);
  L.part_loss = take(BH * L.chunks * 4);
  L.dS = take(BH * F * D * 4);
  L.dz = take(BH * F * 4);
  L.dSb = take(BH * F * D * 2);
  L.total = off;
  return L;
}

bool bw_supported(const as_hybrid_attn_s* h) {
  const auto& d = h->desc;
  return d.phi_layers == 1 && d.phi_dim == d.d;
}

}  // namespace

extern "C" {

as_status_t as_hybrid_attn_backward_workspace_bytes(as_hybrid_attn_t h, size_t* bytes) {
  if (!h || !bytes) return AS_ERR_INVALID_ARG;
  if (!bw_supported(h)) return AS_ERR_UNSUPPORTED;
  *bytes = bw_layout(h).total;
  return AS_OK;
}

as_status_t as_hybrid_attn_backward_phi(as_hybrid_attn_t h, const void* q, const void* k, const void* v,
                                        const as_phi_weights_t* w, const void* y_teacher, const void* y_hat,
                                        const float* aux, const void* forward_workspace, float* dWq, float* dWk,
                                        float* loss, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!h || !q || !k || !v || !y_teacher || !y_hat || !aux || !forward_workspace || !dWq || !dWk) return AS_ERR_INVALID_ARG;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return AS_ERR_CUDA; }
  if (dev != h->device) return AS_ERR_INVALID_ARG;
  if (!bw_supported(h)) return AS_ERR_UNSUPPORTED;
  const auto& d = h->desc;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const size_t HFD = (size_t)d.H * d.phi_dim * d.d;
  if (h->n_l == 0) {
    // no linear tokens: the output does not depend on the feature maps; the loss is not formed on this path
    if (loss) return AS_ERR_INVALID_ARG;
    if (cudaMemsetAsync(dWq, 0, HFD * 4, st) != cudaSuccess || cudaMemsetAsync(dWk, 0, HFD * 4, st) != cudaSuccess) {
      cudaGetLastError(); return AS_ERR_CUDA;
    }
    return AS_OK;
  }
  if (!w || !w->wq1 || !w->wk1) return AS_ERR_INVALID_ARG;
  if (w->bq1 || w->bk1 || w->wq2 || w->wk2 || w->bq2 || w->bk2) return AS_ERR_UNSUPPORTED;
  const BwLayout L = bw_layout(h);
  if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < L.total) return AS_ERR_WORKSPACE;
  char* ws = (char*)workspace;
  const char* fws = (const char*)forward_workspace;
  BwParams p{};
  p.q = (const __nv_bfloat16*)q; p.k = (const __nv_bfloat16*)k; p.v = (const __nv_bfloat16*)v;
  p.wq = (const __nv_bfloat16*)w->wq1; p.wk = (const __nv_bfloat16*)w->wk1;
  p.y = (const __nv_bfloat16*)y_teacher; p.yhat = (const __nv_bfloat16*)y_hat;
  p.aux = aux; p.S = (const float*)(fws + h->ws.S); p.z = (const float*)(fws + h->ws.z);
  p.Sb = (const __nv_bfloat16*)(fws + h->ws.Sb); p.status = h->d_status;
  p.sm_rank = h->d_sm_rank;
  p.part_dS = (float*)(ws + L.part_dS); p.part_dz = (float*)(ws + L.part_dz); p.part_dW = (float*)(ws + L.part_dW);
  p.part_loss = (float*)(ws + L.part_loss); p.dS = (float*)(ws + L.dS); p.dz = (float*)(ws + L.dz);
  p.dSb = (__nv_bfloat16*)(ws + L.dSb);
  p.dWq = dWq; p.dWk = dWk; p.loss = loss;
  p.B = d.B; p.H = d.H; p.N = d.N; p.P = d.poly_degree; p.n_s = h->n_s; p.stab_mode = d.stab_mode;
  p.chunks = L.chunks; p.chunk_tokens = L.chunk_tokens;

  const int BH = d.B * d.H, D = d.d;
  const dim3 grid(L.chunks, BH), rgrid((D * D + D + 255) / 256, std::max(BH, d.H), 2);
  cudaError_t e = cudaSuccess;
  if (D == 128 && d.phi_dim == 128 && d.kernel_path == AS_PATH_TENSOR) {
    // the products on the tensor cores; the same fixed-order reductions
    if ((e = as_bw_tensor_init()) == cudaSuccess && (e = as_bw_tensor_query(p, st)) == cudaSuccess) {
      bw_reduce_kernel<<<rgrid, 256, 0, st>>>(p, D, 0);
      if ((e = as_bw_tensor_key(p, st)) == cudaSuccess) bw_reduce_kernel<<<rgrid, 256, 0, st>>>(p, D, 1);
    }
  } else if (D == 128) {
    if ((e = cudaFuncSetAttribute(bw_query_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)BwSmem<128>::BYTES)) == cudaSuccess &&
        (e = cudaFuncSetAttribute(bw_key_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)BwSmem<128>::BYTES)) == cudaSuccess) {
      bw_query_kernel<128><<<grid, BW_THREADS, BwSmem<128>::BYTES, st>>>(p);
      bw_reduce_kernel<<<rgrid, 256, 0, st>>>(p, D, 0);
      bw_key_kernel<128><<<grid, BW_THREADS, BwSmem<128>::BYTES, st>>>(p);
      bw_reduce_kernel<<<rgrid, 256, 0, st>>>(p, D, 1);
    }
  } else {
    if ((e = cudaFuncSetAttribute(bw_query_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)BwSmem<64>::BYTES)) == cudaSuccess &&
        (e = cudaFuncSetAttribute(bw_key_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)BwSmem<64>::BYTES)) == cudaSuccess) {
      bw_query_kernel<64><<<grid, BW_THREADS, BwSmem<64>::BYTES, st>>>(p);
      bw_reduce_kernel<<<rgrid, 256, 0, st>>>(p, D, 0);
      bw_key_kernel<64><<<grid, BW_THREADS, BwSmem<64>::BYTES, st>>>(p);
      bw_reduce_kernel<<<rgrid, 256, 0, st>>>(p, D, 1);
    }
  }
  if (e != cudaSuccess || cudaGetLastError() != cudaSuccess) { cudaGetLastError(); return AS_ERR_CUDA; }
  h->launches += 4;
  return AS_OK;
}

}  // extern "C"
