// fp32 CUDA-core kernels of the hybrid attention forward (AS_PATH_SIMT), plus the fixed-order
// reduction of the per-chunk linear state that both kernel paths share.
//
// The SIMT kernels are the on-device cross-check of the tensor-core path: same inputs, same
// workspace layout, every product and sum in fp32, no tensor cores, no TMA.
#include "as_internal.h"

namespace {

constexpr int KP_THREADS = 256;
constexpr int KP_TOK = 16;          // tokens staged per step in the K pass

__device__ __forceinline__ float bf2f(__nv_bfloat16 x) { return __bfloat162float(x); }

// phi(x) = [a_1, a_2^2, ...]: part p of the activation to the power p+1 ("Characterization of phi").
__device__ __forceinline__ float poly_part(float a, int f, int part_width) {
  const int p = f / part_width;
  float r = a;
  for (int i = 0; i < p; ++i) r *= a;
  return r;
}

// K pass: for one (batch*head, token chunk) accumulate S = sum phi_k(k_j)^T v_j and z = sum phi_k(k_j)
// over the chunk's linear tokens, and copy the chunk's softmax tokens to the compact K_S / V_S.
template <int D, int F>
__global__ void __launch_bounds__(KP_THREADS) simt_kpass_kernel(as_launch_args a) {
  extern __shared__ float smem[];
  float* sW = smem;                          // [F][D+1]
  float* sK = sW + F * (D + 1);              // [KP_TOK][D]
  float* sV = sK + KP_TOK * D;               // [KP_TOK][D]
  float* sPhi = sV + KP_TOK * D;             // [KP_TOK][F]
  __shared__ int sRank[KP_TOK];

  const int bh = blockIdx.y, chunk = blockIdx.x, tid = threadIdx.x;
  const int h = bh % a.H;
  const int part_width = F / a.P;
  const __nv_bfloat16* W = a.wk + (size_t)h * F * D;
  for (int i = tid; i < F * D; i += KP_THREADS) sW[(i / D) * (D + 1) + (i % D)] = bf2f(W[i]);

  constexpr int TPR = KP_THREADS / F;        // threads per feature row of S
  constexpr int COLS = D / TPR;              // S columns per thread
  const int f_own = tid / TPR, c0 = (tid % TPR) * COLS;
  float acc[COLS];
#pragma unroll
  for (int c = 0; c < COLS; ++c) acc[c] = 0.f;
  float zacc = 0.f;

  const int tok_begin = chunk * a.chunk_tiles * AS_TILE;
  const int tok_end = min(a.N, tok_begin + a.chunk_tiles * AS_TILE);
  const __nv_bfloat16* kb = a.k + (size_t)bh * a.N * D;
  const __nv_bfloat16* vb = a.v + (size_t)bh * a.N * D;
  __syncthreads();

  for (int t0 = tok_begin; t0 < tok_end; t0 += KP_TOK) {
    for (int i = tid; i < KP_TOK * D; i += KP_THREADS) {
      const int tt = i / D, dd = i % D, n = t0 + tt;
      const bool in = n < tok_end;
      sK[i] = in ? bf2f(kb[(size_t)n * D + dd]) : 0.f;
      sV[i] = in ? bf2f(vb[(size_t)n * D + dd]) : 0.f;
    }
    if (tid < KP_TOK) sRank[tid] = (t0 + tid < tok_end) ? a.sm_rank[t0 + tid] : 0;
    __syncthreads();
    // softmax tokens go to the compact arrays
    if (a.ks_w != nullptr) {
      for (int i = tid; i < KP_TOK * D; i += KP_THREADS) {
        const int tt = i / D, dd = i % D, n = t0 + tt;
        if (n < tok_end && sRank[tt] >= 0) {
          const size_t o = ((size_t)bh * a.n_s + sRank[tt]) * D + dd;
          a.ks_w[o] = kb[(size_t)n * D + dd];
          a.vs_w[o] = vb[(size_t)n * D + dd];
        }
      }
    }
    // features of the staged tokens (zero for softmax tokens and past the end)
    for (int i = tid; i < KP_TOK * F; i += KP_THREADS) {
      const int tt = i / F, f = i % F;
      float s = 0.f;
#pragma unroll 8
      for (int dd = 0; dd < D; ++dd) s = fmaf(sW[f * (D + 1) + dd], sK[tt * D + dd], s);
      s = fmaxf(s, 0.f);
      const bool lin = (t0 + tt < tok_end) && sRank[tt] < 0;
      sPhi[tt * F + f] = lin ? poly_part(s, f, part_width) : 0.f;
    }
    __syncthreads();
#pragma unroll 4
    for (int tt = 0; tt < KP_TOK; ++tt) {
      const float p = sPhi[tt * F + f_own];
      if (c0 == 0) zacc += p;
#pragma unroll
      for (int c = 0; c < COLS; ++c) acc[c] = fmaf(p, sV[tt * D + c0 + c], acc[c]);
    }
    __syncthreads();
  }
  float* ps = a.part_s + (((size_t)bh * a.n_chunks + chunk) * F + f_own) * D + c0;
#pragma unroll
  for (int c = 0; c < COLS; ++c) ps[c] = acc[c];
  if (c0 == 0) a.part_z[((size_t)bh * a.n_chunks + chunk) * F + f_own] = zacc;
}

// Sums the per-chunk partial states in chunk order (deterministic) and writes S, z in fp32 and
// S rounded to bf16 (same [F][d] layout: the tensor path reads it like a V tile).
__global__ void reduce_state_kernel(as_launch_args a) {
  const int bh = blockIdx.y;
  const int D = a.d, F = a.F;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;      // over F*D entries, then F entries of z
  // (the loads of eight chunks are issued together, the sum still runs in chunk order)
  if (i < F * D) {
    const float* src = a.part_s + (size_t)bh * a.n_chunks * F * D + i;
    const size_t pitch = (size_t)F * D;
    float s = 0.f;
    int c = 0;
    for (; c + 8 <= a.n_chunks; c += 8) {
      float v[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) v[j] = __ldcs(src + (c + j) * pitch);
#pragma unroll
      for (int j = 0; j < 8; ++j) s += v[j];
    }
    for (; c < a.n_chunks; ++c) s += __ldcs(src + c * pitch);
    a.S[(size_t)bh * F * D + i] = s;
    a.Sb[(size_t)bh * F * D + i] = __float2bfloat16_rn(s);
  } else if (i < F * D + F) {
    const int f = i - F * D;
    float s = 0.f;
    for (int c = 0; c < a.n_chunks; ++c) s += a.part_z[((size_t)bh * a.n_chunks + c) * F + f];
    a.z[(size_t)bh * F + f] = s;
  }
}

__global__ void round_state_kernel(const float* S, __nv_bfloat16* Sb, size_t n) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) Sb[i] = __float2bfloat16_rn(S[i]);
}

constexpr int QP_WARPS = 8;

// Q pass: one warp per query row.  Online softmax over the softmax tokens, then the linear
// branch phi_q(q_i) S and phi_q(q_i).z, merged under the shared denominator.
template <int D, int F>
__global__ void __launch_bounds__(QP_WARPS * 32) simt_qpass_kernel(as_launch_args a) {
  constexpr int EPL = D / 32;               // elements of a row per lane
  constexpr int FPL = F / 32;               // features per lane
  extern __shared__ float smem[];
  float* sQ = smem;                                           // [QP_WARPS][D]
  __nv_bfloat16* sW = (__nv_bfloat16*)(sQ + QP_WARPS * D);    // [F][D+2]
  const int bh = blockIdx.y, h = bh % a.H;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int row = blockIdx.x * QP_WARPS + warp;
  const bool lin = a.n_l > 0;
  if (lin) {
    const __nv_bfloat16* W = a.wq + (size_t)h * F * D;
    for (int i = threadIdx.x; i < F * D; i += QP_WARPS * 32) sW[(i / D) * (D + 2) + (i % D)] = W[i];
  }
  const bool active = row < a.N;
  float qv[EPL];
  if (active) {
    const __nv_bfloat16* qp = a.q + ((size_t)bh * a.N + row) * D + lane * EPL;
#pragma unroll
    for (int e = 0; e < EPL; ++e) { qv[e] = bf2f(qp[e]); sQ[warp * D + lane * EPL + e] = qv[e]; }
  }
  __syncthreads();
  if (!active) return;

  float m = -INFINITY, l = 0.f, o[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) o[e] = 0.f;
  const __nv_bfloat16* kb = a.ks + (size_t)bh * a.n_s * D + lane * EPL;
  const __nv_bfloat16* vb = a.vs + (size_t)bh * a.n_s * D + lane * EPL;
  constexpr int UN = 4;
  for (int j0 = 0; j0 < a.n_s; j0 += UN) {
    float s[UN];
#pragma unroll
    for (int u = 0; u < UN; ++u) {
      const int j = min(j0 + u, a.n_s - 1);
      float p = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) p = fmaf(qv[e], bf2f(kb[(size_t)j * D + e]), p);
      s[u] = p;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
#pragma unroll
      for (int u = 0; u < UN; ++u) s[u] += __shfl_xor_sync(0xffffffffu, s[u], off);
    }
#pragma unroll
    for (int u = 0; u < UN; ++u) {
      if (j0 + u < a.n_s) {
        const float sc = s[u] * a.scale;
        const float mn = fmaxf(m, sc);
        const float corr = __expf(m - mn);      // exp(-inf) = 0 on the first key
        const float p = __expf(sc - mn);
        l = l * corr + p;
#pragma unroll
        for (int e = 0; e < EPL; ++e) o[e] = o[e] * corr + p * bf2f(vb[(size_t)(j0 + u) * D + e]);
        m = mn;
      }
    }
  }
  const float c = a.n_s > 0 ? m : 0.f;
  float den_l = 0.f, lam = 1.f;
  float num[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) num[e] = o[e];
  float den = l;
  if (lin) {
    const int part_width = F / a.P;
    float fi[FPL];
#pragma unroll
    for (int i = 0; i < FPL; ++i) {
      const int f = lane + 32 * i;
      float s = 0.f;
#pragma unroll 8
      for (int dd = 0; dd < D; ++dd) s = fmaf(bf2f(sW[f * (D + 2) + dd]), sQ[warp * D + dd], s);
      fi[i] = poly_part(fmaxf(s, 0.f), f, part_width);
      den_l = fmaf(fi[i], a.z[(size_t)bh * F + f], den_l);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) den_l += __shfl_xor_sync(0xffffffffu, den_l, off);
    if (a.stab_mode == AS_STAB_EXACT && a.n_s > 0) lam = __expf(-c);
    const float* Sb = a.S + (size_t)bh * F * D + lane * EPL;
    float nl[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) nl[e] = 0.f;
#pragma unroll
    for (int i = 0; i < FPL; ++i) {
      for (int src = 0; src < 32; ++src) {
        const float p = __shfl_sync(0xffffffffu, fi[i], src);
        const int f = src + 32 * i;
#pragma unroll
        for (int e = 0; e < EPL; ++e) nl[e] = fmaf(p, Sb[(size_t)f * D + e], nl[e]);
      }
    }
#pragma unroll
    for (int e = 0; e < EPL; ++e) num[e] += lam * nl[e];
    den += lam * den_l;
  }
  __nv_bfloat16* op = a.out + ((size_t)bh * a.N + row) * D + lane * EPL;
#pragma unroll
  for (int e = 0; e < EPL; ++e) op[e] = __float2bfloat16_rn(num[e] / den);
  if (a.aux != nullptr && lane == 0) {
    float* ap = a.aux + ((size_t)bh * a.N + row) * 3;
    ap[0] = c; ap[1] = l; ap[2] = den_l;
  }
}

template <typename K>
cudaError_t set_smem(K kernel, size_t bytes) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

}  // namespace

cudaError_t as_simt_kpass(const as_launch_args& a, cudaStream_t st) {
  dim3 grid(a.n_chunks, a.B * a.H);
  cudaError_t e;
  if (a.d == 128) {
    const size_t sm = sizeof(float) * (128 * 129 + 2 * KP_TOK * 128 + KP_TOK * 128);
    if ((e = set_smem(simt_kpass_kernel<128, 128>, sm)) != cudaSuccess) return e;
    simt_kpass_kernel<128, 128><<<grid, KP_THREADS, sm, st>>>(a);
  } else {
    const size_t sm = sizeof(float) * (64 * 65 + 2 * KP_TOK * 64 + KP_TOK * 64);
    if ((e = set_smem(simt_kpass_kernel<64, 64>, sm)) != cudaSuccess) return e;
    simt_kpass_kernel<64, 64><<<grid, KP_THREADS, sm, st>>>(a);
  }
  return cudaGetLastError();
}

cudaError_t as_reduce_state(const as_launch_args& a, cudaStream_t st) {
  const int n = a.F * a.d + a.F;
  dim3 grid((n + 255) / 256, a.B * a.H);
  reduce_state_kernel<<<grid, 256, 0, st>>>(a);
  return cudaGetLastError();
}

cudaError_t as_round_state(const as_launch_args& a, cudaStream_t st) {
  const size_t n = (size_t)a.B * a.H * a.F * a.d;
  round_state_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(a.S, a.Sb, n);
  return cudaGetLastError();
}

cudaError_t as_simt_qpass(const as_launch_args& a, cudaStream_t st) {
  dim3 grid((a.N + QP_WARPS - 1) / QP_WARPS, a.B * a.H);
  cudaError_t e;
  if (a.d == 128) {
    const size_t sm = sizeof(float) * QP_WARPS * 128 + 2 * 128 * 130;
    if ((e = set_smem(simt_qpass_kernel<128, 128>, sm)) != cudaSuccess) return e;
    simt_qpass_kernel<128, 128><<<grid, QP_WARPS * 32, sm, st>>>(a);
  } else {
    const size_t sm = sizeof(float) * QP_WARPS * 64 + 2 * 64 * 66;
    if ((e = set_smem(simt_qpass_kernel<64, 64>, sm)) != cudaSuccess) return e;
    simt_qpass_kernel<64, 64><<<grid, QP_WARPS * 32, sm, st>>>(a);
  }
  return cudaGetLastError();
}
