// as_hybrid_attn_linear_state_static: the linear state S, z of one layer computed without any
// allocation.  The per-chunk partial sums live in a fixed device array that is part of the
// library image, so the call needs no workspace argument, no handle and no allocator.
//
// Who needs this: code that runs where device memory cannot be requested any more - a serving
// process that handed the whole HBM to its own arena at start-up (a later cudaMalloc fails or is
// forbidden by policy), a plug-in inside another framework that may only use the buffers it was
// given, or a latency-critical loop that must not hit the implicit device-wide synchronisation
// of cudaMalloc / cudaFree.  Such callers pass their inputs and outputs and nothing else.
//
// The arithmetic is the fp32 CUDA-core formulation of the K pass (features, then S and z over
// the linear tokens); the token rule is evaluated on the device from the grid, block and rate.
#include <mutex>

#include "as_internal.h"

namespace {

// Fixed scratch: 8 MiB of fp32 partial sums.  A device holds this array from the moment the driver
// loads this module there (with lazy module loading: the first call below on that device) until the
// process exits.
constexpr size_t kScratchFloats = size_t(2) << 20;
static __device__ __align__(256) float g_static_scratch[kScratchFloats];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
float* g_scratch_addr[kMaxDevices] = {};       // device address of g_static_scratch, per device
bool g_setup_done[kMaxDevices] = {};

constexpr int LS_THREADS = 256;
constexpr int LS_TOK = 16;                     // tokens staged per step

struct LsParams {
  const __nv_bfloat16 *k, *v, *wk;
  float *part_s, *part_z;                      // inside the static scratch
  float *S_out, *z_out;
  int H, N, P;
  int grid_h, grid_w, blk_t, blk_h, blk_w, rate;
  int n_chunks, chunk_tokens;
};

// Token rule: inside each (clipped) spatial block the token with raster index l is a softmax
// token iff l mod R == 0; R == 1 selects every token, R == 0 none.
__device__ __forceinline__ bool is_softmax_token(int n, const LsParams& p) {
  if (p.rate == 0) return false;
  if (p.rate == 1) return true;
  const int w = n % p.grid_w, h = (n / p.grid_w) % p.grid_h, t = n / (p.grid_w * p.grid_h);
  const int ot = t / p.blk_t * p.blk_t, oh = h / p.blk_h * p.blk_h, ow = w / p.blk_w * p.blk_w;
  const int eh = min(p.blk_h, p.grid_h - oh), ew = min(p.blk_w, p.grid_w - ow);
  const int l = ((t - ot) * eh + (h - oh)) * ew + (w - ow);
  return l % p.rate == 0;
}

// One CTA per (token chunk, batch*head): partial S [F][D] and z [F] over the chunk's linear tokens.
template <int D>
__global__ void __launch_bounds__(LS_THREADS) static_partial_kernel(LsParams p) {
  constexpr int F = D;
  extern __shared__ float smem[];
  float* sW = smem;                            // [F][D+1]
  float* sK = sW + F * (D + 1);                // [LS_TOK][D]
  float* sV = sK + LS_TOK * D;                 // [LS_TOK][D]
  float* sPhi = sV + LS_TOK * D;               // [LS_TOK][F]
  __shared__ int sLin[LS_TOK];

  const int bh = blockIdx.y, chunk = blockIdx.x, tid = threadIdx.x;
  const int h = bh % p.H;
  const int part_width = F / p.P;
  const __nv_bfloat16* W = p.wk + (size_t)h * F * D;
  for (int i = tid; i < F * D; i += LS_THREADS) sW[(i / D) * (D + 1) + (i % D)] = __bfloat162float(W[i]);

  constexpr int TPR = LS_THREADS / F;          // threads per feature row
  constexpr int COLS = D / TPR;                // columns of S per thread
  const int f_own = tid / TPR, c0 = (tid % TPR) * COLS;
  float acc[COLS];
#pragma unroll
  for (int c = 0; c < COLS; ++c) acc[c] = 0.f;
  float zacc = 0.f;

  const int tok_begin = chunk * p.chunk_tokens;
  const int tok_end = min(p.N, tok_begin + p.chunk_tokens);
  const __nv_bfloat16* kb = p.k + (size_t)bh * p.N * D;
  const __nv_bfloat16* vb = p.v + (size_t)bh * p.N * D;
  __syncthreads();

  for (int t0 = tok_begin; t0 < tok_end; t0 += LS_TOK) {
    for (int i = tid; i < LS_TOK * D; i += LS_THREADS) {
      const int n = t0 + i / D;
      const bool in = n < tok_end;
      sK[i] = in ? __bfloat162float(kb[(size_t)n * D + i % D]) : 0.f;
      sV[i] = in ? __bfloat162float(vb[(size_t)n * D + i % D]) : 0.f;
    }
    if (tid < LS_TOK) sLin[tid] = (t0 + tid < tok_end) && !is_softmax_token(t0 + tid, p);
    __syncthreads();
    for (int i = tid; i < LS_TOK * F; i += LS_THREADS) {
      const int tt = i / F, f = i % F;
      float a = 0.f;
#pragma unroll 8
      for (int dd = 0; dd < D; ++dd) a = fmaf(sW[f * (D + 1) + dd], sK[tt * D + dd], a);
      a = fmaxf(a, 0.f);
      float r = a;
      for (int q = 0; q < f / part_width; ++q) r *= a;      // part p (0-based) to the power p + 1
      sPhi[i] = sLin[tt] ? r : 0.f;
    }
    __syncthreads();
#pragma unroll 4
    for (int tt = 0; tt < LS_TOK; ++tt) {
      const float ph = sPhi[tt * F + f_own];
      if (c0 == 0) zacc += ph;
#pragma unroll
      for (int c = 0; c < COLS; ++c) acc[c] = fmaf(ph, sV[tt * D + c0 + c], acc[c]);
    }
    __syncthreads();
  }
  const size_t slot = (size_t)bh * p.n_chunks + chunk;
  float* ps = p.part_s + (slot * F + f_own) * D + c0;
#pragma unroll
  for (int c = 0; c < COLS; ++c) ps[c] = acc[c];
  if (c0 == 0) p.part_z[slot * F + f_own] = zacc;
}

// Sums the partials in chunk order (deterministic) into the caller's S and z.
template <int D>
__global__ void static_reduce_kernel(LsParams p) {
  constexpr int F = D;
  const int bh = blockIdx.y;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < F * D) {
    float s = 0.f;
    for (int c = 0; c < p.n_chunks; ++c) s += p.part_s[((size_t)bh * p.n_chunks + c) * F * D + i];
    if (p.S_out) p.S_out[(size_t)bh * F * D + i] = s;
  } else if (i < F * D + F) {
    const int f = i - F * D;
    float s = 0.f;
    for (int c = 0; c < p.n_chunks; ++c) s += p.part_z[((size_t)bh * p.n_chunks + c) * F + f];
    if (p.z_out) p.z_out[(size_t)bh * F + f] = s;
  }
}

template <int D>
constexpr size_t partial_smem_bytes() {
  return sizeof(float) * (D * (D + 1) + 2 * LS_TOK * D + LS_TOK * D);
}

// Once per device, with that device current: resolve the device address of the scratch array
// (its name in host code is only a stand-in for the symbol) and opt the kernels into their
// dynamic shared memory.
as_status_t setup_device(int dev, float** scratch) {
  if (dev < 0 || dev >= kMaxDevices) return AS_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_setup_done[dev]) {
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
      cudaGetLastError(); return AS_ERR_CUDA;
    }
    if (major != 10) return AS_ERR_ARCH;
    float* ptr = nullptr;
    if (cudaGetSymbolAddress((void**)&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) {
      cudaGetLastError(); return AS_ERR_CUDA;
    }
    if (cudaFuncSetAttribute(static_partial_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)partial_smem_bytes<128>()) != cudaSuccess ||
        cudaFuncSetAttribute(static_partial_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)partial_smem_bytes<64>()) != cudaSuccess) {
      cudaGetLastError(); return AS_ERR_CUDA;
    }
    g_scratch_addr[dev] = ptr;
    g_setup_done[dev] = true;
  }
  *scratch = g_scratch_addr[dev];
  return AS_OK;
}

}  // namespace

extern "C" as_status_t as_hybrid_attn_linear_state_static(
    const void* k, const void* v, const void* wk, int32_t B, int32_t H, int32_t N, int32_t d,
    int32_t grid_t, int32_t grid_h, int32_t grid_w, int32_t blk_t, int32_t blk_h, int32_t blk_w,
    int32_t rate_den, int32_t poly_degree, float* S_out, float* z_out, void* cuda_stream) {
  if (!k || !v || !wk || (!S_out && !z_out)) return AS_ERR_INVALID_ARG;
  if (B <= 0 || H <= 0 || N <= 0 || grid_t <= 0 || grid_h <= 0 || grid_w <= 0) return AS_ERR_INVALID_ARG;
  if ((long long)grid_t * grid_h * grid_w != (long long)N) return AS_ERR_INVALID_ARG;
  if (rate_den < 0 || (rate_den > 1 && (blk_t <= 0 || blk_h <= 0 || blk_w <= 0))) return AS_ERR_INVALID_ARG;
  if (poly_degree < 1 || poly_degree > 2) return AS_ERR_UNSUPPORTED;
  if (d != 64 && d != 128) return AS_ERR_UNSUPPORTED;
  if ((((uintptr_t)k | (uintptr_t)v | (uintptr_t)wk) & 1) || (((uintptr_t)S_out | (uintptr_t)z_out) & 3))
    return AS_ERR_INVALID_ARG;
  const long long BH = (long long)B * H;
  const size_t per_slot = (size_t)d * (d + 1);             // floats of one partial (S and z), F == d
  // The fixed scratch must hold at least one partial per (batch, head).
  if (BH > 65535 || (size_t)BH * per_slot > kScratchFloats) return AS_ERR_UNSUPPORTED;

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return AS_ERR_CUDA; }
  float* scratch = nullptr;
  as_status_t s = setup_device(dev, &scratch);
  if (s != AS_OK) return s;

  // Split the token axis into as many chunks as the scratch holds, up to about two CTAs per SM.
  const int max_by_scratch = (int)(kScratchFloats / ((size_t)BH * per_slot));
  const int by_tokens = (N + LS_TOK - 1) / LS_TOK;
  const int by_sms = (int)((296 + BH - 1) / BH);
  int chunks = by_tokens < max_by_scratch ? by_tokens : max_by_scratch;
  if (by_sms < chunks) chunks = by_sms;
  if (chunks < 1) chunks = 1;
  int chunk_tokens = (N + chunks - 1) / chunks;
  chunk_tokens = (chunk_tokens + LS_TOK - 1) / LS_TOK * LS_TOK;
  chunks = (N + chunk_tokens - 1) / chunk_tokens;

  LsParams p{};
  p.k = (const __nv_bfloat16*)k; p.v = (const __nv_bfloat16*)v; p.wk = (const __nv_bfloat16*)wk;
  p.part_s = scratch;
  p.part_z = scratch + (size_t)BH * chunks * d * d;
  p.S_out = S_out; p.z_out = z_out;
  p.H = H; p.N = N; p.P = poly_degree;
  p.grid_h = grid_h; p.grid_w = grid_w; p.blk_t = blk_t; p.blk_h = blk_h; p.blk_w = blk_w; p.rate = rate_den;
  p.n_chunks = chunks; p.chunk_tokens = chunk_tokens;

  cudaStream_t st = (cudaStream_t)cuda_stream;
  const dim3 grid1(chunks, (unsigned)BH), grid2((d * d + d + 255) / 256, (unsigned)BH);
  if (d == 128) {
    static_partial_kernel<128><<<grid1, LS_THREADS, partial_smem_bytes<128>(), st>>>(p);
    static_reduce_kernel<128><<<grid2, 256, 0, st>>>(p);
  } else {
    static_partial_kernel<64><<<grid1, LS_THREADS, partial_smem_bytes<64>(), st>>>(p);
    static_reduce_kernel<64><<<grid2, 256, 0, st>>>(p);
  }
  if (cudaGetLastError() != cudaSuccess) return AS_ERR_CUDA;
  return AS_OK;
}
