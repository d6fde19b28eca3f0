// Host side of libas_hybrid_attn: argument checking, the token split, workspace layout and
// the launch sequence of the forward pass.  No arithmetic of the method runs here except the
// integer token rule.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>

#include "as_internal.h"

namespace {

size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

// Token rule of section "Hybrid Attention" (T_S = { i : i mod R = 1 }, 1-indexed), applied to the
// raster index inside each clipped spatial block; a block equal to the grid is the paper's rule.
void build_token_split(const as_hybrid_attn_desc_t& d, std::vector<int32_t>& idx) {
  idx.clear();
  const int R = d.rate_den;
  if (R == 0) return;
  for (int t = 0; t < d.grid_t; ++t)
    for (int h = 0; h < d.grid_h; ++h)
      for (int w = 0; w < d.grid_w; ++w) {
        const int n = (t * d.grid_h + h) * d.grid_w + w;
        if (R == 1) { idx.push_back(n); continue; }
        const int ot = t / d.blk_t * d.blk_t, oh = h / d.blk_h * d.blk_h, ow = w / d.blk_w * d.blk_w;
        const int eh = std::min(d.blk_h, d.grid_h - oh), ew = std::min(d.blk_w, d.grid_w - ow);
        const int l = ((t - ot) * eh + (h - oh)) * ew + (w - ow);
        if (l % R == 0) idx.push_back(n);
      }
}

as_status_t validate(const as_hybrid_attn_desc_t* d) {
  if (!d) return AS_ERR_INVALID_ARG;
  if (d->struct_size != sizeof(as_hybrid_attn_desc_t)) return AS_ERR_INVALID_ARG;
  if (d->B <= 0 || d->H <= 0 || d->N <= 0) return AS_ERR_INVALID_ARG;
  if (d->grid_t <= 0 || d->grid_h <= 0 || d->grid_w <= 0) return AS_ERR_INVALID_ARG;
  if ((long long)d->grid_t * d->grid_h * d->grid_w != (long long)d->N) return AS_ERR_INVALID_ARG;
  if (d->rate_den < 0) return AS_ERR_INVALID_ARG;
  if (d->softmax_idx == nullptr && d->rate_den > 1 &&
      (d->blk_t <= 0 || d->blk_h <= 0 || d->blk_w <= 0)) return AS_ERR_INVALID_ARG;
  if (d->softmax_idx != nullptr) {
    if (d->n_softmax < 0 || d->n_softmax > d->N) return AS_ERR_INVALID_ARG;
    for (int i = 0; i < d->n_softmax; ++i) {
      if (d->softmax_idx[i] < 0 || d->softmax_idx[i] >= d->N) return AS_ERR_INVALID_ARG;
      if (i > 0 && d->softmax_idx[i] <= d->softmax_idx[i - 1]) return AS_ERR_INVALID_ARG;
    }
  }
  if (d->stab_mode != AS_STAB_PAPER && d->stab_mode != AS_STAB_EXACT) return AS_ERR_INVALID_ARG;
  if (d->kernel_path != AS_PATH_TENSOR && d->kernel_path != AS_PATH_SIMT) return AS_ERR_INVALID_ARG;
  if (!(d->softmax_scale >= 0.f) || !std::isfinite(d->softmax_scale)) return AS_ERR_INVALID_ARG;
  if (d->phi_dim <= 0 || d->poly_degree <= 0 || d->phi_layers <= 0) return AS_ERR_INVALID_ARG;
  if (d->phi_dim % d->poly_degree != 0) return AS_ERR_INVALID_ARG;
  // what the library has kernels for
  if (d->d != 64 && d->d != 128) return AS_ERR_UNSUPPORTED;
  if (d->phi_layers > 2 || d->poly_degree > 4 || d->phi_act != AS_ACT_RELU) return AS_ERR_UNSUPPORTED;
  const int F = d->phi_dim;
  // feature width: d itself, or a multiple of 128 up to 512; parts of the polynomial a multiple of 32 wide
  if (!(F == d->d || (F % 128 == 0 && F <= 512))) return AS_ERR_UNSUPPORTED;
  if ((F / d->poly_degree) % 32 != 0) return AS_ERR_UNSUPPORTED;
  if (d->kernel_path == AS_PATH_SIMT && (F != d->d || d->phi_layers != 1 || d->poly_degree > 2)) return AS_ERR_UNSUPPORTED;
  if (d->phi_layers == 2) {
    // two layers: hidden width d or 2d (d = 128), features d or 2d; at d = 64 both equal to d
    const int hid = d->phi_hidden;
    if (d->d == 128 ? !((hid == 128 || hid == 256) && (F == 128 || F == 256)) : !(hid == 64 && F == 64)) return AS_ERR_UNSUPPORTED;
  }
  if ((long long)d->B * d->H > 65535) return AS_ERR_UNSUPPORTED;
  return AS_OK;
}

void layout_workspace(as_hybrid_attn_s* h) {
  const auto& d = h->desc;
  const size_t BH = (size_t)d.B * d.H;
  as_ws_layout& w = h->ws;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += align256(bytes); return o; };
  const bool compact = h->n_s > 0 && h->n_l > 0;      // at rate 1 the Q pass reads k, v directly
  w.ks = take(compact ? BH * h->n_s * d.d * 2 : 0);
  w.vs = take(compact ? BH * h->n_s * d.d * 2 : 0);
  const bool lin = h->n_l > 0;
  w.part_s = take(lin ? BH * h->n_chunks * d.phi_dim * d.d * 4 : 0);
  w.part_z = take(lin ? BH * h->n_chunks * d.phi_dim * 4 : 0);
  w.S = take(lin ? BH * d.phi_dim * d.d * 4 : 0);
  w.z = take(lin ? BH * d.phi_dim * 4 : 0);
  w.Sb = take(lin ? BH * d.phi_dim * d.d * 2 : 0);
  const bool two = lin && d.phi_layers == 2;
  w.h1k = take(two ? BH * (size_t)d.N * d.phi_hidden * 2 : 0);
  w.total = std::max<size_t>(off, 256);
  const size_t t = BH * d.N * d.d * 2;
  off = w.total;
  w.stage_q = take(t); w.stage_k = take(t); w.stage_v = take(t); w.stage_o = take(t);
  w.total_host = off;
}

struct ProfileScope {
  as_hybrid_attn_s* h; cudaStream_t st; int slot = -1;
  ProfileScope(as_hybrid_attn_s* h_, cudaStream_t st_, int cls) : h(h_), st(st_) {
    h->launches++;
    if (h->profiling && h->ev_used < AS_MAX_PROFILE) {
      slot = h->ev_used++;
      h->ev_class[slot] = cls;
      cudaEventRecord(h->ev[2 * slot], st);
    }
  }
  ~ProfileScope() { if (slot >= 0) cudaEventRecord(h->ev[2 * slot + 1], st); }
};

}  // namespace

// Keys and linear state handed to the query stage from outside (sequence sharding: gathered / summed over ranks).
struct as_ext_state {
  const void *ks, *vs;         // [B*H, n_keys, d] bf16
  int n_keys;
  const float *S, *z;          // [B*H, F, d], [B*H, F] fp32; NULL: no linear tokens anywhere
};
enum { AS_STAGE_KEYS = 1, AS_STAGE_QUERIES = 2 };

static as_status_t launch_heads(as_hybrid_attn_t h, const void* q, const void* k, const void* v,
                                const as_phi_weights_t* w, void* out, float* aux, char* ws, cudaStream_t st,
                                int first, int count, int nb, int nh, int stages = AS_STAGE_KEYS | AS_STAGE_QUERIES,
                                const as_ext_state* ext = nullptr);

// A handle works on the device it was created on: its tables live there and the kernels' shared-memory opt-in
// was made there.
static bool on_handle_device(const as_hybrid_attn_s* h) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return false; }
  return dev == h->device;
}

// The feature-map weights a layer with linear tokens needs: present, 16-byte aligned; biases are optional
// (4-byte aligned), second-layer ones only with a second layer; the fp32 check path takes none.
static as_status_t check_weights(const as_hybrid_attn_s* h, const as_phi_weights_t* w) {
  if (h->n_l == 0) return AS_OK;
  const auto& d = h->desc;
  if (!w || !w->wq1 || !w->wk1) return AS_ERR_INVALID_ARG;
  if (d.phi_layers == 1 && (w->wq2 || w->wk2 || w->bq2 || w->bk2)) return AS_ERR_INVALID_ARG;
  if (d.phi_layers == 2 && (!w->wq2 || !w->wk2)) return AS_ERR_INVALID_ARG;
  if (((uintptr_t)w->wq1 | (uintptr_t)w->wk1 | (uintptr_t)w->wq2 | (uintptr_t)w->wk2) & 15) return AS_ERR_INVALID_ARG;
  if (((uintptr_t)w->bq1 | (uintptr_t)w->bk1 | (uintptr_t)w->bq2 | (uintptr_t)w->bk2) & 3) return AS_ERR_INVALID_ARG;
  if (d.kernel_path == AS_PATH_SIMT && (w->bq1 || w->bk1)) return AS_ERR_UNSUPPORTED;
  return AS_OK;
}

extern "C" {

const char* as_status_string(as_status_t s) {
  switch (s) {
    case AS_OK: return "ok";
    case AS_ERR_INVALID_ARG: return "invalid argument";
    case AS_ERR_UNSUPPORTED: return "unsupported configuration";
    case AS_ERR_ARCH: return "device is not sm_100";
    case AS_ERR_ALLOC: return "allocation failed";
    case AS_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case AS_ERR_CUDA: return "CUDA call failed";
    case AS_ERR_DEVICE_TIMEOUT: return "bounded wait inside a kernel expired";
    case AS_ERR_INFEASIBLE: return "no assignment fits the budget";
  }
  return "unknown status";
}

as_status_t as_hybrid_attn_create(const as_hybrid_attn_desc_t* desc, as_hybrid_attn_t* out) {
  if (!out) return AS_ERR_INVALID_ARG;
  as_status_t vs = validate(desc);
  if (vs != AS_OK) return vs;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return AS_ERR_CUDA; }
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
    cudaGetLastError(); return AS_ERR_CUDA;
  }
  if (major != 10) return AS_ERR_ARCH;

  as_hybrid_attn_s* h = new (std::nothrow) as_hybrid_attn_s();
  if (!h) return AS_ERR_ALLOC;
  h->desc = *desc;
  h->desc.softmax_idx = nullptr;                 // the caller's array is not kept
  h->device = dev;
  h->scale = desc->softmax_scale > 0.f ? desc->softmax_scale : 1.0f / std::sqrt((float)desc->d);
  if (desc->softmax_idx) h->idx_host.assign(desc->softmax_idx, desc->softmax_idx + desc->n_softmax);
  else build_token_split(*desc, h->idx_host);
  h->n_s = (int)h->idx_host.size();
  h->n_l = desc->N - h->n_s;
  h->desc.n_softmax = h->n_s;

  // K-pass split of the token axis: at most one CTA per SM over all (batch, head) pairs.
  const int tiles = (desc->N + AS_TILE - 1) / AS_TILE;
  int sms = 148;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int BH = desc->B * desc->H;
  const int f_chunks = (desc->phi_dim + 127) / 128;       // the tensor K pass runs one CTA per 128 features as well
  int chunks = std::max(1, std::min(tiles, sms / (BH * f_chunks)));
  h->chunk_tiles = (tiles + chunks - 1) / chunks;
  h->n_chunks = (tiles + h->chunk_tiles - 1) / h->chunk_tiles;
  layout_workspace(h);

  std::vector<int32_t> rank(desc->N, -1);
  for (int i = 0; i < h->n_s; ++i) rank[h->idx_host[i]] = i;
  if (cudaMalloc(&h->d_sm_rank, sizeof(int32_t) * ((size_t)desc->N + 8)) != cudaSuccess ||
      cudaMalloc(&h->d_status, 256) != cudaSuccess ||
      cudaMalloc(&h->d_counters, sizeof(uint32_t) * 8 * (size_t)BH) != cudaSuccess) {
    cudaGetLastError(); as_hybrid_attn_destroy(h); return AS_ERR_ALLOC;
  }
  if (cudaMemcpy(h->d_sm_rank, rank.data(), sizeof(int32_t) * desc->N, cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemset(h->d_status, 0, 256) != cudaSuccess ||
      cudaMemset(h->d_counters, 0, sizeof(uint32_t) * 8 * (size_t)BH) != cudaSuccess) {
    cudaGetLastError(); as_hybrid_attn_destroy(h); return AS_ERR_CUDA;
  }
  if (desc->kernel_path == AS_PATH_TENSOR && as_tensor_init() != cudaSuccess) {
    cudaGetLastError(); as_hybrid_attn_destroy(h); return AS_ERR_CUDA;
  }
  *out = h;
  return AS_OK;
}

as_status_t as_hybrid_attn_destroy(as_hybrid_attn_t h) {
  if (!h) return AS_OK;
  if (h->d_sm_rank) cudaFree(h->d_sm_rank);
  if (h->d_status) cudaFree(h->d_status);
  if (h->d_counters) cudaFree(h->d_counters);
  for (cudaEvent_t e : h->ev) cudaEventDestroy(e);
  for (cudaEvent_t e : h->ev_run) cudaEventDestroy(e);
  if (h->side_ready) {
    cudaEventDestroy(h->ev_fork); cudaEventDestroy(h->ev_join);
    cudaStreamDestroy(h->s_in); cudaStreamDestroy(h->s_out);
  }
  delete h;
  return AS_OK;
}

as_status_t as_hybrid_attn_workspace_bytes(as_hybrid_attn_t h, size_t* bytes) {
  if (!h || !bytes) return AS_ERR_INVALID_ARG;
  *bytes = h->ws.total;
  return AS_OK;
}

as_status_t as_hybrid_attn_workspace_bytes_host(as_hybrid_attn_t h, size_t* bytes) {
  if (!h || !bytes) return AS_ERR_INVALID_ARG;
  *bytes = h->ws.total_host;
  return AS_OK;
}

as_status_t as_hybrid_attn_softmax_tokens(as_hybrid_attn_t h, int32_t* count, int32_t* idx_host,
                                          int32_t capacity) {
  if (!h || !count) return AS_ERR_INVALID_ARG;
  if (idx_host) {
    if (capacity < h->n_s) return AS_ERR_INVALID_ARG;
    std::memcpy(idx_host, h->idx_host.data(), sizeof(int32_t) * h->n_s);
  }
  *count = h->n_s;
  return AS_OK;
}

as_status_t as_hybrid_attn_forward(as_hybrid_attn_t h, const void* q, const void* k, const void* v,
                                   const as_phi_weights_t* w, void* out, float* aux,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!h || !q || !k || !v || !out) return AS_ERR_INVALID_ARG;
  if (!on_handle_device(h)) return AS_ERR_INVALID_ARG;
  const auto& d = h->desc;
  const as_status_t ws_ok = check_weights(h, w);
  if (ws_ok != AS_OK) return ws_ok;
  if (((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out) & 15) return AS_ERR_INVALID_ARG;
  if (aux && ((uintptr_t)aux & 3)) return AS_ERR_INVALID_ARG;
  if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < h->ws.total) return AS_ERR_WORKSPACE;
  return launch_heads(h, q, k, v, w, out, aux, (char*)workspace, (cudaStream_t)cuda_stream, 0, d.B * d.H, d.B, d.H);
}

}  // extern "C"

// Launches the kernels for `count` consecutive (batch, head) pairs starting at global pair `first`
// (all of them, or a run of heads inside one batch entry).  q, k, v, out, aux point at the first pair of
// the run; the run is presented to the kernels as nb x nh pairs (nb * nh == count).  Scratch that only
// lives inside one forward (compacted K/V, partial sums) is shared by all runs; S, z and the bf16 S keep
// their place in the full [B*H] arrays, so linear_state sees every pair afterwards.
static as_status_t launch_heads(as_hybrid_attn_t h, const void* q, const void* k, const void* v,
                                const as_phi_weights_t* w, void* out, float* aux, char* ws, cudaStream_t st,
                                int first, int count, int nb, int nh, int stages, const as_ext_state* ext) {
  const auto& d = h->desc;
  // with outside state the linear branch exists when a state is given, whatever this handle's own tokens are
  const bool lin = ext ? (ext->S != nullptr) : (h->n_l > 0);
  const int head0 = first % d.H;                 // the run's first head: where its weights start
  const size_t F = d.phi_dim, dd = d.d;
  (void)count;
  as_launch_args a{};
  a.q = (const __nv_bfloat16*)q; a.k = (const __nv_bfloat16*)k; a.v = (const __nv_bfloat16*)v;
  const bool two = lin && d.phi_layers == 2;
  const size_t hid = two ? d.phi_hidden : 0;
  const size_t w1 = (two ? hid : F) * dd;        // elements of one head's first-layer matrix
  const size_t b1 = two ? hid : F;               // ... and of its bias
  auto at = [](const void* p, size_t off) { return p ? (const __nv_bfloat16*)p + off : nullptr; };
  a.wq = lin ? at(w->wq1, head0 * w1) : nullptr;
  a.wk = lin ? at(w->wk1, head0 * w1) : nullptr;
  a.wq2 = two ? at(w->wq2, head0 * F * hid) : nullptr;
  a.wk2 = two ? at(w->wk2, head0 * F * hid) : nullptr;
  a.bq1 = lin ? at(w->bq1, head0 * b1) : nullptr;
  a.bk1 = lin ? at(w->bk1, head0 * b1) : nullptr;
  a.bq2 = two ? at(w->bq2, head0 * F) : nullptr;
  a.bk2 = two ? at(w->bk2, head0 * F) : nullptr;
  a.h1k = two ? (__nv_bfloat16*)(ws + h->ws.h1k) : nullptr;
  a.layers = d.phi_layers;
  a.hid = (int)hid;
  a.out = (__nv_bfloat16*)out; a.aux = aux;
  const bool compact = h->n_s > 0 && lin;
  a.ks_w = compact ? (__nv_bfloat16*)(ws + h->ws.ks) : nullptr;
  a.vs_w = compact ? (__nv_bfloat16*)(ws + h->ws.vs) : nullptr;
  a.ks = compact ? a.ks_w : a.k;
  a.vs = compact ? a.vs_w : a.v;
  a.part_s = (float*)(ws + h->ws.part_s); a.part_z = (float*)(ws + h->ws.part_z);
  a.S = (float*)(ws + h->ws.S) + (size_t)first * F * dd; a.z = (float*)(ws + h->ws.z) + (size_t)first * F;
  a.Sb = (__nv_bfloat16*)(ws + h->ws.Sb) + (size_t)first * F * dd;
  a.sm_rank = h->d_sm_rank; a.status = h->d_status; a.counters = h->d_counters;
  a.B = nb; a.H = nh; a.N = d.N; a.d = d.d; a.F = d.phi_dim; a.P = d.poly_degree;
  a.n_s = h->n_s; a.n_l = h->n_l; a.n_chunks = h->n_chunks; a.chunk_tiles = h->chunk_tiles;
  a.scale = h->scale; a.stab_mode = d.stab_mode;
  const bool simt = d.kernel_path == AS_PATH_SIMT;
  cudaError_t e = cudaSuccess;
  if (ext) {
    // query stage on gathered keys and a summed state: S as the bf16 operand into this workspace
    a.ks = (const __nv_bfloat16*)ext->ks; a.vs = (const __nv_bfloat16*)ext->vs;
    a.ks_w = a.vs_w = nullptr;
    a.n_s = ext->n_keys; a.n_l = lin ? 1 : 0;
    if (lin) {
      a.S = const_cast<float*>(ext->S); a.z = const_cast<float*>(ext->z);
      { ProfileScope p(h, st, AS_KERNEL_REDUCE);
        e = as_round_state(a, st); }
      if (e != cudaSuccess) { cudaGetLastError(); return AS_ERR_CUDA; }
    }
  }
  if (!(stages & AS_STAGE_KEYS)) goto queries;
  if (two) {
    { ProfileScope p(h, st, AS_KERNEL_KPASS);     // counted with the K pass: it feeds it
      e = as_tensor_phi1(a, st); }
    if (e != cudaSuccess) { cudaGetLastError(); return AS_ERR_CUDA; }
  }
  if (lin) {
    { ProfileScope p(h, st, AS_KERNEL_KPASS);
      e = simt ? as_simt_kpass(a, st) : as_tensor_kpass(a, st); }
    if (e != cudaSuccess) { cudaGetLastError(); return AS_ERR_CUDA; }
    if (simt) {
      // (the tensor K pass adds the chunks up itself, every CTA of a head a slice, once the head's CTAs have all stored)
      { ProfileScope p(h, st, AS_KERNEL_REDUCE);
        e = as_reduce_state(a, st); }
      if (e != cudaSuccess) { cudaGetLastError(); return AS_ERR_CUDA; }
    }
  }
queries:
  if (!(stages & AS_STAGE_QUERIES)) return AS_OK;
  { ProfileScope p(h, st, AS_KERNEL_QPASS);
    e = simt ? as_simt_qpass(a, st) : as_tensor_qpass(a, st); }
  if (e != cudaSuccess) { cudaGetLastError(); return AS_ERR_CUDA; }
  return AS_OK;
}

extern "C" {

as_status_t as_hybrid_attn_forward_host(as_hybrid_attn_t h, const void* q_host, const void* k_host,
                                        const void* v_host, const as_phi_weights_t* w,
                                        void* out_host, void* workspace, size_t workspace_bytes,
                                        void* cuda_stream) {
  if (!h || !q_host || !k_host || !v_host || !out_host) return AS_ERR_INVALID_ARG;
  if (!on_handle_device(h)) return AS_ERR_INVALID_ARG;
  if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < h->ws.total_host) return AS_ERR_WORKSPACE;
  const auto& d = h->desc;
  const as_status_t ws_ok = check_weights(h, w);
  if (ws_ok != AS_OK) return ws_ok;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  char* ws = (char*)workspace;
  // The three copies in, the kernels and the copy out of one run of heads form a pipeline over runs:
  // copies in on one side stream, kernels on the caller's stream, copies out on another side stream, so
  // that both directions of the host link and the kernels work at the same time.  A run is a whole
  // number of heads of one batch entry with at least ~8 MB of q.
  const size_t head_bytes = (size_t)d.N * d.d * 2;
  int run = (int)std::min<size_t>((size_t)d.H, std::max<size_t>(1, ((size_t)8 << 20) / head_bytes));
  const int runs_per_batch = (d.H + run - 1) / run;
  const int n_runs = d.B * runs_per_batch;
  if (!h->side_ready) {
    if (cudaStreamCreateWithFlags(&h->s_in, cudaStreamNonBlocking) != cudaSuccess ||
        cudaStreamCreateWithFlags(&h->s_out, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming) != cudaSuccess) {
      cudaGetLastError(); return AS_ERR_CUDA;
    }
    h->side_ready = true;
  }
  while ((int)h->ev_run.size() < 2 * n_runs) {
    cudaEvent_t e;
    if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) { cudaGetLastError(); return AS_ERR_CUDA; }
    h->ev_run.push_back(e);
  }
  bool ok = cudaEventRecord(h->ev_fork, st) == cudaSuccess &&
            cudaStreamWaitEvent(h->s_in, h->ev_fork, 0) == cudaSuccess &&
            cudaStreamWaitEvent(h->s_out, h->ev_fork, 0) == cudaSuccess;
  as_status_t status = AS_OK;
  for (int r = 0; ok && r < n_runs; ++r) {
    const int b = r / runs_per_batch, h0 = (r % runs_per_batch) * run;
    const int nh = std::min(run, d.H - h0);
    const int first = b * d.H + h0;
    const size_t off = (size_t)first * head_bytes, bytes = (size_t)nh * head_bytes;
    cudaEvent_t ev_in = h->ev_run[2 * r], ev_done = h->ev_run[2 * r + 1];
    ok = cudaMemcpyAsync(ws + h->ws.stage_q + off, (const char*)q_host + off, bytes, cudaMemcpyHostToDevice, h->s_in) == cudaSuccess &&
         cudaMemcpyAsync(ws + h->ws.stage_k + off, (const char*)k_host + off, bytes, cudaMemcpyHostToDevice, h->s_in) == cudaSuccess &&
         cudaMemcpyAsync(ws + h->ws.stage_v + off, (const char*)v_host + off, bytes, cudaMemcpyHostToDevice, h->s_in) == cudaSuccess &&
         cudaEventRecord(ev_in, h->s_in) == cudaSuccess && cudaStreamWaitEvent(st, ev_in, 0) == cudaSuccess;
    if (!ok) break;
    status = launch_heads(h, ws + h->ws.stage_q + off, ws + h->ws.stage_k + off, ws + h->ws.stage_v + off, w,
                          ws + h->ws.stage_o + off, nullptr, ws, st, first, nh, 1, nh);
    if (status != AS_OK) break;
    ok = cudaEventRecord(ev_done, st) == cudaSuccess && cudaStreamWaitEvent(h->s_out, ev_done, 0) == cudaSuccess &&
         cudaMemcpyAsync((char*)out_host + off, ws + h->ws.stage_o + off, bytes, cudaMemcpyDeviceToHost, h->s_out) == cudaSuccess;
  }
  // join: the caller's stream completes only after the last copy out (and, after an error, after
  // whatever the side streams were already given)
  const bool joined = cudaEventRecord(h->ev_join, h->s_out) == cudaSuccess && cudaStreamWaitEvent(st, h->ev_join, 0) == cudaSuccess &&
                      cudaEventRecord(h->ev_fork, h->s_in) == cudaSuccess && cudaStreamWaitEvent(st, h->ev_fork, 0) == cudaSuccess;
  if (status != AS_OK) return status;
  if (!ok || !joined) { cudaGetLastError(); return AS_ERR_CUDA; }
  return AS_OK;
}

as_status_t as_hybrid_attn_linear_state(as_hybrid_attn_t h, const void* workspace, float* S_out,
                                        float* z_out, void* cuda_stream) {
  if (!h || !workspace) return AS_ERR_INVALID_ARG;
  if (h->n_l == 0 || !on_handle_device(h)) return AS_ERR_INVALID_ARG;
  const auto& d = h->desc;
  const size_t BH = (size_t)d.B * d.H;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const char* ws = (const char*)workspace;
  if (S_out && cudaMemcpyAsync(S_out, ws + h->ws.S, BH * d.phi_dim * d.d * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess) {
    cudaGetLastError(); return AS_ERR_CUDA;
  }
  if (z_out && cudaMemcpyAsync(z_out, ws + h->ws.z, BH * d.phi_dim * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess) {
    cudaGetLastError(); return AS_ERR_CUDA;
  }
  return AS_OK;
}

as_status_t as_hybrid_attn_last_status(as_hybrid_attn_t h, void* cuda_stream) {
  if (!h || !on_handle_device(h)) return AS_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  uint32_t word = 0;
  if (cudaStreamSynchronize(st) != cudaSuccess ||
      cudaMemcpy(&word, h->d_status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError(); return AS_ERR_CUDA;
  }
  // after a time-out CTAs have left early: the K pass's arrival counters may stand anywhere
  if (word != 0 && (cudaMemset(h->d_status, 0, 4) != cudaSuccess ||
                    cudaMemset(h->d_counters, 0, sizeof(uint32_t) * 8 * (size_t)h->desc.B * h->desc.H) != cudaSuccess)) {
    cudaGetLastError(); return AS_ERR_CUDA;
  }
  return (word & AS_DEV_TIMEOUT) ? AS_ERR_DEVICE_TIMEOUT : AS_OK;
}

as_status_t as_hybrid_attn_key_pass(as_hybrid_attn_t h, const void* k, const void* v, const as_phi_weights_t* w,
                                    void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!h || !k || !v) return AS_ERR_INVALID_ARG;
  if (!on_handle_device(h)) return AS_ERR_INVALID_ARG;
  const auto& d = h->desc;
  const as_status_t ws_ok = check_weights(h, w);
  if (ws_ok != AS_OK) return ws_ok;
  if (((uintptr_t)k | (uintptr_t)v) & 15) return AS_ERR_INVALID_ARG;
  if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < h->ws.total) return AS_ERR_WORKSPACE;
  if (h->n_l == 0) return AS_OK;                  // nothing to sum and nothing to compact: the keys are k, v themselves
  return launch_heads(h, k, k, v, w, nullptr, nullptr, (char*)workspace, (cudaStream_t)cuda_stream, 0, d.B * d.H, d.B, d.H,
                      AS_STAGE_KEYS, nullptr);
}

as_status_t as_hybrid_attn_workspace_offsets(as_hybrid_attn_t h, size_t* ks, size_t* vs, size_t* S, size_t* z) {
  if (!h || !ks || !vs || !S || !z) return AS_ERR_INVALID_ARG;
  *ks = h->ws.ks; *vs = h->ws.vs; *S = h->ws.S; *z = h->ws.z;
  return AS_OK;
}

as_status_t as_hybrid_attn_query_pass(as_hybrid_attn_t h, const void* q, const as_phi_weights_t* w, const void* ks,
                                      const void* vs, int32_t n_keys, const float* S, const float* z, void* out,
                                      float* aux, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!h || !q || !out || n_keys < 0 || (n_keys > 0 && (!ks || !vs)) || ((S == nullptr) != (z == nullptr))) return AS_ERR_INVALID_ARG;
  if (n_keys == 0 && !S) return AS_ERR_INVALID_ARG;            // nothing to attend to
  if (!on_handle_device(h)) return AS_ERR_INVALID_ARG;
  const auto& d = h->desc;
  if (S) {
    if (!w || !w->wq1) return AS_ERR_INVALID_ARG;
    if (d.phi_layers == 2 && !w->wq2) return AS_ERR_INVALID_ARG;
    if (((uintptr_t)w->wq1 | (uintptr_t)w->wq2) & 15) return AS_ERR_INVALID_ARG;
    if (((uintptr_t)w->bq1 | (uintptr_t)w->bq2) & 3) return AS_ERR_INVALID_ARG;
  }
  if (((uintptr_t)q | (uintptr_t)out | (uintptr_t)ks | (uintptr_t)vs | (uintptr_t)S) & 15) return AS_ERR_INVALID_ARG;
  if (aux && ((uintptr_t)aux & 3)) return AS_ERR_INVALID_ARG;
  if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < h->ws.total) return AS_ERR_WORKSPACE;
  // the workspace must have room for the bf16 copy of S even when this handle's own tokens are all softmax tokens
  if (S && h->n_l == 0) return AS_ERR_UNSUPPORTED;
  const as_ext_state ext{ks, vs, n_keys, S, z};
  as_phi_weights_t none{};
  return launch_heads(h, q, q, q, w ? w : &none, out, aux, (char*)workspace, (cudaStream_t)cuda_stream, 0, d.B * d.H, d.B, d.H,
                      AS_STAGE_QUERIES, &ext);
}

as_status_t as_hybrid_attn_debug_expire_wait(as_hybrid_attn_t h, int64_t limit_cycles, void* cuda_stream) {
  if (!h || !on_handle_device(h)) return AS_ERR_INVALID_ARG;
  if (limit_cycles < 1 || limit_cycles > 100000000) return AS_ERR_INVALID_ARG;      // at most about 50 ms
  if (as_tensor_expire_wait(h->d_status, limit_cycles, (cudaStream_t)cuda_stream) != cudaSuccess) {
    cudaGetLastError(); return AS_ERR_CUDA;
  }
  return AS_OK;
}

as_status_t as_hybrid_attn_profile_enable(as_hybrid_attn_t h, int32_t enable) {
  if (!h) return AS_ERR_INVALID_ARG;
  if (enable && h->ev.empty()) {
    h->ev.reserve(2 * AS_MAX_PROFILE);
    for (int i = 0; i < 2 * AS_MAX_PROFILE; ++i) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) { cudaGetLastError(); return AS_ERR_CUDA; }
      h->ev.push_back(e);
    }
    h->ev_class.assign(AS_MAX_PROFILE, 0);
  }
  h->profiling = enable != 0;
  h->ev_used = 0;
  return AS_OK;
}

as_status_t as_hybrid_attn_profile_read(as_hybrid_attn_t h, float* ms, int32_t* launches) {
  if (!h || !ms || !launches) return AS_ERR_INVALID_ARG;
  float acc[AS_NUM_KERNELS] = {0.f, 0.f, 0.f};
  int32_t cnt[AS_NUM_KERNELS] = {0, 0, 0};
  for (int i = 0; i < h->ev_used; ++i) {
    if (cudaEventSynchronize(h->ev[2 * i + 1]) != cudaSuccess) { cudaGetLastError(); return AS_ERR_CUDA; }
    float t = 0.f;
    if (cudaEventElapsedTime(&t, h->ev[2 * i], h->ev[2 * i + 1]) != cudaSuccess) { cudaGetLastError(); return AS_ERR_CUDA; }
    acc[h->ev_class[i]] += t;
    cnt[h->ev_class[i]]++;
  }
  for (int c = 0; c < AS_NUM_KERNELS; ++c) { ms[c] = acc[c]; launches[c] = cnt[c]; }
  h->ev_used = 0;
  return AS_OK;
}

as_status_t as_hybrid_attn_launch_count(as_hybrid_attn_t h, uint64_t* count) {
  if (!h || !count) return AS_ERR_INVALID_ARG;
  *count = h->launches;
  return AS_OK;
}

}  // extern "C"
