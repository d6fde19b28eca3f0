// Query stage of a layer WITHOUT softmax tokens (rate 0), one-layer feature map with F = d = 128, no bias, degree <= 2:
//   y_i = phi_q(q_i) S / (phi_q(q_i) . z)         (the hybrid-attention equation with T_S empty)
// The work per row is small (two 128 x 128 x 128 products), so the kernel has to stream: q in, y out, both once.
// A persistent CTA owns a contiguous run of 128-row tiles (tiles of one (batch, head) are consecutive, so the
// weights W and the state S of a head are loaded once or twice per CTA) and keeps several tiles in flight:
//
//   TMA warp          Q tiles into a ring of three slots; W and S (bf16) whenever the (batch, head) changes
//   issuing thread 1  Phi = Q W^T           -> TMEM, one accumulator per group (as soon as Q is there and the
//                                              group has read its previous Phi)
//   compute warps     two groups of four warps, tiles alternate between the groups; one thread per row:
//                     phi_q = poly(relu(Phi)) as bf16 into the group's shared-memory tile, phi_q . z on the way;
//                     later O / (phi_q . z) as bf16 into the same tile, one TMA store per warp
//   issuing thread 2  O = phi_q S           -> TMEM, one accumulator per group
//
// Every wait is bounded (status word, abort flag), as in the other kernels.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "tensor_common.cuh"

namespace {

using namespace as_tc;

constexpr int QS_THREADS = 352;          // warps 0-3 / 4-7: compute groups 0 / 1; warp 8: TMA; warps 9, 10: MMA issuers
constexpr int QS_SLOTS = 3;              // Q tiles in flight
constexpr int TILE = 128 * 128 * 2;      // bytes of a [128 x 128] bf16 tile

struct QSParams {
  int N, H, P;
  int nt;                    // 128-row tiles per (batch, head)
  long long tiles;           // tiles over all (batch, head) pairs
  const float* z;            // [B*H][128]
  float* aux;                // [B*H][N][3] or nullptr
  uint32_t* status;
};

struct QSLayout {
  static constexpr int W_OFF = 0, ST_OFF = TILE, Q_OFF = 2 * TILE, PHI_OFF = Q_OFF + QS_SLOTS * TILE;
  static constexpr int BAR_OFF = PHI_OFF + 2 * TILE;
  static constexpr int TOTAL = BAR_OFF + 256 + 1024;         // + slack for the 1024-byte alignment
};
// barriers
constexpr int B_QFULL = 0, B_QEMPTY = B_QFULL + QS_SLOTS, B_WFULL = B_QEMPTY + QS_SLOTS, B_WFREE = B_WFULL + 1,
              B_PHI = B_WFREE + 1, B_PHIF = B_PHI + 2, B_P = B_PHIF + 2, B_O = B_P + 2, B_OF = B_O + 2, B_COUNT = B_OF + 2;

struct QSCtx {
  uint32_t sbase, tmem;
  WaitCtx wc;
  long long t0, t1;          // this CTA's tiles [t0, t1)
  AS_DEV uint32_t bar(int i) const { return sbase + QSLayout::BAR_OFF + 8 * i; }
  AS_DEV bool wait(int b, int phase) const { return mbar_wait(bar(b), phase & 1, wc); }
  AS_DEV bool wait_warp(int b, int phase) const { return mbar_wait_warp(bar(b), phase & 1, wc); }
  AS_DEV uint32_t tPhi(int g) const { return tmem + 128u * g; }
  AS_DEV uint32_t tO(int g) const { return tmem + 256u + 128u * g; }
};

// tile t belongs to (batch, head) pair t / nt
AS_DEV int qs_bh(const QSParams& p, long long t) { return (int)(t / p.nt); }

// ---------------------------------------------------------------- TMA producer
__device__ __noinline__ void qs_produce(const QSParams& p, const QSCtx& c, const CUtensorMap* tmQ, const CUtensorMap* tmW,
                                        const CUtensorMap* tmSt) {
  const int lane = threadIdx.x & 31;
  const int n = (int)(c.t1 - c.t0);
  int seg = -1, bh_prev = -1;
  for (int i = 0; i < n; ++i) {
    const long long t = c.t0 + i;
    const int bh = qs_bh(p, t), row0 = (int)(t % p.nt) * 128, slot = i % QS_SLOTS;
    if (!c.wait_warp(B_QEMPTY + slot, i / QS_SLOTS + 1)) return;      // the product that read the slot has completed
    if (lane == 0) {
      mbar_expect_tx(c.bar(B_QFULL + slot), TILE);
      load_tile<128>(c.sbase + QSLayout::Q_OFF + slot * TILE, tmQ, c.bar(B_QFULL + slot), row0, bh);
    }
    __syncwarp();
    if (bh != bh_prev) {
      // a new (batch, head): its weights and state replace the previous pair's once every product that reads
      // those has completed
      ++seg;
      if (seg > 0 && !c.wait_warp(B_WFREE, seg - 1)) return;
      if (lane == 0) {
        mbar_expect_tx(c.bar(B_WFULL), 2 * TILE);
        load_tile<128>(c.sbase + QSLayout::W_OFF, tmW, c.bar(B_WFULL), 0, bh % p.H);
        load_tile<128>(c.sbase + QSLayout::ST_OFF, tmSt, c.bar(B_WFULL), 0, bh);
      }
      __syncwarp();
      bh_prev = bh;
    }
  }
}

// ---------------------------------------------------------------- issuing thread 1: Phi = Q W^T
__device__ __noinline__ void qs_issue_phi(const QSParams& p, const QSCtx& c) {
  constexpr uint32_t ID = make_idesc(128, 128, 0, 0);
  const int n = (int)(c.t1 - c.t0);
  const uint64_t w0 = kmajor_desc(c.sbase + QSLayout::W_OFF);
  int seg = -1, bh_prev = -1;
  for (int i = 0; i < n; ++i) {
    const int g = i & 1, k = i >> 1, slot = i % QS_SLOTS;
    const int bh = qs_bh(p, c.t0 + i);
    if (bh != bh_prev) {
      ++seg;
      if (!c.wait(B_WFULL, seg)) return;
      bh_prev = bh;
    }
    if (k > 0 && !c.wait(B_PHIF + g, k - 1)) return;                  // the group has read its previous Phi
    if (!c.wait(B_QFULL + slot, i / QS_SLOTS)) return;
    tc_fence_after();
    issue_kmajor<128>(c.tPhi(g), kmajor_desc(c.sbase + QSLayout::Q_OFF + slot * TILE), w0, ID, false);
    tc_commit(c.bar(B_PHI + g));
    tc_commit(c.bar(B_QEMPTY + slot));
  }
}

// ---------------------------------------------------------------- issuing thread 2: O = phi_q S
__device__ __noinline__ void qs_issue_out(const QSParams& p, const QSCtx& c) {
  constexpr uint32_t ID = make_idesc(128, 128, 0, 1);          // S is MN-major (feature rows, d contiguous)
  const int n = (int)(c.t1 - c.t0);
  const uint64_t s0 = mnmajor_desc(c.sbase + QSLayout::ST_OFF);
  for (int i = 0; i < n; ++i) {
    const int g = i & 1, k = i >> 1;
    if (!c.wait(B_P + g, k)) return;                                  // phi_q of this tile is in shared memory
    if (k > 0 && !c.wait(B_OF + g, k - 1)) return;                    // the group has read its previous O
    tc_fence_after();
    const uint64_t a0 = kmajor_desc(c.sbase + QSLayout::PHI_OFF + g * TILE);
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) mma_ss(c.tO(g), a0 + kstep_kmajor(kk), s0 + kstep_mnmajor(kk), ID, kk > 0 ? 1u : 0u);
    tc_commit(c.bar(B_O + g));
    // the last tile of a (batch, head): once its product has completed nothing reads W or S of that pair any more
    const bool last_of_pair = (i + 1 == n) || (qs_bh(p, c.t0 + i + 1) != qs_bh(p, c.t0 + i));
    if (last_of_pair) tc_commit(c.bar(B_WFREE));
  }
}

// ---------------------------------------------------------------- compute group: its tiles i = g, g + 2, ...
__device__ __noinline__ void qs_compute(const QSParams& p, const QSCtx& c, const CUtensorMap* tmO, uint8_t* smem) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = warp >> 2, quad = warp & 3;
  const int r = quad * 32 + lane;                    // row inside the 128-row tile
  const uint32_t lane_off = (uint32_t)(quad * 32) << 16;
  const uint32_t tPhi = c.tPhi(g) + lane_off, tO = c.tO(g) + lane_off;
  uint8_t* tile = smem + QSLayout::PHI_OFF + g * TILE;     // phi_q, then the output rows
  const int n = (int)(c.t1 - c.t0);
  const int part = 128 / p.P;
  uint32_t x[32];
  for (int i = g, k = 0; i < n; i += 2, ++k) {
    const long long t = c.t0 + i;
    const int bh = qs_bh(p, t), row = (int)(t % p.nt) * 128 + r;
    const float2* zrow = reinterpret_cast<const float2*>(p.z + (size_t)bh * 128);
    // ---- phi_q = poly(relu(Phi)) as bf16, and its product with z from the very values the MMA multiplies with S
    if (!c.wait_warp(B_PHI + g, k)) return;
    tc_fence_after();
    if (lane == 0) tma_store_wait_read();            // this warp's previous output store has been read out of the tile
    __syncwarp();
    float dl0 = 0.f, dl1 = 0.f;
#pragma unroll
    for (int cc = 0; cc < 4; ++cc) {
      tmem_ld32(tPhi + cc * 32, x);
      tmem_ld_wait(x);
      const int pw = min((cc * 32) / part, p.P - 1);   // 0: the feature itself, 1: its square
      uint32_t wd[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const float a0 = fmaxf(__uint_as_float(x[2 * j]), 0.f), a1 = fmaxf(__uint_as_float(x[2 * j + 1]), 0.f);
        const float r0 = pw >= 1 ? a0 * a0 : a0, r1 = pw >= 1 ? a1 * a1 : a1;
        wd[j] = pack_bf16(r0, r1);
        const float2 zz = __ldg(zrow + cc * 16 + j);
        dl0 = fmaf(__uint_as_float(wd[j] << 16), zz.x, dl0);
        dl1 = fmaf(__uint_as_float(wd[j] & 0xffff0000u), zz.y, dl1);
      }
      store_row_chunk(tile, r, cc * 32, wd);
    }
    tc_fence_before();
    mbar_arrive(c.bar(B_PHIF + g));                  // the next Phi of this group may land
    fence_proxy_async();
    mbar_arrive(c.bar(B_P + g));
    const float den = dl0 + dl1;
    // ---- y = O / den, staged in the same tile (the product that read phi_q from it has completed with O)
    if (!c.wait_warp(B_O + g, k)) return;
    tc_fence_after();
    const float inv = 1.f / den;
#pragma unroll
    for (int cc = 0; cc < 4; ++cc) {
      tmem_ld32(tO + cc * 32, x);
      tmem_ld_wait(x);
      uint32_t wd[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) wd[j] = pack_bf16(__uint_as_float(x[2 * j]) * inv, __uint_as_float(x[2 * j + 1]) * inv);
      store_row_chunk(tile, r, cc * 32, wd);
    }
    tc_fence_before();
    mbar_arrive(c.bar(B_OF + g));                    // the next O of this group may land
    fence_proxy_async();
    __syncwarp();
    const int wrow0 = row - lane;
    if (lane == 0 && wrow0 < p.N) {
#pragma unroll
      for (int b = 0; b < 2; ++b) tma_store_3d(tmO, smem_u32(tile) + b * BOX_BYTES + quad * 32 * 128, b * 64, wrow0, bh);
      tma_store_commit();
    }
    if (p.aux != nullptr && row < p.N) {
      float* ap = p.aux + ((size_t)bh * p.N + row) * 3;
      ap[0] = 0.f; ap[1] = 0.f; ap[2] = den;
    }
  }
  if (lane == 0) tma_store_wait_read();              // this warp's output stores have read their rows (the writes land by the end of the kernel)
}

__global__ void __launch_bounds__(QS_THREADS, 1)
qstream_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmW,
               const __grid_constant__ CUtensorMap tmSt, const __grid_constant__ CUtensorMap tmO, const __grid_constant__ QSParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t sbase = smem_u32(smem);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + QSLayout::BAR_OFF + 8 * B_COUNT);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + QSLayout::BAR_OFF + 8 * B_COUNT + 4);
  const int warp = threadIdx.x >> 5;

  // an earlier CTA of this or a previous launch timed out: do nothing (decided once per CTA)
  __shared__ uint32_t s_skip;
  if (threadIdx.x == 0) s_skip = *reinterpret_cast<volatile uint32_t*>(p.status);
  __syncthreads();
  if (s_skip != 0u) return;

  if (threadIdx.x == 0) {
    *abort_flag = 0u;
    auto bar = [&](int i) { return sbase + QSLayout::BAR_OFF + 8 * i; };
    for (int s = 0; s < QS_SLOTS; ++s) { mbar_init(bar(B_QFULL + s), 1); mbar_init(bar(B_QEMPTY + s), 1); }
    mbar_init(bar(B_WFULL), 1); mbar_init(bar(B_WFREE), 1);
    for (int g = 0; g < 2; ++g) {
      mbar_init(bar(B_PHI + g), 1); mbar_init(bar(B_PHIF + g), 128); mbar_init(bar(B_P + g), 128);
      mbar_init(bar(B_O + g), 1); mbar_init(bar(B_OF + g), 128);
    }
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 9) { tmem_alloc(smem_u32(tmem_slot), 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // Every CTA gets a contiguous run of tiles.  With at least as many CTAs as (batch, head) pairs no run crosses a
  // pair (a change of pair stalls the pipeline while W and S are replaced): the pairs get floor or ceil(G / pairs)
  // CTAs each, which share the pair's tiles evenly.  Otherwise the tiles of all pairs are cut into G near-equal runs.
  const long long G = gridDim.x, cta = blockIdx.x, pairs = p.tiles / p.nt;
  long long t0, t1;
  if (G >= pairs) {
    const long long base = G / pairs, extra = G % pairs;             // the first `extra` pairs get base + 1 CTAs
    const bool big = cta < extra * (base + 1);
    const long long pair = big ? cta / (base + 1) : extra + (cta - extra * (base + 1)) / base;
    const long long m = big ? base + 1 : base, j = big ? cta % (base + 1) : (cta - extra * (base + 1)) % base;
    t0 = pair * p.nt + j * p.nt / m;
    t1 = pair * p.nt + (j + 1) * p.nt / m;
  } else {
    t0 = cta * p.tiles / G;
    t1 = (cta + 1) * p.tiles / G;
  }
  const QSCtx c{sbase, *tmem_slot, WaitCtx{p.status, abort_flag}, t0, t1};

  if (warp == 8) {
    if ((threadIdx.x & 31) == 0) { tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmW); tma_prefetch_desc(&tmSt); tma_prefetch_desc(&tmO); }
    qs_produce(p, c, &tmQ, &tmW, &tmSt);
  } else if (warp == 9) {
    if ((threadIdx.x & 31) == 0) qs_issue_phi(p, c);
    __syncwarp();
  } else if (warp == 10) {
    if ((threadIdx.x & 31) == 0) qs_issue_out(p, c);
    __syncwarp();
  } else {
    qs_compute(p, c, &tmO, smem);
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 9) {
    tc_fence_after();
    tmem_dealloc(c.tmem, 512);
  }
}

}  // namespace

cudaError_t as_tensor_init_qstream() { return opt_in_smem(qstream_kernel, QSLayout::TOTAL); }

bool as_tensor_qstream_handles(const as_launch_args& a) {
  return a.n_s == 0 && a.n_l > 0 && a.layers == 1 && a.d == 128 && a.F == 128 && a.P <= 2 && a.bq1 == nullptr;
}

cudaError_t as_tensor_qstream(const as_launch_args& a, cudaStream_t st) {
  const int BH = a.B * a.H;
  CUtensorMap tmQ, tmW, tmSt, tmO;
  // the output is stored warp by warp: boxes of 32 rows
  if (!make_map(&tmQ, a.q, a.d, a.N, BH, 128) || !make_map(&tmO, a.out, a.d, a.N, BH, 32) ||
      !make_map(&tmW, a.wq, a.d, a.F, a.H, 128) || !make_map(&tmSt, a.Sb, a.d, a.F, BH, 128))
    return cudaErrorInvalidValue;
  QSParams p{};
  p.N = a.N; p.H = a.H; p.P = a.P;
  p.nt = (a.N + 127) / 128;
  p.tiles = (long long)p.nt * BH;
  p.z = a.z; p.aux = a.aux; p.status = a.status;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
    return cudaErrorInvalidValue;
  const dim3 grid((unsigned)(p.tiles < sms ? p.tiles : sms), 1, 1);   // persistent: one CTA per SM
  qstream_kernel<<<grid, QS_THREADS, QSLayout::TOTAL, st>>>(tmQ, tmW, tmSt, tmO, p);
  return cudaGetLastError();
}
