// K pass of the hybrid attention forward on the tensor cores of sm_100a (phi_k projection, linear
// state, softmax gather) and the first layer of a two-layer feature map for the keys.
//
//   One CTA = (chunk of 128-token tiles, batch*head, chunk of 128 features).  Per token tile:
//     Phi^T = W X^T       tcgen05.mma, smem x smem -> TMEM; TMEM lane = feature, column = token.
//                         One layer: W = W_k rows of the feature chunk, X = the K tile.  Two layers:
//                         W = W_k2[feature chunk, :], X = relu(K W_k1^T + b1) as left by phi1_kernel,
//                         one MMA chain per 128-wide slice of the hidden width.
//     phi   = poly(relu(Phi + b)), zero for softmax tokens and past the sequence end, rounded to bf16
//             into spare TMEM columns (eight feature warps, two per lane quadrant)
//     S    += phi^T-tile V   tcgen05.mma, TMEM x smem -> TMEM accumulator that lives across the chunk
//     z    += the bf16 features, summed per feature in registers
//     the tile's softmax-token rows are copied to the compact K_S / V_S (feature chunk 0 only).
//   All tiles travel through one ring of shared-memory slots filled by TMA; every mbarrier wait is bounded.
#include "tensor_common.cuh"

namespace {

using namespace as_tc;

struct KParams {
  int N, n_s, n_chunks, chunk_tiles, P, F, H;
  const int32_t* sm_rank;              // [N (+ padding)]: position in T_S, or -1 for a linear token
  __nv_bfloat16 *ks_w, *vs_w;          // compact softmax K / V (nullptr when nothing is gathered)
  const __nv_bfloat16* k;              // two-layer maps gather the softmax K rows from here (no K tile in the ring)
  const __nv_bfloat16* bias;           // last-layer bias [H][F], or nullptr
  float *part_s, *part_z;
  float *S, *z;                        // [B*H][F][D], [B*H][F]: the chunks' partials added up ...
  __nv_bfloat16* Sb;                   // ... and S once more rounded to bf16 (the query stage's MMA operand)
  uint32_t* counters;                  // [B*H][feature chunks][2]: CTAs that have stored / that have added; zero between launches
  uint32_t* status;
};

constexpr int K_THREADS = 384;           // warps 0-7: feature warps; 8: TMA; 9: MMA issuer; 10-11: gather
constexpr int K_FEATURE_THREADS = 256;

// LAYERS == 1: ring items per token tile are (K, V), one resident weight tile.
// LAYERS == 2: ring items are (h1 slice 0 .. NH-1, V), NH resident weight tiles W_2[feature chunk, hidden slice].
// Every tile is [128 rows x D columns] bf16 (a hidden slice is D wide).
template <int D, int LAYERS, int NH>
struct KLayout {
  static constexpr int NX = LAYERS == 1 ? 1 : NH;               // tiles that feed the feature product
  static constexpr int IPT = NX + 1;                            // ring items per token tile
  static constexpr int TILE = 128 * D * 2;
  static constexpr int SLOTS = D == 128 ? 7 - NH : 8;
  static constexpr int W_OFF = 0;
  static constexpr int RING_OFF = NH * TILE;
  static constexpr int BAR_OFF = RING_OFF + SLOTS * TILE;
  static constexpr int N_BARS = 1 + 2 * SLOTS + 5;
  static constexpr int PAIR_OFF = BAR_OFF + 8 * N_BARS + 16;    // 2 x 64 words: per token pair, which halves are linear tokens
  static constexpr int Z_OFF = PAIR_OFF + 2 * 64 * 4;           // 128 floats: z of the upper column half
  static constexpr int TOTAL = Z_OFF + 128 * 4 + 1024;          // + slack for the 1024-byte alignment
  // the chunk's partial S leaves through the ring (idle by then): 128 rows of D floats, each row padded by 16
  // bytes so that the 32 lanes of a warp, one row each, write to different banks
  static constexpr int OUT_PITCH = D * 4 + 16;
  static_assert(128 * OUT_PITCH <= SLOTS * TILE, "staging area");
};

// Features of 32 token columns of one TMEM lane: bias, ReLU, power, linear-token mask, bf16.
template <int POW>
AS_DEV void k_features(const uint32_t (&x)[32], const uint4* mask4, float bias, uint32_t (&w)[16], float& z0, float& z1) {
#pragma unroll
  for (int g4 = 0; g4 < 4; ++g4) {
    const uint4 m = mask4[g4];
    const uint32_t mm[4] = {m.x, m.y, m.z, m.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int i = 4 * g4 + e;
      float a0 = fmaxf(__uint_as_float(x[2 * i]) + bias, 0.f), a1 = fmaxf(__uint_as_float(x[2 * i + 1]) + bias, 0.f);
      if (POW == 2) { a0 *= a0; a1 *= a1; }
      if (POW == 3) { a0 = a0 * a0 * a0; a1 = a1 * a1 * a1; }
      if (POW == 4) { a0 *= a0; a1 *= a1; a0 *= a0; a1 *= a1; }
      w[i] = pack_bf16(a0, a1) & mm[e];
      // z sums the features as the MMA sees them: the bf16 values
      add_bf16x2(z0, z1, w[i]);
    }
  }
}

template <int D, int LAYERS, int NH>
__global__ void __launch_bounds__(K_THREADS, 1)
kpass_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
             const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmH, const KParams p) {
  using L = KLayout<D, LAYERS, NH>;
  constexpr int SLOTS = L::SLOTS, IPT = L::IPT, NX = L::NX;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t sbase = smem_u32(smem);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::BAR_OFF);
  enum { B_W = 0, B_FULL = 1, B_EMPTY = B_FULL + SLOTS, B_D1 = B_EMPTY + SLOTS, B_PK = B_D1 + 2, B_DONE = B_PK + 2,
         B_COUNT = B_DONE + 1 };
  static_assert(B_COUNT == L::N_BARS, "barrier count");
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::BAR_OFF + 8 * B_COUNT);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + L::BAR_OFF + 8 * B_COUNT + 4);
  uint32_t* sPair = reinterpret_cast<uint32_t*>(smem + L::PAIR_OFF);
  float* sZ = reinterpret_cast<float*>(smem + L::Z_OFF);
  auto bar = [&](int i) { return smem_u32(bars + i); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int bh = blockIdx.y, h = bh % p.H, chunk = blockIdx.x, fc = blockIdx.z;
  const int tiles_total = (p.N + 127) / 128;
  const int t_begin = chunk * p.chunk_tiles;
  const int nt = min(p.chunk_tiles, tiles_total - t_begin);
  const WaitCtx wc{p.status, abort_flag};
  const bool gathers = (p.ks_w != nullptr) && fc == 0;       // this CTA copies the softmax rows out

  __shared__ uint32_t s_skip;
  if (threadIdx.x == 0) s_skip = *reinterpret_cast<volatile uint32_t*>(p.status);
  __syncthreads();
  if (s_skip != 0u) return;

  auto sW = [&](int j) { return sbase + L::W_OFF + j * L::TILE; };
  auto sSlot = [&](int it) { return sbase + L::RING_OFF + (it % SLOTS) * L::TILE; };
  // one ring item: tile t's K (one layer) or hidden slice i (two layers), or its V tile
  auto load_item = [&](int it) {
    const int st = it % SLOTS, t = it / IPT, i = it % IPT, row = (t_begin + t) * 128;
    mbar_expect_tx(bar(B_FULL + st), L::TILE);
    if (i == NX) load_tile<D>(sSlot(it), &tmV, bar(B_FULL + st), row, bh);
    else if (LAYERS == 1) load_tile<D>(sSlot(it), &tmK, bar(B_FULL + st), row, bh);
    else load_boxes(sSlot(it), &tmH, bar(B_FULL + st), i * D, row, bh, D / 64);
  };
  constexpr int FIRST = SLOTS;                               // items requested before the CTA has finished setting up: the whole ring

  if (threadIdx.x == 0) {
    *abort_flag = 0u;
    for (int b = 0; b < 2; ++b) { mbar_init(bar(B_D1 + b), 1); mbar_init(bar(B_PK + b), K_FEATURE_THREADS); }
    mbar_init(bar(B_DONE), 1);
    fence_barrier_init();
  }
  if (threadIdx.x == 8 * 32) {
    // The producer sets up the barriers of the ring itself and requests the weights and the first tiles at
    // once: the first bytes of a CTA take several microseconds to arrive, and the allocation of tensor memory
    // and the CTA-wide barrier below need not be waited for.
    mbar_init(bar(B_W), 1);
    // a slot is free again when the MMA that read it has completed and, where rows are gathered, when both
    // gather warps are through with it
    for (int s = 0; s < SLOTS; ++s) { mbar_init(bar(B_FULL + s), 1); mbar_init(bar(B_EMPTY + s), gathers ? 3 : 1); }
    fence_barrier_init();
    fence_proxy_async();
    mbar_expect_tx(bar(B_W), NH * L::TILE);
    // rows past F are out of bounds and arrive as zeros
    for (int j = 0; j < NH; ++j) load_boxes(sW(j), &tmW, bar(B_W), j * D, fc * 128, h, D / 64);
    for (int it = 0; it < FIRST && it < nt * IPT; ++it) load_item(it);
  }
  if (warp == 9) { tmem_alloc(smem_u32(tmem_slot), 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tD1[2] = {tmem + 0u, tmem + 128u};          // Phi^T of a tile, fp32
  const uint32_t tAcc = tmem + 256u;                         // S of this feature chunk
  const uint32_t tPA[2] = {tmem + 384u, tmem + 448u};        // the tile's features as packed bf16 (A operand)

  if (warp == 8) {
    // ------------------------------------------------------------ TMA producer
    for (int it = FIRST; it < nt * IPT; ++it) {              // the first items were requested during set-up
      const int st = it % SLOTS;
      if (!mbar_wait_warp(bar(B_EMPTY + st), ((it / SLOTS) & 1) ^ 1, wc)) break;
      if (lane == 0) load_item(it);
      __syncwarp();
    }
  } else if (warp == 9) {
    // ------------------------------------------------------------ MMA issuer (one thread)
    // Two kinds of product per tile: Phi^T(t) as soon as the tile's X items have landed, and S += phi^T V (t) as
    // soon as the feature warps have packed the tile.  The thread issues whichever is ready, so that neither a
    // late tile holds up the accumulation of an earlier one (and with it the release of its V slot) nor the
    // other way round.  Phi^T(t) reuses the columns the feature warps read for tile t - 2 and its features will
    // overwrite the packed operand of S(t - 2): it is only issued once S(t - 2) has been (products of one thread
    // complete in order).
    if (lane == 0) {
      constexpr uint32_t ID_PHI = make_idesc(128, 128, 0, 0);    // Phi^T = W X^T : M = features, N = 128 tokens
      constexpr uint32_t ID_ACC = make_idesc(128, D, 0, 1);      // S += phi^T V  : V is MN-major
      bool ok = mbar_wait(bar(B_W), 0, wc);
      int tp = 0, ts = 0;                                        // next tile for Phi^T / for the accumulation
      long long t0 = 0;
      uint32_t polls = 0;
      while (ok && ts < nt) {
        bool did = false;
        if (ts < tp) {                                           // S(ts): packed features and the V tile
          const int it = ts * IPT + NX;
          if (mbar_try_wait(bar(B_PK + (ts & 1)), (ts >> 1) & 1) && mbar_try_wait(bar(B_FULL + it % SLOTS), (it / SLOTS) & 1)) {
            tc_fence_after();
            issue_tmemA_mnB(tAcc, tPA[ts & 1], mnmajor_desc(sSlot(it)), ID_ACC, ts > 0);
            tc_commit(bar(B_EMPTY + it % SLOTS));
            if (ts == nt - 1) tc_commit(bar(B_DONE));
            ++ts;
            did = true;
          }
        }
        if (tp < nt && tp - ts < 2) {                            // Phi^T(tp): its X items
          bool ready = true;
#pragma unroll
          for (int j = 0; j < NX; ++j) {
            const int it = tp * IPT + j;
            ready = ready && mbar_try_wait(bar(B_FULL + it % SLOTS), (it / SLOTS) & 1);
          }
          if (ready) {
            tc_fence_after();
#pragma unroll
            for (int j = 0; j < NX; ++j) {
              const int it = tp * IPT + j;
              issue_kmajor<D>(tD1[tp & 1], kmajor_desc(sW(j)), kmajor_desc(sSlot(it)), ID_PHI, j > 0);
              tc_commit(bar(B_EMPTY + it % SLOTS));
            }
            tc_commit(bar(B_D1 + (tp & 1)));
            ++tp;
            did = true;
          }
        }
        if (did) { polls = 0; t0 = 0; continue; }
        // nothing was ready: the same bound as every other wait (the clock is looked at every 64 idle rounds)
        if ((++polls & 63u) == 0u) {
          const long long now = clock64();
          if (t0 == 0) t0 = now;
          if (*wc.abort != 0u || now - t0 > kWaitLimitCycles) {
            *wc.abort = 1u;
            atomicOr(wc.status, 1u);
            ok = false;
          }
        }
      }
    }
    __syncwarp();
  } else if (warp >= 10) {
    // ------------------------------------------------------------ gather of softmax-token rows
    if (gathers) {
      const int gw = warp - 10;
      // rows handled by this warp: gw*64 .. gw*64+63; two ranks per lane.  The ranks of tile t + 1 are
      // fetched while tile t is being copied, so that the global-load latency stays off the critical path.
      auto load_ranks = [&](int t, int (&rk)[2]) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int n = (t_begin + t) * 128 + gw * 64 + e * 32 + lane;
          rk[e] = (t < nt && n < p.N) ? p.sm_rank[n] : -1;
        }
      };
      int rk_next[2];
      load_ranks(0, rk_next);
      for (int t = 0; t < nt; ++t) {
        int rk[2] = {rk_next[0], rk_next[1]};
        load_ranks(t + 1, rk_next);
        bool ok = true;
        for (int i = 0; i < IPT; ++i) {
          const int it = t * IPT + i;
          ok = ok && mbar_wait_warp(bar(B_FULL + it % SLOTS), (it / SLOTS) & 1, wc);
        }
        if (!ok) break;
        const uint8_t* kt = LAYERS == 1 ? smem + L::RING_OFF + ((t * IPT) % SLOTS) * L::TILE : nullptr;
        const uint8_t* vt = smem + L::RING_OFF + ((t * IPT + NX) % SLOTS) * L::TILE;
        constexpr int CH = D / 8;                          // 16-byte chunks per row
        for (int e = 0; e < 2; ++e) {
          uint32_t bits = __ballot_sync(0xffffffffu, rk[e] >= 0);
          while (bits) {
            const int src = __ffs(bits) - 1;
            bits &= bits - 1;
            const int rank = __shfl_sync(0xffffffffu, rk[e], src);
            const uint32_t rrow = gw * 64 + e * 32 + src;
            // lanes [0, CH) move the K row, lanes [16, 16 + CH) the V row
            const int c = lane & 15;
            if (c < CH) {
              uint4 val;
              if (lane < 16 && LAYERS == 2) {
                const size_t n = (size_t)(t_begin + t) * 128 + rrow;
                val = *reinterpret_cast<const uint4*>(p.k + ((size_t)bh * p.N + n) * D + c * 8);
              } else {
                const uint8_t* tile = (lane < 16) ? kt : vt;
                val = *reinterpret_cast<const uint4*>(tile + (c / 8) * BOX_BYTES + swz128_chunk_offset(rrow, c % 8));
              }
              __nv_bfloat16* dst = ((lane < 16) ? p.ks_w : p.vs_w) + ((size_t)bh * p.n_s + rank) * D + c * 8;
              *reinterpret_cast<uint4*>(dst) = val;
            }
          }
        }
        __syncwarp();
        if (lane == 0)
          for (int i = 0; i < IPT; ++i) mbar_arrive(bar(B_EMPTY + (t * IPT + i) % SLOTS));
      }
    }
    named_barrier_arrive(2, K_FEATURE_THREADS + 64);           // the feature warps may reuse the ring for the partial S
  } else {
    // ------------------------------------------------------------ feature warps: lane of TMEM = feature
    // warp w works on TMEM lanes 32 * (w % 4) .. + 31 and on token columns 64 * (w / 4) .. + 63
    const int quad = warp & 3, hf = warp >> 2, tid = threadIdx.x;
    const int f_local = quad * 32 + lane, f = fc * 128 + f_local;
    const uint32_t lane_off = (uint32_t)(quad * 32) << 16;
    const int part = p.F / p.P;
    const int pw = min(f / part, p.P - 1) + 1;                 // power of this feature's part (the same in a whole warp
                                                               // whenever the part width is a multiple of 32)
    const float bias = (p.bias != nullptr && f < p.F) ? __bfloat162float(p.bias[(size_t)h * p.F + f]) : 0.f;
    float z0 = 0.f, z1 = 0.f;
    bool ok = true;
    uint32_t x[32];
    // Which tokens of a tile are linear tokens (inside the sequence, not softmax tokens), as one word per
    // token pair that masks the packed bf16 features; the first 64 threads each prepare one pair, one tile ahead.
    auto pair_mask = [&](int t) -> uint32_t {
      if (tid >= 64 || t >= nt) return 0u;
      const int n0 = (t_begin + t) * 128 + 2 * tid;
      uint32_t m = 0u;
      if (n0 < p.N && p.sm_rank[n0] < 0) m |= 0x0000ffffu;
      if (n0 + 1 < p.N && p.sm_rank[n0 + 1] < 0) m |= 0xffff0000u;
      return m;
    };
    uint32_t m_next = pair_mask(0);
    for (int t = 0; t < nt; ++t) {
      const int b = t & 1;
      if (tid < 64) sPair[b * 64 + tid] = m_next;
      m_next = pair_mask(t + 1);
      // every feature thread reaches this barrier in every iteration, also after a failed wait: a warp
      // that left the loop early would leave the others waiting here for good
      named_barrier_sync(1, K_FEATURE_THREADS);
      if (ok) ok = mbar_wait_warp(bar(B_D1 + b), (t >> 1) & 1, wc);
      if (!ok) continue;
      tc_fence_after();
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        const int col = hf * 64 + c * 32;
        tmem_ld32(tD1[b] + lane_off + col, x);
        tmem_ld_wait(x);
        const uint4* mask4 = reinterpret_cast<const uint4*>(sPair + b * 64 + col / 2);
        uint32_t w[16];
        switch (pw) {
          case 1: k_features<1>(x, mask4, bias, w, z0, z1); break;
          case 2: k_features<2>(x, mask4, bias, w, z0, z1); break;
          case 3: k_features<3>(x, mask4, bias, w, z0, z1); break;
          default: k_features<4>(x, mask4, bias, w, z0, z1); break;
        }
        tmem_st16(tPA[b] + lane_off + col / 2, w);
      }
      tmem_st_wait();
      tc_fence_before();
      mbar_arrive(bar(B_PK + b));
    }
    if (ok) ok = mbar_wait_warp(bar(B_DONE), 0, wc);
    // z of the two column halves is added through shared memory.  The partial S leaves through the ring: each
    // thread puts its half row there (rows padded so that a warp's lanes hit different banks), then the row's
    // owner hands the row to the copy engine as one contiguous piece - a row written straight from registers
    // would cost one 32-byte sector per lane and instruction.  The ring is idle once the last product has
    // completed and the gather warps (barrier 2) have read their last tile.  Every feature thread takes part in
    // the barriers whatever its waits returned.
    if (hf == 1) sZ[f_local] = z0 + z1;
    named_barrier_sync(2, K_FEATURE_THREADS + 64);
    uint8_t* stage = smem + L::RING_OFF + f_local * L::OUT_PITCH;
    if (ok) {
      tc_fence_after();
      constexpr int HALF = D / 2;                              // accumulator columns per warp
#pragma unroll
      for (int c = 0; c < HALF / 32; ++c) {
        const int col = hf * HALF + c * 32;
        tmem_ld32(tAcc + lane_off + col, x);                   // warp-collective: also lanes beyond F take part
        tmem_ld_wait(x);
#pragma unroll
        for (int i = 0; i < 8; ++i)
          *reinterpret_cast<uint4*>(stage + (col + 4 * i) * 4) = make_uint4(x[4 * i], x[4 * i + 1], x[4 * i + 2], x[4 * i + 3]);
      }
      fence_proxy_async();
    }
    named_barrier_sync(1, K_FEATURE_THREADS);
    if (ok && hf == 0 && f < p.F) {
      const size_t slot = (size_t)bh * p.n_chunks + chunk;
      bulk_store_1d(p.part_s + (slot * p.F + f) * D, smem_u32(stage), D * 4);
      tma_store_commit();
      p.part_z[slot * p.F + f] = (z0 + z1) + sZ[f_local];
      tma_store_wait_all();                                    // the partial state is in global memory ...
      fence_proxy_async_all();                                 // ... and ordered before what this CTA publishes below
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 9) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
  // ---- The chunks' partial states are added up here, in chunk order (fixed order, no float atomics): every CTA of
  // a (batch, head, feature chunk) takes a slice of the [F x (D + 1)] entries once all of them have stored theirs.
  // The CTAs of one launch are resident together (one per SM, a cooperative launch when there is more than one
  // chunk), so the wait ends; it is bounded like every other wait.  The second counter tells the last CTA to finish
  // its slice that both counters can go back to zero for the next launch.
  __shared__ uint32_t s_go;
  uint32_t* cnt = p.counters + 2 * ((size_t)bh * gridDim.z + fc);
  const uint32_t n_ctas = gridDim.x;
  if (threadIdx.x == 0) {
    __threadfence();
    atomicAdd(cnt, 1u);
    uint32_t go = 1u, it = 0;
    long long t0 = 0;
    while (*reinterpret_cast<volatile uint32_t*>(cnt) < n_ctas) {
      __nanosleep(100);
      if ((++it & 63u) == 0u) {
        const long long now = clock64();
        if (t0 == 0) t0 = now;
        if (*abort_flag != 0u || now - t0 > kWaitLimitCycles) { atomicOr(p.status, 1u); go = 0u; break; }
      }
      // a CTA that found the status word set never arrives: the others stop waiting as soon as they see it too
      if (*reinterpret_cast<volatile uint32_t*>(p.status) != 0u) { go = 0u; break; }
    }
    s_go = go;
  }
  __syncthreads();
  if (s_go == 0u) return;
  __threadfence();
  {
    const int f0 = fc * 128, nf = min(128, p.F - f0);
    const size_t pitch = (size_t)p.F * D;                      // floats between two chunks' partials
    const float* src = p.part_s + ((size_t)bh * p.n_chunks * p.F + f0) * D;
    float* dS = p.S + ((size_t)bh * p.F + f0) * D;
    __nv_bfloat16* dSb = p.Sb + ((size_t)bh * p.F + f0) * D;
    const int n4 = nf * D / 4, per = (n4 + (int)n_ctas - 1) / (int)n_ctas;       // float4 entries, this CTA's slice
    const int i_end = min(n4, (chunk + 1) * per);
    for (int i = chunk * per + (int)threadIdx.x; i < i_end; i += K_THREADS) {
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      int c = 0;
      for (; c + 4 <= p.n_chunks; c += 4) {                    // four chunks' loads in flight, added in chunk order
        float4 v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = __ldcg(reinterpret_cast<const float4*>(src + (c + j) * pitch) + i);
#pragma unroll
        for (int j = 0; j < 4; ++j) { acc.x += v[j].x; acc.y += v[j].y; acc.z += v[j].z; acc.w += v[j].w; }
      }
      for (; c < p.n_chunks; ++c) {
        const float4 v = __ldcg(reinterpret_cast<const float4*>(src + c * pitch) + i);
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
      }
      reinterpret_cast<float4*>(dS)[i] = acc;
      reinterpret_cast<uint2*>(dSb)[i] = make_uint2(pack_bf16(acc.x, acc.y), pack_bf16(acc.z, acc.w));
    }
    if (chunk == 0) {
      for (int f = threadIdx.x; f < nf; f += K_THREADS) {
        float acc = 0.f;
        for (int c = 0; c < p.n_chunks; ++c) acc += __ldcg(p.part_z + ((size_t)bh * p.n_chunks + c) * p.F + f0 + f);
        p.z[(size_t)bh * p.F + f0 + f] = acc;
      }
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const uint32_t done = atomicAdd(cnt + 1, 1u);
    if (done + 1u == n_ctas) { cnt[0] = 0u; cnt[1] = 0u; }     // everyone has read the first counter: ready for the next launch
  }
}

// ======================================================================================
// First layer of a two-layer feature map for the keys ("Characterization of phi": the embedding
// network): h1 = relu(k W_1^T + b_1), [B*H, N, hidden] bf16.  One 128-token tile per CTA, all hidden slices.
// ======================================================================================
struct P1Params { int H, hid; const __nv_bfloat16* bias; uint32_t* status; };
constexpr int P1_THREADS = 160;          // warps 0-3: epilogue (one thread per token row); warp 4: TMA + MMA

template <int D, int NH>
struct P1Layout {
  static constexpr int TILE = 128 * D * 2;
  static constexpr int X_OFF = 0, W_OFF = TILE, BAR_OFF = (1 + NH) * TILE;
  static constexpr int BIAS_OFF = BAR_OFF + 64;                 // NH * D floats
  static constexpr int TOTAL = BIAS_OFF + NH * D * 4 + 1024;
};

template <int D, int NH>
__global__ void __launch_bounds__(P1_THREADS)
phi1_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW,
            const __grid_constant__ CUtensorMap tmH, const P1Params p) {
  using L = P1Layout<D, NH>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t sbase = smem_u32(smem);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::BAR_OFF);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::BAR_OFF + 16);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + L::BAR_OFF + 20);
  float* sBias = reinterpret_cast<float*>(smem + L::BIAS_OFF);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int bh = blockIdx.y, h = bh % p.H, row0 = blockIdx.x * 128;
  const WaitCtx wc{p.status, abort_flag};
  const uint32_t bar_full = smem_u32(bars), bar_done = smem_u32(bars + 1);
  constexpr int TM_COLS = NH * 128;                             // 128 or 256: a power of two

  __shared__ uint32_t s_skip;
  if (threadIdx.x == 0) s_skip = *reinterpret_cast<volatile uint32_t*>(p.status);
  __syncthreads();
  if (s_skip != 0u) return;
  if (threadIdx.x == 0) {
    *abort_flag = 0u;
    mbar_init(bar_full, 1); mbar_init(bar_done, 1);
    fence_barrier_init();
    fence_proxy_async();
  }
  for (int i = threadIdx.x; i < NH * D; i += P1_THREADS)
    sBias[i] = (p.bias != nullptr && i < p.hid) ? __bfloat162float(p.bias[(size_t)h * p.hid + i]) : 0.f;
  if (warp == 4) { tmem_alloc(smem_u32(tmem_slot), TM_COLS); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t sX = sbase + L::X_OFF;
  auto sW = [&](int j) { return sbase + L::W_OFF + j * L::TILE; };
  // hidden slice j is staged for its store where an operand sat: slice 0 over the X tile, slice j over W tile j - 1
  auto stage_off = [&](int j) { return j == 0 ? L::X_OFF : L::W_OFF + (j - 1) * L::TILE; };

  if (warp == 4) {
    if (lane == 0) {
      mbar_expect_tx(bar_full, (1 + NH) * L::TILE);
      load_tile<D>(sX, &tmX, bar_full, row0, bh);
      for (int j = 0; j < NH; ++j) load_tile<D>(sW(j), &tmW, bar_full, j * 128, h);   // W_1[h] rows of slice j (past hid: zeros)
    }
    __syncwarp();
    if (mbar_wait_warp(bar_full, 0, wc)) {
      tc_fence_after();
      if (lane == 0) {
        for (int j = 0; j < NH; ++j)      // X W_1^T, N = 128 hidden units of slice j (N = D when the hidden width is 64)
          issue_kmajor<D>(tmem + j * 128, kmajor_desc(sX), kmajor_desc(sW(j)), make_idesc(128, NH == 1 ? D : 128, 0, 0), false);
        tc_commit(bar_done);
      }
      __syncwarp();
    }
  } else {
    const int r = warp * 32 + lane;
    const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
    bool ok = mbar_wait_warp(bar_done, 0, wc);
    if (ok) {
      tc_fence_after();
      uint32_t x[32];
#pragma unroll
      for (int j = 0; j < NH; ++j) {
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          tmem_ld32(tmem + lane_off + j * 128 + c * 32, x);
          tmem_ld_wait(x);
          const float* bb = sBias + j * D + c * 32;
          uint32_t w[16];
#pragma unroll
          for (int i = 0; i < 16; ++i)
            w[i] = pack_bf16(fmaxf(__uint_as_float(x[2 * i]) + bb[2 * i], 0.f), fmaxf(__uint_as_float(x[2 * i + 1]) + bb[2 * i + 1], 0.f));
          store_row_chunk(smem + stage_off(j), r, c * 32, w);   // every MMA has completed: the operand tiles are free
        }
      }
      fence_proxy_async();
    }
    named_barrier_sync(1, 128);                               // reached by every epilogue thread, also after a failed wait
    if (ok && r == 0) {
      for (int j = 0; j < NH; ++j)
#pragma unroll
        for (int b = 0; b < D / 64; ++b) tma_store_3d(&tmH, sbase + stage_off(j) + b * BOX_BYTES, j * D + b * 64, row0, bh);
      tma_store_commit();
      tma_store_wait_all();
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 4) {
    tc_fence_after();
    tmem_dealloc(tmem, TM_COLS);
  }
}

template <int D, int LAYERS, int NH>
cudaError_t launch_kpass(const CUtensorMap& tmK, const CUtensorMap& tmV, const CUtensorMap& tmW, const CUtensorMap& tmH,
                         const KParams& p, dim3 grid, cudaStream_t st) {
  if (grid.x == 1) {                   // one chunk per head: no CTA waits for another
    kpass_kernel<D, LAYERS, NH><<<grid, K_THREADS, KLayout<D, LAYERS, NH>::TOTAL, st>>>(tmK, tmV, tmW, tmH, p);
    return cudaGetLastError();
  }
  // several chunks per head: the CTAs wait for one another at the end, so they must be resident together
  void* args[] = {(void*)&tmK, (void*)&tmV, (void*)&tmW, (void*)&tmH, (void*)&p};
  return cudaLaunchCooperativeKernel((const void*)kpass_kernel<D, LAYERS, NH>, grid, dim3(K_THREADS), args,
                                     (size_t)KLayout<D, LAYERS, NH>::TOTAL, st);
}

}  // namespace

cudaError_t as_tensor_init_kpass() {
  cudaError_t e;
  if ((e = opt_in_smem(kpass_kernel<128, 1, 1>, KLayout<128, 1, 1>::TOTAL)) != cudaSuccess) return e;
  if ((e = opt_in_smem(kpass_kernel<64, 1, 1>, KLayout<64, 1, 1>::TOTAL)) != cudaSuccess) return e;
  if ((e = opt_in_smem(kpass_kernel<128, 2, 1>, KLayout<128, 2, 1>::TOTAL)) != cudaSuccess) return e;
  if ((e = opt_in_smem(kpass_kernel<128, 2, 2>, KLayout<128, 2, 2>::TOTAL)) != cudaSuccess) return e;
  if ((e = opt_in_smem(kpass_kernel<64, 2, 1>, KLayout<64, 2, 1>::TOTAL)) != cudaSuccess) return e;
  if ((e = opt_in_smem(phi1_kernel<128, 1>, P1Layout<128, 1>::TOTAL)) != cudaSuccess) return e;
  if ((e = opt_in_smem(phi1_kernel<128, 2>, P1Layout<128, 2>::TOTAL)) != cudaSuccess) return e;
  if ((e = opt_in_smem(phi1_kernel<64, 1>, P1Layout<64, 1>::TOTAL)) != cudaSuccess) return e;
  return cudaSuccess;
}

// First layer of the key feature map: h1k = relu(k W_k1^T + b_k1).
cudaError_t as_tensor_phi1(const as_launch_args& a, cudaStream_t st) {
  const int BH = a.B * a.H;
  CUtensorMap tmX, tmW, tmH;
  if (!make_map(&tmX, a.k, a.d, a.N, BH, 128) || !make_map(&tmW, a.wk, a.d, a.hid, a.H, 128) ||
      !make_map(&tmH, a.h1k, a.hid, a.N, BH, 128))
    return cudaErrorInvalidValue;
  P1Params p{a.H, a.hid, a.bk1, a.status};
  dim3 grid((a.N + 127) / 128, BH, 1);
  if (a.d == 128 && a.hid == 256) phi1_kernel<128, 2><<<grid, P1_THREADS, P1Layout<128, 2>::TOTAL, st>>>(tmX, tmW, tmH, p);
  else if (a.d == 128) phi1_kernel<128, 1><<<grid, P1_THREADS, P1Layout<128, 1>::TOTAL, st>>>(tmX, tmW, tmH, p);
  else phi1_kernel<64, 1><<<grid, P1_THREADS, P1Layout<64, 1>::TOTAL, st>>>(tmX, tmW, tmH, p);
  return cudaGetLastError();
}

cudaError_t as_tensor_kpass(const as_launch_args& a, cudaStream_t st) {
  const int BH = a.B * a.H;
  const bool two = a.layers == 2;
  CUtensorMap tmK, tmV, tmW, tmH;
  if (!make_map(&tmK, a.k, a.d, a.N, BH, 128) || !make_map(&tmV, a.v, a.d, a.N, BH, 128)) return cudaErrorInvalidValue;
  // last-layer weights [H][F][width of their input]
  if (!make_map(&tmW, two ? a.wk2 : a.wk, two ? a.hid : a.d, a.F, a.H, 128)) return cudaErrorInvalidValue;
  if (two) { if (!make_map(&tmH, a.h1k, a.hid, a.N, BH, 128)) return cudaErrorInvalidValue; }
  else tmH = tmK;               // never used with a one-layer map
  KParams p{};
  p.N = a.N; p.n_s = a.n_s; p.n_chunks = a.n_chunks; p.chunk_tiles = a.chunk_tiles; p.P = a.P; p.F = a.F;
  p.H = a.H; p.sm_rank = a.sm_rank; p.ks_w = a.ks_w; p.vs_w = a.vs_w; p.k = a.k;
  p.bias = two ? a.bk2 : a.bk1;
  p.part_s = a.part_s; p.part_z = a.part_z; p.status = a.status;
  p.S = a.S; p.z = a.z; p.Sb = a.Sb; p.counters = a.counters;
  dim3 grid(a.n_chunks, BH, (a.F + 127) / 128);
  if (a.d == 128) {
    if (!two) return launch_kpass<128, 1, 1>(tmK, tmV, tmW, tmH, p, grid, st);
    if (a.hid == 256) return launch_kpass<128, 2, 2>(tmK, tmV, tmW, tmH, p, grid, st);
    return launch_kpass<128, 2, 1>(tmK, tmV, tmW, tmH, p, grid, st);
  }
  if (!two) return launch_kpass<64, 1, 1>(tmK, tmV, tmW, tmH, p, grid, st);
  return launch_kpass<64, 2, 1>(tmK, tmV, tmW, tmH, p, grid, st);
}
