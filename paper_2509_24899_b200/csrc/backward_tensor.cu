// Gradient of the value-distillation loss w.r.t. the feature-map weights ("Attention Distillation"; Algorithm 1
// updates the feature maps only) on the tensor cores, for one-layer maps with d = F = 128 and no bias.  The chain rule
// (formulas in backward_simt.cu) is a handful of products per 128-token tile:
//
//   query side   A  = Q W_q^T                  pre-activations                   [tokens x F]
//                U  = g S^T                     g = sign(y_hat - y) / den         [tokens x F]
//                dS  += (lambda phi_q)^T g      state gradient                    [F x d]
//                dW_q += (dL/da_q)^T Q          dL/da_q = lambda (U + z s) phi'    [F x d]
//   key side     A  = K W_k^T,  T = V dS^T,     dW_k += (dL/da_k)^T K             dL/da_k = (T + dz) phi' on linear tokens
//
// bf16 operands, fp32 accumulation in TMEM.  dz = sum_i lambda phi_q,i s_i is summed, in token order, from the very
// bf16 values the dS product multiplies (through shared memory).  One CTA per (token chunk, batch*head): sixteen
// compute warps - a token row (= TMEM lane) is shared by four threads, each taking 32 of its 128 columns - and lane
// 0 of warp 16, which loads the tiles and issues the products, one tile at a time.  The chunks' partial results leave
// in the layout of the CUDA-core version and are added up by its fixed-order reduction kernels.  Every wait is
// bounded (status word, abort flag).
#include "backward_common.h"
#include "tensor_common.cuh"

namespace {

using namespace as_tc;

constexpr int BT_COMPUTE = 512;          // warps 0-15: row = thread % 128, column quarter = thread / 128
constexpr int BT_THREADS = BT_COMPUTE + 32;   // warp 16: TMA + MMA issue (lane 0)
constexpr int TILE = 128 * 128 * 2;      // bytes of a [128 x 128] bf16 tile
constexpr uint32_t ID_KK = make_idesc(128, 128, 0, 0);      // both operands K-major
constexpr uint32_t ID_MM = make_idesc(128, 128, 1, 1);      // both operands MN-major (token rows are the K index)

// barriers (per-tile ones are used once per tile: phase = tile index)
constexpr int B_FULL1 = 3;                  // key side: the second K/V set's "full" barrier (the slot of B_GRDY)
constexpr int B_WFULL = 0, B_FULL = 1, B_ARDY = 2, B_GRDY = 3, B_URDY = 4, B_PRDY = 5, B_DONE = 6, B_DZ = 7, B_COUNT = 8;

struct BtLayout {
  static constexpr int W_OFF = 0;                 // weights [F][d]
  static constexpr int S_OFF = TILE;              // S (query side) / dS (key side) in bf16 [F][d]
  static constexpr int X_OFF = 2 * TILE;          // Q / K tile
  static constexpr int Y_OFF = 3 * TILE;          // query side: y, then g in place.  key side: V, then dL/da_k in place
  static constexpr int H_OFF = 4 * TILE;          // query side: y_hat, then lambda phi_q in place
  static constexpr int A_OFF = 5 * TILE;          // query side: dL/da_q
  static constexpr int BAR_OFF = 6 * TILE;
  static constexpr int SVEC_OFF = BAR_OFF + 128;  // 2 x 4 x 128 floats: the column quarters' shares of G . y_hat, per tile parity
  static constexpr int ZVEC_OFF = SVEC_OFF + 4096;   // 128 floats: z (query side) / dz (key side)
  static constexpr int SROW_OFF = ZVEC_OFF + 512; // 2 x 128 floats: s of the tile's rows, per tile parity
  static constexpr int RED_OFF = SROW_OFF + 1024; // 512 floats: the token quarters' shares of dz at the end, then the warps' loss sums
  static constexpr int TOTAL = RED_OFF + 2048 + 1024;   // + slack for the 1024-byte alignment
};

// phi = r^p and its slope p r^(p-1) for r = relu(a); the power is a compile-time constant (a thread's 32 features
// belong to one part of the feature map)
template <int PW>
AS_DEV void bt_poly(float a, float& phi, float& slope) {
  const float r = fmaxf(a, 0.f);
  float rp1 = 1.f;                                // r^(p-1)
#pragma unroll
  for (int i = 1; i < PW; ++i) rp1 *= r;
  phi = rp1 * r;
  slope = a > 0.f ? (float)PW * rp1 : 0.f;
}
// Query side, 32 features of one row: lambda phi_q and dL/da_q = lambda (U + z s) phi' as bf16 pairs.
template <int PW>
AS_DEV void bt_q_features(const uint32_t (&xa)[32], const uint32_t (&xu)[32], const float* zv, float s_i, float lam,
                          uint32_t (&wp)[16], uint32_t (&wa)[16]) {
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    float ph0, sl0, ph1, sl1;
    bt_poly<PW>(__uint_as_float(xa[2 * i]), ph0, sl0);
    bt_poly<PW>(__uint_as_float(xa[2 * i + 1]), ph1, sl1);
    const float u0 = fmaf(zv[2 * i], s_i, __uint_as_float(xu[2 * i])), u1 = fmaf(zv[2 * i + 1], s_i, __uint_as_float(xu[2 * i + 1]));
    wp[i] = pack_bf16(lam * ph0, lam * ph1);
    wa[i] = pack_bf16(lam * u0 * sl0, lam * u1 * sl1);
  }
}
// Key side, 32 features of one row: dL/da_k = (T + dz) phi' on linear tokens, zero on softmax tokens.
template <int PW>
AS_DEV void bt_k_features(const uint32_t (&xa)[32], const uint32_t (&xt)[32], const float* zv, bool lin, uint32_t (&wa)[16]) {
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    float ph0, sl0, ph1, sl1;
    bt_poly<PW>(__uint_as_float(xa[2 * i]), ph0, sl0);
    bt_poly<PW>(__uint_as_float(xa[2 * i + 1]), ph1, sl1);
    const float t0 = (__uint_as_float(xt[2 * i]) + zv[2 * i]) * sl0, t1 = (__uint_as_float(xt[2 * i + 1]) + zv[2 * i + 1]) * sl1;
    wa[i] = lin ? pack_bf16(t0, t1) : 0u;
  }
}
AS_DEV float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
AS_DEV float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Writes 32 columns of one accumulator row (TMEM lane = feature row) to dst.
AS_DEV void bt_store_acc(uint32_t tacc, float* dst) {
  uint32_t x[32];
  tmem_ld32(tacc, x);
  tmem_ld_wait(x);
#pragma unroll
  for (int i = 0; i < 8; ++i) reinterpret_cast<uint4*>(dst)[i] = make_uint4(x[4 * i], x[4 * i + 1], x[4 * i + 2], x[4 * i + 3]);
}

// ---------------------------------------------------------------------------------------------- query side
__global__ void __launch_bounds__(BT_THREADS, 1)
btq_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmY, const __grid_constant__ CUtensorMap tmH,
           const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmS, const __grid_constant__ BwParams p) {
  using L = BtLayout;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t sbase = smem_u32(smem);
  auto bar = [&](int i) { return sbase + L::BAR_OFF + 8 * i; };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::BAR_OFF + 8 * B_COUNT);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + L::BAR_OFF + 8 * B_COUNT + 4);
  float* svec = reinterpret_cast<float*>(smem + L::SVEC_OFF);
  float* zvec = reinterpret_cast<float*>(smem + L::ZVEC_OFF);
  float* red = reinterpret_cast<float*>(smem + L::RED_OFF);
  float* srow = reinterpret_cast<float*>(smem + L::SROW_OFF);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int bh = blockIdx.y, chunk = blockIdx.x, h = bh % p.H;
  const int tok_begin = chunk * p.chunk_tokens;
  const int tok_end = min(p.N, tok_begin + p.chunk_tokens);
  const int nt = (tok_end - tok_begin + 127) / 128;

  __shared__ uint32_t s_skip;
  if (threadIdx.x == 0) s_skip = *reinterpret_cast<volatile uint32_t*>(p.status);
  __syncthreads();
  if (s_skip != 0u) return;
  if (threadIdx.x == 0) {
    *abort_flag = 0u;
    mbar_init(bar(B_WFULL), 1); mbar_init(bar(B_FULL), 1); mbar_init(bar(B_ARDY), 1); mbar_init(bar(B_GRDY), BT_COMPUTE);
    mbar_init(bar(B_URDY), 1); mbar_init(bar(B_PRDY), BT_COMPUTE); mbar_init(bar(B_DONE), 1); mbar_init(bar(B_DZ), BT_COMPUTE);
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 16) { tmem_alloc(smem_u32(tmem_slot), 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tA = tmem, tU = tmem + 128, tdS = tmem + 256, tdW = tmem + 384;
  const WaitCtx wc{p.status, abort_flag};

  if (warp == 16) {
    if (lane == 0) {
      tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmY); tma_prefetch_desc(&tmH);
      mbar_expect_tx(bar(B_WFULL), 2 * TILE);
      load_tile<128>(sbase + L::W_OFF, &tmW, bar(B_WFULL), 0, h);
      load_tile<128>(sbase + L::S_OFF, &tmS, bar(B_WFULL), 0, bh);
      bool ok = true;
      for (int t = 0; t < nt && ok; ++t) {
        // the previous tile's products and its dz pass have read the tiles
        if (t > 0) ok = mbar_wait(bar(B_DONE), (t - 1) & 1, wc) && mbar_wait(bar(B_DZ), (t - 1) & 1, wc);
        if (!ok) break;
        const int row0 = tok_begin + t * 128;
        mbar_expect_tx(bar(B_FULL), 3 * TILE);
        load_tile<128>(sbase + L::X_OFF, &tmQ, bar(B_FULL), row0, bh);
        load_tile<128>(sbase + L::Y_OFF, &tmY, bar(B_FULL), row0, bh);
        load_tile<128>(sbase + L::H_OFF, &tmH, bar(B_FULL), row0, bh);
        if (t == 0 && !mbar_wait(bar(B_WFULL), 0, wc)) break;
        if (!mbar_wait(bar(B_FULL), t & 1, wc)) break;
        tc_fence_after();
        issue_kmajor<128>(tA, kmajor_desc(sbase + L::X_OFF), kmajor_desc(sbase + L::W_OFF), ID_KK, false);
        tc_commit(bar(B_ARDY));
        if (!mbar_wait(bar(B_GRDY), t & 1, wc)) break;
        tc_fence_after();
        issue_kmajor<128>(tU, kmajor_desc(sbase + L::Y_OFF), kmajor_desc(sbase + L::S_OFF), ID_KK, false);
        tc_commit(bar(B_URDY));
        if (!mbar_wait(bar(B_PRDY), t & 1, wc)) break;
        tc_fence_after();
        const uint64_t aP = mnmajor_desc(sbase + L::H_OFF), bG = mnmajor_desc(sbase + L::Y_OFF);
        const uint64_t aD = mnmajor_desc(sbase + L::A_OFF), bQ = mnmajor_desc(sbase + L::X_OFF);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) mma_ss(tdS, aP + kstep_mnmajor(kk), bG + kstep_mnmajor(kk), ID_MM, (t > 0 || kk > 0) ? 1u : 0u);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) mma_ss(tdW, aD + kstep_mnmajor(kk), bQ + kstep_mnmajor(kk), ID_MM, (t > 0 || kk > 0) ? 1u : 0u);
        tc_commit(bar(B_DONE));
      }
    }
    __syncwarp();
  } else {
    const int r = threadIdx.x & 127, qt = threadIdx.x >> 7;    // token row of the tile (= TMEM lane) and column quarter
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const int part = 128 / p.P;
    if (qt == 0) zvec[r] = p.z[(size_t)bh * 128 + r];
    named_barrier_sync(1, BT_COMPUTE);
    float dz_acc = 0.f, loss = 0.f;
    bool ok = true;
    uint8_t* sY = smem + L::Y_OFF;
    uint8_t* sH = smem + L::H_OFF;
    uint8_t* sA = smem + L::A_OFF;
    // the row's statistics of the forward pass (c_i, the two parts of the denominator), fetched one tile ahead
    auto row_stats = [&](int t, float (&a)[3]) {
      const int n = tok_begin + t * 128 + r;
      if (t < nt && n < tok_end) {
        const float* ap = p.aux + ((size_t)bh * p.N + n) * 3;
        a[0] = ap[0]; a[1] = ap[1]; a[2] = ap[2];
      } else {
        a[0] = 0.f; a[1] = 1.f; a[2] = 0.f;
      }
    };
    float st_next[3];
    row_stats(0, st_next);
    for (int t = 0; t < nt; ++t) {
      const float st_c[3] = {st_next[0], st_next[1], st_next[2]};
      row_stats(t + 1, st_next);
      if (ok) ok = mbar_wait_warp(bar(B_FULL), t & 1, wc);
      const int n = tok_begin + t * 128 + r;
      const bool in = ok && n < tok_end;
      float lam = 0.f, den = 1.f;
      if (in) {
        lam = (p.stab_mode == AS_STAB_EXACT && p.n_s > 0) ? __expf(-st_c[0]) : 1.f;
        den = st_c[1] + lam * st_c[2];
      }
      const float inv_den = 1.f / den;
      float* sv = svec + (t & 1) * 512;
      {
        // g = sign(y_hat - y) / den over this thread's 32 columns of the row, written over y; its share of G . y_hat
        // and of the loss on the way
        float sdot = 0.f;
        if (ok) {
#pragma unroll
          for (int c4 = 0; c4 < 4; ++c4) {
            const int c = qt * 4 + c4;
            const uint32_t off = (c >> 3) * BOX_BYTES + swz128_chunk_offset(r, c & 7);
            const uint4 yv = *reinterpret_cast<const uint4*>(sY + off);
            const uint4 hv = *reinterpret_cast<const uint4*>(sH + off);
            const uint32_t yw[4] = {yv.x, yv.y, yv.z, yv.w}, hw[4] = {hv.x, hv.y, hv.z, hv.w};
            uint32_t gw[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float h0 = bf_lo(hw[i]), h1 = bf_hi(hw[i]);
              const float d0 = h0 - bf_lo(yw[i]), d1 = h1 - bf_hi(yw[i]);
              // (rows past the end of the sequence arrive as zeros: no difference, no sign, nothing added)
              const float G0 = d0 == 0.f ? 0.f : copysignf(1.f, d0), G1 = d1 == 0.f ? 0.f : copysignf(1.f, d1);
              loss += fabsf(d0) + fabsf(d1);
              sdot = fmaf(G0, h0, fmaf(G1, h1, sdot));
              gw[i] = pack_bf16(G0 * inv_den, G1 * inv_den);
            }
            *reinterpret_cast<uint4*>(sY + off) = make_uint4(gw[0], gw[1], gw[2], gw[3]);
          }
        }
        sv[qt * 128 + r] = sdot;
      }
      fence_proxy_async();
      mbar_arrive(bar(B_GRDY));
      if (ok) ok = mbar_wait_warp(bar(B_ARDY), t & 1, wc);
      if (ok) ok = mbar_wait_warp(bar(B_URDY), t & 1, wc);
      // (U is complete only after every thread has arrived on the g barrier: the quarters' shares are all there)
      const float s_i = in ? -((sv[r] + sv[128 + r]) + (sv[256 + r] + sv[384 + r])) * inv_den : 0.f;
      if (qt == 0) srow[(t & 1) * 128 + r] = s_i;    // for the dz pass below (read after the barrier of all compute threads)
      if (ok) {
        tc_fence_after();
        uint32_t xa[32], xu[32];
        const int cc = qt;                           // this thread's 32 features
        tmem_ld32(tA + lane_off + cc * 32, xa);
        tmem_ld32(tU + lane_off + cc * 32, xu);
        tmem_ld_wait(xa);
        tmem_ld_wait(xu);
        const int pw = min((cc * 32) / part, p.P - 1) + 1;            // power of these 32 features
        uint32_t wp[16], wa[16];
        switch (pw) {
          case 1: bt_q_features<1>(xa, xu, zvec + cc * 32, s_i, lam, wp, wa); break;
          case 2: bt_q_features<2>(xa, xu, zvec + cc * 32, s_i, lam, wp, wa); break;
          case 3: bt_q_features<3>(xa, xu, zvec + cc * 32, s_i, lam, wp, wa); break;
          default: bt_q_features<4>(xa, xu, zvec + cc * 32, s_i, lam, wp, wa); break;
        }
        store_row_chunk(sH, r, cc * 32, wp);         // lambda phi_q over y_hat (consumed: every thread is past the g barrier)
        store_row_chunk(sA, r, cc * 32, wa);
        tc_fence_before();
      }
      fence_proxy_async();
      mbar_arrive(bar(B_PRDY));
      // dz[f] += sum over the tile's tokens of (lambda phi)[token][f] * s[token]: feature f = r, tokens of quarter qt
      named_barrier_sync(1, BT_COMPUTE);             // every row of lambda phi of the tile is in shared memory
      if (ok) {
        const uint32_t col = (uint32_t)(r >> 6) * BOX_BYTES + (uint32_t)(r & 7) * 2, chunk8 = (uint32_t)((r & 63) >> 3);
        const float* st = srow + (t & 1) * 128;
#pragma unroll 8
        for (int k = 0; k < 32; ++k) {
          const int tok = qt * 32 + k;
          const uint16_t hbits = *reinterpret_cast<const uint16_t*>(sH + col + swz128_chunk_offset(tok, chunk8));
          dz_acc = fmaf(__uint_as_float((uint32_t)hbits << 16), st[tok], dz_acc);
        }
      }
      mbar_arrive(bar(B_DZ));
    }
    // ---- the chunk's partial results
    if (ok && nt > 0) ok = mbar_wait_warp(bar(B_DONE), (nt - 1) & 1, wc);
    const size_t slot = (size_t)bh * p.chunks + chunk;
    if (ok && nt > 0) {
      tc_fence_after();
      bt_store_acc(tdS + lane_off + qt * 32, p.part_dS + (slot * 128 + r) * 128 + qt * 32);
      bt_store_acc(tdW + lane_off + qt * 32, p.part_dW + (slot * 128 + r) * 128 + qt * 32);
      tc_fence_before();
    }
    // dz of the chunk: the four token quarters' shares in quarter order; the loss: the sixteen warps' sums in warp order
    red[qt * 128 + r] = dz_acc;
    named_barrier_sync(1, BT_COMPUTE);
    if (qt == 0) p.part_dz[slot * 128 + r] = (red[r] + red[128 + r]) + (red[256 + r] + red[384 + r]);
    named_barrier_sync(1, BT_COMPUTE);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) loss += __shfl_xor_sync(0xffffffffu, loss, off);
    if (lane == 0) red[warp] = loss;
    named_barrier_sync(1, BT_COMPUTE);
    if (threadIdx.x == 0) {
      float l = 0.f;
      for (int w = 0; w < 16; ++w) l += red[w];
      p.part_loss[slot] = l;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 16) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// ---------------------------------------------------------------------------------------------- key side
__global__ void __launch_bounds__(BT_THREADS, 1)
btk_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmW,
           const __grid_constant__ CUtensorMap tmS, const __grid_constant__ BwParams p) {
  using L = BtLayout;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t sbase = smem_u32(smem);
  auto bar = [&](int i) { return sbase + L::BAR_OFF + 8 * i; };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::BAR_OFF + 8 * B_COUNT);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + L::BAR_OFF + 8 * B_COUNT + 4);
  float* zvec = reinterpret_cast<float*>(smem + L::ZVEC_OFF);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int bh = blockIdx.y, chunk = blockIdx.x, h = bh % p.H;
  const int tok_begin = chunk * p.chunk_tokens;
  const int tok_end = min(p.N, tok_begin + p.chunk_tokens);
  const int nt = (tok_end - tok_begin + 127) / 128;

  __shared__ uint32_t s_skip;
  if (threadIdx.x == 0) s_skip = *reinterpret_cast<volatile uint32_t*>(p.status);
  __syncthreads();
  if (s_skip != 0u) return;
  if (threadIdx.x == 0) {
    *abort_flag = 0u;
    mbar_init(bar(B_WFULL), 1); mbar_init(bar(B_FULL), 1); mbar_init(bar(B_FULL1), 1); mbar_init(bar(B_ARDY), 1);
    mbar_init(bar(B_PRDY), BT_COMPUTE); mbar_init(bar(B_DONE), 1);
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 16) { tmem_alloc(smem_u32(tmem_slot), 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tA = tmem, tT = tmem + 128, tdW = tmem + 256;
  const WaitCtx wc{p.status, abort_flag};

  if (warp == 16) {
    if (lane == 0) {
      tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
      mbar_expect_tx(bar(B_WFULL), 2 * TILE);
      load_tile<128>(sbase + L::W_OFF, &tmW, bar(B_WFULL), 0, h);
      load_tile<128>(sbase + L::S_OFF, &tmS, bar(B_WFULL), 0, bh);
      // K and V tiles are double-buffered: tile t lives in set t & 1 (its own "full" barrier), and the tile after the
      // next is requested as soon as the last product that reads the set has completed
      auto sK = [&](int t) { return sbase + ((t & 1) ? L::H_OFF : L::X_OFF); };
      auto sVt = [&](int t) { return sbase + ((t & 1) ? L::A_OFF : L::Y_OFF); };
      auto full = [&](int t) { return bar((t & 1) ? B_FULL1 : B_FULL); };
      auto request = [&](int t) {
        mbar_expect_tx(full(t), 2 * TILE);
        load_tile<128>(sK(t), &tmK, full(t), tok_begin + t * 128, bh);
        load_tile<128>(sVt(t), &tmV, full(t), tok_begin + t * 128, bh);
      };
      auto first_products = [&](int t) {           // A = K W_k^T and T = V dS^T of tile t
        tc_fence_after();
        issue_kmajor<128>(tA, kmajor_desc(sK(t)), kmajor_desc(sbase + L::W_OFF), ID_KK, false);
        issue_kmajor<128>(tT, kmajor_desc(sVt(t)), kmajor_desc(sbase + L::S_OFF), ID_KK, false);
        tc_commit(bar(B_ARDY));
      };
      bool ok = nt > 0;
      if (ok) {
        request(0);
        if (nt > 1) request(1);
        ok = mbar_wait(bar(B_WFULL), 0, wc) && mbar_wait(full(0), 0, wc);
        if (ok) first_products(0);
      }
      for (int t = 0; t < nt && ok; ++t) {
        if (!mbar_wait(bar(B_PRDY), t & 1, wc)) break;                   // dL/da_k of tile t is in shared memory (over V)
        tc_fence_after();
        const uint64_t aD = mnmajor_desc(sVt(t)), bK = mnmajor_desc(sK(t));
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) mma_ss(tdW, aD + kstep_mnmajor(kk), bK + kstep_mnmajor(kk), ID_MM, (t > 0 || kk > 0) ? 1u : 0u);
        tc_commit(bar(B_DONE));
        // the threads have read A and T of tile t (they arrived on the barrier above): the next tile's may land
        if (t + 1 < nt) {
          if (!mbar_wait(full(t + 1), ((t + 1) >> 1) & 1, wc)) break;
          first_products(t + 1);
        }
        if (t + 2 < nt) {
          if (!mbar_wait(bar(B_DONE), t & 1, wc)) break;                 // the set of tile t is free
          request(t + 2);
        }
      }
    }
    __syncwarp();
  } else {
    const int r = threadIdx.x & 127, qt = threadIdx.x >> 7;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const int part = 128 / p.P;
    if (qt == 0) zvec[r] = p.dz[(size_t)bh * 128 + r];
    named_barrier_sync(1, BT_COMPUTE);
    bool ok = true;
    auto is_linear = [&](int t) { const int n = tok_begin + t * 128 + r; return t < nt && n < tok_end && p.sm_rank[n] < 0; };
    bool lin_next = is_linear(0);                    // fetched one tile ahead
    for (int t = 0; t < nt; ++t) {
      uint8_t* sV = smem + ((t & 1) ? L::A_OFF : L::Y_OFF);      // the V tile of the set tile t lives in
      const bool lin_c = lin_next;
      lin_next = is_linear(t + 1);
      if (ok) ok = mbar_wait_warp(bar(B_ARDY), t & 1, wc);
      const bool lin = ok && lin_c;
      if (ok) {
        tc_fence_after();
        uint32_t xa[32], xt[32];
        const int cc = qt;                           // this thread's 32 features
        tmem_ld32(tA + lane_off + cc * 32, xa);
        tmem_ld32(tT + lane_off + cc * 32, xt);
        tmem_ld_wait(xa);
        tmem_ld_wait(xt);
        const int pw = min((cc * 32) / part, p.P - 1) + 1;
        uint32_t wa[16];
        switch (pw) {
          case 1: bt_k_features<1>(xa, xt, zvec + cc * 32, lin, wa); break;
          case 2: bt_k_features<2>(xa, xt, zvec + cc * 32, lin, wa); break;
          case 3: bt_k_features<3>(xa, xt, zvec + cc * 32, lin, wa); break;
          default: bt_k_features<4>(xa, xt, zvec + cc * 32, lin, wa); break;
        }
        store_row_chunk(sV, r, cc * 32, wa);         // dL/da_k over v (the product that read v has completed)
        tc_fence_before();
      }
      fence_proxy_async();
      mbar_arrive(bar(B_PRDY));
    }
    if (ok && nt > 0) ok = mbar_wait_warp(bar(B_DONE), (nt - 1) & 1, wc);
    if (ok && nt > 0) {
      tc_fence_after();
      const size_t slot = (size_t)bh * p.chunks + chunk;
      bt_store_acc(tdW + lane_off + qt * 32, p.part_dW + (slot * 128 + r) * 128 + qt * 32);
      tc_fence_before();
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 16) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

}  // namespace

cudaError_t as_bw_tensor_init() {
  cudaError_t e;
  if ((e = opt_in_smem(btq_kernel, BtLayout::TOTAL)) != cudaSuccess) return e;
  return opt_in_smem(btk_kernel, BtLayout::TOTAL);
}

cudaError_t as_bw_tensor_query(const BwParams& p, cudaStream_t st) {
  const int BH = p.B * p.H;
  CUtensorMap tmQ, tmY, tmH, tmW, tmS;
  if (!make_map(&tmQ, p.q, 128, p.N, BH, 128) || !make_map(&tmY, p.y, 128, p.N, BH, 128) ||
      !make_map(&tmH, p.yhat, 128, p.N, BH, 128) || !make_map(&tmW, p.wq, 128, 128, p.H, 128) ||
      !make_map(&tmS, p.Sb, 128, 128, BH, 128))
    return cudaErrorInvalidValue;
  btq_kernel<<<dim3(p.chunks, BH), BT_THREADS, BtLayout::TOTAL, st>>>(tmQ, tmY, tmH, tmW, tmS, p);
  return cudaGetLastError();
}

cudaError_t as_bw_tensor_key(const BwParams& p, cudaStream_t st) {
  const int BH = p.B * p.H;
  CUtensorMap tmK, tmV, tmW, tmS;
  if (!make_map(&tmK, p.k, 128, p.N, BH, 128) || !make_map(&tmV, p.v, 128, p.N, BH, 128) ||
      !make_map(&tmW, p.wk, 128, 128, p.H, 128) || !make_map(&tmS, p.dSb, 128, 128, BH, 128))
    return cudaErrorInvalidValue;
  btk_kernel<<<dim3(p.chunks, BH), BT_THREADS, BtLayout::TOTAL, st>>>(tmK, tmV, tmW, tmS, p);
  return cudaGetLastError();
}
