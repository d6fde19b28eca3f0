// Q pass of the hybrid attention forward on the tensor cores of sm_100a: softmax branch, phi_q
// projection, linear apply and merge, fused in one persistent kernel.
//
//   persistent, one CTA per SM (units left over after the full rounds are split into 128-row halves
//   over twice as many CTAs); per unit of 2 x 128 query rows a flash-style loop over 128-key tiles
//   of K_S / V_S:        S = Q K_S^T -> TMEM; the softmax threads (one per row) read their row and
//                        release the score columns at once, so the next tile's Q K_S^T runs under the
//                        exponentials; running max / sum per row; P = exp2(.) as bf16 -> shared memory,
//                        O += P V_S (smem x smem -> TMEM).  Two issuing threads: one for what writes
//                        the score columns, one for what accumulates into O.
//   tail:                Phi = Q W_q^T -> TMEM (in the place of a next tile's scores), phi_q scaled per
//                        row as bf16 where P sat, O += phi_q S (S in bf16 read like a V tile),
//                        den = l + phi_q.z, y = O / den -> bf16 -> staged in the P tile -> TMA store.
// All tiles are staged by TMA with the 128-byte swizzle; every mbarrier wait is bounded.
#include "tensor_common.cuh"

namespace {

using namespace as_tc;

// ======================================================================================
// Q pass
// ======================================================================================
struct QParams {
  int N, n_s, nkv, lin, stab_mode, P, H;
  int layers;                // depth of the feature map: with 2, tmH holds relu(q W_1^T) and tmW is W_2
  int nx, n_units;           // 256-row units per (batch, head); units over all (batch, head) pairs
  int n_rounds;              // rounds in which every CTA has a unit (n_units / gridDim.x)
  int split_last;            // 1: the units left over after those rounds are cut in two 128-row halves, one per CTA
  float scale_log2;          // softmax scale * log2(e)
  const float* z;            // [B*H][F]
  float* aux;                // [B*H][N][3] or nullptr
  uint32_t* status;
};

constexpr int Q_THREADS = 352;           // warps 0-3 / 4-7: softmax groups 0 / 1; warp 8: TMA; warps 9, 10: MMA issuers
constexpr int KV_STAGES = 3;
constexpr float RESCALE_THRESHOLD = 8.f; // log2 units: rescale O only when the row max grew by > 2^8

template <int D>
struct QLayout {
  static constexpr int TILE = 128 * D * 2;                 // bytes of a [128 x D] bf16 tile
  static constexpr int PTILE = 128 * 128 * 2;              // bytes of a [128 rows x 128 keys] bf16 P tile
  static constexpr int Q_OFF = 0;
  static constexpr int P_OFF = 2 * TILE;                   // per group: P, then phi_q, then the output rows
  static constexpr int KV_OFF = P_OFF + 2 * PTILE;
  static constexpr int BAR_OFF = KV_OFF + KV_STAGES * TILE;
  static constexpr int TOTAL = BAR_OFF + 256 + 1024;       // + slack for the 1024-byte alignment
};

// Persistent: one CTA per SM walks over 256-row units (unit w = blockIdx.x + u * gridDim.x; the units of
// one (batch, head) are consecutive, so the CTAs that run at the same time share K_S / V_S in L2).
// Barrier phases and the K/V ring run on across units.
//
// Scores and probabilities live in different memories: S = Q K^T lands in TMEM, the softmax threads read
// their rows into registers and release the S columns at once, so the next tile's Q K^T is computed while
// the exponentials run; P goes to shared memory as bf16 and is the A operand of O += P V.  A group's
// softmax therefore never waits for the tensor pipe in the steady state, and the pipe sees, per key tile
// and group, one Q K^T block as soon as S is free and one P V block as soon as P is there.
//
// The work of one unit is a function per role, kept out of line: each role then gets a register
// allocation of its own (the softmax rows need nearly the whole budget, and the issuing thread must
// not spill).  Everything about a unit is derived from its index u inside the function.
struct QCtx {
  uint32_t sbase;            // shared-memory window address of the 1024-aligned base
  uint32_t tmem;             // TMEM base address
  WaitCtx wc;
};

// Unit u of this CTA: which 256-row unit, which row it starts at, and how many of the two 128-row groups
// work on it.  In the rounds every CTA takes part in, CTA c has unit c + u * gridDim.x.  What is left
// over afterwards would keep less than half of the SMs busy for a whole unit's time; a single group, which
// has the tensor and XU pipes to itself, needs little more than half of that, so the left-over units are
// cut into their two 128-row halves and spread over twice as many CTAs.
struct QUnit { int w, row0, ng; };
AS_DEV QUnit q_unit(const QParams& p, int u) {
  const int c = (int)blockIdx.x, n = (int)gridDim.x;
  if (u < p.n_rounds) { const int w = c + u * n; return QUnit{w, (w % p.nx) * 256, 2}; }
  if (p.split_last) { const int w = p.n_rounds * n + (c >> 1); return QUnit{w, (w % p.nx) * 256 + (c & 1) * 128, 1}; }
  const int w = p.n_rounds * n + c;
  return QUnit{w, (w % p.nx) * 256, 2};
}
// number of units CTA c walks over
AS_DEV int q_units_of_cta(const QParams& p) {
  const int left = p.n_units - p.n_rounds * (int)gridDim.x;
  const int extra = p.split_last ? ((int)blockIdx.x < 2 * left) : ((int)blockIdx.x < left);
  return p.n_rounds + (extra ? 1 : 0);
}

template <int D>
struct QRing {
  using L = QLayout<D>;
  // barrier indices; per group: S (scores or Phi landed), SF (score columns read out), P (P or phi_q in
  // shared memory), PF (the product that reads the P buffer has completed), O (output accumulator final),
  // QF (nothing of the unit reads the Q tile any more)
  static constexpr int B_Q0 = 0, B_FULL = 2, B_EMPTY = B_FULL + KV_STAGES, B_S = B_EMPTY + KV_STAGES, B_SF = B_S + 2,
                       B_P = B_SF + 2, B_PF = B_P + 2, B_O = B_PF + 2, B_QF = B_O + 2, B_COUNT = B_QF + 2;
  const QCtx c;              // by value: nothing here is re-read from memory after a barrier or an MMA
  int nkv, lin, two;
  int it_h, it_w, it_vlast, it_st, n_items, n_sp;
  // Ring items of one unit, in the order they are consumed: K_0; then K_{j+1}, V_j for j = 0 .. nkv-2;
  // then for the linear tail (two-layer map: the two groups' first-layer activations,) the last-layer
  // weights; V_{nkv-1}; S in bf16.
  AS_DEV QRing(int nkv_, int lin_, int layers, const QCtx& c_) : c(c_), nkv(nkv_), lin(lin_), two(lin_ && layers == 2) {
    int next = nkv > 0 ? 2 * nkv - 1 : 0;
    it_h = next; if (two) next += 2;
    it_w = next; if (lin) next += 1;
    it_vlast = next; if (nkv > 0) next += 1;
    it_st = next; if (lin) next += 1;
    n_items = next;
    n_sp = nkv + lin;                    // per unit and group: S completions = P hand-overs = P-buffer releases
  }
  AS_DEV int item_k(int j) const { return j == 0 ? 0 : 2 * j - 1; }
  AS_DEV int item_v(int j) const { return j + 1 < nkv ? 2 * j + 2 : it_vlast; }
  AS_DEV uint32_t bar(int i) const { return c.sbase + L::BAR_OFF + 8 * i; }
  AS_DEV uint32_t sQ(int g) const { return c.sbase + L::Q_OFF + g * L::TILE; }
  AS_DEV uint32_t sP(int g) const { return c.sbase + L::P_OFF + g * L::PTILE; }
  // The K/V ring is indexed by a running item number that does not restart with a unit.
  AS_DEV uint32_t sKV(int item) const { return c.sbase + L::KV_OFF + (item % KV_STAGES) * L::TILE; }
  AS_DEV uint32_t tS(int g) const { return c.tmem + 128u * g; }
  AS_DEV uint32_t tO(int g) const { return c.tmem + 256u + 128u * g; }
  AS_DEV bool wait(int b, int phase) const { return mbar_wait_warp(bar(b), phase & 1, c.wc); }
  AS_DEV void release(int item) const { tc_commit(bar(B_EMPTY + item % KV_STAGES)); }
  // single-thread forms for the issuing thread (no warp vote): a wait that is already satisfied still
  // costs a round trip to shared memory, so barriers needed together are probed together
  AS_DEV bool wait1(int b, int phase) const { return mbar_wait(bar(b), phase & 1, c.wc); }
  AS_DEV bool probe(int b, int phase) const { return mbar_try_wait(bar(b), phase & 1); }
  AS_DEV bool wait_full(int item) const { return wait1(B_FULL + item % KV_STAGES, item / KV_STAGES); }
  // barrier b0 and, when use1, the ring item's full barrier
  AS_DEV bool wait2(int b0, int ph0, bool use1, int item) const {
    const int b1 = B_FULL + item % KV_STAGES, ph1 = item / KV_STAGES;
    const bool r0 = probe(b0, ph0);
    const bool r1 = use1 ? probe(b1, ph1) : true;
    if (r0 && r1) return true;
    if (!r1 && !wait1(b1, ph1)) return false;
    return r0 || wait1(b0, ph0);
  }
};

// ---------------------------------------------------------------- TMA producer, one unit
template <int D>
__device__ __noinline__ bool q_produce_unit(const QParams& p, const QCtx& c, const CUtensorMap* tmQ, const CUtensorMap* tmK,
                                            const CUtensorMap* tmV, const CUtensorMap* tmW, const CUtensorMap* tmSt,
                                            const CUtensorMap* tmH, int u) {
  using R = QRing<D>;
  using L = QLayout<D>;
  const int nkv = p.nkv;
  const R q(nkv, p.lin, p.layers, c);
  const int lane = threadIdx.x & 31;
  const QUnit un = q_unit(p, u);
  const int bh = un.w / p.nx, h = bh % p.H, row0 = un.row0;
  const int base = u * q.n_items;
  const int n_stream = nkv > 0 ? 2 * nkv - 1 : 0;     // K_0, then K_{j+1}, V_j alternating
  const int q_at = nkv > 0 ? 1 : 0;                   // the Q tiles are requested right after the unit's first K tile
  for (int it = 0; it < q.n_items; ++it) {
    if (it == q_at) {
      for (int g = 0; g < un.ng; ++g) {
        // the previous unit's last product that reads this Q buffer has completed
        if (u > 0 && !q.wait(R::B_QF + g, u - 1)) return false;
        if (lane == 0) {
          mbar_expect_tx(q.bar(R::B_Q0 + g), L::TILE);
          load_tile<D>(q.sQ(g), tmQ, q.bar(R::B_Q0 + g), row0 + g * 128, bh);
        }
        __syncwarp();
      }
    }
    const int gi = base + it, st = gi % KV_STAGES;
    if (!q.wait(R::B_EMPTY + st, gi / KV_STAGES + 1)) return false;
    if (lane == 0) {
      mbar_expect_tx(q.bar(R::B_FULL + st), L::TILE);
      const uint32_t fb = q.bar(R::B_FULL + st);
      if (it < n_stream) {
        if (it == 0 || (it & 1)) load_tile<D>(q.sKV(gi), tmK, fb, ((it + 1) >> 1) * 128, bh);   // K_0 at 0, K_j at 2j-1
        else load_tile<D>(q.sKV(gi), tmV, fb, ((it >> 1) - 1) * 128, bh);                        // V_j at 2j+2
      } else if (q.two && it < q.it_w) {
        load_tile<D>(q.sKV(gi), tmH, fb, row0 + (it - q.it_h) * 128, bh);    // relu(q W_1^T) of group it - it_h
      } else if (q.lin && it == q.it_w) {
        load_tile<D>(q.sKV(gi), tmW, fb, 0, h);                              // last-layer W_q[h]: [F rows][D]
      } else if (nkv > 0 && it == q.it_vlast) {
        load_tile<D>(q.sKV(gi), tmV, fb, (nkv - 1) * 128, bh);
      } else {
        load_tile<D>(q.sKV(gi), tmSt, fb, 0, bh);                            // S[bh] in bf16: [F rows][D]
      }
    }
    __syncwarp();
  }
  return true;
}

// ---------------------------------------------------------------- MMA issuers, one unit
// Two issuing threads (lane 0 of warps 9 and 10; the other lanes wait at the end of the role): one issues
// what writes the score columns (Q K^T per tile, Phi at the end) as soon as the softmax threads have read
// them out, the other what accumulates into O (P V per tile, phi_q S at the end) as soon as P is in
// shared memory.  The two streams touch different TMEM columns and release different ring items, so they
// need no ordering between them; each thread's commits cover its own MMAs.  An issuing thread is the
// busiest resource of the CTA - every clock it spends outside the MMA instructions is a clock the tensor
// pipe may idle - so it takes no warp votes or warp barriers, probes the barriers it needs together, and
// has its operands ready before it looks at a barrier.
template <int D>
__device__ __noinline__ bool q_score_unit(const QParams& p, const QCtx& c, int u) {
  using R = QRing<D>;
  constexpr int F = D;
  constexpr uint32_t ID_QK = make_idesc(128, 128, 0, 0);      // S = Q K^T      (N = 128 keys)
  constexpr uint32_t ID_PHI = make_idesc(128, F, 0, 0);       // Phi = Q W_q^T  (N = F)
  const int nkv = p.nkv, lin = p.lin;
  const R q(nkv, lin, p.layers, c);
  const int base = u * q.n_items, pb = u * q.n_sp;            // first ring item / first barrier phase of the unit
  const int ng = q_unit(p, u).ng;                             // groups at work on this unit (the last one of a group: ng - 1)
  uint64_t dq[2][8];                                          // the Q tiles do not move within a unit
#pragma unroll
  for (int g = 0; g < 2; ++g) {
    const uint64_t q0 = kmajor_desc(q.sQ(g));
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) dq[g][kk] = q0 + kstep_kmajor(kk);
  }
  // Phi = X W^T with X = Q (one layer) or the first-layer activations (two layers), N = F
  auto issue_phi = [&](int g) {
    const uint64_t w0 = kmajor_desc(q.sKV(base + q.it_w));
    if (q.two) {
      const uint64_t x0 = kmajor_desc(q.sKV(base + q.it_h + g));
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk) mma_ss(q.tS(g), x0 + kstep_kmajor(kk), w0 + kstep_kmajor(kk), ID_PHI, kk > 0 ? 1u : 0u);
    } else {
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk) mma_ss(q.tS(g), dq[g][kk], w0 + kstep_kmajor(kk), ID_PHI, kk > 0 ? 1u : 0u);
    }
    tc_commit(q.bar(R::B_S + g));
    tc_commit(q.bar(R::B_QF + g));                   // nothing of this unit reads the group's Q tile any more
    if (q.two) q.release(base + q.it_h + g);
    if (g == ng - 1) {
      // a lone group: the other group's first-layer tile was loaded all the same and only has to be let go
      if (q.two && ng == 1) { q.wait_full(base + q.it_h + 1); q.release(base + q.it_h + 1); }
      q.release(base + q.it_w);
    }
  };
  // The first product of a unit overwrites score columns the previous unit's threads read last: wait for
  // that read (the last S-free phase of the previous unit) together with the Q tile.
  for (int g = 0; g < ng; ++g) {
    if (u > 0 && !q.wait1(R::B_SF + g, pb - 1)) return false;
    if (nkv == 0) {
      if (!q.wait1(R::B_Q0 + g, u)) return false;
      if (lin) {
        // no softmax tokens at all: the feature product opens the unit
        if (!q.wait_full(base + q.it_w)) return false;
        if (q.two && !q.wait_full(base + q.it_h + g)) return false;
        tc_fence_after();
        issue_phi(g);
      }
    } else {
      if (!q.wait2(R::B_Q0 + g, u, g == 0, base)) return false;
      tc_fence_after();
      const uint64_t k0 = kmajor_desc(q.sKV(base));
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk) mma_ss(q.tS(g), dq[g][kk], k0 + kstep_kmajor(kk), ID_QK, kk > 0 ? 1u : 0u);
      tc_commit(q.bar(R::B_S + g));
      if (g == ng - 1) q.release(base);
      if (nkv == 1 && !lin) tc_commit(q.bar(R::B_QF + g));
    }
  }
  for (int j = 0; j < nkv; ++j) {
    const bool last = (j + 1 == nkv);
    // as soon as the groups have read their score rows: the next tile's Q K^T, or Phi after the last tile
    if (!last) {
      const int ik = base + q.item_k(j + 1);
      const uint64_t k0 = kmajor_desc(q.sKV(ik));
#pragma unroll
      for (int g = 0; g < 2; ++g) {
        if (g >= ng) break;
        if (!q.wait2(R::B_SF + g, pb + j, g == 0, ik)) return false;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) mma_ss(q.tS(g), dq[g][kk], k0 + kstep_kmajor(kk), ID_QK, kk > 0 ? 1u : 0u);
        tc_commit(q.bar(R::B_S + g));
        if (j + 2 == nkv && !lin) tc_commit(q.bar(R::B_QF + g));   // the unit's last read of the Q tile
      }
      q.release(ik);
    } else if (lin) {
      for (int g = 0; g < ng; ++g) {
        if (!q.wait2(R::B_SF + g, pb + j, g == 0, base + q.it_w)) return false;
        if (q.two && !q.wait_full(base + q.it_h + g)) return false;
        tc_fence_after();
        issue_phi(g);
      }
    }
  }
  return true;
}

template <int D>
__device__ __noinline__ bool q_accum_unit(const QParams& p, const QCtx& c, int u) {
  using R = QRing<D>;
  constexpr int F = D;
  constexpr uint32_t ID_PV = make_idesc(128, D, 0, 1);        // O += P V and O += phi_q S  (V, S are MN-major)
  const int nkv = p.nkv, lin = p.lin;
  const R q(nkv, lin, p.layers, c);
  const int base = u * q.n_items, pb = u * q.n_sp;            // first ring item / first barrier phase of the unit
  const int ng = q_unit(p, u).ng;
  uint64_t dp[2][8];                                          // the P tiles never move
#pragma unroll
  for (int g = 0; g < 2; ++g) {
    const uint64_t p0 = kmajor_desc(q.sP(g));
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) dp[g][kk] = p0 + kstep_kmajor(kk);
  }
  for (int j = 0; j < nkv; ++j) {
    const bool last = (j + 1 == nkv);
    // as soon as P is in shared memory: O += P V
    const int iv = base + q.item_v(j);
    const uint64_t v0 = mnmajor_desc(q.sKV(iv));
#pragma unroll
    for (int g = 0; g < 2; ++g) {
      if (g >= ng) break;
      if (!q.wait2(R::B_P + g, pb + j, g == 0, iv)) return false;
      tc_fence_after();
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) mma_ss(q.tO(g), dp[g][kk], v0 + kstep_mnmajor(kk), ID_PV, (j > 0 || kk > 0) ? 1u : 0u);
      tc_commit(q.bar(R::B_PF + g));
      if (last && !lin) tc_commit(q.bar(R::B_O + g));
    }
    q.release(iv);
  }
  if (lin) {
    const int is = base + q.it_st;
    const uint64_t s0 = mnmajor_desc(q.sKV(is));
    for (int g = 0; g < ng; ++g) {
      if (!q.wait2(R::B_P + g, pb + nkv, g == 0, is)) return false;
      tc_fence_after();
      // phi_q sits where P sits, S plays the part of a V tile
#pragma unroll
      for (int kk = 0; kk < F / 16; ++kk) mma_ss(q.tO(g), dp[g][kk], s0 + kstep_mnmajor(kk), ID_PV, (nkv > 0 || kk > 0) ? 1u : 0u);
      tc_commit(q.bar(R::B_PF + g));
      tc_commit(q.bar(R::B_O + g));
      if (g == ng - 1) q.release(is);
    }
  }
  return true;
}

// ---------------------------------------------------------------- softmax / merge group, one unit
template <int D>
__device__ __noinline__ bool q_softmax_unit(const QParams& p, const QCtx& c, const CUtensorMap* tmO, uint8_t* smem, int u) {
  using R = QRing<D>;
  using L = QLayout<D>;
  constexpr int F = D;
  const int nkv = p.nkv, n_s = p.n_s;
  const float scale_log2 = p.scale_log2;
  const R q(nkv, p.lin, p.layers, c);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = warp >> 2;                          // group 0 or 1
  const int r = (warp & 3) * 32 + lane;             // row inside the group's 128-row tile
  const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
  const uint32_t tSg = q.tS(g) + lane_off, tOg = q.tO(g) + lane_off;
  uint8_t* sPg = smem + L::P_OFF + g * L::PTILE;    // this group's P / phi_q / output staging tile
  const int pb = u * q.n_sp;
  float m_ref = 0.f, m_true = -INFINITY, l = 0.f;
  uint32_t x[32];

  // The P buffer may be written once the product that read its previous contents has completed; the very
  // first use only has to wait for this warp's output store of the previous unit to have been read out.
  auto p_buffer_free = [&](int use) -> bool {       // use: running index of the buffer's uses
    if (lane == 0) tma_store_wait_read();
    if (use == 0) { __syncwarp(); return true; }
    return q.wait(R::B_PF + g, use - 1);
  };

  for (int j = 0; j < nkv; ++j) {
    if (!q.wait(R::B_S + g, pb + j)) return false;
    tc_fence_after();
    uint32_t sv[128];                               // this thread's row of the 128 x 128 score tile
    tmem_ld128_sync(tSg, sv);
    tc_fence_before();
    mbar_arrive(q.bar(R::B_SF + g));                // the score columns may be overwritten
    const int valid = n_s - j * 128;                // keys of this tile that exist (>= 128: all)
    if (valid < 128) {
#pragma unroll
      for (int i = 0; i < 128; ++i) sv[i] = (i < valid) ? sv[i] : 0xff800000u;   // -inf: exp2 gives 0
    }
    float mx0 = fmax3(__uint_as_float(sv[0]), __uint_as_float(sv[1]), __uint_as_float(sv[2]));
    float mx1 = fmax3(__uint_as_float(sv[3]), __uint_as_float(sv[4]), __uint_as_float(sv[5]));
#pragma unroll
    for (int i = 6; i + 3 < 128; i += 4) {
      mx0 = fmax3(mx0, __uint_as_float(sv[i]), __uint_as_float(sv[i + 1]));
      mx1 = fmax3(mx1, __uint_as_float(sv[i + 2]), __uint_as_float(sv[i + 3]));
    }
    float mx = fmax3(mx0, mx1, fmaxf(__uint_as_float(sv[126]), __uint_as_float(sv[127])));
    mx *= scale_log2;
    m_true = fmaxf(m_true, mx);
    // The reference maximum only moves when the row maximum grew by more than 2^8; then O and l
    // are rescaled (once the previous tile's P V has completed, before this tile's P is handed over).
    const bool need = (j > 0) && (mx > m_ref + RESCALE_THRESHOLD);
    const float resc = need ? ex2(m_ref - mx) : 1.f;
    if (j == 0 || need) m_ref = mx;
    // P = exp2(s * scale_log2 - m_ref) as bf16 into the group's P tile in shared memory
    const float neg_m = -m_ref;
    // packed fp32x2 arithmetic halves the instruction count of the scaling and of the row sum
    const float2 scale2 = make_float2(scale_log2, scale_log2), negm2 = make_float2(neg_m, neg_m);
    float2 la = make_float2(0.f, 0.f), lb = make_float2(0.f, 0.f);
#pragma unroll
    for (int cc = 0; cc < 4; ++cc) {
      uint32_t pw[16];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int k = cc * 32 + 4 * i;
        const float2 xa = __ffma2_rn(make_float2(__uint_as_float(sv[k]), __uint_as_float(sv[k + 1])), scale2, negm2);
        const float2 xb = __ffma2_rn(make_float2(__uint_as_float(sv[k + 2]), __uint_as_float(sv[k + 3])), scale2, negm2);
        const float2 pa = make_float2(ex2(xa.x), ex2(xa.y)), pc = make_float2(ex2(xb.x), ex2(xb.y));
        la = __fadd2_rn(la, pa);
        lb = __fadd2_rn(lb, pc);
        pw[2 * i] = pack_bf16(pa.x, pa.y);
        pw[2 * i + 1] = pack_bf16(pc.x, pc.y);
      }
      if (cc == 0 && !p_buffer_free(pb + j)) return false;   // the previous tile's P V has read the buffer
      store_row_chunk(sPg, r, cc * 32, pw);
    }
    // The sum above adds the unrounded probabilities while the MMA multiplies their bf16 roundings with V.
    // Over many keys the rounding errors average out, but the error of a probability that dominates its
    // row does not, and a result close to one large v_j would be off by up to 2^-9 of its value.  So the
    // sum takes over the rounding error of the tile's largest probability.
    const float p_top = ex2(mx - m_ref);
    const float p_top_err = __uint_as_float(pack_bf16(0.f, p_top) & 0xffff0000u) - p_top;
    l = l * resc + (((la.x + la.y) + (lb.x + lb.y)) + p_top_err);
    if (__any_sync(0xffffffffu, need)) {
      // the previous tile's P V has completed (waited for above) and this tile's has not been released yet
      tc_fence_after();
#pragma unroll
      for (int cc = 0; cc < D / 32; ++cc) {
        tmem_ld32(tOg + cc * 32, x);
        tmem_ld_wait(x);
#pragma unroll
        for (int i = 0; i < 32; ++i) x[i] = __float_as_uint(__uint_as_float(x[i]) * resc);
        tmem_st32(tOg + cc * 32, x);
      }
      tmem_st_wait();
      tc_fence_before();
    }
    fence_proxy_async();
    mbar_arrive(q.bar(R::B_P + g));
  }

  const QUnit un = q_unit(p, u);
  const int bh = un.w / p.nx;
  const int row = un.row0 + g * 128 + r;
  float den = l, den_l_out = 0.f;
  if (p.lin) {
    // per-row factor applied to phi_q so that the linear branch lands on the scale of O and l
    float e = 0.f;
    if (nkv > 0) e = (p.stab_mode == AS_STAB_EXACT) ? -m_ref : (m_true - m_ref);
    e = fminf(fmaxf(e, -100.f), 100.f);
    const float lam = ex2(e);
    const float2* zrow = reinterpret_cast<const float2*>(p.z + (size_t)bh * F);
    if (!q.wait(R::B_S + g, pb + nkv)) return false;
    tc_fence_after();
    uint32_t ph[F];                                  // this thread's row of Phi: read at once, columns released
    float dl0 = 0.f, dl1 = 0.f;
    const bool two_parts = (p.P == 2);
#pragma unroll
    for (int cc = 0; cc < F / 32; ++cc) {
      tmem_ld32(tSg + cc * 32, x);
      tmem_ld_wait(x);
#pragma unroll
      for (int i = 0; i < 32; ++i) ph[cc * 32 + i] = x[i];
    }
    tc_fence_before();
    mbar_arrive(q.bar(R::B_SF + g));                 // the next unit's first Q K^T may overwrite the columns
    if (!p_buffer_free(pb + nkv)) return false;      // the last tile's P V has read the buffer
#pragma unroll
    for (int cc = 0; cc < F / 32; ++cc) {
      const bool squared = two_parts && (cc * 32 >= F / 2);
      uint32_t wd[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        float a0 = fmaxf(__uint_as_float(ph[cc * 32 + 2 * i]), 0.f), a1 = fmaxf(__uint_as_float(ph[cc * 32 + 2 * i + 1]), 0.f);
        if (squared) { a0 *= a0; a1 *= a1; }
        wd[i] = pack_bf16(a0 * lam, a1 * lam);
        // the denominator uses the very bf16 values the MMA multiplies with S
        const float2 zz = __ldg(zrow + cc * 16 + i);   // same address in every lane: one broadcast load
        dl0 = fmaf(__uint_as_float(wd[i] << 16), zz.x, dl0);
        dl1 = fmaf(__uint_as_float(wd[i] & 0xffff0000u), zz.y, dl1);
      }
      store_row_chunk(sPg, r, cc * 32, wd);          // phi_q takes P's place as the A operand
    }
    const float dl = dl0 + dl1;
    fence_proxy_async();
    mbar_arrive(q.bar(R::B_P + g));
    den = l + dl;
    den_l_out = dl / lam;
  }
  if (!q.wait(R::B_O + g, u)) return false;
  tc_fence_after();
  const float inv = 1.f / den;
  // The output rows are staged in the group's P tile (the product that read it has completed with the O
  // barrier); each warp stores its own 32 rows (rows past N are clipped by the tensor map).
  const int wrow0 = row - lane;
#pragma unroll
  for (int cc = 0; cc < D / 32; ++cc) {
    tmem_ld32(tOg + cc * 32, x);
    tmem_ld_wait(x);
    uint32_t wd[16];
#pragma unroll
    for (int i = 0; i < 16; ++i)
      wd[i] = pack_bf16(__uint_as_float(x[2 * i]) * inv, __uint_as_float(x[2 * i + 1]) * inv);
    store_row_chunk(sPg, r, cc * 32, wd);
  }
  fence_proxy_async();
  __syncwarp();
  if (lane == 0 && wrow0 < p.N) {
#pragma unroll
    for (int b = 0; b < D / 64; ++b)
      tma_store_3d(tmO, smem_u32(sPg) + b * BOX_BYTES + (warp & 3) * 32 * 128, b * 64, wrow0, bh);
    tma_store_commit();
  }
  if (p.aux != nullptr && row < p.N) {
    const float ln2 = 0.6931471805599453f;
    float* ap = p.aux + ((size_t)bh * p.N + row) * 3;
    ap[0] = nkv > 0 ? m_true * ln2 : 0.f;
    ap[1] = nkv > 0 ? l * ex2(m_ref - m_true) : 0.f;
    ap[2] = den_l_out;
  }
  // The next unit's first P V overwrites O: every tcgen05.ld above has completed (tmem_ld_wait), and
  // the arrive on the P barrier that releases that MMA follows in program order.
  tc_fence_before();
  return true;
}

template <int D>
__global__ void __launch_bounds__(Q_THREADS, 1)
qpass_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
             const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmW,
             const __grid_constant__ CUtensorMap tmSt, const __grid_constant__ CUtensorMap tmH,
             const __grid_constant__ CUtensorMap tmO, const __grid_constant__ QParams p) {
  using L = QLayout<D>;
  using R = QRing<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::BAR_OFF + 8 * R::B_COUNT);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + L::BAR_OFF + 8 * R::B_COUNT + 4);
  auto bar = [&](int i) { return sbase + L::BAR_OFF + 8 * i; };
  const int warp = threadIdx.x >> 5;

  // an earlier CTA of this or a previous launch timed out: do nothing (decided once per CTA)
  __shared__ uint32_t s_skip;
  if (threadIdx.x == 0) s_skip = *reinterpret_cast<volatile uint32_t*>(p.status);
  __syncthreads();
  if (s_skip != 0u) return;

  if (threadIdx.x == 0) {
    *abort_flag = 0u;
    mbar_init(bar(R::B_Q0), 1); mbar_init(bar(R::B_Q0 + 1), 1);
    for (int s = 0; s < KV_STAGES; ++s) { mbar_init(bar(R::B_FULL + s), 1); mbar_init(bar(R::B_EMPTY + s), 1); }
    for (int g = 0; g < 2; ++g) {
      mbar_init(bar(R::B_S + g), 1); mbar_init(bar(R::B_SF + g), 128); mbar_init(bar(R::B_P + g), 128);
      mbar_init(bar(R::B_PF + g), 1); mbar_init(bar(R::B_O + g), 1); mbar_init(bar(R::B_QF + g), 1);
    }
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 9) { tmem_alloc(smem_u32(tmem_slot), 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const QCtx c{sbase, *tmem_slot, WaitCtx{p.status, abort_flag}};
  const int n_mine = q_units_of_cta(p);               // units of this CTA

  if (warp == 8) {
    if ((threadIdx.x & 31) == 0) { tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmO); }
    for (int u = 0; u < n_mine; ++u)
      if (!q_produce_unit<D>(p, c, &tmQ, &tmK, &tmV, &tmW, &tmSt, &tmH, u)) break;
  } else if (warp == 9) {
    if ((threadIdx.x & 31) == 0) {
      for (int u = 0; u < n_mine; ++u)
        if (!q_score_unit<D>(p, c, u)) break;
    }
    __syncwarp();
  } else if (warp == 10) {
    if ((threadIdx.x & 31) == 0) {
      for (int u = 0; u < n_mine; ++u)
        if (!q_accum_unit<D>(p, c, u)) break;
    }
    __syncwarp();
  } else {
    // a unit worked on by one group only (a left-over half) is the CTA's last one: group 1 stops before it
    const int n_grp = (n_mine > p.n_rounds && p.split_last && warp >= 4) ? p.n_rounds : n_mine;
    for (int u = 0; u < n_grp; ++u)
      if (!q_softmax_unit<D>(p, c, &tmO, smem, u)) break;
    if ((threadIdx.x & 31) == 0) tma_store_wait_all();   // this warp's output stores have completed
  }

  // ------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 9) {
    tc_fence_after();
    tmem_dealloc(c.tmem, 512);
  }
}

}  // namespace

cudaError_t as_tensor_init_qpass() {
  cudaError_t e;
  if ((e = opt_in_smem(qpass_kernel<128>, QLayout<128>::TOTAL)) != cudaSuccess) return e;
  if ((e = opt_in_smem(qpass_kernel<64>, QLayout<64>::TOTAL)) != cudaSuccess) return e;
  return cudaSuccess;
}

cudaError_t as_tensor_qpass(const as_launch_args& a, cudaStream_t st) {
  const int BH = a.B * a.H;
  const bool lin = a.n_l > 0;
  CUtensorMap tmQ, tmK, tmV, tmW, tmSt, tmH, tmO;
  // the output is stored warp by warp: boxes of 32 rows
  if (!make_map(&tmQ, a.q, a.d, a.N, BH, 128) || !make_map(&tmO, a.out, a.d, a.N, BH, 32)) return cudaErrorInvalidValue;
  if (a.n_s > 0) {
    if (!make_map(&tmK, a.ks, a.d, a.n_s, BH, 128) || !make_map(&tmV, a.vs, a.d, a.n_s, BH, 128)) return cudaErrorInvalidValue;
  } else {
    tmK = tmQ; tmV = tmQ;       // never used: the key loop is empty
  }
  if (lin) {
    // boxes are always 128 rows: rows past F (or d) are out of bounds and arrive as zeros
    if (!make_map(&tmW, a.layers == 2 ? a.wq2 : a.wq, a.d, a.F, a.H, 128) || !make_map(&tmSt, a.Sb, a.d, a.F, BH, 128)) return cudaErrorInvalidValue;
  } else {
    tmW = tmQ; tmSt = tmQ;      // never used: no linear branch at rate 1
  }
  if (lin && a.layers == 2) { if (!make_map(&tmH, a.h1q, a.d, a.N, BH, 128)) return cudaErrorInvalidValue; }
  else tmH = tmQ;             // never used with a one-layer map
  QParams p{};
  p.layers = lin ? a.layers : 1;
  p.N = a.N; p.n_s = a.n_s; p.nkv = (a.n_s + 127) / 128; p.lin = lin ? 1 : 0; p.stab_mode = a.stab_mode; p.P = a.P;
  p.H = a.H;
  p.scale_log2 = a.scale * 1.4426950408889634f;
  p.z = a.z; p.aux = a.aux; p.status = a.status;
  p.nx = (a.N + 255) / 256;
  p.n_units = p.nx * BH;
  // persistent: one CTA per SM (the kernel's shared memory and its 512 TMEM columns allow no second one)
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
    return cudaErrorInvalidValue;
  dim3 grid(p.n_units < sms ? p.n_units : sms, 1, 1);
  p.n_rounds = p.n_units / (int)grid.x;
  const int left = p.n_units - p.n_rounds * (int)grid.x;
  // left-over units as 128-row halves when twice their number still fits the grid
  p.split_last = (left > 0 && 2 * left <= (int)grid.x) ? 1 : 0;
  if (a.d == 128) qpass_kernel<128><<<grid, Q_THREADS, QLayout<128>::TOTAL, st>>>(tmQ, tmK, tmV, tmW, tmSt, tmH, tmO, p);
  else qpass_kernel<64><<<grid, Q_THREADS, QLayout<64>::TOTAL, st>>>(tmQ, tmK, tmV, tmW, tmSt, tmH, tmO, p);
  return cudaGetLastError();
}
