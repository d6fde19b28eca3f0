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
//   tail, per chunk c of 128 features:
//                        Phi_c = Q W_q[c]^T -> TMEM (in the place of a next tile's scores), phi_q scaled per
//                        row as bf16 where P sat, O += phi_q,c S_c (S in bf16 read like a V tile),
//                        den = l + phi_q.z, y = O / den -> bf16 -> staged in the P tile -> TMA store.
//   two-layer feature map: the hidden activations relu(Q W_q1^T + b1) are formed in the same way first
//                        (128 hidden units at a time) and kept as bf16 in the P tile and, once nothing reads
//                        Q any more, in the Q tile; Phi_c = sum over the hidden slices of h1_j W_q2[c, j]^T.
// All tiles are staged by TMA with the 128-byte swizzle; every mbarrier wait is bounded.
#include "tensor_common.cuh"

namespace {

using namespace as_tc;

// ======================================================================================
// Q pass
// ======================================================================================
struct QParams {
  int N, n_s, nkv, lin, stab_mode, P, H;
  int layers;                // depth of the feature map (1 or 2)
  int F, fc, fcw;            // feature width, its chunks of 128 (ceil), width of a chunk (min(F, 128))
  int nh;                    // two layers: slices of the hidden width (each D wide)
  const __nv_bfloat16* b1;   // two layers: first-layer bias of this launch's first head [H][hidden], or nullptr
  const __nv_bfloat16* b2;   // last-layer bias [H][F], or nullptr
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
  // barrier indices; per group: S (scores, hidden activations or Phi landed in the score columns), SF (score
  // columns read out), P (P or phi_q in shared memory), PF (the product that reads the P tile has completed),
  // O (output accumulator final), QF (nothing of the unit reads the Q tile any more), H (two layers: the
  // hidden activations are in shared memory)
  static constexpr int B_Q0 = 0, B_FULL = 2, B_EMPTY = B_FULL + KV_STAGES, B_S = B_EMPTY + KV_STAGES, B_SF = B_S + 2,
                       B_P = B_SF + 2, B_PF = B_P + 2, B_O = B_PF + 2, B_QF = B_O + 2, B_H = B_QF + 2, B_COUNT = B_H + 2;
  const QCtx c;              // by value: nothing here is re-read from memory after a barrier or an MMA
  int nkv, lin, two, fc, nh, vl;
  int n_stream, n_items;
  int n_s, n_p, n_pf;        // per unit and group: uses of the score columns, P hand-overs, releases of the P tile
  // Ring items of one unit, in the order they are consumed: K_0; then K_{j+1}, V_j for j = 0 .. nkv-2; then
  // the linear tail with V_{nkv-1} in second place:
  //   one layer:   W[0], V_last, then W[c], S[c-1] for c = 1 .. fc-1, then S[fc-1]
  //   two layers:  W1[0], V_last, W1[1 .. nh-1], then W2[c, j] (c slow), then S[0 .. fc-1]
  // addresses and waits only (the key loop needs nothing else)
  AS_DEV explicit QRing(const QCtx& c_) : c(c_), nkv(0), lin(0), two(0), fc(0), nh(0), vl(0), n_stream(0), n_items(0), n_s(0), n_p(0), n_pf(0) {}
  AS_DEV QRing(const QParams& p, const QCtx& c_)
      : c(c_), nkv(p.nkv), lin(p.lin), two(p.lin && p.layers == 2), fc(p.lin ? p.fc : 0), nh(p.nh), vl(p.nkv > 0 ? 1 : 0) {
    n_stream = nkv > 0 ? 2 * nkv - 1 : 0;
    n_items = n_stream + vl + (two ? nh + fc * nh + fc : 2 * fc);
    n_s = nkv + (two ? nh + fc : fc);
    n_p = nkv + fc;
    n_pf = nkv + (two ? 1 : fc);
  }
  AS_DEV int item_k(int j) const { return j == 0 ? 0 : 2 * j - 1; }
  AS_DEV int it_vlast() const { return n_stream + (lin ? 1 : 0); }   // after the tail's first weight tile, if there is a tail
  AS_DEV int item_v(int j) const { return j + 1 < nkv ? 2 * j + 2 : it_vlast(); }
  // one layer: last-layer weights of feature chunk ch; two layers: first-layer weights of hidden slice ch
  AS_DEV int it_w(int ch) const { return ch == 0 ? n_stream : (two ? n_stream + vl + ch : n_stream + vl + 2 * ch - 1); }
  AS_DEV int it_w2(int ch, int j) const { return n_stream + vl + nh + ch * nh + j; }
  AS_DEV int it_st(int ch) const {
    if (two) return n_stream + vl + nh + fc * nh + ch;
    return ch + 1 < fc ? n_stream + vl + 2 * ch + 2 : n_stream + vl + 2 * fc - 1;
  }
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
template <int D, bool TWO, bool GEN>
__device__ __noinline__ bool q_produce_unit(const QParams& p, const QCtx& c, const CUtensorMap* tmQ, const CUtensorMap* tmK,
                                            const CUtensorMap* tmV, const CUtensorMap* tmW, const CUtensorMap* tmSt,
                                            const CUtensorMap* tmW1, int u) {
  using R = QRing<D>;
  using L = QLayout<D>;
  const int nkv = p.nkv;
  const R q(p, c);
  const int lane = threadIdx.x & 31;
  const QUnit un = q_unit(p, u);
  const int bh = un.w / p.nx, h = bh % p.H, row0 = un.row0;
  const int base = u * q.n_items;
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
      const uint32_t fb = q.bar(R::B_FULL + st), dst = q.sKV(gi);
      if (it < q.n_stream) {
        if (it == 0 || (it & 1)) load_tile<D>(dst, tmK, fb, ((it + 1) >> 1) * 128, bh);   // K_0 at 0, K_j at 2j-1
        else load_tile<D>(dst, tmV, fb, ((it >> 1) - 1) * 128, bh);                        // V_j at 2j+2
      } else if (q.vl && it == q.it_vlast()) {
        load_tile<D>(dst, tmV, fb, (nkv - 1) * 128, bh);
      } else if (!TWO) {
        // W[ch] / S[ch] in bf16: [128 feature rows][D]; rows past F arrive as zeros
        const int r = it - q.n_stream - (it > q.n_stream ? q.vl : 0);     // 0: W[0]; 2ch-1: W[ch]; 2ch+2 (and the last): S[ch]
        if (r == 0) load_tile<D>(dst, tmW, fb, 0, h);
        else if (r == 2 * q.fc - 1) load_tile<D>(dst, tmSt, fb, (q.fc - 1) * 128, bh);
        else if (r & 1) load_tile<D>(dst, tmW, fb, ((r + 1) >> 1) * 128, h);
        else load_tile<D>(dst, tmSt, fb, ((r >> 1) - 1) * 128, bh);
      } else {
        const int r = it - q.n_stream - (it > q.n_stream ? q.vl : 0);     // W1[0 .. nh-1], W2[c, j], S[c]
        if (r < q.nh) load_tile<D>(dst, tmW1, fb, r * 128, h);                                  // hidden rows of slice r
        else if (r < q.nh + q.fc * q.nh) {
          const int e = r - q.nh;
          load_boxes(dst, tmW, fb, (e % q.nh) * D, (e / q.nh) * 128, h, D / 64);                // W2[feature chunk, hidden slice]
        } else load_tile<D>(dst, tmSt, fb, (r - q.nh - q.fc * q.nh) * 128, bh);
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
template <int D, bool TWO, bool GEN>
__device__ __noinline__ bool q_score_unit(const QParams& p, const QCtx& c, int u) {
  using R = QRing<D>;
  constexpr uint32_t ID_QK = make_idesc(128, 128, 0, 0);      // S = Q K^T      (N = 128 keys)
  const int nkv = p.nkv, lin = p.lin;
  const R q(p, c);
  const uint32_t id_phi = make_idesc(128, D == 128 ? 128 : p.fcw, 0, 0);   // Phi_c = X W^T  (N = features of a chunk; 128 at d = 128)
  constexpr uint32_t ID_HID = make_idesc(128, D, 0, 0);       // hidden slice = Q W_1[j]^T (N = D hidden units)
  const int base = u * q.n_items, ps = u * q.n_s;             // first ring item / first score-column phase of the unit
  const int ng = q_unit(p, u).ng;                             // groups at work on this unit (the last one of a group: ng - 1)
  uint64_t dq[2][8];                                          // the Q tiles do not move within a unit
#pragma unroll
  for (int g = 0; g < 2; ++g) {
    const uint64_t q0 = kmajor_desc(q.sQ(g));
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) dq[g][kk] = q0 + kstep_kmajor(kk);
  }
  // The i-th product of the unit into a group's score columns overwrites what the threads read last: the
  // (i-1)-th use, or the previous unit's last one.
  auto s_free = [&](int g, int i) -> bool { return (u == 0 && i == 0) ? true : q.wait1(R::B_SF + g, ps + i - 1); };

  // ---- first key tile (its product opens the unit)
  if (nkv > 0) {
    for (int g = 0; g < ng; ++g) {
      if (!s_free(g, 0)) return false;
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
  // ---- as soon as the groups have read their score rows: the next tile's Q K^T
  for (int j = 0; j + 1 < nkv; ++j) {
    const int ik = base + q.item_k(j + 1);
    const uint64_t k0 = kmajor_desc(q.sKV(ik));
#pragma unroll
    for (int g = 0; g < 2; ++g) {
      if (g >= ng) break;
      if (!q.wait2(R::B_SF + g, ps + j, g == 0, ik)) return false;
      tc_fence_after();
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk) mma_ss(q.tS(g), dq[g][kk], k0 + kstep_kmajor(kk), ID_QK, kk > 0 ? 1u : 0u);
      tc_commit(q.bar(R::B_S + g));
      if (j + 2 == nkv && !lin) tc_commit(q.bar(R::B_QF + g));   // the unit's last read of the Q tile
    }
    q.release(ik);
  }
  if (!lin) return true;

  // ---- linear tail: what lands in the score columns after the last key tile
  if constexpr (!TWO) {
    // Phi_c = Q W[c]^T, one chunk of features after the other
    for (int ch = 0; ch < q.fc; ++ch) {
      const int iw = base + q.it_w(ch);
      const uint64_t w0 = kmajor_desc(q.sKV(iw));
      for (int g = 0; g < ng; ++g) {
        if (!s_free(g, nkv + ch)) return false;
        if (nkv == 0 && ch == 0 && !q.wait1(R::B_Q0 + g, u)) return false;
        if (g == 0 && !q.wait_full(iw)) return false;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) mma_ss(q.tS(g), dq[g][kk], w0 + kstep_kmajor(kk), id_phi, kk > 0 ? 1u : 0u);
        tc_commit(q.bar(R::B_S + g));
        if (ch == q.fc - 1) tc_commit(q.bar(R::B_QF + g));     // nothing of this unit reads the group's Q tile any more
      }
      q.release(iw);
    }
    return true;
  } else {
  // two layers: hidden slices first (A = Q), then Phi_c = sum_j h1_j W2[c, j]^T with the hidden slices read from
  // where the threads put them: slice 0 in the group's P tile, slice 1 in its Q tile
  for (int j = 0; j < q.nh; ++j) {
    const int iw = base + q.it_w(j);
    const uint64_t w0 = kmajor_desc(q.sKV(iw));
    for (int g = 0; g < ng; ++g) {
      if (!s_free(g, nkv + j)) return false;
      if (nkv == 0 && j == 0 && !q.wait1(R::B_Q0 + g, u)) return false;
      if (g == 0 && !q.wait_full(iw)) return false;
      tc_fence_after();
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk) mma_ss(q.tS(g), dq[g][kk], w0 + kstep_kmajor(kk), ID_HID, kk > 0 ? 1u : 0u);
      tc_commit(q.bar(R::B_S + g));
      if (q.nh == 1 && q.fc == 1) tc_commit(q.bar(R::B_QF + g));   // the Q tile is not reused as a buffer in this shape
    }
    q.release(iw);
  }
  for (int ch = 0; ch < q.fc; ++ch) {
    for (int j = 0; j < q.nh; ++j) {
      const int iw = base + q.it_w2(ch, j);
      const uint64_t w0 = kmajor_desc(q.sKV(iw));
      if (!q.wait_full(iw)) return false;
      for (int g = 0; g < ng; ++g) {
        if (j == 0) {
          if (!s_free(g, nkv + q.nh + ch)) return false;
          if (ch == 0 && !q.wait1(R::B_H + g, u)) return false;   // the group's hidden activations are in shared memory
        }
        tc_fence_after();
        const uint64_t a0 = kmajor_desc(j == 0 ? q.sP(g) : q.sQ(g));
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk)
          mma_ss(q.tS(g), a0 + kstep_kmajor(kk), w0 + kstep_kmajor(kk), id_phi, (j > 0 || kk > 0) ? 1u : 0u);
        if (j == q.nh - 1) {
          tc_commit(q.bar(R::B_S + g));
          // two hidden slices, one feature chunk: this was the last read of the Q tile (as a buffer)
          if (q.nh == 2 && q.fc == 1) tc_commit(q.bar(R::B_QF + g));
        }
      }
      q.release(iw);
    }
  }
  return true;
  }
}

template <int D, bool TWO, bool GEN>
__device__ __noinline__ bool q_accum_unit(const QParams& p, const QCtx& c, int u) {
  using R = QRing<D>;
  constexpr uint32_t ID_PV = make_idesc(128, D, 0, 1);        // O += P V and O += phi_q S  (V, S are MN-major)
  const int nkv = p.nkv, lin = p.lin;
  const R q(p, c);
  const int base = u * q.n_items, pp = u * q.n_p;             // first ring item / first P hand-over phase of the unit
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
      if (!q.wait2(R::B_P + g, pp + j, g == 0, iv)) return false;
      tc_fence_after();
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) mma_ss(q.tO(g), dp[g][kk], v0 + kstep_mnmajor(kk), ID_PV, (j > 0 || kk > 0) ? 1u : 0u);
      tc_commit(q.bar(R::B_PF + g));
      if (last && !lin) tc_commit(q.bar(R::B_O + g));
    }
    q.release(iv);
  }
  if (!lin) return true;
  // O += phi_q,c S_c per feature chunk: phi_q sits where P sits (two layers, second chunk: in the Q tile),
  // S plays the part of a V tile
  const int ksteps = (D == 128 ? 128 : p.fcw) / 16;           // a constant at d = 128: the chains below unroll
  for (int ch = 0; ch < q.fc; ++ch) {
    const int is = base + q.it_st(ch);
    const uint64_t s0 = mnmajor_desc(q.sKV(is));
    const bool in_q_tile = TWO && ch == 1;
    for (int g = 0; g < ng; ++g) {
      if (!q.wait2(R::B_P + g, pp + nkv + ch, g == 0, is)) return false;
      tc_fence_after();
      const uint64_t a0 = in_q_tile ? kmajor_desc(q.sQ(g)) : dp[g][0];
#pragma unroll
      for (int kk = 0; kk < 8; ++kk)
        if (kk < ksteps) mma_ss(q.tO(g), a0 + kstep_kmajor(kk), s0 + kstep_mnmajor(kk), ID_PV, (nkv > 0 || ch > 0 || kk > 0) ? 1u : 0u);
      if (!in_q_tile) tc_commit(q.bar(R::B_PF + g));           // a reader of the P tile has completed
      if (ch == q.fc - 1) {
        tc_commit(q.bar(R::B_O + g));
        if (in_q_tile) tc_commit(q.bar(R::B_QF + g));          // ... and the last reader of the Q tile
      }
    }
    q.release(is);
  }
  return true;
}

// ---------------------------------------------------------------- feature rows of the linear tail
// One row of Phi (feature chunk ch), already read out of the score columns into ph -> bf16(lam * poly(relu(Phi + b)))
// -> row r of `tile` (the A operand of the apply product).  Returns the row's share of phi_q.z, formed with the very
// bf16 values the MMA multiplies with S.  GEN = false is the common case (no bias, polynomial degree <= 2).
template <int D, bool GEN>
AS_DEV float q_features_to_tile(const QParams& p, const uint32_t (&ph)[128], uint8_t* tile, int r, int bh, int ch, float lam) {
  const int fcw = D == 128 ? 128 : p.fcw;            // a chunk is narrower than 128 only at d = F = 64
  const int part = p.F / p.P;
  const float2* zrow = reinterpret_cast<const float2*>(p.z + (size_t)bh * p.F + ch * 128);
  const uint32_t* brow = nullptr;
  if (GEN && p.b2 != nullptr) brow = reinterpret_cast<const uint32_t*>(p.b2 + (size_t)(bh % p.H) * p.F + ch * 128);
  float dl0 = 0.f, dl1 = 0.f;
#pragma unroll
  for (int cc = 0; cc < 4; ++cc) {
    if (cc * 32 < fcw) {
      const int pw = min((ch * 128 + cc * 32) / part, p.P - 1);     // 0-based part of these 32 features
      uint32_t wd[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        float a0 = __uint_as_float(ph[cc * 32 + 2 * i]), a1 = __uint_as_float(ph[cc * 32 + 2 * i + 1]);
        if (GEN && brow != nullptr) {
          const uint32_t bb = __ldg(brow + cc * 16 + i);            // same address in every lane: one broadcast load
          a0 += __uint_as_float(bb << 16);
          a1 += __uint_as_float(bb & 0xffff0000u);
        }
        a0 = fmaxf(a0, 0.f); a1 = fmaxf(a1, 0.f);
        float r0 = a0, r1 = a1;
        if (pw >= 1) { r0 *= a0; r1 *= a1; }
        if (GEN) {
          if (pw >= 2) { r0 *= a0; r1 *= a1; }
          if (pw >= 3) { r0 *= a0; r1 *= a1; }
        }
        wd[i] = pack_bf16(r0 * lam, r1 * lam);
        const float2 zz = __ldg(zrow + cc * 16 + i);
        dl0 = fmaf(__uint_as_float(wd[i] << 16), zz.x, dl0);
        dl1 = fmaf(__uint_as_float(wd[i] & 0xffff0000u), zz.y, dl1);
      }
      store_row_chunk(tile, r, cc * 32, wd);
    }
  }
  fence_proxy_async();
  return dl0 + dl1;
}

// The same for the one-layer tail, 32 columns at a time straight from the score columns (the loop is not unrolled:
// the tail runs once per unit, and on a CTA's first unit its instructions come from L2 line by line, so its
// size is its cost).  Arrives on `sf_bar` once the last columns are in registers.
template <int D, bool GEN>
AS_DEV float q_features_from_tmem(const QParams& p, uint32_t tSg, uint32_t sf_bar, uint8_t* tile, int r, int bh, int ch, float lam) {
  const int fcw = D == 128 ? 128 : p.fcw;
  const int part = p.F / p.P;
  const float2* zrow = reinterpret_cast<const float2*>(p.z + (size_t)bh * p.F + ch * 128);
  const uint32_t* brow = nullptr;
  if (GEN && p.b2 != nullptr) brow = reinterpret_cast<const uint32_t*>(p.b2 + (size_t)(bh % p.H) * p.F + ch * 128);
  const float2 lam2 = make_float2(lam, lam);
  float2 dl2 = make_float2(0.f, 0.f);
  uint32_t x[32];
#pragma unroll 1
  for (int cc = 0; cc * 32 < fcw; ++cc) {
    tmem_ld32(tSg + cc * 32, x);
    tmem_ld_wait(x);
    if (cc * 32 + 32 >= fcw) {
      tc_fence_before();
      mbar_arrive(sf_bar);                             // the next product into the score columns may follow
    }
    const int pw = min((ch * 128 + cc * 32) / part, p.P - 1);     // 0-based part of these 32 features
    uint32_t wd[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      float a0 = __uint_as_float(x[2 * i]), a1 = __uint_as_float(x[2 * i + 1]);
      if (GEN && brow != nullptr) {
        const uint32_t bb = __ldg(brow + cc * 16 + i);            // same address in every lane: one broadcast load
        a0 += __uint_as_float(bb << 16);
        a1 += __uint_as_float(bb & 0xffff0000u);
      }
      const float2 a = make_float2(fmaxf(a0, 0.f), fmaxf(a1, 0.f));
      float2 rr = a;
      if (pw >= 1) rr = __fmul2_rn(rr, a);
      if (GEN) {
        if (pw >= 2) rr = __fmul2_rn(rr, a);
        if (pw >= 3) rr = __fmul2_rn(rr, a);
      }
      rr = __fmul2_rn(rr, lam2);
      wd[i] = pack_bf16(rr.x, rr.y);
      const float2 zz = __ldg(zrow + cc * 16 + i);
      dl2 = __ffma2_rn(make_float2(__uint_as_float(wd[i] << 16), __uint_as_float(wd[i] & 0xffff0000u)), zz, dl2);
    }
    store_row_chunk(tile, r, cc * 32, wd);
  }
  fence_proxy_async();
  return dl2.x + dl2.y;
}

// Reads one row of the score columns (ncols of them) at once and releases the columns.
template <int D>
AS_DEV void q_read_row(const QRing<D>& q, int g, uint32_t tSg, int ncols, uint32_t (&ph)[128]) {
  using R = QRing<D>;
  uint32_t x[32];
#pragma unroll
  for (int cc = 0; cc < 4; ++cc) {
    if (cc * 32 < ncols) {
      tmem_ld32(tSg + cc * 32, x);
      tmem_ld_wait(x);
#pragma unroll
      for (int i = 0; i < 32; ++i) ph[cc * 32 + i] = x[i];
    }
  }
  tc_fence_before();
  mbar_arrive(q.bar(R::B_SF + g));                   // the next product into the score columns may follow
}

// Two-layer feature map, one unit and group: hidden slices relu(Q W_1[j]^T + b_1) as bf16 (slice 0 into the P tile,
// slice 1 into the Q tile, free once the product that made slice 1, the last reader of Q, has completed), then the
// feature chunks.  Returns phi_q.z, or -1 when a wait ran out.
template <int D, bool GEN>
__device__ __noinline__ float q_two_layer_tail(const QParams& p, const QRing<D>& q, int g, uint32_t tSg, uint8_t* sPg, uint8_t* sQg,
                                               int r, int bh, int ps, int ppf, float lam) {
  using R = QRing<D>;
  const int nkv = p.nkv, h = bh % p.H, lane = threadIdx.x & 31;
  const __nv_bfloat16* b1 = (GEN && p.b1) ? p.b1 + (size_t)h * (q.nh * D) : nullptr;
  uint32_t x[32];
  for (int j = 0; j < q.nh; ++j) {
    if (!q.wait(R::B_S + g, ps + nkv + j)) return -1.f;
    tc_fence_after();
    if (j == 0) {                                    // the last tile's P V has read the P tile (cf. the key loop)
      if (lane == 0) tma_store_wait_read();
      if (ppf + nkv == 0) __syncwarp();
      else if (!q.wait(R::B_PF + g, ppf + nkv - 1)) return -1.f;
    }
    const uint32_t* brow = b1 ? reinterpret_cast<const uint32_t*>(b1 + j * D) : nullptr;
    uint8_t* tile = j == 0 ? sPg : sQg;
#pragma unroll
    for (int cc = 0; cc < D / 32; ++cc) {
      tmem_ld32(tSg + cc * 32, x);
      tmem_ld_wait(x);
      uint32_t wd[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        float a0 = __uint_as_float(x[2 * i]), a1 = __uint_as_float(x[2 * i + 1]);
        if (brow != nullptr) {
          const uint32_t bb = __ldg(brow + cc * 16 + i);
          a0 += __uint_as_float(bb << 16);
          a1 += __uint_as_float(bb & 0xffff0000u);
        }
        wd[i] = pack_bf16(fmaxf(a0, 0.f), fmaxf(a1, 0.f));
      }
      store_row_chunk(tile, r, cc * 32, wd);
    }
    tc_fence_before();
    mbar_arrive(q.bar(R::B_SF + g));
    fence_proxy_async();
    mbar_arrive(q.bar(R::B_H + g));
  }
  // Feature chunks.  The hidden slices stay in their buffers until the last chunk's product has completed, so with
  // two chunks the first one's features wait in shared memory nobody else uses at that time: the rows of the group's
  // P tile are still the hidden slice, but ... (see below)
  if (!q.wait(R::B_S + g, ps + nkv + q.nh)) return -1.f;
  tc_fence_after();
  if (q.fc == 1) {
    uint32_t ph[128];
    q_read_row<D>(q, g, tSg, D == 128 ? 128 : p.fcw, ph);
    const float dl = q_features_to_tile<D, GEN>(p, ph, sPg, r, bh, 0, lam);   // Phi_0 is complete: nothing reads the slices any more
    mbar_arrive(q.bar(R::B_P + g));
    return dl;
  }
  // two chunks: chunk 0 is kept as bf16 pairs in registers until Phi_1 has landed (then the slices are free)
  float dl0 = 0.f, dl1 = 0.f;
  uint32_t pk[64];
  {
    const int part = p.F / p.P;
    const float2* zrow = reinterpret_cast<const float2*>(p.z + (size_t)bh * p.F);
    const uint32_t* brow = (GEN && p.b2) ? reinterpret_cast<const uint32_t*>(p.b2 + (size_t)h * p.F) : nullptr;
#pragma unroll
    for (int cc = 0; cc < 4; ++cc) {
      tmem_ld32(tSg + cc * 32, x);
      tmem_ld_wait(x);
      const int pw = min((cc * 32) / part, p.P - 1);
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        float a0 = __uint_as_float(x[2 * i]), a1 = __uint_as_float(x[2 * i + 1]);
        if (brow != nullptr) {
          const uint32_t bb = __ldg(brow + cc * 16 + i);
          a0 += __uint_as_float(bb << 16);
          a1 += __uint_as_float(bb & 0xffff0000u);
        }
        a0 = fmaxf(a0, 0.f); a1 = fmaxf(a1, 0.f);
        float r0 = a0, r1 = a1;
        if (pw >= 1) { r0 *= a0; r1 *= a1; }
        if (pw >= 2) { r0 *= a0; r1 *= a1; }
        if (pw >= 3) { r0 *= a0; r1 *= a1; }
        const uint32_t wv = pack_bf16(r0 * lam, r1 * lam);
        pk[cc * 16 + i] = wv;
        const float2 zz = __ldg(zrow + cc * 16 + i);
        dl0 = fmaf(__uint_as_float(wv << 16), zz.x, dl0);
        dl1 = fmaf(__uint_as_float(wv & 0xffff0000u), zz.y, dl1);
      }
    }
    tc_fence_before();
    mbar_arrive(q.bar(R::B_SF + g));                 // Phi_1 may overwrite the score columns
  }
  if (!q.wait(R::B_S + g, ps + nkv + q.nh + 1)) return -1.f;     // Phi_1 is there: nothing reads the hidden slices any more
  tc_fence_after();
#pragma unroll
  for (int cc = 0; cc < 4; ++cc) {
    uint32_t wd[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) wd[i] = pk[cc * 16 + i];
    store_row_chunk(sPg, r, cc * 32, wd);
  }
  fence_proxy_async();
  mbar_arrive(q.bar(R::B_P + g));
  uint32_t ph[128];
  q_read_row<D>(q, g, tSg, 128, ph);
  const float dlb = q_features_to_tile<D, GEN>(p, ph, sQg, r, bh, 1, lam);
  mbar_arrive(q.bar(R::B_P + g));
  return (dl0 + dl1) + dlb;
}

// ---------------------------------------------------------------- softmax / merge group, one unit
template <int D, bool TWO, bool GEN>
__device__ __noinline__ bool q_softmax_unit(const QParams& p, const QCtx& c, const CUtensorMap* tmO, uint8_t* smem, int u) {
  using R = QRing<D>;
  using L = QLayout<D>;
  const int nkv = p.nkv, n_s = p.n_s;
  const float scale_log2 = p.scale_log2;
  const R q(p, c);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = warp >> 2;                          // group 0 or 1
  const int r = (warp & 3) * 32 + lane;             // row inside the group's 128-row tile
  const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
  const uint32_t tSg = q.tS(g) + lane_off, tOg = q.tO(g) + lane_off;
  uint8_t* sPg = smem + L::P_OFF + g * L::PTILE;    // this group's P / phi_q / output staging tile
  const int ps = u * q.n_s, ppf = u * q.n_pf;       // first phases of the unit (cf. QRing)
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
    if (!q.wait(R::B_S + g, ps + j)) return false;
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
      if (cc == 0 && !p_buffer_free(ppf + j)) return false;  // the previous tile's P V has read the buffer
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
    float dl;
    dl = 0.f;
    if constexpr (!TWO) {
      for (int ch = 0; ch < q.fc; ++ch) {
        if (!q.wait(R::B_S + g, ps + nkv + ch)) return false;
        tc_fence_after();
        if (!p_buffer_free(ppf + nkv + ch)) return false;   // the last tile's P V / the previous chunk's product has read the P tile
        dl += q_features_from_tmem<D, GEN>(p, tSg, q.bar(R::B_SF + g), sPg, r, bh, ch, lam);   // phi_q takes P's place as the A operand
        mbar_arrive(q.bar(R::B_P + g));
      }
    }
    if constexpr (TWO) {
      uint8_t* sQg = smem + L::Q_OFF + g * L::TILE;    // the group's Q tile: a second buffer once Q is done with
      dl = q_two_layer_tail<D, GEN>(p, q, g, tSg, sPg, sQg, r, bh, ps, ppf, lam);
      if (dl < 0.f) return false;                      // a wait ran out (the sum itself is never negative)
    }
    den = l + dl;
    den_l_out = dl / lam;
  }
  if (!q.wait(R::B_O + g, u)) return false;
  tc_fence_after();
  const float inv = 1.f / den;
  // The output rows are staged in the group's P tile (the product that read it has completed with the O
  // barrier); each warp stores its own 32 rows (rows past N are clipped by the tensor map).
  const int wrow0 = row - lane;
#pragma unroll 1
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

// ---------------------------------------------------------------- layers without softmax tokens (rate 0)
// With no key loop a unit is: Phi = Q W^T, phi_q, O = phi_q S, y = O / (phi_q . z), store.  The tensor pipe has
// little to do and the kernel is bound by how fast the threads turn rows around, so this variant of the kernel runs
// SIXTEEN compute warps: each 128-row group is worked on by two warps per TMEM lane quadrant, each taking one half of
// the columns of a row (features on the way in, output columns on the way out).  Producer and issuing threads are the
// ones of the general kernel; a row's two threads add their shares of phi_q . z through shared memory.
constexpr int QL_THREADS = 608;          // warps 0-15: compute (group = bit 2, quadrant = bits 0-1, column half = bit 3);
                                         // warp 16: TMA; warps 17, 18: MMA issuers

template <int D, bool GEN>
__device__ __noinline__ bool q_linear_unit(const QParams& p, const QCtx& c, const CUtensorMap* tmO, uint8_t* smem, float* sDl, int u) {
  using R = QRing<D>;
  using L = QLayout<D>;
  const R q(p, c);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = (warp >> 2) & 1, quad = warp & 3, hf = warp >> 3;
  const int r = quad * 32 + lane;                   // row inside the group's 128-row tile
  const uint32_t lane_off = (uint32_t)(quad * 32) << 16;
  const uint32_t tSg = q.tS(g) + lane_off, tOg = q.tO(g) + lane_off;
  uint8_t* sPg = smem + L::P_OFF + g * L::PTILE;    // phi_q, then the output rows
  float* dl_slot = sDl + g * 128 + r;
  const int ps = u * q.n_s, ppf = u * q.n_pf;
  const int fcw = D == 128 ? 128 : p.fcw;           // width of a feature chunk; this thread takes columns [hf, hf + 1) * half
  const int half = fcw / 2;
  const QUnit un = q_unit(p, u);
  const int bh = un.w / p.nx, row = un.row0 + g * 128 + r;
  const int part = p.F / p.P;
  uint32_t x[32];
  float dl = 0.f;
  for (int ch = 0; ch < q.fc; ++ch) {
    if (!q.wait(R::B_S + g, ps + ch)) return false;
    tc_fence_after();
    // the P tile may be written once the product that read it has completed and the previous unit's output store
    // has been read out (the stores are issued by the warps of column half 0)
    if (hf == 0 && lane == 0) tma_store_wait_read();
    if (ppf + ch > 0 && !q.wait(R::B_PF + g, ppf + ch - 1)) return false;
    named_barrier_sync(1 + g, 256);
    const float2* zrow = reinterpret_cast<const float2*>(p.z + (size_t)bh * p.F + ch * 128 + hf * half);
    const uint32_t* brow = nullptr;
    if (GEN && p.b2 != nullptr) brow = reinterpret_cast<const uint32_t*>(p.b2 + (size_t)(bh % p.H) * p.F + ch * 128 + hf * half);
    float dl0 = 0.f, dl1 = 0.f;
#pragma unroll
    for (int cc = 0; cc < 2; ++cc) {
      if (cc * 32 < half) {
        const int col = hf * half + cc * 32;
        tmem_ld32(tSg + col, x);
        tmem_ld_wait(x);
        const int pw = min((ch * 128 + col) / part, p.P - 1);
        uint32_t wd[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          float a0 = __uint_as_float(x[2 * i]), a1 = __uint_as_float(x[2 * i + 1]);
          if (GEN && brow != nullptr) {
            const uint32_t bb = __ldg(brow + cc * 16 + i);
            a0 += __uint_as_float(bb << 16);
            a1 += __uint_as_float(bb & 0xffff0000u);
          }
          a0 = fmaxf(a0, 0.f); a1 = fmaxf(a1, 0.f);
          float r0 = a0, r1 = a1;
          if (pw >= 1) { r0 *= a0; r1 *= a1; }
          if (GEN) {
            if (pw >= 2) { r0 *= a0; r1 *= a1; }
            if (pw >= 3) { r0 *= a0; r1 *= a1; }
          }
          wd[i] = pack_bf16(r0, r1);
          const float2 zz = __ldg(zrow + cc * 16 + i);
          dl0 = fmaf(__uint_as_float(wd[i] << 16), zz.x, dl0);
          dl1 = fmaf(__uint_as_float(wd[i] & 0xffff0000u), zz.y, dl1);
        }
        store_row_chunk(sPg, r, col, wd);
      }
    }
    dl += dl0 + dl1;
    tc_fence_before();
    mbar_arrive(q.bar(R::B_SF + g));                 // the next product into the score columns may follow
    fence_proxy_async();
    mbar_arrive(q.bar(R::B_P + g));
  }
  // the row's denominator: both column halves' shares of phi_q . z
  if (hf == 1) *dl_slot = dl;
  named_barrier_sync(1 + g, 256);
  if (hf == 0) dl += *dl_slot;
  named_barrier_sync(1 + g, 256);
  if (hf == 0) *dl_slot = dl;
  if (!q.wait(R::B_O + g, u)) return false;          // (the products run meanwhile)
  named_barrier_sync(1 + g, 256);
  const float den = *dl_slot;
  tc_fence_after();
  const float inv = 1.f / den;
  const int ohalf = D / 2;                           // output columns per thread
#pragma unroll
  for (int cc = 0; cc < 2; ++cc) {
    if (cc * 32 < ohalf) {
      const int col = hf * ohalf + cc * 32;
      tmem_ld32(tOg + col, x);
      tmem_ld_wait(x);
      uint32_t wd[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) wd[i] = pack_bf16(__uint_as_float(x[2 * i]) * inv, __uint_as_float(x[2 * i + 1]) * inv);
      store_row_chunk(sPg, r, col, wd);
    }
  }
  fence_proxy_async();
  tc_fence_before();
  named_barrier_sync(1 + g, 256);                    // both halves of every row are staged
  const int wrow0 = row - lane;
  if (hf == 0 && lane == 0 && wrow0 < p.N) {
#pragma unroll
    for (int b = 0; b < D / 64; ++b)
      tma_store_3d(tmO, smem_u32(sPg) + b * BOX_BYTES + quad * 32 * 128, b * 64, wrow0, bh);
    tma_store_commit();
  }
  if (hf == 0 && p.aux != nullptr && row < p.N) {
    float* ap = p.aux + ((size_t)bh * p.N + row) * 3;
    ap[0] = 0.f; ap[1] = 0.f; ap[2] = den;
  }
  return true;
}

template <int D, bool GEN>
__global__ void __launch_bounds__(QL_THREADS, 1)
qlin_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmW,
            const __grid_constant__ CUtensorMap tmSt, const __grid_constant__ CUtensorMap tmO, const __grid_constant__ QParams p) {
  using L = QLayout<D>;
  using R = QRing<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t sbase = smem_u32(smem);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::BAR_OFF + 8 * R::B_COUNT);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + L::BAR_OFF + 8 * R::B_COUNT + 4);
  auto bar = [&](int i) { return sbase + L::BAR_OFF + 8 * i; };
  const int warp = threadIdx.x >> 5;
  __shared__ float sDl[2 * 128];                     // per group and row: share of phi_q . z, then the denominator

  __shared__ uint32_t s_skip;
  if (threadIdx.x == 0) s_skip = *reinterpret_cast<volatile uint32_t*>(p.status);
  __syncthreads();
  if (s_skip != 0u) return;

  if (threadIdx.x == 0) {
    *abort_flag = 0u;
    mbar_init(bar(R::B_Q0), 1); mbar_init(bar(R::B_Q0 + 1), 1);
    for (int s = 0; s < KV_STAGES; ++s) { mbar_init(bar(R::B_FULL + s), 1); mbar_init(bar(R::B_EMPTY + s), 1); }
    for (int g = 0; g < 2; ++g) {
      mbar_init(bar(R::B_S + g), 1); mbar_init(bar(R::B_SF + g), 256); mbar_init(bar(R::B_P + g), 256);
      mbar_init(bar(R::B_PF + g), 1); mbar_init(bar(R::B_O + g), 1); mbar_init(bar(R::B_QF + g), 1);
      mbar_init(bar(R::B_H + g), 128);
    }
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 17) { tmem_alloc(smem_u32(tmem_slot), 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const QCtx c{sbase, *tmem_slot, WaitCtx{p.status, abort_flag}};
  const int n_mine = q_units_of_cta(p);

  if (warp == 16) {
    if ((threadIdx.x & 31) == 0) { tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmW); tma_prefetch_desc(&tmSt); tma_prefetch_desc(&tmO); }
    for (int u = 0; u < n_mine; ++u)
      if (!q_produce_unit<D, false, GEN>(p, c, &tmQ, &tmQ, &tmQ, &tmW, &tmSt, &tmW, u)) break;
  } else if (warp == 17) {
    if ((threadIdx.x & 31) == 0) {
      for (int u = 0; u < n_mine; ++u)
        if (!q_score_unit<D, false, GEN>(p, c, u)) break;
    }
    __syncwarp();
  } else if (warp == 18) {
    if ((threadIdx.x & 31) == 0) {
      for (int u = 0; u < n_mine; ++u)
        if (!q_accum_unit<D, false, GEN>(p, c, u)) break;
    }
    __syncwarp();
  } else {
    const int g = (warp >> 2) & 1;
    // a unit worked on by one group only (a left-over half) is the CTA's last one: group 1 stops before it
    const int n_grp = (n_mine > p.n_rounds && p.split_last && g == 1) ? p.n_rounds : n_mine;
    for (int u = 0; u < n_grp; ++u)
      if (!q_linear_unit<D, GEN>(p, c, &tmO, smem, sDl, u)) break;
    if ((threadIdx.x & 31) == 0) tma_store_wait_read();
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 17) {
    tc_fence_after();
    tmem_dealloc(c.tmem, 512);
  }
}

template <int D, bool TWO, bool GEN>
__global__ void __launch_bounds__(Q_THREADS, 1)
qpass_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
             const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmW,
             const __grid_constant__ CUtensorMap tmSt, const __grid_constant__ CUtensorMap tmW1,
             const __grid_constant__ CUtensorMap tmO, const __grid_constant__ QParams p) {
  using L = QLayout<D>;
  using R = QRing<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
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
      mbar_init(bar(R::B_H + g), 128 * (p.nh > 0 ? p.nh : 1));   // one arrival per thread and hidden slice
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
      if (!q_produce_unit<D, TWO, GEN>(p, c, &tmQ, &tmK, &tmV, &tmW, &tmSt, &tmW1, u)) break;
  } else if (warp == 9) {
    if ((threadIdx.x & 31) == 0) {
      for (int u = 0; u < n_mine; ++u)
        if (!q_score_unit<D, TWO, GEN>(p, c, u)) break;
    }
    __syncwarp();
  } else if (warp == 10) {
    if ((threadIdx.x & 31) == 0) {
      for (int u = 0; u < n_mine; ++u)
        if (!q_accum_unit<D, TWO, GEN>(p, c, u)) break;
    }
    __syncwarp();
  } else {
    // a unit worked on by one group only (a left-over half) is the CTA's last one: group 1 stops before it
    const int n_grp = (n_mine > p.n_rounds && p.split_last && warp >= 4) ? p.n_rounds : n_mine;
    for (int u = 0; u < n_grp; ++u)
      if (!q_softmax_unit<D, TWO, GEN>(p, c, &tmO, smem, u)) break;
    if ((threadIdx.x & 31) == 0) tma_store_wait_read();  // this warp's output stores have read their rows (the writes land by the end of the kernel)
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
  if ((e = opt_in_smem(qpass_kernel<128, false, false>, QLayout<128>::TOTAL)) != cudaSuccess) return e;
  if ((e = opt_in_smem(qpass_kernel<128, false, true>, QLayout<128>::TOTAL)) != cudaSuccess) return e;
  if ((e = opt_in_smem(qpass_kernel<128, true, false>, QLayout<128>::TOTAL)) != cudaSuccess) return e;
  if ((e = opt_in_smem(qpass_kernel<128, true, true>, QLayout<128>::TOTAL)) != cudaSuccess) return e;
  if ((e = opt_in_smem(qpass_kernel<64, false, false>, QLayout<64>::TOTAL)) != cudaSuccess) return e;
  if ((e = opt_in_smem(qpass_kernel<64, false, true>, QLayout<64>::TOTAL)) != cudaSuccess) return e;
  if ((e = opt_in_smem(qpass_kernel<64, true, false>, QLayout<64>::TOTAL)) != cudaSuccess) return e;
  if ((e = opt_in_smem(qpass_kernel<64, true, true>, QLayout<64>::TOTAL)) != cudaSuccess) return e;
  if ((e = opt_in_smem(qlin_kernel<128, false>, QLayout<128>::TOTAL)) != cudaSuccess) return e;
  if ((e = opt_in_smem(qlin_kernel<128, true>, QLayout<128>::TOTAL)) != cudaSuccess) return e;
  if ((e = opt_in_smem(qlin_kernel<64, false>, QLayout<64>::TOTAL)) != cudaSuccess) return e;
  if ((e = opt_in_smem(qlin_kernel<64, true>, QLayout<64>::TOTAL)) != cudaSuccess) return e;
  return cudaSuccess;
}

cudaError_t as_tensor_qpass(const as_launch_args& a, cudaStream_t st) {
  if (as_tensor_qstream_handles(a)) return as_tensor_qstream(a, st);   // no softmax tokens, the common feature map
  const int BH = a.B * a.H;
  const bool lin = a.n_l > 0;
  CUtensorMap tmQ, tmK, tmV, tmW, tmSt, tmW1, tmO;
  // the output is stored warp by warp: boxes of 32 rows
  if (!make_map(&tmQ, a.q, a.d, a.N, BH, 128) || !make_map(&tmO, a.out, a.d, a.N, BH, 32)) return cudaErrorInvalidValue;
  if (a.n_s > 0) {
    if (!make_map(&tmK, a.ks, a.d, a.n_s, BH, 128) || !make_map(&tmV, a.vs, a.d, a.n_s, BH, 128)) return cudaErrorInvalidValue;
  } else {
    tmK = tmQ; tmV = tmQ;       // never used: the key loop is empty
  }
  const bool two = lin && a.layers == 2;
  if (lin) {
    // boxes are always 128 rows: rows past F (or the hidden width) are out of bounds and arrive as zeros.
    // tmW: last-layer weights [H][F][width of their input]; tmW1: first-layer weights of a two-layer map.
    if (!make_map(&tmW, two ? a.wq2 : a.wq, two ? a.hid : a.d, a.F, a.H, 128) || !make_map(&tmSt, a.Sb, a.d, a.F, BH, 128))
      return cudaErrorInvalidValue;
  } else {
    tmW = tmQ; tmSt = tmQ;      // never used: no linear branch at rate 1
  }
  if (two) { if (!make_map(&tmW1, a.wq, a.d, a.hid, a.H, 128)) return cudaErrorInvalidValue; }
  else tmW1 = tmQ;            // never used with a one-layer map
  QParams p{};
  p.layers = lin ? a.layers : 1;
  p.N = a.N; p.n_s = a.n_s; p.nkv = (a.n_s + 127) / 128; p.lin = lin ? 1 : 0; p.stab_mode = a.stab_mode; p.P = a.P;
  p.H = a.H;
  p.F = a.F; p.fc = (a.F + 127) / 128; p.fcw = a.F < 128 ? a.F : 128;
  p.nh = two ? a.hid / a.d : 0;
  p.b1 = two ? a.bq1 : nullptr;
  p.b2 = two ? a.bq2 : a.bq1;
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
  // the general kernels carry the bias and the powers beyond 2; the common case does without them
  const bool gen = lin && (a.P > 2 || p.b1 != nullptr || p.b2 != nullptr);
  if (p.nkv == 0 && lin && !two) {
    // no softmax tokens, one-layer map: the variant with sixteen compute warps
    if (a.d == 128) {
      if (gen) qlin_kernel<128, true><<<grid, QL_THREADS, QLayout<128>::TOTAL, st>>>(tmQ, tmW, tmSt, tmO, p);
      else qlin_kernel<128, false><<<grid, QL_THREADS, QLayout<128>::TOTAL, st>>>(tmQ, tmW, tmSt, tmO, p);
    } else {
      if (gen) qlin_kernel<64, true><<<grid, QL_THREADS, QLayout<64>::TOTAL, st>>>(tmQ, tmW, tmSt, tmO, p);
      else qlin_kernel<64, false><<<grid, QL_THREADS, QLayout<64>::TOTAL, st>>>(tmQ, tmW, tmSt, tmO, p);
    }
    return cudaGetLastError();
  }
#define AS_LAUNCH_Q(D_, TWO_, GEN_) \
  qpass_kernel<D_, TWO_, GEN_><<<grid, Q_THREADS, QLayout<D_>::TOTAL, st>>>(tmQ, tmK, tmV, tmW, tmSt, tmW1, tmO, p)
  if (a.d == 128) {
    if (two) { if (gen) AS_LAUNCH_Q(128, true, true); else AS_LAUNCH_Q(128, true, false); }
    else { if (gen) AS_LAUNCH_Q(128, false, true); else AS_LAUNCH_Q(128, false, false); }
  } else {
    if (two) { if (gen) AS_LAUNCH_Q(64, true, true); else AS_LAUNCH_Q(64, true, false); }
    else { if (gen) AS_LAUNCH_Q(64, false, true); else AS_LAUNCH_Q(64, false, false); }
  }
#undef AS_LAUNCH_Q
  return cudaGetLastError();
}
