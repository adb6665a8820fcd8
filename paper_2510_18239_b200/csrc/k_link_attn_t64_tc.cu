// Links attend over the history on the 5th-generation tensor cores at d = 256, 64-token tiles (bf16 storage, rows
// LayerNorm-ed already):
//
//   O[T]_h = phi( Q[T]_h K[S]_h^T * scale ) V[S]_h,  K[S] = X W_K,  V[S] = X W_V,  X = LN(S)                (Eq. 3 / Eq. 7)
//
// Same algebra as k_link_attn_tc.cu: W_K is folded into the link queries (Q2, k_link_prep.cu; scores arrive in the log2
// domain) and W_V is applied after the attention, so both contractions run against the stored history rows X, streamed
// once by TMA and used as keys and as values:
//   scores [128 x 64]   = Q2_block [128 x d] . X_tile^T          (one block of 128 stacked (head, link) rows per work item)
//   acc    [128 x d]   += P [128 x 64] . X_tile
// At d = 256 the accumulator takes 256 TMEM columns and a block of folded queries 64 KB of shared memory, which only fits
// with a 64-token tile (32 KB per stage, four stages; three score buffers of 64 columns; two P buffers of 16 KB: all of
// the CTA's shared memory but 1 KB, so the index arrays stay in global memory and are read an item ahead).  The rows
// read must be LayerNorm-ed already (the lookup or the previous layer's history update stores them so); there is no
// on-the-fly LayerNorm in this kernel.  Online softmax in the log2 domain with lazy rescale, or SiLU(s) / N(U) with `silu`
// (Algorithms 1-2).
//
// Persistent CTAs walk (user, chunk) x row-block items - the four CTAs of a group take the same items, one row block
// each, in the order the schedule kernel dealt them so that every group gets the same number of token tiles; warp 0 TMA producer, warp 1 MMA issuer, warps 2-9 softmax.  What
// a softmax warp does for a tile is a chain of waits (scores in TMEM -> TMEM load -> row maximum -> exponentials -> P in
// shared memory -> fence -> signal) whose latency, not its arithmetic, sets the tile period, so the eight warps form TWO
// GROUPS that take alternate tiles: while one group is in the middle of its chain the other starts the next tile's.  A
// group is four warps, ONE thread per stacked row (the row's 64 scores of the tile in registers: no exchange between
// threads for the maximum, and with 320 threads per CTA no register spills - with shared memory configured to its
// maximum a spill is a round trip to L2), and owns the P buffer of its tile parity; tile g's scores sit in buffer g % 3
// and are issued two tiles ahead of its value contraction.  The running
// reference maximum of a row is shared by both groups: the group that handles tile g publishes it (after its own decision
// whether to raise it) and the other group picks it up for tile g + 1; each group keeps the partial row sums of its own
// tiles, relative to the last reference it saw, and the two threads of a row combine them when the item ends.
// Two d = 128 builds of this kernel were measured against k_link_attn_tc.cu (25 us per launch on 256 users x 512 tokens)
// and dropped: 64-token tiles with two CTAs per SM (only two token stages fit per CTA, so the tile period is bound by the
// latency of the copies: 31 us), and 128-token tiles with the two groups of this file (a thread then owns 128 scores of a
// row, taken from TMEM in four pieces twice over: 28 us; 0.90 against 0.72 ms on 32 users x 32768 tokens).
#include "lime_common.cuh"
#include "tc_common.cuh"

namespace lime {

// Geometry: D features per row, XSTAGES token stages.
template <int D_, int XSTAGES_>
struct LbCfg {
  static constexpr int D = D_, TILE = 64, XSTAGES = XSTAGES_;
  static constexpr int GROUPS = 2;                              // softmax groups (alternate tiles), one thread per row in each
  static constexpr int COLS = TILE;                             // token columns per thread: the whole row of the tile
  static constexpr int OUT = D / GROUPS;                        // accumulator columns a thread reads out (the two threads of a row)
  static constexpr int SOFTMAX_WARPS = 4 * GROUPS, GROUP_WARPS = 4, THREADS = 64 + 32 * SOFTMAX_WARPS;
  static constexpr uint32_t XSUB = 64 * 128;                    // [64 tokens x 64 features]
  static constexpr uint32_t X_STAGE = (D / 64) * XSUB;
  static constexpr uint32_t QSUB = 128 * 128;                   // [128 rows x 64 features]
  static constexpr uint32_t Q_BUF = (D / 64) * QSUB;
  static constexpr int PBUFS = 2;                               // one per group
  static constexpr int SBUFS = 3;                               // score buffers in TMEM: tile g uses buffer g % 3
  static constexpr uint32_t P_BUF = 128 * 128;                  // [128 rows x 64 tokens]
  static constexpr uint32_t OFF_X = 0;
  static constexpr uint32_t OFF_Q2 = XSTAGES * X_STAGE;
  static constexpr uint32_t OFF_P = OFF_Q2 + Q_BUF;
  // exchange area (floats): published reference maxima [2 tile parities][128], row sums [GROUPS][128]
  static constexpr uint32_t OFF_EXCH = OFF_P + PBUFS * P_BUF;
  static constexpr uint32_t EXCH_FLOATS = (2 + GROUPS) * 128;
  static constexpr uint32_t OFF_BAR = OFF_EXCH + EXCH_FLOATS * 4;
  static constexpr uint32_t SMEM = OFF_BAR + 256;
  static constexpr uint32_t COL_S = 0, COL_O = 256;             // scores: 3 x 64 columns; accumulator: D columns
  static constexpr uint32_t TMEM_COLS = 512;
  static_assert(OUT % 32 == 0 && COLS == 64 && D <= 256, "column split of a row");
  static_assert(SMEM <= 232448, "shared memory budget of one CTA");
};
constexpr float LB_RESCALE_THRESHOLD = 8.0f;                  // in log2 units

struct LinkAttn64Params {
  const int32_t* off;
  const int32_t* chunk_start;     // [B+1] prefix of per-user chunk counts
  const int32_t* chunk_user;      // [chunk items] user of each (user, chunk) item
  const int32_t* group_start;     // [groups + 1] the items of a group of CTAs (one CTA per row block) are
  const int32_t* group_items;     //              group_items[group_start[j] .. group_start[j + 1])
  int B, chunk, shared, ell, H;
  int silu;
  int HL, RB;                     // stacked (head, link) rows in all, and 128-row blocks of them (one per work item)
  float *part_m, *part_s, *part_acc;   // [items x HL], [items x HL], [items x HL x d]
  __nv_bfloat16* Ohat;                 // [B*ell x H*d]: final rows of single-chunk users
  int* err;
};

__device__ __forceinline__ uint32_t lb_chunk_addr(uint32_t r, uint32_t c) { return r * 128u + ((c ^ (r & 7u)) << 4); }
__device__ __forceinline__ uint32_t lb_pack(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float lb_silu(float x) {
  const float hx = 0.5f * x;
  float th;
  asm("tanh.approx.f32 %0, %1;" : "=f"(th) : "f"(hx));
  return fmaf(hx, th, hx);
}
__device__ __forceinline__ float lb_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ bool lb_group_sync(uint64_t* bar, uint32_t& uses, int lane, int* err, int where) {
  __syncwarp();
  if (lane == 0) tc::mbar_arrive(bar);
  const bool ok = tc::mbar_wait(bar, uses & 1u, err, where);
  ++uses;
  return ok;
}

// p = 2^(s - m_ref) (or SiLU(s)) for this thread's COLS token columns, as bf16 into the A-operand buffer (K-major over
// the tile's tokens, 128-byte swizzle: one K-block of 64 tokens).  Columns past the end of a ragged last tile were set to
// -inf (0 for SiLU) by the caller and give 0.  Returns the sum.
template <bool SILU, int COLS>
__device__ __forceinline__ float lb_probabilities(const float (&v)[COLS], float m_ref, int col0, uint8_t* pbuf, uint32_t r) {
  float ls0 = 0.f, ls1 = 0.f;
#pragma unroll
  for (int c8 = 0; c8 < COLS / 8; ++c8) {
    uint32_t packed[4];
#pragma unroll
    for (int j2 = 0; j2 < 4; ++j2) {
      const int j = c8 * 8 + 2 * j2;
      float e0 = SILU ? lb_silu(v[j]) : lb_ex2(v[j] - m_ref), e1 = SILU ? lb_silu(v[j + 1]) : lb_ex2(v[j + 1] - m_ref);
      ls0 += e0;
      ls1 += e1;
      packed[j2] = lb_pack(e0, e1);
    }
    *reinterpret_cast<uint4*>(pbuf + lb_chunk_addr(r, (uint32_t)(col0 >> 3) + (uint32_t)c8)) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
  }
  return ls0 + ls1;
}

// Walk over the (user, chunk) items of a CTA's group, in the order the schedule dealt them (even token counts across
// the groups).  The index arrays stay in global memory (shared memory is all tiles), so the items and users of the
// next two steps and the token range of the next item are fetched an item ahead.
struct LbItemWalk {
  int pos, end;             // position in group_items of the current item, and of the group's end
  int ci, ci1, ci2;         // (user, chunk) index of the current item, the next, and the one after
  int b0, b1, b2;           // their users (-1: none)
  int tok0, tok1, single;   // token range of the current item; 1 if its user has this chunk only
  int ntok0, ntok1, nsingle;
  const int32_t* items; const int32_t* chunk_user; const int32_t* chunk_start; const int32_t* off;
  int chunk;
  __device__ __forceinline__ void range(int ci_, int b, int& t0, int& t1, int& sg) const {
    const int c0 = __ldg(chunk_start + b), c1 = __ldg(chunk_start + b + 1), o0 = __ldg(off + b), o1 = __ldg(off + b + 1);
    t0 = o0 + (ci_ - c0) * chunk;
    t1 = min(o1, t0 + chunk);
    sg = (c1 - c0 == 1) ? 1 : 0;
  }
  __device__ __forceinline__ void init(const int32_t* it, const int32_t* cu, const int32_t* cs, const int32_t* of, int ch, int first, int last) {
    items = it; chunk_user = cu; chunk_start = cs; off = of; chunk = ch;
    pos = first; end = last;
    ci = pos < end ? __ldg(items + pos) : -1;
    ci1 = pos + 1 < end ? __ldg(items + pos + 1) : -1;
    ci2 = -1;
    b0 = ci >= 0 ? __ldg(chunk_user + ci) : -1;
    b1 = ci1 >= 0 ? __ldg(chunk_user + ci1) : -1;
    b2 = -1;
    tok0 = tok1 = single = ntok0 = ntok1 = nsingle = 0;
    if (b0 >= 0) range(ci, b0, tok0, tok1, single);
    if (b1 >= 0) range(ci1, b1, ntok0, ntok1, nsingle);
  }
  __device__ __forceinline__ bool valid() const { return pos < end; }
  __device__ __forceinline__ void prefetch() {
    ci2 = pos + 2 < end ? __ldg(items + pos + 2) : -1;
    b2 = ci2 >= 0 ? __ldg(chunk_user + ci2) : -1;
  }
  __device__ __forceinline__ void advance() {
    ++pos; ci = ci1; ci1 = ci2; b0 = b1; b1 = b2;
    tok0 = ntok0; tok1 = ntok1; single = nsingle;
    if (b1 >= 0) range(ci1, b1, ntok0, ntok1, nsingle);
  }
};

template <class G>
__global__ void __launch_bounds__(G::THREADS, 1)
k_link_attn_t64_tc(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmQ2, const LinkAttn64Params p) {
  using namespace tc;
  constexpr int D = G::D, TILE = G::TILE, COLS = G::COLS, OUT = G::OUT, XSTAGES = G::XSTAGES, PBUFS = G::PBUFS, SBUFS = G::SBUFS;
  // work items: (user, chunk) x row block.  gridDim % RB == 0: a CTA keeps one row block for its whole life, and the RB
  // CTAs of a group walk the same items, so the history rows they share meet in L2.
  const int grp_first = __ldg(p.group_start + (int)blockIdx.x / p.RB), grp_end = __ldg(p.group_start + (int)blockIdx.x / p.RB + 1);
  if (grp_first >= grp_end) return;
  extern __shared__ __align__(1024) uint8_t smem[];
  if ((smem_u32(smem) & 1023u) != 0) {                     // the swizzled tiles need a 1024-byte aligned base
    if (threadIdx.x == 0) atomicCAS(p.err, 0, 97);
    return;
  }
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + G::OFF_BAR);
  uint64_t* x_full = bars;             // [XSTAGES]
  uint64_t* x_empty = bars + 4;        // [XSTAGES]  second MMA of the tile done
  uint64_t* s_full = bars + 8;         // [SBUFS]  score tile in TMEM
  uint64_t* p_ready = bars + 11;       // [2]  per tile and P buffer: P in smem (the four warps of that buffer's group)
  uint64_t* p_free = bars + 13;        // [2]  per tile and P buffer: second MMA done reading P (and accumulator up to date)
  uint64_t* o_free = bars + 15;        //      accumulator of the item read out (all softmax warps)
  uint64_t* row_bar = bars + 16;       // [4]  rendezvous of the two warps that share a TMEM lane quarter (end of an item)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 20);
  uint64_t* q_full = bars + 21;        //      folded queries of a user landed
  uint64_t* q_empty = bars + 22;       //      every score MMA that reads them has run
  uint64_t* mref_bar = bars + 23;      // [2 tile parities][4 quarters]  reference maxima after the tile published (and the
                                       //                                previous ones read) by the handling group's warp
  static_assert(XSTAGES <= 4 && SBUFS == 3 && PBUFS == 2, "barrier table above");

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < XSTAGES; ++s) { mbar_init(&x_full[s], 1); mbar_init(&x_empty[s], 1); }
    mbar_init(q_full, 1); mbar_init(q_empty, 1);
    for (int i = 0; i < SBUFS; ++i) mbar_init(&s_full[i], 1);
    mbar_init(&p_ready[0], G::GROUP_WARPS); mbar_init(&p_ready[1], G::GROUP_WARPS); mbar_init(&p_free[0], 1); mbar_init(&p_free[1], 1);
    mbar_init(o_free, G::SOFTMAX_WARPS);
    for (int i = 0; i < 4; ++i) mbar_init(&row_bar[i], G::GROUPS);
    for (int i = 0; i < 8; ++i) mbar_init(&mref_bar[i], 1);
    fence_barrier_init();
    prefetch_tmap(&tmX); prefetch_tmap(&tmQ2);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, G::TMEM_COLS); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  constexpr uint32_t COL_S = G::COL_S, COL_O = G::COL_O;

  const int rb = (int)blockIdx.x % p.RB;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      const uint64_t pol_stream = policy_evict_first(), pol_keep = policy_evict_last();
      bool ok = true;
      int g = 0, qn = 0, prev_user = -1;
      LbItemWalk w;
      for (w.init(p.group_items, p.chunk_user, p.chunk_start, p.off, p.chunk, grp_first, grp_end); w.valid() && ok; w.advance()) {
        w.prefetch();
        const int b = w.b0;
        const int tok0 = w.tok0, tok1 = w.tok1;
        const bool load_q = p.shared ? (qn == 0) : (b != prev_user);
        prev_user = b;
        if (load_q) {
          if (!mbar_wait(q_empty, ((uint32_t)qn & 1u) ^ 1u, p.err, 42)) { ok = false; break; }
          mbar_arrive_expect_tx(q_full, G::Q_BUF);
          for (int kb = 0; kb < D / 64; ++kb)
            tma_load_2d_hint(smem + G::OFF_Q2 + kb * G::QSUB, &tmQ2, kb * 64, (p.shared ? 0 : b) * p.HL + rb * 128, q_full, pol_keep);
          ++qn;
        }
        const int n_tiles = (tok1 - tok0 + TILE - 1) / TILE;
        for (int t = 0; t < n_tiles; ++t, ++g) {
          const int s = g % XSTAGES;
          if (!mbar_wait(&x_empty[s], ((uint32_t)(g / XSTAGES) & 1u) ^ 1u, p.err, 41)) { ok = false; break; }
          mbar_arrive_expect_tx(&x_full[s], G::X_STAGE);
          for (int kb = 0; kb < D / 64; ++kb)
            tma_load_2d_hint(smem + G::OFF_X + s * G::X_STAGE + kb * G::XSUB, &tmX, kb * 64, tok0 + t * TILE, &x_full[s], pol_stream);
        }
      }
      if (!ok || *(volatile int*)p.err != 0) {
        // giving up: let the copies already issued land (bounded) before this CTA's shared memory goes away
        for (int j = 0; j < g && j < XSTAGES; ++j)
          mbar_wait_quiet(&x_full[(g - 1 - j) % XSTAGES], (uint32_t)((g - 1 - j) / XSTAGES) & 1u);
        if (qn > 0) mbar_wait_quiet(q_full, (uint32_t)(qn - 1) & 1u);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_s = make_idesc_bf16(128, TILE);               // Q2 . X^T  : both K-major
      constexpr uint32_t idesc_o = make_idesc_bf16(128, D, false, true);     // P . X     : B is MN-major
      const uint32_t sbase = smem_u32(smem);
      auto issue_scores = [&](int g) -> bool {
        const int s = g % XSTAGES;
        if (!mbar_wait(&x_full[s], (uint32_t)(g / XSTAGES) & 1u, p.err, 51)) return false;
        tc_fence_after();
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t oa = (uint32_t)(kk >> 2) * G::QSUB + (uint32_t)(kk & 3) * 32;
          const uint32_t ob = (uint32_t)(kk >> 2) * G::XSUB + (uint32_t)(kk & 3) * 32;
          mma_bf16_ss(tmem_base + COL_S + (uint32_t)(g % SBUFS) * TILE, make_sdesc_k_sw128(sbase + G::OFF_Q2 + oa),
                      make_sdesc_k_sw128(sbase + G::OFF_X + s * G::X_STAGE + ob), idesc_s, kk != 0);
        }
        mma_commit(&s_full[g % SBUFS]);
        return true;
      };
      bool ok = true;
      int g = 0, qn = 0, k = 0, prev_user = -1;
      LbItemWalk w;
      for (w.init(p.group_items, p.chunk_user, p.chunk_start, p.off, p.chunk, grp_first, grp_end); w.valid() && ok; w.advance(), ++k) {
        w.prefetch();
        const int b = w.b0;
        const int tok0 = w.tok0, tok1 = w.tok1;
        const bool load_q = p.shared ? (qn == 0) : (b != prev_user);
        prev_user = b;
        if (load_q) {
          if (!mbar_wait(q_full, (uint32_t)qn & 1u, p.err, 50)) { ok = false; break; }
          ++qn;
        }
        // will the producer replace the queries after this item?
        const bool next_reloads = !p.shared && w.b1 >= 0 && w.b1 != b;
        const int n_tiles = (tok1 - tok0 + TILE - 1) / TILE;
        // The scores run two tiles ahead of the second contraction: while the group of tile g is in its chain, the
        // tensor pipe holds the value contraction of tile g - 1 and the scores of tile g + 1, so it never waits for a
        // chain that has not even started.  Score buffer (g + 2) % 3 was read before p_ready(g - 1).  (Measured and
        // dropped: the next scores issued before the wait for P, two tiles ahead - the fourth token stage then has no slack
        // and the issuer waits for the copy - or one tile ahead - the chain is then exposed again; an L2 prefetch of the
        // tile five tiles ahead did not change either.  In steady state a tile takes 1.18 us of which the tensor pipe is
        // issued to for 0.88 (scores 0.57, values 0.31).  The rest is not the issuing thread: descriptors formed by one
        // add each, a single commit per tile, and the waits taken in the middle of a batch so that MMAs stay queued
        // across them were all measured and left the period unchanged or longer.)
        if (!issue_scores(g)) { ok = false; break; }
        if (n_tiles > 1 && !issue_scores(g + 1)) { ok = false; break; }
        if (n_tiles <= 2 && next_reloads) mma_commit(q_empty);
        for (int t = 0; t < n_tiles; ++t, ++g) {
          const int s = g % XSTAGES;
          if (!mbar_wait(&p_ready[g % PBUFS], (uint32_t)(g / PBUFS) & 1u, p.err, 52)) { ok = false; break; }
          // the first tile of an item overwrites the accumulator: the previous item must have been read out
          if (t == 0 && k > 0 && !mbar_wait(o_free, (uint32_t)(k - 1) & 1u, p.err, 53)) { ok = false; break; }
          tc_fence_after();
          for (int kk = 0; kk < TILE / 16; ++kk)      // contraction over the tile's 64 tokens, 16 per instruction
            mma_bf16_ss(tmem_base + COL_O, make_sdesc_k_sw128(sbase + G::OFF_P + (uint32_t)(g % PBUFS) * G::P_BUF + (uint32_t)kk * 32),
                        make_sdesc_mn_sw128(sbase + G::OFF_X + s * G::X_STAGE + (uint32_t)kk * 2048, G::XSUB), idesc_o, (t | kk) != 0);
          mma_commit(&x_empty[s]);
          mma_commit(&p_free[g % PBUFS]);
          if (t + 2 < n_tiles) {
            if (!issue_scores(g + 2)) { ok = false; break; }
            if (t + 3 == n_tiles && next_reloads) mma_commit(q_empty);
          }
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax warps (2..9), two groups of four
    const int q = warp & 3;                                    // TMEM lane quarter of this warp
    const int grp = (warp - 2) >> 2;                           // handles the tiles with g % 2 == grp
    const uint32_t r = (uint32_t)(q * 32 + lane);              // (head, link) row == TMEM lane; the thread owns the whole row
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
    float* mref = reinterpret_cast<float*>(smem + G::OFF_EXCH);              // [2 tile parities][128]
    float* exch_sum = mref + 2 * 128;                                        // [GROUPS][128]
    const int R = rb * 128 + (int)r;                            // row among all H * ell
    const int64_t ohat_off = (int64_t)(R % p.ell) * (p.H * D) + (R / p.ell) * D + grp * OUT;
    bool ok = true;
    int g = 0, k = 0;
    uint32_t row_uses = 0;
    LbItemWalk w;
    for (w.init(p.group_items, p.chunk_user, p.chunk_start, p.off, p.chunk, grp_first, grp_end); w.valid() && ok; w.advance(), ++k) {
      w.prefetch();
      const int b = w.b0;
      const int tok0 = w.tok0, tok1 = w.tok1;
      const int n_tiles = (tok1 - tok0 + TILE - 1) / TILE;
      // m_own: the reference maximum this thread's row sum is relative to; l_sum: sum over the tiles of this group
      float m_own = -INFINITY, l_sum = 0.f;
      for (int t = 0; t < n_tiles && ok; ++t, ++g) {
        if ((g & 1) != grp) continue;                          // the other group's tile
        const int pb = grp;                                    // P buffer of this group
        const int sb = g % SBUFS;                              // score buffer of the tile
        const int nvalid = min(TILE, tok1 - tok0 - t * TILE);
        if (!mbar_wait(&s_full[sb], (uint32_t)(g / SBUFS) & 1u, p.err, 63)) { ok = false; break; }
        tc_fence_after();
        float v[COLS];
        {
          float v0[32], v1[32];
          tmem_ld_32x32(lane_addr + COL_S + sb * TILE, v0);
          tmem_ld_32x32(lane_addr + COL_S + sb * TILE + 32, v1);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j) { v[j] = v0[j]; v[32 + j] = v1[j]; }
        }
        if (nvalid < TILE) {
          // ragged last tile of the item: the columns past its end (rows of the next user, or the fill value) drop out
          const float dead = p.silu ? 0.f : -INFINITY;
#pragma unroll
          for (int j = 0; j < COLS; ++j)
            if (j >= nvalid) v[j] = dead;
        }
        uint8_t* pbuf = smem + G::OFF_P + pb * G::P_BUF;
        if (p.silu) {
          // SiLU(s) / N(U) needs neither a reference maximum nor row sums: one pass, nothing shared between threads
          if (g >= PBUFS && !mbar_wait(&p_free[pb], (uint32_t)((g - PBUFS) >> 1) & 1u, p.err, 65)) { ok = false; break; }
          lb_probabilities<true, COLS>(v, 0.f, 0, pbuf, r);
          tc_fence_before();
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) mbar_arrive(&p_ready[pb]);
          continue;
        }
        // four independent chains for the row maximum (a ragged tile's dead columns hold -inf)
        float mx0 = v[0], mx1 = v[1], mx2 = v[2], mx3 = v[3];
#pragma unroll
        for (int j = 4; j < COLS; j += 4) {
          mx0 = fmaxf(mx0, v[j]); mx1 = fmaxf(mx1, v[j + 1]); mx2 = fmaxf(mx2, v[j + 2]); mx3 = fmaxf(mx3, v[j + 3]);
        }
        const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
        // the reference the other group left after the previous tile (every tile but the very first waits, whether or
        // not it uses the value: the two groups then never drift more than one tile apart)
        float m_prev = -INFINITY;
        if (g > 0) {
          if (!mbar_wait(&mref_bar[((g - 1) & 1) * 4 + q], (uint32_t)((g - 1) >> 1) & 1u, p.err, 69)) { ok = false; break; }
          if (t > 0) m_prev = mref[((g - 1) & 1) * 128 + r];
        }
        if (m_prev != m_own && l_sum != 0.f) l_sum *= lb_ex2(m_own - m_prev);       // bring this group's sum up to date
        // raise the reference maximum only when it is exceeded by more than the threshold (or unset)
        const bool need = mx > m_prev + LB_RESCALE_THRESHOLD;
        const float m_new = need ? mx : m_prev;
        const float factor = (need && m_prev != -INFINITY) ? lb_ex2(m_prev - m_new) : 1.0f;
        mref[(g & 1) * 128 + r] = m_new;
        __syncwarp();
        if (lane == 0) mbar_arrive(&mref_bar[(g & 1) * 4 + q]);
        if (__any_sync(0xffffffffu, need && t > 0)) {
          // the accumulator must be quiescent: wait for the previous tile's second MMA, then scale the row
          if (!mbar_wait(&p_free[(g - 1) & 1], (uint32_t)((g - 1) >> 1) & 1u, p.err, 64)) { ok = false; break; }
          tc_fence_after();
#pragma unroll 1
          for (int c = 0; c < D; c += 32) {
            float a[32];
            tmem_ld_32x32(lane_addr + COL_O + c, a);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 32; ++j) a[j] *= factor;
            tmem_st_32x32(lane_addr + COL_O + c, a);
          }
          tmem_wait_st();
        }
        l_sum *= factor;
        m_own = m_new;

        // the P that last sat in this group's buffer must have been consumed
        if (g >= PBUFS && !mbar_wait(&p_free[pb], (uint32_t)((g - PBUFS) >> 1) & 1u, p.err, 65)) { ok = false; break; }
        l_sum += lb_probabilities<false, COLS>(v, m_own, 0, pbuf, r);
        tc_fence_before();
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_ready[pb]);
      }
      if (!ok) break;
      // item result: the final reference (published with the last tile), the two partial sums, then the accumulator
      const int gl = g - 1;
      if (!p.silu) {
        if ((gl & 1) != grp) {
          if (!mbar_wait(&mref_bar[(gl & 1) * 4 + q], (uint32_t)(gl >> 1) & 1u, p.err, 70)) { ok = false; break; }
          const float m_fin = mref[(gl & 1) * 128 + r];
          if (m_fin != m_own && l_sum != 0.f) l_sum *= lb_ex2(m_own - m_fin);
          m_own = m_fin;
        }
        exch_sum[grp * 128 + r] = l_sum;
      }
      if (!lb_group_sync(&row_bar[q], row_uses, lane, p.err, 68)) { ok = false; break; }
      float l_tot;
      if (!p.silu) l_tot = exch_sum[r] + exch_sum[128 + r];
      else l_tot = (float)(tok1 - tok0);   // SiLU mode normalises by the number of keys (Algorithm 1): this chunk's tokens, summed over the chunks by the merge
      if (!mbar_wait(&p_free[gl & 1], (uint32_t)(gl >> 1) & 1u, p.err, 66)) { ok = false; break; }
      tc_fence_after();
      const bool single = w.single != 0;
      const float inv = 1.0f / l_tot;
      __nv_bfloat16* dst_o = p.Ohat + (int64_t)b * p.ell * (p.H * D) + ohat_off;
      float* dst_p = p.part_acc + ((int64_t)w.ci * p.HL + R) * D + grp * OUT;
#pragma unroll 1
      for (int c = 0; c < OUT; c += 32) {
        float a[32];
        tmem_ld_32x32(lane_addr + COL_O + grp * OUT + c, a);
        tmem_wait_ld();
        if (single) {
          // the whole history of this user was one chunk: normalise and write the attention row directly
#pragma unroll
          for (int j = 0; j < 32; j += 8) {
            uint4 o;
            o.x = lb_pack(a[j] * inv, a[j + 1] * inv); o.y = lb_pack(a[j + 2] * inv, a[j + 3] * inv);
            o.z = lb_pack(a[j + 4] * inv, a[j + 5] * inv); o.w = lb_pack(a[j + 6] * inv, a[j + 7] * inv);
            *reinterpret_cast<uint4*>(dst_o + c + j) = o;
          }
        } else {
#pragma unroll
          for (int j = 0; j < 32; j += 4) *reinterpret_cast<float4*>(dst_p + c + j) = make_float4(a[j], a[j + 1], a[j + 2], a[j + 3]);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(o_free);
      if (!single && grp == 0) {
        const int64_t prow = (int64_t)w.ci * p.HL + R;
        p.part_m[prow] = p.silu ? 0.f : m_own;        // log2 domain; equal weights for the chunks in SiLU mode
        p.part_s[prow] = l_tot;
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, G::TMEM_COLS);
  }
}

using LbD256 = LbCfg<256, 4>;             // d = 256, four token stages

bool link_attn_d256_tc_supported(int dtype, int d, int H, int ell, int phi) {
  return dtype == LIME_BF16 && d == 256 && (H * ell) % 128 == 0 && H * ell <= 512 && ell % 4 == 0 &&
         (phi == LIME_PHI_SOFTMAX || phi == LIME_PHI_SILU);
}

int link_attn_d256_groups(int n_chunk_upper, int H, int ell) {
  const int RB = H * ell / 128;
  if (RB < 1) return 0;
  const int grid = n_chunk_upper * RB < kSMs ? n_chunk_upper * RB : kSMs;
  return grid / RB;
}

template <class G>
static lime_status launch_link_attn_t64(const LinkAttnArgs& a, cudaStream_t st, const char* name, bool (&smem_set)[kMaxDeviceOrdinals]) {
  if (a.n_chunk_upper <= 0 || a.total == 0) return LIME_OK;   // no history: the merge step writes zeros
  if (a.ln) return LIME_INVALID_ARG;                           // rows must arrive LayerNorm-ed
  CUtensorMap tmX, tmQ2;
  const uint64_t users = a.shared ? 1 : (uint64_t)a.B;
  if (!make_tmap_bf16_sw128(&tmX, a.hist, (uint64_t)a.total, G::D, G::D, G::TILE) ||
      !make_tmap_bf16_sw128(&tmQ2, a.Q2, users * (uint64_t)(a.H * a.ell), G::D, G::D, 128))
    return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
  if (a.group_start == nullptr || a.group_items == nullptr) return LIME_INVALID_ARG;
  LinkAttn64Params p;
  p.group_start = a.group_start; p.group_items = a.group_items;
  p.off = a.off; p.chunk_start = a.chunk_start; p.chunk_user = a.chunk_user; p.silu = a.silu; p.B = a.B; p.chunk = a.chunk; p.shared = a.shared;
  p.ell = a.ell; p.H = a.H; p.HL = a.H * a.ell; p.RB = p.HL / 128; p.part_m = a.part_m; p.part_s = a.part_s; p.part_acc = a.part_acc;
  p.Ohat = (__nv_bfloat16*)a.Ohat; p.err = a.err;
  const int grid = link_attn_d256_groups(a.n_chunk_upper, a.H, a.ell) * p.RB;
  if (a.n_groups * p.RB != grid) return LIME_INVALID_ARG;      // the schedule was dealt for another grid
  lime_status es = ensure_dynamic_smem((const void*)k_link_attn_t64_tc<G>, (int)G::SMEM, smem_set);
  if (es != LIME_OK) return es;
  ProfScope _p(name, st);
  k_link_attn_t64_tc<G><<<grid, G::THREADS, G::SMEM, st>>>(tmX, tmQ2, p);
  LIME_LAUNCH_CHECK(name);
  return LIME_OK;
}

lime_status launch_link_attn_d256_tc(const LinkAttnArgs& a, cudaStream_t st) {
  static bool smem_set[kMaxDeviceOrdinals] = {};
  return launch_link_attn_t64<LbD256>(a, st, "k_link_attn_d256_tc", smem_set);
}

}  // namespace lime
