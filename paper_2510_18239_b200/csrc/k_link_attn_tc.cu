// Links attend over the history on the 5th-generation tensor cores (bf16 storage):
//
//   O[T]_h = softmax_j( Q[T]_h K[S]_h^T * scale ) V[S]_h,  K[S] = LN(S) W_K,  V[S] = LN(S) W_V          (Eq. 3 / Eq. 7)
//
// With W_K folded into the link queries (Q2, see k_link_prep.cu; the fold also carries scale * log2(e), so scores
// arrive in the log2 domain) and W_V applied after the attention, both contractions run against the *stored*
// history rows X, which are streamed exactly once (TMA) and used both as keys and as values - K[S] and V[S] are
// never materialised:
//   scores [HL x 128]   = Q2 [HL x d] . X_tile^T            LayerNorm folded in afterwards:
//                         s_ij = rstd_j * (raw_ij - mu_j * rowsum(Q2)_i)
//   acc    [HL x d]    += P' [HL x 128] . X_tile            P'_ij = p_ij * rstd_j;  the mean term sum_j P'_ij mu_j is
//                                                           a per-row scalar subtracted from every column at the end
//   O[T]_{l,h} = (acc_(h,l) / sum) . W_V[:, head h]         (W_V is folded into the GEMM that follows)
// The H * ell stacked (head, link) rows are processed in blocks of 128 = the TMEM lanes (one block per work item; a
// second block of the same tokens finds them in L2).  Online softmax whose reference maximum is only raised
// when the true maximum exceeds it by more than 8 (then the accumulator row is rescaled in TMEM), so most tiles need
// no correction pass.  With LN = false the rows of X are LayerNorm-ed already and the corrections vanish.
// With `silu` set the activation is SiLU(s) / N(U) (Algorithms 1-2): one pass per tile, no maximum, no row sums; the
// divisor is the number of keys, and per-chunk partials are summed with equal weights.
// Shared memory: three token stages, the folded queries of the current user, two P' buffers (the second MMA of a
// tile runs while the next tile's P' is written).
//
// Persistent CTAs walk (user, chunk-of-history) items.  Warp roles: warp 0 TMA producer (runs ahead across items),
// warp 1 MMA issuer, warps 2-17 softmax: four threads per (head, link) row, each owning 32 of the tile's 128 token
// columns (a warp may only touch the TMEM lane quarter warp_id % 4, so the four parts of a row sit in warps w,
// w + 4, w + 8, w + 12 and exchange their row maximum through shared memory).  Four warps per scheduler keep the
// issue slots busy while TMEM loads and exponentials are in flight.  A user whose history is a single chunk is
// normalised and written directly; longer histories leave (max, sum, accumulator) partials per chunk that
// k_link_attn_merge_norm combines.
//
// Built for d = 128 and H * ell a multiple of 128.
#include "lime_common.cuh"
#include "tc_common.cuh"

namespace lime {

constexpr int LA_D = 128, LA_TILE = 128, LA_XSTAGES = 3;
constexpr int LA_PARTS = 4;                                   // threads per row
constexpr int LA_COLS = LA_TILE / LA_PARTS;                   // token columns per thread
constexpr int LA_SOFTMAX_WARPS = 4 * LA_PARTS, LA_THREADS = 64 + 32 * LA_SOFTMAX_WARPS;
constexpr uint32_t LA_SUB = 128 * 128;
constexpr uint32_t LA_X_STAGE = 2 * LA_SUB;
constexpr uint32_t LA_OFF_X = 0;
constexpr uint32_t LA_OFF_Q2 = LA_XSTAGES * LA_X_STAGE;
constexpr uint32_t LA_Q2_BUF = 2 * LA_SUB;                    // folded queries of one user's row block
constexpr int LA_Q2_BUFS = 1;                                // buffers of them (a user's queries are replaced after its last
                                                             // score MMA, a tile before the item ends)
constexpr int LA_PBUFS = 2;                                  // buffers of P': the second MMA of a tile runs while the
constexpr uint32_t LA_P_BUF = 2 * LA_SUB;                    // softmax warps already write the next tile's P'
constexpr uint32_t LA_OFF_P = LA_OFF_Q2 + LA_Q2_BUFS * LA_Q2_BUF;   // P' [128 rows x 128 tokens] x LA_PBUFS
constexpr uint32_t LA_OFF_STATS = LA_OFF_P + LA_PBUFS * LA_P_BUF;   // per X stage: float2 {rstd, mu} x 128 tokens
constexpr uint32_t LA_OFF_EXCH = LA_OFF_STATS + LA_XSTAGES * 128 * 8;   // [2 tile parities][PARTS][128] maxima, then
                                                                        // [PARTS][128] sums and [PARTS][128] mean terms
constexpr uint32_t LA_OFF_BAR = LA_OFF_EXCH + 4 * LA_PARTS * 128 * 4;
constexpr int LA_IDX_CAP = 1025;                             // users + 1 whose offsets are staged in shared memory
constexpr uint32_t LA_OFF_IDX = LA_OFF_BAR + 256;            // chunk_start[0..B], off[0..B] (a search over them per work item
                                                             // costs a chain of dependent reads: microseconds from global memory)
constexpr uint32_t LA_SMEM = LA_OFF_IDX + 2 * LA_IDX_CAP * 4 + 8;
constexpr float LA_RESCALE_THRESHOLD = 8.0f;                 // in log2 units

struct LinkAttnParams {
  const float* cQ;                // [users x HL]
  const int32_t* off;
  const int32_t* chunk_start;     // [B+1] prefix of per-user chunk counts
  const int32_t* chunk_user;      // [chunk items] user of each (user, chunk) item
  int B, chunk, shared, ell, H;
  int silu;                       // attention activation: 0 softmax (online, log2 domain), 1 SiLU(s) / N(U) (Algorithm 2)
  int HL, RB;                     // stacked (head, link) rows in all, and 128-row blocks of them (one per work item)
  float ln_eps;
  float *part_m, *part_s, *part_acc;   // [items x HL], [items x HL], [items x HL x d]
  __nv_bfloat16* Ohat;                 // [B*ell x H*d]: final rows of single-chunk users
  float2* stats_out;                   // nullable: {rstd, mean} per history row (written by the CTAs of row block 0)
  int* err;
};

__device__ __forceinline__ uint32_t la_chunk_addr(uint32_t r, uint32_t c) { return r * 128u + ((c ^ (r & 7u)) << 4); }
__device__ __forceinline__ uint32_t la_pack(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
// SiLU(x) = x * sigmoid(x) = x/2 * (1 + tanh(x/2)): one SFU operation
__device__ __forceinline__ float la_silu(float x) {
  const float hx = 0.5f * x;
  float th;
  asm("tanh.approx.f32 %0, %1;" : "=f"(th) : "f"(hx));
  return fmaf(hx, th, hx);
}
__device__ __forceinline__ float la_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Rendezvous of the warps that arrive on `bar` (every wait in this kernel is bounded, so no bar.sync): shared-memory
// writes made by any lane before the call are visible to every participant after it.
__device__ __forceinline__ bool la_group_sync(uint64_t* bar, uint32_t& uses, int lane, int* err, int where) {
  __syncwarp();
  if (lane == 0) tc::mbar_arrive(bar);
  const bool ok = tc::mbar_wait(bar, uses & 1u, err, where);
  ++uses;
  return ok;
}

// Pass 1 over this thread's LA_COLS scores: LayerNorm correction (LN) and the maximum over the valid columns.
template <bool LN, bool MASK>
__device__ __forceinline__ float la_pass1(float (&v)[LA_COLS], const float2* __restrict__ st, float cq, int col0, int nvalid) {
  float mx = -INFINITY;
#pragma unroll
  for (int j = 0; j < LA_COLS; ++j) {
    if (LN) {
      const float2 c2 = st[col0 + j];
      v[j] = (v[j] - cq * c2.y) * c2.x;
    }
    if (!MASK || col0 + j < nvalid) mx = fmaxf(mx, v[j]);
  }
  return mx;
}

// Pass 2: p = 2^(s - m_ref) (softmax) or SiLU(s) (SILU: no reference maximum, no row sum), P' = p * rstd as bf16 into
// the A-operand buffer (K-major over the tile's tokens, 128-byte swizzle); returns the sums of p and of P' * mu
// through l_sum / mean_corr.
template <bool LN, bool MASK, bool SILU>
__device__ __forceinline__ void la_pass2(const float (&v)[LA_COLS], const float2* __restrict__ st, float m_ref, int col0, int nvalid,
                                         uint8_t* prow_base, uint32_t r, uint32_t chunk0, float& l_sum, float& mean_corr) {
  float ls0 = 0.f, ls1 = 0.f, mc0 = 0.f, mc1 = 0.f;
#pragma unroll
  for (int c8 = 0; c8 < LA_COLS / 8; ++c8) {
    uint32_t packed[4];
#pragma unroll
    for (int j2 = 0; j2 < 4; ++j2) {
      const int j = c8 * 8 + 2 * j2;
      float e0 = SILU ? la_silu(v[j]) : la_ex2(v[j] - m_ref), e1 = SILU ? la_silu(v[j + 1]) : la_ex2(v[j + 1] - m_ref);
      if (MASK) {
        if (col0 + j >= nvalid) e0 = 0.f;
        if (col0 + j + 1 >= nvalid) e1 = 0.f;
      }
      ls0 += e0;
      ls1 += e1;
      if (LN) {
        const float2 a = st[col0 + j], b = st[col0 + j + 1];
        // what the MMA will see is the bf16-rounded P'; use the same rounded values for the mean term
        const uint32_t pk = la_pack(e0 * a.x, e1 * b.x);
        mc0 = fmaf(__uint_as_float(pk << 16), a.y, mc0);
        mc1 = fmaf(__uint_as_float(pk & 0xffff0000u), b.y, mc1);
        packed[j2] = pk;
      } else {
        packed[j2] = la_pack(e0, e1);
      }
    }
    *reinterpret_cast<uint4*>(prow_base + la_chunk_addr(r, chunk0 + (uint32_t)c8)) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
  }
  l_sum += ls0 + ls1;
  mean_corr += mc0 + mc1;
}

// Walk over this CTA's work items.  The user of an item comes from the chunk_user table, read two items ahead, and the
// token range from the offset tables staged in shared memory: the code between two items is executed once per item by
// every role, so it is kept to a few instructions with no dependent chain of global reads.
struct ItemWalk {
  int ci, stride, n_ci;     // (user, chunk) index of the current item, its step, and the number of such items
  int b0, b1, b2;           // users of the current item, the next, and the one after (-1: none)
  __device__ __forceinline__ void init(const int32_t* __restrict__ chunk_user, int first, int step, int n) {
    ci = first; stride = step; n_ci = n;
    b0 = ci < n ? __ldg(chunk_user + ci) : -1;
    b1 = ci + step < n ? __ldg(chunk_user + ci + step) : -1;
    b2 = -1;
  }
  __device__ __forceinline__ bool valid() const { return ci < n_ci; }
  __device__ __forceinline__ void prefetch(const int32_t* __restrict__ chunk_user) {
    b2 = ci + 2 * stride < n_ci ? __ldg(chunk_user + ci + 2 * stride) : -1;
  }
  __device__ __forceinline__ void advance() { ci += stride; b0 = b1; b1 = b2; }
};

template <bool LN>
__global__ void __launch_bounds__(LA_THREADS, 1)
k_link_attn_tc(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmQ2, const LinkAttnParams p) {
  using namespace tc;
  extern __shared__ __align__(1024) uint8_t smem[];
  if ((smem_u32(smem) & 1023u) != 0) {
    if (threadIdx.x == 0) atomicCAS(p.err, 0, 91);
    return;
  }
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + LA_OFF_BAR);
  uint64_t* x_full = bars;             // [LA_XSTAGES]
  uint64_t* x_empty = bars + 4;        // [LA_XSTAGES]  second MMA of the tile done
  uint64_t* q_full = bars + 22;        // [2]  folded queries of a user landed in buffer i
  uint64_t* q_empty = bars + 24;       // [2]  every score MMA that reads buffer i has run
  uint64_t* s_full = bars + 8;         // [2]  score tile in TMEM
  uint64_t* p_ready = bars + 10;       // [2]  per tile and P' buffer: P' in smem (all softmax warps)
  uint64_t* p_free = bars + 12;        // [2]  per tile and P' buffer: second MMA done reading P' (and accumulator up to date)
  uint64_t* o_free = bars + 14;        //      accumulator of the item read out (all softmax warps)
  uint64_t* stats_bar = bars + 15;     //      rendezvous of the softmax warps (token statistics written)
  uint64_t* row_bar = bars + 16;       // [4]  rendezvous of the warps that share a TMEM lane quarter
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 20);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < LA_XSTAGES; ++s) { mbar_init(&x_full[s], 1); mbar_init(&x_empty[s], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&q_full[i], 1); mbar_init(&q_empty[i], 1); }
    for (int i = 0; i < 2; ++i) mbar_init(&s_full[i], 1);
    mbar_init(&p_ready[0], LA_SOFTMAX_WARPS); mbar_init(&p_ready[1], LA_SOFTMAX_WARPS); mbar_init(&p_free[0], 1); mbar_init(&p_free[1], 1);
    mbar_init(o_free, LA_SOFTMAX_WARPS);
    mbar_init(stats_bar, LA_SOFTMAX_WARPS);
    for (int i = 0; i < 4; ++i) mbar_init(&row_bar[i], LA_PARTS);
    fence_barrier_init();
    prefetch_tmap(&tmX); prefetch_tmap(&tmQ2);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // set-up done: the next kernel's CTAs may become resident; nothing an earlier kernel wrote is read before this wait
  pdl_launch_dependents();
  pdl_wait();
  // work items: (user, chunk) x row block; gridDim % RB == 0, so a CTA keeps one row block for its whole life
  const int n_items = p.chunk_start[p.B] * p.RB;
  const bool active = (int)blockIdx.x < n_items;           // a CTA without items goes straight to the end
  const int32_t* chunk_start = p.chunk_start;
  const int32_t* off = p.off;
  if (p.B + 1 <= LA_IDX_CAP) {
    int32_t* idx = reinterpret_cast<int32_t*>(smem + LA_OFF_IDX);
    for (int i = threadIdx.x; i <= p.B; i += LA_THREADS) { idx[i] = p.chunk_start[i]; idx[LA_IDX_CAP + i] = p.off[i]; }
    chunk_start = idx;
    off = idx + LA_IDX_CAP;
    __syncthreads();
  }
  constexpr uint32_t COL_S = 0, COL_O = 256;      // scores: 2 x 128 columns; accumulator: d columns

  // item -> token range; identical in every role
  const int rb = (int)blockIdx.x % p.RB;
  const int ci_first = (int)blockIdx.x / p.RB, ci_step = (int)gridDim.x / p.RB, n_ci = n_items / p.RB;
  auto item_range = [&](int ci, int b, int& tok0, int& tok1) {
    tok0 = off[b] + (ci - chunk_start[b]) * p.chunk;
    tok1 = min(off[b + 1], tok0 + p.chunk);
  };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0 && active) {
      const uint64_t pol_stream = policy_evict_first(), pol_keep = policy_evict_last();
      bool ok = true;
      int g = 0, qn = 0, prev_user = -1;
      ItemWalk w;
      for (w.init(p.chunk_user, ci_first, ci_step, n_ci); w.valid() && ok; w.advance()) {
        w.prefetch(p.chunk_user);
        const int b = w.b0;
        int tok0, tok1;
        item_range(w.ci, b, tok0, tok1);
        const bool load_q = p.shared ? (qn == 0) : (b != prev_user);
        prev_user = b;
        if (load_q) {
          const int qb = qn % LA_Q2_BUFS;
          if (!mbar_wait(&q_empty[qb], ((uint32_t)(qn / LA_Q2_BUFS) & 1u) ^ 1u, p.err, 42)) { ok = false; break; }
          mbar_arrive_expect_tx(&q_full[qb], LA_Q2_BUF);
          for (int kb = 0; kb < 2; ++kb)
            tma_load_2d_hint(smem + LA_OFF_Q2 + qb * LA_Q2_BUF + kb * LA_SUB, &tmQ2, kb * 64, (p.shared ? 0 : b) * p.HL + rb * 128,
                             &q_full[qb], pol_keep);
          ++qn;
        }
        const int n_tiles = (tok1 - tok0 + LA_TILE - 1) / LA_TILE;
        for (int t = 0; t < n_tiles; ++t, ++g) {
          const int s = g % LA_XSTAGES;
          if (!mbar_wait(&x_empty[s], ((uint32_t)(g / LA_XSTAGES) & 1u) ^ 1u, p.err, 41)) { ok = false; break; }
          mbar_arrive_expect_tx(&x_full[s], LA_X_STAGE);
          for (int kb = 0; kb < 2; ++kb)
            tma_load_2d_hint(smem + LA_OFF_X + s * LA_X_STAGE + kb * LA_SUB, &tmX, kb * 64, tok0 + t * LA_TILE, &x_full[s],
                             pol_stream);
        }
      }
      if (!ok || *(volatile int*)p.err != 0) {
        // giving up: let the copies already issued land (bounded) before this CTA's shared memory goes away
        for (int j = 0; j < g && j < LA_XSTAGES; ++j)
          mbar_wait_quiet(&x_full[(g - 1 - j) % LA_XSTAGES], (uint32_t)((g - 1 - j) / LA_XSTAGES) & 1u);
        for (int j = 0; j < qn && j < LA_Q2_BUFS; ++j)
          mbar_wait_quiet(&q_full[(qn - 1 - j) % LA_Q2_BUFS], (uint32_t)((qn - 1 - j) / LA_Q2_BUFS) & 1u);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && active) {
      constexpr uint32_t idesc_s = make_idesc_bf16(128, 128);                 // Q2 . X^T  : both K-major
      constexpr uint32_t idesc_o = make_idesc_bf16(128, 128, false, true);    // P' . X    : B is MN-major
      const uint32_t sbase = smem_u32(smem);
      uint32_t q2_off = LA_OFF_Q2;                 // buffer of the current user's folded queries
      auto issue_scores = [&](int g) -> bool {
        const int s = g % LA_XSTAGES;
        if (!mbar_wait(&x_full[s], (uint32_t)(g / LA_XSTAGES) & 1u, p.err, 51)) return false;
        tc_fence_after();
        for (int kk = 0; kk < 8; ++kk) {
          const uint32_t o = (uint32_t)(kk >> 2) * LA_SUB + (uint32_t)(kk & 3) * 32;
          mma_bf16_ss(tmem_base + COL_S + (uint32_t)(g & 1) * 128, make_sdesc_k_sw128(sbase + q2_off + o),
                      make_sdesc_k_sw128(sbase + LA_OFF_X + s * LA_X_STAGE + o), idesc_s, kk != 0);
        }
        mma_commit(&s_full[g & 1]);
        return true;
      };
      bool ok = true;
      int g = 0, qn = 0, k = 0, prev_user = -1;
      ItemWalk w;
      for (w.init(p.chunk_user, ci_first, ci_step, n_ci); w.valid() && ok; w.advance(), ++k) {
        w.prefetch(p.chunk_user);
        const int b = w.b0;
        int tok0, tok1;
        item_range(w.ci, b, tok0, tok1);
        const bool load_q = p.shared ? (qn == 0) : (b != prev_user);
        prev_user = b;
        if (load_q) {
          if (!mbar_wait(&q_full[qn % LA_Q2_BUFS], (uint32_t)(qn / LA_Q2_BUFS) & 1u, p.err, 50)) { ok = false; break; }
          q2_off = LA_OFF_Q2 + (uint32_t)(qn % LA_Q2_BUFS) * LA_Q2_BUF;
          ++qn;
        }
        // will the producer replace the queries after this item?
        const bool next_reloads = !p.shared && w.b1 >= 0 && w.b1 != b;
        const int n_tiles = (tok1 - tok0 + LA_TILE - 1) / LA_TILE;
        if (!issue_scores(g)) { ok = false; break; }
        if (n_tiles == 1 && next_reloads) mma_commit(&q_empty[(qn - 1) % LA_Q2_BUFS]);
        for (int t = 0; t < n_tiles; ++t, ++g) {
          // the next tile's scores overlap this tile's softmax (its score buffer was read before p_ready(g-1))
          if (t + 1 < n_tiles) {
            if (!issue_scores(g + 1)) { ok = false; break; }
            if (t + 2 == n_tiles && next_reloads) mma_commit(&q_empty[(qn - 1) % LA_Q2_BUFS]);
          }
          const int s = g % LA_XSTAGES;
          if (!mbar_wait(&p_ready[g % LA_PBUFS], (uint32_t)(g / LA_PBUFS) & 1u, p.err, 52)) { ok = false; break; }
          // the first tile of an item overwrites the accumulator: the previous item must have been read out
          if (t == 0 && k > 0 && !mbar_wait(o_free, (uint32_t)(k - 1) & 1u, p.err, 53)) { ok = false; break; }
          tc_fence_after();
          for (int kk = 0; kk < 8; ++kk) {      // contraction over the tile's 128 tokens, 16 per instruction
            const uint32_t oa = (uint32_t)(kk >> 2) * LA_SUB + (uint32_t)(kk & 3) * 32;
            mma_bf16_ss(tmem_base + COL_O, make_sdesc_k_sw128(sbase + LA_OFF_P + (uint32_t)(g % LA_PBUFS) * LA_P_BUF + oa),
                        make_sdesc_mn_sw128(sbase + LA_OFF_X + s * LA_X_STAGE + (uint32_t)kk * 2048, LA_SUB), idesc_o,
                        (t | kk) != 0);
          }
          mma_commit(&x_empty[s]);
          mma_commit(&p_free[g % LA_PBUFS]);
        }
      }
    }
  } else if (active) {
    // ------------------------------------------------------------------ softmax warps (2..17)
    const int sw = warp - 2;                                   // 0..15
    const int q = warp & 3;                                    // TMEM lane quarter of this warp
    const int part = sw >> 2;                                  // which LA_COLS token columns of the tile
    const int col0 = part * LA_COLS;
    const uint32_t r = (uint32_t)(q * 32 + lane);              // (head, link) row == TMEM lane
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
    float2* stats = reinterpret_cast<float2*>(smem + LA_OFF_STATS);
    float* exch_max = reinterpret_cast<float*>(smem + LA_OFF_EXCH);          // [2 tile parities][PARTS][128]
    float* exch_sum = exch_max + 2 * LA_PARTS * 128;                         // [PARTS][128]
    float* exch_mean = exch_sum + LA_PARTS * 128;                            // [PARTS][128]
    // where this thread's part of its (head, link) row goes: fixed for the life of the CTA
    const int R = rb * 128 + (int)r;                            // row among all H * ell
    // final rows are stored after a 4 x 4 transpose of 16-byte chunks inside each group of four lanes: lane 4j+i then
    // holds chunk i of rows 4j..4j+3, so every store instruction writes whole 64-byte row parts.  Four consecutive
    // rows share a head (ell is a multiple of 4), so they are H * d elements apart.
    const int R4 = rb * 128 + q * 32 + (lane & ~3);
    const int64_t ohat_off = (int64_t)(R4 % p.ell) * (p.H * LA_D) + (R4 / p.ell) * LA_D + col0 + (lane & 3) * 8;
    bool ok = true;
    int g = 0, k = 0;
    uint32_t stats_uses = 0, row_uses = 0;
    ItemWalk w;
    for (w.init(p.chunk_user, ci_first, ci_step, n_ci); w.valid() && ok; w.advance(), ++k) {
      w.prefetch(p.chunk_user);
      const int b = w.b0;
      int tok0, tok1;
      item_range(w.ci, b, tok0, tok1);
      const int n_tiles = (tok1 - tok0 + LA_TILE - 1) / LA_TILE;
      const float cq = LN ? p.cQ[(int64_t)(p.shared ? 0 : b) * p.HL + rb * 128 + r] : 0.f;
      float m_ref = -INFINITY, l_sum = 0.f, mean_corr = 0.f;
      for (int t = 0; t < n_tiles && ok; ++t, ++g) {
        const int s = g % LA_XSTAGES, pb = g & 1;
        const int nvalid = min(LA_TILE, tok1 - tok0 - t * LA_TILE);
        const float2* st = stats + s * 128;
        if (LN) {
          // LayerNorm statistics of the tile's tokens: four lanes per token, 32 features each, held in registers
          if (!mbar_wait(&x_full[s], (uint32_t)(g / LA_XSTAGES) & 1u, p.err, 61)) { ok = false; break; }
          const int tok = 8 * sw + (lane >> 2), p4 = lane & 3;
          const uint8_t* xs = smem + LA_OFF_X + s * LA_X_STAGE + (p4 >> 1) * LA_SUB + tok * 128;
          uint4 u[4];
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const int ch = (p4 & 1) * 4 + ((c + (p4 >> 1)) & 3);             // this lane's 4 chunks, rotated start
            u[c] = *reinterpret_cast<const uint4*>(xs + ((ch ^ (tok & 7)) << 4));
          }
          float sum = 0.f;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const uint32_t w[4] = {u[c].x, u[c].y, u[c].z, u[c].w};
#pragma unroll
            for (int j = 0; j < 4; ++j) sum += __uint_as_float(w[j] << 16) + __uint_as_float(w[j] & 0xffff0000u);
          }
          sum += __shfl_xor_sync(0xffffffffu, sum, 1);
          sum += __shfl_xor_sync(0xffffffffu, sum, 2);
          const float mu = sum * (1.0f / LA_D);
          float var = 0.f;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const uint32_t w[4] = {u[c].x, u[c].y, u[c].z, u[c].w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float a = __uint_as_float(w[j] << 16) - mu, bb = __uint_as_float(w[j] & 0xffff0000u) - mu;
              var = fmaf(a, a, var);
              var = fmaf(bb, bb, var);
            }
          }
          var += __shfl_xor_sync(0xffffffffu, var, 1);
          var += __shfl_xor_sync(0xffffffffu, var, 2);
          if (p4 == 0) {
            const float2 rm = make_float2(rsqrtf(var * (1.0f / LA_D) + p.ln_eps), mu);
            stats[s * 128 + tok] = rm;
            if (p.stats_out != nullptr && rb == 0 && tok < nvalid) p.stats_out[tok0 + t * LA_TILE + tok] = rm;
          }
          if (!la_group_sync(stats_bar, stats_uses, lane, p.err, 62)) { ok = false; break; }
        }
        if (!mbar_wait(&s_full[pb], (uint32_t)(g >> 1) & 1u, p.err, 63)) { ok = false; break; }
        tc_fence_after();

        // pass 1: this thread's scores (log2 domain) into registers, and their maximum
        float v[LA_COLS];
        tmem_ld_32x32(lane_addr + COL_S + pb * 128 + col0, v);
        tmem_wait_ld();
        float mx = nvalid == LA_TILE ? la_pass1<LN, false>(v, st, cq, col0, nvalid) : la_pass1<LN, true>(v, st, cq, col0, nvalid);
        if (p.silu) {
          // SiLU(s) / N(U) needs neither a reference maximum nor row sums: one pass, no exchange between the row's threads
          if (g >= LA_PBUFS && !mbar_wait(&p_free[g % LA_PBUFS], (uint32_t)((g - LA_PBUFS) / LA_PBUFS) & 1u, p.err, 65)) { ok = false; break; }
          uint8_t* pbuf = smem + LA_OFF_P + (g % LA_PBUFS) * LA_P_BUF + (col0 >> 6) * LA_SUB;
          const uint32_t chunk0 = (uint32_t)(col0 & 63) >> 3;
          if (nvalid == LA_TILE) la_pass2<LN, false, true>(v, st, 0.f, col0, nvalid, pbuf, r, chunk0, l_sum, mean_corr);
          else la_pass2<LN, true, true>(v, st, 0.f, col0, nvalid, pbuf, r, chunk0, l_sum, mean_corr);
          tc_fence_before();
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) mbar_arrive(&p_ready[g % LA_PBUFS]);
          continue;
        }
        exch_max[(pb * LA_PARTS + part) * 128 + r] = mx;
        if (!la_group_sync(&row_bar[q], row_uses, lane, p.err, 67)) { ok = false; break; }
#pragma unroll
        for (int i = 1; i < LA_PARTS; ++i) mx = fmaxf(mx, exch_max[(pb * LA_PARTS + ((part + i) & (LA_PARTS - 1))) * 128 + r]);

        // raise the reference maximum only when it is exceeded by more than the threshold (or unset)
        const bool need = mx > m_ref + LA_RESCALE_THRESHOLD;
        const float m_new = need ? mx : m_ref;
        const float factor = (need && m_ref != -INFINITY) ? la_ex2(m_ref - m_new) : 1.0f;
        if (__any_sync(0xffffffffu, need && t > 0)) {
          // the accumulator must be quiescent: wait for the previous tile's second MMA, then scale this part of the row
          if (!mbar_wait(&p_free[(g - 1) % LA_PBUFS], (uint32_t)((g - 1) / LA_PBUFS) & 1u, p.err, 64)) { ok = false; break; }
          tc_fence_after();
          float a[LA_COLS];
          tmem_ld_32x32(lane_addr + COL_O + col0, a);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < LA_COLS; ++j) a[j] *= factor;
          tmem_st_32x32(lane_addr + COL_O + col0, a);
          tmem_wait_st();
        }
        l_sum *= factor;
        mean_corr *= factor;
        m_ref = m_new;

        // the P' that last sat in this buffer must have been consumed
        if (g >= LA_PBUFS && !mbar_wait(&p_free[g % LA_PBUFS], (uint32_t)((g - LA_PBUFS) / LA_PBUFS) & 1u, p.err, 65)) { ok = false; break; }
        // pass 2: P' -> smem; K index = token column, so columns col0.. live in K-block col0 / 64, chunk (col0 % 64) / 8..
        uint8_t* pbuf = smem + LA_OFF_P + (g % LA_PBUFS) * LA_P_BUF + (col0 >> 6) * LA_SUB;
        const uint32_t chunk0 = (uint32_t)(col0 & 63) >> 3;
        if (nvalid == LA_TILE) la_pass2<LN, false, false>(v, st, m_ref, col0, nvalid, pbuf, r, chunk0, l_sum, mean_corr);
        else la_pass2<LN, true, false>(v, st, m_ref, col0, nvalid, pbuf, r, chunk0, l_sum, mean_corr);
        tc_fence_before();
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_ready[g % LA_PBUFS]);
      }
      if (!ok) break;
      // item result: wait for the last second MMA, combine the parts' sums, read this part of the accumulator row
      const int gl = g - 1;
      if (!mbar_wait(&p_free[gl % LA_PBUFS], (uint32_t)(gl / LA_PBUFS) & 1u, p.err, 66)) { ok = false; break; }
      tc_fence_after();
      exch_sum[part * 128 + r] = l_sum;
      exch_mean[part * 128 + r] = mean_corr;
      if (!la_group_sync(&row_bar[q], row_uses, lane, p.err, 68)) { ok = false; break; }
      float l_tot = 0.f, c_tot = 0.f;
#pragma unroll
      for (int i = 0; i < LA_PARTS; ++i) { l_tot += exch_sum[i * 128 + r]; c_tot += exch_mean[i * 128 + r]; }
      // SiLU mode normalises by the number of keys (Algorithm 1): this chunk's tokens, summed over the chunks by the merge
      if (p.silu) l_tot = (float)(tok1 - tok0);
      float a[LA_COLS];
      tmem_ld_32x32(lane_addr + COL_O + col0, a);
      tmem_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(o_free);
      const bool single = chunk_start[b + 1] - chunk_start[b] == 1;
      const int64_t prow = (int64_t)w.ci * p.HL + R;            // row of the per-chunk partials
      // 4 x 4 transpose of 16-byte chunks inside each group of four lanes (two butterfly steps of warp shuffles)
      auto xchg = [&](uint4& keep_lo, uint4& keep_hi, bool upper, int dist) {
        // lanes with `upper` clear give away keep_hi and receive into it; lanes with it set give away keep_lo
        uint4 send = upper ? keep_lo : keep_hi, recv;
        recv.x = __shfl_xor_sync(0xffffffffu, send.x, dist); recv.y = __shfl_xor_sync(0xffffffffu, send.y, dist);
        recv.z = __shfl_xor_sync(0xffffffffu, send.z, dist); recv.w = __shfl_xor_sync(0xffffffffu, send.w, dist);
        if (upper) keep_lo = recv; else keep_hi = recv;
      };
      auto transpose4 = [&](uint4 (&t)[4]) {
        xchg(t[0], t[1], (lane & 1) != 0, 1);
        xchg(t[2], t[3], (lane & 1) != 0, 1);
        xchg(t[0], t[2], (lane & 2) != 0, 2);
        xchg(t[1], t[3], (lane & 2) != 0, 2);
      };
      if (single) {
        // the whole history of this user was one chunk: normalise and write the attention rows directly
        const float inv = 1.0f / l_tot;
        static_assert(LA_COLS == 32, "the chunk transpose below moves four 16-byte chunks per thread");
        uint4 tch[4];
#pragma unroll
        for (int c8 = 0; c8 < 4; ++c8) {
          tch[c8].x = la_pack((a[c8 * 8 + 0] - c_tot) * inv, (a[c8 * 8 + 1] - c_tot) * inv);
          tch[c8].y = la_pack((a[c8 * 8 + 2] - c_tot) * inv, (a[c8 * 8 + 3] - c_tot) * inv);
          tch[c8].z = la_pack((a[c8 * 8 + 4] - c_tot) * inv, (a[c8 * 8 + 5] - c_tot) * inv);
          tch[c8].w = la_pack((a[c8 * 8 + 6] - c_tot) * inv, (a[c8 * 8 + 7] - c_tot) * inv);
        }
        transpose4(tch);
        __nv_bfloat16* dst = p.Ohat + (int64_t)b * p.ell * (p.H * LA_D) + ohat_off;
#pragma unroll
        for (int m = 0; m < 4; ++m) *reinterpret_cast<uint4*>(dst + (int64_t)m * (p.H * LA_D)) = tch[m];
      } else {
        // fp32 partial accumulator: this thread's 32 columns are two runs of four 16-byte chunks; after the transposes
        // lane 4j+i holds chunk i of rows 4j..4j+3, so a store instruction writes whole 64-byte pieces of rows
        float* dst = p.part_acc + ((int64_t)w.ci * p.HL + R4) * LA_D + col0 + (lane & 3) * 4;
#pragma unroll
        for (int run = 0; run < 2; ++run) {
          uint4 t[4];
#pragma unroll
          for (int c4 = 0; c4 < 4; ++c4) {
            const int j = run * 16 + c4 * 4;
            t[c4] = make_uint4(__float_as_uint(a[j] - c_tot), __float_as_uint(a[j + 1] - c_tot), __float_as_uint(a[j + 2] - c_tot),
                               __float_as_uint(a[j + 3] - c_tot));
          }
          transpose4(t);
#pragma unroll
          for (int m = 0; m < 4; ++m) *reinterpret_cast<uint4*>(dst + (int64_t)m * LA_D + run * 16) = t[m];
        }
        if (part == 0) {
          p.part_m[prow] = p.silu ? 0.f : m_ref;        // log2 domain; equal weights for the chunks in SiLU mode
          p.part_s[prow] = l_tot;
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

bool link_attn_tc_supported(int dtype, int d, int H, int ell, int phi) {
  return dtype == LIME_BF16 && d == LA_D && (H * ell) % 128 == 0 && H * ell <= 512 &&
         (phi == LIME_PHI_SOFTMAX || phi == LIME_PHI_SILU);
}

lime_status launch_link_attn_tc(const LinkAttnArgs& a, cudaStream_t st) {
  if (a.n_chunk_upper <= 0 || a.total == 0) return LIME_OK;   // no history: the merge step writes zeros
  CUtensorMap tmX, tmQ2;
  const uint64_t users = a.shared ? 1 : (uint64_t)a.B;
  if (!make_tmap_bf16_sw128(&tmX, a.hist, (uint64_t)a.total, LA_D, LA_D, LA_TILE) ||
      !make_tmap_bf16_sw128(&tmQ2, a.Q2, users * (uint64_t)(a.H * a.ell), LA_D, LA_D, 128))
    return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
  LinkAttnParams p;
  p.cQ = a.cQ; p.off = a.off; p.chunk_start = a.chunk_start; p.chunk_user = a.chunk_user; p.silu = a.silu; p.B = a.B; p.chunk = a.chunk; p.shared = a.shared;
  p.ell = a.ell; p.H = a.H; p.HL = a.H * a.ell; p.RB = p.HL / 128; p.ln_eps = a.ln_eps; p.part_m = a.part_m; p.part_s = a.part_s; p.part_acc = a.part_acc;
  p.Ohat = (__nv_bfloat16*)a.Ohat; p.stats_out = a.ln ? a.stats_out : nullptr; p.err = a.err;
  int grid = a.n_chunk_upper * p.RB < kSMs ? a.n_chunk_upper * p.RB : kSMs;
  grid -= grid % p.RB;                              // a CTA's work items then all share its row block
  static bool smem_ln[kMaxDeviceOrdinals] = {}, smem_plain[kMaxDeviceOrdinals] = {};
  lime_status es = a.ln ? ensure_dynamic_smem((const void*)k_link_attn_tc<true>, (int)LA_SMEM, smem_ln)
                        : ensure_dynamic_smem((const void*)k_link_attn_tc<false>, (int)LA_SMEM, smem_plain);
  if (es != LIME_OK) return es;
  ProfScope _p("k_link_attn_tc", st);
  if (a.ln) launch_pdl(k_link_attn_tc<true>, dim3(grid), dim3(LA_THREADS), LA_SMEM, st, tmX, tmQ2, p);
  else launch_pdl(k_link_attn_tc<false>, dim3(grid), dim3(LA_THREADS), LA_SMEM, st, tmX, tmQ2, p);
  LIME_LAUNCH_CHECK("k_link_attn_tc");
  return LIME_OK;
}

}  // namespace lime
