// History update of one XOR layer on tcgen05 for more stacked (head, link) rows than one SM can keep resident
// (H * ell = 256 .. 512 at d = d_ff = 128, e.g. 4 heads x 64 links):
//
//   S'[t,:] = GatedMLP( O[S]_t ),   O[S]_t = concat_h softmax_l( Q[S]_{t,h} K[T]_{l,h}^T * scale ) V[T]_{l,h}     (Eq. 7, Eq. 5)
//
// Same chain of contractions per 128-token tile as k_hist_update_tc.cu (scores -> per-head softmax -> [gate | up] ->
// SiLU(gate) * up -> W_o), but the folded link-side operands K2 [HL x d] and [G2 | U2] [2f x HL] (k_link_prep.cu) no
// longer fit in shared memory next to the token tile.  The (head, link) rows are therefore walked in groups of 128:
//   for each group c:  scores_c = X . K2_c^T  ->  softmax per head  ->  [gate | up] += P_c . [G2 | U2]_c
// with K2_c (32 KB) and [G2 | U2]_c (64 KB) streamed from L2 into one buffer each, per tile and group (they are
// per-user data of a few hundred KB that every tile of the user re-reads: L2 traffic, not HBM traffic).  K2_{c+1}
// arrives while group c is in its softmax, [G2 | U2]_{c+1} while group c+1 is.
//
// Warp 0 TMA producer, warp 1 MMA issuer, warps 2-9 token rows: two threads per token (TMEM lane), 64 columns each -
// whole heads of the softmax (ell in {32, 64}).  TMEM: 128 columns of scores, 256 [gate | up], 128 S'.
// With `out_ln` the rows are written LayerNorm-ed for the next layer (see k_hist_update_tc.cu).
#include "lime_common.cuh"
#include "tc_common.cuh"

namespace lime {

constexpr int H2_D = 128, H2_F = 128, H2_TILE = 128;
constexpr int H2_ROW_WARPS = 8, H2_THREADS = 64 + 32 * H2_ROW_WARPS;
constexpr uint32_t H2_SUB = 128 * 128;                  // bytes of one [128 rows x 64 bf16] swizzled sub-tile
constexpr uint32_t H2_OFF_X = 0;                        // token tile: 2 K-blocks
constexpr uint32_t H2_OFF_K2 = 2 * H2_SUB;              // K2_c [128 x d]: 2 K-blocks
constexpr uint32_t H2_OFF_GU = H2_OFF_K2 + 2 * H2_SUB;  // [G2 | U2]_c [2f x 128]: 2 K-blocks x 32 KB (gate rows, then up rows)
constexpr uint32_t H2_OFF_WO = H2_OFF_GU + 4 * H2_SUB;  // [d x f]: 2 K-blocks
constexpr uint32_t H2_OFF_PU = H2_OFF_WO + 2 * H2_SUB;  // P_c, then U: 2 K-blocks
constexpr uint32_t H2_OFF_STATS = H2_OFF_PU + 2 * H2_SUB;    // 2 (tile parity) x 128 float2 {rstd, mu}
constexpr uint32_t H2_OFF_EXCH = H2_OFF_STATS + 2 * 128 * 8; // pair exchange: [2 tile parities][2 halves][128] float2 {mean, M2}
constexpr uint32_t H2_OFF_CK = H2_OFF_EXCH + 4 * 128 * 8;    // the current user's HL key row sums (up to 512 floats)
constexpr uint32_t H2_OFF_BAR = H2_OFF_CK + 512 * 4;
constexpr int H2_IDX_CAP = 1025;                            // users + 1 whose offsets are staged in shared memory (the
constexpr uint32_t H2_OFF_IDX = H2_OFF_BAR + 256;           // search for a tile's user is a chain of dependent reads:
constexpr uint32_t H2_SMEM = H2_OFF_IDX + 2 * H2_IDX_CAP * 4 + 8;   // microseconds from global memory)
static_assert(H2_SMEM <= 232448, "shared memory budget of one CTA");

struct HistUpdate2Params {
  __nv_bfloat16* out;            // [total x d]
  const float* cK;               // [users x HL] row sums of K2
  const int32_t* off;            // [B+1]
  const int32_t* tile_start;     // [B+1] prefix of per-user tile counts (tile = 128 tokens)
  int B, HL, NG, shared, out_ln; // NG = HL / 128 groups
  int silu;                      // 1: P = SiLU(scores) / ell (Algorithm 2) instead of the per-head softmax
  float ln_eps;
  int* err;
};

__device__ __forceinline__ uint32_t h2_chunk(uint32_t r, uint32_t c) { return r * 128u + ((c ^ (r & 7u)) << 4); }
__device__ __forceinline__ uint32_t h2_pack(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float h2_tanh(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float h2_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ bool h2_group_sync(uint64_t* bar, uint32_t& uses, int lane, int* err, int where) {
  __syncwarp();
  if (lane == 0) tc::mbar_arrive(bar);
  const bool ok = tc::mbar_wait(bar, uses & 1u, err, where);
  ++uses;
  return ok;
}
struct H2TileUser {
  int b = -1, lo = 0, hi = 0;
  __device__ __forceinline__ int of(const int32_t* __restrict__ tile_start, int B, int t) {
    if (t < lo || t >= hi) {
      // the user is a neighbour of the cached one: step through tile_start (staged in shared memory), no search
      if (b < 0) b = upper_user(tile_start, B, t);
      else if (t >= hi) { do { ++b; } while (tile_start[b + 1] <= t); }
      else { do { --b; } while (tile_start[b] > t); }
      lo = tile_start[b];
      hi = tile_start[b + 1];
    }
    return b;
  }
};

template <int ELL, bool LN>
__global__ void __launch_bounds__(H2_THREADS, 1)
k_hist_update2_tc(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmK2,
                  const __grid_constant__ CUtensorMap tmG, const __grid_constant__ CUtensorMap tmU,
                  const __grid_constant__ CUtensorMap tmWo, const HistUpdate2Params p) {
  using namespace tc;
  static_assert(64 % ELL == 0, "a thread owns whole heads");
  extern __shared__ __align__(1024) uint8_t smem[];
  if ((smem_u32(smem) & 1023u) != 0) {
    if (threadIdx.x == 0) atomicCAS(p.err, 0, 94);
    return;
  }
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + H2_OFF_BAR);
  uint64_t* x_full = bars;           // per tile
  uint64_t* x_empty = bars + 1;      // per tile: last scores MMA done (1) + statistics taken (8 warps)
  uint64_t* k2_full = bars + 2;      // per (tile, group)
  uint64_t* k2_empty = bars + 3;     // per (tile, group): scores MMA done
  uint64_t* ops_full = bars + 4;     // per (tile, group): [G2 | U2]_c landed
  uint64_t* ops_empty = bars + 5;    // per (tile, group): mix MMA done (producer's view)
  uint64_t* wo_full = bars + 6;
  uint64_t* s2_full = bars + 20;     // [2] per (tile, group), by parity of the group counter: scores in TMEM
  uint64_t* p_ready = bars + 8;      // per (tile, group): P_c in smem (8 warps)
  uint64_t* p_free = bars + 9;       // per (tile, group): mix MMA done (row warps' view)
  uint64_t* gu_full = bars + 10;     // per tile: [gate | up] complete
  uint64_t* u_ready = bars + 11;     // per tile: U in smem (8 warps)
  uint64_t* sp_full = bars + 12;     // per tile: S' in TMEM (and U read)
  uint64_t* sp_free = bars + 13;     // per tile: S' read out (8 warps)
  uint64_t* stats_bar = bars + 14;   // rendezvous of the 8 row warps
  uint64_t* pair_bar = bars + 15;    // [4] rendezvous of the two warps sharing a TMEM lane quarter
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 19);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int NG = p.NG;

  if (threadIdx.x == 0) {
    mbar_init(x_full, 1); mbar_init(x_empty, 1 + H2_ROW_WARPS);
    mbar_init(k2_full, 1); mbar_init(k2_empty, 1); mbar_init(ops_full, 1); mbar_init(ops_empty, 1); mbar_init(wo_full, 1);
    mbar_init(&s2_full[0], 1); mbar_init(&s2_full[1], 1); mbar_init(p_ready, H2_ROW_WARPS); mbar_init(p_free, 1); mbar_init(gu_full, 1);
    mbar_init(u_ready, H2_ROW_WARPS); mbar_init(sp_full, 1); mbar_init(sp_free, H2_ROW_WARPS); mbar_init(stats_bar, H2_ROW_WARPS);
    for (int i = 0; i < 4; ++i) mbar_init(&pair_bar[i], 2);
    fence_barrier_init();
    prefetch_tmap(&tmX); prefetch_tmap(&tmK2); prefetch_tmap(&tmG); prefetch_tmap(&tmU); prefetch_tmap(&tmWo);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // set-up done: the next kernel's CTAs may become resident; nothing an earlier kernel wrote is read before this wait
  pdl_launch_dependents();
  pdl_wait();
  const int n_tiles_all = p.tile_start[p.B];
  const int t_begin = (int)(((int64_t)blockIdx.x * n_tiles_all) / gridDim.x);
  const int t_end = (int)(((int64_t)(blockIdx.x + 1) * n_tiles_all) / gridDim.x);
  const int n = t_end - t_begin;
  const int32_t* tile_start = p.tile_start;
  const int32_t* off = p.off;
  if (p.B + 1 <= H2_IDX_CAP) {
    int32_t* idx = reinterpret_cast<int32_t*>(smem + H2_OFF_IDX);
    for (int i = threadIdx.x; i <= p.B; i += H2_THREADS) { idx[i] = p.tile_start[i]; idx[H2_IDX_CAP + i] = p.off[i]; }
    tile_start = idx;
    off = idx + H2_IDX_CAP;
    __syncthreads();
  }
  // Two 128-column buffers take the scores of the groups and S' in rotation: use u of this CTA (per tile NG score uses,
  // then S') goes to buffer u & 1, so the scores of the next group are formed while the row warps still read this one's.
  constexpr uint32_t COL_A = 0, COL_GU = 128, COL_B = 384;
  auto col_of = [&](int u) -> uint32_t { return (u & 1) ? COL_B : COL_A; };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0 && n > 0) {
      const uint64_t pol_stream = policy_evict_first(), pol_keep = policy_evict_last();
      mbar_arrive_expect_tx(wo_full, 2 * H2_SUB);
      for (int kb = 0; kb < 2; ++kb) tma_load_2d_hint(smem + H2_OFF_WO + kb * H2_SUB, &tmWo, kb * 64, 0, wo_full, pol_keep);
      bool ok = true;
      int g = 0, q = 0;
      H2TileUser tu;
      for (; g < n && ok; ++g) {
        const int t = t_begin + g;
        const int b = tu.of(tile_start, p.B, t);
        const int urow = p.shared ? 0 : b;
        if (g > 0 && !mbar_wait(x_empty, (uint32_t)(g - 1) & 1u, p.err, 12)) { ok = false; break; }
        const int row0 = off[b] + (t - tu.lo) * H2_TILE;
        mbar_arrive_expect_tx(x_full, 2 * H2_SUB);
        for (int kb = 0; kb < 2; ++kb) tma_load_2d_hint(smem + H2_OFF_X + kb * H2_SUB, &tmX, kb * 64, row0, x_full, pol_stream);
        for (int c = 0; c < NG; ++c, ++q) {
          if (q > 0 && !mbar_wait(k2_empty, (uint32_t)(q - 1) & 1u, p.err, 11)) { ok = false; break; }
          mbar_arrive_expect_tx(k2_full, 2 * H2_SUB);
          for (int kb = 0; kb < 2; ++kb)
            tma_load_2d_hint(smem + H2_OFF_K2 + kb * H2_SUB, &tmK2, kb * 64, urow * p.HL + c * 128, k2_full, pol_keep);
          if (q > 0 && !mbar_wait(ops_empty, (uint32_t)(q - 1) & 1u, p.err, 13)) { ok = false; break; }
          mbar_arrive_expect_tx(ops_full, 4 * H2_SUB);
          for (int kb = 0; kb < 2; ++kb) {
            // contraction index = (head, link) rows of group c: columns c * 128 + kb * 64 .. of the transposed operands
            tma_load_2d_hint(smem + H2_OFF_GU + kb * 2 * H2_SUB, &tmG, c * 128 + kb * 64, urow * H2_F, ops_full, pol_keep);
            tma_load_2d_hint(smem + H2_OFF_GU + kb * 2 * H2_SUB + H2_SUB, &tmU, c * 128 + kb * 64, urow * H2_F, ops_full, pol_keep);
          }
        }
      }
      if (!ok || *(volatile int*)p.err != 0) {
        // giving up: let the copies already issued land (bounded) before this CTA's shared memory goes away
        if (g > 0 || q > 0) mbar_wait_quiet(x_full, (uint32_t)(g < n ? g : n - 1) & 1u);
        if (q > 0) { mbar_wait_quiet(k2_full, (uint32_t)(q - 1) & 1u); mbar_wait_quiet(ops_full, (uint32_t)(q - 1) & 1u); }
        mbar_wait_quiet(wo_full, 0);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && n > 0) {
      constexpr uint32_t idesc_128 = make_idesc_bf16(128, 128);
      constexpr uint32_t idesc_256 = make_idesc_bf16(128, 256);
      const uint32_t sbase = smem_u32(smem);
      const uint32_t pu = sbase + H2_OFF_PU;
      bool ok = mbar_wait(wo_full, 0, p.err, 21);
      int q = 0;
      // scores of group qq (tile-local use index u): X . K2_c^T
      auto issue_scores = [&](int qq, int u, bool last_of_tile) -> bool {
        if (!mbar_wait(k2_full, (uint32_t)qq & 1u, p.err, 22)) return false;
        tc_fence_after();
        for (int kk = 0; kk < 8; ++kk) {
          const uint32_t o = (uint32_t)(kk >> 2) * H2_SUB + (uint32_t)(kk & 3) * 32;
          mma_bf16_ss(tmem_base + col_of(u), make_sdesc_k_sw128(sbase + H2_OFF_X + o), make_sdesc_k_sw128(sbase + H2_OFF_K2 + o),
                      idesc_128, kk != 0);
        }
        mma_commit(&s2_full[qq & 1]);
        mma_commit(k2_empty);
        if (last_of_tile) mma_commit(x_empty);
        return true;
      };
      for (int g = 0; g < n && ok; ++g) {
        if (!mbar_wait(x_full, (uint32_t)g & 1u, p.err, 23)) break;
        const int u0 = g * (NG + 1);
        // 1. scores of the first group (its buffer last held the scores of the previous tile's last group: consumed)
        if (!issue_scores(q, u0, NG == 1)) { ok = false; break; }
        for (int c = 0; c < NG && ok; ++c, ++q) {
          if (c + 1 < NG) {
            // 1'. scores of the next group, under this group's softmax; for c = 0 the buffer last held S' of the previous tile
            if (c == 0 && g > 0 && !mbar_wait(sp_free, (uint32_t)(g - 1) & 1u, p.err, 26)) { ok = false; break; }
            if (!issue_scores(q + 1, u0 + c + 1, c + 1 == NG - 1)) { ok = false; break; }
          }
          // 3. [gate | up] (+)= P_c . [G2 | U2]_c
          if (!mbar_wait(ops_full, (uint32_t)q & 1u, p.err, 27)) { ok = false; break; }
          if (!mbar_wait(p_ready, (uint32_t)q & 1u, p.err, 24)) { ok = false; break; }
          tc_fence_after();
          for (int kk = 0; kk < 8; ++kk) {
            const uint32_t oa = (uint32_t)(kk >> 2) * H2_SUB + (uint32_t)(kk & 3) * 32;
            const uint32_t ob = (uint32_t)(kk >> 2) * 2 * H2_SUB + (uint32_t)(kk & 3) * 32;
            mma_bf16_ss(tmem_base + COL_GU, make_sdesc_k_sw128(pu + oa), make_sdesc_k_sw128(sbase + H2_OFF_GU + ob), idesc_256,
                        (c | kk) != 0);
          }
          mma_commit(ops_empty);
          mma_commit(p_free);
          if (c == NG - 1) mma_commit(gu_full);
        }
        if (!ok) break;
        // 5. S'(g) = U(g) . W_o, into the buffer after the last group's (with one group that one last held S'(g-1))
        if (!mbar_wait(u_ready, (uint32_t)g & 1u, p.err, 25)) break;
        if (NG == 1 && g > 0 && !mbar_wait(sp_free, (uint32_t)(g - 1) & 1u, p.err, 26)) break;
        tc_fence_after();
        for (int kk = 0; kk < 8; ++kk) {
          const uint32_t o = (uint32_t)(kk >> 2) * H2_SUB + (uint32_t)(kk & 3) * 32;
          mma_bf16_ss(tmem_base + col_of(u0 + NG), make_sdesc_k_sw128(pu + o), make_sdesc_k_sw128(sbase + H2_OFF_WO + o), idesc_128,
                      kk != 0);
        }
        mma_commit(sp_full);
      }
    }
  } else if (n > 0) {
    // ------------------------------------------------------------------ token-row warps (2..9)
    const int rw = warp - 2;                                 // 0..7
    const int q4 = warp & 3;                                 // TMEM lane quarter of this warp
    const int half = rw >> 2;                                // which 64 columns of every step
    const uint32_t r = (uint32_t)(q4 * 32 + lane);           // token row of the tile == TMEM lane
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q4 * 32) << 16);
    float2* stats = reinterpret_cast<float2*>(smem + H2_OFF_STATS);
    float* exch = reinterpret_cast<float*>(smem + H2_OFF_EXCH);
    float* ck_all = reinterpret_cast<float*>(smem + H2_OFF_CK);
    uint8_t* pu = smem + H2_OFF_PU + half * H2_SUB;          // K-block `half` holds this thread's 64 columns
    uint32_t stats_uses = 0, pair_uses = 0;
    int ck_user = -1, q = 0;
    bool ok = true;
    H2TileUser tu;
    for (int g = 0; g < n && ok; ++g) {
      const int t = t_begin + g;
      const int b = tu.of(tile_start, p.B, t);
      const int row0 = off[b] + (t - tu.lo) * H2_TILE;
      // ---- LayerNorm statistics of the tile (two lanes per token, 64 features each), then this row's constants
      float rstd_r = 1.f, mu_r = 0.f;
      if (LN) {
        if (!mbar_wait(x_full, (uint32_t)g & 1u, p.err, 31)) { ok = false; break; }
        const int tok = 16 * rw + (lane >> 1), hf = lane & 1;
        const uint8_t* xs = smem + H2_OFF_X + hf * H2_SUB + tok * 128;
        uint4 u[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) u[c] = *reinterpret_cast<const uint4*>(xs + (((c + tok + 4 * hf) & 7) << 4));
        float sum = 0.f;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const uint32_t w[4] = {u[c].x, u[c].y, u[c].z, u[c].w};
#pragma unroll
          for (int j = 0; j < 4; ++j) sum += __uint_as_float(w[j] << 16) + __uint_as_float(w[j] & 0xffff0000u);
        }
        sum += __shfl_xor_sync(0xffffffffu, sum, 1);
        const float mu = sum * (1.0f / H2_D);
        float var = 0.f;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const uint32_t w[4] = {u[c].x, u[c].y, u[c].z, u[c].w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float a = __uint_as_float(w[j] << 16) - mu, bb = __uint_as_float(w[j] & 0xffff0000u) - mu;
            var = fmaf(a, a, var);
            var = fmaf(bb, bb, var);
          }
        }
        var += __shfl_xor_sync(0xffffffffu, var, 1);
        if (hf == 0) stats[(g & 1) * 128 + tok] = make_float2(rsqrtf(var * (1.0f / H2_D) + p.ln_eps), mu);
        __syncwarp();
        if (lane == 0) mbar_arrive(x_empty);
        if (!h2_group_sync(stats_bar, stats_uses, lane, p.err, 35)) { ok = false; break; }
        const float2 st = stats[(g & 1) * 128 + r];
        rstd_r = st.x; mu_r = st.y;
        if (b != ck_user && (ck_user < 0 || !p.shared)) {
          // every warp has passed the rendezvous, i.e. finished the previous tile: nobody still reads the old sums.
          // Warps of a half write identical values.
          for (int i = half * 64 + lane; i < p.HL; i += 128) ck_all[i] = p.cK[(int64_t)(p.shared ? 0 : b) * p.HL + i];
          for (int i = half * 64 + 32 + lane; i < p.HL; i += 128) ck_all[i] = p.cK[(int64_t)(p.shared ? 0 : b) * p.HL + i];
          __syncwarp();
        }
        ck_user = b;
      } else {
        if (lane == 0) mbar_arrive(x_empty);
      }
      // ---- per group: softmax over the links of this thread's heads, P_c -> smem
      for (int c = 0; c < NG && ok; ++c, ++q) {
        if (!mbar_wait(&s2_full[q & 1], (uint32_t)(q >> 1) & 1u, p.err, 32)) { ok = false; break; }
        tc_fence_after();
        float v[64];
        {
          float v0[32], v1[32];
          const uint32_t cs = col_of(g * (NG + 1) + c);
          tmem_ld_32x32(lane_addr + cs + half * 64, v0);
          tmem_ld_32x32(lane_addr + cs + half * 64 + 32, v1);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j) { v[j] = v0[j]; v[32 + j] = v1[j]; }
        }
        const float* ck_s = ck_all + c * 128 + half * 64;
#pragma unroll
        for (int h = 0; h < 64 / ELL; ++h) {
          float mx = -INFINITY;
#pragma unroll
          for (int j = 0; j < ELL; ++j) {
            const int cc = h * ELL + j;
            if (LN) v[cc] = (v[cc] - mu_r * ck_s[cc]) * rstd_r;
            mx = fmaxf(mx, v[cc]);
          }
          float inv;
          if (p.silu) {
            // SiLU(s) / ell: every history query attends to the ell links of the head (Algorithm 1)
#pragma unroll
            for (int j = 0; j < ELL; ++j) { const float hx = 0.5f * v[h * ELL + j]; v[h * ELL + j] = fmaf(hx, h2_tanh(hx), hx); }
            inv = 1.0f / ELL;
          } else {
            float s0 = 0.f, s1 = 0.f;
#pragma unroll
            for (int j = 0; j < ELL; j += 2) {
              v[h * ELL + j] = h2_ex2(v[h * ELL + j] - mx);
              v[h * ELL + j + 1] = h2_ex2(v[h * ELL + j + 1] - mx);
              s0 += v[h * ELL + j];
              s1 += v[h * ELL + j + 1];
            }
            inv = __fdividef(1.f, s0 + s1);
          }
#pragma unroll
          for (int j = 0; j < ELL; ++j) v[h * ELL + j] *= inv;
        }
        // P_{q-1} must have been consumed by its mix MMA before the buffer is rewritten; the probabilities above were
        // formed while that MMA ran
        if (c > 0 && !mbar_wait(p_free, (uint32_t)(q - 1) & 1u, p.err, 36)) { ok = false; break; }
#pragma unroll
        for (int c8 = 0; c8 < 8; ++c8) {
          const int cc = c8 * 8;
          uint4 o;
          o.x = h2_pack(v[cc + 0], v[cc + 1]);
          o.y = h2_pack(v[cc + 2], v[cc + 3]);
          o.z = h2_pack(v[cc + 4], v[cc + 5]);
          o.w = h2_pack(v[cc + 6], v[cc + 7]);
          *reinterpret_cast<uint4*>(pu + h2_chunk(r, (uint32_t)c8)) = o;
        }
        tc_fence_before();
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(p_ready);
      }
      if (!ok) break;
      // ---- U = SiLU(gate) * up for this thread's 64 hidden columns -> smem (over the last P, which the mix has read)
      if (!mbar_wait(gu_full, (uint32_t)g & 1u, p.err, 33)) { ok = false; break; }
      tc_fence_after();
#pragma unroll
      for (int c = 0; c < 64; c += 32) {
        float gt[32], up[32];
        tmem_ld_32x32(lane_addr + COL_GU + half * 64 + c, gt);
        tmem_ld_32x32(lane_addr + COL_GU + H2_F + half * 64 + c, up);
        tmem_wait_ld();
#pragma unroll
        for (int c8 = 0; c8 < 4; ++c8) {
          float y[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float hx = 0.5f * gt[c8 * 8 + j];
            y[j] = fmaf(hx, h2_tanh(hx), hx) * up[c8 * 8 + j];
          }
          uint4 o;
          o.x = h2_pack(y[0], y[1]); o.y = h2_pack(y[2], y[3]); o.z = h2_pack(y[4], y[5]); o.w = h2_pack(y[6], y[7]);
          *reinterpret_cast<uint4*>(pu + h2_chunk(r, (uint32_t)(c >> 3) + c8)) = o;
        }
      }
      tc_fence_before();
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(u_ready);
      // ---- this thread's 64 columns of its S' row -> (LayerNorm) -> bf16 -> staged in the P/U buffer -> whole rows to global
      if (!mbar_wait(sp_full, (uint32_t)g & 1u, p.err, 34)) { ok = false; break; }
      tc_fence_after();
      float v[64];
      {
        float v0[32], v1[32];
        const uint32_t cs = col_of(g * (NG + 1) + NG);
        tmem_ld_32x32(lane_addr + cs + half * 64, v0);
        tmem_ld_32x32(lane_addr + cs + half * 64 + 32, v1);
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < 32; ++j) { v[j] = v0[j]; v[32 + j] = v1[j]; }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(sp_free);
      if (p.out_ln) {
        // one exchange per row: each half sends the mean of its 64 columns and their squared deviations from it; the
        // two pairs combine exactly.  Slots alternate by tile parity (rewritten only after a later rendezvous).
        float s = 0.f;
#pragma unroll
        for (int j = 0; j < 64; ++j) s += v[j];
        const float m_half = s * (1.0f / 64);
        float m2 = 0.f;
#pragma unroll
        for (int j = 0; j < 64; ++j) { const float dv = v[j] - m_half; m2 = fmaf(dv, dv, m2); }
        float2* ex2 = reinterpret_cast<float2*>(exch) + (g & 1) * 256;
        ex2[half * 128 + r] = make_float2(m_half, m2);
        if (!h2_group_sync(&pair_bar[q4], pair_uses, lane, p.err, 37)) { ok = false; break; }
        const float2 other = ex2[(half ^ 1) * 128 + r];
        const float mu = 0.5f * (m_half + other.x);
        const float dm = m_half - mu;
        const float rstd = rsqrtf((m2 + other.y + 128.0f * dm * dm) * (1.0f / H2_D) + p.ln_eps);
#pragma unroll
        for (int j = 0; j < 64; ++j) v[j] = (v[j] - mu) * rstd;
      }
      {
        // A thread owns half a row (128 bytes): stored directly, every instruction would touch 32 lines.  S'(g) has
        // consumed U, so the P/U buffer is free until the next tile's first P: the tile is staged there (row r at
        // r * 256 bytes, 16-byte chunk c at position c ^ (r & 15) to spread the banks) and each warp then writes whole
        // 256-byte rows.
        uint8_t* stage = smem + H2_OFF_PU;
#pragma unroll
        for (int c8 = 0; c8 < 8; ++c8) {
          uint4 o;
          o.x = h2_pack(v[c8 * 8 + 0], v[c8 * 8 + 1]); o.y = h2_pack(v[c8 * 8 + 2], v[c8 * 8 + 3]);
          o.z = h2_pack(v[c8 * 8 + 4], v[c8 * 8 + 5]); o.w = h2_pack(v[c8 * 8 + 6], v[c8 * 8 + 7]);
          *reinterpret_cast<uint4*>(stage + r * 256u + ((((uint32_t)(half * 8 + c8)) ^ (r & 15u)) << 4)) = o;
        }
        if (!h2_group_sync(stats_bar, stats_uses, lane, p.err, 38)) { ok = false; break; }
        const int row_end = off[b + 1];
#pragma unroll 4
        for (int i = rw; i < H2_TILE; i += H2_ROW_WARPS) {
          if (row0 + i >= row_end) break;
          const uint2 o = *reinterpret_cast<const uint2*>(stage + i * 256 + ((((uint32_t)lane >> 1) ^ ((uint32_t)i & 15u)) << 4) + (lane & 1) * 8);
          *reinterpret_cast<uint2*>(p.out + (int64_t)(row0 + i) * H2_D + lane * 4) = o;
        }
        // the next tile's first P goes into the same buffer: with LayerNorm on the fly its statistics rendezvous comes
        // first, otherwise wait here until every warp has copied its rows out
        if (!LN && !h2_group_sync(stats_bar, stats_uses, lane, p.err, 40)) { ok = false; break; }
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

bool hist_update2_tc_supported(int dtype, int d, int f, int H, int ell, int phi, int gated_mlp) {
  const int HL = H * ell;
  return dtype == LIME_BF16 && d == H2_D && f == H2_F && HL % 128 == 0 && HL >= 256 && HL <= 512 && (ell == 32 || ell == 64) &&
         (phi == LIME_PHI_SOFTMAX || phi == LIME_PHI_SILU) && gated_mlp != 0;
}

template <int ELL>
static lime_status launch_hu2(const HistUpdateArgs& a, int HL, cudaStream_t st) {
  CUtensorMap tmX, tmK2, tmG, tmU, tmWo;
  const uint64_t users = a.shared ? 1 : (uint64_t)a.B;
  if (!make_tmap_bf16_sw128(&tmX, a.hist_in, (uint64_t)a.total, H2_D, H2_D, H2_TILE) ||
      !make_tmap_bf16_sw128(&tmK2, a.K2, users * HL, H2_D, H2_D, 128) ||
      !make_tmap_bf16_sw128(&tmG, a.G2t, users * H2_F, (uint64_t)HL, (uint64_t)HL, 128) ||
      !make_tmap_bf16_sw128(&tmU, a.U2t, users * H2_F, (uint64_t)HL, (uint64_t)HL, 128) ||
      !make_tmap_bf16_sw128(&tmWo, a.WoT, H2_D, H2_F, H2_F, 128))
    return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
  HistUpdate2Params p;
  p.out = (__nv_bfloat16*)a.hist_out; p.cK = a.cK; p.off = a.off; p.tile_start = a.tile_start; p.B = a.B; p.HL = HL;
  p.NG = HL / 128; p.shared = a.shared; p.silu = a.silu; p.out_ln = a.out_ln; p.ln_eps = a.ln_eps; p.err = a.err;
  int grid = a.n_tile_upper < kSMs ? a.n_tile_upper : kSMs;
  if (grid < 1) return LIME_OK;
  static bool smem_ln[kMaxDeviceOrdinals] = {}, smem_plain[kMaxDeviceOrdinals] = {};
  lime_status es = a.ln ? ensure_dynamic_smem((const void*)k_hist_update2_tc<ELL, true>, (int)H2_SMEM, smem_ln)
                        : ensure_dynamic_smem((const void*)k_hist_update2_tc<ELL, false>, (int)H2_SMEM, smem_plain);
  if (es != LIME_OK) return es;
  ProfScope _p("k_hist_update2_tc", st);
  if (a.ln) launch_pdl(k_hist_update2_tc<ELL, true>, dim3(grid), dim3(H2_THREADS), H2_SMEM, st, tmX, tmK2, tmG, tmU, tmWo, p);
  else launch_pdl(k_hist_update2_tc<ELL, false>, dim3(grid), dim3(H2_THREADS), H2_SMEM, st, tmX, tmK2, tmG, tmU, tmWo, p);
  LIME_LAUNCH_CHECK("k_hist_update2_tc");
  return LIME_OK;
}

lime_status launch_hist_update2_tc(const HistUpdateArgs& a, int H, cudaStream_t st) {
  if (a.total == 0) return LIME_OK;
  switch (a.ell) {
    case 32: return launch_hu2<32>(a, H * a.ell, st);
    case 64: return launch_hu2<64>(a, H * a.ell, st);
  }
  return LIME_UNSUPPORTED_SHAPE;
}

}  // namespace lime
