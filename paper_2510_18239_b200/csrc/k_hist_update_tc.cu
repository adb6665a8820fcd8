// History update of one XOR layer on the 5th-generation tensor cores (bf16 storage):
//
//   S'[t,:] = GatedMLP( O[S]_t ),   O[S]_t = concat_h softmax_l( Q[S]_{t,h} K[T]_{l,h}^T * scale ) V[T]_{l,h}     (Eq. 7, Eq. 5)
//
// fused per 128-token tile into three chained tensor-core contractions whose operands never leave the SM:
//   1. scores  [128 x HL]  = X_tile [128 x d] . K2^T               (K2 = folded link keys, see k_link_prep.cu; the fold
//      carries scale * log2(e)).  LayerNorm is applied afterwards as s = rstd_t * (raw - mu_t * rowsum(K2)), exact
//      for the bf16 operands
//   2. per-head softmax over the ell links of each token (registers only) -> P (bf16, smem)
//   3. [gate | up] [128 x 2f] = P [128 x HL] . [G2 | U2]           (value mix and first GatedMLP layer folded)
//   4. U = SiLU(gate) * up (bf16, smem)       5. S' = U [128 x f] . W_o [f x d]  -> bf16 rows to global
// HL = H * ell stacked (head, link) rows.  History is read once (TMA) and written once per layer.
//
// Warp roles: warp 0 TMA producer, warp 1 MMA issuer, warps 2-17 token rows: four threads per token (TMEM lane), each
// owning 32 of the 128 columns of every step - one head of the softmax when ell = 32 (a warp may only touch the TMEM
// lane quarter warp_id % 4, so the four parts of a row sit in warps w, w + 4, w + 8, w + 12).  Four warps per
// scheduler keep the issue slots busy while TMEM loads and transcendentals are in flight.  The steps of consecutive
// tiles are software-pipelined so that the tensor pipe works on one tile while the token warps work on the other:
//   token warps, tile g :  SiLU(g) | statistics of tile g+1 | softmax(g+1) | store S'(g)
//   MMA issuer,  tile g :  [gate|up](g) , scores(g+1) | S'(g)             | [gate|up](g+1) ...
// TMEM: two 128-column buffers that hold a tile's scores and later its S' (alternating by tile), 256 columns
// [gate | up].  Shared memory: one token stage (32 KB), K2, [G2 | U2], W_o (128 KB), one P/U buffer (32 KB).
//
// With `out_ln` the rows are written already LayerNorm-ed (the next layer applies LayerNorm to every row it reads and
// nothing else reads them, Eq. 8), so that the next layer's kernels run with LN = false.
//
// Built for d = d_ff = 128, H * ell = 128 and ell in {16, 32}.
#include "lime_common.cuh"
#include "tc_common.cuh"

namespace lime {

constexpr int HU_D = 128, HU_F = 128, HU_HL = 128, HU_TILE = 128;
constexpr int HU_PARTS = 4;                            // threads per token row
constexpr int HU_COLS = 128 / HU_PARTS;                // columns per thread in every step
constexpr int HU_ROW_WARPS = 4 * HU_PARTS, HU_THREADS = 64 + 32 * HU_ROW_WARPS;
constexpr uint32_t HU_SUB = 128 * 128;                 // bytes of one [128 rows x 64 bf16] swizzled sub-tile
constexpr uint32_t HU_OFF_X = 0;                       // token tile: 2 K-blocks
constexpr uint32_t HU_OFF_K2 = 2 * HU_SUB;             // [HL x d]      2 K-blocks x 16 KB
constexpr uint32_t HU_OFF_GU = HU_OFF_K2 + 2 * HU_SUB; // [2f x HL]     2 K-blocks x 32 KB (gate rows, then up rows)
constexpr uint32_t HU_OFF_WO = HU_OFF_GU + 4 * HU_SUB; // [d x f]       2 K-blocks x 16 KB
constexpr uint32_t HU_OFF_PU = HU_OFF_WO + 2 * HU_SUB; // P, then U, of the current tile: 2 K-blocks
constexpr uint32_t HU_OFF_STATS = HU_OFF_PU + 2 * HU_SUB;   // 2 (tile parity) x 128 float2 {rstd, mu}
constexpr uint32_t HU_OFF_EXCH = HU_OFF_STATS + 2 * 128 * 8;   // row exchange: [2 tile parities][PARTS][128] float2 {mean, M2}
constexpr uint32_t HU_OFF_CK = HU_OFF_EXCH + 2 * HU_PARTS * 128 * 8;   // the current user's HL key row sums (fp32)
constexpr uint32_t HU_OFF_BAR = HU_OFF_CK + HU_HL * 4;
constexpr int HU_IDX_CAP = 1025;                            // users + 1 whose offsets are staged in shared memory (the
constexpr uint32_t HU_OFF_IDX = HU_OFF_BAR + 256;           // search for a tile's user is a chain of dependent reads:
constexpr uint32_t HU_SMEM = HU_OFF_IDX + 2 * HU_IDX_CAP * 4 + 8;   // microseconds from global memory)
static_assert(HU_SMEM <= 232448, "shared memory budget of one CTA");

struct HistUpdateParams {
  __nv_bfloat16* out;            // [total x d]
  const float* cK;               // [users x HL] row sums of K2
  const float2* stats_in;        // nullable (LN): {rstd, mean} of every history row, computed by the attention kernel
  const int32_t* off;            // [B+1]
  const int32_t* tile_start;     // [B+1] prefix of per-user tile counts (tile = 128 tokens)
  int B, ell, shared, out_ln;
  int silu;                      // 1: P = SiLU(scores) / ell (Algorithm 2) instead of the per-head softmax
  float ln_eps;
  int* err;
};

// address of 16-byte chunk `c` (0..7) of row r inside a 128B-swizzled [rows x 64 bf16] sub-tile
__device__ __forceinline__ uint32_t sw128_chunk(uint32_t r, uint32_t c) { return r * 128u + ((c ^ (r & 7u)) << 4); }

// user of tile t, cached: consecutive tiles are the same user most of the time, and when they are not the user is a
// neighbour of the cached one, found by stepping through tile_start (staged in shared memory) instead of a search
struct TileUser {
  int b = -1, lo = 0, hi = 0;
  __device__ __forceinline__ int of(const int32_t* __restrict__ tile_start, int B, int t) {
    if (t < lo || t >= hi) {
      if (b < 0) b = upper_user(tile_start, B, t);
      else if (t >= hi) { do { ++b; } while (tile_start[b + 1] <= t); }
      else { do { --b; } while (tile_start[b] > t); }
      lo = tile_start[b];
      hi = tile_start[b + 1];
    }
    return b;
  }
};
// the same walk for code that needs the token rows of a tile: the user's row range is cached with the tile range
struct TileRows {
  TileUser tu;
  int row_lo = 0, row_hi = 0;
  // first token row of tile t; row_hi is the end of its user's rows
  __device__ __forceinline__ int first_row(const int32_t* __restrict__ tile_start, const int32_t* __restrict__ off, int B,
                                           int t, int tile) {
    const int before = tu.b;
    const int b = tu.of(tile_start, B, t);
    if (b != before) { row_lo = off[b]; row_hi = off[b + 1]; }
    return row_lo + (t - tu.lo) * tile;
  }
};

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float tanh_approx(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float hu_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Rendezvous of the warps that arrive on `bar`, with a bounded wait; shared-memory writes made by any lane before the
// call are visible to every participant after it.
__device__ __forceinline__ bool hu_group_sync(uint64_t* bar, uint32_t& uses, int lane, int* err, int where) {
  __syncwarp();
  if (lane == 0) tc::mbar_arrive(bar);
  const bool ok = tc::mbar_wait(bar, uses & 1u, err, where);
  ++uses;
  return ok;
}

template <int ELL, bool LN>
__global__ void __launch_bounds__(HU_THREADS, 1)
k_hist_update_tc(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmK2,
                 const __grid_constant__ CUtensorMap tmG, const __grid_constant__ CUtensorMap tmU,
                 const __grid_constant__ CUtensorMap tmWo, const HistUpdateParams p) {
  using namespace tc;
  static_assert(HU_COLS % ELL == 0, "a thread owns whole heads");
  extern __shared__ __align__(1024) uint8_t smem[];
  if ((smem_u32(smem) & 1023u) != 0) {                       // swizzled tiles need a 1024-byte aligned base
    if (threadIdx.x == 0) atomicCAS(p.err, 0, 90);
    return;
  }
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + HU_OFF_BAR);
  uint64_t* x_full = bars;           // token tile landed
  uint64_t* x_empty = bars + 1;      // scores MMA done (1) + statistics taken by the row warps
  uint64_t* k2_full = bars + 2;      // per user segment
  uint64_t* k2_empty = bars + 3;
  uint64_t* ops_full = bars + 4;     // per user segment: G2, U2
  uint64_t* ops_empty = bars + 5;
  uint64_t* wo_full = bars + 6;
  uint64_t* s2_full = bars + 7;      // per tile: scores in TMEM
  uint64_t* p_ready = bars + 8;      // per tile: P in smem (all row warps)
  uint64_t* gu_full = bars + 9;      // per tile: [gate | up] in TMEM
  uint64_t* u_ready = bars + 10;     // per tile: U in smem (all row warps)
  uint64_t* sp_full = bars + 11;     // per tile: S' in TMEM (and U read)
  uint64_t* sp_free = bars + 12;     // per tile: S' read out (all row warps)
  uint64_t* stats_bar = bars + 13;   // rendezvous of the row warps (token statistics written)
  uint64_t* row_bar = bars + 14;     // [4] rendezvous of the warps sharing a TMEM lane quarter
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 18);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    mbar_init(x_full, 1); mbar_init(x_empty, 1 + HU_ROW_WARPS);
    mbar_init(k2_full, 1); mbar_init(k2_empty, 1); mbar_init(ops_full, 1); mbar_init(ops_empty, 1); mbar_init(wo_full, 1);
    mbar_init(s2_full, 1); mbar_init(p_ready, HU_ROW_WARPS); mbar_init(gu_full, 1); mbar_init(u_ready, HU_ROW_WARPS);
    mbar_init(sp_full, 1); mbar_init(sp_free, HU_ROW_WARPS); mbar_init(stats_bar, HU_ROW_WARPS);
    for (int i = 0; i < 4; ++i) mbar_init(&row_bar[i], HU_PARTS);
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
  const int n = t_end - t_begin;                            // tiles of this CTA, g = 0..n-1
  const int32_t* tile_start = p.tile_start;
  const int32_t* off = p.off;
  if (p.B + 1 <= HU_IDX_CAP) {
    int32_t* idx = reinterpret_cast<int32_t*>(smem + HU_OFF_IDX);
    for (int i = threadIdx.x; i <= p.B; i += HU_THREADS) { idx[i] = p.tile_start[i]; idx[HU_IDX_CAP + i] = p.off[i]; }
    tile_start = idx;
    off = idx + HU_IDX_CAP;
    __syncthreads();
  }
  constexpr uint32_t COL_SS = 0, COL_GU = 256;      // scores / S' buffer of tile g: COL_SS + (g & 1) * 128

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0 && n > 0) {
      const uint64_t pol_stream = policy_evict_first(), pol_keep = policy_evict_last();
      mbar_arrive_expect_tx(wo_full, 2 * HU_SUB);
      for (int kb = 0; kb < 2; ++kb) tma_load_2d_hint(smem + HU_OFF_WO + kb * HU_SUB, &tmWo, kb * 64, 0, wo_full, pol_keep);
      int cur_user = -1, seg = 0, g = 0;
      bool ok = true;
      TileUser tu;
      for (; g < n && ok; ++g) {
        const int t = t_begin + g;
        const int b = tu.of(tile_start, p.B, t);
        if (b != cur_user && (seg == 0 || !p.shared)) {
          const int urow = p.shared ? 0 : b;
          if (seg > 0 && !mbar_wait(k2_empty, (uint32_t)(seg - 1) & 1u, p.err, 11)) { ok = false; break; }
          mbar_arrive_expect_tx(k2_full, 2 * HU_SUB);
          for (int kb = 0; kb < 2; ++kb)
            tma_load_2d_hint(smem + HU_OFF_K2 + kb * HU_SUB, &tmK2, kb * 64, urow * HU_HL, k2_full, pol_keep);
          if (seg > 0 && !mbar_wait(ops_empty, (uint32_t)(seg - 1) & 1u, p.err, 13)) { ok = false; break; }
          mbar_arrive_expect_tx(ops_full, 4 * HU_SUB);
          for (int kb = 0; kb < 2; ++kb) {
            tma_load_2d_hint(smem + HU_OFF_GU + kb * 2 * HU_SUB, &tmG, kb * 64, urow * HU_F, ops_full, pol_keep);
            tma_load_2d_hint(smem + HU_OFF_GU + kb * 2 * HU_SUB + HU_SUB, &tmU, kb * 64, urow * HU_F, ops_full, pol_keep);
          }
          ++seg;
        }
        cur_user = b;
        if (g > 0 && !mbar_wait(x_empty, (uint32_t)(g - 1) & 1u, p.err, 12)) { ok = false; break; }
        const int row0 = off[b] + (t - tu.lo) * HU_TILE;
        mbar_arrive_expect_tx(x_full, 2 * HU_SUB);
        for (int kb = 0; kb < 2; ++kb) tma_load_2d_hint(smem + HU_OFF_X + kb * HU_SUB, &tmX, kb * 64, row0, x_full, pol_stream);
      }
      if (!ok || *(volatile int*)p.err != 0) {
        // giving up: let the copies already issued land (bounded) before this CTA's shared memory goes away
        if (g > 0) mbar_wait_quiet(x_full, (uint32_t)(g - 1) & 1u);
        if (seg > 0) { mbar_wait_quiet(k2_full, (uint32_t)(seg - 1) & 1u); mbar_wait_quiet(ops_full, (uint32_t)(seg - 1) & 1u); }
        mbar_wait_quiet(wo_full, 0);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && n > 0) {
      constexpr uint32_t idesc_128 = make_idesc_bf16(128, 128);
      constexpr uint32_t idesc_256 = make_idesc_bf16(128, 256);
      const uint32_t sbase = smem_u32(smem);
      const uint32_t pu = sbase + HU_OFF_PU;
      TileUser tu;
      int user_of_scores = -1, user_of_mix = -1, seg_k = 0, seg_o = 0;
      // does tile g close its user's run of tiles inside this CTA (so that the user's operands may be replaced)?
      auto last_of_user = [&](int g) {
        if (p.shared) return false;
        const int t = t_begin + g;
        tu.of(tile_start, p.B, t);
        return g + 1 < n && t + 1 >= tu.hi;
      };
      // 1. scores(g) = X . K2^T
      auto issue_scores = [&](int g) -> bool {
        const int b = tu.of(tile_start, p.B, t_begin + g);
        if (b != user_of_scores && (seg_k == 0 || !p.shared)) {
          if (!mbar_wait(k2_full, (uint32_t)seg_k & 1u, p.err, 22)) return false;
          ++seg_k;
        }
        user_of_scores = b;
        if (g >= 2 && !mbar_wait(sp_free, (uint32_t)(g - 2) & 1u, p.err, 26)) return false;   // S'(g-2) shared the buffer
        if (!mbar_wait(x_full, (uint32_t)g & 1u, p.err, 23)) return false;
        tc_fence_after();
        for (int kk = 0; kk < 8; ++kk) {
          const uint32_t o = (uint32_t)(kk >> 2) * HU_SUB + (uint32_t)(kk & 3) * 32;
          mma_bf16_ss(tmem_base + COL_SS + (uint32_t)(g & 1) * 128, make_sdesc_k_sw128(sbase + HU_OFF_X + o),
                      make_sdesc_k_sw128(sbase + HU_OFF_K2 + o), idesc_128, kk != 0);
        }
        mma_commit(x_empty);
        mma_commit(s2_full);
        if (last_of_user(g)) mma_commit(k2_empty);
        return true;
      };
      bool ok = mbar_wait(wo_full, 0, p.err, 21);
      if (ok) ok = issue_scores(0);
      for (int g = 0; g < n && ok; ++g) {
        const uint32_t tp = (uint32_t)g & 1u;
        // 3. [gate | up](g) = P(g) . [G2 | U2]
        const int b = tu.of(tile_start, p.B, t_begin + g);
        if (b != user_of_mix && (seg_o == 0 || !p.shared)) {
          if (!mbar_wait(ops_full, (uint32_t)seg_o & 1u, p.err, 27)) break;
          ++seg_o;
        }
        user_of_mix = b;
        if (!mbar_wait(p_ready, tp, p.err, 24)) break;
        tc_fence_after();
        for (int kk = 0; kk < 8; ++kk) {
          const uint32_t oa = (uint32_t)(kk >> 2) * HU_SUB + (uint32_t)(kk & 3) * 32;
          const uint32_t ob = (uint32_t)(kk >> 2) * 2 * HU_SUB + (uint32_t)(kk & 3) * 32;
          mma_bf16_ss(tmem_base + COL_GU, make_sdesc_k_sw128(pu + oa), make_sdesc_k_sw128(sbase + HU_OFF_GU + ob), idesc_256,
                      kk != 0);
        }
        mma_commit(gu_full);
        if (last_of_user(g)) mma_commit(ops_empty);
        // 1'. scores of the next tile, while the row warps turn [gate | up](g) into U(g)
        if (g + 1 < n && !issue_scores(g + 1)) break;
        // 5. S'(g) = U(g) . W_o, into the buffer that held scores(g)
        if (!mbar_wait(u_ready, tp, p.err, 25)) break;
        tc_fence_after();
        for (int kk = 0; kk < 8; ++kk) {
          const uint32_t o = (uint32_t)(kk >> 2) * HU_SUB + (uint32_t)(kk & 3) * 32;
          mma_bf16_ss(tmem_base + COL_SS + (uint32_t)(g & 1) * 128, make_sdesc_k_sw128(pu + o),
                      make_sdesc_k_sw128(sbase + HU_OFF_WO + o), idesc_128, kk != 0);
        }
        mma_commit(sp_full);
      }
    }
  } else if (n > 0) {
    // ------------------------------------------------------------------ token-row warps (2..17)
    const int rw = warp - 2;                                 // 0..15
    const int q = warp & 3;                                  // TMEM lane quarter of this warp
    const int part = rw >> 2;                                // which 32 columns of every step
    const int col0 = part * HU_COLS;
    const uint32_t r = (uint32_t)(q * 32 + lane);            // token row of the tile == TMEM lane
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
    float2* stats = reinterpret_cast<float2*>(smem + HU_OFF_STATS);
    float* exch = reinterpret_cast<float*>(smem + HU_OFF_EXCH);                 // [2 tile parities][PARTS][128] float2
    const float* ck_s = reinterpret_cast<const float*>(smem + HU_OFF_CK) + col0;   // key row sums of this thread's columns
    // K index = column, so this thread's columns live in K-block col0 / 64, chunks (col0 % 64) / 8 ..
    uint8_t* pu = smem + HU_OFF_PU + (col0 >> 6) * HU_SUB;
    const uint32_t chunk0 = (uint32_t)(col0 & 63) >> 3;
    uint32_t stats_uses = 0, row_uses = 0;
    int ck_user = -1;
    bool ok = true;
    float rstd_r = 1.f, mu_r = 0.f;                          // LayerNorm constants of this thread's token row

    // LayerNorm statistics of tile g: four lanes per token, 32 features each; then this thread's own row constants.
    // Two slots by tile parity: a warp past the rendezvous of tile g+1 knows every warp has read tile g's.
    // With statistics handed over by the attention kernel, a thread needs only those of its own row: one 8-byte read,
    // issued a tile ahead (fetch_stats) and taken here.
    TileRows tr_next, tr_out;       // walkers over the tile being prepared (g + 1) and the tile being stored (g)
    float2 st_ahead = make_float2(1.f, 0.f);
    auto fetch_stats = [&](int g) {
      const int row = tr_next.first_row(tile_start, off, p.B, t_begin + g, HU_TILE) + (int)r;
      st_ahead = row < tr_next.row_hi ? __ldg(p.stats_in + row) : make_float2(1.f, 0.f);
    };
    auto take_stats = [&](int g) -> bool {
      if (LN && p.stats_in != nullptr) {
        rstd_r = st_ahead.x; mu_r = st_ahead.y;
        if (lane == 0) mbar_arrive(x_empty);
        return true;
      }
      if (LN) {
        if (!mbar_wait(x_full, (uint32_t)g & 1u, p.err, 31)) return false;
        const int tok = 8 * rw + (lane >> 2), p4 = lane & 3;
        const uint8_t* xs = smem + HU_OFF_X + (p4 >> 1) * HU_SUB + tok * 128;
        uint4 u[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int ch = (p4 & 1) * 4 + ((c + (p4 >> 1)) & 3);
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
        const float mu = sum * (1.0f / HU_D);
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
        if (p4 == 0) stats[(g & 1) * 128 + tok] = make_float2(rsqrtf(var * (1.0f / HU_D) + p.ln_eps), mu);
        __syncwarp();
        if (lane == 0) mbar_arrive(x_empty);                 // this warp is done with the staged tile
        if (!hu_group_sync(stats_bar, stats_uses, lane, p.err, 35)) return false;
        const float2 st = stats[(g & 1) * 128 + r];
        rstd_r = st.x; mu_r = st.y;
      } else {
        if (lane == 0) mbar_arrive(x_empty);
      }
      return true;
    };

    // 2. per-head softmax over the links of this thread's heads (32 score columns), P -> smem
    auto softmax = [&](int g) -> bool {
      float v[HU_COLS];
      tr_next.first_row(tile_start, off, p.B, t_begin + g, HU_TILE);
      const int b = tr_next.tu.b;
      if (!mbar_wait(s2_full, (uint32_t)g & 1u, p.err, 32)) return false;
      tc_fence_after();
      if (LN && b != ck_user && (ck_user < 0 || !p.shared)) {
        // scores(g) exist, so every warp has finished the softmax of tile g-1 (its P was needed first): nobody still
        // reads the previous user's sums.  Every warp of a part writes the same values.
        float* ckw = reinterpret_cast<float*>(smem + HU_OFF_CK) + col0;
        ckw[lane] = p.cK[(int64_t)(p.shared ? 0 : b) * HU_HL + col0 + lane];
        __syncwarp();
      }
      ck_user = b;
      tmem_ld_32x32(lane_addr + COL_SS + (uint32_t)(g & 1) * 128 + col0, v);
      tmem_wait_ld();
#pragma unroll
      for (int h = 0; h < HU_COLS / ELL; ++h) {
        float mx = -INFINITY;
#pragma unroll
        for (int j = 0; j < ELL; ++j) {
          const int c = h * ELL + j;
          if (LN) v[c] = (v[c] - mu_r * ck_s[c]) * rstd_r;
          mx = fmaxf(mx, v[c]);
        }
        float inv;
        if (p.silu) {
          // SiLU(s) / ell: every history query attends to the ell links of the head (Algorithm 1)
#pragma unroll
          for (int j = 0; j < ELL; ++j) { const float hx = 0.5f * v[h * ELL + j]; v[h * ELL + j] = fmaf(hx, tanh_approx(hx), hx); }
          inv = 1.0f / ELL;
        } else {
          float s0 = 0.f, s1 = 0.f;
#pragma unroll
          for (int j = 0; j < ELL; j += 2) {
            v[h * ELL + j] = hu_ex2(v[h * ELL + j] - mx);
            v[h * ELL + j + 1] = hu_ex2(v[h * ELL + j + 1] - mx);
            s0 += v[h * ELL + j];
            s1 += v[h * ELL + j + 1];
          }
          inv = __fdividef(1.f, s0 + s1);
        }
#pragma unroll
        for (int j = 0; j < ELL; ++j) v[h * ELL + j] *= inv;
      }
#pragma unroll
      for (int c8 = 0; c8 < HU_COLS / 8; ++c8) {
        const int c = c8 * 8;                                // first of 8 consecutive contraction indices
        uint4 o;
        o.x = pack_bf16(v[c + 0], v[c + 1]);
        o.y = pack_bf16(v[c + 2], v[c + 3]);
        o.z = pack_bf16(v[c + 4], v[c + 5]);
        o.w = pack_bf16(v[c + 6], v[c + 7]);
        *reinterpret_cast<uint4*>(pu + sw128_chunk(r, chunk0 + (uint32_t)c8)) = o;
      }
      tc_fence_before();
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(p_ready);
      return true;
    };

    // 4. U = SiLU(gate) * up for this thread's 32 hidden columns -> smem (over P(g), which [gate|up](g) has read)
    auto silu_mul = [&](int g) -> bool {
      if (!mbar_wait(gu_full, (uint32_t)g & 1u, p.err, 33)) return false;
      tc_fence_after();
      float gt[HU_COLS], up[HU_COLS];
      tmem_ld_32x32(lane_addr + COL_GU + col0, gt);
      tmem_ld_32x32(lane_addr + COL_GU + HU_F + col0, up);
      tmem_wait_ld();
#pragma unroll
      for (int c8 = 0; c8 < HU_COLS / 8; ++c8) {
        float y[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float hx = 0.5f * gt[c8 * 8 + j];
          y[j] = fmaf(hx, tanh_approx(hx), hx) * up[c8 * 8 + j];    // x * sigmoid(x) = x/2 * (1 + tanh(x/2))
        }
        uint4 o;
        o.x = pack_bf16(y[0], y[1]); o.y = pack_bf16(y[2], y[3]); o.z = pack_bf16(y[4], y[5]); o.w = pack_bf16(y[6], y[7]);
        *reinterpret_cast<uint4*>(pu + sw128_chunk(r, chunk0 + (uint32_t)c8)) = o;
      }
      tc_fence_before();
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(u_ready);
      return true;
    };

    // 6. this thread's 32 columns of its S' row -> (LayerNorm) -> bf16 -> global.  The caller has waited for sp_full(g).
    auto store_rows = [&](int g) -> bool {
      const int row0 = tr_out.first_row(tile_start, off, p.B, t_begin + g, HU_TILE);
      float v[HU_COLS];
      tmem_ld_32x32(lane_addr + COL_SS + (uint32_t)(g & 1) * 128 + col0, v);
      tmem_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(sp_free);
      if (p.out_ln) {
        // one exchange per row: every part sends the mean of its columns and their squared deviations from it, and
        // the four pairs are combined exactly (sum of the parts' deviations + the spread of the parts' means).  Two
        // slots by tile parity: a slot is rewritten only after a later rendezvous of the same row group.
        float s = 0.f;
#pragma unroll
        for (int j = 0; j < HU_COLS; ++j) s += v[j];
        const float m_part = s * (1.0f / HU_COLS);
        float m2 = 0.f;
#pragma unroll
        for (int j = 0; j < HU_COLS; ++j) { const float dv = v[j] - m_part; m2 = fmaf(dv, dv, m2); }
        float2* ex2 = reinterpret_cast<float2*>(exch) + (g & 1) * HU_PARTS * 128;
        ex2[part * 128 + r] = make_float2(m_part, m2);
        if (!hu_group_sync(&row_bar[q], row_uses, lane, p.err, 37)) return false;
        float2 pm[HU_PARTS];
        float mu = 0.f;
#pragma unroll
        for (int i = 0; i < HU_PARTS; ++i) { pm[i] = ex2[i * 128 + r]; mu += pm[i].x; }
        mu *= (1.0f / HU_PARTS);
        float vt = 0.f;
#pragma unroll
        for (int i = 0; i < HU_PARTS; ++i) { const float dm = pm[i].x - mu; vt += pm[i].y + (float)HU_COLS * dm * dm; }
        const float rstd = rsqrtf(vt * (1.0f / HU_D) + p.ln_eps);
#pragma unroll
        for (int j = 0; j < HU_COLS; ++j) v[j] = (v[j] - mu) * rstd;
      }
      // bf16 row part = 4 chunks of 16 bytes.  A 4 x 4 transpose of chunks inside each group of four lanes (two
      // butterfly steps of warp shuffles) leaves lane 4j+i with chunk i of rows 4j..4j+3, so that every store
      // instruction writes whole 64-byte row parts (full sectors) instead of 32 scattered 16-byte pieces.
      uint4 tch[4];
#pragma unroll
      for (int c8 = 0; c8 < 4; ++c8) {
        tch[c8].x = pack_bf16(v[c8 * 8 + 0], v[c8 * 8 + 1]); tch[c8].y = pack_bf16(v[c8 * 8 + 2], v[c8 * 8 + 3]);
        tch[c8].z = pack_bf16(v[c8 * 8 + 4], v[c8 * 8 + 5]); tch[c8].w = pack_bf16(v[c8 * 8 + 6], v[c8 * 8 + 7]);
      }
      auto xchg = [&](uint4& keep_lo, uint4& keep_hi, bool upper, int dist) {
        // lanes with `upper` clear give away keep_hi and receive into it; lanes with it set give away keep_lo
        uint4 send = upper ? keep_lo : keep_hi, recv;
        recv.x = __shfl_xor_sync(0xffffffffu, send.x, dist); recv.y = __shfl_xor_sync(0xffffffffu, send.y, dist);
        recv.z = __shfl_xor_sync(0xffffffffu, send.z, dist); recv.w = __shfl_xor_sync(0xffffffffu, send.w, dist);
        if (upper) keep_lo = recv; else keep_hi = recv;
      };
      xchg(tch[0], tch[1], (lane & 1) != 0, 1);
      xchg(tch[2], tch[3], (lane & 1) != 0, 1);
      xchg(tch[0], tch[2], (lane & 2) != 0, 2);
      xchg(tch[1], tch[3], (lane & 2) != 0, 2);
      const int rbase = row0 + q * 32 + (lane & ~3);          // first of the four rows this lane group holds
      const int row_end = tr_out.row_hi;
#pragma unroll
      for (int m = 0; m < 4; ++m)
        if (rbase + m < row_end)
          *reinterpret_cast<uint4*>(p.out + (int64_t)(rbase + m) * HU_D + col0 + (lane & 3) * 8) = tch[m];
      return true;
    };

    if (LN && p.stats_in != nullptr) fetch_stats(0);
    ok = take_stats(0) && softmax(0);
    for (int g = 0; g < n && ok; ++g) {
      if (LN && p.stats_in != nullptr && g + 1 < n) fetch_stats(g + 1);
      if (!silu_mul(g)) { ok = false; break; }                                   // [gate|up](g) ran under store(g-1)
      // statistics of the next tile while S'(g) is formed, so that its stage can be refilled a whole tile early
      if (g + 1 < n && !take_stats(g + 1)) { ok = false; break; }
      // P(g+1) overwrites U(g): wait until S'(g) has consumed it
      if (!mbar_wait(sp_full, (uint32_t)g & 1u, p.err, 34)) { ok = false; break; }
      tc_fence_after();
      if (g + 1 < n && !softmax(g + 1)) { ok = false; break; }
      if (!store_rows(g)) { ok = false; break; }                                 // runs under [gate|up](g+1)
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

bool hist_update_tc_supported(int dtype, int d, int f, int H, int ell, int phi, int gated_mlp) {
  return dtype == LIME_BF16 && d == HU_D && f == HU_F && H * ell == HU_HL && (ell == 16 || ell == 32) &&
         (phi == LIME_PHI_SOFTMAX || phi == LIME_PHI_SILU) && gated_mlp != 0;
}

template <int ELL>
static lime_status launch_hu(const HistUpdateArgs& a, cudaStream_t st) {
  CUtensorMap tmX, tmK2, tmG, tmU, tmWo;
  const uint64_t users = a.shared ? 1 : (uint64_t)a.B;
  if (!make_tmap_bf16_sw128(&tmX, a.hist_in, (uint64_t)a.total, HU_D, HU_D, HU_TILE) ||
      !make_tmap_bf16_sw128(&tmK2, a.K2, users * HU_HL, HU_D, HU_D, 128) ||
      !make_tmap_bf16_sw128(&tmG, a.G2t, users * HU_F, HU_HL, HU_HL, 128) ||
      !make_tmap_bf16_sw128(&tmU, a.U2t, users * HU_F, HU_HL, HU_HL, 128) ||
      !make_tmap_bf16_sw128(&tmWo, a.WoT, HU_D, HU_F, HU_F, 128))
    return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
  HistUpdateParams p;
  p.out = (__nv_bfloat16*)a.hist_out; p.cK = a.cK; p.stats_in = a.ln ? a.stats_in : nullptr; p.off = a.off; p.tile_start = a.tile_start; p.B = a.B; p.silu = a.silu; p.ell = ELL;
  p.shared = a.shared; p.out_ln = a.out_ln; p.ln_eps = a.ln_eps; p.err = a.err;
  int grid = a.n_tile_upper < kSMs ? a.n_tile_upper : kSMs;
  if (grid < 1) return LIME_OK;
  static bool smem_ln[kMaxDeviceOrdinals] = {}, smem_plain[kMaxDeviceOrdinals] = {};
  lime_status es = a.ln ? ensure_dynamic_smem((const void*)k_hist_update_tc<ELL, true>, (int)HU_SMEM, smem_ln)
                        : ensure_dynamic_smem((const void*)k_hist_update_tc<ELL, false>, (int)HU_SMEM, smem_plain);
  if (es != LIME_OK) return es;
  ProfScope _p("k_hist_update_tc", st);
  if (a.ln) launch_pdl(k_hist_update_tc<ELL, true>, dim3(grid), dim3(HU_THREADS), HU_SMEM, st, tmX, tmK2, tmG, tmU, tmWo, p);
  else launch_pdl(k_hist_update_tc<ELL, false>, dim3(grid), dim3(HU_THREADS), HU_SMEM, st, tmX, tmK2, tmG, tmU, tmWo, p);
  LIME_LAUNCH_CHECK("k_hist_update_tc");
  return LIME_OK;
}

lime_status launch_hist_update_tc(const HistUpdateArgs& a, cudaStream_t st) {
  if (a.total == 0) return LIME_OK;
  switch (a.ell) {
    case 16: return launch_hu<16>(a, st);
    case 32: return launch_hu<32>(a, st);
  }
  return LIME_UNSUPPORTED_SHAPE;
}

}  // namespace lime
