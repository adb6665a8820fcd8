// History update of one XOR layer on tcgen05 at d = d_ff = 256 with ell = 64 links and H in {2, 4, 8} heads (bf16 storage,
// rows LayerNorm-ed already):
//
//   S'[t,:] = GatedMLP( O[S]_t ),   O[S]_t = concat_h phi( Q[S]_{t,h} K[T]_{l,h}^T * scale ) V[T]_{l,h}          (Eq. 7, Eq. 5)
//   GatedMLP(A) = ( SiLU(A W_g) * (A W_u) ) W_o
//
// Per 128-token tile the chain of contractions never leaves the SM.  Scores are taken against the folded link keys K2
// (k_link_prep.cu: Q[S] is never formed), the value mix is done head by head against the plain link values V[T], and
// the GatedMLP weights follow unfolded - at this width folding W_V W_g into the link side (as the d = 128 kernels do)
// would cost twice the tensor work and twice the operand traffic:
//   scores [128 x H*64] = X . K2^T, 256 stacked (head, link) rows = four heads per contraction
//   per group c of two heads: per-head softmax over the 64 links, unnormalised (or SiLU(s) / 64) -> P_c (bf16);
//                             O[:, head] = P_head [128 x 64] . V_head [64 x d_h]
//   O * 1 / (row sum of the head) -> bf16
//   per half hf of the hidden columns:   [gate | up] = O . [W_g | W_u][:, hf]  ->  U = SiLU(gate) * up (bf16)
//                                        S' (+)= U . W_o[hf rows, :]
//   S' -> (LayerNorm) -> bf16 -> global memory
// Every contraction but the value mix is issued 256 columns wide: at 128 columns an MMA re-reads its A operand from
// shared memory twice as often per flop, and shared-memory bandwidth (operands in, TMA writes, the row warps) is what
// the tensor pipe waits for here.
// TMEM (512 columns) as two regions that swap roles every tile.  R0: scores of heads 0-3, overwritten head by head by
// O as its scores are consumed, later S'.  R1: scores of heads 4-7, later [gate | up] of one half.  The next tile's
// R0 is this tile's R1, which is free before S' is even complete.
// Shared memory: X tile 64 KB (dead once the scores are formed: then the two P buffers, then O); V[T]^T of the user, later
// U, later the patches S' leaves through, 32 KB; a ring of three 32 KB operand slabs ([256 rows x 64 of the contraction
// index]) through which K2, [W_g | W_u] and W_o stream from L2 in the order the MMA issuer consumes them.  (Seven
// 16 KB slabs of 32 of the contraction index, 64-byte swizzle - half again as many bytes in flight - were measured:
// 8.3 against 7.4 ms per production_ragged step; what limits the stream is not its depth but the 64-byte pieces.)
// Warp 0 TMA producer, warp 1 MMA issuer, warps 2-17 token rows.  For the softmax the row warps form two groups that
// take alternate groups of two heads, one thread per (token, head): no exchange between threads, and one group's
// exponentials overlap the other group's value mix.  Elsewhere four threads share a token, a quarter of the columns each.
#include "lime_common.cuh"
#include "tc_common.cuh"

namespace lime {

constexpr int HC_D = 256, HC_F = 256, HC_TILE = 128, HC_ELL = 64;
constexpr int HC_PARTS = 4, HC_ROW_WARPS = 4 * HC_PARTS, HC_THREADS = 64 + 32 * HC_ROW_WARPS;
constexpr int HC_RING = 3;
constexpr uint32_t HC_SUB = 128 * 128;                          // bytes of one [128 rows x 64 bf16] swizzled sub-tile
constexpr uint32_t HC_SLAB = 2 * HC_SUB;                        // one ring slot: [256 rows x 64 bf16]
constexpr uint32_t HC_OFF_XO = 0;                               // token tile, then P of two groups, then O: 4 K-blocks
constexpr uint32_t HC_OFF_PU = HC_OFF_XO + 4 * HC_SUB;          // V[T]^T [256 features x 64 links], later U: 2 K-blocks
constexpr uint32_t HC_OFF_RING = HC_OFF_PU + 2 * HC_SUB;
constexpr uint32_t HC_OFF_EXCH = HC_OFF_RING + HC_RING * HC_SLAB;     // [2 parities][PARTS][128] float2
constexpr uint32_t HC_OFF_INV = HC_OFF_EXCH + 2 * HC_PARTS * 128 * 8; // [8 heads][128 rows] 1 / softmax row sum
constexpr uint32_t HC_OFF_BAR = HC_OFF_INV + 8 * 128 * 4;
constexpr int HC_IDX_CAP = 1025;                                // users + 1 whose offsets are staged in shared memory
constexpr uint32_t HC_OFF_IDX = HC_OFF_BAR + 512;
constexpr uint32_t HC_SMEM = HC_OFF_IDX + 2 * HC_IDX_CAP * 4 + 8;
static_assert(HC_SMEM <= 232448, "shared memory budget of one CTA");

struct HistUpdate256Params {
  __nv_bfloat16* out;            // [total x d]
  const int32_t* off;            // [B+1]
  const int32_t* tile_start;     // [B+1] prefix of per-user tile counts (tile = 128 tokens)
  int B, H, HL, NG, shared, out_ln;   // NG = HL / 128 groups of two heads
  int silu;                      // 1: P = SiLU(scores) / ell (Algorithm 2) instead of the per-head softmax
  float ln_eps;
  int* err;
};

__device__ __forceinline__ uint32_t hc_chunk(uint32_t r, uint32_t c) { return r * 128u + ((c ^ (r & 7u)) << 4); }
__device__ __forceinline__ uint32_t hc_pack(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float hc_tanh(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float hc_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ bool hc_group_sync(uint64_t* bar, uint32_t& uses, int lane, int* err, int where) {
  __syncwarp();
  if (lane == 0) tc::mbar_arrive(bar);
  const bool ok = tc::mbar_wait(bar, uses & 1u, err, where);
  ++uses;
  return ok;
}
struct HcTileUser {
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

__global__ void __launch_bounds__(HC_THREADS, 1)
k_hist_update_d256_tc(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmK2,
                      const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmWgu,
                      const __grid_constant__ CUtensorMap tmWo, const HistUpdate256Params p) {
  using namespace tc;
  extern __shared__ __align__(1024) uint8_t smem[];
  if ((smem_u32(smem) & 1023u) != 0) {
    if (threadIdx.x == 0) atomicCAS(p.err, 0, 96);
    return;
  }
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + HC_OFF_BAR);
  uint64_t* full = bars;              // [HC_RING] operand slab landed
  uint64_t* empty = bars + 3;         // [HC_RING] the MMAs that read the slab have run
  uint64_t* x_full = bars + 6;        // per tile
  uint64_t* x_free = bars + 7;        // per tile: the last contraction that reads the X / P / O buffer has run
  uint64_t* v_full = bars + 8;        // per tile: V[T]^T of the tile's user landed
  uint64_t* pu_free = bars + 9;       // per tile: every row warp is done with its patch of the V / U buffer (16 warps)
  uint64_t* s_full = bars + 10;       // [2] per tile: scores of heads 0-3 / 4-7 in TMEM
  uint64_t* p_ready = bars + 12;      // [2] per group, by row-warp group: P_c in smem (8 warps)
  uint64_t* pv_done = bars + 14;      // [2] per group: value mix done (that P buffer free)
  uint64_t* o_full = bars + 16;       // per tile: O complete in TMEM
  uint64_t* o_ready = bars + 17;      // per tile: O as bf16 in smem (16 warps)
  uint64_t* gu_full = bars + 18;      // per (tile, half): [gate | up] complete
  uint64_t* u_ready = bars + 19;      // per (tile, half): U in smem, [gate | up] read (16 warps)
  uint64_t* sp_full = bars + 20;      // per tile: S' complete
  uint64_t* sp_read = bars + 21;      // per tile: S' read out of TMEM (16 warps)
  uint64_t* row_bar = bars + 22;      // [4] rendezvous of the four warps sharing a TMEM lane quarter
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 26);
  static_assert(HC_RING == 3, "barrier table above");

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_tiles_all = p.tile_start[p.B];
  const int t_begin = (int)(((int64_t)blockIdx.x * n_tiles_all) / gridDim.x);
  const int t_end = (int)(((int64_t)(blockIdx.x + 1) * n_tiles_all) / gridDim.x);
  const int n = t_end - t_begin;
  const int NG = p.NG;                                       // groups of two heads
  const int d_h = HC_D / p.H;
  const int n_sg = (p.HL + 255) / 256;                       // score contractions per tile (four heads each)
  const int sc_boxes = p.HL >= 256 ? 2 : 1;                  // 128-row boxes of K2 per score slab

  if (threadIdx.x == 0) {
    for (int i = 0; i < HC_RING; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    mbar_init(x_full, 1); mbar_init(x_free, 1); mbar_init(v_full, 1); mbar_init(pu_free, HC_ROW_WARPS);
    for (int i = 0; i < 2; ++i) { mbar_init(&s_full[i], 1); mbar_init(&p_ready[i], HC_ROW_WARPS / 2); mbar_init(&pv_done[i], 1); }
    mbar_init(o_full, 1); mbar_init(o_ready, HC_ROW_WARPS); mbar_init(gu_full, 1); mbar_init(u_ready, HC_ROW_WARPS);
    mbar_init(sp_full, 1); mbar_init(sp_read, HC_ROW_WARPS);
    for (int i = 0; i < 4; ++i) mbar_init(&row_bar[i], HC_PARTS);
    fence_barrier_init();
    prefetch_tmap(&tmX); prefetch_tmap(&tmK2); prefetch_tmap(&tmV); prefetch_tmap(&tmWgu); prefetch_tmap(&tmWo);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  const int32_t* tile_start = p.tile_start;
  const int32_t* off = p.off;
  if (p.B + 1 <= HC_IDX_CAP) {
    int32_t* idx = reinterpret_cast<int32_t*>(smem + HC_OFF_IDX);
    for (int i = threadIdx.x; i <= p.B; i += HC_THREADS) { idx[i] = p.tile_start[i]; idx[HC_IDX_CAP + i] = p.off[i]; }
    tile_start = idx;
    off = idx + HC_IDX_CAP;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0 && n > 0) {
      const uint64_t pol_stream = policy_evict_first(), pol_keep = policy_evict_last();
      bool ok = true;
      int g = 0, sl = 0;
      bool v_sent = false;
      // one ring slab: one or two boxes of 128 rows at contraction offset x
      auto slab = [&](const CUtensorMap* m, int x, int y0, int y1, int boxes) -> bool {
        const int s = sl % HC_RING;
        if (!mbar_wait(&empty[s], ((uint32_t)(sl / HC_RING) & 1u) ^ 1u, p.err, 11)) return false;
        mbar_arrive_expect_tx(&full[s], (uint32_t)boxes * HC_SUB);
        tma_load_2d_hint(smem + HC_OFF_RING + s * HC_SLAB, m, x, y0, &full[s], pol_keep);
        if (boxes == 2) tma_load_2d_hint(smem + HC_OFF_RING + s * HC_SLAB + HC_SUB, m, x, y1, &full[s], pol_keep);
        ++sl;
        return true;
      };
      HcTileUser tu;
      for (; g < n && ok; ++g) {
        const int t = t_begin + g;
        const int b = tu.of(tile_start, p.B, t);
        const int urow = p.shared ? 0 : b;
        auto k2_slab = [&](int sg, int kb) -> bool {
          const int y = urow * p.HL + sg * 256;
          return slab(&tmK2, kb * 64, y, y + 128, sc_boxes);
        };
        // Operand slabs go out in the order of use.  The first K2 slab is requested BEFORE the wait for the X buffer: it
        // only needs a free ring slot, so it travels while the previous tile is still being finished.
        ok = k2_slab(0, 0);
        if (!ok) break;
        // the X / P / O buffer is free once the previous tile's last contraction over O has run
        if (g > 0 && !mbar_wait(x_free, (uint32_t)(g - 1) & 1u, p.err, 12)) { ok = false; break; }
        const int row0 = off[b] + (t - tu.lo) * HC_TILE;
        mbar_arrive_expect_tx(x_full, 4 * HC_SUB);
        for (int kb = 0; kb < 4; ++kb) tma_load_2d_hint(smem + HC_OFF_XO + kb * HC_SUB, &tmX, kb * 64, row0, x_full, pol_stream);
        for (int kb = 1; kb < 4 && ok; ++kb) ok = k2_slab(0, kb);
        for (int sg = 1; sg < n_sg && ok; ++sg)
          for (int kb = 0; kb < 4 && ok; ++kb) ok = k2_slab(sg, kb);
        if (!ok) break;
        // the user's link values go where U of the previous tile was and where its rows left through
        if (g > 0 && !mbar_wait(pu_free, (uint32_t)(g - 1) & 1u, p.err, 13)) { ok = false; break; }
        mbar_arrive_expect_tx(v_full, 2 * HC_SUB);
        tma_load_2d_hint(smem + HC_OFF_PU, &tmV, 0, urow * HC_D, v_full, pol_keep);
        v_sent = true;
        // then per half of the hidden columns the gate and up columns of W_g / W_u (contraction over d) and that half's
        // rows of W_o (all output columns)
        for (int hf = 0; hf < 2 && ok; ++hf) {
          if (hf == 1)
            for (int kb = 0; kb < 2 && ok; ++kb) ok = slab(&tmWo, kb * 64, 0, 128, 2);             // S'(0): hidden columns 0..127
          for (int kb = 0; kb < 4 && ok; ++kb) ok = slab(&tmWgu, kb * 64, hf * 128, HC_F + hf * 128, 2);
        }
        for (int kb = 0; kb < 2 && ok; ++kb) ok = slab(&tmWo, 128 + kb * 64, 0, 128, 2);           // S'(1): hidden columns 128..255
      }
      if (!ok || *(volatile int*)p.err != 0) {
        // giving up: let the copies already issued land (bounded) before this CTA's shared memory goes away
        const int gl = g < n ? g : n - 1;
        if (g > 0 || sl > 0) mbar_wait_quiet(x_full, (uint32_t)gl & 1u);
        if (v_sent) mbar_wait_quiet(v_full, (uint32_t)gl & 1u);
        for (int j = 0; j < sl && j < HC_RING; ++j) mbar_wait_quiet(&full[(sl - 1 - j) % HC_RING], (uint32_t)((sl - 1 - j) / HC_RING) & 1u);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && n > 0) {
      constexpr uint32_t idesc_256 = make_idesc_bf16(128, 256);
      const uint32_t idesc_sc = p.HL >= 256 ? idesc_256 : make_idesc_bf16(128, 128);
      const uint32_t idesc_v = make_idesc_bf16(128, d_h);
      const uint32_t sbase = smem_u32(smem);
      const uint32_t xo = sbase + HC_OFF_XO, pu = sbase + HC_OFF_PU;
      bool ok = true;
      int sl = 0;
      uint32_t p_uses[2] = {0u, 0u};
      // one operand slab (64 of the contraction index): D[128 x N] (+)= A_kblock . slab^T
      auto slab_mma = [&](uint32_t d_col, uint32_t a_kblock, uint32_t idesc, bool first) -> bool {
        const int s = sl % HC_RING;
        if (!mbar_wait(&full[s], (uint32_t)(sl / HC_RING) & 1u, p.err, 22)) return false;
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < 4; ++k)
          mma_bf16_ss(tmem_base + d_col, make_sdesc_k_sw128(a_kblock + k * 32), make_sdesc_k_sw128(sbase + HC_OFF_RING + s * HC_SLAB + k * 32),
                      idesc, (first && k == 0) ? 0u : 1u);
        mma_commit(&empty[s]);
        ++sl;
        return true;
      };
      for (int g = 0; g < n && ok; ++g) {
        const uint32_t R0 = (uint32_t)(g & 1) * 256u, R1 = 256u - R0;
        if (!mbar_wait(x_full, (uint32_t)g & 1u, p.err, 23)) break;
        // 1. scores.  R0 was [gate | up] of the previous tile (u_ready waited); R1 was its S'.
        for (int kb = 0; kb < 4 && ok; ++kb) ok = slab_mma(R0, xo + kb * HC_SUB, idesc_sc, kb == 0);
        if (!ok) break;
        mma_commit(&s_full[0]);
        if (g > 0 && !mbar_wait(sp_read, (uint32_t)(g - 1) & 1u, p.err, 26)) break;
        tc_fence_after();
        if (n_sg == 2) {
          for (int kb = 0; kb < 4 && ok; ++kb) ok = slab_mma(R1, xo + kb * HC_SUB, idesc_256, kb == 0);
          if (!ok) break;
          mma_commit(&s_full[1]);
        }
        if (!mbar_wait(v_full, (uint32_t)g & 1u, p.err, 28)) break;
        // 2. value mix, head by head: O[:, head] = P_head . V_head  (contraction over the 64 links of the head).  The O
        //    columns of group c lie inside score columns that groups <= c / 2 held, all consumed once P_c exists and the
        //    groups are taken in order.
        for (int c = 0; c < NG && ok; ++c) {
          const int rg = c & 1;
          if (!mbar_wait(&p_ready[rg], p_uses[rg] & 1u, p.err, 24)) { ok = false; break; }
          ++p_uses[rg];
          tc_fence_after();
          for (int hl = 0; hl < 2; ++hl) {
            const int h = c * 2 + hl;
            for (int kk = 0; kk < 4; ++kk)
              mma_bf16_ss(tmem_base + R0 + (uint32_t)(h * d_h), make_sdesc_k_sw128(xo + (uint32_t)(rg * 2 + hl) * HC_SUB + kk * 32),
                          make_sdesc_k_sw128(pu + (uint32_t)(h * d_h) * 128 + kk * 32), idesc_v, kk != 0);
          }
          mma_commit(&pv_done[rg]);
          if (c == NG - 1) mma_commit(o_full);
        }
        if (!ok) break;
        // 3. GatedMLP on O (bf16 in the X / P / O buffer), the hidden columns in two halves
        if (!mbar_wait(o_ready, (uint32_t)g & 1u, p.err, 25)) break;
        tc_fence_after();
        for (int hf = 0; hf < 2 && ok; ++hf) {
          if (hf == 1) {
            // S' = U(0) . W_o[0..127, :] first: it frees the U buffer for the second half
            for (int kb = 0; kb < 2 && ok; ++kb) ok = slab_mma(R0, pu + kb * HC_SUB, idesc_256, kb == 0);
          }
          for (int kb = 0; kb < 4 && ok; ++kb) ok = slab_mma(R1, xo + kb * HC_SUB, idesc_256, kb == 0);
          if (!ok) break;
          mma_commit(gu_full);
          if (hf == 1) mma_commit(x_free);
          if (!mbar_wait(u_ready, (uint32_t)(2 * g + hf) & 1u, p.err, 27)) { ok = false; break; }
          tc_fence_after();
        }
        if (!ok) break;
        for (int kb = 0; kb < 2 && ok; ++kb) ok = slab_mma(R0, pu + kb * HC_SUB, idesc_256, false);
        if (!ok) break;
        mma_commit(sp_full);
      }
    }
  } else if (n > 0) {
    // ------------------------------------------------------------------ token-row warps (2..17)
    const int rw = warp - 2;                                 // 0..15
    const int q4 = warp & 3;                                 // TMEM lane quarter of this warp
    const int part = rw >> 2;                                // which quarter of the columns of every step
    const int rg = part >> 1, hh = part & 1;                 // softmax: row-warp group, head within a group of two
    const uint32_t r = (uint32_t)(q4 * 32 + lane);           // token row of the tile == TMEM lane
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q4 * 32) << 16);
    float2* exch = reinterpret_cast<float2*>(smem + HC_OFF_EXCH);         // [2][PARTS][128]
    float* inv_sum = reinterpret_cast<float*>(smem + HC_OFF_INV);         // [8][128]
    uint8_t* p_head = smem + HC_OFF_XO + (uint32_t)(rg * 2 + hh) * HC_SUB;   // P of this thread's head: one K-block
    uint8_t* pu_part = smem + HC_OFF_PU + (part >> 1) * HC_SUB;           // U: K-block part / 2, chunks (part % 2) * 4 ..
    const uint32_t pu_chunk0 = (uint32_t)(part & 1) * 4;
    uint32_t row_uses = 0, my_p = 0;
    bool ok = true;
    HcTileUser tu;
    for (int g = 0; g < n && ok; ++g) {
      const int t = t_begin + g;
      const int b = tu.of(tile_start, p.B, t);
      const int row0 = off[b] + (t - tu.lo) * HC_TILE;
      const uint32_t R0 = (uint32_t)(g & 1) * 256u, R1 = 256u - R0;
      // ---- this row-warp group's groups of two heads: softmax over the 64 links of this thread's head, P_c -> smem
      for (int c = rg; c < NG && ok; c += 2, ++my_p) {
        const int sg = c >> 1;
        if (!mbar_wait(&s_full[sg], (uint32_t)g & 1u, p.err, 32)) { ok = false; break; }
        tc_fence_after();
        const uint32_t col = lane_addr + (sg ? R1 : R0) + (uint32_t)(c & 1) * 128u + (uint32_t)hh * 64u;
        float v[32];
        float mx = 0.f, sum = 0.f;
        if (!p.silu) {
          tmem_ld_32x32(col, v);
          tmem_wait_ld();
          mx = v[0];
#pragma unroll
          for (int j = 1; j < 32; ++j) mx = fmaxf(mx, v[j]);
          tmem_ld_32x32(col + 32, v);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j) mx = fmaxf(mx, v[j]);
        }
        // the P buffers lie over the token tile: every score contraction of the tile must have read it, and the value mix
        // that read this buffer last must have run
        if (!mbar_wait(&s_full[n_sg - 1], (uint32_t)g & 1u, p.err, 35)) { ok = false; break; }
        if (my_p > 0 && !mbar_wait(&pv_done[rg], (my_p - 1) & 1u, p.err, 36)) { ok = false; break; }
#pragma unroll
        for (int hv = 0; hv < 2; ++hv) {
          tmem_ld_32x32(col + hv * 32, v);
          tmem_wait_ld();
          if (p.silu) {
            // SiLU(s) / ell: every history query attends to the ell links of the head (Algorithm 1)
#pragma unroll
            for (int j = 0; j < 32; ++j) { const float hx = 0.5f * v[j]; v[j] = fmaf(hx, hc_tanh(hx), hx) * (1.0f / HC_ELL); }
          } else {
            float s0 = 0.f, s1 = 0.f;
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
              v[j] = hc_ex2(v[j] - mx);
              v[j + 1] = hc_ex2(v[j + 1] - mx);
              s0 += v[j];
              s1 += v[j + 1];
            }
            sum += s0 + s1;
          }
#pragma unroll
          for (int c8 = 0; c8 < 4; ++c8) {
            uint4 o;
            o.x = hc_pack(v[c8 * 8 + 0], v[c8 * 8 + 1]); o.y = hc_pack(v[c8 * 8 + 2], v[c8 * 8 + 3]);
            o.z = hc_pack(v[c8 * 8 + 4], v[c8 * 8 + 5]); o.w = hc_pack(v[c8 * 8 + 6], v[c8 * 8 + 7]);
            *reinterpret_cast<uint4*>(p_head + hc_chunk(r, (uint32_t)(hv * 4 + c8))) = o;
          }
        }
        // the exponentials go to the value mix unnormalised; O is divided by the row sum of its head afterwards
        inv_sum[(c * 2 + hh) * 128 + (int)r] = p.silu ? 1.0f : __fdividef(1.0f, sum);
        tc_fence_before();
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_ready[rg]);
      }
      if (!ok) break;
      // ---- O: this thread's 64 columns / row sum of their heads -> bf16 -> K-block `part` of the X / P / O buffer
      if (!mbar_wait(o_full, (uint32_t)g & 1u, p.err, 33)) { ok = false; break; }
      tc_fence_after();
#pragma unroll
      for (int c = 0; c < 64; c += 32) {
        float a[32];
        tmem_ld_32x32(lane_addr + R0 + part * 64 + c, a);
        const float sc = inv_sum[((part * 64 + c) / d_h) * 128 + (int)r];
        tmem_wait_ld();
#pragma unroll
        for (int c8 = 0; c8 < 4; ++c8) {
          uint4 o;
          o.x = hc_pack(a[c8 * 8 + 0] * sc, a[c8 * 8 + 1] * sc); o.y = hc_pack(a[c8 * 8 + 2] * sc, a[c8 * 8 + 3] * sc);
          o.z = hc_pack(a[c8 * 8 + 4] * sc, a[c8 * 8 + 5] * sc); o.w = hc_pack(a[c8 * 8 + 6] * sc, a[c8 * 8 + 7] * sc);
          *reinterpret_cast<uint4*>(smem + HC_OFF_XO + part * HC_SUB + hc_chunk(r, (uint32_t)(c >> 3) + c8)) = o;
        }
      }
      tc_fence_before();
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(o_ready);
      // ---- per half of the hidden columns: U = SiLU(gate) * up for this thread's 32 columns -> smem
      for (int hf = 0; hf < 2 && ok; ++hf) {
        if (!mbar_wait(gu_full, (uint32_t)(2 * g + hf) & 1u, p.err, 34)) { ok = false; break; }
        tc_fence_after();
        float gt[32], up[32];
        tmem_ld_32x32(lane_addr + R1 + part * 32, gt);
        tmem_ld_32x32(lane_addr + R1 + 128 + part * 32, up);
        tmem_wait_ld();
#pragma unroll
        for (int c8 = 0; c8 < 4; ++c8) {
          float y[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float hx = 0.5f * gt[c8 * 8 + j];
            y[j] = fmaf(hx, hc_tanh(hx), hx) * up[c8 * 8 + j];
          }
          uint4 o;
          o.x = hc_pack(y[0], y[1]); o.y = hc_pack(y[2], y[3]); o.z = hc_pack(y[4], y[5]); o.w = hc_pack(y[6], y[7]);
          *reinterpret_cast<uint4*>(pu_part + hc_chunk(r, pu_chunk0 + (uint32_t)c8)) = o;
        }
        tc_fence_before();
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(u_ready);
      }
      if (!ok) break;
      // ---- S': this thread's 64 columns of its row -> (LayerNorm) -> bf16 -> global, straight from registers
      if (!mbar_wait(sp_full, (uint32_t)g & 1u, p.err, 37)) { ok = false; break; }
      tc_fence_after();
      float a0[32], a1[32];
      tmem_ld_32x32(lane_addr + R0 + part * 64, a0);
      tmem_ld_32x32(lane_addr + R0 + part * 64 + 32, a1);
      tmem_wait_ld();
      // S' is in registers: the columns may take the next tile's value mix while this tile is normalised and stored
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(sp_read);
      float mu = 0.f, rstd = 1.f;
      if (p.out_ln) {
        // each quarter sends the mean of its 64 columns and their squared deviations from it; the four combine exactly
        float s = 0.f;
#pragma unroll
        for (int j = 0; j < 32; ++j) s += a0[j] + a1[j];
        const float m_q = s * (1.0f / 64);
        float m2 = 0.f;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float d0 = a0[j] - m_q, d1 = a1[j] - m_q;
          m2 = fmaf(d0, d0, m2);
          m2 = fmaf(d1, d1, m2);
        }
        float2* ex = exch + (row_uses & 1u) * (HC_PARTS * 128);
        ex[part * 128 + r] = make_float2(m_q, m2);
        if (!hc_group_sync(&row_bar[q4], row_uses, lane, p.err, 38)) { ok = false; break; }
        float2 e[HC_PARTS];
#pragma unroll
        for (int i = 0; i < HC_PARTS; ++i) e[i] = ex[i * 128 + r];
        mu = 0.25f * (e[0].x + e[1].x + e[2].x + e[3].x);
        float tot = 0.f;
#pragma unroll
        for (int i = 0; i < HC_PARTS; ++i) { const float dm = e[i].x - mu; tot += e[i].y + 64.0f * dm * dm; }
        rstd = rsqrtf(tot * (1.0f / HC_D) + p.ln_eps);
      }
      // Out through a 2 KB patch of the V / U buffer that belongs to this warp alone (S' has consumed U): the warp stages
      // 32 columns of its 32 rows (row R at R * 64 bytes, 16-byte chunk c at position c ^ ((R >> 1) & 3): conflict-free
      // both ways), then writes them with four lanes per row, 64 contiguous bytes each.  Only the warp itself has to
      // rendezvous.
      {
        uint8_t* patch = smem + HC_OFF_PU + (part >> 1) * HC_SUB + q4 * 4096 + (part & 1) * 2048;
        const int row_end = off[b + 1];
        const uint32_t rr = (uint32_t)lane >> 2, rc = (uint32_t)lane & 3u;
#pragma unroll
        for (int hcol = 0; hcol < 2; ++hcol) {
          const float* a = hcol ? a1 : a0;
#pragma unroll
          for (int c8 = 0; c8 < 4; ++c8) {
            uint4 o;
            o.x = hc_pack((a[c8 * 8 + 0] - mu) * rstd, (a[c8 * 8 + 1] - mu) * rstd);
            o.y = hc_pack((a[c8 * 8 + 2] - mu) * rstd, (a[c8 * 8 + 3] - mu) * rstd);
            o.z = hc_pack((a[c8 * 8 + 4] - mu) * rstd, (a[c8 * 8 + 5] - mu) * rstd);
            o.w = hc_pack((a[c8 * 8 + 6] - mu) * rstd, (a[c8 * 8 + 7] - mu) * rstd);
            *reinterpret_cast<uint4*>(patch + lane * 64 + (((uint32_t)c8 ^ (((uint32_t)lane >> 1) & 3u)) << 4)) = o;
          }
          __syncwarp();
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const uint32_t R = (uint32_t)i * 8 + rr;
            const uint4 o = *reinterpret_cast<const uint4*>(patch + R * 64 + ((rc ^ ((R >> 1) & 3u)) << 4));
            const int grow = row0 + q4 * 32 + (int)R;
            if (grow < row_end)
              *reinterpret_cast<uint4*>(p.out + (int64_t)grow * HC_D + part * 64 + hcol * 32 + rc * 8) = o;
          }
          __syncwarp();
        }
      }
      // the V / U buffer may take the next tile's link values
      if (lane == 0) mbar_arrive(pu_free);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

bool hist_update_d256_tc_supported(int dtype, int d, int f, int H, int ell, int phi, int gated_mlp) {
  return dtype == LIME_BF16 && d == HC_D && f == HC_F && ell == HC_ELL && (H == 2 || H == 4 || H == 8) &&
         (phi == LIME_PHI_SOFTMAX || phi == LIME_PHI_SILU) && gated_mlp != 0;
}

lime_status launch_hist_update_d256_tc(const HistUpdate256Args& a, cudaStream_t st) {
  if (a.total == 0) return LIME_OK;
  const int HL = a.H * HC_ELL;
  CUtensorMap tmX, tmK2, tmV, tmWgu, tmWo;
  const uint64_t users = a.shared ? 1 : (uint64_t)a.B;
  if (!make_tmap_bf16_sw128(&tmX, a.hist_in, (uint64_t)a.total, HC_D, HC_D, HC_TILE) ||
      !make_tmap_bf16_sw128(&tmK2, a.K2, users * HL, HC_D, HC_D, 128) ||
      !make_tmap_bf16_sw128(&tmV, a.V2t, users * HC_D, HC_ELL, HC_ELL, 256) ||
      !make_tmap_bf16_sw128(&tmWgu, a.WguT, 2 * HC_F, HC_D, HC_D, 128) ||
      !make_tmap_bf16_sw128(&tmWo, a.WoT, HC_D, HC_F, HC_F, 128))
    return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
  HistUpdate256Params p;
  p.out = (__nv_bfloat16*)a.hist_out; p.off = a.off; p.tile_start = a.tile_start; p.B = a.B; p.H = a.H; p.HL = HL;
  p.NG = HL / 128; p.shared = a.shared; p.silu = a.silu; p.out_ln = a.out_ln; p.ln_eps = a.ln_eps; p.err = a.err;
  int grid = a.n_tile_upper < kSMs ? a.n_tile_upper : kSMs;
  if (grid < 1) return LIME_OK;
  static bool smem_set[kMaxDeviceOrdinals] = {};
  lime_status es = ensure_dynamic_smem((const void*)k_hist_update_d256_tc, (int)HC_SMEM, smem_set);
  if (es != LIME_OK) return es;
  ProfScope _p("k_hist_update_d256_tc", st);
  k_hist_update_d256_tc<<<grid, HC_THREADS, HC_SMEM, st>>>(tmX, tmK2, tmV, tmWgu, tmWo, p);
  LIME_LAUNCH_CHECK("k_hist_update_d256_tc");
  return LIME_OK;
}

}  // namespace lime
