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
//   per group c of 128 stacked (head, link) rows = 2 heads:
//     scores_c [128 x 128] = X . K2_c^T            -> per-head softmax over the 64 links (or SiLU(s) / 64) -> P_c (bf16)
//     O[:, head]           = P_head [128 x 64] . V_head [64 x d_h]          (both heads of the group)
//   O -> bf16 (over the X tile, which nothing reads any more)
//   per half hf of the hidden columns:   [gate | up] = O . [W_g | W_u][:, hf]  ->  U = SiLU(gate) * up (bf16)
//                                        S' (+)= U . W_o[hf rows, :]
//   S' -> (LayerNorm) -> bf16 -> whole rows to global memory
// TMEM (512 columns): [0, 256) two score buffers, later [gate | up] of one half; [256, 512) O, later S'.
// Shared memory: X / O tile 64 KB, P / U 32 KB, and a ring of seven 16 KB operand slabs ([128 rows x 64
// of the contraction index]) through which K2, the link values of each group of two heads, W_g, W_u and W_o stream from
// L2 in the order the MMA issuer consumes them (44 slabs per tile with 8 heads).  What bounds the kernel is how many
// operand bytes are in flight from L2 per SM, so everything that is not the token tile or the P / U buffer is ring.
// Warp 0 TMA producer, warp 1 MMA issuer, warps 2-17 token rows: four threads per token (TMEM lane), a quarter of the
// columns of every step each; the two threads that share a head of the softmax exchange (max, sum) once per group.
#include "lime_common.cuh"
#include "tc_common.cuh"

namespace lime {

constexpr int HC_D = 256, HC_F = 256, HC_TILE = 128, HC_ELL = 64;
constexpr int HC_PARTS = 4, HC_ROW_WARPS = 4 * HC_PARTS, HC_THREADS = 64 + 32 * HC_ROW_WARPS;
constexpr int HC_RING = 7;
constexpr uint32_t HC_SUB = 128 * 128;                          // bytes of one [128 rows x 64 bf16] swizzled sub-tile
constexpr uint32_t HC_OFF_XO = 0;                               // token tile, later O: 4 K-blocks
constexpr uint32_t HC_OFF_PU = HC_OFF_XO + 4 * HC_SUB;          // P_c, later U: 2 K-blocks
constexpr uint32_t HC_OFF_RING = HC_OFF_PU + 2 * HC_SUB;
constexpr uint32_t HC_OFF_EXCH = HC_OFF_RING + HC_RING * HC_SUB;      // [2 parities][PARTS][128] float2
constexpr uint32_t HC_OFF_BAR = HC_OFF_EXCH + 2 * HC_PARTS * 128 * 8;
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
  uint64_t* empty = bars + 7;         // [HC_RING] the MMAs that read the slab have run
  uint64_t* x_full = bars + 14;       // per tile
  uint64_t* x_free = bars + 15;       // per tile: the last contraction that reads the X / O buffer has run
  uint64_t* s_full = bars + 16;       // [2] per group, by parity of the group counter: scores in TMEM
  uint64_t* p_ready = bars + 18;      // per group: P_c in smem (16 warps)
  uint64_t* pv_done = bars + 19;      // per group: value mix done (P buffer free)
  uint64_t* o_full = bars + 20;       // per tile: O complete in TMEM
  uint64_t* o_ready = bars + 21;      // per tile: O as bf16 in smem (16 warps)
  uint64_t* gu_full = bars + 22;      // per (tile, half): [gate | up] complete
  uint64_t* u_ready = bars + 23;      // per (tile, half): U in smem, [gate | up] read (16 warps)
  uint64_t* sp_full = bars + 24;      // per tile: S' complete
  uint64_t* sp_read = bars + 25;      // per tile: S' read out (16 warps)
  uint64_t* row_bar = bars + 27;      // [4] rendezvous of the four warps sharing a TMEM lane quarter
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 31);
  static_assert(HC_RING == 7, "barrier table above");

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_tiles_all = p.tile_start[p.B];
  const int t_begin = (int)(((int64_t)blockIdx.x * n_tiles_all) / gridDim.x);
  const int t_end = (int)(((int64_t)(blockIdx.x + 1) * n_tiles_all) / gridDim.x);
  const int n = t_end - t_begin;
  const int NG = p.NG;
  const int d_h = HC_D / p.H;
  // link values of a group of two heads: 2 * d_h feature rows of V[T]^T, in slabs of up to 128 rows
  const int v_rows = 2 * d_h < 128 ? 2 * d_h : 128;
  const int v_slabs = (2 * d_h + 127) / 128;

  if (threadIdx.x == 0) {
    for (int i = 0; i < HC_RING; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    mbar_init(x_full, 1); mbar_init(x_free, 1);
    mbar_init(&s_full[0], 1); mbar_init(&s_full[1], 1); mbar_init(p_ready, HC_ROW_WARPS); mbar_init(pv_done, 1);
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
  constexpr uint32_t COL_SC = 0, COL_GU = 0, COL_O = 256, COL_SP = 256;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0 && n > 0) {
      const uint64_t pol_stream = policy_evict_first(), pol_keep = policy_evict_last();
      bool ok = true;
      int g = 0, sl = 0;
      auto slab_n = [&](const CUtensorMap* m, int x, int y, uint32_t bytes) -> bool {
        const int s = sl % HC_RING;
        if (!mbar_wait(&empty[s], ((uint32_t)(sl / HC_RING) & 1u) ^ 1u, p.err, 11)) return false;
        mbar_arrive_expect_tx(&full[s], bytes);
        tma_load_2d_hint(smem + HC_OFF_RING + s * HC_SUB, m, x, y, &full[s], pol_keep);
        ++sl;
        return true;
      };
      auto slab = [&](const CUtensorMap* m, int x, int y) -> bool { return slab_n(m, x, y, HC_SUB); };
      HcTileUser tu;
      for (; g < n && ok; ++g) {
        const int t = t_begin + g;
        const int b = tu.of(tile_start, p.B, t);
        const int urow = p.shared ? 0 : b;
        auto k2_group = [&](int c) {
          for (int kb = 0; kb < 4 && ok; ++kb) ok = slab(&tmK2, kb * 64, urow * p.HL + c * 128);
        };
        // Operand slabs go out in the order of use.  The first group's K2 slabs are requested BEFORE the wait for the
        // X / O buffer: they only need free ring slots (which the previous tile's last contractions release one by one),
        // so they travel while that tile is still being finished and stored.
        k2_group(0);
        if (!ok) break;
        // the X / O buffer is free once the previous tile's last contraction over O has run
        if (g > 0 && !mbar_wait(x_free, (uint32_t)(g - 1) & 1u, p.err, 12)) { ok = false; break; }
        const int row0 = off[b] + (t - tu.lo) * HC_TILE;
        mbar_arrive_expect_tx(x_full, 4 * HC_SUB);
        for (int kb = 0; kb < 4; ++kb) tma_load_2d_hint(smem + HC_OFF_XO + kb * HC_SUB, &tmX, kb * 64, row0, x_full, pol_stream);
        // per group: the next group's K2 (its scores are formed under this group's softmax), then this group's values
        for (int c = 0; c < NG && ok; ++c) {
          if (c + 1 < NG) k2_group(c + 1);
          for (int j = 0; j < v_slabs && ok; ++j)
            ok = slab_n(&tmV, 0, urow * HC_D + c * 2 * d_h + j * 128, (uint32_t)v_rows * 128u);
        }
        // then per half of the hidden columns the gate and up columns of W_g / W_u (contraction over d) and that half's
        // rows of W_o (both halves of the output columns)
        for (int hf = 0; hf < 2 && ok; ++hf) {
          if (hf == 1) {
            for (int nh = 0; nh < 2 && ok; ++nh)
              for (int kb = 0; kb < 2 && ok; ++kb) ok = slab(&tmWo, kb * 64, nh * 128);            // S'(0): hidden columns 0..127
          }
          for (int kb = 0; kb < 4 && ok; ++kb) {
            ok = slab(&tmWgu, kb * 64, hf * 128);
            ok = ok && slab(&tmWgu, kb * 64, HC_F + hf * 128);
          }
        }
        for (int nh = 0; nh < 2 && ok; ++nh)
          for (int kb = 0; kb < 2 && ok; ++kb) ok = slab(&tmWo, 128 + kb * 64, nh * 128);          // S'(1): hidden columns 128..255
      }
      if (!ok || *(volatile int*)p.err != 0) {
        // giving up: let the copies already issued land (bounded) before this CTA's shared memory goes away
        if (g > 0 || sl > 0) mbar_wait_quiet(x_full, (uint32_t)(g < n ? g : n - 1) & 1u);
        for (int j = 0; j < sl && j < HC_RING; ++j) mbar_wait_quiet(&full[(sl - 1 - j) % HC_RING], (uint32_t)((sl - 1 - j) / HC_RING) & 1u);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && n > 0) {
      constexpr uint32_t idesc_128 = make_idesc_bf16(128, 128);
      const uint32_t idesc_v = make_idesc_bf16(128, d_h);
      const uint32_t sbase = smem_u32(smem);
      const uint32_t xo = sbase + HC_OFF_XO, pu = sbase + HC_OFF_PU;
      bool ok = true;
      int sl = 0, q = 0;
      // one operand slab (64 of the contraction index): D[128 x 128] (+)= A_kblock . slab^T
      auto slab_mma = [&](uint32_t d_col, uint32_t a_kblock, bool first) -> bool {
        const int s = sl % HC_RING;
        if (!mbar_wait(&full[s], (uint32_t)(sl / HC_RING) & 1u, p.err, 22)) return false;
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < 4; ++k)
          mma_bf16_ss(tmem_base + d_col, make_sdesc_k_sw128(a_kblock + k * 32), make_sdesc_k_sw128(sbase + HC_OFF_RING + s * HC_SUB + k * 32),
                      idesc_128, (first && k == 0) ? 0u : 1u);
        mma_commit(&empty[s]);
        ++sl;
        return true;
      };
      auto issue_scores = [&](int qq) -> bool {
        for (int kb = 0; kb < 4; ++kb)
          if (!slab_mma(COL_SC + (uint32_t)(qq & 1) * 128, xo + kb * HC_SUB, kb == 0)) return false;
        mma_commit(&s_full[qq & 1]);
        return true;
      };
      for (int g = 0; g < n && ok; ++g) {
        if (!mbar_wait(x_full, (uint32_t)g & 1u, p.err, 23)) break;
        // 1. scores of the first group (both score buffers were last read as [gate | up] of the previous tile: u_ready waited)
        if (!issue_scores(q)) { ok = false; break; }
        for (int c = 0; c < NG && ok; ++c, ++q) {
          if (c + 1 < NG && !issue_scores(q + 1)) { ok = false; break; }
          if (!mbar_wait(p_ready, (uint32_t)q & 1u, p.err, 24)) { ok = false; break; }
          // the O columns last held S' of the previous tile
          if (c == 0 && g > 0 && !mbar_wait(sp_read, (uint32_t)(g - 1) & 1u, p.err, 26)) { ok = false; break; }
          // the group's link values: one or two ring slabs
          const int sv = sl;
          for (int j = 0; j < v_slabs && ok; ++j)
            ok = mbar_wait(&full[(sv + j) % HC_RING], (uint32_t)((sv + j) / HC_RING) & 1u, p.err, 28);
          if (!ok) break;
          tc_fence_after();
          // 2. value mix, head by head: O[:, head] = P_head . V_head  (contraction over the 64 links of the head)
          for (int hl = 0; hl < 2; ++hl) {
            const int h = c * 2 + hl;
            const int fo = hl * d_h;                         // the head's first feature row among the group's rows
            const uint32_t vb = sbase + HC_OFF_RING + (uint32_t)((sv + fo / 128) % HC_RING) * HC_SUB + (uint32_t)(fo % 128) * 128u;
            for (int kk = 0; kk < 4; ++kk)
              mma_bf16_ss(tmem_base + COL_O + (uint32_t)(h * d_h), make_sdesc_k_sw128(pu + hl * HC_SUB + kk * 32),
                          make_sdesc_k_sw128(vb + kk * 32), idesc_v, kk != 0);
          }
          for (int j = 0; j < v_slabs; ++j) mma_commit(&empty[(sv + j) % HC_RING]);
          sl += v_slabs;
          mma_commit(pv_done);
          if (c == NG - 1) mma_commit(o_full);
        }
        if (!ok) break;
        // 3. GatedMLP on O (bf16 in the X / O buffer), the hidden columns in two halves
        if (!mbar_wait(o_ready, (uint32_t)g & 1u, p.err, 25)) break;
        for (int hf = 0; hf < 2 && ok; ++hf) {
          if (hf == 1) {
            // S' = U(0) . W_o[0..127, :] first: it frees the U buffer for the second half
            for (int nh = 0; nh < 2 && ok; ++nh)
              for (int kb = 0; kb < 2 && ok; ++kb) ok = slab_mma(COL_SP + (uint32_t)nh * 128, pu + kb * HC_SUB, kb == 0);
          }
          for (int kb = 0; kb < 4 && ok; ++kb) {
            ok = slab_mma(COL_GU, xo + kb * HC_SUB, kb == 0);
            ok = ok && slab_mma(COL_GU + 128, xo + kb * HC_SUB, kb == 0);
          }
          if (!ok) break;
          mma_commit(gu_full);
          if (hf == 1) mma_commit(x_free);
          if (!mbar_wait(u_ready, (uint32_t)(2 * g + hf) & 1u, p.err, 27)) { ok = false; break; }
          tc_fence_after();
        }
        if (!ok) break;
        for (int nh = 0; nh < 2 && ok; ++nh)
          for (int kb = 0; kb < 2 && ok; ++kb) ok = slab_mma(COL_SP + (uint32_t)nh * 128, pu + kb * HC_SUB, false);
        if (!ok) break;
        mma_commit(sp_full);
      }
    }
  } else if (n > 0) {
    // ------------------------------------------------------------------ token-row warps (2..17)
    const int rw = warp - 2;                                 // 0..15
    const int q4 = warp & 3;                                 // TMEM lane quarter of this warp
    const int part = rw >> 2;                                // which quarter of the columns of every step
    const uint32_t r = (uint32_t)(q4 * 32 + lane);           // token row of the tile == TMEM lane
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q4 * 32) << 16);
    float2* exch = reinterpret_cast<float2*>(smem + HC_OFF_EXCH);         // [2][PARTS][128]
    uint8_t* pu_part = smem + HC_OFF_PU + (part >> 1) * HC_SUB;           // K-block part / 2, chunks (part % 2) * 4 ..
    const uint32_t pu_chunk0 = (uint32_t)(part & 1) * 4;
    uint32_t row_uses = 0;
    int q = 0;
    bool ok = true;
    HcTileUser tu;
    for (int g = 0; g < n && ok; ++g) {
      const int t = t_begin + g;
      const int b = tu.of(tile_start, p.B, t);
      const int row0 = off[b] + (t - tu.lo) * HC_TILE;
      // ---- per group: softmax over the 64 links of a head (two threads per head), P_c -> smem
      for (int c = 0; c < NG && ok; ++c, ++q) {
        if (!mbar_wait(&s_full[q & 1], (uint32_t)(q >> 1) & 1u, p.err, 32)) { ok = false; break; }
        tc_fence_after();
        float v[32];
        tmem_ld_32x32(lane_addr + COL_SC + (uint32_t)(q & 1) * 128 + part * 32, v);
        tmem_wait_ld();
        if (p.silu) {
          // SiLU(s) / ell: every history query attends to the ell links of the head (Algorithm 1)
#pragma unroll
          for (int j = 0; j < 32; ++j) { const float hx = 0.5f * v[j]; v[j] = fmaf(hx, hc_tanh(hx), hx) * (1.0f / HC_ELL); }
        } else {
          float mx = v[0];
#pragma unroll
          for (int j = 1; j < 32; ++j) mx = fmaxf(mx, v[j]);
          float s0 = 0.f, s1 = 0.f;
#pragma unroll
          for (int j = 0; j < 32; j += 2) {
            v[j] = hc_ex2(v[j] - mx);
            v[j + 1] = hc_ex2(v[j + 1] - mx);
            s0 += v[j];
            s1 += v[j + 1];
          }
          // one exchange with the thread that holds the other half of the head
          float2* ex = exch + (row_uses & 1u) * (HC_PARTS * 128);
          ex[part * 128 + r] = make_float2(mx, s0 + s1);
          if (!hc_group_sync(&row_bar[q4], row_uses, lane, p.err, 35)) { ok = false; break; }
          const float2 other = ex[(part ^ 1) * 128 + r];
          const float M = fmaxf(mx, other.x);
          const float mine = hc_ex2(mx - M);
          const float scale = __fdividef(mine, fmaf(s0 + s1, mine, other.y * hc_ex2(other.x - M)));
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] *= scale;
        }
        // P_{q-1} must have been consumed by its value mix before the buffer is rewritten
        if (q > 0 && !mbar_wait(pv_done, (uint32_t)(q - 1) & 1u, p.err, 36)) { ok = false; break; }
#pragma unroll
        for (int c8 = 0; c8 < 4; ++c8) {
          uint4 o;
          o.x = hc_pack(v[c8 * 8 + 0], v[c8 * 8 + 1]); o.y = hc_pack(v[c8 * 8 + 2], v[c8 * 8 + 3]);
          o.z = hc_pack(v[c8 * 8 + 4], v[c8 * 8 + 5]); o.w = hc_pack(v[c8 * 8 + 6], v[c8 * 8 + 7]);
          *reinterpret_cast<uint4*>(pu_part + hc_chunk(r, pu_chunk0 + (uint32_t)c8)) = o;
        }
        tc_fence_before();
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(p_ready);
      }
      if (!ok) break;
      // ---- O: this thread's 64 columns -> bf16 -> K-block `part` of the X / O buffer (every scores MMA has run)
      if (!mbar_wait(o_full, (uint32_t)g & 1u, p.err, 33)) { ok = false; break; }
      tc_fence_after();
#pragma unroll
      for (int c = 0; c < 64; c += 32) {
        float a[32];
        tmem_ld_32x32(lane_addr + COL_O + part * 64 + c, a);
        tmem_wait_ld();
#pragma unroll
        for (int c8 = 0; c8 < 4; ++c8) {
          uint4 o;
          o.x = hc_pack(a[c8 * 8 + 0], a[c8 * 8 + 1]); o.y = hc_pack(a[c8 * 8 + 2], a[c8 * 8 + 3]);
          o.z = hc_pack(a[c8 * 8 + 4], a[c8 * 8 + 5]); o.w = hc_pack(a[c8 * 8 + 6], a[c8 * 8 + 7]);
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
        tmem_ld_32x32(lane_addr + COL_GU + part * 32, gt);
        tmem_ld_32x32(lane_addr + COL_GU + 128 + part * 32, up);
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
      tmem_ld_32x32(lane_addr + COL_SP + part * 64, a0);
      tmem_ld_32x32(lane_addr + COL_SP + part * 64 + 32, a1);
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
      // Out through a 2 KB patch of the P / U buffer that belongs to this warp alone (S' has consumed U): the warp stages
      // 32 columns of its 32 rows (row R at R * 64 bytes, 16-byte chunk c at position c ^ ((R >> 1) & 3): conflict-free
      // both ways), then writes them with four lanes per row, 64 contiguous bytes each.  Only the warp itself has to
      // rendezvous; the patch lies inside the rows of the P / U buffer that this warp and its column neighbour write.
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
      // without the softmax exchange nothing else keeps the column neighbour from writing the next P over this patch
      if (p.silu && !hc_group_sync(&row_bar[q4], row_uses, lane, p.err, 39)) { ok = false; break; }
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
  const int v_rows = 2 * (HC_D / a.H) < 128 ? 2 * (HC_D / a.H) : 128;      // value rows of one slab: a group of two heads
  if (!make_tmap_bf16_sw128(&tmX, a.hist_in, (uint64_t)a.total, HC_D, HC_D, HC_TILE) ||
      !make_tmap_bf16_sw128(&tmK2, a.K2, users * HL, HC_D, HC_D, 128) ||
      !make_tmap_bf16_sw128(&tmV, a.V2t, users * HC_D, HC_ELL, HC_ELL, v_rows) ||
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
