// History update of one XOR layer on the 5th-generation tensor cores (bf16 storage):
//
//   S'[t,:] = GatedMLP( O[S]_t ),   O[S]_t = concat_h softmax_l( Q[S]_{t,h} K[T]_{l,h}^T * scale ) V[T]_{l,h}     (Eq. 7, Eq. 5)
//
// fused per 128-token tile into three chained tensor-core contractions whose operands never leave the SM:
//   1. scores  [128 x HL]  = X_tile [128 x d] . K2^T               (K2 = folded link keys, see k_link_prep.cu)
//      LayerNorm is applied afterwards as s = rstd_t * (raw - mu_t * rowsum(K2)), exact for the bf16 operands
//   2. per-head softmax over the ell links of each token (one thread per token, registers only) -> P (bf16, smem)
//   3. [gate | up] [128 x 2f] = P [128 x HL] . [G2 | U2]           (value mix and first GatedMLP layer folded)
//   4. U = SiLU(gate) * up (bf16, smem)       5. S' = U [128 x f] . W_o [f x d]  -> bf16 rows to global
// HL = H * ell stacked (head, link) rows.  Warp roles: warp 0 TMA producer, warp 1 MMA issuer, warps 2-5 one
// thread per token row (TMEM lane).  History is read once (TMA) and written once per layer.
//
// Built for d = d_ff = 128 and H * ell = 128 (shared memory: 2 x 32 KB token stages + 160 KB of operands;
// TMEM: 128 + 256 + 128 columns).
#include "lime_common.cuh"
#include "tc_common.cuh"

namespace lime {

constexpr int HU_D = 128, HU_F = 128, HU_HL = 128, HU_TILE = 128, HU_THREADS = 192;
constexpr uint32_t HU_SUB = 128 * 128;                 // bytes of one [128 rows x 64 bf16] swizzled sub-tile
constexpr uint32_t HU_X_STAGE = 2 * HU_SUB;            // token tile: 2 K-blocks
constexpr uint32_t HU_OFF_X = 0;                       // 2 stages
constexpr uint32_t HU_OFF_K2 = 2 * HU_X_STAGE;         // [HL x d]      2 K-blocks x 16 KB
constexpr uint32_t HU_OFF_GU = HU_OFF_K2 + 2 * HU_SUB; // [2f x HL]     2 K-blocks x 32 KB (gate rows, then up rows)
constexpr uint32_t HU_OFF_WO = HU_OFF_GU + 4 * HU_SUB; // [d x f]       2 K-blocks x 16 KB
constexpr uint32_t HU_OFF_PU = HU_OFF_WO + 2 * HU_SUB; // P, then U     2 K-blocks x 16 KB
constexpr uint32_t HU_OFF_BAR = HU_OFF_PU + 2 * HU_SUB;
constexpr uint32_t HU_OFF_CK = HU_OFF_BAR + 128;       // 4 per-warp copies of the [HL] key row sums (fp32)
constexpr uint32_t HU_SMEM = HU_OFF_CK + 4 * HU_HL * 4; // 231,680 B of the 232,448 B an SM offers one CTA

struct HistUpdateParams {
  __nv_bfloat16* out;            // [total x d]
  const float* cK;               // [users x HL] row sums of K2
  const int32_t* off;            // [B+1]
  const int32_t* tile_start;     // [B+1] prefix of per-user tile counts (tile = 128 tokens)
  int B, ell, shared, ln;
  float ln_eps;
  int* err;
};

// address of 16-byte chunk `c` (0..7) of row r inside a 128B-swizzled [rows x 64 bf16] sub-tile
__device__ __forceinline__ uint32_t sw128_chunk(uint32_t r, uint32_t c) { return r * 128u + ((c ^ (r & 7u)) << 4); }

// user of tile t, cached: the tile ranges of consecutive tiles are the same user most of the time
struct TileUser {
  int b = -1, lo = 0, hi = 0;
  __device__ __forceinline__ int of(const int32_t* __restrict__ tile_start, int B, int t) {
    if (t < lo || t >= hi) {
      b = upper_user(tile_start, B, t);
      lo = tile_start[b];
      hi = tile_start[b + 1];
    }
    return b;
  }
};

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

template <int ELL>
__global__ void __launch_bounds__(HU_THREADS, 1)
k_hist_update_tc(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmK2,
                 const __grid_constant__ CUtensorMap tmG, const __grid_constant__ CUtensorMap tmU,
                 const __grid_constant__ CUtensorMap tmWo, const HistUpdateParams p) {
  using namespace tc;
  extern __shared__ __align__(1024) uint8_t smem[];
  if ((smem_u32(smem) & 1023u) != 0) {                       // swizzled tiles need a 1024-byte aligned base
    if (threadIdx.x == 0) atomicCAS(p.err, 0, 90);
    return;
  }
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + HU_OFF_BAR);
  uint64_t* x_full = bars;          // [2]  TMA -> MMA, epilogue
  uint64_t* x_empty = bars + 2;     // [2]  MMA commit (1) + epilogue warps (4)
  uint64_t* uops_full = bars + 4;   //      per user segment: K2, G2, U2 landed
  uint64_t* uops_empty = bars + 5;  //      per user segment: last MMA reading them done
  uint64_t* wo_full = bars + 6;
  uint64_t* s2_full = bars + 7;     // per tile, MMA1 done
  uint64_t* p_ready = bars + 8;     // per tile, P in smem (4 warps)
  uint64_t* gu_full = bars + 9;     // per tile, MMA2 done
  uint64_t* u_ready = bars + 10;    // per tile, U in smem (4 warps)
  uint64_t* sp_full = bars + 11;    // per tile, MMA3 done
  uint64_t* sp_free = bars + 12;    // per tile, S' read out of TMEM (4 warps)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 13);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_tiles = p.tile_start[p.B];
  const int t_begin = (int)(((int64_t)blockIdx.x * n_tiles) / gridDim.x);
  const int t_end = (int)(((int64_t)(blockIdx.x + 1) * n_tiles) / gridDim.x);

  if (threadIdx.x == 0) {
    for (int s = 0; s < 2; ++s) { mbar_init(&x_full[s], 1); mbar_init(&x_empty[s], 5); }
    mbar_init(uops_full, 1); mbar_init(uops_empty, 1); mbar_init(wo_full, 1);
    mbar_init(s2_full, 1); mbar_init(p_ready, 4); mbar_init(gu_full, 1); mbar_init(u_ready, 4);
    mbar_init(sp_full, 1); mbar_init(sp_free, 4);
    fence_barrier_init();
    prefetch_tmap(&tmX); prefetch_tmap(&tmK2); prefetch_tmap(&tmG); prefetch_tmap(&tmU); prefetch_tmap(&tmWo);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  constexpr uint32_t COL_S2 = 0, COL_GU = 128, COL_SP = 384;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0 && t_begin < t_end) {
      const uint64_t pol_stream = policy_evict_first(), pol_keep = policy_evict_last();
      mbar_arrive_expect_tx(wo_full, 2 * HU_SUB);
      for (int kb = 0; kb < 2; ++kb) tma_load_2d_hint(smem + HU_OFF_WO + kb * HU_SUB, &tmWo, kb * 64, 0, wo_full, pol_keep);
      int cur_user = -1, seg = 0, it = 0;
      bool ok = true;
      TileUser tu;
      for (int t = t_begin; t < t_end && ok; ++t, ++it) {
        const int b = tu.of(p.tile_start, p.B, t);
        if (b != cur_user) {
          if (seg > 0 && !mbar_wait(uops_empty, (uint32_t)(seg - 1) & 1u, p.err, 11)) { ok = false; break; }
          const int urow = p.shared ? 0 : b;
          mbar_arrive_expect_tx(uops_full, 6 * HU_SUB);
          for (int kb = 0; kb < 2; ++kb) {
            tma_load_2d_hint(smem + HU_OFF_K2 + kb * HU_SUB, &tmK2, kb * 64, urow * HU_HL, uops_full, pol_keep);
            tma_load_2d_hint(smem + HU_OFF_GU + kb * 2 * HU_SUB, &tmG, kb * 64, urow * HU_F, uops_full, pol_keep);
            tma_load_2d_hint(smem + HU_OFF_GU + kb * 2 * HU_SUB + HU_SUB, &tmU, kb * 64, urow * HU_F, uops_full, pol_keep);
          }
          cur_user = b;
          ++seg;
        }
        const int s = it & 1;
        if (!mbar_wait(&x_empty[s], ((uint32_t)(it >> 1) & 1u) ^ 1u, p.err, 12)) { ok = false; break; }
        const int row0 = p.off[b] + (t - tu.lo) * HU_TILE;
        mbar_arrive_expect_tx(&x_full[s], HU_X_STAGE);
        for (int kb = 0; kb < 2; ++kb)
          tma_load_2d_hint(smem + HU_OFF_X + s * HU_X_STAGE + kb * HU_SUB, &tmX, kb * 64, row0, &x_full[s], pol_stream);
      }
      if (!ok || *(volatile int*)p.err != 0) {
        for (int j = 0; j < it && j < 2; ++j) mbar_wait_quiet(&x_full[(it - 1 - j) & 1], (uint32_t)((it - 1 - j) >> 1) & 1u);
        if (seg > 0) mbar_wait_quiet(uops_full, (uint32_t)(seg - 1) & 1u);
        mbar_wait_quiet(wo_full, 0);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && t_begin < t_end) {
      constexpr uint32_t idesc_128 = make_idesc_bf16(128, 128);
      constexpr uint32_t idesc_256 = make_idesc_bf16(128, 256);
      const uint32_t sbase = smem_u32(smem);
      int cur_user = -1, seg = 0, it = 0;
      bool ok = mbar_wait(wo_full, 0, p.err, 21);
      TileUser tu;
      for (int t = t_begin; t < t_end && ok; ++t, ++it) {
        const int b = tu.of(p.tile_start, p.B, t);
        const uint32_t tp = (uint32_t)it & 1u;
        if (b != cur_user) {
          if (!mbar_wait(uops_full, (uint32_t)seg & 1u, p.err, 22)) break;
          cur_user = b;
          ++seg;
        }
        const int s = it & 1;
        if (!mbar_wait(&x_full[s], (uint32_t)(it >> 1) & 1u, p.err, 23)) break;
        tc_fence_after();
        // 1. scores = X . K2^T
        for (int kk = 0; kk < 8; ++kk) {
          const uint32_t o = (uint32_t)(kk >> 2) * HU_SUB + (uint32_t)(kk & 3) * 32;
          mma_bf16_ss(tmem_base + COL_S2, make_sdesc_k_sw128(sbase + HU_OFF_X + s * HU_X_STAGE + o),
                      make_sdesc_k_sw128(sbase + HU_OFF_K2 + o), idesc_128, kk != 0);
        }
        mma_commit(&x_empty[s]);
        mma_commit(s2_full);
        // 3. [gate | up] = P . [G2 | U2]
        if (!mbar_wait(p_ready, tp, p.err, 24)) break;
        tc_fence_after();
        for (int kk = 0; kk < 8; ++kk) {
          const uint32_t oa = (uint32_t)(kk >> 2) * HU_SUB + (uint32_t)(kk & 3) * 32;
          const uint32_t ob = (uint32_t)(kk >> 2) * 2 * HU_SUB + (uint32_t)(kk & 3) * 32;
          mma_bf16_ss(tmem_base + COL_GU, make_sdesc_k_sw128(sbase + HU_OFF_PU + oa),
                      make_sdesc_k_sw128(sbase + HU_OFF_GU + ob), idesc_256, kk != 0);
        }
        mma_commit(gu_full);
        // the user's operands are free once the last tile of the segment has issued its MMAs on them
        const bool last_of_user = (t + 1 == t_end) || (t + 1 >= tu.hi);
        if (last_of_user) mma_commit(uops_empty);
        // 5. S' = U . W_o
        if (!mbar_wait(u_ready, tp, p.err, 25)) break;
        if (it > 0 && !mbar_wait(sp_free, (uint32_t)(it - 1) & 1u, p.err, 26)) break;
        tc_fence_after();
        for (int kk = 0; kk < 8; ++kk) {
          const uint32_t o = (uint32_t)(kk >> 2) * HU_SUB + (uint32_t)(kk & 3) * 32;
          mma_bf16_ss(tmem_base + COL_SP, make_sdesc_k_sw128(sbase + HU_OFF_PU + o),
                      make_sdesc_k_sw128(sbase + HU_OFF_WO + o), idesc_128, kk != 0);
        }
        mma_commit(sp_full);
      }
    }
  } else {
    // ------------------------------------------------------------------ token-row warps (2..5)
    const int q = warp & 3;
    const uint32_t r = (uint32_t)(q * 32 + lane);           // token row of the tile == TMEM lane
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
    uint8_t* pu = smem + HU_OFF_PU;
    float* ck_s = reinterpret_cast<float*>(smem + HU_OFF_CK) + (warp - 2) * HU_HL;   // this warp's own copy
    int cur_user = -1, it = 0;
    constexpr int H = HU_HL / ELL;
    TileUser tu;
    for (int t = t_begin; t < t_end; ++t, ++it) {
      const int b = tu.of(p.tile_start, p.B, t);
      const uint32_t tp = (uint32_t)it & 1u;
      const int s = it & 1;
      if (b != cur_user) {
        __syncwarp();                                         // every lane is done with the previous user's sums
        for (int i = lane; i < HU_HL; i += 32) ck_s[i] = p.cK[(int64_t)(p.shared ? 0 : b) * HU_HL + i];
        __syncwarp();
        cur_user = b;
      }
      const int row0 = p.off[b] + (t - tu.lo) * HU_TILE;
      const bool valid = row0 + (int)r < p.off[b + 1];
      // LayerNorm statistics of this thread's token from the staged tile (two passes, rotated chunk order)
      if (!mbar_wait(&x_full[s], (uint32_t)(it >> 1) & 1u, p.err, 31)) break;
      float mu = 0.f, rstd = 1.f;
      if (p.ln) {
        const uint8_t* xs = smem + HU_OFF_X + s * HU_X_STAGE + r * 128u;
        float sum = 0.f;
#pragma unroll
        for (int c = 0; c < 16; ++c) {
          const int cc = (c + (int)r) & 7;
          const uint4 u = *reinterpret_cast<const uint4*>(xs + (c >> 3) * HU_SUB + cc * 16);
          const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) sum += __uint_as_float(w[j] << 16) + __uint_as_float(w[j] & 0xffff0000u);
        }
        mu = sum * (1.0f / HU_D);
        float var = 0.f;
#pragma unroll
        for (int c = 0; c < 16; ++c) {
          const int cc = (c + (int)r) & 7;
          const uint4 u = *reinterpret_cast<const uint4*>(xs + (c >> 3) * HU_SUB + cc * 16);
          const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float a = __uint_as_float(w[j] << 16) - mu, bb = __uint_as_float(w[j] & 0xffff0000u) - mu;
            var = fmaf(a, a, var);
            var = fmaf(bb, bb, var);
          }
        }
        rstd = rsqrtf(var * (1.0f / HU_D) + p.ln_eps);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&x_empty[s]);

      // 2. per-head softmax over the links, P -> smem (A operand of the next MMA, K-major, 128B swizzle)
      if (!mbar_wait(s2_full, tp, p.err, 32)) break;
      tc_fence_after();
#pragma unroll
      for (int h = 0; h < H; ++h) {
        float sc[ELL];
#pragma unroll
        for (int c = 0; c < ELL; c += 16) {
          float v[16];
          tmem_ld_32x16(lane_addr + COL_S2 + h * ELL + c, v);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 16; ++j) sc[c + j] = (v[j] - mu * ck_s[h * ELL + c + j]) * rstd;
        }
        float mx = sc[0];
#pragma unroll
        for (int j = 1; j < ELL; ++j) mx = fmaxf(mx, sc[j]);
        float sum = 0.f;
#pragma unroll
        for (int j = 0; j < ELL; ++j) { sc[j] = __expf(sc[j] - mx); sum += sc[j]; }
        const float inv = 1.f / sum;
#pragma unroll
        for (int c8 = 0; c8 < ELL / 8; ++c8) {
          const int k = h * ELL + c8 * 8;                    // first of 8 consecutive contraction indices
          uint4 o;
          o.x = pack_bf16(sc[c8 * 8 + 0] * inv, sc[c8 * 8 + 1] * inv);
          o.y = pack_bf16(sc[c8 * 8 + 2] * inv, sc[c8 * 8 + 3] * inv);
          o.z = pack_bf16(sc[c8 * 8 + 4] * inv, sc[c8 * 8 + 5] * inv);
          o.w = pack_bf16(sc[c8 * 8 + 6] * inv, sc[c8 * 8 + 7] * inv);
          *reinterpret_cast<uint4*>(pu + (k >> 6) * HU_SUB + sw128_chunk(r, (uint32_t)(k & 63) >> 3)) = o;
        }
      }
      tc_fence_before();
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(p_ready);

      // 4. U = SiLU(gate) * up -> smem (over P, which the second MMA has finished reading)
      if (!mbar_wait(gu_full, tp, p.err, 33)) break;
      tc_fence_after();
#pragma unroll
      for (int c = 0; c < HU_F; c += 16) {
        float g[16], u[16];
        tmem_ld_32x16(lane_addr + COL_GU + c, g);
        tmem_ld_32x16(lane_addr + COL_GU + HU_F + c, u);
        tmem_wait_ld();
        float y[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) y[j] = silu_f(g[j]) * u[j];
#pragma unroll
        for (int c8 = 0; c8 < 2; ++c8) {
          const int k = c + c8 * 8;
          uint4 o;
          o.x = pack_bf16(y[c8 * 8 + 0], y[c8 * 8 + 1]);
          o.y = pack_bf16(y[c8 * 8 + 2], y[c8 * 8 + 3]);
          o.z = pack_bf16(y[c8 * 8 + 4], y[c8 * 8 + 5]);
          o.w = pack_bf16(y[c8 * 8 + 6], y[c8 * 8 + 7]);
          *reinterpret_cast<uint4*>(pu + (k >> 6) * HU_SUB + sw128_chunk(r, (uint32_t)(k & 63) >> 3)) = o;
        }
      }
      tc_fence_before();
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(u_ready);

      // 6. S' row -> bf16 -> global
      if (!mbar_wait(sp_full, tp, p.err, 34)) break;
      tc_fence_after();
      uint4* dst = reinterpret_cast<uint4*>(p.out + (int64_t)(row0 + (int)r) * HU_D);
#pragma unroll
      for (int c = 0; c < HU_D; c += 16) {
        float v[16];
        tmem_ld_32x16(lane_addr + COL_SP + c, v);
        tmem_wait_ld();
        if (valid) {
          uint4 o0, o1;
          o0.x = pack_bf16(v[0], v[1]); o0.y = pack_bf16(v[2], v[3]); o0.z = pack_bf16(v[4], v[5]); o0.w = pack_bf16(v[6], v[7]);
          o1.x = pack_bf16(v[8], v[9]); o1.y = pack_bf16(v[10], v[11]); o1.z = pack_bf16(v[12], v[13]); o1.w = pack_bf16(v[14], v[15]);
          dst[c / 8] = o0;
          dst[c / 8 + 1] = o1;
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(sp_free);
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
  return dtype == LIME_BF16 && d == HU_D && f == HU_F && H * ell == HU_HL && (ell == 16 || ell == 32 || ell == 64) &&
         phi == LIME_PHI_SOFTMAX && gated_mlp != 0;
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
  p.out = (__nv_bfloat16*)a.hist_out; p.cK = a.cK; p.off = a.off; p.tile_start = a.tile_start; p.B = a.B; p.ell = ELL;
  p.shared = a.shared; p.ln = a.ln; p.ln_eps = a.ln_eps; p.err = a.err;
  int grid = a.n_tile_upper < kSMs ? a.n_tile_upper : kSMs;
  if (grid < 1) return LIME_OK;
  LIME_CUDA(cudaFuncSetAttribute(k_hist_update_tc<ELL>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)HU_SMEM));
  ProfScope _p("k_hist_update_tc", st);
  k_hist_update_tc<ELL><<<grid, HU_THREADS, HU_SMEM, st>>>(tmX, tmK2, tmG, tmU, tmWo, p);
  LIME_LAUNCH_CHECK("k_hist_update_tc");
  return LIME_OK;
}

lime_status launch_hist_update_tc(const HistUpdateArgs& a, cudaStream_t st) {
  if (a.total == 0) return LIME_OK;
  switch (a.ell) {
    case 16: return launch_hu<16>(a, st);
    case 32: return launch_hu<32>(a, st);
    case 64: return launch_hu<64>(a, st);
  }
  return LIME_UNSUPPORTED_SHAPE;
}

}  // namespace lime
