// Candidate scoring through the interaction network on the 5th-generation tensor cores (bf16 storage, one hidden layer):
//
//   O_c     = sum_l W[c,l] LS[l,:]                                            (Eq. 4, the LIME embedding of candidate c)
//   logit_c = w_2 . ReLU( [O_c | T_c] W_1 + b_1 ) + b_2                       (Sec. 3.3 "Lightweight User-Item Interaction":
//                                                                              a shallow interaction network scores O_c)
// With W_1 = [W_1a ; W_1b] split over the two halves of its input, O_c W_1a = sum_l W[c,l] (LS W_1a)[l,:], so the
// hidden pre-activation of a tile of 128 candidates is two chained contractions into one TMEM accumulator,
//   acc [128 x n1] = T_tile [128 x d] . W_1b [d x n1]  +  W_tile [128 x ell] . LSW_b [ell x n1],   LSW_b = LS_b W_1a,
// and O is never formed: per candidate the kernel still streams only its weight row and its embedding row.  LSW_b
// ([ell x n1] per user) is formed by k_head_lsw before this kernel; W_1b is weights only.
// Same streaming structure as k_score_tc.cu: warp 0 TMA producer (candidate tile + weight rows into a ring of stages,
// the user's LSW into its own one or two buffers), warp 1 MMA issuer, warps 2-5 epilogue (thread r = candidate row r =
// TMEM lane r: bias, ReLU and the n1-term dot with w_2 in registers).
#include "lime_common.cuh"
#include "tc_common.cuh"

namespace lime {

constexpr int SH_TILE = 128, SH_THREADS = 192, SH_MAX_STAGES = 6;

struct ScoreHeadParams {
  float* logits;
  const float* b1;       // [n1] or NULL
  const float* w2;       // [n1]
  const float* b2;       // [1] or NULL
  int B, C, d, n1;
  int tiles_per_user, n_tiles;
  int stages, lsw_bufs;
  int* err;
};

template <int ELL>
__global__ void __launch_bounds__(SH_THREADS, 1)
k_score_head_tc(const __grid_constant__ CUtensorMap tmT, const __grid_constant__ CUtensorMap tmW,
                const __grid_constant__ CUtensorMap tmLSW, const __grid_constant__ CUtensorMap tmW1b, const ScoreHeadParams p) {
  using namespace tc;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);

  constexpr int WKB = ELL > 64 ? ELL / 64 : 1;                   // K blocks of the weight-row operand
  constexpr int WK = ELL > 64 ? 64 : ELL;                        // elements per K block (row pitch WK * 2 bytes)
  constexpr uint32_t W_ROW = WK * 2;                             // swizzle span of the weight-row operands
  const int KB = p.d / 64, n1 = p.n1;
  const uint32_t t_bytes = (uint32_t)KB * SH_TILE * 128;
  constexpr uint32_t w_bytes = (uint32_t)SH_TILE * ELL * 2;
  const uint32_t stage_bytes = t_bytes + w_bytes;
  const uint32_t lsw_bytes = ((uint32_t)n1 * ELL * 2 + 1023u) & ~1023u;
  const uint32_t w1b_bytes = (uint32_t)KB * n1 * 128;
  const int S = p.stages, LB = p.lsw_bufs;

  uint8_t* lsw_base = smem + (size_t)S * stage_bytes;
  uint8_t* w1b_base = lsw_base + (size_t)LB * lsw_bytes;
  float* consts = reinterpret_cast<float*>(w1b_base + ((w1b_bytes + 1023u) & ~1023u));     // b1 [n1], w2 [n1], b2
  uint64_t* full = reinterpret_cast<uint64_t*>(consts + 2 * 256 + 4);
  uint64_t* empty = full + SH_MAX_STAGES;
  uint64_t* tmem_full = empty + SH_MAX_STAGES;
  uint64_t* tmem_empty = tmem_full + 2;
  uint64_t* lsw_full = tmem_empty + 2;        // [2]
  uint64_t* lsw_empty = lsw_full + 2;         // [2]
  uint64_t* w1b_full = lsw_empty + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(w1b_full + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t acc_cols = n1 <= 32 ? 32u : (n1 <= 64 ? 64u : (n1 <= 128 ? 128u : 256u));   // one accumulator buffer
  const uint32_t tmem_cols = 2 * acc_cols;

  const int t_begin = (int)(((int64_t)blockIdx.x * p.n_tiles) / gridDim.x);
  const int t_end = (int)(((int64_t)(blockIdx.x + 1) * p.n_tiles) / gridDim.x);

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&tmem_full[b], 1); mbar_init(&tmem_empty[b], 4);
      mbar_init(&lsw_full[b], 1); mbar_init(&lsw_empty[b], 1);
    }
    mbar_init(w1b_full, 1);
    fence_barrier_init();
    prefetch_tmap(&tmT); prefetch_tmap(&tmW); prefetch_tmap(&tmLSW); prefetch_tmap(&tmW1b);
  }
  for (int i = threadIdx.x; i < n1; i += SH_THREADS) {
    consts[i] = p.b1 ? p.b1[i] : 0.f;
    consts[256 + i] = p.w2[i];
  }
  if (threadIdx.x == 0) consts[512] = p.b2 ? p.b2[0] : 0.f;
  if (warp == 1) { tmem_alloc(tmem_slot, tmem_cols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0 && t_begin < t_end) {
      const uint64_t pol_stream = policy_evict_first(), pol_keep = policy_evict_last();
      mbar_arrive_expect_tx(w1b_full, w1b_bytes);
      for (int kb = 0; kb < KB; ++kb) tma_load_2d_hint(w1b_base + (size_t)kb * n1 * 128, &tmW1b, kb * 64, 0, w1b_full, pol_keep);
      int it = 0, un = 0, prev_user = -1;
      bool ok = true;
      for (int t = t_begin; t < t_end && ok; ++t, ++it) {
        const int b = t / p.tiles_per_user;
        if (b != prev_user) {
          const int lb = un % LB;
          if (!mbar_wait(&lsw_empty[lb], ((uint32_t)(un / LB) & 1u) ^ 1u, p.err, 101)) { ok = false; break; }
          mbar_arrive_expect_tx(&lsw_full[lb], (uint32_t)n1 * ELL * 2);
          for (int kb = 0; kb < WKB; ++kb)
            tma_load_2d_hint(lsw_base + (size_t)lb * lsw_bytes + (size_t)kb * n1 * W_ROW, &tmLSW, kb * WK, b * n1, &lsw_full[lb], pol_keep);
          ++un;
          prev_user = b;
        }
        const int s = it % S;
        if (!mbar_wait(&empty[s], ((uint32_t)(it / S) & 1u) ^ 1u, p.err, 102)) { ok = false; break; }
        const int row0 = b * p.C + (t % p.tiles_per_user) * SH_TILE;
        uint8_t* st = smem + (size_t)s * stage_bytes;
        mbar_arrive_expect_tx(&full[s], stage_bytes);
        for (int kb = 0; kb < KB; ++kb) tma_load_2d_hint(st + (size_t)kb * SH_TILE * 128, &tmT, kb * 64, row0, &full[s], pol_stream);
        for (int kb = 0; kb < WKB; ++kb)
          tma_load_2d_hint(st + t_bytes + (size_t)kb * SH_TILE * W_ROW, &tmW, kb * WK, row0, &full[s], pol_stream);
      }
      if (!ok || *(volatile int*)p.err != 0) {
        // giving up: let the copies already issued land (bounded) before this CTA's shared memory goes away
        for (int j = 0; j < it && j < S; ++j) mbar_wait_quiet(&full[(it - 1 - j) % S], (uint32_t)((it - 1 - j) / S) & 1u);
        for (int j = 0; j < un && j < LB; ++j) mbar_wait_quiet(&lsw_full[(un - 1 - j) % LB], (uint32_t)((un - 1 - j) / LB) & 1u);
        mbar_wait_quiet(w1b_full, 0);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && t_begin < t_end) {
      const uint32_t idesc = make_idesc_bf16(SH_TILE, n1);
      bool ok = mbar_wait(w1b_full, 0, p.err, 103);
      int it = 0, un = 0, prev_user = -1;
      uint32_t lsw_addr = 0;
      for (int t = t_begin; t < t_end && ok; ++t, ++it) {
        const int b = t / p.tiles_per_user;
        if (b != prev_user) {
          const int lb = un % LB;
          if (!mbar_wait(&lsw_full[lb], (uint32_t)(un / LB) & 1u, p.err, 104)) break;
          lsw_addr = smem_u32(lsw_base + (size_t)lb * lsw_bytes);
          ++un;
          prev_user = b;
        }
        const int s = it % S, buf = it & 1;
        if (!mbar_wait(&tmem_empty[buf], ((uint32_t)(it >> 1) & 1u) ^ 1u, p.err, 105)) break;
        if (!mbar_wait(&full[s], (uint32_t)(it / S) & 1u, p.err, 106)) break;
        tc_fence_after();
        const uint32_t a0 = smem_u32(smem + (size_t)s * stage_bytes);
        const uint32_t d_tmem = tmem_base + (uint32_t)buf * acc_cols;
        // T_tile . W_1b  (contraction over d)
        for (int kb = 0; kb < KB; ++kb) {
#pragma unroll
          for (int k = 0; k < 4; ++k)
            mma_bf16_ss(d_tmem, make_sdesc_k_sw128(a0 + (uint32_t)kb * SH_TILE * 128 + k * 32),
                        make_sdesc_k_sw128(smem_u32(w1b_base) + (uint32_t)kb * n1 * 128 + k * 32), idesc, (kb | k) != 0 ? 1u : 0u);
        }
        // + W_tile . LSW_b  (contraction over the links)
#pragma unroll
        for (int kb = 0; kb < WKB; ++kb) {
#pragma unroll
          for (int k = 0; k < WK / 16; ++k)
            mma_bf16_ss(d_tmem, make_sdesc_k_sw(a0 + t_bytes + (uint32_t)kb * SH_TILE * W_ROW + k * 32, W_ROW),
                        make_sdesc_k_sw(lsw_addr + (uint32_t)kb * n1 * W_ROW + k * 32, W_ROW), idesc, 1u);
        }
        mma_commit(&empty[s]);
        mma_commit(&tmem_full[buf]);
        // the last tile of this user inside the CTA frees the user's LSW buffer
        const bool user_ends = (t + 1 < t_end) && ((t + 1) / p.tiles_per_user != b);
        if (user_ends) mma_commit(&lsw_empty[(un - 1) % LB]);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int q = warp & 3;
    const int r = q * 32 + lane;
    const float* b1s = consts;
    const float* w2s = consts + 256;
    const float b2 = consts[512];
    int it = 0;
    for (int t = t_begin; t < t_end; ++t, ++it) {
      const int buf = it & 1;
      const int b = t / p.tiles_per_user;
      const int c0 = (t % p.tiles_per_user) * SH_TILE;
      if (!mbar_wait(&tmem_full[buf], (uint32_t)(it >> 1) & 1u, p.err, 107)) break;
      tc_fence_after();
      float acc4[4] = {0.f, 0.f, 0.f, 0.f};
      const uint32_t ta = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)buf * acc_cols;
      for (int c = 0; c < n1; c += 16) {
        float v[16];
        tmem_ld_32x16(ta + (uint32_t)c, v);
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < 16; ++j) acc4[j & 3] = fmaf(fmaxf(v[j] + b1s[c + j], 0.f), w2s[c + j], acc4[j & 3]);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tmem_empty[buf]);
      if (c0 + r < p.C) p.logits[(int64_t)b * p.C + c0 + r] = (acc4[0] + acc4[1]) + (acc4[2] + acc4[3]) + b2;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, tmem_cols);
  }
}

// Shared-memory plan: S stages of (candidate tile + weight rows), one or two LSW buffers, W_1b, constants, barriers.
static bool score_head_plan(int ell, int d, int n1, int* stages, int* lsw_bufs, size_t* smem_bytes) {
  const size_t stage = (size_t)(d / 64) * SH_TILE * 128 + (size_t)SH_TILE * ell * 2;
  const size_t lsw = ((size_t)n1 * ell * 2 + 1023) & ~(size_t)1023;
  const size_t w1b = ((size_t)(d / 64) * n1 * 128 + 1023) & ~(size_t)1023;
  const size_t fixed = 1024 + (2 * 256 + 4) * 4 + (2 * SH_MAX_STAGES + 9) * 8 + 16;
  const size_t budget = 226 * 1024;
  for (int lb = 2; lb >= 1; --lb) {
    if (fixed + w1b + lb * lsw + 2 * stage > budget) continue;
    int S = (int)((budget - fixed - w1b - lb * lsw) / stage);
    if (S > SH_MAX_STAGES) S = SH_MAX_STAGES;
    *stages = S; *lsw_bufs = lb; *smem_bytes = fixed + w1b + lb * lsw + (size_t)S * stage;
    return true;
  }
  return false;
}

bool score_head_tc_supported(const ScoreArgs& a, int n1) {
  if (a.dtype != LIME_BF16 || a.cand_off != nullptr || a.cand_ids != nullptr) return false;
  if (!(a.ell == 32 || a.ell == 64 || a.ell == 128)) return false;
  if (a.d % 64 != 0 || a.d > 512) return false;
  if (n1 % 16 != 0 || n1 < 16 || n1 > 256) return false;
  if (a.C <= 0 || a.total != (int64_t)a.B * a.C) return false;
  int S, lb;
  size_t smem;
  return score_head_plan(a.ell, a.d, n1, &S, &lb, &smem);
}

template <int ELL>
static lime_status launch_score_head_tc_t(const ScoreArgs& a, const ScoreHeadArgs& h, int* err, cudaStream_t st) {
  int S, lb;
  size_t smem;
  if (!score_head_plan(ELL, a.d, h.n1, &S, &lb, &smem)) return LIME_UNSUPPORTED_SHAPE;
  constexpr int WK = ELL > 64 ? 64 : ELL;
  CUtensorMap tmT, tmW, tmLSW, tmW1b;
  if (!make_tmap_bf16_sw128(&tmT, a.T, (uint64_t)a.total, (uint64_t)a.d, (uint64_t)a.d, SH_TILE) ||
      !make_tmap_bf16_kmajor(&tmW, a.W, (uint64_t)a.total, ELL, ELL, SH_TILE, WK) ||
      !make_tmap_bf16_kmajor(&tmLSW, h.LSWt, (uint64_t)a.B * h.n1, ELL, ELL, (uint32_t)h.n1, WK) ||
      !make_tmap_bf16_sw128(&tmW1b, h.W1bT, (uint64_t)h.n1, (uint64_t)a.d, (uint64_t)a.d, (uint32_t)h.n1))
    return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
  ScoreHeadParams p;
  p.logits = a.logits; p.b1 = h.b1; p.w2 = h.w2; p.b2 = h.b2; p.B = a.B; p.C = a.C; p.d = a.d; p.n1 = h.n1;
  p.tiles_per_user = (a.C + SH_TILE - 1) / SH_TILE;
  p.n_tiles = p.tiles_per_user * a.B;
  p.stages = S; p.lsw_bufs = lb; p.err = err;
  const int grid = p.n_tiles < kSMs ? p.n_tiles : kSMs;
  LIME_CUDA(cudaFuncSetAttribute(k_score_head_tc<ELL>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  ProfScope _p("k_score_head_tc", st);
  k_score_head_tc<ELL><<<grid, SH_THREADS, smem, st>>>(tmT, tmW, tmLSW, tmW1b, p);
  LIME_LAUNCH_CHECK("k_score_head_tc");
  return LIME_OK;
}

lime_status launch_score_head_tc(const ScoreArgs& a, const ScoreHeadArgs& h, int* err, cudaStream_t st) {
  switch (a.ell) {
    case 32: return launch_score_head_tc_t<32>(a, h, err, st);
    case 64: return launch_score_head_tc_t<64>(a, h, err, st);
    case 128: return launch_score_head_tc_t<128>(a, h, err, st);
  }
  return LIME_UNSUPPORTED_SHAPE;
}

}  // namespace lime
