// Candidate scoring on the 5th-generation tensor cores (Eq. 4, per-candidate stage), bf16 storage.
//
//   logit[c] = < sum_l W[c,l] LS[l,:], T[c,:] >  =  sum_l W[c,l] * A[c,l],   A = T_tile [128 x d] . LS^T [d x ell]
//
// The contraction T.LS^T is a real dense GEMM (25-50 flop per streamed byte, more than the CUDA cores can
// sustain at HBM rate), so it runs as tcgen05.mma with the accumulator in TMEM; what remains per candidate is an
// ell-term dot product with the cached weight row.  The kernel is a persistent, warp-specialised stream:
//   warp 0    : TMA producer  - candidate tile [128 x d], its cached weight rows [128 x ell] (+ the user's link
//                               states when the stage holds another user's) into a ring of shared-memory stages
//   warp 1    : MMA issuer    - d/16 tcgen05.mma (M=128, N=ell, K=16) per tile into one of two TMEM accumulators
//   warps 2-5 : epilogue      - thread r owns candidate row r of the tile (TMEM lane r): takes its weight row from
//                               the stage, reads the accumulator row with tcgen05.ld, writes one logit
// Every HBM stream is therefore prefetched a whole ring ahead of its use; no warp waits on a global load.
// HBM traffic per candidate is the algorithmic minimum: its weight row, its embedding row, one fp32 logit.
#include "lime_common.cuh"
#include "tc_common.cuh"

namespace lime {

constexpr int SCT_TILE = 128;
constexpr int SCT_THREADS = 192;
constexpr int SCT_MAX_STAGES = 8;

struct ScoreTcParams {
  float* logits;
  int B, C, d;
  int tiles_per_user, n_tiles;
  int stages;
  int* err;
};

template <int ELL>
__global__ void __launch_bounds__(SCT_THREADS, 1)
k_score_tc(const __grid_constant__ CUtensorMap tmT, const __grid_constant__ CUtensorMap tmLS,
           const __grid_constant__ CUtensorMap tmW, const ScoreTcParams p) {
  using namespace tc;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);

  const int KB = p.d / 64;                       // 64-element (128-byte) K blocks
  const uint32_t t_bytes = (uint32_t)KB * SCT_TILE * 128;
  const uint32_t ls_bytes = (uint32_t)KB * ELL * 128;
  constexpr uint32_t w_bytes = (uint32_t)SCT_TILE * ELL * 2;     // weight rows, not swizzled: row r at r * ELL * 2
  const uint32_t stage_bytes = t_bytes + ls_bytes + w_bytes;
  const int S = p.stages;

  uint64_t* full = reinterpret_cast<uint64_t*>(smem + (size_t)S * stage_bytes);
  uint64_t* empty = full + SCT_MAX_STAGES;
  uint64_t* tmem_full = empty + SCT_MAX_STAGES;
  uint64_t* tmem_empty = tmem_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tmem_empty + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr uint32_t TMEM_COLS = (2 * ELL < 32) ? 32 : 2 * ELL;

  // contiguous tile range per CTA: consecutive tiles share a user, so link states are re-fetched rarely
  const int t_begin = (int)(((int64_t)blockIdx.x * p.n_tiles) / gridDim.x);
  const int t_end = (int)(((int64_t)(blockIdx.x + 1) * p.n_tiles) / gridDim.x);

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 5); }   // MMA commit + 4 epilogue warps
    for (int b = 0; b < 2; ++b) { mbar_init(&tmem_full[b], 1); mbar_init(&tmem_empty[b], 4); }
    fence_barrier_init();
    prefetch_tmap(&tmT);
    prefetch_tmap(&tmLS);
    prefetch_tmap(&tmW);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // set-up done: the next kernel's CTAs may become resident; nothing an earlier kernel wrote is read before this wait
  pdl_launch_dependents();
  pdl_wait();

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage_user[SCT_MAX_STAGES];
#pragma unroll
      for (int s = 0; s < SCT_MAX_STAGES; ++s) stage_user[s] = -1;
      const uint64_t pol_stream = policy_evict_first();
      const uint64_t pol_keep = policy_evict_last();
      int it = 0;
      bool ok = true;
      for (int t = t_begin; t < t_end; ++t, ++it) {
        const int s = it % S;
        const uint32_t ph = (uint32_t)(it / S) & 1u;
        if (!mbar_wait(&empty[s], ph ^ 1u, p.err, 1)) { ok = false; break; }
        const int b = t / p.tiles_per_user;
        const int row0 = b * p.C + (t % p.tiles_per_user) * SCT_TILE;
        bool load_ls = false;
#pragma unroll
        for (int q = 0; q < SCT_MAX_STAGES; ++q)
          if (q == s) { load_ls = stage_user[q] != b; stage_user[q] = b; }
        uint8_t* st = smem + (size_t)s * stage_bytes;
        mbar_arrive_expect_tx(&full[s], t_bytes + w_bytes + (load_ls ? ls_bytes : 0u));
        for (int kb = 0; kb < KB; ++kb)
          tma_load_2d_hint(st + (size_t)kb * SCT_TILE * 128, &tmT, kb * 64, row0, &full[s], pol_stream);
        tma_load_2d_hint(st + t_bytes + ls_bytes, &tmW, 0, row0, &full[s], pol_stream);
        if (load_ls)
          for (int kb = 0; kb < KB; ++kb)
            tma_load_2d_hint(st + t_bytes + (size_t)kb * ELL * 128, &tmLS, kb * 64, b * ELL, &full[s], pol_keep);
      }
      if (!ok || *(volatile int*)p.err != 0) {
        // giving up: let the copies already issued land (bounded) before this CTA's shared memory goes away
        for (int j = 0; j < it && j < S; ++j) {
          const int last = it - 1 - j;                    // most recent arming of stage last % S
          mbar_wait_quiet(&full[last % S], (uint32_t)(last / S) & 1u);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(SCT_TILE, ELL);
      int it = 0;
      for (int t = t_begin; t < t_end; ++t, ++it) {
        const int s = it % S;
        const uint32_t ph = (uint32_t)(it / S) & 1u;
        const int buf = it & 1;
        const uint32_t bph = (uint32_t)(it >> 1) & 1u;
        if (!mbar_wait(&tmem_empty[buf], bph ^ 1u, p.err, 2)) break;
        if (!mbar_wait(&full[s], ph, p.err, 3)) break;
        tc_fence_after();
        const uint32_t a0 = smem_u32(smem + (size_t)s * stage_bytes);
        const uint32_t b0 = a0 + t_bytes;
        const uint32_t d_tmem = tmem_base + (uint32_t)buf * ELL;
        for (int kb = 0; kb < KB; ++kb) {
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const uint64_t ad = make_sdesc_k_sw128(a0 + (uint32_t)kb * SCT_TILE * 128 + k * 32);
            const uint64_t bd = make_sdesc_k_sw128(b0 + (uint32_t)kb * ELL * 128 + k * 32);
            mma_bf16_ss(d_tmem, ad, bd, idesc, (kb | k) != 0 ? 1u : 0u);
          }
        }
        mma_commit(&empty[s]);         // the stage may be refilled once these MMAs have read it
        mma_commit(&tmem_full[buf]);   // the accumulator is complete
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int q = warp & 3;                       // TMEM lane quarter this warp may read
    const int r = q * 32 + lane;                  // candidate row of the tile owned by this thread
    int it = 0;
    for (int t = t_begin; t < t_end; ++t, ++it) {
      const int buf = it & 1;
      const uint32_t bph = (uint32_t)(it >> 1) & 1u;
      const int b = t / p.tiles_per_user;
      const int c0 = (t % p.tiles_per_user) * SCT_TILE;
      const bool valid = c0 + r < p.C;
      const int64_t grow = (int64_t)b * p.C + c0 + r;
      const int s = it % S;
      if (!mbar_wait(&full[s], (uint32_t)(it / S) & 1u, p.err, 5)) break;
      uint4 w[ELL / 8];
      {
        const uint4* wp = reinterpret_cast<const uint4*>(smem + (size_t)s * stage_bytes + t_bytes + ls_bytes) + r * (ELL / 8);
#pragma unroll
        for (int i = 0; i < ELL / 8; ++i) w[i] = wp[i];
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[s]);       // this warp has taken its rows out of the stage
      if (!mbar_wait(&tmem_full[buf], bph, p.err, 4)) break;
      tc_fence_after();
      // dot of the weight row with the accumulator row, CH columns per TMEM load, four independent partial sums
      constexpr int CH = ELL >= 32 ? 32 : 16;
      float acc4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int c = 0; c < ELL; c += CH) {
        float v[CH];
        const uint32_t ta = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * ELL + c);
        if constexpr (CH == 32) tmem_ld_32x32(ta, v); else tmem_ld_32x16(ta, v);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < CH / 8; ++i) {
          const uint4 u = w[c / 8 + i];
          const uint32_t uu[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float lo = __uint_as_float(uu[j] << 16);
            const float hi = __uint_as_float(uu[j] & 0xffff0000u);
            acc4[j] = fmaf(lo, v[i * 8 + 2 * j], acc4[j]);
            acc4[j] = fmaf(hi, v[i * 8 + 2 * j + 1], acc4[j]);
          }
        }
      }
      const float acc = (acc4[0] + acc4[1]) + (acc4[2] + acc4[3]);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tmem_empty[buf]);
      if (valid) p.logits[grow] = acc;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// Shared-memory budget: S stages of (candidate tile + link states) + barriers + alignment slack.
static int score_tc_stages(int ell, int d, size_t* smem_bytes) {
  const size_t stage = (size_t)(d / 64) * (SCT_TILE + ell) * 128 + (size_t)SCT_TILE * ell * 2;
  const size_t fixed = 1024 + 2 * SCT_MAX_STAGES * 8 + 4 * 8 + 16;
  int S = (int)((226 * 1024 - fixed) / stage);
  if (S > SCT_MAX_STAGES) S = SCT_MAX_STAGES;
  *smem_bytes = (size_t)S * stage + fixed;
  return S;
}

bool score_tc_supported(const ScoreArgs& a) {
  if (a.dtype != LIME_BF16 || a.cand_off != nullptr || a.cand_ids != nullptr) return false;
  if (!(a.ell == 16 || a.ell == 32 || a.ell == 64 || a.ell == 128)) return false;
  if (a.d % 64 != 0 || a.d > 512) return false;
  if (a.C <= 0 || a.total != (int64_t)a.B * a.C) return false;
  size_t smem;
  return score_tc_stages(a.ell, a.d, &smem) >= 2;
}

template <int ELL>
static lime_status launch_score_tc_t(const ScoreArgs& a, int* err, cudaStream_t st) {
  size_t smem;
  const int S = score_tc_stages(ELL, a.d, &smem);
  CUtensorMap tmT, tmLS, tmW;
  if (!make_tmap_bf16_sw128(&tmT, a.T, (uint64_t)a.total, (uint64_t)a.d, (uint64_t)a.d, SCT_TILE) ||
      !make_tmap_bf16_sw128(&tmLS, a.LS, (uint64_t)a.B * ELL, (uint64_t)a.d, (uint64_t)a.d, ELL) ||
      !make_tmap_bf16_plain(&tmW, a.W, (uint64_t)a.total, ELL, ELL, SCT_TILE))
    return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
  ScoreTcParams p;
  p.logits = a.logits; p.B = a.B; p.C = a.C; p.d = a.d;
  p.tiles_per_user = (a.C + SCT_TILE - 1) / SCT_TILE;
  p.n_tiles = p.tiles_per_user * a.B;
  p.stages = S; p.err = err;
  int grid = p.n_tiles < kSMs ? p.n_tiles : kSMs;
  LIME_CUDA(cudaFuncSetAttribute(k_score_tc<ELL>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  ProfScope _p("k_score_tc", st);
  launch_pdl(k_score_tc<ELL>, dim3(grid), dim3(SCT_THREADS), smem, st, tmT, tmLS, tmW, p);
  LIME_LAUNCH_CHECK("k_score_tc");
  return LIME_OK;
}

lime_status launch_score_tc(const ScoreArgs& a, int* err, cudaStream_t st) {
  switch (a.ell) {
    case 16: return launch_score_tc_t<16>(a, err, st);
    case 32: return launch_score_tc_t<32>(a, err, st);
    case 64: return launch_score_tc_t<64>(a, err, st);
    case 128: return launch_score_tc_t<128>(a, err, st);
  }
  return LIME_UNSUPPORTED_SHAPE;
}

}  // namespace lime
