// Candidate scoring straight from the corpus-level caches (Eq. 4, Sec. 3.3 "QK cache"), bf16 storage:
//
//   logit[b, c] = < sum_l W[id, l] LS_b[l, :], T[id, :] >,   id = cand_ids[b * C + c]
//
// where T [V x d] is the item-embedding table and W [V x ell] the cached candidate->link weights of the whole corpus.
// Same structure as k_score_tc.cu (A = T_tile . LS^T on tcgen05 with the accumulator in TMEM, then an ell-term dot
// with the weight row per candidate), but the rows of a tile are not adjacent in memory, so one tiled copy cannot
// fetch them.  The producer warps fetch them with the gather form of the TMA tile load: one copy takes a column
// offset and FOUR row indices and lands the four rows (box one row high) as consecutive rows of the stage, with the
// 128-byte swizzle the MMA expects applied from the destination address as for a full tile.  Per tile that is
// 32 x d/64 copies of embedding rows and 32 of weight rows (not swizzled).  Measured alternatives: per-thread 16-byte
// cp.async copies (2.3 TB/s: the load/store path keeps too few sectors in flight) and one-row TMA boxes (1.7 TB/s:
// bound by the copy-issue rate).  This removes the separate gather of candidate rows (a write and a re-read of
// d + ell elements per candidate) from the serving path.
//   warps 0-3 : producers  - 32 x (d/64 + 1) gather copies per tile spread over the threads; thread 0 also fetches the user's link states when the stage held another user's
//   warp  4   : MMA issuer
//   warps 5-8 : epilogue   - thread r owns candidate row r (TMEM lane r)
// With packed corpus records ([embedding row | weight row] per item, row pitch d + ell: lime_pack_corpus_cache) the
// same copies run over two views of the one array, and a candidate's embedding and weights come from one place in DRAM.
// An id outside [0, V) fetches row 0 instead (the copies of a stage keep their fixed byte count and never leave the
// caches); the epilogue thread of that slot writes logit 0 and lowers the caller's flag to the slot index.
#include "lime_common.cuh"
#include "tc_common.cuh"

namespace lime {

constexpr int SG_TILE = 128;
constexpr int SG_THREADS = 128 + 32 + 128;
constexpr int SG_MAX_STAGES = 8;

struct ScoreGatherParams {
  const int32_t* ids;           // [B x C]
  int32_t V;                    // rows of the corpus caches
  int32_t* flag;                // nullable: smallest slot whose id was outside [0, V)
  float* logits;                // [B x C]
  int B, C, d;
  int tiles_per_user, n_tiles;
  int stages;
  int* err;
};

template <int ELL>
__global__ void __launch_bounds__(SG_THREADS, 1)
k_score_gather_tc(const __grid_constant__ CUtensorMap tmLS, const __grid_constant__ CUtensorMap tmT,
                  const __grid_constant__ CUtensorMap tmW, const ScoreGatherParams p) {
  using namespace tc;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);

  const int KB = p.d / 64;                       // 64-element (128-byte) K blocks
  const uint32_t t_bytes = (uint32_t)KB * SG_TILE * 128;
  const uint32_t ls_bytes = (uint32_t)KB * ELL * 128;
  constexpr uint32_t w_bytes = (uint32_t)SG_TILE * ELL * 2;      // weight rows, not swizzled: row r at r * ELL * 2
  const uint32_t stage_bytes = t_bytes + ls_bytes + w_bytes;
  const int S = p.stages;

  uint64_t* full = reinterpret_cast<uint64_t*>(smem + (size_t)S * stage_bytes);
  uint64_t* empty = full + SG_MAX_STAGES;
  uint64_t* tmem_full = empty + SG_MAX_STAGES;
  uint64_t* tmem_empty = tmem_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tmem_empty + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr uint32_t TMEM_COLS = (2 * ELL < 32) ? 32 : 2 * ELL;

  // contiguous tile range per CTA: consecutive tiles share a user, so link states are re-fetched rarely
  const int t_begin = (int)(((int64_t)blockIdx.x * p.n_tiles) / gridDim.x);
  const int t_end = (int)(((int64_t)(blockIdx.x + 1) * p.n_tiles) / gridDim.x);

  if (threadIdx.x == 0) {
    // full: one arrival per producer thread, each carrying its byte count; empty: MMA commit + 4 epilogue warps
    for (int s = 0; s < S; ++s) { mbar_init(&full[s], 128); mbar_init(&empty[s], 5); }
    for (int b = 0; b < 2; ++b) { mbar_init(&tmem_full[b], 1); mbar_init(&tmem_empty[b], 4); }
    fence_barrier_init();
    prefetch_tmap(&tmLS); prefetch_tmap(&tmT); prefetch_tmap(&tmW);
  }
  if (warp == 4) {
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

  if (warp < 4) {
    // ------------------------------------------------------------------ producers: thread r fetches row r of the tile
    const uint32_t r = threadIdx.x;
    int stage_user[SG_MAX_STAGES];
#pragma unroll
    for (int s = 0; s < SG_MAX_STAGES; ++s) stage_user[s] = -1;
    const uint64_t pol_keep = policy_evict_last(), pol_stream = policy_evict_first();
    const int n_jobs = 32 * (KB + 1);              // per tile: 32 row quads x (KB embedding blocks + the weight rows)
    // Thread (warp w, lane g) issues the copies of row quad g (rows 4g..4g+3 of the tile) for K blocks w, w+4, ... and,
    // as job KB, the weight rows.  Its four ids are read two tiles ahead of their use, so the round trip of that read
    // is off the path that refills a freed stage.
    auto read_ids = [&](int t, int (&id)[4]) {
#pragma unroll
      for (int i = 0; i < 4; ++i) id[i] = 0;
      if (t >= t_end) return;
      const int b = t / p.tiles_per_user;
      const int c = (t % p.tiles_per_user) * SG_TILE + 4 * lane;
      const int32_t* src = p.ids + (int64_t)b * p.C + c;
      // rows past the user's last candidate fetch row 0 (a stage's byte count stays fixed; their logits are never written)
      if (c + 3 < p.C && (reinterpret_cast<uintptr_t>(src) & 15) == 0) {
        const int4 v = __ldg(reinterpret_cast<const int4*>(src));
        id[0] = v.x; id[1] = v.y; id[2] = v.z; id[3] = v.w;
      } else {
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (c + i < p.C) id[i] = __ldg(src + i);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (id[i] < 0 || id[i] >= p.V) id[i] = 0;      // out of range: row 0 stands in; the epilogue zeroes the logit
    };
    int id_now[4], id_next[4], id_after[4];
    read_ids(t_begin, id_next);
    read_ids(t_begin + 1, id_after);
    int it = 0;
    bool ok = true;
    for (int t = t_begin; t < t_end; ++t, ++it) {
      const int s = it % S;
#pragma unroll
      for (int i = 0; i < 4; ++i) { id_now[i] = id_next[i]; id_next[i] = id_after[i]; }
      read_ids(t + 2, id_after);
      if (!mbar_wait(&empty[s], ((uint32_t)(it / S) & 1u) ^ 1u, p.err, 101)) { ok = false; break; }
      const int b = t / p.tiles_per_user;
      uint8_t* st = smem + (size_t)s * stage_bytes;
      // every thread announces its own bytes before it issues its copies, so the phase cannot complete early
      bool load_ls = false;
      if (r == 0) {
#pragma unroll
        for (int q = 0; q < SG_MAX_STAGES; ++q)
          if (q == s) { load_ls = stage_user[q] != b; stage_user[q] = b; }
      }
      uint32_t my_bytes = load_ls ? ls_bytes : 0u;
      for (int j = (int)r; j < n_jobs; j += 128) my_bytes += (j >> 5) < KB ? 512u : (uint32_t)(4 * ELL * 2);
      mbar_arrive_expect_tx(&full[s], my_bytes);
      if (load_ls)
        for (int kb = 0; kb < KB; ++kb)
          tma_load_2d_hint(st + t_bytes + (size_t)kb * ELL * 128, &tmLS, kb * 64, b * ELL, &full[s], pol_keep);
      for (int j = (int)r; j < n_jobs; j += 128) {
        const int what = j >> 5;                   // what < KB: K block of the embedding rows, else the weight rows
        if (what < KB)
          tma_gather4_2d_hint(st + (size_t)what * SG_TILE * 128 + (size_t)lane * 512, &tmT, what * 64, id_now[0],
                              id_now[1], id_now[2], id_now[3], &full[s], pol_stream);
        else
          tma_gather4_2d_hint(st + t_bytes + ls_bytes + (size_t)lane * (4 * ELL * 2), &tmW, 0, id_now[0], id_now[1],
                              id_now[2], id_now[3], &full[s], pol_stream);
      }
    }
    if (r == 0 && (!ok || *(volatile int*)p.err != 0)) {
      // giving up: let the copies already issued land (bounded) before this CTA's shared memory goes away
      for (int j = 0; j < it && j < S; ++j) {
        const int last = it - 1 - j;
        mbar_wait_quiet(&full[last % S], (uint32_t)(last / S) & 1u);
      }
    }
  } else if (warp == 4) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(SG_TILE, ELL);
      int it = 0;
      for (int t = t_begin; t < t_end; ++t, ++it) {
        const int s = it % S;
        const uint32_t ph = (uint32_t)(it / S) & 1u;
        const int buf = it & 1;
        const uint32_t bph = (uint32_t)(it >> 1) & 1u;
        if (!mbar_wait(&tmem_empty[buf], bph ^ 1u, p.err, 102)) break;
        if (!mbar_wait(&full[s], ph, p.err, 103)) break;
        tc_fence_after();
        const uint32_t a0 = smem_u32(smem + (size_t)s * stage_bytes);
        const uint32_t b0 = a0 + t_bytes;
        const uint32_t d_tmem = tmem_base + (uint32_t)buf * ELL;
        for (int kb = 0; kb < KB; ++kb) {
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const uint64_t ad = make_sdesc_k_sw128(a0 + (uint32_t)kb * SG_TILE * 128 + k * 32);
            const uint64_t bd = make_sdesc_k_sw128(b0 + (uint32_t)kb * ELL * 128 + k * 32);
            mma_bf16_ss(d_tmem, ad, bd, idesc, (kb | k) != 0 ? 1u : 0u);
          }
        }
        mma_commit(&empty[s]);         // the stage may be refilled once these MMAs have read it
        mma_commit(&tmem_full[buf]);   // the accumulator is complete
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 5..8)
    const int q = warp & 3;                       // TMEM lane quarter this warp may read
    const int r = q * 32 + lane;                  // candidate row of the tile owned by this thread
    int it = 0;
    for (int t = t_begin; t < t_end; ++t, ++it) {
      const int buf = it & 1;
      const uint32_t bph = (uint32_t)(it >> 1) & 1u;
      const int b = t / p.tiles_per_user;
      const int c0 = (t % p.tiles_per_user) * SG_TILE;
      const bool valid = c0 + r < p.C;
      const int64_t grow = (int64_t)b * p.C + c0 + r;
      const int s = it % S;
      const int32_t my_id = valid ? __ldg(p.ids + grow) : 0;        // in L2 since the producers read it; used at the very end
      if (!mbar_wait(&full[s], (uint32_t)(it / S) & 1u, p.err, 105)) break;
      uint4 w[ELL / 8];
      {
        const uint4* wp = reinterpret_cast<const uint4*>(smem + (size_t)s * stage_bytes + t_bytes + ls_bytes) + r * (ELL / 8);
#pragma unroll
        for (int i = 0; i < ELL / 8; ++i) w[i] = wp[i];
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[s]);       // this warp has taken its rows out of the stage
      if (!mbar_wait(&tmem_full[buf], bph, p.err, 104)) break;
      tc_fence_after();
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
      if (valid) {
        const bool in_range = my_id >= 0 && my_id < p.V;
        p.logits[grow] = in_range ? acc : 0.f;
        if (!in_range && p.flag != nullptr) atomicMin(p.flag, (int32_t)grow);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 4) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

static int score_gather_stages(int ell, int d, size_t* smem_bytes) {
  const size_t stage = (size_t)(d / 64) * (SG_TILE + ell) * 128 + (size_t)SG_TILE * ell * 2;
  const size_t fixed = 1024 + 2 * SG_MAX_STAGES * 8 + 4 * 8 + 16;
  int S = (int)((226 * 1024 - fixed) / stage);
  if (S > SG_MAX_STAGES) S = SG_MAX_STAGES;
  *smem_bytes = (size_t)S * stage + fixed;
  return S;
}

bool score_gather_tc_supported(const ScoreArgs& a) {
  if (a.dtype != LIME_BF16 || a.cand_off != nullptr || a.cand_ids == nullptr) return false;
  if (!(a.ell == 16 || a.ell == 32 || a.ell == 64 || a.ell == 128)) return false;
  if (a.d % 64 != 0 || a.d > 512) return false;
  if (a.C <= 0 || a.total != (int64_t)a.B * a.C) return false;
  if ((reinterpret_cast<uintptr_t>(a.T) | reinterpret_cast<uintptr_t>(a.W)) & 15) return false;   // bulk copies want 16-byte alignment
  size_t smem;
  return score_gather_stages(a.ell, a.d, &smem) >= 2;
}

template <int ELL>
static lime_status launch_score_gather_t(const ScoreArgs& a, int* err, cudaStream_t st) {
  size_t smem;
  const int S = score_gather_stages(ELL, a.d, &smem);
  CUtensorMap tmLS, tmT, tmW;
  if (!make_tmap_bf16_sw128(&tmLS, a.LS, (uint64_t)a.B * ELL, (uint64_t)a.d, (uint64_t)a.d, ELL) ||
      !make_tmap_bf16_sw128(&tmT, a.T, (uint64_t)a.corpus_rows, (uint64_t)a.d, (uint64_t)(a.ldt ? a.ldt : a.d), 1) ||
      !make_tmap_bf16_plain(&tmW, a.W, (uint64_t)a.corpus_rows, ELL, (uint64_t)(a.ldw ? a.ldw : ELL), 1))
    return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
  ScoreGatherParams p;
  p.ids = a.cand_ids; p.logits = a.logits; p.V = (int32_t)a.corpus_rows; p.flag = a.dev_flag;
  p.B = a.B; p.C = a.C; p.d = a.d;
  p.tiles_per_user = (a.C + SG_TILE - 1) / SG_TILE;
  p.n_tiles = p.tiles_per_user * a.B;
  p.stages = S; p.err = err;
  const int grid = p.n_tiles < kSMs ? p.n_tiles : kSMs;
  LIME_CUDA(cudaFuncSetAttribute(k_score_gather_tc<ELL>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  ProfScope _p("k_score_gather_tc", st);
  launch_pdl(k_score_gather_tc<ELL>, dim3(grid), dim3(SG_THREADS), smem, st, tmLS, tmT, tmW, p);
  LIME_LAUNCH_CHECK("k_score_gather_tc");
  return LIME_OK;
}

lime_status launch_score_gather_tc(const ScoreArgs& a, int* err, cudaStream_t st) {
  switch (a.ell) {
    case 16: return launch_score_gather_t<16>(a, err, st);
    case 32: return launch_score_gather_t<32>(a, err, st);
    case 64: return launch_score_gather_t<64>(a, err, st);
    case 128: return launch_score_gather_t<128>(a, err, st);
  }
  return LIME_UNSUPPORTED_SHAPE;
}

}  // namespace lime
