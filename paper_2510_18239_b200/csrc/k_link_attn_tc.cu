// Links attend over the history on the 5th-generation tensor cores (bf16 storage):
//
//   O[T]_h = softmax_j( Q[T]_h K[S]_h^T * scale ) V[S]_h,  K[S] = LN(S) W_K,  V[S] = LN(S) W_V          (Eq. 3 / Eq. 7)
//
// With W_K folded into the link queries (Q2, see k_link_prep.cu) and W_V applied after the attention, both
// contractions run against the *stored* history rows X, which are streamed exactly once (TMA) and used both as
// keys and as values - K[S] and V[S] are never materialised:
//   scores [HL x 128]   = Q2 [HL x d] . X_tile^T            LayerNorm folded in afterwards:
//                         s_ij = rstd_j * (raw_ij - mu_j * rowsum(Q2)_i)
//   acc    [HL x d]    += P' [HL x 128] . X_tile            P'_ij = p_ij * rstd_j;  the mean term sum_j P'_ij mu_j is
//                                                           a per-row scalar subtracted from every column at the end
//   O[T]_{l,h} = (acc_(h,l) / sum) . W_V[:, head h]         (chunks merged in k_link_prep.cu, W_V folded into the GEMM after)
// HL = H * ell stacked (head, link) rows = 128 TMEM lanes; thread i of the softmax warps owns row i: an online
// softmax whose reference maximum is only raised when the true maximum exceeds it by more than 8 (then the
// accumulator row is rescaled in TMEM), so most tiles need no correction pass.
// One CTA per (user, chunk of the history); warp 0 TMA producer, warp 1 MMA issuer, warps 2-5 softmax.
//
// Built for d = 128 and H * ell = 128.
#include "lime_common.cuh"
#include "tc_common.cuh"

namespace lime {

constexpr int LA_D = 128, LA_HL = 128, LA_TILE = 128, LA_THREADS = 192, LA_XSTAGES = 3;
constexpr uint32_t LA_SUB = 128 * 128;
constexpr uint32_t LA_X_STAGE = 2 * LA_SUB;
constexpr uint32_t LA_OFF_X = 0;
constexpr uint32_t LA_OFF_Q2 = LA_XSTAGES * LA_X_STAGE;
constexpr uint32_t LA_OFF_P = LA_OFF_Q2 + 2 * LA_SUB;        // 2 buffers of [HL x 128 tokens]
constexpr uint32_t LA_OFF_STATS = LA_OFF_P + 4 * LA_SUB;     // per X stage: mu[128], rstd[128]
constexpr uint32_t LA_OFF_BAR = LA_OFF_STATS + LA_XSTAGES * 2 * 128 * 4;
constexpr uint32_t LA_SMEM = LA_OFF_BAR + 256;
constexpr float LA_RESCALE_THRESHOLD = 8.0f;

struct LinkAttnParams {
  const float* cQ;                // [users x HL]
  const int32_t* off;
  const int32_t* chunk_start;     // [B+1] prefix of per-user chunk counts
  int B, chunk, shared, ln;
  float ln_eps;
  float *part_m, *part_s, *part_acc;   // [items x HL], [items x HL], [items x HL x d]
  int* err;
};

__device__ __forceinline__ uint32_t la_chunk_addr(uint32_t r, uint32_t c) { return r * 128u + ((c ^ (r & 7u)) << 4); }
__device__ __forceinline__ uint32_t la_pack(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

__global__ void __launch_bounds__(LA_THREADS, 1)
k_link_attn_tc(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmQ2, const LinkAttnParams p) {
  using namespace tc;
  const int item = blockIdx.x;
  if (item >= p.chunk_start[p.B]) return;
  extern __shared__ __align__(1024) uint8_t smem[];
  if ((smem_u32(smem) & 1023u) != 0) {
    if (threadIdx.x == 0) atomicCAS(p.err, 0, 91);
    return;
  }
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + LA_OFF_BAR);
  uint64_t* x_full = bars;             // [3]
  uint64_t* x_empty = bars + 3;        // [3]  second MMA of the tile done
  uint64_t* stats_ready = bars + 6;    // [3]  128 arrivals
  uint64_t* q_full = bars + 9;
  uint64_t* s_full = bars + 10;        // [2]  score tile in TMEM
  uint64_t* p_ready = bars + 12;       // [2]  P' in smem (4 warps)
  uint64_t* p_free = bars + 14;        // [2]  second MMA done reading P' (and accumulator up to date)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 16);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = upper_user(p.chunk_start, p.B, item);
  const int tok0 = p.off[b] + (item - p.chunk_start[b]) * p.chunk;
  const int tok1 = min(p.off[b + 1], tok0 + p.chunk);
  const int n_tiles = (tok1 - tok0 + LA_TILE - 1) / LA_TILE;

  if (threadIdx.x == 0) {
    for (int s = 0; s < LA_XSTAGES; ++s) { mbar_init(&x_full[s], 1); mbar_init(&x_empty[s], 1); mbar_init(&stats_ready[s], 128); }
    mbar_init(q_full, 1);
    for (int i = 0; i < 2; ++i) { mbar_init(&s_full[i], 1); mbar_init(&p_ready[i], 4); mbar_init(&p_free[i], 1); }
    fence_barrier_init();
    prefetch_tmap(&tmX); prefetch_tmap(&tmQ2);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  constexpr uint32_t COL_S = 0, COL_O = 256;      // scores: 2 x 128 columns; accumulator: d columns

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      const uint64_t pol_stream = policy_evict_first(), pol_keep = policy_evict_last();
      mbar_arrive_expect_tx(q_full, 2 * LA_SUB);
      for (int kb = 0; kb < 2; ++kb)
        tma_load_2d_hint(smem + LA_OFF_Q2 + kb * LA_SUB, &tmQ2, kb * 64, (p.shared ? 0 : b) * LA_HL, q_full, pol_keep);
      bool ok = true;
      int t = 0;
      for (; t < n_tiles; ++t) {
        const int s = t % LA_XSTAGES;
        if (!mbar_wait(&x_empty[s], ((uint32_t)(t / LA_XSTAGES) & 1u) ^ 1u, p.err, 41)) { ok = false; break; }
        mbar_arrive_expect_tx(&x_full[s], LA_X_STAGE);
        for (int kb = 0; kb < 2; ++kb)
          tma_load_2d_hint(smem + LA_OFF_X + s * LA_X_STAGE + kb * LA_SUB, &tmX, kb * 64, tok0 + t * LA_TILE, &x_full[s],
                           pol_stream);
      }
      if (!ok || *(volatile int*)p.err != 0) {
        for (int j = 0; j < t && j < LA_XSTAGES; ++j)
          mbar_wait_quiet(&x_full[(t - 1 - j) % LA_XSTAGES], (uint32_t)((t - 1 - j) / LA_XSTAGES) & 1u);
        mbar_wait_quiet(q_full, 0);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_s = make_idesc_bf16(128, 128);                 // Q2 . X^T  : both K-major
      constexpr uint32_t idesc_o = make_idesc_bf16(128, 128, false, true);    // P' . X    : B is MN-major
      const uint32_t sbase = smem_u32(smem);
      auto issue_scores = [&](int t) -> bool {
        const int s = t % LA_XSTAGES;
        if (!mbar_wait(&x_full[s], (uint32_t)(t / LA_XSTAGES) & 1u, p.err, 51)) return false;
        tc_fence_after();
        for (int kk = 0; kk < 8; ++kk) {
          const uint32_t o = (uint32_t)(kk >> 2) * LA_SUB + (uint32_t)(kk & 3) * 32;
          mma_bf16_ss(tmem_base + COL_S + (uint32_t)(t & 1) * 128, make_sdesc_k_sw128(sbase + LA_OFF_Q2 + o),
                      make_sdesc_k_sw128(sbase + LA_OFF_X + s * LA_X_STAGE + o), idesc_s, kk != 0);
        }
        mma_commit(&s_full[t & 1]);
        return true;
      };
      bool ok = mbar_wait(q_full, 0, p.err, 50);
      if (ok && n_tiles > 0) ok = issue_scores(0);
      for (int t = 0; t < n_tiles && ok; ++t) {
        // the next tile's scores overlap this tile's softmax (its score buffer was released by p_ready(t-1))
        if (t + 1 < n_tiles && !issue_scores(t + 1)) { ok = false; break; }
        const int s = t % LA_XSTAGES, pb = t & 1;
        if (!mbar_wait(&p_ready[pb], (uint32_t)(t >> 1) & 1u, p.err, 52)) { ok = false; break; }
        tc_fence_after();
        for (int kk = 0; kk < 8; ++kk) {      // contraction over the tile's 128 tokens, 16 per instruction
          const uint32_t oa = (uint32_t)(kk >> 2) * LA_SUB + (uint32_t)(kk & 3) * 32;
          mma_bf16_ss(tmem_base + COL_O, make_sdesc_k_sw128(sbase + LA_OFF_P + pb * 2 * LA_SUB + oa),
                      make_sdesc_mn_sw128(sbase + LA_OFF_X + s * LA_X_STAGE + (uint32_t)kk * 2048, LA_SUB), idesc_o,
                      (t | kk) != 0);
        }
        mma_commit(&x_empty[s]);
        mma_commit(&p_free[pb]);
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax warps (2..5): thread i owns row i
    const int q = warp & 3;
    const uint32_t r = (uint32_t)(q * 32 + lane);
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
    const float cq = p.cQ[(int64_t)(p.shared ? 0 : b) * LA_HL + r];
    float m_ref = -INFINITY, l_sum = 0.f, mean_corr = 0.f;
    bool ok = true;
    for (int t = 0; t < n_tiles && ok; ++t) {
      const int s = t % LA_XSTAGES, pb = t & 1;
      const uint32_t xph = (uint32_t)(t / LA_XSTAGES) & 1u;
      float* mu_s = reinterpret_cast<float*>(smem + LA_OFF_STATS) + s * 256;
      float* rstd_s = mu_s + 128;
      const int nvalid = min(LA_TILE, tok1 - tok0 - t * LA_TILE);
      // LayerNorm statistics of token r of this tile (each thread one token), shared through smem
      if (!mbar_wait(&x_full[s], xph, p.err, 61)) { ok = false; break; }
      {
        float mu = 0.f, rstd = 1.f;
        if (p.ln) {
          const uint8_t* xs = smem + LA_OFF_X + s * LA_X_STAGE + r * 128u;
          float sum = 0.f;
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            const int cc = (c + (int)r) & 7;
            const uint4 u = *reinterpret_cast<const uint4*>(xs + (c >> 3) * LA_SUB + cc * 16);
            const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) sum += __uint_as_float(w[j] << 16) + __uint_as_float(w[j] & 0xffff0000u);
          }
          mu = sum * (1.0f / LA_D);
          float var = 0.f;
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            const int cc = (c + (int)r) & 7;
            const uint4 u = *reinterpret_cast<const uint4*>(xs + (c >> 3) * LA_SUB + cc * 16);
            const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float a = __uint_as_float(w[j] << 16) - mu, bb = __uint_as_float(w[j] & 0xffff0000u) - mu;
              var = fmaf(a, a, var);
              var = fmaf(bb, bb, var);
            }
          }
          rstd = rsqrtf(var * (1.0f / LA_D) + p.ln_eps);
        }
        mu_s[r] = mu;
        rstd_s[r] = rstd;
        mbar_arrive(&stats_ready[s]);
      }
      if (!mbar_wait(&stats_ready[s], xph, p.err, 62)) { ok = false; break; }
      if (!mbar_wait(&s_full[pb], (uint32_t)(t >> 1) & 1u, p.err, 63)) { ok = false; break; }
      tc_fence_after();

      // pass 1: row maximum of the tile's valid scores
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < LA_TILE; c += 16) {
        float v[16];
        tmem_ld_32x16(lane_addr + COL_S + pb * 128 + c, v);
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const float sc = (v[j] - cq * mu_s[c + j]) * rstd_s[c + j];
          if (c + j < nvalid) mx = fmaxf(mx, sc);
        }
      }
      // raise the reference maximum only when it is exceeded by more than the threshold (or unset)
      const bool need = mx > m_ref + LA_RESCALE_THRESHOLD;
      const float m_new = need ? mx : m_ref;
      const float factor = (need && m_ref != -INFINITY) ? __expf(m_ref - m_new) : 1.0f;
      if (__any_sync(0xffffffffu, need && t > 0)) {
        // the accumulator must be quiescent: wait for the previous tile's second MMA, then scale this row
        if (!mbar_wait(&p_free[(t - 1) & 1], (uint32_t)((t - 1) >> 1) & 1u, p.err, 64)) { ok = false; break; }
        tc_fence_after();
#pragma unroll
        for (int c = 0; c < LA_D; c += 16) {
          float v[16];
          tmem_ld_32x16(lane_addr + COL_O + c, v);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 16; ++j) v[j] *= factor;
          tmem_st_32x16(lane_addr + COL_O + c, v);
        }
        tmem_wait_st();
      }
      l_sum *= factor;
      mean_corr *= factor;
      m_ref = m_new;

      // the P' buffer of two tiles ago must have been consumed
      if (t >= 2 && !mbar_wait(&p_free[pb], (uint32_t)((t - 2) >> 1) & 1u, p.err, 65)) { ok = false; break; }
      // pass 2: p = exp(s - m_ref); P' = p * rstd -> smem (A operand, K-major over the tile's tokens)
      uint8_t* pbuf = smem + LA_OFF_P + pb * 2 * LA_SUB;
#pragma unroll
      for (int c = 0; c < LA_TILE; c += 16) {
        float v[16];
        tmem_ld_32x16(lane_addr + COL_S + pb * 128 + c, v);
        tmem_wait_ld();
        float pp[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const float rs = rstd_s[c + j], mj = mu_s[c + j];
          const float sc = (v[j] - cq * mj) * rs;
          const float e = (c + j < nvalid) ? __expf(sc - m_ref) : 0.f;
          l_sum += e;
          // what the MMA will see is the bf16-rounded P'; use the same rounded value for the mean term
          const float pr = __bfloat162float(__float2bfloat16_rn(e * rs));
          mean_corr = fmaf(pr, mj, mean_corr);
          pp[j] = pr;
        }
#pragma unroll
        for (int c8 = 0; c8 < 2; ++c8) {
          const int k = c + c8 * 8;
          uint4 o;
          o.x = la_pack(pp[c8 * 8 + 0], pp[c8 * 8 + 1]);
          o.y = la_pack(pp[c8 * 8 + 2], pp[c8 * 8 + 3]);
          o.z = la_pack(pp[c8 * 8 + 4], pp[c8 * 8 + 5]);
          o.w = la_pack(pp[c8 * 8 + 6], pp[c8 * 8 + 7]);
          *reinterpret_cast<uint4*>(pbuf + (k >> 6) * LA_SUB + la_chunk_addr(r, (uint32_t)(k & 63) >> 3)) = o;
        }
      }
      tc_fence_before();
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(&p_ready[pb]);
    }
    // chunk result: (m_ref, sum, accumulator row minus the mean term) -> scratch, merged per user afterwards
    if (ok && n_tiles > 0) ok = mbar_wait(&p_free[(n_tiles - 1) & 1], (uint32_t)((n_tiles - 1) >> 1) & 1u, p.err, 66);
    if (ok) {
      tc_fence_after();
      float* dst = p.part_acc + ((int64_t)item * LA_HL + r) * LA_D;
#pragma unroll
      for (int c = 0; c < LA_D; c += 16) {
        float v[16];
        tmem_ld_32x16(lane_addr + COL_O + c, v);
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < 16; j += 4)
          *reinterpret_cast<float4*>(dst + c + j) =
              make_float4(v[j] - mean_corr, v[j + 1] - mean_corr, v[j + 2] - mean_corr, v[j + 3] - mean_corr);
      }
      p.part_m[(int64_t)item * LA_HL + r] = m_ref;
      p.part_s[(int64_t)item * LA_HL + r] = l_sum;
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
  return dtype == LIME_BF16 && d == LA_D && H * ell == LA_HL && phi == LIME_PHI_SOFTMAX;
}

lime_status launch_link_attn_tc(const LinkAttnArgs& a, cudaStream_t st) {
  if (a.n_chunk_upper <= 0 || a.total == 0) return LIME_OK;   // no history: the merge step writes zeros
  CUtensorMap tmX, tmQ2;
  const uint64_t users = a.shared ? 1 : (uint64_t)a.B;
  if (!make_tmap_bf16_sw128(&tmX, a.hist, (uint64_t)a.total, LA_D, LA_D, LA_TILE) ||
      !make_tmap_bf16_sw128(&tmQ2, a.Q2, users * LA_HL, LA_D, LA_D, 128))
    return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
  LinkAttnParams p;
  p.cQ = a.cQ; p.off = a.off; p.chunk_start = a.chunk_start; p.B = a.B; p.chunk = a.chunk; p.shared = a.shared;
  p.ln = a.ln; p.ln_eps = a.ln_eps; p.part_m = a.part_m; p.part_s = a.part_s; p.part_acc = a.part_acc; p.err = a.err;
  LIME_CUDA(cudaFuncSetAttribute(k_link_attn_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)LA_SMEM));
  {
    ProfScope _p("k_link_attn_tc", st);
    k_link_attn_tc<<<a.n_chunk_upper, LA_THREADS, LA_SMEM, st>>>(tmX, tmQ2, p);
    LIME_LAUNCH_CHECK("k_link_attn_tc");
  }
  return LIME_OK;
}

}  // namespace lime
