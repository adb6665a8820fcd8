// Link-side preparation GEMM of the XOR layers on tcgen05 (bf16 in, fp32 accumulate in TMEM).
//
//   PREP   LN(T) [rows x d] . Wprep [d x N]  -> folded queries Q2, folded keys K2 (+ their row sums) and either the
//          folded gate / up operands G2t, U2t (N = 2*H*d + 2*H*f) or the plain link values V[T], stored transposed
//          (N = 2*H*d + d), that the streaming kernels contract against the history (Eq. 7); weights folded once at
//          set-up, see k_link_prep.cu.  d and f are multiples of 128.
// Persistent CTAs walk the 128-row x 128-column output tiles: warp 0 streams K blocks of A and B with TMA through a stage
// ring that runs on across tiles, warp 1 issues the MMAs into one of two TMEM accumulators, warps 2-9 (two threads per
// output row = TMEM lane, half of the tile's columns each) run the epilogue of a tile while the next tile's copies and MMAs proceed.  The GatedMLP on the
// link rows lives in k_link_mlp_tc.cu.
#include "lime_common.cuh"
#include "tc_common.cuh"

namespace lime {

constexpr int GM_THREADS = 64 + 256, GM_MAX_STAGES = 6;   // producer, MMA issuer, eight epilogue warps
constexpr uint32_t GM_SUB = 128 * 128;    // [128 rows x 64 bf16]

enum { GM_EPI_PREP = 0, GM_EPI_ROWS_T = 1 };

struct GemmParams {
  int64_t M;            // valid rows of A / C
  int kblocks;          // K / 64
  int stages;
  int m_tiles, n_tiles; // output tiles of 128 rows x NT columns
  // PREP
  int ell, H, shared_rows;          // rows are (user, link): user = row / ell
  int d, f, plain_v;                // output widths; plain_v: the third segment is V[T] (d columns) instead of G2 | U2
  __nv_bfloat16 *Q2, *K2, *G2t, *U2t, *V2t;
  float *cQ, *cK;                   // row sums of Q2 / K2 (only with d = 128: one n-tile per row)
  // ROWS_T: out[(row / group) * n_cols + col][row % group] for col < n_cols (bf16): the product transposed per group of rows
  __nv_bfloat16* out_t;
  int group, n_cols;
  int* err;
};

__device__ __forceinline__ uint32_t gm_pack(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

template <int EPI, int NT>
__global__ void __launch_bounds__(GM_THREADS, 1)
k_gemm_tc(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmParams p) {
  using namespace tc;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  constexpr uint32_t B_SUB = (uint32_t)NT * 128;
  constexpr uint32_t STAGE = GM_SUB + B_SUB;
  const int S = p.stages;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)S * STAGE);
  uint64_t* full = bars;
  uint64_t* empty = bars + GM_MAX_STAGES;
  uint64_t* acc_full = bars + 2 * GM_MAX_STAGES;          // [2] accumulator of a tile complete
  uint64_t* acc_empty = acc_full + 2;                      // [2] read out by the four epilogue warps
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // persistent: output tiles (m-tile, n-tile), n fastest, dealt round-robin to the CTAs; the stage ring and the two
  // accumulators run on across tiles, so the copies and MMAs of the next tile overlap this tile's epilogue
  const int n_tiles = p.m_tiles * p.n_tiles;
  const int KB = p.kblocks;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 8); }
    fence_barrier_init();
    prefetch_tmap(&tmA); prefetch_tmap(&tmB);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 2 * NT); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // set-up done: the next kernel's CTAs may become resident; nothing an earlier kernel wrote is read before this wait
  pdl_launch_dependents();
  pdl_wait();

  if (warp == 0) {
    if (lane == 0) {
      const uint64_t pol = policy_evict_last();
      bool ok = true;
      int it = 0;
      for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
        const int m0 = (t / p.n_tiles) * 128, nt = t % p.n_tiles;
        for (int kb = 0; kb < KB; ++kb, ++it) {
          const int s = it % S;
          if (!mbar_wait(&empty[s], ((uint32_t)(it / S) & 1u) ^ 1u, p.err, 71)) { ok = false; break; }
          uint8_t* st = smem + (size_t)s * STAGE;
          mbar_arrive_expect_tx(&full[s], STAGE);
          tma_load_2d_hint(st, &tmA, kb * 64, m0, &full[s], pol);
          tma_load_2d_hint(st + GM_SUB, &tmB, kb * 64, nt * NT, &full[s], pol);
        }
      }
      if (!ok || *(volatile int*)p.err != 0)
        for (int j = 0; j < it && j < S; ++j) mbar_wait_quiet(&full[(it - 1 - j) % S], (uint32_t)((it - 1 - j) / S) & 1u);
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(128, NT);
      const uint32_t sbase = smem_u32(smem);
      bool ok = true;
      int it = 0, n = 0;
      for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++n) {
        const int buf = n & 1;
        if (!mbar_wait(&acc_empty[buf], ((uint32_t)(n >> 1) & 1u) ^ 1u, p.err, 74)) { ok = false; break; }
        tc_fence_after();
        for (int kb = 0; kb < KB && ok; ++kb, ++it) {
          const int s = it % S;
          if (!mbar_wait(&full[s], (uint32_t)(it / S) & 1u, p.err, 72)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int k = 0; k < 4; ++k)
            mma_bf16_ss(tmem_base + (uint32_t)buf * NT, make_sdesc_k_sw128(sbase + s * STAGE + k * 32),
                        make_sdesc_k_sw128(sbase + s * STAGE + GM_SUB + k * 32), idesc, (kb | k) != 0);
          mma_commit(&empty[s]);
        }
        if (ok) mma_commit(&acc_full[buf]);
      }
    }
  } else {
    const int q = warp & 3;
    const int r = q * 32 + lane;
    const int half = (warp - 2) >> 2;                  // which half of the tile's columns this warp reads out
    const int cb = half * (NT / 2), ce = cb + NT / 2;
    int n = 0;
    for (int t = blockIdx.x; t < n_tiles; t += gridDim.x, ++n) {
      const int buf = n & 1;
      const int m0 = (t / p.n_tiles) * 128, nt = t % p.n_tiles;
      const int64_t row = (int64_t)m0 + r;
      const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)buf * NT;
      if (!mbar_wait(&acc_full[buf], (uint32_t)(n >> 1) & 1u, p.err, 73)) break;
      tc_fence_after();
      const bool valid = row < p.M;
      if (EPI == GM_EPI_PREP) {
        // n-tile -> (segment, head, 128-column part); row -> (user, link)
        const int n0 = nt * 128, qk_cols = 2 * p.H * p.d;
        const int64_t u = row / p.ell;
        const int l = (int)(row % p.ell);
        const int HL = p.H * p.ell;
        if (n0 < qk_cols) {
          const int seg = n0 / (p.H * p.d), h = (n0 / p.d) % p.H, i0 = n0 % p.d;
          __nv_bfloat16* dst = (seg == 0 ? p.Q2 : p.K2) + ((u * HL) + h * p.ell + l) * p.d + i0;
          float* cs = seg == 0 ? p.cQ : p.cK;
          float rs = 0.f;
#pragma unroll
          for (int c = cb; c < ce; c += 16) {
            float v[16];
            tmem_ld_32x16(lane_addr + c, v);
            tmem_wait_ld();
            uint4 o0, o1;
            o0.x = gm_pack(v[0], v[1]); o0.y = gm_pack(v[2], v[3]); o0.z = gm_pack(v[4], v[5]); o0.w = gm_pack(v[6], v[7]);
            o1.x = gm_pack(v[8], v[9]); o1.y = gm_pack(v[10], v[11]); o1.z = gm_pack(v[12], v[13]); o1.w = gm_pack(v[14], v[15]);
#pragma unroll
            for (int j = 0; j < 16; ++j) rs += __bfloat162float(__float2bfloat16_rn(v[j]));   // sum of what is stored
            if (valid) {
              *reinterpret_cast<uint4*>(dst + c) = o0;
              *reinterpret_cast<uint4*>(dst + c + 8) = o1;
            }
          }
          if (cs != nullptr && half == 0) {
            // the row sum spans the whole tile: this warp also reads the other half's columns for it
#pragma unroll
            for (int c = ce; c < NT; c += 16) {
              float v[16];
              tmem_ld_32x16(lane_addr + c, v);
              tmem_wait_ld();
#pragma unroll
              for (int j = 0; j < 16; ++j) rs += __bfloat162float(__float2bfloat16_rn(v[j]));
            }
            if (valid) cs[u * HL + h * p.ell + l] = rs;
          }
        } else {
          // transposed stores: G2t / U2t [user][f][(h, l)], or V2t [user][d][l]
          __nv_bfloat16* dst;
          int64_t ld;
          if (p.plain_v) {
            dst = p.V2t + (u * p.d + (n0 - qk_cols)) * p.ell + l;
            ld = p.ell;
          } else {
            const int n1 = n0 - qk_cols;
            const int seg = n1 / (p.H * p.f), h = (n1 / p.f) % p.H, i0 = n1 % p.f;
            dst = (seg == 0 ? p.G2t : p.U2t) + (u * p.f + i0) * HL + h * p.ell + l;
            ld = HL;
          }
#pragma unroll
          for (int c = cb; c < ce; c += 16) {
            float v[16];
            tmem_ld_32x16(lane_addr + c, v);
            tmem_wait_ld();
            if (valid) {
#pragma unroll
              for (int j = 0; j < 16; ++j) dst[(int64_t)(c + j) * ld] = __float2bfloat16_rn(v[j]);
            }
          }
        }
      } else if (EPI == GM_EPI_ROWS_T) {
        const int64_t u = row / p.group;
        const int l = (int)(row % p.group);
        __nv_bfloat16* dst = p.out_t + (u * p.n_cols + (int64_t)nt * NT) * p.group + l;
#pragma unroll
        for (int c = cb; c < ce; c += 16) {
          float v[16];
          tmem_ld_32x16(lane_addr + c, v);
          tmem_wait_ld();
          if (valid) {
#pragma unroll
            for (int j = 0; j < 16; ++j)
              if (nt * NT + c + j < p.n_cols) dst[(int64_t)(c + j) * p.group] = __float2bfloat16_rn(v[j]);
          }
        }
      }
      // the accumulator has been read: the MMA issuer may reuse it for the tile after next
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[buf]);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 2 * NT);
  }
}

template <int EPI, int NT>
static lime_status launch_gemm(const void* A, int64_t M, int K, const void* Bt, int n_rows_b, int n_tiles, GemmParams p,
                               const char* name, cudaStream_t st) {
  if (M == 0) return LIME_OK;
  CUtensorMap tmA, tmB;
  if (!make_tmap_bf16_sw128(&tmA, A, (uint64_t)M, (uint64_t)K, (uint64_t)K, 128) ||
      !make_tmap_bf16_sw128(&tmB, Bt, (uint64_t)n_rows_b, (uint64_t)K, (uint64_t)K, 128))
    return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
  constexpr size_t stage = GM_SUB + (size_t)NT * 128;
  const int64_t m_tiles = (M + 127) / 128;
  if (m_tiles * n_tiles > 0x7fffffffLL) return LIME_UNSUPPORTED_SHAPE;
  p.M = M; p.kblocks = K / 64; p.m_tiles = (int)m_tiles; p.n_tiles = n_tiles;
  p.stages = GM_MAX_STAGES;
  const size_t smem = p.stages * stage + 256 + 1024;
  LIME_CUDA(cudaFuncSetAttribute(k_gemm_tc<EPI, NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  ProfScope _p(name, st);
  const int64_t tiles = m_tiles * n_tiles;
  const unsigned grid = (unsigned)(tiles < kSMs ? tiles : kSMs);
  launch_pdl(k_gemm_tc<EPI, NT>, dim3(grid), dim3(GM_THREADS), smem, st, tmA, tmB, p);
  LIME_LAUNCH_CHECK(name);
  return LIME_OK;
}

lime_status launch_gemm_prep(const LinkGemmArgs& a, cudaStream_t st) {
  GemmParams p{};
  p.ell = a.ell; p.H = a.H; p.d = a.K; p.f = a.f; p.plain_v = a.plain_v;
  p.Q2 = (__nv_bfloat16*)a.Q2; p.K2 = (__nv_bfloat16*)a.K2; p.G2t = (__nv_bfloat16*)a.G2t;
  p.U2t = (__nv_bfloat16*)a.U2t; p.V2t = (__nv_bfloat16*)a.V2t; p.cQ = a.cQ; p.cK = a.cK; p.err = a.err;
  if (a.K % 128 || a.f % 128 || a.K < 128) return LIME_UNSUPPORTED_SHAPE;
  // column segments: Q2 | K2 | (G2 | U2, or V); the last layer needs only the queries
  const int cols_all = 2 * a.H * a.K + (a.plain_v ? a.K : 2 * a.H * a.f);
  const int n_tiles = (a.need_hist ? cols_all : a.H * a.K) / 128;
  return launch_gemm<GM_EPI_PREP, 128>(a.A, a.M, a.K, a.Bt, cols_all, n_tiles, p, "k_gemm_tc_prep", st);
}

// A [M x K] . Bt^T with Bt [n_cols x K] (bf16, K a multiple of 64): the product as bf16, transposed per group of `group`
// consecutive rows: out_t [M / group][n_cols][group]
lime_status launch_gemm_rows_t(const void* A, int64_t M, int K, const void* Bt, int n_cols, int group, void* out_t, int* err,
                               const char* name, cudaStream_t st) {
  if (K % 64 || K < 64 || n_cols < 1 || group < 1) return LIME_UNSUPPORTED_SHAPE;
  GemmParams p{};
  p.out_t = (__nv_bfloat16*)out_t; p.group = group; p.n_cols = n_cols; p.err = err;
  return launch_gemm<GM_EPI_ROWS_T, 128>(A, M, K, Bt, n_cols, (n_cols + 127) / 128, p, name, st);
}

}  // namespace lime
