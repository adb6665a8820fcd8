// Offline candidate->link attention weights on the 5th-generation tensor cores (Eq. 4, "pre-computed and cached"),
// bf16 storage:
//
//   W[c, :] = softmax_l( <T_c, keff_l> ),   keff = ((L W_K^c)(W_Q^c)^T) * cand_scale   (fp32, formed at set-up)
//
// The scores T [M x d] . keff^T [d x ell] are a dense contraction streamed over the M catalogue items, so they run
// as tcgen05.mma with the accumulator in TMEM.  To keep fp32-level accuracy of the effective keys with bf16
// operands, keff is split into a bf16 high part and a bf16 remainder (keff = hi + lo up to 2^-17 relative) stacked
// as one B operand [2 ell x d]: one MMA of N = 2 ell yields both partial scores, which the epilogue adds.
// Persistent, warp-specialised stream like the scorer:
//   warp 0    : TMA producer - item tile [128 x d] into a ring of 128B-swizzled stages (keys once, resident)
//   warp 1    : MMA issuer   - d/16 tcgen05.mma (M=128, N=2 ell, K=16) per tile into one of two TMEM accumulators
//   warps 2-5 : epilogue     - thread r owns item row r (TMEM lane r): row softmax in registers, bf16 row to global
//                              (GROUP < ELL: the ELL keys are ELL / GROUP heads' keys and the softmax runs per head)
// HBM traffic per item is the algorithmic minimum: its embedding row in, its weight row out.
#include "lime_common.cuh"
#include "tc_common.cuh"

namespace lime {

constexpr int PCT_TILE = 128;
constexpr int PCT_THREADS = 192;
constexpr int PCT_MAX_STAGES = 8;

struct PrecomputeTcParams {
  __nv_bfloat16* out;     // [M x ELL]
  int64_t M;
  int d, n_tiles, stages;
  int* err;
};

// keff fp32 [ell x d] -> bf16 [2 ell x d]: rows 0..ell-1 the rounded value, rows ell..2ell-1 the rounded remainder
__global__ void k_keff_split(const float* __restrict__ keff, int n, __nv_bfloat16* __restrict__ out) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const float v = keff[i];
  const __nv_bfloat16 hi = __float2bfloat16_rn(v);
  out[i] = hi;
  out[n + i] = __float2bfloat16_rn(v - __bfloat162float(hi));
}

lime_status launch_keff_split(const float* keff, int ell, int d, void* out, cudaStream_t st) {
  const int n = ell * d;
  ProfScope _p("k_keff_split", st);
  k_keff_split<<<(n + 255) / 256, 256, 0, st>>>(keff, n, (__nv_bfloat16*)out);
  LIME_LAUNCH_CHECK("k_keff_split");
  return LIME_OK;
}

__device__ __forceinline__ uint32_t pct_pack(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

template <int ELL, int GROUP>
__global__ void __launch_bounds__(PCT_THREADS, 1)
k_precompute_tc(const __grid_constant__ CUtensorMap tmT, const __grid_constant__ CUtensorMap tmK, const PrecomputeTcParams p) {
  using namespace tc;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);

  const int KB = p.d / 64;
  const uint32_t t_bytes = (uint32_t)KB * PCT_TILE * 128;
  const uint32_t k_bytes = (uint32_t)KB * 2 * ELL * 128;
  const int S = p.stages;
  uint8_t* keys = smem;                         // [KB][2 ELL rows x 128 B]
  uint8_t* ring = smem + k_bytes;               // S stages of [KB][128 rows x 128 B]

  uint64_t* full = reinterpret_cast<uint64_t*>(ring + (size_t)S * t_bytes);
  uint64_t* empty = full + PCT_MAX_STAGES;
  uint64_t* tmem_full = empty + PCT_MAX_STAGES;
  uint64_t* tmem_empty = tmem_full + 2;
  uint64_t* keys_full = tmem_empty + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(keys_full + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr uint32_t TMEM_COLS = (4 * ELL < 32) ? 32 : 4 * ELL;      // two accumulators of 2 ELL columns

  const int t_begin = (int)(((int64_t)blockIdx.x * p.n_tiles) / gridDim.x);
  const int t_end = (int)(((int64_t)(blockIdx.x + 1) * p.n_tiles) / gridDim.x);

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&tmem_full[b], 1); mbar_init(&tmem_empty[b], 4); }
    mbar_init(keys_full, 1);
    fence_barrier_init();
    prefetch_tmap(&tmT);
    prefetch_tmap(&tmK);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0 && t_begin < t_end) {
      const uint64_t pol_stream = policy_evict_first(), pol_keep = policy_evict_last();
      mbar_arrive_expect_tx(keys_full, k_bytes);
      for (int kb = 0; kb < KB; ++kb) {
        // rows of the stacked [hi | lo] keys, in boxes of at most 128 rows
        for (int r0 = 0; r0 < 2 * ELL; r0 += (2 * ELL < 128 ? 2 * ELL : 128))
          tma_load_2d_hint(keys + (size_t)kb * 2 * ELL * 128 + (size_t)r0 * 128, &tmK, kb * 64, r0, keys_full, pol_keep);
      }
      int it = 0;
      bool ok = true;
      for (int t = t_begin; t < t_end; ++t, ++it) {
        const int s = it % S;
        if (!mbar_wait(&empty[s], ((uint32_t)(it / S) & 1u) ^ 1u, p.err, 81)) { ok = false; break; }
        uint8_t* st = ring + (size_t)s * t_bytes;
        mbar_arrive_expect_tx(&full[s], t_bytes);
        for (int kb = 0; kb < KB; ++kb)
          tma_load_2d_hint(st + (size_t)kb * PCT_TILE * 128, &tmT, kb * 64, t * PCT_TILE, &full[s], pol_stream);
      }
      if (!ok || *(volatile int*)p.err != 0) {
        for (int j = 0; j < it && j < S; ++j) {
          const int last = it - 1 - j;
          mbar_wait_quiet(&full[last % S], (uint32_t)(last / S) & 1u);
        }
        mbar_wait_quiet(keys_full, 0);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && t_begin < t_end) {
      constexpr uint32_t idesc = make_idesc_bf16(PCT_TILE, 2 * ELL);
      bool ok = mbar_wait(keys_full, 0, p.err, 82);
      int it = 0;
      for (int t = t_begin; t < t_end && ok; ++t, ++it) {
        const int s = it % S;
        const int buf = it & 1;
        if (!mbar_wait(&tmem_empty[buf], ((uint32_t)(it >> 1) & 1u) ^ 1u, p.err, 83)) break;
        if (!mbar_wait(&full[s], (uint32_t)(it / S) & 1u, p.err, 84)) break;
        tc_fence_after();
        const uint32_t a0 = smem_u32(ring + (size_t)s * t_bytes);
        const uint32_t b0 = smem_u32(keys);
        const uint32_t d_tmem = tmem_base + (uint32_t)buf * 2 * ELL;
        for (int kb = 0; kb < KB; ++kb) {
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const uint64_t ad = make_sdesc_k_sw128(a0 + (uint32_t)kb * PCT_TILE * 128 + k * 32);
            const uint64_t bd = make_sdesc_k_sw128(b0 + (uint32_t)kb * 2 * ELL * 128 + k * 32);
            mma_bf16_ss(d_tmem, ad, bd, idesc, (kb | k) != 0 ? 1u : 0u);
          }
        }
        mma_commit(&empty[s]);
        mma_commit(&tmem_full[buf]);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int q = warp & 3;
    const int r = q * 32 + lane;
    int it = 0;
    for (int t = t_begin; t < t_end; ++t, ++it) {
      const int buf = it & 1;
      const int64_t row = (int64_t)t * PCT_TILE + r;
      if (!mbar_wait(&tmem_full[buf], (uint32_t)(it >> 1) & 1u, p.err, 85)) break;
      tc_fence_after();
      const uint32_t ta = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * 2 * ELL);
      float sc[ELL];
#pragma unroll
      for (int c = 0; c < ELL; c += 16) {
        float hi[16], lo[16];
        tmem_ld_32x16(ta + c, hi);
        tmem_ld_32x16(ta + ELL + c, lo);
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < 16; ++j) sc[c + j] = hi[j] + lo[j];
      }
      // the accumulator is in registers: hand the TMEM buffer back before the arithmetic
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tmem_empty[buf]);
#pragma unroll
      for (int g0 = 0; g0 < ELL; g0 += GROUP) {
        float mx = sc[g0];
#pragma unroll
        for (int j = 1; j < GROUP; ++j) mx = fmaxf(mx, sc[g0 + j]);
        float s0 = 0.f, s1 = 0.f;
#pragma unroll
        for (int j = 0; j < GROUP; j += 2) {
          sc[g0 + j] = __expf(sc[g0 + j] - mx);
          sc[g0 + j + 1] = __expf(sc[g0 + j + 1] - mx);
          s0 += sc[g0 + j];
          s1 += sc[g0 + j + 1];
        }
        const float inv = 1.f / (s0 + s1);
#pragma unroll
        for (int j = 0; j < GROUP; ++j) sc[g0 + j] *= inv;
      }
      if (row < p.M) {
        uint4* dst = reinterpret_cast<uint4*>(p.out + row * ELL);
#pragma unroll
        for (int c8 = 0; c8 < ELL / 8; ++c8) {
          uint4 o;
          o.x = pct_pack(sc[c8 * 8 + 0], sc[c8 * 8 + 1]);
          o.y = pct_pack(sc[c8 * 8 + 2], sc[c8 * 8 + 3]);
          o.z = pct_pack(sc[c8 * 8 + 4], sc[c8 * 8 + 5]);
          o.w = pct_pack(sc[c8 * 8 + 6], sc[c8 * 8 + 7]);
          __stcs(dst + c8, o);
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

static int precompute_tc_stages(int ell, int d, size_t* smem_bytes) {
  const size_t stage = (size_t)(d / 64) * PCT_TILE * 128;
  const size_t keys = (size_t)(d / 64) * 2 * ell * 128;
  const size_t fixed = 1024 + keys + (2 * PCT_MAX_STAGES + 5) * 8 + 16;
  if (fixed + 2 * stage > 226 * 1024) { *smem_bytes = 0; return 0; }
  int S = (int)((226 * 1024 - fixed) / stage);
  if (S > PCT_MAX_STAGES) S = PCT_MAX_STAGES;
  *smem_bytes = (size_t)S * stage + fixed;
  return S;
}

bool precompute_tc_supported(int dtype, int d, int ell, int group) {
  if (dtype != LIME_BF16) return false;
  if (!(ell == 16 || ell == 32 || ell == 64 || ell == 128)) return false;
  if (!(group == ell || group == 16 || group == 32 || group == 64) || group > ell) return false;
  if (d % 64 != 0 || d > 512) return false;
  size_t smem;
  return precompute_tc_stages(ell, d, &smem) >= 2;
}

template <int ELL, int GROUP>
static lime_status launch_precompute_tc_t(const void* cand, int64_t M, int d, const void* keff_hl, void* out_w, int* err,
                                          cudaStream_t st) {
  size_t smem;
  const int S = precompute_tc_stages(ELL, d, &smem);
  CUtensorMap tmT, tmK;
  if (!make_tmap_bf16_sw128(&tmT, cand, (uint64_t)M, (uint64_t)d, (uint64_t)d, PCT_TILE) ||
      !make_tmap_bf16_sw128(&tmK, keff_hl, (uint64_t)2 * ELL, (uint64_t)d, (uint64_t)d, 2 * ELL < 128 ? 2 * ELL : 128))
    return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
  PrecomputeTcParams p;
  p.out = (__nv_bfloat16*)out_w; p.M = M; p.d = d;
  p.n_tiles = (int)((M + PCT_TILE - 1) / PCT_TILE);
  p.stages = S; p.err = err;
  const int grid = p.n_tiles < kSMs ? p.n_tiles : kSMs;
  LIME_CUDA(cudaFuncSetAttribute(k_precompute_tc<ELL, GROUP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  ProfScope _p("k_precompute_tc", st);
  k_precompute_tc<ELL, GROUP><<<grid, PCT_THREADS, smem, st>>>(tmT, tmK, p);
  LIME_LAUNCH_CHECK("k_precompute_tc");
  return LIME_OK;
}

template <int ELL>
static lime_status launch_precompute_tc_g(const void* cand, int64_t M, int d, int group, const void* keff_hl, void* out_w, int* err,
                                          cudaStream_t st) {
  if (group == ELL) return launch_precompute_tc_t<ELL, ELL>(cand, M, d, keff_hl, out_w, err, st);
  if constexpr (ELL > 16) if (group == 16) return launch_precompute_tc_t<ELL, 16>(cand, M, d, keff_hl, out_w, err, st);
  if constexpr (ELL > 32) if (group == 32) return launch_precompute_tc_t<ELL, 32>(cand, M, d, keff_hl, out_w, err, st);
  if constexpr (ELL > 64) if (group == 64) return launch_precompute_tc_t<ELL, 64>(cand, M, d, keff_hl, out_w, err, st);
  return LIME_UNSUPPORTED_SHAPE;
}

lime_status launch_precompute_tc(const void* cand, int64_t M, int d, int rows, int group, const void* keff_hl, void* out_w,
                                 int* err, cudaStream_t st) {
  if (M == 0) return LIME_OK;
  if (M > (int64_t)0x7fffffff * PCT_TILE / 2) return LIME_UNSUPPORTED_SHAPE;
  switch (rows) {
    case 16: return launch_precompute_tc_g<16>(cand, M, d, group, keff_hl, out_w, err, st);
    case 32: return launch_precompute_tc_g<32>(cand, M, d, group, keff_hl, out_w, err, st);
    case 64: return launch_precompute_tc_g<64>(cand, M, d, group, keff_hl, out_w, err, st);
    case 128: return launch_precompute_tc_g<128>(cand, M, d, group, keff_hl, out_w, err, st);
  }
  return LIME_UNSUPPORTED_SHAPE;
}

}  // namespace lime
