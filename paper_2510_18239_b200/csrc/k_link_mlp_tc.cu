// GatedMLP on the link rows of one XOR layer, fused with everything that consumes its result (bf16 operands, fp32
// accumulation in TMEM):
//
//   T^j = GatedMLP(O[T]) = ( SiLU(O[T] W_g) * (O[T] W_u) ) W_o                                   (Eq. 5 on link rows, Eq. 8)
//
// The attention kernel leaves Ohat [rows x H*d]: per (user, link) row the H un-projected head outputs side by side;
// W_V is folded into the gate / up weights (k_link_prep.cu), so, per block of 128 hidden columns (one pass for
// d_ff = 128, two for d_ff = 256):
//   1. [gate | up] [128 x 2*128] = Ohat_tile [128 x H*d] . [Mvg | Mvu]  streamed over K = H*d through a TMA stage ring
//   2. U = SiLU(gate) * up -> bf16 -> shared memory (A operand of the next contraction)
//   3. T^j (+)= U [128 x 128] . W_o [128 of the f rows x d]
// and the epilogue of step 3, one thread pair per row, writes what the rest of the layer stack needs:
//   - T^j as fp32 (only when the caller asks for the layer's link rows)
//   - L^P (+)= T^j, the running sum of Eq. 8
//   - LN(T^j) as bf16, the A operand of the next layer's link-side GEMM (LayerNorm before the projections, App. C)
//   - on the last layer, the link states bf16(L^P) of Eq. 4 when no candidate-side value projection follows
// One CTA per 128 rows.  Warp 0 TMA producer, warp 1 MMA issuer, warps 2-9 epilogue (two threads per row, half of the
// columns each; a warp may only touch the TMEM lane quarter warp_id % 4).
//
// Built for d = d_ff in {128, 256} (template parameter D).
#include "lime_common.cuh"
#include "tc_common.cuh"

namespace lime {

constexpr int LM_THREADS = 64 + 256;
constexpr uint32_t LM_SUB = 128 * 128;                       // [128 rows x 64 bf16]
constexpr uint32_t LM_STAGE = 3 * LM_SUB;                    // A tile + 256 rows of B

template <int D> struct LmLayout {
  static constexpr int PASSES = D / 128;                               // blocks of 128 hidden columns
  static constexpr int STAGES = D == 128 ? 3 : 2;
  static constexpr uint32_t OFF_WO = STAGES * LM_STAGE;                // W_o^T rows of one pass: D/128 x 2 sub-tiles
  static constexpr uint32_t WO_BYTES = (uint32_t)(D / 128) * 2 * LM_SUB;
  static constexpr uint32_t OFF_U = OFF_WO + WO_BYTES;                 // U [128 x 128]: 2 K-blocks
  static constexpr uint32_t OPS_END = OFF_U + 2 * LM_SUB;
  // the output tile is staged over the operand buffers once the last contraction has finished
  static constexpr int TS_LD = D + 4;                                  // floats per staged fp32 row (16-byte aligned, spread banks)
  static constexpr int TH_LD = D + 8;                                  // bf16 per staged LN row
  static constexpr uint32_t OFF_TH = 128 * TS_LD * 4;
  static constexpr uint32_t STAGE_END = OFF_TH + 128 * TH_LD * 2;
  static constexpr uint32_t OFF_EXCH = OPS_END > STAGE_END ? OPS_END : STAGE_END;   // [2 slots][2 halves][128] floats
  static constexpr uint32_t OFF_BAR = OFF_EXCH + 4 * 128 * 4;
  static constexpr uint32_t SMEM = OFF_BAR + 256;
  static_assert(SMEM <= 232448, "shared memory budget of one CTA");
};

struct LinkMlpParams {
  int64_t M;                    // rows (users x links)
  int kblocks;                  // H*d / 64
  float* T_out;                 // nullable: fp32 [M x d]
  float* LP;                    // nullable: fp32 [M x d] running sum
  int lp_accumulate;            // 0: LP = T, 1: LP += T
  __nv_bfloat16* That_next;     // nullable: bf16 [M x d] = LN(T) (or T when ln == 0)
  __nv_bfloat16* link_states;   // nullable: bf16 [M x d] = LP after this layer
  int ln;
  float ln_eps;
  int* err;
};

__device__ __forceinline__ uint32_t lm_pack(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float lm_tanh(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t lm_chunk(uint32_t r, uint32_t c) { return r * 128u + ((c ^ (r & 7u)) << 4); }

template <int D>
__global__ void __launch_bounds__(LM_THREADS, 1)
k_link_mlp_tc(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
              const __grid_constant__ CUtensorMap tmWo, const LinkMlpParams p) {
  using namespace tc;
  using Lay = LmLayout<D>;
  constexpr int PASSES = Lay::PASSES, STAGES = Lay::STAGES, F = D;
  extern __shared__ __align__(1024) uint8_t smem[];
  if ((smem_u32(smem) & 1023u) != 0) {
    if (threadIdx.x == 0) atomicCAS(p.err, 0, 93);
    return;
  }
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Lay::OFF_BAR);
  uint64_t* full = bars;                 // [STAGES]
  uint64_t* empty = bars + 3;            // [STAGES]
  uint64_t* wo_full = bars + 6;          // per pass: this pass's rows of W_o^T landed
  uint64_t* gu_full = bars + 7;          // per pass: [gate | up] complete
  uint64_t* u_ready = bars + 8;          // per pass: U in shared memory, [gate | up] read (8 warps)
  uint64_t* out_full = bars + 9;         // per pass: the pass's part of step 3 done (W_o^T buffer and U free again)
  uint64_t* pair_bar = bars + 10;        // [4], 2 warps each
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 14);
  uint64_t* all_bar = bars + 15;         // rendezvous of the 8 epilogue warps (tiles staged in shared memory)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.x * 128;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(wo_full, 1); mbar_init(gu_full, 1); mbar_init(u_ready, 8); mbar_init(out_full, 1);
    for (int i = 0; i < 4; ++i) mbar_init(&pair_bar[i], 2);
    mbar_init(all_bar, 8);
    fence_barrier_init();
    prefetch_tmap(&tmA); prefetch_tmap(&tmB); prefetch_tmap(&tmWo);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  constexpr uint32_t COL_GU = 0, COL_OUT = 256;
  // set-up done: the next kernel's CTAs may become resident; nothing an earlier kernel wrote is read before this wait
  pdl_launch_dependents();
  pdl_wait();

  if (warp == 0) {
    if (lane == 0) {
      const uint64_t pol = policy_evict_last();
      auto load_wo = [&](int pass) {
        // rows = output columns of W_o (D of them, 128 per sub-tile pair), contraction index = this pass's 128 hidden columns
        mbar_arrive_expect_tx(wo_full, Lay::WO_BYTES);
        for (int nh = 0; nh < D / 128; ++nh)
          for (int kb = 0; kb < 2; ++kb)
            tma_load_2d_hint(smem + Lay::OFF_WO + (uint32_t)(nh * 2 + kb) * LM_SUB, &tmWo, pass * 128 + kb * 64, nh * 128, wo_full, pol);
      };
      load_wo(0);
      bool ok = true;
      int it = 0;                                          // ring use counter over all passes
      for (int pass = 0; pass < PASSES && ok; ++pass) {
        for (int kb = 0; kb < p.kblocks; ++kb, ++it) {
          const int s = it % STAGES;
          if (!mbar_wait(&empty[s], ((uint32_t)(it / STAGES) & 1u) ^ 1u, p.err, 71)) { ok = false; break; }
          uint8_t* st = smem + (size_t)s * LM_STAGE;
          mbar_arrive_expect_tx(&full[s], LM_STAGE);
          tma_load_2d_hint(st, &tmA, kb * 64, m0, &full[s], pol);
          tma_load_2d_hint(st + LM_SUB, &tmB, kb * 64, pass * 128, &full[s], pol);           // gate rows of this pass
          tma_load_2d_hint(st + 2 * LM_SUB, &tmB, kb * 64, F + pass * 128, &full[s], pol);   // up rows
        }
        // the next pass's rows of W_o^T replace this pass's once its part of step 3 has run
        if (ok && pass + 1 < PASSES) {
          if (!mbar_wait(out_full, (uint32_t)pass & 1u, p.err, 81)) { ok = false; break; }
          load_wo(pass + 1);
        }
      }
      if (!ok || *(volatile int*)p.err != 0) {
        for (int j = 0; j < it && j < STAGES; ++j)
          mbar_wait_quiet(&full[(it - 1 - j) % STAGES], (uint32_t)((it - 1 - j) / STAGES) & 1u);
        mbar_wait_quiet(wo_full, 0);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc_256 = make_idesc_bf16(128, 256);
      constexpr uint32_t idesc_128 = make_idesc_bf16(128, 128);
      const uint32_t sbase = smem_u32(smem);
      bool ok = true;
      int it = 0;
      for (int pass = 0; pass < PASSES && ok; ++pass) {
        // 1. [gate | up] of this pass; its columns were last read by the previous pass's step 2 (u_ready, waited below)
        for (int kb = 0; kb < p.kblocks && ok; ++kb, ++it) {
          const int s = it % STAGES;
          if (!mbar_wait(&full[s], (uint32_t)(it / STAGES) & 1u, p.err, 72)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int k = 0; k < 4; ++k)
            mma_bf16_ss(tmem_base + COL_GU, make_sdesc_k_sw128(sbase + s * LM_STAGE + k * 32),
                        make_sdesc_k_sw128(sbase + s * LM_STAGE + LM_SUB + k * 32), idesc_256, (kb | k) != 0);
          mma_commit(&empty[s]);
        }
        if (!ok) break;
        mma_commit(gu_full);
        ok = mbar_wait(wo_full, (uint32_t)pass & 1u, p.err, 74) && mbar_wait(u_ready, (uint32_t)pass & 1u, p.err, 75);
        if (!ok) break;
        // 3. T (+)= U . W_o (this pass's hidden columns)
        tc_fence_after();
        for (int nh = 0; nh < D / 128; ++nh)
          for (int kk = 0; kk < 8; ++kk) {
            const uint32_t o = (uint32_t)(kk >> 2) * LM_SUB + (uint32_t)(kk & 3) * 32;
            mma_bf16_ss(tmem_base + COL_OUT + (uint32_t)nh * 128, make_sdesc_k_sw128(sbase + Lay::OFF_U + o),
                        make_sdesc_k_sw128(sbase + Lay::OFF_WO + (uint32_t)nh * 2 * LM_SUB + o), idesc_128, (pass | kk) != 0);
          }
        mma_commit(out_full);
      }
    }
  } else {
    const int ew = warp - 2;                                   // 0..7
    const int q = warp & 3;
    const int half = ew >> 2;
    const uint32_t r = (uint32_t)(q * 32 + lane);
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
    float* exch = reinterpret_cast<float*>(smem + Lay::OFF_EXCH);
    bool ok = true;
    for (int pass = 0; pass < PASSES && ok; ++pass) {
      if (!mbar_wait(gu_full, (uint32_t)pass & 1u, p.err, 73)) { ok = false; break; }
      tc_fence_after();
      // 2. U = SiLU(gate) * up for this thread's 64 hidden columns of the pass (K-block `half` of the A operand); the
      //    previous pass's step 3 has read U (gu_full is committed after it)
      uint8_t* ub = smem + Lay::OFF_U + half * LM_SUB;
#pragma unroll
      for (int c = 0; c < 64; c += 32) {
        float gt[32], up[32];
        tmem_ld_32x32(lane_addr + COL_GU + half * 64 + c, gt);
        tmem_ld_32x32(lane_addr + COL_GU + 128 + half * 64 + c, up);
        tmem_wait_ld();
#pragma unroll
        for (int c8 = 0; c8 < 4; ++c8) {
          float y[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float hx = 0.5f * gt[c8 * 8 + j];
            y[j] = fmaf(hx, lm_tanh(hx), hx) * up[c8 * 8 + j];
          }
          uint4 o;
          o.x = lm_pack(y[0], y[1]); o.y = lm_pack(y[2], y[3]); o.z = lm_pack(y[4], y[5]); o.w = lm_pack(y[6], y[7]);
          *reinterpret_cast<uint4*>(ub + lm_chunk(r, (uint32_t)(c >> 3) + c8)) = o;
        }
      }
      tc_fence_before();
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(u_ready);
    }

    // 3'. epilogue of T = U . W_o: this thread's D/2 columns of its row, 64 at a time
    constexpr int CH = D / 128;                                  // 64-column pieces per thread
    if (ok && mbar_wait(out_full, (uint32_t)(PASSES - 1) & 1u, p.err, 76)) {
      tc_fence_after();
      auto load64 = [&](int ch, float (&v)[64]) {
        float v0[32], v1[32];
        tmem_ld_32x32(lane_addr + COL_OUT + half * (D / 2) + ch * 64, v0);
        tmem_ld_32x32(lane_addr + COL_OUT + half * (D / 2) + ch * 64 + 32, v1);
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < 32; ++j) { v[j] = v0[j]; v[32 + j] = v1[j]; }
      };
      // T, the running sum of Eq. 8 and (last layer) the link states leave row by row: a thread owns half a row, so
      // direct accesses would touch 32 lines per instruction.  The tile is staged as fp32 over the operand buffers
      // (free since the last contraction finished) and each warp then moves whole rows.
      constexpr int TS_LD = Lay::TS_LD;
      float* Ts = reinterpret_cast<float*>(smem);
      float s = 0.f;
#pragma unroll
      for (int ch = 0; ch < CH; ++ch) {
        float v[64];
        load64(ch, v);
#pragma unroll
        for (int j = 0; j < 64; j += 4)
          *reinterpret_cast<float4*>(Ts + r * TS_LD + half * (D / 2) + ch * 64 + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
#pragma unroll
        for (int j = 0; j < 64; ++j) s += v[j];
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(all_bar);
      if (mbar_wait(all_bar, 0, p.err, 79)) {
        // a warp takes rows ew, ew + 8, ...; the reads of the running sum for a batch of rows are issued together
        constexpr int BATCH = 8;
        const int n_valid = (int)(p.M - m0 < 128 ? p.M - m0 : 128);
        const bool acc = p.LP != nullptr && p.lp_accumulate != 0;
#pragma unroll 1
        for (int cb = 0; cb < D; cb += 128) {                    // 128 columns (one float4 per lane) at a time
          for (int i0 = ew; i0 < 128; i0 += 8 * BATCH) {
            float4 prev[BATCH];
#pragma unroll
            for (int k = 0; k < BATCH; ++k) {
              const int i = i0 + 8 * k;
              prev[k] = (acc && i < n_valid) ? *reinterpret_cast<const float4*>(p.LP + ((int64_t)m0 + i) * D + cb + lane * 4)
                                             : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int k = 0; k < BATCH; ++k) {
              const int i = i0 + 8 * k;
              if (i >= n_valid) continue;
              float4 t = *reinterpret_cast<const float4*>(Ts + i * TS_LD + cb + lane * 4);
              const int64_t o = ((int64_t)m0 + i) * D + cb + lane * 4;
              if (p.T_out) *reinterpret_cast<float4*>(p.T_out + o) = t;
              if (p.LP) {
                t.x += prev[k].x; t.y += prev[k].y; t.z += prev[k].z; t.w += prev[k].w;
                *reinterpret_cast<float4*>(p.LP + o) = t;
                if (p.link_states) *reinterpret_cast<uint2*>(p.link_states + o) = make_uint2(lm_pack(t.x, t.y), lm_pack(t.z, t.w));
              }
            }
          }
        }
      }
      if (p.That_next) {
        // LN(T) for the next layer's link-side GEMM: the two halves of a row exchange their partial sums
        float mu = 0.f, rstd = 1.f;
        if (p.ln) {
          uint32_t uses = 0;
          auto pair_sync = [&](int where) {
            __syncwarp();
            if (lane == 0) mbar_arrive(&pair_bar[q]);
            const bool w = mbar_wait(&pair_bar[q], uses & 1u, p.err, where);
            ++uses;
            return w;
          };
          exch[half * 128 + r] = s;
          ok = pair_sync(77);
          mu = (s + exch[(half ^ 1) * 128 + r]) * (1.0f / D);
          float var = 0.f;
#pragma unroll
          for (int ch = 0; ch < CH; ++ch) {
            float v[64];
            load64(ch, v);
#pragma unroll
            for (int j = 0; j < 64; ++j) { const float c = v[j] - mu; var = fmaf(c, c, var); }
          }
          exch[256 + half * 128 + r] = var;
          ok = ok && pair_sync(78);
          rstd = rsqrtf((var + exch[256 + (half ^ 1) * 128 + r]) * (1.0f / D) + p.ln_eps);
        }
        // the same way out for the bf16 rows: staged behind the fp32 tile, then whole rows per warp
        constexpr int TH_LD = Lay::TH_LD;
        __nv_bfloat16* Th = reinterpret_cast<__nv_bfloat16*>(smem + Lay::OFF_TH);
#pragma unroll
        for (int ch = 0; ch < CH; ++ch) {
          float v[64];
          load64(ch, v);
#pragma unroll
          for (int j = 0; j < 64; j += 8) {
            uint4 o;
            o.x = lm_pack((v[j] - mu) * rstd, (v[j + 1] - mu) * rstd); o.y = lm_pack((v[j + 2] - mu) * rstd, (v[j + 3] - mu) * rstd);
            o.z = lm_pack((v[j + 4] - mu) * rstd, (v[j + 5] - mu) * rstd); o.w = lm_pack((v[j + 6] - mu) * rstd, (v[j + 7] - mu) * rstd);
            *reinterpret_cast<uint4*>(Th + r * TH_LD + half * (D / 2) + ch * 64 + j) = o;
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(all_bar);
        if (ok && mbar_wait(all_bar, 1, p.err, 80)) {
#pragma unroll 4
          for (int i = ew; i < 128; i += 8) {
            const int64_t grow = (int64_t)m0 + i;
            if (grow >= p.M) break;
#pragma unroll
            for (int cb = 0; cb < D; cb += 128)
              *reinterpret_cast<uint2*>(p.That_next + grow * D + cb + lane * 4) = *reinterpret_cast<const uint2*>(Th + i * TH_LD + cb + lane * 4);
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

template <int D>
static lime_status launch_lm(const LinkMlpArgs& a, cudaStream_t st) {
  using Lay = LmLayout<D>;
  CUtensorMap tmA, tmB, tmWo;
  if (!make_tmap_bf16_sw128(&tmA, a.Ohat, (uint64_t)a.M, (uint64_t)a.K, (uint64_t)a.K, 128) ||
      !make_tmap_bf16_sw128(&tmB, a.WpostT, 2 * D, (uint64_t)a.K, (uint64_t)a.K, 128) ||
      !make_tmap_bf16_sw128(&tmWo, a.WoT, D, D, D, 128))
    return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
  LinkMlpParams p;
  p.M = a.M; p.kblocks = a.K / 64; p.T_out = a.T_out; p.LP = a.LP; p.lp_accumulate = a.lp_accumulate;
  p.That_next = (__nv_bfloat16*)a.That_next; p.link_states = (__nv_bfloat16*)a.link_states; p.ln = a.ln; p.ln_eps = a.ln_eps;
  p.err = a.err;
  static bool smem_set[kMaxDeviceOrdinals] = {};
  lime_status es = ensure_dynamic_smem((const void*)k_link_mlp_tc<D>, (int)Lay::SMEM, smem_set);
  if (es != LIME_OK) return es;
  ProfScope _p("k_link_mlp_tc", st);
  launch_pdl(k_link_mlp_tc<D>, dim3((unsigned)((a.M + 127) / 128)), dim3(LM_THREADS), Lay::SMEM, st, tmA, tmB, tmWo, p);
  LIME_LAUNCH_CHECK("k_link_mlp_tc");
  return LIME_OK;
}

// a.K = H * d; d = d_ff = a.d
lime_status launch_link_mlp_tc(const LinkMlpArgs& a, cudaStream_t st) {
  if (a.M == 0) return LIME_OK;
  if (a.d == 128) return launch_lm<128>(a, st);
  if (a.d == 256) return launch_lm<256>(a, st);
  return LIME_UNSUPPORTED_SHAPE;
}

}  // namespace lime
