// CUDA-core XOR attention (both directions of Eq. 7), any d_h <= 128, fp32 arithmetic.
// These kernels define the reference behaviour of the CUDA path for every shape and storage type; the bf16
// tensor-core kernels replace them where the tiles are dense contractions of supported size.
#include "lime_common.cuh"

namespace lime {

constexpr int ATT_TN = 32;       // history tokens per tile (one per lane)
constexpr int ATT_WARPS = 4;

// ----------------------------------------------------------------------------- links attend over history
// O[T] = phi(Q[T] K[S]^T) V[S]  (App. H.1), one block per (chunk of a user's history, head).
// Online softmax: every link row keeps a running max m, running sum s and un-normalised accumulator; the
// chunk's (m, s, acc) go to scratch and k_attn_link_merge combines a user's chunks in a fixed order.
template <typename TS>
__global__ void __launch_bounds__(ATT_WARPS * 32)
k_attn_link_simt(const float* __restrict__ QT, int64_t qt_user_stride, const TS* __restrict__ KS,
                 const TS* __restrict__ VS, const int32_t* __restrict__ off, int B, int ell, int d, int H, int phi,
                 float scale, int chunk, const int32_t* __restrict__ chunk_start, float* __restrict__ part_m,
                 float* __restrict__ part_s, float* __restrict__ part_acc) {
  const int ci = blockIdx.x;
  if (ci >= chunk_start[B]) return;
  const int b = upper_user(chunk_start, B, ci);
  const int h = blockIdx.y;
  const int d_h = d / H;
  const int64_t t0 = (int64_t)off[b] + (int64_t)(ci - chunk_start[b]) * chunk;
  const int64_t t1 = min((int64_t)off[b + 1], t0 + chunk);

  extern __shared__ float smem[];
  float* Qs = smem;                          // [ell][d_h]
  float* Kt = Qs + ell * d_h;                // [d_h][33]  (transposed tile)
  float* Vs = Kt + d_h * (ATT_TN + 1);       // [32][d_h]
  float* acc_s = Vs + ATT_TN * d_h;          // [ell][d_h]
  float* m_s = acc_s + ell * d_h;            // [ell]
  float* s_s = m_s + ell;                    // [ell]

  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const float* q = QT + (int64_t)b * qt_user_stride + h * d_h;
  for (int i = tid; i < ell * d_h; i += blockDim.x) {
    Qs[i] = q[(i / d_h) * d + (i % d_h)];
    acc_s[i] = 0.f;
  }
  for (int i = tid; i < ell; i += blockDim.x) { m_s[i] = -INFINITY; s_s[i] = 0.f; }

  for (int64_t tt = t0; tt < t1; tt += ATT_TN) {
    __syncthreads();
    for (int i = tid; i < ATT_TN * d_h; i += blockDim.x) {
      const int t = i / d_h, k = i % d_h;
      float kv = 0.f, vv = 0.f;
      if (tt + t < t1) {
        const int64_t g = (tt + t) * d + h * d_h + k;
        kv = Store<TS>::ld(KS + g);
        vv = Store<TS>::ld(VS + g);
      }
      Kt[k * (ATT_TN + 1) + t] = kv;
      Vs[t * d_h + k] = vv;
    }
    __syncthreads();
    const bool valid = tt + lane < t1;
    for (int l = wid; l < ell; l += ATT_WARPS) {
      float sc = 0.f;
      const float* ql = Qs + l * d_h;
      for (int k = 0; k < d_h; ++k) sc = fmaf(ql[k], Kt[k * (ATT_TN + 1) + lane], sc);
      float p, corr;
      if (phi == LIME_PHI_SOFTMAX) {
        sc = valid ? sc * scale : -INFINITY;
        const float m_old = m_s[l];
        const float m_new = fmaxf(m_old, warp_max(sc));
        p = valid ? __expf(sc - m_new) : 0.f;
        corr = (m_old == -INFINITY) ? 0.f : __expf(m_old - m_new);
        const float ps = warp_sum(p);
        __syncwarp();
        if (lane == 0) { m_s[l] = m_new; s_s[l] = s_s[l] * corr + ps; }
      } else {
        p = valid ? silu_f(sc) : 0.f;
        corr = 1.f;
      }
      for (int k0 = 0; k0 < d_h; k0 += 32) {
        const int k = k0 + lane;
        float a = 0.f;
#pragma unroll 8
        for (int t = 0; t < ATT_TN; ++t) {
          const float pt = __shfl_sync(0xffffffffu, p, t);
          if (k < d_h) a = fmaf(pt, Vs[t * d_h + k], a);
        }
        if (k < d_h) acc_s[l * d_h + k] = acc_s[l * d_h + k] * corr + a;
      }
      __syncwarp();
    }
  }
  __syncthreads();
  const int64_t pbase = ((int64_t)ci * H + h) * ell;
  for (int i = tid; i < ell; i += blockDim.x) { part_m[pbase + i] = m_s[i]; part_s[pbase + i] = s_s[i]; }
  for (int i = tid; i < ell * d_h; i += blockDim.x) part_acc[pbase * d_h + i] = acc_s[i];
}

__global__ void __launch_bounds__(128)
k_attn_link_merge(const int32_t* __restrict__ off, int ell, int d, int H, int phi,
                  const int32_t* __restrict__ chunk_start, const float* __restrict__ part_m,
                  const float* __restrict__ part_s, const float* __restrict__ part_acc, float* __restrict__ AT) {
  const int b = blockIdx.x, h = blockIdx.y;
  const int d_h = d / H;
  const int c0 = chunk_start[b], c1 = chunk_start[b + 1];
  const float n_hist = (float)(off[b + 1] - off[b]);
  for (int i = threadIdx.x; i < ell * d_h; i += blockDim.x) {
    const int l = i / d_h, k = i % d_h;
    float out = 0.f;
    if (c1 > c0) {
      if (phi == LIME_PHI_SOFTMAX) {
        float M = -INFINITY;
        for (int c = c0; c < c1; ++c) M = fmaxf(M, part_m[((int64_t)c * H + h) * ell + l]);
        float S = 0.f, O = 0.f;
        for (int c = c0; c < c1; ++c) {
          const int64_t r = ((int64_t)c * H + h) * ell + l;
          const float w = __expf(part_m[r] - M);
          S = fmaf(part_s[r], w, S);
          O = fmaf(part_acc[r * d_h + k], w, O);
        }
        out = O / S;
      } else {
        float O = 0.f;
        for (int c = c0; c < c1; ++c) O += part_acc[(((int64_t)c * H + h) * ell + l) * d_h + k];
        out = O / n_hist;
      }
    }
    AT[((int64_t)b * ell + l) * d + h * d_h + k] = out;
  }
}

static size_t attn_link_smem(int ell, int d_h) {
  return sizeof(float) * ((size_t)2 * ell * d_h + (size_t)d_h * (ATT_TN + 1) + (size_t)ATT_TN * d_h + 2 * (size_t)ell);
}

lime_status launch_attn_link_simt(const AttnLinkArgs& a, cudaStream_t st) {
  if (a.n_chunk_upper <= 0) return LIME_OK;
  const int d_h = a.d / a.H;
  const size_t smem = attn_link_smem(a.ell, d_h);
  if (smem > 200 * 1024) return LIME_UNSUPPORTED_SHAPE;
  ProfScope _p("k_attn_link_simt", st);
  dim3 grid(a.n_chunk_upper, a.H);
  if (a.s_dtype == LIME_F32) {
    LIME_CUDA(cudaFuncSetAttribute(k_attn_link_simt<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k_attn_link_simt<float><<<grid, ATT_WARPS * 32, smem, st>>>(
        a.QT, a.qt_user_stride, (const float*)a.KS, (const float*)a.VS, a.off, a.B, a.ell, a.d, a.H, a.phi, a.scale,
        a.chunk, a.chunk_start, a.part_m, a.part_s, a.part_acc);
  } else {
    LIME_CUDA(cudaFuncSetAttribute(k_attn_link_simt<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)smem));
    k_attn_link_simt<__nv_bfloat16><<<grid, ATT_WARPS * 32, smem, st>>>(
        a.QT, a.qt_user_stride, (const __nv_bfloat16*)a.KS, (const __nv_bfloat16*)a.VS, a.off, a.B, a.ell, a.d, a.H,
        a.phi, a.scale, a.chunk, a.chunk_start, a.part_m, a.part_s, a.part_acc);
  }
  LIME_LAUNCH_CHECK("k_attn_link_simt");
  return LIME_OK;
}

lime_status launch_attn_link_merge(const AttnLinkArgs& a, cudaStream_t st) {
  if (a.B == 0) return LIME_OK;
  ProfScope _p("k_attn_link_merge", st);
  dim3 grid(a.B, a.H);
  k_attn_link_merge<<<grid, 128, 0, st>>>(a.off, a.ell, a.d, a.H, a.phi, a.chunk_start, a.part_m, a.part_s,
                                          a.part_acc, a.AT);
  LIME_LAUNCH_CHECK("k_attn_link_merge");
  return LIME_OK;
}

// ----------------------------------------------------------------------------- history attends over links
// O[S] = phi(Q[S] K[T]^T) V[T]: per history token, a softmax over the user's ell link rows per head.
// One block per tile of tokens of one user; the user's K[T], V[T] (fp32 [ell x d]) sit in shared memory.
template <typename TS>
__global__ void __launch_bounds__(ATT_WARPS * 32)
k_attn_hist_simt(const TS* QS, TS* AS, const float* __restrict__ KT, const float* __restrict__ VT,
                 int64_t t_user_stride, const int32_t* __restrict__ off, int B, int ell, int d, int H, int phi,
                 float scale, int tile, const int32_t* __restrict__ tile_start) {
  const int ti = blockIdx.x;
  if (ti >= tile_start[B]) return;
  const int b = upper_user(tile_start, B, ti);
  const int d_h = d / H;
  const int64_t t0 = (int64_t)off[b] + (int64_t)(ti - tile_start[b]) * tile;
  const int64_t t1 = min((int64_t)off[b + 1], t0 + tile);

  extern __shared__ float smem[];
  const int ldk = d + 1;
  float* Ks = smem;                   // [ell][d+1]
  float* Vs = Ks + ell * ldk;         // [ell][d+1]
  float* qs = Vs + ell * ldk;         // [warps][d]
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const float* kt = KT + (int64_t)b * t_user_stride;
  const float* vt = VT + (int64_t)b * t_user_stride;
  for (int i = tid; i < ell * d; i += blockDim.x) {
    const int l = i / d, k = i % d;
    Ks[l * ldk + k] = kt[i];
    Vs[l * ldk + k] = vt[i];
  }
  __syncthreads();
  float* qw = qs + wid * d;
  constexpr int MAXL = 8;             // ell <= 256 -> at most 8 links per lane
  for (int64_t t = t0 + wid; t < t1; t += ATT_WARPS) {
    for (int k = lane; k < d; k += 32) qw[k] = Store<TS>::ld(QS + t * d + k);
    __syncwarp();
    for (int h = 0; h < H; ++h) {
      float p[MAXL];
      float mx = -INFINITY;
#pragma unroll
      for (int j = 0; j < MAXL; ++j) {
        const int l = lane + 32 * j;
        float sc = -INFINITY;
        if (l < ell) {
          sc = 0.f;
          const float* kr = Ks + l * ldk + h * d_h;
          const float* qh = qw + h * d_h;
          for (int k = 0; k < d_h; ++k) sc = fmaf(qh[k], kr[k], sc);
          if (phi == LIME_PHI_SOFTMAX) sc *= scale;
        }
        p[j] = sc;
        mx = fmaxf(mx, sc);
      }
      if (phi == LIME_PHI_SOFTMAX) {
        mx = warp_max(mx);
        float sum = 0.f;
#pragma unroll
        for (int j = 0; j < MAXL; ++j) {
          p[j] = (lane + 32 * j < ell) ? __expf(p[j] - mx) : 0.f;
          sum += p[j];
        }
        const float inv = 1.f / warp_sum(sum);
#pragma unroll
        for (int j = 0; j < MAXL; ++j) p[j] *= inv;
      } else {
        const float inv = 1.f / (float)ell;
#pragma unroll
        for (int j = 0; j < MAXL; ++j) p[j] = (lane + 32 * j < ell) ? silu_f(p[j]) * inv : 0.f;
      }
      for (int k0 = 0; k0 < d_h; k0 += 32) {
        const int k = k0 + lane;
        float a = 0.f;
#pragma unroll
        for (int j = 0; j < MAXL; ++j) {
          if (32 * j < ell) {
            for (int ll = 0; ll < 32; ++ll) {
              const float pl = __shfl_sync(0xffffffffu, p[j], ll);
              const int l = 32 * j + ll;
              if (l < ell && k < d_h) a = fmaf(pl, Vs[l * ldk + h * d_h + k], a);
            }
          }
        }
        if (k < d_h) Store<TS>::st(AS + t * d + h * d_h + k, a);
      }
    }
    __syncwarp();
  }
}

lime_status launch_attn_hist_simt(const AttnHistArgs& a, cudaStream_t st) {
  if (a.n_tile_upper <= 0) return LIME_OK;
  const size_t smem = sizeof(float) * ((size_t)2 * a.ell * (a.d + 1) + (size_t)ATT_WARPS * a.d);
  if (smem > 200 * 1024) return LIME_UNSUPPORTED_SHAPE;
  ProfScope _p("k_attn_hist_simt", st);
  if (a.s_dtype == LIME_F32) {
    LIME_CUDA(cudaFuncSetAttribute(k_attn_hist_simt<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k_attn_hist_simt<float><<<a.n_tile_upper, ATT_WARPS * 32, smem, st>>>(
        (const float*)a.QS, (float*)a.AS, a.KT, a.VT, a.t_user_stride, a.off, a.B, a.ell, a.d, a.H, a.phi, a.scale,
        a.tile, a.tile_start);
  } else {
    LIME_CUDA(cudaFuncSetAttribute(k_attn_hist_simt<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)smem));
    k_attn_hist_simt<__nv_bfloat16><<<a.n_tile_upper, ATT_WARPS * 32, smem, st>>>(
        (const __nv_bfloat16*)a.QS, (__nv_bfloat16*)a.AS, a.KT, a.VT, a.t_user_stride, a.off, a.B, a.ell, a.d, a.H,
        a.phi, a.scale, a.tile, a.tile_start);
  }
  LIME_LAUNCH_CHECK("k_attn_hist_simt");
  return LIME_OK;
}

}  // namespace lime
