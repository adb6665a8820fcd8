// The two small feed-forward networks around the XOR layers, on CUDA cores (any storage type, any widths):
//   - link contextualisation  L^C_b = MLP(L (+) E^C_b)                         (Eq. 2)
//   - the interaction network that scores the LIME embedding, logit_c = FFN([O_c | T_c])     (Sec. 3.3, widths of App. C)
// Both are x <- ReLU(x W_i + b_i) for every hidden layer and a linear last layer.  Both first layers see a
// concatenation and are split over it, so neither input row is ever formed:
//   (L_l (+) E^C_b) W_0 = (L W_0[:d])_l + E^C_b W_0[d:]          the first term is weights only (formed at set-up)
//   [O_c | T_c] W_0     = sum_l W[c,l] (LS_b W_0[:d])_l + T_c W_0[d:]          LSW_b = LS_b W_0[:d] once per user
// The bf16 one-hidden-layer interaction network on dense candidate streams runs on tensor cores (k_score_head_tc.cu);
// everything else (fp32 storage, deeper networks, ragged candidate lists, candidates taken by id) runs here.
#include "lime_common.cuh"

namespace lime {

// ----------------------------------------------------------------------------- Y[r, :] = X[r, :] . W (+ b)
// Small dense product with fp32 accumulation.  A block takes FR_ROWS rows of X and FR_COLS output columns; the rows sit in
// shared memory, the block's slice of W is staged there too in pieces of FR_KC contraction indices (read once, coalesced
// over the columns), and a thread forms FR_ROWS / 4 x 1 outputs per piece from shared memory only.  Outputs: fp32 [M x N]
// and / or bf16 transposed per group of `group` rows ([M/group][N][group], the K-major operand layout of
// k_score_head_tc.cu).
constexpr int FR_ROWS = 32, FR_COLS = 32, FR_KC = 64, FR_THREADS = 128;      // thread (ty, tx): rows ty*8..ty*8+7, column tx
template <typename TX, typename TW>
__global__ void __launch_bounds__(FR_THREADS)
k_rows_times_w(const TX* __restrict__ X, int64_t M, int K, const TW* __restrict__ W, int ldw, int N, const float* __restrict__ bias,
               float* __restrict__ Y, __nv_bfloat16* __restrict__ Yt, int group) {
  extern __shared__ float fr_sm[];
  float* xs = fr_sm;                                 // [FR_ROWS][K + 1]
  float* wsm = xs + FR_ROWS * (K + 1);               // [FR_KC][FR_COLS]
  const int64_t r0 = (int64_t)blockIdx.x * FR_ROWS;
  const int c0 = blockIdx.y * FR_COLS;
  const int nr = (int)min((int64_t)FR_ROWS, M - r0);
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  for (int i = threadIdx.x; i < FR_ROWS * K; i += FR_THREADS) {
    const int r = i / K, k = i % K;
    xs[r * (K + 1) + k] = r < nr ? Store<TX>::ld(X + (r0 + r) * K + k) : 0.f;
  }
  constexpr int RPT = FR_ROWS / 4;                   // rows per thread
  float acc[RPT];
  const int col = c0 + tx;
  const float b = (bias && col < N) ? bias[col] : 0.f;
#pragma unroll
  for (int r = 0; r < RPT; ++r) acc[r] = b;
  for (int k0 = 0; k0 < K; k0 += FR_KC) {
    __syncthreads();
    for (int i = threadIdx.x; i < FR_KC * FR_COLS; i += FR_THREADS) {
      const int kk = i / FR_COLS, c = i % FR_COLS;
      wsm[i] = (k0 + kk < K && c0 + c < N) ? Store<TW>::ld(W + (int64_t)(k0 + kk) * ldw + c0 + c) : 0.f;
    }
    __syncthreads();
    const int kn = min(FR_KC, K - k0);
    for (int kk = 0; kk < kn; ++kk) {
      const float w = wsm[kk * FR_COLS + tx];
#pragma unroll
      for (int r = 0; r < RPT; ++r) acc[r] = fmaf(xs[(ty * RPT + r) * (K + 1) + k0 + kk], w, acc[r]);
    }
  }
  if (col < N) {
    for (int r = 0; r < RPT; ++r) {
      const int rr = ty * RPT + r;
      if (rr >= nr) break;
      const int64_t row = r0 + rr;
      if (Y) Y[row * N + col] = acc[r];
      if (Yt) Yt[((row / group) * N + col) * group + (row % group)] = __float2bfloat16_rn(acc[r]);
    }
  }
}

lime_status launch_rows_times_w(const void* X, int x_dtype, int64_t M, int K, const void* W, int w_dtype, int ldw, int N,
                                const float* bias, float* Y, void* Yt, int group, const char* name, cudaStream_t st) {
  if (M == 0 || N == 0) return LIME_OK;
  const size_t smem = sizeof(float) * (FR_ROWS * ((size_t)K + 1) + FR_KC * FR_COLS);
  if (smem > 200 * 1024) return LIME_UNSUPPORTED_SHAPE;
  const dim3 grid((unsigned)((M + FR_ROWS - 1) / FR_ROWS), (unsigned)((N + FR_COLS - 1) / FR_COLS));
  ProfScope _p(name, st);
#define LIME_RTW(TX, TW)                                                                                                  \
  do {                                                                                                                    \
    LIME_CUDA(cudaFuncSetAttribute(k_rows_times_w<TX, TW>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));       \
    k_rows_times_w<TX, TW><<<grid, FR_THREADS, smem, st>>>((const TX*)X, M, K, (const TW*)W, ldw, N, bias, Y,              \
                                                          (__nv_bfloat16*)Yt, group);                                      \
  } while (0)
  if (x_dtype == LIME_F32 && w_dtype == LIME_F32) LIME_RTW(float, float);
  else if (x_dtype == LIME_F32) LIME_RTW(float, __nv_bfloat16);
  else if (w_dtype == LIME_F32) LIME_RTW(__nv_bfloat16, float);
  else LIME_RTW(__nv_bfloat16, __nv_bfloat16);
#undef LIME_RTW
  LIME_LAUNCH_CHECK(name);
  return LIME_OK;
}

// ----------------------------------------------------------------------------- Eq. 2: L^C = MLP(L (+) E^C)
// A block takes CM_LINKS links of one user.  first[l, :] = (L W_0[:d])_l + b_0 comes from set-up; the block adds the
// user's E^C_b W_0[d:], applies ReLU and walks the remaining layers with the activations in shared memory.
constexpr int CM_LINKS = 8, CM_THREADS = 128;
struct FfnLayers {
  int n_layers;                      // layers after the first one's split (>= 1): weights W[i] [in_i x out_i], bias b[i]
  int in_w[LIME_FFN_MAX_HIDDEN + 1], out_w[LIME_FFN_MAX_HIDDEN + 1];
  const void* W[LIME_FFN_MAX_HIDDEN + 1];
  const float* b[LIME_FFN_MAX_HIDDEN + 1];
};

template <typename T>
__global__ void __launch_bounds__(CM_THREADS)
k_link_ctx_mlp(const float* __restrict__ first, const T* __restrict__ user_ctx, int d_c, const T* __restrict__ W0c, int w0,
               int ell, int max_w, FfnLayers L, float* __restrict__ out) {
  extern __shared__ float sm[];
  float* ec = sm;                          // [d_c]
  float* ha = ec + d_c;                    // [CM_LINKS][max_w]
  float* hb = ha + CM_LINKS * max_w;       // [CM_LINKS][max_w]
  const int b = blockIdx.y, l0 = blockIdx.x * CM_LINKS;
  const int nl = min(CM_LINKS, ell - l0);
  for (int c = threadIdx.x; c < d_c; c += CM_THREADS) ec[c] = Store<T>::ld(user_ctx + (int64_t)b * d_c + c);
  __syncthreads();
  for (int j = threadIdx.x; j < w0; j += CM_THREADS) {
    float u = 0.f;
    for (int c = 0; c < d_c; ++c) u = fmaf(ec[c], Store<T>::ld(W0c + (int64_t)c * w0 + j), u);
    for (int r = 0; r < nl; ++r) {
      const float v = first[(int64_t)(l0 + r) * w0 + j] + u;
      ha[r * max_w + j] = L.n_layers > 0 ? fmaxf(v, 0.f) : v;
    }
  }
  __syncthreads();
  for (int i = 0; i < L.n_layers; ++i) {
    const bool last = i + 1 == L.n_layers;
    const T* W = (const T*)L.W[i];
    const int K = L.in_w[i], N = L.out_w[i];
    for (int j = threadIdx.x; j < N; j += CM_THREADS) {
      float acc[CM_LINKS];
      const float bj = L.b[i] ? L.b[i][j] : 0.f;
#pragma unroll
      for (int r = 0; r < CM_LINKS; ++r) acc[r] = bj;
      for (int k = 0; k < K; ++k) {
        const float w = Store<T>::ld(W + (int64_t)k * N + j);
#pragma unroll
        for (int r = 0; r < CM_LINKS; ++r) acc[r] = fmaf(ha[r * max_w + k], w, acc[r]);
      }
      for (int r = 0; r < nl; ++r) {
        if (last) out[((int64_t)b * ell + l0 + r) * N + j] = acc[r];
        else hb[r * max_w + j] = fmaxf(acc[r], 0.f);
      }
    }
    __syncthreads();
    float* t = ha; ha = hb; hb = t;
  }
  if (L.n_layers == 0)
    for (int j = threadIdx.x; j < w0; j += CM_THREADS)
      for (int r = 0; r < nl; ++r) out[((int64_t)b * ell + l0 + r) * w0 + j] = ha[r * max_w + j];
}

lime_status launch_link_ctx_mlp(int dtype, const float* first, const void* user_ctx, int d_c, const void* W0c, int w0, int B,
                                int ell, const FfnArgs& f, float* out, cudaStream_t st) {
  if (B == 0) return LIME_OK;
  FfnLayers L{};
  L.n_layers = f.n_layers;
  int max_w = w0;
  for (int i = 0; i < f.n_layers; ++i) {
    L.in_w[i] = f.in_w[i]; L.out_w[i] = f.out_w[i]; L.W[i] = f.W[i]; L.b[i] = f.b[i];
    if (f.out_w[i] > max_w) max_w = f.out_w[i];
  }
  const size_t smem = sizeof(float) * ((size_t)d_c + 2 * (size_t)CM_LINKS * max_w);
  if (smem > 96 * 1024) return LIME_UNSUPPORTED_SHAPE;
  dim3 grid((unsigned)((ell + CM_LINKS - 1) / CM_LINKS), (unsigned)B);
  ProfScope _p("k_link_ctx_mlp", st);
  if (dtype == LIME_F32) {
    LIME_CUDA(cudaFuncSetAttribute(k_link_ctx_mlp<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k_link_ctx_mlp<float><<<grid, CM_THREADS, smem, st>>>(first, (const float*)user_ctx, d_c, (const float*)W0c, w0, ell, max_w, L, out);
  } else {
    LIME_CUDA(cudaFuncSetAttribute(k_link_ctx_mlp<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k_link_ctx_mlp<__nv_bfloat16><<<grid, CM_THREADS, smem, st>>>(first, (const __nv_bfloat16*)user_ctx, d_c,
                                                                 (const __nv_bfloat16*)W0c, w0, ell, max_w, L, out);
  }
  LIME_LAUNCH_CHECK("k_link_ctx_mlp");
  return LIME_OK;
}

// ----------------------------------------------------------------------------- interaction network, generic scorer
// A block owns HS_SLOTS consecutive candidate slots and walks the users they belong to, keeping the user's LSW_b
// ([ell x w0], fp32) in shared memory; a warp takes HS_CPW candidates at a time so that every weight it reads serves
// all of them.  Candidate ids outside the corpus caches score 0 and lower the flag, as in the plain scorer.
constexpr int HS_WARPS = 4, HS_CPW = 4, HS_SLOTS = 64;
template <typename T>
__global__ void __launch_bounds__(HS_WARPS * 32)
k_score_head_simt(const float* __restrict__ LSW, const T* __restrict__ W, const T* __restrict__ Tc, int B, int ell, int d,
                  const int32_t* __restrict__ cand_off, int C, int64_t total, const int32_t* __restrict__ cand_ids,
                  int64_t corpus_rows, int32_t* __restrict__ dev_flag, const T* __restrict__ W0t, const float* __restrict__ b0, int w0,
                  int max_w, FfnLayers L, float* __restrict__ logits) {
  extern __shared__ float sm[];
  float* lsw = sm;                                   // [ell][w0]
  float* per_warp = lsw + ell * w0;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  float* ww = per_warp + wid * HS_CPW * (ell + d + 2 * max_w);    // [CPW][ell]
  float* tt = ww + HS_CPW * ell;                                  // [CPW][d]
  float* ha = tt + HS_CPW * d;                                    // [CPW][max_w]
  float* hb = ha + HS_CPW * max_w;
  int64_t i0 = (int64_t)blockIdx.x * HS_SLOTS;
  const int64_t i1 = min(total, i0 + HS_SLOTS);
  if (i0 >= i1) return;
  int b = cand_off ? upper_user(cand_off, B, (int)i0) : (int)(i0 / C);
  while (i0 < i1) {
    int64_t uend = cand_off ? (int64_t)cand_off[b + 1] : (int64_t)(b + 1) * C;
    while (uend <= i0 && b + 1 < B) { ++b; uend = cand_off ? (int64_t)cand_off[b + 1] : (int64_t)(b + 1) * C; }
    if (uend <= i0) return;
    const int64_t e = min(i1, uend);
    __syncthreads();
    for (int k = tid; k < ell * w0; k += blockDim.x) lsw[k] = LSW[(int64_t)b * ell * w0 + k];
    __syncthreads();
    for (int64_t g0 = i0 + (int64_t)wid * HS_CPW; g0 < e; g0 += HS_WARPS * HS_CPW) {
      const int nc = (int)min((int64_t)HS_CPW, e - g0);
      bool live[HS_CPW];
#pragma unroll
      for (int c = 0; c < HS_CPW; ++c) {
        live[c] = false;
        if (c < nc) {
          const int64_t i = g0 + c;
          const int64_t row = cand_ids ? (int64_t)cand_ids[i] : i;
          live[c] = !(cand_ids && (row < 0 || row >= corpus_rows));
          if (live[c]) {
            for (int l = lane; l < ell; l += 32) ww[c * ell + l] = Store<T>::ld(W + row * ell + l);
            for (int k = lane; k < d; k += 32) tt[c * d + k] = Store<T>::ld(Tc + row * d + k);
          } else {
            for (int l = lane; l < ell; l += 32) ww[c * ell + l] = 0.f;
            for (int k = lane; k < d; k += 32) tt[c * d + k] = 0.f;
            if (lane == 0) {
              logits[i] = 0.f;
              if (dev_flag != nullptr) atomicMin(dev_flag, (int32_t)min(i, (int64_t)INT32_MAX));
            }
          }
        } else {
          for (int l = lane; l < ell; l += 32) ww[c * ell + l] = 0.f;
          for (int k = lane; k < d; k += 32) tt[c * d + k] = 0.f;
        }
      }
      __syncwarp();
      // first layer, split over [O | T]
      for (int j = lane; j < w0; j += 32) {
        float acc[HS_CPW];
        const float bj = b0 ? b0[j] : 0.f;
#pragma unroll
        for (int c = 0; c < HS_CPW; ++c) acc[c] = bj;
        for (int l = 0; l < ell; ++l) {
          const float v = lsw[l * w0 + j];
#pragma unroll
          for (int c = 0; c < HS_CPW; ++c) acc[c] = fmaf(ww[c * ell + l], v, acc[c]);
        }
        for (int k = 0; k < d; ++k) {
          const float v = Store<T>::ld(W0t + (int64_t)k * w0 + j);
#pragma unroll
          for (int c = 0; c < HS_CPW; ++c) acc[c] = fmaf(tt[c * d + k], v, acc[c]);
        }
#pragma unroll
        for (int c = 0; c < HS_CPW; ++c) ha[c * max_w + j] = fmaxf(acc[c], 0.f);
      }
      __syncwarp();
      float* hin = ha;
      float* hout = hb;
      for (int i = 0; i < L.n_layers; ++i) {
        const bool last = i + 1 == L.n_layers;
        const T* Wi = (const T*)L.W[i];
        const int K = L.in_w[i], N = L.out_w[i];
        if (last) {
          // one output: the logit; lanes split the contraction
          float acc[HS_CPW];
#pragma unroll
          for (int c = 0; c < HS_CPW; ++c) acc[c] = 0.f;
          for (int k = lane; k < K; k += 32) {
            const float v = Store<T>::ld(Wi + k);
#pragma unroll
            for (int c = 0; c < HS_CPW; ++c) acc[c] = fmaf(hin[c * max_w + k], v, acc[c]);
          }
#pragma unroll
          for (int c = 0; c < HS_CPW; ++c) {
            const float s = warp_sum(acc[c]) + (L.b[i] ? L.b[i][0] : 0.f);
            if (lane == 0 && c < nc && live[c]) logits[g0 + c] = s;
          }
        } else {
          for (int j = lane; j < N; j += 32) {
            float acc[HS_CPW];
            const float bj = L.b[i] ? L.b[i][j] : 0.f;
#pragma unroll
            for (int c = 0; c < HS_CPW; ++c) acc[c] = bj;
            for (int k = 0; k < K; ++k) {
              const float v = Store<T>::ld(Wi + (int64_t)k * N + j);
#pragma unroll
              for (int c = 0; c < HS_CPW; ++c) acc[c] = fmaf(hin[c * max_w + k], v, acc[c]);
            }
#pragma unroll
            for (int c = 0; c < HS_CPW; ++c) hout[c * max_w + j] = fmaxf(acc[c], 0.f);
          }
          __syncwarp();
          float* t = hin; hin = hout; hout = t;
        }
      }
      __syncwarp();
    }
    i0 = e;
  }
}

lime_status launch_score_head_simt(const ScoreArgs& a, const float* LSW, const void* W0t, const float* b0, int w0,
                                   const FfnArgs& f, cudaStream_t st) {
  if (a.total == 0) return LIME_OK;
  FfnLayers L{};
  L.n_layers = f.n_layers;
  int max_w = w0;
  for (int i = 0; i < f.n_layers; ++i) {
    L.in_w[i] = f.in_w[i]; L.out_w[i] = f.out_w[i]; L.W[i] = f.W[i]; L.b[i] = f.b[i];
    if (f.out_w[i] > max_w) max_w = f.out_w[i];
  }
  const size_t smem = sizeof(float) * ((size_t)a.ell * w0 + (size_t)HS_WARPS * HS_CPW * (a.ell + a.d + 2 * (size_t)max_w));
  if (smem > 200 * 1024) return LIME_UNSUPPORTED_SHAPE;
  const int64_t blocks = (a.total + HS_SLOTS - 1) / HS_SLOTS;
  if (blocks > 0x7fffffffLL) return LIME_UNSUPPORTED_SHAPE;
  ProfScope _p("k_score_head_simt", st);
  if (a.dtype == LIME_F32) {
    LIME_CUDA(cudaFuncSetAttribute(k_score_head_simt<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k_score_head_simt<float><<<(int)blocks, HS_WARPS * 32, smem, st>>>(
        LSW, (const float*)a.W, (const float*)a.T, a.B, a.ell, a.d, a.cand_off, a.C, a.total, a.cand_ids, a.corpus_rows,
        a.dev_flag, (const float*)W0t, b0, w0, max_w, L, a.logits);
  } else {
    LIME_CUDA(cudaFuncSetAttribute(k_score_head_simt<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k_score_head_simt<__nv_bfloat16><<<(int)blocks, HS_WARPS * 32, smem, st>>>(
        LSW, (const __nv_bfloat16*)a.W, (const __nv_bfloat16*)a.T, a.B, a.ell, a.d, a.cand_off, a.C, a.total, a.cand_ids,
        a.corpus_rows, a.dev_flag, (const __nv_bfloat16*)W0t, b0, w0, max_w, L, a.logits);
  }
  LIME_LAUNCH_CHECK("k_score_head_simt");
  return LIME_OK;
}

}  // namespace lime
