// CUDA-core (fp32 FFMA) row-block linear layer: Y = epilogue( LN?(X) . W ).
// Serves the fp32 storage path and the fp32 link-row algebra (B*ell rows per layer: a few percent of the
// history rows).  The bf16 history rows go through the tensor-core kernels instead.
#include "lime_common.cuh"

namespace lime {

constexpr int LBM = 64, LBN = 64, LBK = 16;

template <typename TX, typename TW, typename TY, bool GLU>
__global__ void __launch_bounds__(256)
k_linear_simt(const TX* __restrict__ X, int64_t M, int K, int N,
              const TW* __restrict__ W0, const TW* __restrict__ W1, const TW* __restrict__ W2,
              TY* __restrict__ Y0, TY* __restrict__ Y1, TY* __restrict__ Y2,
              int ln, float ln_eps, int accumulate) {
  __shared__ float As[LBK][LBM + 4];
  __shared__ float Bs[GLU ? 2 : 1][LBK][LBN + 4];
  __shared__ float mu_s[LBM], rstd_s[LBM];

  const int tid = threadIdx.x;
  const int64_t row0 = (int64_t)blockIdx.x * LBM;
  const int col0 = blockIdx.y * LBN;
  const TW* Wa = blockIdx.z == 0 ? W0 : (blockIdx.z == 1 ? W1 : W2);
  const TW* Wb = W1;  // GLU: gate = W0, up = W1
  TY* Y = blockIdx.z == 0 ? Y0 : (blockIdx.z == 1 ? Y1 : Y2);

  // LayerNorm statistics of this block's rows (two passes over the row: mean, then centred variance)
  if (ln) {
    const int lane = tid & 31, wid = tid >> 5;
    for (int r = wid; r < LBM; r += 8) {
      const int64_t row = row0 + r;
      float mu = 0.f, rs = 0.f;
      if (row < M) {
        const TX* xr = X + row * K;
        float s = 0.f;
        for (int k = lane; k < K; k += 32) s += Store<TX>::ld(xr + k);
        mu = warp_sum(s) / (float)K;
        float v = 0.f;
        for (int k = lane; k < K; k += 32) { float c = Store<TX>::ld(xr + k) - mu; v += c * c; }
        rs = rsqrtf(warp_sum(v) / (float)K + ln_eps);
      }
      if (lane == 0) { mu_s[r] = mu; rstd_s[r] = rs; }
    }
  } else {
    if (tid < LBM) { mu_s[tid] = 0.f; rstd_s[tid] = 1.f; }
  }
  __syncthreads();

  const int ty = tid >> 4, tx = tid & 15;
  float acc[GLU ? 2 : 1][4][4];
#pragma unroll
  for (int g = 0; g < (GLU ? 2 : 1); ++g)
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[g][i][j] = 0.f;

  for (int k0 = 0; k0 < K; k0 += LBK) {
    // A tile: 64 rows x 16 k -> As[k][row]
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int idx = tid + e * 256;
      const int r = idx >> 4, k = idx & 15;
      const int64_t row = row0 + r;
      float v = 0.f;
      if (row < M && k0 + k < K) v = (Store<TX>::ld(X + row * K + k0 + k) - mu_s[r]) * rstd_s[r];
      As[k][r] = v;
    }
    // B tile(s): 16 k x 64 cols
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int idx = tid + e * 256;
      const int k = idx >> 6, c = idx & 63;
      const int kk = k0 + k, col = col0 + c;
      float v = 0.f, v2 = 0.f;
      if (kk < K && col < N) {
        v = Wa ? Store<TW>::ld(Wa + (int64_t)kk * N + col) : (kk == col ? 1.f : 0.f);
        if (GLU) v2 = Store<TW>::ld(Wb + (int64_t)kk * N + col);
      }
      Bs[0][k][c] = v;
      if (GLU) Bs[GLU ? 1 : 0][k][c] = v2;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < LBK; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[k][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[0][k][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[0][i][j] = fmaf(a[i], b[j], acc[0][i][j]);
      if (GLU) {
#pragma unroll
        for (int j = 0; j < 4; ++j) b[j] = Bs[GLU ? 1 : 0][k][tx * 4 + j];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[GLU ? 1 : 0][i][j] = fmaf(a[i], b[j], acc[GLU ? 1 : 0][i][j]);
      }
    }
    __syncthreads();
  }

#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t row = row0 + ty * 4 + i;
    if (row >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int col = col0 + tx * 4 + j;
      if (col >= N) continue;
      float v = acc[0][i][j];
      if (GLU) v = silu_f(v) * acc[GLU ? 1 : 0][i][j];
      TY* p = Y + row * N + col;
      if (accumulate) v += Store<TY>::ld(p);
      Store<TY>::st(p, v);
    }
  }
}

template <typename TX, typename TW, typename TY>
static lime_status launch_t(const LinearArgs& a, cudaStream_t st) {
  if (a.M == 0) return LIME_OK;
  ProfScope _p(a.glu ? "k_linear_simt_glu" : (a.ln ? "k_linear_simt_ln" : "k_linear_simt"), st);
  dim3 grid((unsigned)((a.M + LBM - 1) / LBM), (unsigned)((a.N + LBN - 1) / LBN), a.glu ? 1 : a.n_out);
  if (a.glu)
    k_linear_simt<TX, TW, TY, true><<<grid, 256, 0, st>>>(
        (const TX*)a.X, a.M, a.K, a.N, (const TW*)a.W[0], (const TW*)a.W[1], nullptr, (TY*)a.Y[0], nullptr, nullptr,
        a.ln, a.ln_eps, a.accumulate);
  else
    k_linear_simt<TX, TW, TY, false><<<grid, 256, 0, st>>>(
        (const TX*)a.X, a.M, a.K, a.N, (const TW*)a.W[0], (const TW*)a.W[1], (const TW*)a.W[2], (TY*)a.Y[0],
        (TY*)a.Y[1], (TY*)a.Y[2], a.ln, a.ln_eps, a.accumulate);
  LIME_LAUNCH_CHECK("k_linear_simt");
  return LIME_OK;
}

lime_status launch_linear_simt(const LinearArgs& a, cudaStream_t st) {
  const int x = a.x_dtype, w = a.w_dtype, y = a.y_dtype;
  if (x == LIME_F32 && w == LIME_F32 && y == LIME_F32) return launch_t<float, float, float>(a, st);
  if (x == LIME_F32 && w == LIME_BF16 && y == LIME_F32) return launch_t<float, __nv_bfloat16, float>(a, st);
  if (x == LIME_BF16 && w == LIME_BF16 && y == LIME_BF16)
    return launch_t<__nv_bfloat16, __nv_bfloat16, __nv_bfloat16>(a, st);
  if (x == LIME_BF16 && w == LIME_BF16 && y == LIME_F32) return launch_t<__nv_bfloat16, __nv_bfloat16, float>(a, st);
  return LIME_INVALID_ARG;
}

}  // namespace lime
