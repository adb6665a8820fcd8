// Link-side operand preparation for the tensor-core XOR layer kernels.
//
// Both attention directions of Eq. 7 touch the history only through LN(S): K[S] = LN(S) W_K, V[S] = LN(S) W_V,
// Q[S] = LN(S) W_Q.  Because the link side is tiny (ell rows per user), the projections are folded into it, so
// that the streaming kernels contract directly against the stored history rows and never materialise Q/K/V of
// the history:
//   links <- history scores   Q[T]_h K[S]_h^T = Q2_(h,l) . LN(S)^T     Q2[(h,l), :] = scale * Q[T]_{l,h} W_{K,h}^T
//   history <- links scores   Q[S]_h K[T]_h^T = LN(S) . K2_(h,l)^T     K2[(h,l), :] = scale * K[T]_{l,h} W_{Q,h}^T
//   GatedMLP input O[S] W_g = P . G2,  O[S] W_u = P . U2               G2[(h,l), :] = V[T]_{l,h} W_g[h rows, :]
// (h, l) = head-major stacked link rows, H*ell of them.  Outputs are bf16 in the layouts the MMA operands want.
#include "lime_common.cuh"

namespace lime {

// out[(h,l), i] = scale * sum_{k < d_h} A[l, h*d_h + k] * W[i, h*d_h + k]      (W row-major [d_out x d], NULL = I)
// grid (users, H), block 256.  A fp32 [ell x d] per user.
__global__ void __launch_bounds__(256)
k_fold_rows(const float* __restrict__ A, int64_t a_user_stride, const __nv_bfloat16* __restrict__ W, int ell, int d,
            int H, int d_out, float scale, __nv_bfloat16* __restrict__ out, int64_t out_user_stride) {
  extern __shared__ float smem[];
  const int d_h = d / H;
  float* As = smem;                      // [ell][d_h]
  float* Ws = As + ell * d_h;            // [d_out][d_h + 1]
  const int u = blockIdx.x, h = blockIdx.y, tid = threadIdx.x;
  const float* a = A + (int64_t)u * a_user_stride;
  for (int i = tid; i < ell * d_h; i += blockDim.x) As[i] = a[(i / d_h) * d + h * d_h + (i % d_h)];
  for (int i = tid; i < d_out * d_h; i += blockDim.x) {
    const int r = i / d_h, k = i % d_h;
    Ws[r * (d_h + 1) + k] = W ? __bfloat162float(W[(int64_t)r * d + h * d_h + k]) : (r == h * d_h + k ? 1.f : 0.f);
  }
  __syncthreads();
  __nv_bfloat16* o = out + (int64_t)u * out_user_stride + (int64_t)h * ell * d_out;
  for (int i = tid; i < ell * d_out; i += blockDim.x) {
    const int l = i / d_out, r = i % d_out;
    float acc = 0.f;
    const float* ar = As + l * d_h;
    const float* wr = Ws + r * (d_h + 1);
    for (int k = 0; k < d_h; ++k) acc = fmaf(ar[k], wr[k], acc);
    o[(int64_t)l * d_out + r] = __float2bfloat16_rn(acc * scale);
  }
}

// outT[n, (h,l)] = sum_{k < d_h} A[l, h*d_h + k] * W[h*d_h + k, n]             (W row-major [d x f])
// i.e. the transposed fold, stored [f x H*ell] so that (h,l) is the contiguous (contraction) index.
__global__ void __launch_bounds__(256)
k_fold_cols_t(const float* __restrict__ A, int64_t a_user_stride, const __nv_bfloat16* __restrict__ W, int ell, int d,
              int H, int f, __nv_bfloat16* __restrict__ outT, int64_t out_user_stride) {
  extern __shared__ float smem[];
  const int d_h = d / H;
  float* As = smem;                      // [ell][d_h + 1]
  float* Ws = As + ell * (d_h + 1);      // [d_h][f]
  const int u = blockIdx.x, h = blockIdx.y, tid = threadIdx.x;
  const float* a = A + (int64_t)u * a_user_stride;
  for (int i = tid; i < ell * d_h; i += blockDim.x) As[(i / d_h) * (d_h + 1) + (i % d_h)] = a[(i / d_h) * d + h * d_h + (i % d_h)];
  for (int i = tid; i < d_h * f; i += blockDim.x) Ws[i] = __bfloat162float(W[(int64_t)(h * d_h + i / f) * f + (i % f)]);
  __syncthreads();
  const int HL = H * ell;
  __nv_bfloat16* o = outT + (int64_t)u * out_user_stride;
  for (int i = tid; i < ell * f; i += blockDim.x) {
    const int n = i / ell, l = i % ell;
    float acc = 0.f;
    const float* ar = As + l * (d_h + 1);
    for (int k = 0; k < d_h; ++k) acc = fmaf(ar[k], Ws[k * f + n], acc);
    o[(int64_t)n * HL + h * ell + l] = __float2bfloat16_rn(acc);
  }
}

// sums[r] = sum_i bf16 X[r, i]  (of the rounded values, so that the LayerNorm fold cancels exactly what the MMA sees)
__global__ void __launch_bounds__(256)
k_rowsum_bf16(const __nv_bfloat16* __restrict__ X, int64_t rows, int cols, float* __restrict__ sums) {
  const int lane = threadIdx.x & 31;
  const int64_t r = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (r >= rows) return;
  float s = 0.f;
  for (int i = lane; i < cols; i += 32) s += __bfloat162float(X[r * cols + i]);
  s = warp_sum(s);
  if (lane == 0) sums[r] = s;
}

// W [rows x cols] -> WT [cols x rows]  (bf16), set-up time only
__global__ void k_transpose_bf16(const __nv_bfloat16* __restrict__ W, int rows, int cols, __nv_bfloat16* __restrict__ WT) {
  __shared__ __nv_bfloat16 t[32][33];
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  for (int j = threadIdx.y; j < 32; j += blockDim.y) {
    const int r = r0 + j, c = c0 + threadIdx.x;
    if (r < rows && c < cols) t[j][threadIdx.x] = W[(int64_t)r * cols + c];
  }
  __syncthreads();
  for (int j = threadIdx.y; j < 32; j += blockDim.y) {
    const int c = c0 + j, r = r0 + threadIdx.x;
    if (r < rows && c < cols) WT[(int64_t)c * rows + r] = t[threadIdx.x][j];
  }
}

lime_status launch_transpose_bf16(const void* W, int rows, int cols, void* WT, cudaStream_t st) {
  ProfScope _p("k_transpose_bf16", st);
  dim3 grid((cols + 31) / 32, (rows + 31) / 32), block(32, 8);
  k_transpose_bf16<<<grid, block, 0, st>>>((const __nv_bfloat16*)W, rows, cols, (__nv_bfloat16*)WT);
  LIME_LAUNCH_CHECK("k_transpose_bf16");
  return LIME_OK;
}

lime_status launch_link_prep(const LinkPrepArgs& a, cudaStream_t st) {
  const int d_h = a.d / a.H, HL = a.H * a.ell;
  dim3 grid(a.users, a.H);
  const size_t smem_rows = sizeof(float) * ((size_t)a.ell * d_h + (size_t)a.d * (d_h + 1));
  const size_t smem_cols = sizeof(float) * ((size_t)a.ell * (d_h + 1) + (size_t)d_h * a.f);
  if (smem_rows > 200 * 1024 || smem_cols > 200 * 1024) return LIME_UNSUPPORTED_SHAPE;
  ProfScope _p("k_link_prep", st);
  LIME_CUDA(cudaFuncSetAttribute(k_fold_rows, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_rows));
  LIME_CUDA(cudaFuncSetAttribute(k_fold_cols_t, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_cols));
  const int64_t ustride = a.shared ? 0 : (int64_t)a.ell * a.d;
  if (a.Q2) {
    k_fold_rows<<<grid, 256, smem_rows, st>>>(a.QT, ustride, (const __nv_bfloat16*)a.Wk, a.ell, a.d, a.H, a.d, a.scale,
                                              (__nv_bfloat16*)a.Q2, (int64_t)HL * a.d);
    k_rowsum_bf16<<<(unsigned)(((int64_t)a.users * HL + 7) / 8), 256, 0, st>>>((const __nv_bfloat16*)a.Q2,
                                                                              (int64_t)a.users * HL, a.d, a.cQ);
  }
  if (a.K2) {
    k_fold_rows<<<grid, 256, smem_rows, st>>>(a.KT, ustride, (const __nv_bfloat16*)a.Wq, a.ell, a.d, a.H, a.d, a.scale,
                                              (__nv_bfloat16*)a.K2, (int64_t)HL * a.d);
    k_rowsum_bf16<<<(unsigned)(((int64_t)a.users * HL + 7) / 8), 256, 0, st>>>((const __nv_bfloat16*)a.K2,
                                                                              (int64_t)a.users * HL, a.d, a.cK);
    k_fold_cols_t<<<grid, 256, smem_cols, st>>>(a.VT, ustride, (const __nv_bfloat16*)a.Wg, a.ell, a.d, a.H, a.f,
                                                (__nv_bfloat16*)a.G2t, (int64_t)a.f * HL);
    k_fold_cols_t<<<grid, 256, smem_cols, st>>>(a.VT, ustride, (const __nv_bfloat16*)a.Wu, a.ell, a.d, a.H, a.f,
                                                (__nv_bfloat16*)a.U2t, (int64_t)a.f * HL);
  }
  LIME_LAUNCH_CHECK("k_link_prep");
  return LIME_OK;
}

}  // namespace lime
