// Link-side preparation for the tensor-core XOR layer kernels.
//
// Both attention directions of Eq. 7 touch the history only through LN(S): K[S] = LN(S) W_K, V[S] = LN(S) W_V,
// Q[S] = LN(S) W_Q.  Because the link side is tiny (ell rows per user), the history-side projections are folded
// into it, so that the streaming kernels contract directly against the stored history rows and never materialise
// Q/K/V of the history.  With That = LN(T) the link rows entering the layer and (h, l) the head-major stacked rows:
//   links <- history scores  Q[T]_h K[S]_h^T = Q2_(h,l) . LN(S)^T    Q2_(h,l) = That_l (scale W_{Q,h} W_{K,h}^T)
//   history <- links scores  Q[S]_h K[T]_h^T = LN(S) . K2_(h,l)^T    K2_(h,l) = That_l (scale W_{K,h} W_{Q,h}^T)
//   GatedMLP input           O[S] W_g = P . G2,  O[S] W_u = P . U2   G2_(h,l) = That_l (W_{V,h} W_g[h rows, :])
//   link rows                O[T] W_g = sum_h Ohat_(h,l) (W_{V,h} W_g[h rows, :])        (same folded matrices)
// The bracketed products depend on the weights only and are formed once, here, at lime_set_weights time; `scale`
// is the softmax scale times log2(e), so that the streaming kernels exponentiate with ex2 directly.
#include "lime_common.cuh"

namespace lime {

__device__ __forceinline__ float w_at(const __nv_bfloat16* W, int r, int c, int ld) {
  return W ? __bfloat162float(W[(int64_t)r * ld + c]) : (r == c ? 1.f : 0.f);
}

// WprepT (B operand of the PREP GEMM: one row per output column, contraction index j contiguous), row segments
//   [H*d] folded queries | [H*d] folded keys | then, with `plain_v` clear, [H*f] folded gate | [H*f] folded up;
//   with `plain_v` set, [d] rows of W_V^T (the link values V[T] = LN(T) W_V are then formed as they stand, for the
//   kernels that mix values head by head and apply the GatedMLP weights afterwards)
// WpostT [2f x H*d]     (B operand of the GLU GEMM on link rows)
__global__ void k_fold_weights(const __nv_bfloat16* __restrict__ Wq, const __nv_bfloat16* __restrict__ Wk,
                               const __nv_bfloat16* __restrict__ Wv, const __nv_bfloat16* __restrict__ Wg,
                               const __nv_bfloat16* __restrict__ Wu, int d, int H, int f, float scale, int plain_v,
                               __nv_bfloat16* __restrict__ WprepT, __nv_bfloat16* __restrict__ WpostT) {
  const int d_h = d / H;
  const int rows_qk = 2 * H * d;
  const int n_prep = (rows_qk + (plain_v ? d : 2 * H * f)) * d, n_post = 2 * f * H * d;
  for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < n_prep + n_post; idx += gridDim.x * blockDim.x) {
    float acc = 0.f;
    if (idx < n_prep) {
      const int R = idx / d, j = idx % d;
      if (R < rows_qk) {
        const int seg = R / (H * d), h = (R / d) % H, i = R % d;
        for (int k = h * d_h; k < (h + 1) * d_h; ++k)
          acc = seg == 0 ? fmaf(w_at(Wq, j, k, d), w_at(Wk, i, k, d), acc) : fmaf(w_at(Wk, j, k, d), w_at(Wq, i, k, d), acc);
        acc *= scale;
      } else if (plain_v) {
        acc = w_at(Wv, j, R - rows_qk, d);
      } else {
        const int R2 = R - rows_qk;
        const int seg = R2 / (H * f), h = (R2 / f) % H, i = R2 % f;
        const __nv_bfloat16* Wx = seg == 0 ? Wg : Wu;
        for (int k = h * d_h; k < (h + 1) * d_h; ++k) acc = fmaf(w_at(Wv, j, k, d), __bfloat162float(Wx[(int64_t)k * f + i]), acc);
      }
      WprepT[idx] = __float2bfloat16_rn(acc);
    } else {
      const int e = idx - n_prep;
      const int R = e / (H * d), c = e % (H * d);
      const int n = R % f, h = c / d, i = c % d;
      const __nv_bfloat16* Wx = R < f ? Wg : Wu;
      for (int k = h * d_h; k < (h + 1) * d_h; ++k) acc = fmaf(w_at(Wv, i, k, d), __bfloat162float(Wx[(int64_t)k * f + n]), acc);
      WpostT[e] = __float2bfloat16_rn(acc);
    }
  }
}

lime_status launch_fold_weights(const void* Wq, const void* Wk, const void* Wv, const void* Wg, const void* Wu, int d,
                                int H, int f, float scale, int plain_v, void* WprepT, void* WpostT, cudaStream_t st) {
  ProfScope _p("k_fold_weights", st);
  k_fold_weights<<<kSMs * 2, 256, 0, st>>>((const __nv_bfloat16*)Wq, (const __nv_bfloat16*)Wk, (const __nv_bfloat16*)Wv,
                                           (const __nv_bfloat16*)Wg, (const __nv_bfloat16*)Wu, d, H, f, scale, plain_v,
                                           (__nv_bfloat16*)WprepT, (__nv_bfloat16*)WpostT);
  LIME_LAUNCH_CHECK("k_fold_weights");
  return LIME_OK;
}

// out[r, :] = bf16( LN(T[r, :]) )  (or bf16(T) when ln == 0); one warp per row
__global__ void __launch_bounds__(256)
k_ln_rows_bf16(const float* __restrict__ T, int64_t rows, int d, int ln, float eps, __nv_bfloat16* __restrict__ out) {
  const int lane = threadIdx.x & 31;
  const int64_t r = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (r >= rows) return;
  const float* x = T + r * d;
  float mu = 0.f, rstd = 1.f;
  if (ln) {
    float s = 0.f;
    for (int k = lane; k < d; k += 32) s += x[k];
    mu = warp_sum(s) / (float)d;
    float v = 0.f;
    for (int k = lane; k < d; k += 32) { const float c = x[k] - mu; v = fmaf(c, c, v); }
    rstd = rsqrtf(warp_sum(v) / (float)d + eps);
  }
  for (int k = lane; k < d; k += 32) out[r * d + k] = __float2bfloat16_rn((x[k] - mu) * rstd);
}

lime_status launch_ln_rows_bf16(const float* T, int64_t rows, int d, int ln, float eps, void* out, cudaStream_t st) {
  if (rows == 0) return LIME_OK;
  ProfScope _p("k_ln_rows_bf16", st);
  k_ln_rows_bf16<<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(T, rows, d, ln, eps, (__nv_bfloat16*)out);
  LIME_LAUNCH_CHECK("k_ln_rows_bf16");
  return LIME_OK;
}

// Combine the chunks of a user with log-sum-exp weights and normalise (maxima are kept in the log2 domain):
//   Ohat[(u*ell + l), h*d + i] = sum_c w_c acc_c[(h,l), i] / sum_c w_c s_c,   w_c = 2^(m_c - max_c m_c)
// One warp per (user, stacked row), walked with a grid stride: lane c first takes chunk c's (m, s) (32 chunks at a time),
// the warp reduces the maximum and the weighted sum with shuffles, then every lane owns four consecutive columns per
// 128-column piece of the row and reads the chunks' partial accumulators as 128-bit words, four chunks in flight.
// d is a multiple of 4.  A user without history gets zeros; a user with a single chunk was already written by the
// attention kernel (its warps move on at once); when the schedule says that every user is such a user (*merge_needed == 0)
// the whole grid returns after one read.
__global__ void __launch_bounds__(256)
k_link_attn_merge_norm(const int32_t* __restrict__ chunk_start, const int32_t* __restrict__ merge_needed, int B, int ell, int d,
                       int H, const float* __restrict__ part_m, const float* __restrict__ part_s,
                       const float* __restrict__ part_acc, __nv_bfloat16* __restrict__ Ohat) {
  pdl_launch_dependents();     // simple kernel: the next one may set itself up beside it
  pdl_wait();                  // nothing is read or written before the previous kernel is complete
  if (merge_needed != nullptr && *merge_needed == 0) return;
  const int HL = H * ell;
  const int lane = threadIdx.x & 31;
  const int64_t n_rows = (int64_t)B * HL;
  const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
  for (int64_t wr = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); wr < n_rows; wr += warps) {
    const int u = (int)(wr / HL), row = (int)(wr % HL);
    const int c0 = chunk_start[u], c1 = chunk_start[u + 1];
    if (c1 - c0 == 1) continue;
    const int h = row / ell, l = row % ell;
    __nv_bfloat16* dst = Ohat + ((int64_t)u * ell + l) * (H * d) + h * d;
    // maximum over the chunks, then the normaliser
    float M = -INFINITY;
    for (int c = c0 + lane; c < c1; c += 32) M = fmaxf(M, part_m[(int64_t)c * HL + row]);
    M = warp_max(M);
    float S = 0.f;
    for (int c = c0 + lane; c < c1; c += 32) S = fmaf(part_s[(int64_t)c * HL + row], exp2f(part_m[(int64_t)c * HL + row] - M), S);
    S = warp_sum(S);
    const float inv = c1 > c0 ? 1.0f / S : 0.f;
    for (int i = lane * 4; i < d; i += 128) {
      float4 O = make_float4(0.f, 0.f, 0.f, 0.f);
      int c = c0;
      for (; c + 4 <= c1; c += 4) {
        float4 a[4];
        float w[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          a[k] = *reinterpret_cast<const float4*>(part_acc + ((int64_t)(c + k) * HL + row) * d + i);
          w[k] = exp2f(part_m[(int64_t)(c + k) * HL + row] - M);
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          O.x = fmaf(a[k].x, w[k], O.x); O.y = fmaf(a[k].y, w[k], O.y);
          O.z = fmaf(a[k].z, w[k], O.z); O.w = fmaf(a[k].w, w[k], O.w);
        }
      }
      for (; c < c1; ++c) {
        const float4 a = *reinterpret_cast<const float4*>(part_acc + ((int64_t)c * HL + row) * d + i);
        const float w = exp2f(part_m[(int64_t)c * HL + row] - M);
        O.x = fmaf(a.x, w, O.x); O.y = fmaf(a.y, w, O.y); O.z = fmaf(a.z, w, O.z); O.w = fmaf(a.w, w, O.w);
      }
      __nv_bfloat162 lo = __floats2bfloat162_rn(O.x * inv, O.y * inv), hi = __floats2bfloat162_rn(O.z * inv, O.w * inv);
      uint2 o;
      o.x = *reinterpret_cast<uint32_t*>(&lo);
      o.y = *reinterpret_cast<uint32_t*>(&hi);
      *reinterpret_cast<uint2*>(dst + i) = o;
    }
  }
}

lime_status launch_link_attn_merge_norm(const int32_t* chunk_start, const int32_t* merge_needed, int B, int ell, int d, int H,
                                        const float* part_m, const float* part_s, const float* part_acc, void* Ohat, cudaStream_t st) {
  if (B == 0) return LIME_OK;
  ProfScope _p("k_link_attn_merge_norm", st);
  const int64_t blocks_needed = ((int64_t)B * H * ell + 7) / 8;           // 8 warps (rows) per block
  const int grid = (int)(blocks_needed < (int64_t)kSMs * 8 ? blocks_needed : (int64_t)kSMs * 8);
  launch_pdl(k_link_attn_merge_norm, dim3(grid), dim3(256), 0, st, chunk_start, merge_needed, B, ell, d, H, part_m, part_s, part_acc,
             (__nv_bfloat16*)Ohat);
  LIME_LAUNCH_CHECK("k_link_attn_merge_norm");
  return LIME_OK;
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

}  // namespace lime
