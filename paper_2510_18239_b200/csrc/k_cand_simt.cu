// Candidate side of Eq. 4 on CUDA cores: the offline candidate->link weights and the generic scorer.
// The generic scorer serves fp32 storage, odd shapes and id-indirected (corpus-cache) candidates; the bf16
// streaming scorer on tensor cores lives in k_score_tc.cu.
#include "lime_common.cuh"

namespace lime {

// ----------------------------------------------------------------------------- effective link keys
// keff[l, i] = scale * sum_j (L Wk)[l, j] * Wq[i, j]   so that <T_c Wq, L_l Wk> * scale = <T_c, keff_l>.
// With `heads` > 1 (candidate side head by head) there is one key per (head, link): row h * ell + l sums only over
// head h's columns j, so that <T_c, keff_(h,l)> is head h's score of candidate c against link l.
template <typename T>
__global__ void k_keff_stage1(const T* __restrict__ L, const T* __restrict__ Wk, int ell, int d, float* __restrict__ tmp) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= ell * d) return;
  const int l = i / d, j = i % d;
  float acc;
  if (Wk) {
    acc = 0.f;
    for (int k = 0; k < d; ++k) acc = fmaf(Store<T>::ld(L + l * d + k), Store<T>::ld(Wk + (int64_t)k * d + j), acc);
  } else {
    acc = Store<T>::ld(L + i);
  }
  tmp[i] = acc;
}
template <typename T>
__global__ void k_keff_stage2(const float* __restrict__ tmp, const T* __restrict__ Wq, int ell, int d, int heads, float scale,
                              float* __restrict__ keff) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= heads * ell * d) return;
  const int row = i / d, r = i % d;
  const int h = row / ell, l = row % ell;
  const int dh = d / heads, j0 = h * dh, j1 = j0 + dh;      // head h's columns (all of them with one head)
  float acc;
  if (Wq) {
    acc = 0.f;
    for (int j = j0; j < j1; ++j) acc = fmaf(tmp[l * d + j], Store<T>::ld(Wq + (int64_t)r * d + j), acc);
  } else {
    acc = (r >= j0 && r < j1) ? tmp[l * d + r] : 0.f;
  }
  keff[i] = acc * scale;
}

lime_status launch_keff(int dtype, const void* L, const void* Wk, const void* Wq, int ell, int d, int heads, float scale,
                        float* keff, cudaStream_t st) {
  // stage 1 writes behind the keys (the caller provides 2 * heads * ell * d floats)
  float* tmp = keff + (size_t)heads * ell * d;
  const int n = ell * d, blocks = (n + 127) / 128, blocks2 = (heads * n + 127) / 128;
  ProfScope _p("k_keff", st);
  if (dtype == LIME_F32) {
    k_keff_stage1<float><<<blocks, 128, 0, st>>>((const float*)L, (const float*)Wk, ell, d, tmp);
    k_keff_stage2<float><<<blocks2, 128, 0, st>>>(tmp, (const float*)Wq, ell, d, heads, scale, keff);
  } else {
    k_keff_stage1<__nv_bfloat16><<<blocks, 128, 0, st>>>((const __nv_bfloat16*)L, (const __nv_bfloat16*)Wk, ell, d, tmp);
    k_keff_stage2<__nv_bfloat16><<<blocks2, 128, 0, st>>>(tmp, (const __nv_bfloat16*)Wq, ell, d, heads, scale, keff);
  }
  LIME_LAUNCH_CHECK("k_keff");
  return LIME_OK;
}

// ----------------------------------------------------------------------------- candidate -> link weights
// W[c, :] = softmax over links of <T_c, keff_l>.  keff (fp32) sits in shared memory, one warp per candidate.  The
// `rows` keys form rows / ell groups (one per head of the candidate side); the softmax runs inside each group.
constexpr int PC_WARPS = 8;
template <typename T>
__global__ void __launch_bounds__(PC_WARPS * 32)
k_precompute(const T* __restrict__ cand, int64_t M, int d, int rows, int ell, const float* __restrict__ keff, T* __restrict__ out_w) {
  extern __shared__ float smem[];
  const int ldk = d + 1;
  float* Ks = smem;                  // [ell][d+1]
  float* ts = Ks + rows * ldk;       // [warps][d]
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  for (int i = tid; i < rows * d; i += blockDim.x) Ks[(i / d) * ldk + (i % d)] = keff[i];
  __syncthreads();
  float* tw = ts + wid * d;
  constexpr int MAXL = 8;
  for (int64_t c = (int64_t)blockIdx.x * PC_WARPS + wid; c < M; c += (int64_t)gridDim.x * PC_WARPS) {
    for (int k = lane; k < d; k += 32) tw[k] = Store<T>::ld(cand + c * d + k);
    __syncwarp();
    for (int g0 = 0; g0 < rows; g0 += ell) {
      float p[MAXL];
      float mx = -INFINITY;
#pragma unroll
      for (int j = 0; j < MAXL; ++j) {
        const int l = lane + 32 * j;
        float sc = -INFINITY;
        if (l < ell) {
          sc = 0.f;
          const float* kr = Ks + (g0 + l) * ldk;
          for (int k = 0; k < d; ++k) sc = fmaf(tw[k], kr[k], sc);
        }
        p[j] = sc;
        mx = fmaxf(mx, sc);
      }
      mx = warp_max(mx);
      float sum = 0.f;
#pragma unroll
      for (int j = 0; j < MAXL; ++j) {
        p[j] = (lane + 32 * j < ell) ? __expf(p[j] - mx) : 0.f;
        sum += p[j];
      }
      const float inv = 1.f / warp_sum(sum);
#pragma unroll
      for (int j = 0; j < MAXL; ++j) {
        const int l = lane + 32 * j;
        if (l < ell) Store<T>::st(out_w + c * rows + g0 + l, p[j] * inv);
      }
    }
    __syncwarp();
  }
}

lime_status launch_precompute(int dtype, const void* cand, int64_t M, int d, int rows, int ell, const float* keff, void* out_w,
                              cudaStream_t st) {
  if (M == 0) return LIME_OK;
  const size_t smem = sizeof(float) * ((size_t)rows * (d + 1) + (size_t)PC_WARPS * d);
  if (smem > 200 * 1024) return LIME_UNSUPPORTED_SHAPE;
  int64_t blocks = (M + PC_WARPS - 1) / PC_WARPS;
  const int64_t cap = (int64_t)kSMs * 4;
  if (blocks > cap) blocks = cap;
  ProfScope _p("k_precompute", st);
  if (dtype == LIME_F32) {
    LIME_CUDA(cudaFuncSetAttribute(k_precompute<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k_precompute<float><<<(int)blocks, PC_WARPS * 32, smem, st>>>((const float*)cand, M, d, rows, ell, keff, (float*)out_w);
  } else {
    LIME_CUDA(cudaFuncSetAttribute(k_precompute<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k_precompute<__nv_bfloat16><<<(int)blocks, PC_WARPS * 32, smem, st>>>((const __nv_bfloat16*)cand, M, d, rows, ell, keff,
                                                                        (__nv_bfloat16*)out_w);
  }
  LIME_LAUNCH_CHECK("k_precompute");
  return LIME_OK;
}

// ----------------------------------------------------------------------------- generic scorer
// logit[i] = < sum_l W[i, l] LS_b[l, :], T[i, :] >.  A block owns SC_SLOTS consecutive candidate slots, walks the
// users those slots belong to, keeps that user's link states in shared memory (fp32) and gives each warp one
// candidate at a time.
constexpr int SC_WARPS = 8, SC_SLOTS = 64;
template <typename T>
__global__ void __launch_bounds__(SC_WARPS * 32)
k_score_simt(const T* __restrict__ LS, const T* __restrict__ W, const T* __restrict__ Tc, int B, int ell, int d,
             const int32_t* __restrict__ cand_off, int C, int64_t total, const int32_t* __restrict__ cand_ids,
             int64_t corpus_rows, int32_t* __restrict__ dev_flag, float* __restrict__ logits, int64_t ldw, int64_t ldt) {
  extern __shared__ float smem[];
  float* Ls = smem;                  // [ell][d]
  float* ws = Ls + ell * d;          // [warps][ell]
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  int64_t i0 = (int64_t)blockIdx.x * SC_SLOTS;
  const int64_t i1 = min(total, i0 + SC_SLOTS);
  if (i0 >= i1) return;
  int b = cand_off ? upper_user(cand_off, B, (int)i0) : (int)(i0 / C);
  float* ww = ws + wid * ell;
  while (i0 < i1) {
    int64_t uend = cand_off ? (int64_t)cand_off[b + 1] : (int64_t)(b + 1) * C;
    while (uend <= i0 && b + 1 < B) { ++b; uend = cand_off ? (int64_t)cand_off[b + 1] : (int64_t)(b + 1) * C; }
    if (uend <= i0) return;  // slots past the last user's range: nothing owns them
    const int64_t e = min(i1, uend);
    __syncthreads();
    const T* ls = LS + (int64_t)b * ell * d;
    for (int k = tid; k < ell * d; k += blockDim.x) Ls[k] = Store<T>::ld(ls + k);
    __syncthreads();
    for (int64_t i = i0 + wid; i < e; i += SC_WARPS) {
      const int64_t row = cand_ids ? (int64_t)cand_ids[i] : i;
      if (cand_ids && (row < 0 || row >= corpus_rows)) {
        // an id outside the corpus caches reads nothing: logit 0 and the smallest offending slot recorded
        if (lane == 0) {
          logits[i] = 0.f;
          if (dev_flag != nullptr) atomicMin(dev_flag, (int32_t)min(i, (int64_t)INT32_MAX));
        }
        continue;
      }
      for (int l = lane; l < ell; l += 32) ww[l] = Store<T>::ld(W + row * ldw + l);
      __syncwarp();
      float dot = 0.f;
      for (int k = lane; k < d; k += 32) {
        float o = 0.f;
        for (int l = 0; l < ell; ++l) o = fmaf(ww[l], Ls[l * d + k], o);
        dot = fmaf(o, Store<T>::ld(Tc + row * ldt + k), dot);
      }
      dot = warp_sum(dot);
      if (lane == 0) logits[i] = dot;
      __syncwarp();
    }
    i0 = e;
  }
}

lime_status launch_score_simt(const ScoreArgs& a, cudaStream_t st) {
  if (a.total == 0) return LIME_OK;
  const size_t smem = sizeof(float) * ((size_t)a.ell * a.d + (size_t)SC_WARPS * a.ell);
  if (smem > 200 * 1024) return LIME_UNSUPPORTED_SHAPE;
  const int64_t blocks = (a.total + SC_SLOTS - 1) / SC_SLOTS;
  if (blocks > 0x7fffffffLL) return LIME_UNSUPPORTED_SHAPE;
  const int64_t ldw = a.ldw ? a.ldw : a.ell, ldt = a.ldt ? a.ldt : a.d;
  ProfScope _p("k_score_simt", st);
  if (a.dtype == LIME_F32) {
    LIME_CUDA(cudaFuncSetAttribute(k_score_simt<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k_score_simt<float><<<(int)blocks, SC_WARPS * 32, smem, st>>>((const float*)a.LS, (const float*)a.W, (const float*)a.T,
                                                                 a.B, a.ell, a.d, a.cand_off, a.C, a.total, a.cand_ids,
                                                                 a.corpus_rows, a.dev_flag, a.logits, ldw, ldt);
  } else {
    LIME_CUDA(cudaFuncSetAttribute(k_score_simt<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    k_score_simt<__nv_bfloat16><<<(int)blocks, SC_WARPS * 32, smem, st>>>(
        (const __nv_bfloat16*)a.LS, (const __nv_bfloat16*)a.W, (const __nv_bfloat16*)a.T, a.B, a.ell, a.d, a.cand_off,
        a.C, a.total, a.cand_ids, a.corpus_rows, a.dev_flag, a.logits, ldw, ldt);
  }
  LIME_LAUNCH_CHECK("k_score_simt");
  return LIME_OK;
}

// ----------------------------------------------------------------------------- packed corpus records
// One record per item: its embedding row followed by its cached candidate->link weights (Sec. 3.3: the "QK cache" sits
// beside the item embedding), so that scoring by id touches one place in memory per candidate instead of two.
template <typename T>
__global__ void __launch_bounds__(256)
k_pack_corpus(const T* __restrict__ emb, const T* __restrict__ w, int64_t V, int d, int ell, T* __restrict__ out) {
  const int rec = d + ell;
  const int64_t n = V * rec;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t v = i / rec;
    const int c = (int)(i % rec);
    out[i] = c < d ? emb[v * d + c] : w[v * ell + (c - d)];
  }
}

lime_status launch_pack_corpus(int dtype, const void* emb, const void* w, int64_t V, int d, int ell, void* out, cudaStream_t st) {
  if (V == 0) return LIME_OK;
  ProfScope _p("k_pack_corpus", st);
  if (dtype == LIME_F32) k_pack_corpus<float><<<kSMs * 8, 256, 0, st>>>((const float*)emb, (const float*)w, V, d, ell, (float*)out);
  else k_pack_corpus<__nv_bfloat16><<<kSMs * 8, 256, 0, st>>>((const __nv_bfloat16*)emb, (const __nv_bfloat16*)w, V, d, ell, (__nv_bfloat16*)out);
  LIME_LAUNCH_CHECK("k_pack_corpus");
  return LIME_OK;
}

}  // namespace lime
