// Shared declarations of the CUDA side of the LIME hot path (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "lime.h"

namespace lime {

constexpr int kSMs = 148;  // B200: 2 dies x 74 SMs; grids of persistent kernels are sized from this

// ----------------------------------------------------------------------------- storage helpers
template <typename T> struct Store;
template <> struct Store<float> {
  static __device__ __forceinline__ float ld(const float* p) { return *p; }
  static __device__ __forceinline__ void st(float* p, float v) { *p = v; }
};
template <> struct Store<__nv_bfloat16> {
  static __device__ __forceinline__ float ld(const __nv_bfloat16* p) { return __bfloat162float(*p); }
  static __device__ __forceinline__ void st(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
};

__device__ __forceinline__ float silu_f(float x) { return x / (1.0f + __expf(-x)); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Largest b in [0, B) with start[b] <= x, for a non-decreasing start[0..B] (start[0] = 0).
__device__ __forceinline__ int upper_user(const int32_t* __restrict__ start, int B, int x) {
  int lo = 0, hi = B;  // invariant: start[lo] <= x, answer in [lo, hi)
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (start[mid] <= x) lo = mid; else hi = mid;
  }
  return lo;
}

// ----------------------------------------------------------------------------- context
struct Ctx {
  lime_config cfg;
  lime_weights w;
  bool have_weights;
  int device;
  int cand_heads;   // heads of the candidate side: 1 (one weight row per candidate) or H (one per head)
  int ell_c;        // weight columns per candidate = cand_heads * ell; also the rows of a user's link states
  float* keff;      // [ell x d] fp32: (L W_K^c) W_Q^c^T * cand_scale, the effective link keys of Eq. 4
  void* keff_hl;    // [2 ell x d] bf16: keff split into a rounded part and its remainder (tensor-core precompute)
  float* links32;   // [ell x d] fp32 copy of L (layer-1 link rows when no L^C is given)
  int tc_mode;                   // 0: generic kernels; 1: tensor-core layer kernels at d = 128; 2: at d = 256
  void* WoT[LIME_MAX_LAYERS];    // tensor-core path, per layer (NULL otherwise): W_o transposed [d x d_ff] bf16,
  void* WprepT[LIME_MAX_LAYERS]; //   folded PREP operand (k_link_prep.cu), folded link-row GLU operand [2*d_ff x H*d],
  void* WpostT[LIME_MAX_LAYERS]; //   and (tc_mode 2) [W_g | W_u] transposed [2*d_ff x d]
  void* WguT[LIME_MAX_LAYERS];
  // link-side operands of the first layer for the shared links T^0 = L (weights only, formed at lime_set_weights)
  void *sh_That, *sh_Q2, *sh_K2, *sh_G2t, *sh_U2t, *sh_V2t;
  float *sh_cQ, *sh_cK;
  // feed-forward networks (k_ffn_simt.cu, k_score_head_tc.cu): the caller's description plus derived device data
  bool have_head, have_ctx_mlp;
  lime_ffn head, ctx_mlp;
  int ctx_dc;            // context features per user
  void* head_W1bT;       // [w0 x d] bf16: the T half of the head's first layer, transposed (tensor-core path)
  void* head_W1aT;       // [w0 x d] bf16: its O half, transposed (B operand of the per-user link-state product)
  float* head_w2;        // [w_last] fp32 copy of the head's last layer
  float* ctx_first;      // [ell x w0] fp32: (L W_0[:d]) + b_0 of the context MLP
  int* dev_err;     // device word: 0, or the code of the first bounded wait that gave up in a kernel of this context
  float attn_scale, cand_scale, ln_eps;
  int d_ff, d_h;
};

// record a CUDA error for lime_last_cuda_error(); returns LIME_CUDA_ERROR
lime_status cuda_fail(cudaError_t e, const char* where);
#define LIME_CUDA(expr)                                          \
  do {                                                           \
    cudaError_t _e = (expr);                                     \
    if (_e != cudaSuccess) return ::lime::cuda_fail(_e, #expr);  \
  } while (0)
#define LIME_LAUNCH_CHECK(name)                                  \
  do {                                                           \
    cudaError_t _e = cudaGetLastError();                         \
    if (_e != cudaSuccess) return ::lime::cuda_fail(_e, name);   \
  } while (0)

// ----------------------------------------------------------------------------- programmatic dependent launch
// The kernels of one step run back to back on one stream.  Launched with the programmatic-serialization attribute, a
// kernel's CTAs may become resident while its predecessor still runs (as soon as every CTA of the predecessor has
// executed pdl_launch_dependents() or exited), set up their barriers and tensor memory, and then block in pdl_wait()
// until the predecessor has completed and its writes are visible.  Rules kept by every kernel launched this way:
//  - nothing produced by an earlier kernel is read, and no global memory is written, before pdl_wait();
//  - a kernel that allocates tensor memory calls pdl_launch_dependents() only after its allocation, so a dependent CTA
//    that shares the SM can never hold the columns a CTA of the running kernel still waits for.
// A kernel launched the ordinary way after such a kernel still waits for its completion, as always.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif
bool pdl_enabled();      // environment LIME_PDL=0 turns the attribute off (every launch then serialises fully)
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = pdl_enabled() ? 1 : 0;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ----------------------------------------------------------------------------- per-kernel event timing
// While a profile is open (lime_profile_start .. lime_profile_stop) every launcher brackets its kernel with two
// CUDA events on the launching stream.  Closed, a scope costs one predictable branch.
struct ProfScope {
  ProfScope(const char* name, cudaStream_t st);
  ~ProfScope();
  int slot;
  cudaStream_t st;
};

// ----------------------------------------------------------------------------- kernel launchers (host)
// Each returns LIME_OK or a status; all launch on `st` and never synchronise.

lime_status launch_offsets(const int32_t* len, int B, int32_t* off, cudaStream_t st);

lime_status launch_gather(int dtype, const void* table, int64_t V, int d, const int32_t* ids, int64_t total,
                          void* out, int32_t* dev_flag, cudaStream_t st);
// the same lookup with the non-affine LayerNorm of the row applied before it is stored
lime_status launch_gather_ln(int dtype, const void* table, int64_t V, int d, float eps, const int32_t* ids, int64_t total,
                             void* out, int32_t* dev_flag, cudaStream_t st);

// Work lists of the XOR layers in one launch: chunk_start[b] = sum_{b' < b} ceil(len_b' / chunk) and
// tile_start[b] = sum_{b' < b} ceil(len_b' / tile) for b = 0..B; chunk_user[item] = user of the chunk item (may be NULL);
// *merge_needed (may be NULL) = 1 if any user has several chunks or none (its attention rows come from the merge step)
// Optional: the chunk items dealt to n_groups groups of CTAs with even token-tile counts (tiles of att_tile tokens);
// group_start == NULL: not wanted.  group_start[n_groups + 1], group_items[items], scratch[4 x items].
struct GroupSchedule {
  int n_groups = 0, att_tile = 0;
  int32_t* group_start = nullptr; int32_t* group_items = nullptr; int32_t* scratch = nullptr;
};
lime_status launch_layer_schedules(const int32_t* off, int B, int chunk, int32_t* chunk_start, int tile, int32_t* tile_start,
                                   int32_t* chunk_user, int32_t* merge_needed, const GroupSchedule& gs, cudaStream_t st);

// Y[r, n] (+)= epilogue( LN?(X[r, :]) . W[:, n] ) for up to three weight matrices sharing X.
struct LinearArgs {
  const void* X; int x_dtype;   // [M x K], lime_dtype
  int64_t M; int K; int N;      // every W is [K x N], stored w_dtype; a NULL W means identity (K == N)
  const void* W[3]; int w_dtype;
  void* Y[3]; int y_dtype;      // outputs [M x N] each (ldy = N)
  int n_out;                    // 1..3 (ignored when glu)
  int ln; float ln_eps;         // LayerNorm rows of X first
  int glu;                      // 1: Y[0] = SiLU(X W[0]) * (X W[1])
  int accumulate;               // 1: Y[0] += result (y_dtype must be F32, n_out == 1)
  const float* also_add_to;     // unused (reserved)
};
lime_status launch_linear_simt(const LinearArgs& a, cudaStream_t st);

// link <- history attention partials: per (user, chunk of `chunk` tokens, head, link row): running max, sum,
// un-normalised weighted values.
struct AttnLinkArgs {
  const float* QT; int64_t qt_user_stride;   // [B x ell x d] fp32 (stride 0: shared)
  const void* KS; const void* VS; int s_dtype; // [total x d]
  const int32_t* off; int B; int64_t total;
  int ell, d, H; int phi; float scale;
  int chunk; const int32_t* chunk_start; int n_chunk_upper;  // work list from launch_layer_schedules
  float* part_m; float* part_s; float* part_acc;             // [n_chunk_upper x H x ell], same, [.. x d_h]
  float* AT;                                                  // out [B x ell x d] fp32
};
lime_status launch_attn_link_simt(const AttnLinkArgs& a, cudaStream_t st);
lime_status launch_attn_link_merge(const AttnLinkArgs& a, cudaStream_t st);

// history <- links attention: AS[t, :] = phi(Q[S]_t K[T]^T) V[T] per head, over the ell links of t's user
struct AttnHistArgs {
  const void* QS; void* AS; int s_dtype;     // [total x d]; AS may alias QS
  const float* KT; const float* VT; int64_t t_user_stride;  // [B x ell x d] fp32
  const int32_t* off; int B; int64_t total;
  int ell, d, H; int phi; float scale;
  int tile; const int32_t* tile_start; int n_tile_upper;
};
lime_status launch_attn_hist_simt(const AttnHistArgs& a, cudaStream_t st);

// out[r, :] (storage dtype) = in[r, :] fp32, optionally accumulate into acc fp32 first
lime_status launch_cast_rows(const float* in, int64_t n, void* out, int dtype, cudaStream_t st);
lime_status launch_axpy(const float* x, float* y, int64_t n, int zero_first, cudaStream_t st);
lime_status launch_widen(const void* in, int dtype, float* out, int64_t n, cudaStream_t st);

// candidate -> link weights: W[c, :] = softmax_l( <T_c, keff_l> )  (keff already carries cand_scale); `rows` keys
// in groups of `ell` (one group per head of the candidate side), the softmax inside each group
lime_status launch_precompute(int dtype, const void* cand, int64_t M, int d, int rows, int ell, const float* keff,
                              void* out_w, cudaStream_t st);
// keff = ((L Wk) Wq^T) * scale, fp32 [heads * ell x d]: one key per link, or per (head, link) restricted to the
// head's columns; the buffer holds 2 * heads * ell * d floats
lime_status launch_keff(int dtype, const void* L, const void* Wk, const void* Wq, int ell, int d, int heads, float scale,
                        float* keff, cudaStream_t st);
// link states for the per-head candidate side: out[b, h * ell + l, :] = src[b, l, :] on head h's columns, 0 elsewhere
lime_status launch_expand_heads(const float* src, int64_t rows_in, int ell, int d, int heads, void* out, int dtype, cudaStream_t st);

// bf16 precompute on tcgen05 tensor cores (ell in {16,32,64,128}, d % 64 == 0); keff_hl from launch_keff_split
// `ell` keys in all, softmax per group of `group` consecutive keys (group == ell: one softmax per row)
bool precompute_tc_supported(int dtype, int d, int ell, int group);
lime_status launch_keff_split(const float* keff, int ell, int d, void* keff_hl, cudaStream_t st);
lime_status launch_precompute_tc(const void* cand, int64_t M, int d, int rows, int group, const void* keff_hl, void* out_w,
                                 int* err, cudaStream_t st);

struct ScoreArgs {
  const void* LS; const void* W; const void* T; int dtype;
  int B; int ell, d;
  const int32_t* cand_off; int C; int64_t total;
  const int32_t* cand_ids;      // nullable; with ids, W and T have `corpus_rows` rows and ids outside [0, corpus_rows) score 0
  int64_t corpus_rows;
  int32_t* dev_flag;            // nullable: lowered to the smallest slot whose id was out of range
  float* logits;
  int64_t ldw, ldt;             // row pitch of W and T in elements; 0 = dense (ell, d).  Packed corpus records: d + ell both
};
// out[v, :] = [ emb[v, 0..d) | w[v, 0..ell) ]: one record per item of the corpus caches (k_cand_simt.cu)
lime_status launch_pack_corpus(int dtype, const void* emb, const void* w, int64_t V, int d, int ell, void* out, cudaStream_t st);
lime_status launch_score_simt(const ScoreArgs& a, cudaStream_t st);
// bf16 streaming scorer on tcgen05 tensor cores (fixed C per user, dense rows, ell in {16,32,64,128}, d % 64 == 0)
bool score_tc_supported(const ScoreArgs& a);
lime_status launch_score_tc(const ScoreArgs& a, int* err, cudaStream_t st);
// the same with rows taken from corpus-level caches by cand_ids (fixed C per user), k_score_gather_tc.cu
bool score_gather_tc_supported(const ScoreArgs& a);
lime_status launch_score_gather_tc(const ScoreArgs& a, int* err, cudaStream_t st);

// one-thread kernel whose only wait can never be satisfied (self-test of the bounded waits, tc_host.cu)
lime_status launch_wait_expiry(int* err, uint64_t limit_ns, int code, cudaStream_t st);

// ---- feed-forward networks: Eq. 2 and the interaction network of Sec. 3.3 ------------------------------------------
// layers after the first (whose input is a concatenation and is handled split): W[i] [in_w[i] x out_w[i]], b[i] nullable
struct FfnArgs {
  int n_layers;
  int in_w[LIME_FFN_MAX_HIDDEN + 1], out_w[LIME_FFN_MAX_HIDDEN + 1];
  const void* W[LIME_FFN_MAX_HIDDEN + 1];
  const float* b[LIME_FFN_MAX_HIDDEN + 1];
};
// Y = X . W (+ bias) for a few rows: fp32 [M x N] and / or bf16 transposed per group of rows [M/group][N][group]
lime_status launch_rows_times_w(const void* X, int x_dtype, int64_t M, int K, const void* W, int w_dtype, int ldw, int N,
                                const float* bias, float* Y, void* Yt, int group, const char* name, cudaStream_t st);
lime_status launch_link_ctx_mlp(int dtype, const float* first, const void* user_ctx, int d_c, const void* W0c, int w0, int B,
                                int ell, const FfnArgs& f, float* out, cudaStream_t st);
// generic scorer through the interaction network; LSW fp32 [B x ell x w0], W0t = rows d.. of the first layer [d x w0]
lime_status launch_score_head_simt(const ScoreArgs& a, const float* LSW, const void* W0t, const float* b0, int w0,
                                   const FfnArgs& f, cudaStream_t st);
// one hidden layer of n1 units on tensor cores; LSWt bf16 [B x n1 x ell], W1bT bf16 [n1 x d], w2 fp32 [n1]
struct ScoreHeadArgs {
  const void* LSWt; const void* W1bT; const float* b1; const float* w2; const float* b2; int n1;
};
bool score_head_tc_supported(const ScoreArgs& a, int n1);
lime_status launch_score_head_tc(const ScoreArgs& a, const ScoreHeadArgs& h, int* err, cudaStream_t st);

// ---- tensor-core XOR layer (bf16, d = d_ff = 128, H * ell = 128) ----------------------------------------------
// plain_v: WprepT's third segment is W_V^T (link values formed as they stand) instead of the folded gate / up products
lime_status launch_fold_weights(const void* Wq, const void* Wk, const void* Wv, const void* Wg, const void* Wu, int d,
                                int H, int f, float scale, int plain_v, void* WprepT, void* WpostT, cudaStream_t st);
lime_status launch_ln_rows_bf16(const float* T, int64_t rows, int d, int ln, float eps, void* out, cudaStream_t st);
lime_status launch_link_attn_merge_norm(const int32_t* chunk_start, const int32_t* merge_needed, int B, int ell, int d, int H,
                                        const float* part_m, const float* part_s, const float* part_acc, void* Ohat, cudaStream_t st);
lime_status launch_transpose_bf16(const void* W, int rows, int cols, void* WT, cudaStream_t st);

// link-row GEMMs on tensor cores (k_gemm_tc.cu); A [M x K] bf16 row-major, Bt [N x K] bf16 (weights, pre-folded)
struct LinkGemmArgs {
  const void* A; int64_t M; int K; const void* Bt; void* out;   // K = d
  int ell, H, need_hist;                       // PREP: rows are (user, link); need_hist = also K2 and G2t / U2t (or V2t)
  int f, plain_v;                              // GatedMLP width; plain_v: V2t [users x d x ell] instead of G2t / U2t
  void *Q2, *K2, *G2t, *U2t, *V2t; float *cQ, *cK;   // PREP outputs (cQ / cK nullable; only formed with d = 128)
  int* err;
};
lime_status launch_gemm_prep(const LinkGemmArgs& a, cudaStream_t st);
// A [M x K] . Bt^T, Bt [n_cols x K] (bf16, K % 64 == 0, 16-byte aligned): bf16 result transposed per group of rows,
// out_t [M / group][n_cols][group]
lime_status launch_gemm_rows_t(const void* A, int64_t M, int K, const void* Bt, int n_cols, int group, void* out_t, int* err,
                               const char* name, cudaStream_t st);

// GatedMLP on link rows fused with its consumers (k_link_mlp_tc.cu); d = d_ff in {128, 256}
struct LinkMlpArgs {
  const void* Ohat; int64_t M; int K; int d;   // attention rows [M x K = H*d] bf16
  const void* WpostT; const void* WoT;         // folded [2f x H*d] and transposed [d x f] weights, bf16
  float* T_out;                                // nullable: the layer's link rows, fp32 [M x d]
  float* LP; int lp_accumulate;                // nullable running sum of Eq. 8 (0: assign, 1: add)
  void* That_next;                             // nullable: bf16 LN(T) for the next layer's link-side GEMM
  void* link_states;                           // nullable: bf16 copy of LP after this layer
  int ln; float ln_eps;
  int* err;
};
lime_status launch_link_mlp_tc(const LinkMlpArgs& a, cudaStream_t st);

struct LinkAttnArgs {
  const void* hist; int64_t total;          // [total x d] bf16
  const void* Q2; const float* cQ;          // folded link queries [users x H*ell x d] bf16 and their row sums
  const int32_t* off; const int32_t* chunk_start; int B, chunk, n_chunk_upper;
  const int32_t* chunk_user;                // [items] user of each (user, chunk) work item
  const int32_t* group_start; const int32_t* group_items; int n_groups;   // balanced deal of the items (d = 256 kernel)
  int ell, d, H, shared, ln; float ln_eps;
  int silu;                                 // 1: SiLU(s) / N(U) instead of softmax (Algorithm 2)
  float *part_m, *part_s, *part_acc;        // scratch: [items x H*ell], same, [items x H*ell x d]
  void* Ohat;                               // [B*ell x H*d] bf16: rows of users whose history is one chunk
  float2* stats_out;                        // nullable, ln only: {rstd, mean} of every history row, for the history update
  int* err;
};
bool link_attn_tc_supported(int dtype, int d, int H, int ell, int phi);
int link_attn_d256_groups(int n_chunk_upper, int H, int ell);   // groups of CTAs (one CTA per 128-row block) of that kernel
lime_status launch_link_attn_tc(const LinkAttnArgs& a, cudaStream_t st);

struct HistUpdateArgs {
  const void* hist_in; void* hist_out; int64_t total;
  const void *K2, *G2t, *U2t; const float* cK; const void* WoT;   // WoT [d x f] bf16 (W_o transposed)
  const int32_t* off; const int32_t* tile_start; int B, n_tile_upper;
  int ell, shared, ln; float ln_eps;    // ln: apply LayerNorm to the rows read (0 when they were stored normalised)
  int out_ln;                           // 1: store LayerNorm(S') instead of S'
  int silu;                             // 1: SiLU(s) / ell instead of the per-head softmax (Algorithm 2)
  const float2* stats_in;               // nullable, ln only: {rstd, mean} of every row read, as left by the attention kernel
  int* err;
};
bool hist_update_tc_supported(int dtype, int d, int f, int H, int ell, int phi, int gated_mlp);
lime_status launch_hist_update_tc(const HistUpdateArgs& a, cudaStream_t st);
// same step for H * ell in {256, 384, 512} (link-side operands streamed per tile, k_hist_update2_tc.cu)
bool hist_update2_tc_supported(int dtype, int d, int f, int H, int ell, int phi, int gated_mlp);
lime_status launch_hist_update2_tc(const HistUpdateArgs& a, int H, cudaStream_t st);

// ---- tensor-core XOR layer at d = d_ff = 256 (bf16, ell = 64, H in {2, 4, 8}; history rows LayerNorm-ed already) ----
bool link_attn_d256_tc_supported(int dtype, int d, int H, int ell, int phi);
lime_status launch_link_attn_d256_tc(const LinkAttnArgs& a, cudaStream_t st);   // a.ln must be 0

struct HistUpdate256Args {
  const void* hist_in; void* hist_out; int64_t total;
  const void* K2;                       // folded link keys [users x H*ell x d] bf16
  const void* V2t;                      // link values, transposed [users x d x ell] bf16
  const void* WguT; const void* WoT;    // [W_g | W_u]^T [2f x d] and W_o^T [d x f], bf16
  const int32_t* off; const int32_t* tile_start; int B, n_tile_upper;
  int H, shared;
  int out_ln;                           // 1: store LayerNorm(S') instead of S'
  int silu;                             // 1: SiLU(s) / ell instead of the per-head softmax (Algorithm 2)
  float ln_eps;
  int* err;
};
bool hist_update_d256_tc_supported(int dtype, int d, int f, int H, int ell, int phi, int gated_mlp);
lime_status launch_hist_update_d256_tc(const HistUpdate256Args& a, cudaStream_t st);

}  // namespace lime
