// C-ABI entry points: argument validation, workspace carving and launch sequencing.  No arithmetic of the
// method lives here; every step runs in the kernels of this directory.
#include <cstdio>
#include <cstring>
#include <new>

#include "lime_common.cuh"

namespace lime {

static thread_local char g_err[256] = "";

lime_status cuda_fail(cudaError_t e, const char* where) {
  snprintf(g_err, sizeof(g_err), "%s: %s (%s)", where, cudaGetErrorName(e), cudaGetErrorString(e));
  return LIME_CUDA_ERROR;
}

// ---- per-kernel event timing (process-wide, single-threaded use) -------------------------------------------
struct ProfState {
  bool open = false;
  int capacity = 0, count = 0;
  cudaEvent_t* ev = nullptr;      // 2 per record
  const char** names = nullptr;
};
static ProfState g_prof;

ProfScope::ProfScope(const char* name, cudaStream_t s) : slot(-1), st(s) {
  if (!g_prof.open || g_prof.count >= g_prof.capacity) return;
  slot = g_prof.count++;
  g_prof.names[slot] = name;
  cudaEventRecord(g_prof.ev[2 * slot], st);
}
ProfScope::~ProfScope() {
  if (slot >= 0) cudaEventRecord(g_prof.ev[2 * slot + 1], st);
}

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline size_t align_up(size_t x) { return (x + 255) & ~(size_t)255; }
static inline int elem_size(int dtype) { return dtype == LIME_F32 ? 4 : 2; }

// Tokens per work item of the link<-history attention: a power of two in [lo, 2048] giving about three work items per
// SM (`row_blocks` items per chunk).  Every chunk of a multi-chunk history costs a set of fp32 partials and a pipeline
// refill, so long histories take long chunks.
static int pick_chunk(int64_t total_tokens, int row_blocks, int lo, int hi = 2048) {
  const int64_t target = total_tokens * row_blocks / (3 * kSMs);
  int c = lo;
  while (c < hi && c < target) c <<= 1;
  return c;
}

// Which kernels serve the XOR layers of this shape: 1 = the tensor-core kernels built for d = d_ff = 128, 2 = those
// built for d = d_ff = 256, 0 = the generic CUDA-core path.
static int tensor_core_mode(const lime_config& g, int d_ff) {
  if (link_attn_tc_supported(g.dtype, g.d, g.H, g.ell, g.phi) &&
      (hist_update_tc_supported(g.dtype, g.d, d_ff, g.H, g.ell, g.phi, g.gated_mlp) ||
       hist_update2_tc_supported(g.dtype, g.d, d_ff, g.H, g.ell, g.phi, g.gated_mlp)))
    return 1;
  if (link_attn_d256_tc_supported(g.dtype, g.d, g.H, g.ell, g.phi) &&
      hist_update_d256_tc_supported(g.dtype, g.d, d_ff, g.H, g.ell, g.phi, g.gated_mlp))
    return 2;
  return 0;
}
constexpr int kHistTile = 128;  // tokens per block of the history<-links attention

struct Workspace {
  // history rows, storage dtype
  void *S, *Q, *K, *V, *U;
  // link rows, fp32
  float *T, *QT, *KT, *VT, *AT, *UT, *LP, *LS32;
  int32_t *chunk_start, *tile_start, *chunk_user, *merge_needed;
  GroupSchedule groups;          // balanced deal of the chunk items (d = 256 kernels only)
  float *part_m, *part_s, *part_acc;
  // tensor-core path: folded link-side operands (bf16) and their row sums
  void *Q2, *K2, *G2t, *U2t, *V2t;
  float *cQ, *cK;
  float2* row_stats;   // LayerNorm {rstd, mean} of the history rows of the layer being processed
  void *That, *Ohat, *UTb;   // LN(T) [B*ell x d], merged attention rows [B*ell x H*d], GLU output [B*ell x d_ff] (bf16)
  int chunk, n_chunk_upper, n_tile_upper;
  size_t bytes;
};

static Workspace carve(const Ctx* c, void* base, int32_t B, int64_t total) {
  Workspace w;
  const lime_config& g = c->cfg;
  const size_t es = elem_size(g.dtype);
  size_t o = 0;
  char* p = static_cast<char*>(base);
  auto take = [&](size_t nbytes) { void* r = p ? p + o : nullptr; o += align_up(nbytes); return r; };
  const size_t hd = (size_t)total * g.d * es, hf = (size_t)total * c->d_ff * es;
  w.S = take(hd); w.Q = take(hd); w.K = take(hd); w.V = take(hd); w.U = take(hf);
  const size_t ld = (size_t)B * g.ell * g.d * 4, lf = (size_t)B * g.ell * c->d_ff * 4;
  w.T = (float*)take(ld); w.QT = (float*)take(ld); w.KT = (float*)take(ld); w.VT = (float*)take(ld);
  w.AT = (float*)take(ld); w.UT = (float*)take(lf); w.LP = (float*)take(ld); w.LS32 = (float*)take(ld);
  w.chunk_start = (int32_t*)take((size_t)(B + 1) * 4);
  w.tile_start = (int32_t*)take((size_t)(B + 1) * 4);
  w.merge_needed = (int32_t*)take(4);
  const bool tc_link = c->tc_mode != 0;
  // tensor-core path: at least 4 token tiles per work item, one item per 128-row block of H * ell (at d = 256 a set of
  // partials is 4 x larger and the batches served have many users, so chunks may be longer still)
  w.chunk = c->tc_mode == 2 ? pick_chunk(total, (g.H * g.ell + 127) / 128, 512, 4096)
                            : (tc_link ? pick_chunk(total, (g.H * g.ell + 127) / 128, 512) : pick_chunk(total, 1, 64));
  w.n_chunk_upper = (int)((total + w.chunk - 1) / w.chunk + B);
  w.n_tile_upper = (int)((total + kHistTile - 1) / kHistTile + B);
  w.chunk_user = (int32_t*)take((size_t)w.n_chunk_upper * 4);
  if (c->tc_mode == 2) {
    w.groups.n_groups = link_attn_d256_groups(w.n_chunk_upper, g.H, g.ell);
    w.groups.att_tile = 64;
    w.groups.group_start = (int32_t*)take((size_t)(w.groups.n_groups + 1) * 4);
    w.groups.group_items = (int32_t*)take((size_t)w.n_chunk_upper * 4);
    w.groups.scratch = (int32_t*)take((size_t)w.n_chunk_upper * 16);
  }
  const size_t rows = (size_t)w.n_chunk_upper * g.H * g.ell;
  w.part_m = (float*)take(rows * 4);
  w.part_s = (float*)take(rows * 4);
  w.part_acc = (float*)take(rows * (tc_link ? g.d : c->d_h) * 4);
  const size_t HL = (size_t)g.H * g.ell;
  w.Q2 = take((size_t)B * HL * g.d * 2); w.K2 = take((size_t)B * HL * g.d * 2);
  w.G2t = take((size_t)B * c->d_ff * HL * 2); w.U2t = take((size_t)B * c->d_ff * HL * 2);
  w.V2t = take((size_t)B * g.d * g.ell * 2);
  w.cQ = (float*)take((size_t)B * HL * 4); w.cK = (float*)take((size_t)B * HL * 4);
  w.row_stats = (float2*)take((size_t)total * 8);
  w.That = take((size_t)B * g.ell * g.d * 2); w.Ohat = take((size_t)B * g.ell * g.H * g.d * 2);
  w.UTb = take((size_t)B * g.ell * c->d_ff * 2);
  w.bytes = o;
  return w;
}

// True when the whole layer runs on the tensor-core kernels (their set-up data exists for this layer).
static bool layer_on_tensor_cores(const Ctx* c, int layer) {
  return c->tc_mode != 0 && c->WoT[layer] && c->WprepT[layer] && c->WpostT[layer] && (c->tc_mode == 1 || c->WguT[layer]);
}

// One XOR layer, tensor-core path: three link-row GEMMs around the two streaming attention kernels.
// Link-side operands of one layer's two attention directions (folded through the weights, k_link_prep.cu).
struct LinkOperands {
  const void *Q2, *K2, *G2t, *U2t, *V2t;   // G2t / U2t with tc_mode 1, V2t with tc_mode 2
  const float *cQ, *cK;
  int shared;                 // one set for every user (T^0 = L) or one per user
};

// LN(links_in) -> bf16 -> PREP GEMM: the operands of `layer` for `rows` link rows, written to the given buffers.
static lime_status make_link_operands(Ctx* c, int layer, const void* That, int64_t rows, int need_hist, void* Q2, void* K2,
                                      void* G2t, void* U2t, void* V2t, float* cQ, float* cK, cudaStream_t st) {
  const lime_config& g = c->cfg;
  LinkGemmArgs gp{};
  gp.A = That; gp.M = rows; gp.K = g.d; gp.Bt = c->WprepT[layer]; gp.ell = g.ell; gp.H = g.H;
  gp.f = c->d_ff; gp.plain_v = c->tc_mode == 2;
  gp.need_hist = need_hist; gp.Q2 = Q2; gp.K2 = K2; gp.G2t = G2t; gp.U2t = U2t; gp.V2t = V2t;
  // the row sums serve the LayerNorm folded into the d = 128 kernels; the d = 256 kernels read normalised rows
  gp.cQ = c->tc_mode == 1 ? cQ : nullptr; gp.cK = c->tc_mode == 1 ? cK : nullptr;
  gp.err = c->dev_err;
  return launch_gemm_prep(gp, st);
}

// The streaming part of one XOR layer on tensor cores: links<-history attention, GatedMLP on the link rows with its
// fused consumers (`mlp` carries the outputs wanted), and the history update.  `hist_ln`: apply LayerNorm to the rows
// read (0 when they were stored normalised by the previous layer); `out_ln`: store LayerNorm(S').
static lime_status tc_layer_core(Ctx* c, int layer, const void* hist_in, const int32_t* off, int32_t B, int64_t total,
                                 const LinkOperands& ops, void* hist_out, int hist_ln, int out_ln, LinkMlpArgs mlp,
                                 const Workspace& w, cudaStream_t st) {
  const lime_config& g = c->cfg;
  lime_status s;
  if (c->tc_mode == 2 && hist_ln && total > 0) {
    // the d = 256 kernels read LayerNorm-ed rows only: normalise the raw rows once into a scratch copy (what the
    // fused lookup + LayerNorm would have stored)
    if ((s = launch_gather_ln(g.dtype, hist_in, total, g.d, c->ln_eps, nullptr, total, w.Q, nullptr, st)) != LIME_OK) return s;
    hist_in = w.Q;
    hist_ln = 0;
  }
  // O[T]: links attend over the stored history (keys = values = history rows), chunks merged and normalised
  LinkAttnArgs la{};
  la.hist = hist_in; la.total = total; la.Q2 = ops.Q2; la.cQ = ops.cQ; la.off = off; la.chunk_start = w.chunk_start; la.chunk_user = w.chunk_user; la.B = B;
  la.group_start = w.groups.group_start; la.group_items = w.groups.group_items; la.n_groups = w.groups.n_groups;
  la.chunk = w.chunk; la.n_chunk_upper = w.n_chunk_upper; la.ell = g.ell; la.d = g.d; la.H = g.H; la.shared = ops.shared;
  la.ln = hist_ln; la.ln_eps = c->ln_eps; la.silu = g.phi == LIME_PHI_SILU; la.part_m = w.part_m; la.part_s = w.part_s; la.part_acc = w.part_acc; la.Ohat = w.Ohat;
  la.err = c->dev_err;
  // the attention kernel forms the LayerNorm statistics of every history row anyway; the history update reuses them
  const bool one_block_update = c->tc_mode == 1 && hist_update_tc_supported(g.dtype, g.d, c->d_ff, g.H, g.ell, g.phi, g.gated_mlp);
  const bool pass_stats = hist_ln && hist_out && one_block_update && total > 0;
  la.stats_out = pass_stats ? w.row_stats : nullptr;
  if ((s = c->tc_mode == 2 ? launch_link_attn_d256_tc(la, st) : launch_link_attn_tc(la, st)) != LIME_OK) return s;
  if ((s = launch_link_attn_merge_norm(w.chunk_start, w.merge_needed, B, g.ell, g.d, g.H, w.part_m, w.part_s, w.part_acc, w.Ohat, st)) != LIME_OK)
    return s;
  // T^j = GatedMLP(O[T]) with W_V folded into the gate / up weights, and what the next step needs from it
  mlp.Ohat = w.Ohat; mlp.M = (int64_t)B * g.ell; mlp.K = g.H * g.d; mlp.d = g.d; mlp.WpostT = c->WpostT[layer]; mlp.WoT = c->WoT[layer];
  mlp.ln = g.ln; mlp.ln_eps = c->ln_eps; mlp.err = c->dev_err;
  if ((s = launch_link_mlp_tc(mlp, st)) != LIME_OK) return s;
  if (hist_out && c->tc_mode == 2) {
    HistUpdate256Args hu{};
    hu.hist_in = hist_in; hu.hist_out = hist_out; hu.total = total; hu.K2 = ops.K2; hu.V2t = ops.V2t; hu.WguT = c->WguT[layer];
    hu.WoT = c->WoT[layer]; hu.off = off; hu.tile_start = w.tile_start; hu.B = B; hu.n_tile_upper = w.n_tile_upper; hu.H = g.H;
    hu.shared = ops.shared; hu.out_ln = out_ln; hu.silu = g.phi == LIME_PHI_SILU; hu.ln_eps = c->ln_eps; hu.err = c->dev_err;
    if ((s = launch_hist_update_d256_tc(hu, st)) != LIME_OK) return s;
  } else if (hist_out) {
    // history attends back over the links; scores, per-head softmax, value mix and GatedMLP in one fused kernel
    HistUpdateArgs hu{};
    hu.hist_in = hist_in; hu.hist_out = hist_out; hu.total = total; hu.K2 = ops.K2; hu.G2t = ops.G2t; hu.U2t = ops.U2t;
    hu.cK = ops.cK; hu.WoT = c->WoT[layer]; hu.off = off; hu.tile_start = w.tile_start; hu.B = B;
    hu.n_tile_upper = w.n_tile_upper; hu.ell = g.ell; hu.shared = ops.shared; hu.ln = hist_ln; hu.ln_eps = c->ln_eps;
    hu.out_ln = out_ln; hu.silu = g.phi == LIME_PHI_SILU; hu.err = c->dev_err;
    hu.stats_in = pass_stats ? w.row_stats : nullptr;
    if (one_block_update) s = launch_hist_update_tc(hu, st);
    else s = launch_hist_update2_tc(hu, g.H, st);
    if (s != LIME_OK) return s;
  }
  return LIME_OK;
}

// One XOR layer, tensor-core path, for the public layer call: link rows in and out as fp32.
static lime_status xor_layer_tc(Ctx* c, int layer, const void* hist_in, const int32_t* off, int32_t B, int64_t total,
                                const float* links_in, int links_shared, void* hist_out, float* links_out,
                                const Workspace& w, cudaStream_t st) {
  const lime_config& g = c->cfg;
  lime_status s;
  const int64_t link_rows = links_shared ? g.ell : (int64_t)B * g.ell;
  if ((s = launch_ln_rows_bf16(links_in, link_rows, g.d, g.ln, c->ln_eps, w.That, st)) != LIME_OK) return s;
  if ((s = make_link_operands(c, layer, w.That, link_rows, hist_out != nullptr, w.Q2, w.K2, w.G2t, w.U2t, w.V2t, w.cQ, w.cK, st)) != LIME_OK)
    return s;
  LinkOperands ops{w.Q2, w.K2, w.G2t, w.U2t, w.V2t, w.cQ, w.cK, links_shared};
  LinkMlpArgs mlp{};
  mlp.T_out = links_out;
  return tc_layer_core(c, layer, hist_in, off, B, total, ops, hist_out, g.ln, 0, mlp, w, st);
}

// lime_encode_user on the tensor-core path: per layer one link-side GEMM (none on the first layer when the links are
// the shared L: its operands are weights-only and were formed at lime_set_weights), then the streaming kernels.
// Between layers the history is kept LayerNorm-ed (every consumer normalises it first, Eq. 1 with App. C's LayerNorm),
// so only the first layer pays for the statistics.
static lime_status encode_user_tc(Ctx* c, const void* hist, bool hist_normalized, const int32_t* off, int32_t B, int64_t total,
                                  const float* link_ctx, void* link_states, const Workspace& w, cudaStream_t st) {
  const lime_config& g = c->cfg;
  lime_status s;
  const int64_t BL = (int64_t)B * g.ell;
  for (int j = 0; j < g.n_layers; ++j) {
    const bool last = j == g.n_layers - 1;
    LinkOperands ops;
    if (j == 0 && !link_ctx) {
      ops = LinkOperands{c->sh_Q2, c->sh_K2, c->sh_G2t, c->sh_U2t, c->sh_V2t, c->sh_cQ, c->sh_cK, 1};
    } else {
      if (j == 0 && (s = launch_ln_rows_bf16(link_ctx, BL, g.d, g.ln, c->ln_eps, w.That, st)) != LIME_OK) return s;
      if ((s = make_link_operands(c, j, w.That, BL, !last, w.Q2, w.K2, w.G2t, w.U2t, w.V2t, w.cQ, w.cK, st)) != LIME_OK) return s;
      ops = LinkOperands{w.Q2, w.K2, w.G2t, w.U2t, w.V2t, w.cQ, w.cK, 0};
    }
    LinkMlpArgs mlp{};
    mlp.LP = w.LP; mlp.lp_accumulate = j > 0;                                   // L^P = sum_j T^j  (Eq. 8)
    mlp.That_next = last ? nullptr : w.That;
    mlp.link_states = (last && !c->w.cand_Wv && c->cand_heads == 1) ? link_states : nullptr;
    s = tc_layer_core(c, j, j == 0 ? hist : w.S, off, B, total, ops, last ? nullptr : w.S, (g.ln && j == 0 && !hist_normalized) ? 1 : 0,
                      (g.ln && !last) ? 1 : 0, mlp, w, st);
    if (s != LIME_OK) return s;
  }
  return LIME_OK;
}

// One XOR layer on a carved workspace (see lime_xor_layer in lime.h for the contract).
static lime_status xor_layer_impl(Ctx* c, int layer, const void* hist_in, const int32_t* off, int32_t B,
                                  int64_t total, const float* links_in, int links_shared, void* hist_out,
                                  float* links_out, const Workspace& w, bool schedules_ready, int hist_ln, cudaStream_t st) {
  // hist_ln: LayerNorm the history rows read (config.ln, except on the first layer of an encode whose rows arrive
  // normalised).  The tensor-core branch is only taken by the single-layer call, whose input is never normalised.
  const lime_config& g = c->cfg;
  lime_status s;
  if (!schedules_ready) {
    if ((s = launch_layer_schedules(off, B, w.chunk, w.chunk_start, kHistTile, w.tile_start, w.chunk_user, w.merge_needed, w.groups, st)) != LIME_OK) return s;
  }
  if (layer_on_tensor_cores(c, layer))
    return xor_layer_tc(c, layer, hist_in, off, B, total, links_in, links_shared, hist_out, links_out, w, st);

  // ---- generic path on CUDA cores (fp32 storage, other shapes, SiLU attention, no GatedMLP) ----
  const int64_t link_rows = links_shared ? g.ell : (int64_t)B * g.ell;

  // link rows: Q[T], K[T], V[T] = LN(T) W_{Q,K,V}
  LinearArgs la{};
  la.X = links_in; la.x_dtype = LIME_F32; la.M = link_rows; la.K = g.d; la.N = g.d;
  la.W[0] = c->w.Wq[layer]; la.W[1] = c->w.Wk[layer]; la.W[2] = c->w.Wv[layer]; la.w_dtype = g.dtype;
  la.Y[0] = w.QT; la.Y[1] = w.KT; la.Y[2] = w.VT; la.y_dtype = LIME_F32; la.n_out = 3;
  la.ln = g.ln; la.ln_eps = c->ln_eps;
  if ((s = launch_linear_simt(la, st)) != LIME_OK) return s;

  // history rows: K[S], V[S] (and Q[S] when the history is updated) = LN(S) W
  LinearArgs lh{};
  lh.X = hist_in; lh.x_dtype = g.dtype; lh.M = total; lh.K = g.d; lh.N = g.d; lh.w_dtype = g.dtype; lh.y_dtype = g.dtype;
  lh.W[0] = c->w.Wk[layer]; lh.W[1] = c->w.Wv[layer]; lh.W[2] = c->w.Wq[layer];
  lh.Y[0] = w.K; lh.Y[1] = w.V; lh.Y[2] = w.Q; lh.n_out = hist_out ? 3 : 2;
  lh.ln = hist_ln; lh.ln_eps = c->ln_eps;
  if ((s = launch_linear_simt(lh, st)) != LIME_OK) return s;

  // O[T] = phi(Q[T] K[S]^T) V[S]
  AttnLinkArgs al{};
  al.QT = w.QT; al.qt_user_stride = links_shared ? 0 : (int64_t)g.ell * g.d;
  al.KS = w.K; al.VS = w.V; al.s_dtype = g.dtype; al.off = off; al.B = B; al.total = total;
  al.ell = g.ell; al.d = g.d; al.H = g.H; al.phi = g.phi; al.scale = c->attn_scale;
  al.chunk = w.chunk; al.chunk_start = w.chunk_start; al.n_chunk_upper = w.n_chunk_upper;
  al.part_m = w.part_m; al.part_s = w.part_s; al.part_acc = w.part_acc; al.AT = w.AT;
  if ((s = launch_attn_link_simt(al, st)) != LIME_OK) return s;
  if ((s = launch_attn_link_merge(al, st)) != LIME_OK) return s;

  // links_out = GatedMLP(O[T])
  const int64_t BL = (int64_t)B * g.ell;
  if (g.gated_mlp) {
    LinearArgs lg{};
    lg.X = w.AT; lg.x_dtype = LIME_F32; lg.M = BL; lg.K = g.d; lg.N = c->d_ff; lg.w_dtype = g.dtype;
    lg.W[0] = c->w.Wg[layer]; lg.W[1] = c->w.Wu[layer]; lg.Y[0] = w.UT; lg.y_dtype = LIME_F32; lg.n_out = 1; lg.glu = 1;
    if ((s = launch_linear_simt(lg, st)) != LIME_OK) return s;
    LinearArgs lo{};
    lo.X = w.UT; lo.x_dtype = LIME_F32; lo.M = BL; lo.K = c->d_ff; lo.N = g.d; lo.w_dtype = g.dtype;
    lo.W[0] = c->w.Wo[layer]; lo.Y[0] = links_out; lo.y_dtype = LIME_F32; lo.n_out = 1;
    if ((s = launch_linear_simt(lo, st)) != LIME_OK) return s;
  } else {
    if ((s = launch_axpy(w.AT, links_out, BL * g.d, 1, st)) != LIME_OK) return s;
  }

  if (hist_out) {
    // O[S] = phi(Q[S] K[T]^T) V[T], written over Q[S]; then hist_out = GatedMLP(O[S])
    AttnHistArgs ah{};
    ah.QS = w.Q; ah.AS = w.Q; ah.s_dtype = g.dtype; ah.KT = w.KT; ah.VT = w.VT;
    ah.t_user_stride = links_shared ? 0 : (int64_t)g.ell * g.d;
    ah.off = off; ah.B = B; ah.total = total; ah.ell = g.ell; ah.d = g.d; ah.H = g.H; ah.phi = g.phi;
    ah.scale = c->attn_scale; ah.tile = kHistTile; ah.tile_start = w.tile_start; ah.n_tile_upper = w.n_tile_upper;
    if ((s = launch_attn_hist_simt(ah, st)) != LIME_OK) return s;
    if (g.gated_mlp) {
      LinearArgs lg{};
      lg.X = w.Q; lg.x_dtype = g.dtype; lg.M = total; lg.K = g.d; lg.N = c->d_ff; lg.w_dtype = g.dtype;
      lg.W[0] = c->w.Wg[layer]; lg.W[1] = c->w.Wu[layer]; lg.Y[0] = w.U; lg.y_dtype = g.dtype; lg.n_out = 1; lg.glu = 1;
      if ((s = launch_linear_simt(lg, st)) != LIME_OK) return s;
      LinearArgs lo{};
      lo.X = w.U; lo.x_dtype = g.dtype; lo.M = total; lo.K = c->d_ff; lo.N = g.d; lo.w_dtype = g.dtype;
      lo.W[0] = c->w.Wo[layer]; lo.Y[0] = hist_out; lo.y_dtype = g.dtype; lo.n_out = 1;
      if ((s = launch_linear_simt(lo, st)) != LIME_OK) return s;
    } else if (total > 0) {
      LIME_CUDA(cudaMemcpyAsync(hist_out, w.Q, (size_t)total * g.d * elem_size(g.dtype), cudaMemcpyDeviceToDevice, st));
    }
  }
  return LIME_OK;
}

static lime_status check_layer_weights(const Ctx* c, int layer) {
  if (c->cfg.gated_mlp && (!c->w.Wg[layer] || !c->w.Wu[layer] || !c->w.Wo[layer])) return LIME_INVALID_ARG;
  return LIME_OK;
}

}  // namespace lime

using namespace lime;

extern "C" {

const char* lime_last_cuda_error(void) { return g_err; }
const char* lime_version(void) { return "lime-b200 0.1 sm_100a"; }

lime_status lime_profile_start(int32_t capacity) {
  if (capacity <= 0 || g_prof.open) return LIME_INVALID_ARG;
  g_prof.ev = new (std::nothrow) cudaEvent_t[2 * (size_t)capacity];
  g_prof.names = new (std::nothrow) const char*[capacity];
  if (!g_prof.ev || !g_prof.names) return LIME_INVALID_ARG;
  for (int i = 0; i < 2 * capacity; ++i) {
    cudaError_t e = cudaEventCreate(&g_prof.ev[i]);
    if (e != cudaSuccess) {
      for (int j = 0; j < i; ++j) cudaEventDestroy(g_prof.ev[j]);
      delete[] g_prof.ev; delete[] g_prof.names;
      g_prof = ProfState();
      return cuda_fail(e, "lime_profile_start");
    }
  }
  g_prof.capacity = capacity; g_prof.count = 0; g_prof.open = true;
  return LIME_OK;
}

lime_status lime_profile_stop(char* names, size_t names_bytes, float* ms, int32_t ms_capacity, int32_t* count) {
  if (!g_prof.open || !count) return LIME_INVALID_ARG;
  g_prof.open = false;
  lime_status ret = LIME_OK;
  const int n = g_prof.count < ms_capacity ? g_prof.count : ms_capacity;
  size_t pos = 0;
  if (names && names_bytes) names[0] = 0;
  for (int i = 0; i < n; ++i) {
    cudaError_t e = cudaEventSynchronize(g_prof.ev[2 * i + 1]);
    float t = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&t, g_prof.ev[2 * i], g_prof.ev[2 * i + 1]);
    if (e != cudaSuccess) ret = cuda_fail(e, "lime_profile_stop");
    if (ms) ms[i] = t;
    if (names) {
      const size_t len = strlen(g_prof.names[i]);
      if (pos + len + 2 <= names_bytes) {
        memcpy(names + pos, g_prof.names[i], len);
        pos += len;
        names[pos++] = '\n';
        names[pos] = 0;
      }
    }
  }
  *count = g_prof.count;
  for (int i = 0; i < 2 * g_prof.capacity; ++i) cudaEventDestroy(g_prof.ev[i]);
  delete[] g_prof.ev; delete[] g_prof.names;
  g_prof = ProfState();
  return ret;
}

lime_status lime_create(const lime_config* cfg, lime_ctx** out) {
  if (!cfg || !out) return LIME_INVALID_ARG;
  *out = nullptr;
  const lime_config& g = *cfg;
  if (g.d <= 0 || g.H <= 0 || g.ell <= 0 || g.n_layers <= 0 || g.d_ff < 0) return LIME_INVALID_ARG;
  if (g.dtype != LIME_F32 && g.dtype != LIME_BF16) return LIME_INVALID_ARG;
  if (g.phi != LIME_PHI_SOFTMAX && g.phi != LIME_PHI_SILU) return LIME_INVALID_ARG;
  if (g.attn_scale < 0.f || g.cand_scale < 0.f || g.ln_eps < 0.f) return LIME_INVALID_ARG;
  if (g.cand_heads != 0 && g.cand_heads != 1 && g.cand_heads != g.H) return LIME_INVALID_ARG;
  const int cand_heads = g.cand_heads == g.H ? g.H : 1;
  if (cand_heads * g.ell > 256) return LIME_UNSUPPORTED_SHAPE;
  const int d_ff = g.d_ff ? g.d_ff : g.d;
  if (g.d % 8 || d_ff % 8 || g.d % g.H || g.d / g.H > 128 || g.ell > 256 || g.n_layers > LIME_MAX_LAYERS ||
      g.d > 1024 || d_ff > 1024)
    return LIME_UNSUPPORTED_SHAPE;
  // a user's K[T], V[T] (fp32) must fit in one SM's shared memory for the history<-links attention
  if (sizeof(float) * ((size_t)2 * g.ell * (g.d + 1) + 4 * (size_t)g.d) > 200 * 1024) return LIME_UNSUPPORTED_SHAPE;
  Ctx* c = new (std::nothrow) Ctx();
  if (!c) return LIME_INVALID_ARG;
  c->cfg = g;
  memset(&c->w, 0, sizeof(c->w));
  c->have_weights = false;
  c->d_ff = d_ff;
  c->d_h = g.d / g.H;
  c->attn_scale = g.attn_scale > 0.f ? g.attn_scale : 1.0f / sqrtf((float)c->d_h);
  c->cand_heads = cand_heads;
  c->ell_c = cand_heads * g.ell;
  // per-head scores are scaled like any head of Eq. 1; the single-row form by the full width
  c->cand_scale = g.cand_scale > 0.f ? g.cand_scale : 1.0f / sqrtf((float)(cand_heads > 1 ? c->d_h : g.d));
  c->ln_eps = g.ln_eps > 0.f ? g.ln_eps : 1e-5f;
  c->keff = nullptr; c->keff_hl = nullptr; c->links32 = nullptr; c->dev_err = nullptr;
  c->have_head = c->have_ctx_mlp = false; c->ctx_dc = 0;
  c->head_W1bT = nullptr; c->head_W1aT = nullptr; c->head_w2 = nullptr; c->ctx_first = nullptr;
  c->tc_mode = tensor_core_mode(g, d_ff);
  for (int j = 0; j < LIME_MAX_LAYERS; ++j) c->WoT[j] = c->WprepT[j] = c->WpostT[j] = c->WguT[j] = nullptr;
  c->sh_That = c->sh_Q2 = c->sh_K2 = c->sh_G2t = c->sh_U2t = c->sh_V2t = nullptr; c->sh_cQ = c->sh_cK = nullptr;
  cudaError_t e = cudaGetDevice(&c->device);
  if (e == cudaSuccess) e = cudaMalloc(&c->keff, sizeof(float) * 2 * (size_t)c->ell_c * g.d);
  if (e == cudaSuccess) e = cudaMalloc(&c->keff_hl, 2 * (size_t)2 * c->ell_c * g.d);
  if (e == cudaSuccess) e = cudaMalloc(&c->links32, sizeof(float) * (size_t)g.ell * g.d);
  if (e == cudaSuccess) e = cudaMalloc(&c->dev_err, sizeof(int));
  if (e == cudaSuccess) e = cudaMemset(c->dev_err, 0, sizeof(int));
  if (e != cudaSuccess) {
    if (c->keff) cudaFree(c->keff);
    if (c->keff_hl) cudaFree(c->keff_hl);
    if (c->links32) cudaFree(c->links32);
    if (c->dev_err) cudaFree(c->dev_err);
    delete c;
    return cuda_fail(e, "lime_create");
  }
  *out = reinterpret_cast<lime_ctx*>(c);
  return LIME_OK;
}

lime_status lime_destroy(lime_ctx* ctx) {
  if (!ctx) return LIME_OK;
  Ctx* c = reinterpret_cast<Ctx*>(ctx);
  cudaFree(c->keff);
  cudaFree(c->keff_hl);
  cudaFree(c->links32);
  cudaFree(c->dev_err);
  for (int j = 0; j < LIME_MAX_LAYERS; ++j) { cudaFree(c->WoT[j]); cudaFree(c->WprepT[j]); cudaFree(c->WpostT[j]); cudaFree(c->WguT[j]); }
  cudaFree(c->sh_That); cudaFree(c->sh_Q2); cudaFree(c->sh_K2); cudaFree(c->sh_G2t); cudaFree(c->sh_U2t); cudaFree(c->sh_V2t);
  cudaFree(c->sh_cQ); cudaFree(c->sh_cK);
  cudaFree(c->head_W1bT); cudaFree(c->head_W1aT); cudaFree(c->head_w2); cudaFree(c->ctx_first);
  delete c;
  return LIME_OK;
}

lime_status lime_set_weights(lime_ctx* ctx, const lime_weights* w, void* stream) {
  if (!ctx || !w || !w->links) return LIME_INVALID_ARG;
  Ctx* c = reinterpret_cast<Ctx*>(ctx);
  const lime_config& g = c->cfg;
  if (!aligned16(w->links)) return LIME_INVALID_ARG;
  for (int j = 0; j < g.n_layers; ++j) {
    const void* ps[6] = {w->Wq[j], w->Wk[j], w->Wv[j], w->Wg[j], w->Wu[j], w->Wo[j]};
    for (const void* p : ps) if (!aligned16(p)) return LIME_INVALID_ARG;
    if (g.gated_mlp && (!w->Wg[j] || !w->Wu[j] || !w->Wo[j])) return LIME_INVALID_ARG;
  }
  if (!aligned16(w->cand_Wq) || !aligned16(w->cand_Wk) || !aligned16(w->cand_Wv)) return LIME_INVALID_ARG;
  c->w = *w;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  lime_status s = launch_widen(w->links, g.dtype, c->links32, (int64_t)g.ell * g.d, st);
  if (s != LIME_OK) return s;
  s = launch_keff(g.dtype, w->links, w->cand_Wk, w->cand_Wq, g.ell, g.d, c->cand_heads, c->cand_scale, c->keff, st);
  if (s != LIME_OK) return s;
  if (precompute_tc_supported(g.dtype, g.d, c->ell_c, g.ell) &&
      (s = launch_keff_split(c->keff, c->ell_c, g.d, c->keff_hl, st)) != LIME_OK)
    return s;
  // tensor-core path: per layer, W_o as a K-major B operand ([d x d_ff], contraction index contiguous) and the
  // weight-only products that fold the history-side projections into the link rows
  if (c->tc_mode != 0) {
    const bool plain_v = c->tc_mode == 2;
    const size_t prep_rows = 2 * (size_t)g.H * g.d + (plain_v ? (size_t)g.d : 2 * (size_t)g.H * c->d_ff);
    auto need = [](void** p, size_t bytes) -> cudaError_t { return *p ? cudaSuccess : cudaMalloc(p, bytes); };
    for (int j = 0; j < g.n_layers; ++j) {
      LIME_CUDA(need(&c->WoT[j], (size_t)g.d * c->d_ff * 2));
      LIME_CUDA(need(&c->WprepT[j], prep_rows * g.d * 2));
      LIME_CUDA(need(&c->WpostT[j], (size_t)2 * c->d_ff * g.H * g.d * 2));
      if ((s = launch_transpose_bf16(w->Wo[j], c->d_ff, g.d, c->WoT[j], st)) != LIME_OK) return s;
      if (plain_v) {
        // [W_g | W_u]^T [2f x d]: the history update applies the GatedMLP weights as they stand
        LIME_CUDA(need(&c->WguT[j], (size_t)2 * c->d_ff * g.d * 2));
        if ((s = launch_transpose_bf16(w->Wg[j], g.d, c->d_ff, c->WguT[j], st)) != LIME_OK) return s;
        if ((s = launch_transpose_bf16(w->Wu[j], g.d, c->d_ff, (char*)c->WguT[j] + (size_t)c->d_ff * g.d * 2, st)) != LIME_OK) return s;
      }
      if ((s = launch_fold_weights(w->Wq[j], w->Wk[j], w->Wv[j], w->Wg[j], w->Wu[j], g.d, g.H, c->d_ff,
                                   // softmax: scores leave the fold scaled and in the log2 domain; SiLU(s) takes the raw scores
                                   g.phi == LIME_PHI_SILU ? 1.0f : c->attn_scale * 1.4426950408889634f, plain_v ? 1 : 0,
                                   c->WprepT[j], c->WpostT[j], st)) != LIME_OK)
        return s;
    }
    // first-layer operands for the shared links T^0 = L: LN(L) through the PREP GEMM, once
    const size_t HL = (size_t)g.H * g.ell;
    LIME_CUDA(need(&c->sh_That, (size_t)g.ell * g.d * 2));
    LIME_CUDA(need(&c->sh_Q2, HL * g.d * 2));
    LIME_CUDA(need(&c->sh_K2, HL * g.d * 2));
    if (plain_v) {
      LIME_CUDA(need(&c->sh_V2t, (size_t)g.d * g.ell * 2));
    } else {
      LIME_CUDA(need(&c->sh_G2t, (size_t)c->d_ff * HL * 2));
      LIME_CUDA(need(&c->sh_U2t, (size_t)c->d_ff * HL * 2));
    }
    LIME_CUDA(need((void**)&c->sh_cQ, HL * 4));
    LIME_CUDA(need((void**)&c->sh_cK, HL * 4));
    if ((s = launch_ln_rows_bf16(c->links32, g.ell, g.d, g.ln, c->ln_eps, c->sh_That, st)) != LIME_OK) return s;
    if ((s = make_link_operands(c, 0, c->sh_That, g.ell, g.n_layers > 1, c->sh_Q2, c->sh_K2, c->sh_G2t, c->sh_U2t, c->sh_V2t,
                                c->sh_cQ, c->sh_cK, st)) != LIME_OK)
      return s;
  }
  c->have_weights = true;
  return LIME_OK;
}

size_t lime_workspace_bytes(const lime_ctx* ctx, int32_t B, int64_t total_tokens) {
  if (!ctx || B < 0 || total_tokens < 0 || total_tokens > 0x7fffffffLL) return 0;
  const Ctx* c = reinterpret_cast<const Ctx*>(ctx);
  return carve(c, nullptr, B, total_tokens).bytes + 256;
}

lime_status lime_lengths_to_offsets(lime_ctx* ctx, const int32_t* len, int32_t B, int32_t* off, void* stream) {
  if (!ctx || !off || B < 0 || (B > 0 && !len)) return LIME_INVALID_ARG;
  return launch_offsets(len, B, off, static_cast<cudaStream_t>(stream));
}

lime_status lime_gather_history(lime_ctx* ctx, const void* table, int64_t V, const int32_t* ids, int64_t total_tokens,
                                void* out, int32_t* dev_flag, void* stream) {
  if (!ctx || total_tokens < 0 || V < 0) return LIME_INVALID_ARG;
  if (total_tokens == 0) return LIME_OK;
  if (!table || !ids || !out || !aligned16(table) || !aligned16(out)) return LIME_INVALID_ARG;
  const Ctx* c = reinterpret_cast<const Ctx*>(ctx);
  return launch_gather(c->cfg.dtype, table, V, c->cfg.d, ids, total_tokens, out, dev_flag,
                       static_cast<cudaStream_t>(stream));
}

lime_status lime_gather_history_normalized(lime_ctx* ctx, const void* table, int64_t V, const int32_t* ids,
                                           int64_t total_tokens, void* out, int32_t* dev_flag, void* stream) {
  if (!ctx || total_tokens < 0 || V < 0) return LIME_INVALID_ARG;
  if (total_tokens == 0) return LIME_OK;
  if (!table || !ids || !out || !aligned16(table) || !aligned16(out)) return LIME_INVALID_ARG;
  const Ctx* c = reinterpret_cast<const Ctx*>(ctx);
  if (!c->cfg.ln)
    return launch_gather(c->cfg.dtype, table, V, c->cfg.d, ids, total_tokens, out, dev_flag, static_cast<cudaStream_t>(stream));
  return launch_gather_ln(c->cfg.dtype, table, V, c->cfg.d, c->ln_eps, ids, total_tokens, out, dev_flag,
                          static_cast<cudaStream_t>(stream));
}

lime_status lime_precompute_candidate_links(lime_ctx* ctx, const void* cand_emb, int64_t M, void* out_w, void* stream) {
  if (!ctx || M < 0) return LIME_INVALID_ARG;
  Ctx* c = reinterpret_cast<Ctx*>(ctx);
  if (!c->have_weights) return LIME_NOT_READY;
  if (M == 0) return LIME_OK;
  if (!cand_emb || !out_w || !aligned16(cand_emb) || !aligned16(out_w)) return LIME_INVALID_ARG;
  if (precompute_tc_supported(c->cfg.dtype, c->cfg.d, c->ell_c, c->cfg.ell))
    return launch_precompute_tc(cand_emb, M, c->cfg.d, c->ell_c, c->cfg.ell, c->keff_hl, out_w, c->dev_err,
                                static_cast<cudaStream_t>(stream));
  return launch_precompute(c->cfg.dtype, cand_emb, M, c->cfg.d, c->ell_c, c->cfg.ell, c->keff, out_w,
                           static_cast<cudaStream_t>(stream));
}

lime_status lime_xor_layer(lime_ctx* ctx, int32_t layer, const void* hist_in, const int32_t* off, int32_t B,
                           int64_t total_tokens, const float* links_in, int32_t links_shared, void* hist_out,
                           float* links_out, void* ws, size_t ws_bytes, void* stream) {
  if (!ctx || B < 0 || total_tokens < 0 || total_tokens > 0x7fffffffLL) return LIME_INVALID_ARG;
  Ctx* c = reinterpret_cast<Ctx*>(ctx);
  if (!c->have_weights) return LIME_NOT_READY;
  if (layer < 0 || layer >= c->cfg.n_layers) return LIME_INVALID_ARG;
  if (B == 0) return LIME_OK;
  if (!off || !links_in || !links_out || !ws || (total_tokens > 0 && !hist_in)) return LIME_INVALID_ARG;
  if (!aligned16(hist_in) || !aligned16(hist_out) || !aligned16(links_in) || !aligned16(links_out)) return LIME_INVALID_ARG;
  if (check_layer_weights(c, layer) != LIME_OK) return LIME_INVALID_ARG;
  char* base = reinterpret_cast<char*>(align_up(reinterpret_cast<uintptr_t>(ws)));
  const size_t pad = base - static_cast<char*>(ws);
  Workspace w = carve(c, base, B, total_tokens);
  if (w.bytes + pad > ws_bytes) return LIME_WORKSPACE_TOO_SMALL;
  return xor_layer_impl(c, layer, hist_in, off, B, total_tokens, links_in, links_shared, hist_out, links_out, w, false,
                        c->cfg.ln, static_cast<cudaStream_t>(stream));
}

static lime_status encode_user_impl(lime_ctx* ctx, const void* hist, bool hist_normalized, const int32_t* off, int32_t B,
                                    int64_t total_tokens, const float* link_ctx, void* link_states, void* ws, size_t ws_bytes,
                                    void* stream) {
  if (!ctx || B < 0 || total_tokens < 0 || total_tokens > 0x7fffffffLL) return LIME_INVALID_ARG;
  Ctx* c = reinterpret_cast<Ctx*>(ctx);
  if (!c->have_weights) return LIME_NOT_READY;
  if (B == 0) return LIME_OK;
  if (!off || !link_states || !ws || (total_tokens > 0 && !hist)) return LIME_INVALID_ARG;
  if (!aligned16(hist) || !aligned16(link_ctx) || !aligned16(link_states)) return LIME_INVALID_ARG;
  const lime_config& g = c->cfg;
  for (int j = 0; j < g.n_layers; ++j)
    if (check_layer_weights(c, j) != LIME_OK) return LIME_INVALID_ARG;
  char* base = reinterpret_cast<char*>(align_up(reinterpret_cast<uintptr_t>(ws)));
  const size_t pad = base - static_cast<char*>(ws);
  Workspace w = carve(c, base, B, total_tokens);
  if (w.bytes + pad > ws_bytes) return LIME_WORKSPACE_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  lime_status s;
  if ((s = launch_layer_schedules(off, B, w.chunk, w.chunk_start, kHistTile, w.tile_start, w.chunk_user, w.merge_needed, w.groups, st)) != LIME_OK) return s;
  const int64_t BLd = (int64_t)B * g.ell * g.d;
  if (layer_on_tensor_cores(c, 0)) {
    if ((s = encode_user_tc(c, hist, hist_normalized, off, B, total_tokens, link_ctx, link_states, w, st)) != LIME_OK) return s;
    if (!c->w.cand_Wv && c->cand_heads == 1) return LIME_OK;        // the last layer's kernel wrote the link states
  } else {
    for (int j = 0; j < g.n_layers; ++j) {
      const bool last = j == g.n_layers - 1;
      const float* lin = j == 0 ? (link_ctx ? link_ctx : c->links32) : w.T;
      const int shared = (j == 0 && !link_ctx) ? 1 : 0;
      s = xor_layer_impl(c, j, j == 0 ? hist : w.S, off, B, total_tokens, lin, shared, last ? nullptr : w.S, w.T, w, true,
                         (g.ln && !(j == 0 && hist_normalized)) ? 1 : 0, st);
      if (s != LIME_OK) return s;
      if ((s = launch_axpy(w.T, w.LP, BLd, j == 0, st)) != LIME_OK) return s;   // L^P = sum_j T^j  (Eq. 8)
    }
  }
  // link states = L^P W_V^c (Eq. 4's values), stored as the run's dtype
  const float* src = w.LP;
  if (c->w.cand_Wv) {
    LinearArgs lv{};
    lv.X = w.LP; lv.x_dtype = LIME_F32; lv.M = (int64_t)B * g.ell; lv.K = g.d; lv.N = g.d; lv.w_dtype = g.dtype;
    lv.W[0] = c->w.cand_Wv; lv.Y[0] = w.LS32; lv.y_dtype = LIME_F32; lv.n_out = 1;
    if ((s = launch_linear_simt(lv, st)) != LIME_OK) return s;
    src = w.LS32;
  }
  if (c->cand_heads > 1) return launch_expand_heads(src, (int64_t)B * g.ell, g.ell, g.d, c->cand_heads, link_states, g.dtype, st);
  return launch_cast_rows(src, BLd, link_states, g.dtype, st);
}

lime_status lime_encode_user(lime_ctx* ctx, const void* hist, const int32_t* off, int32_t B, int64_t total_tokens,
                             const float* link_ctx, void* link_states, void* ws, size_t ws_bytes, void* stream) {
  return encode_user_impl(ctx, hist, false, off, B, total_tokens, link_ctx, link_states, ws, ws_bytes, stream);
}

lime_status lime_encode_user_normalized(lime_ctx* ctx, const void* hist_normalized, const int32_t* off, int32_t B,
                                        int64_t total_tokens, const float* link_ctx, void* link_states, void* ws,
                                        size_t ws_bytes, void* stream) {
  return encode_user_impl(ctx, hist_normalized, true, off, B, total_tokens, link_ctx, link_states, ws, ws_bytes, stream);
}

lime_status lime_score_candidates(lime_ctx* ctx, const void* link_states, int32_t B, const void* cand_w,
                                  const void* cand_emb, const int32_t* cand_off, int32_t C, int64_t total_cands,
                                  const int32_t* cand_ids, int64_t corpus_rows, int32_t* dev_flag, float* logits,
                                  void* stream) {
  if (!ctx || B < 0 || C < 0 || total_cands < 0 || total_cands > 0x7fffffffLL) return LIME_INVALID_ARG;
  if (cand_ids && (corpus_rows <= 0 || corpus_rows > 0x7fffffffLL)) return LIME_INVALID_ARG;
  if (!cand_off && total_cands != (int64_t)B * C) return LIME_INVALID_ARG;
  if (B == 0 || total_cands == 0) return LIME_OK;
  if (!link_states || !cand_w || !cand_emb || !logits) return LIME_INVALID_ARG;
  if (!aligned16(link_states) || !aligned16(cand_w) || !aligned16(cand_emb)) return LIME_INVALID_ARG;
  Ctx* c = reinterpret_cast<Ctx*>(ctx);
  ScoreArgs a{};
  a.LS = link_states; a.W = cand_w; a.T = cand_emb; a.dtype = c->cfg.dtype; a.B = B; a.ell = c->ell_c; a.d = c->cfg.d;
  a.cand_off = cand_off; a.C = C; a.total = total_cands; a.cand_ids = cand_ids; a.logits = logits;
  a.corpus_rows = cand_ids ? corpus_rows : 0; a.dev_flag = cand_ids ? dev_flag : nullptr;
  if (score_tc_supported(a)) return launch_score_tc(a, c->dev_err, static_cast<cudaStream_t>(stream));
  if (score_gather_tc_supported(a)) return launch_score_gather_tc(a, c->dev_err, static_cast<cudaStream_t>(stream));
  return launch_score_simt(a, static_cast<cudaStream_t>(stream));
}

// ---- feed-forward networks (Eq. 2; Sec. 3.3 interaction network) ----------------------------------------------------
static bool ffn_valid(const lime_ffn* f, int min_hidden) {
  if (!f || f->n_hidden < min_hidden || f->n_hidden > LIME_FFN_MAX_HIDDEN) return false;
  for (int i = 0; i < f->n_hidden; ++i)
    if (f->widths[i] < 1 || f->widths[i] > 1024) return false;
  for (int i = 0; i <= f->n_hidden; ++i)
    if (!f->W[i] || !aligned16(f->W[i])) return false;
  return true;
}
// layers after the first: layer i maps widths[i-1] to widths[i] (the last one to `out_last`)
static FfnArgs ffn_tail(const lime_ffn& f, int out_last) {
  FfnArgs a{};
  a.n_layers = f.n_hidden;
  for (int i = 1; i <= f.n_hidden; ++i) {
    a.in_w[i - 1] = f.widths[i - 1];
    a.out_w[i - 1] = i < f.n_hidden ? f.widths[i] : out_last;
    a.W[i - 1] = f.W[i];
    a.b[i - 1] = f.b[i];
  }
  return a;
}

lime_status lime_set_context_mlp(lime_ctx* ctx, int32_t d_c, const lime_ffn* mlp, void* stream) {
  if (!ctx || d_c < 1 || d_c > 4096 || !ffn_valid(mlp, 0)) return LIME_INVALID_ARG;
  Ctx* c = reinterpret_cast<Ctx*>(ctx);
  if (!c->have_weights) return LIME_NOT_READY;
  const lime_config& g = c->cfg;
  const int w0 = mlp->n_hidden > 0 ? mlp->widths[0] : g.d;
  cudaFree(c->ctx_first);
  c->ctx_first = nullptr;
  c->have_ctx_mlp = false;
  LIME_CUDA(cudaMalloc(&c->ctx_first, sizeof(float) * (size_t)g.ell * w0));
  // weights-only part of the first layer: (L W_0[:d]) + b_0
  lime_status s = launch_rows_times_w(c->w.links, g.dtype, g.ell, g.d, mlp->W[0], g.dtype, w0, w0, mlp->b[0], c->ctx_first, nullptr,
                                      1, "k_ctx_first", static_cast<cudaStream_t>(stream));
  if (s != LIME_OK) return s;
  c->ctx_mlp = *mlp;
  c->ctx_dc = d_c;
  c->have_ctx_mlp = true;
  return LIME_OK;
}

lime_status lime_contextualize_links(lime_ctx* ctx, const void* user_ctx, int32_t B, float* link_ctx, void* stream) {
  if (!ctx || B < 0) return LIME_INVALID_ARG;
  Ctx* c = reinterpret_cast<Ctx*>(ctx);
  if (!c->have_ctx_mlp) return LIME_NOT_READY;
  if (B == 0) return LIME_OK;
  if (!user_ctx || !link_ctx || !aligned16(link_ctx)) return LIME_INVALID_ARG;
  const lime_config& g = c->cfg;
  const lime_ffn& f = c->ctx_mlp;
  const int w0 = f.n_hidden > 0 ? f.widths[0] : g.d;
  const char* W0c = static_cast<const char*>(f.W[0]) + (size_t)g.d * w0 * elem_size(g.dtype);     // rows d.. act on E^C
  return launch_link_ctx_mlp(g.dtype, c->ctx_first, user_ctx, c->ctx_dc, W0c, w0, B, g.ell, ffn_tail(f, g.d), link_ctx,
                             static_cast<cudaStream_t>(stream));
}

lime_status lime_set_head(lime_ctx* ctx, const lime_ffn* head, void* stream) {
  if (!ctx || !ffn_valid(head, 1)) return LIME_INVALID_ARG;
  Ctx* c = reinterpret_cast<Ctx*>(ctx);
  const lime_config& g = c->cfg;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int w0 = head->widths[0], w_last = head->widths[head->n_hidden - 1];
  cudaFree(c->head_W1bT); cudaFree(c->head_W1aT); cudaFree(c->head_w2);
  c->head_W1bT = nullptr; c->head_W1aT = nullptr; c->head_w2 = nullptr;
  c->have_head = false;
  LIME_CUDA(cudaMalloc(&c->head_w2, sizeof(float) * (size_t)w_last));
  lime_status s = launch_widen(head->W[head->n_hidden], g.dtype, c->head_w2, w_last, st);
  if (s != LIME_OK) return s;
  if (g.dtype == LIME_BF16) {
    // the T half of the first layer as a K-major B operand [w0 x d]
    LIME_CUDA(cudaMalloc(&c->head_W1bT, (size_t)w0 * g.d * 2));
    const char* W0t = static_cast<const char*>(head->W[0]) + (size_t)g.d * w0 * 2;
    if ((s = launch_transpose_bf16(W0t, g.d, w0, c->head_W1bT, st)) != LIME_OK) return s;
    LIME_CUDA(cudaMalloc(&c->head_W1aT, (size_t)w0 * g.d * 2));
    if ((s = launch_transpose_bf16(head->W[0], g.d, w0, c->head_W1aT, st)) != LIME_OK) return s;
  }
  c->head = *head;
  c->have_head = true;
  return LIME_OK;
}

size_t lime_head_workspace_bytes(const lime_ctx* ctx, int32_t B) {
  if (!ctx || B < 0) return 0;
  const Ctx* c = reinterpret_cast<const Ctx*>(ctx);
  if (!c->have_head) return 0;
  const size_t n = (size_t)B * c->ell_c * c->head.widths[0];
  return align_up(n * 4) + align_up(n * 2) + 256;
}

lime_status lime_score_candidates_head(lime_ctx* ctx, const void* link_states, int32_t B, const void* cand_w,
                                       const void* cand_emb, const int32_t* cand_off, int32_t C, int64_t total_cands,
                                       const int32_t* cand_ids, int64_t corpus_rows, int32_t* dev_flag, float* logits,
                                       void* ws, size_t ws_bytes, void* stream) {
  if (!ctx || B < 0 || C < 0 || total_cands < 0 || total_cands > 0x7fffffffLL) return LIME_INVALID_ARG;
  if (cand_ids && (corpus_rows <= 0 || corpus_rows > 0x7fffffffLL)) return LIME_INVALID_ARG;
  if (!cand_off && total_cands != (int64_t)B * C) return LIME_INVALID_ARG;
  Ctx* c = reinterpret_cast<Ctx*>(ctx);
  if (!c->have_head) return LIME_NOT_READY;
  if (B == 0 || total_cands == 0) return LIME_OK;
  if (!link_states || !cand_w || !cand_emb || !logits || !ws) return LIME_INVALID_ARG;
  if (!aligned16(link_states) || !aligned16(cand_w) || !aligned16(cand_emb)) return LIME_INVALID_ARG;
  const lime_config& g = c->cfg;
  const lime_ffn& f = c->head;
  const int w0 = f.widths[0];
  char* base = reinterpret_cast<char*>(align_up(reinterpret_cast<uintptr_t>(ws)));
  const size_t n = (size_t)B * c->ell_c * w0;
  if ((size_t)(base - static_cast<char*>(ws)) + align_up(n * 4) + align_up(n * 2) > ws_bytes) return LIME_WORKSPACE_TOO_SMALL;
  float* LSW = reinterpret_cast<float*>(base);
  void* LSWt = base + align_up(n * 4);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ScoreArgs a{};
  a.LS = link_states; a.W = cand_w; a.T = cand_emb; a.dtype = g.dtype; a.B = B; a.ell = c->ell_c; a.d = g.d;
  a.cand_off = cand_off; a.C = C; a.total = total_cands; a.cand_ids = cand_ids; a.logits = logits;
  a.corpus_rows = cand_ids ? corpus_rows : 0; a.dev_flag = cand_ids ? dev_flag : nullptr;
  const bool tc = f.n_hidden == 1 && c->head_W1bT && score_head_tc_supported(a, w0);
  // per user: LSW_b = LS_b W_0[:d]  (the O half of the first layer applied to the link states, so O is never formed)
  lime_status s;
  if (tc && c->head_W1aT && g.d % 64 == 0)      // on tensor cores when the scorer is (link states and W_0 are bf16)
    s = launch_gemm_rows_t(link_states, (int64_t)B * c->ell_c, g.d, c->head_W1aT, w0, c->ell_c, LSWt, c->dev_err, "k_gemm_tc_lsw", st);
  else
    s = launch_rows_times_w(link_states, g.dtype, (int64_t)B * c->ell_c, g.d, f.W[0], g.dtype, w0, w0, nullptr,
                            tc ? nullptr : LSW, tc ? LSWt : nullptr, c->ell_c, "k_head_lsw", st);
  if (s != LIME_OK) return s;
  if (tc) {
    ScoreHeadArgs h{LSWt, c->head_W1bT, f.b[0], c->head_w2, f.b[1], w0};
    return launch_score_head_tc(a, h, c->dev_err, st);
  }
  const char* W0t = static_cast<const char*>(f.W[0]) + (size_t)g.d * w0 * elem_size(g.dtype);
  return launch_score_head_simt(a, LSW, W0t, f.b[0], w0, ffn_tail(f, 1), st);
}

lime_status lime_pack_corpus_cache(lime_ctx* ctx, const void* cand_emb, const void* cand_w, int64_t corpus_rows, void* packed,
                                   void* stream) {
  if (!ctx || corpus_rows < 0 || corpus_rows > 0x7fffffffLL) return LIME_INVALID_ARG;
  if (corpus_rows == 0) return LIME_OK;
  if (!cand_emb || !cand_w || !packed || !aligned16(cand_emb) || !aligned16(cand_w) || !aligned16(packed)) return LIME_INVALID_ARG;
  const Ctx* c = reinterpret_cast<const Ctx*>(ctx);
  return launch_pack_corpus(c->cfg.dtype, cand_emb, cand_w, corpus_rows, c->cfg.d, c->ell_c, packed, static_cast<cudaStream_t>(stream));
}

lime_status lime_score_candidates_packed(lime_ctx* ctx, const void* link_states, int32_t B, const void* packed,
                                         int64_t corpus_rows, const int32_t* cand_ids, const int32_t* cand_off, int32_t C,
                                         int64_t total_cands, int32_t* dev_flag, float* logits, void* stream) {
  if (!ctx || B < 0 || C < 0 || total_cands < 0 || total_cands > 0x7fffffffLL) return LIME_INVALID_ARG;
  if (corpus_rows <= 0 || corpus_rows > 0x7fffffffLL) return LIME_INVALID_ARG;
  if (!cand_off && total_cands != (int64_t)B * C) return LIME_INVALID_ARG;
  if (B == 0 || total_cands == 0) return LIME_OK;
  if (!link_states || !packed || !cand_ids || !logits || !aligned16(link_states) || !aligned16(packed)) return LIME_INVALID_ARG;
  Ctx* c = reinterpret_cast<Ctx*>(ctx);
  const int es = elem_size(c->cfg.dtype);
  ScoreArgs a{};
  a.LS = link_states; a.T = packed; a.W = static_cast<const char*>(packed) + (size_t)c->cfg.d * es;
  a.ldt = a.ldw = c->cfg.d + c->ell_c;
  a.dtype = c->cfg.dtype; a.B = B; a.ell = c->ell_c; a.d = c->cfg.d;
  a.cand_off = cand_off; a.C = C; a.total = total_cands; a.cand_ids = cand_ids; a.logits = logits;
  a.corpus_rows = corpus_rows; a.dev_flag = dev_flag;
  if (score_gather_tc_supported(a)) return launch_score_gather_tc(a, c->dev_err, static_cast<cudaStream_t>(stream));
  return launch_score_simt(a, static_cast<cudaStream_t>(stream));
}

lime_status lime_selftest_wait_expiry(lime_ctx* ctx, int32_t limit_us, void* stream) {
  if (!ctx || limit_us < 1 || limit_us > 1000000) return LIME_INVALID_ARG;
  Ctx* c = reinterpret_cast<Ctx*>(ctx);
  return launch_wait_expiry(c->dev_err, (uint64_t)limit_us * 1000ull, LIME_SELFTEST_WAIT_CODE, static_cast<cudaStream_t>(stream));
}

lime_status lime_device_status(lime_ctx* ctx, int32_t* code) {
  if (!ctx || !code) return LIME_INVALID_ARG;
  Ctx* c = reinterpret_cast<Ctx*>(ctx);
  int v = 0;
  LIME_CUDA(cudaMemcpy(&v, c->dev_err, sizeof(int), cudaMemcpyDeviceToHost));
  *code = v;
  if (v != 0) {
    LIME_CUDA(cudaMemset(c->dev_err, 0, sizeof(int)));
    return LIME_DEVICE_TIMEOUT;
  }
  return LIME_OK;
}

}  // extern "C"
