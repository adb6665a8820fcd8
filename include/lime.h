/*
 * lime.h -- C ABI of the B200 (sm_100a) LIME ranking-inference hot path.
 *
 * LIME (link embeddings + XOR attention + decoupled candidate attention) splits ranking inference
 * into three stages (Sec. 3.3 of the paper):
 *   offline : candidate->link attention weights phi(T L^t), independent of the user        (Eq. 4)
 *   online  : per user, n stacked XOR layers turn the shared links L into personalised
 *             links L^P by attending over the user's N(U) history items                     (Eq. 3, 6-8)
 *   per candidate : weighted sum of the user's link states, then a score                    (Eq. 4)
 *
 * Conventions shared by every entry point
 *   - Every tensor pointer is a DEVICE pointer owned by the caller unless the comment says "host".
 *     The library never frees or keeps caller memory beyond the call, except the weight pointers given
 *     to lime_set_weights, which are borrowed until the next lime_set_weights / lime_destroy.
 *   - Row-major, innermost dimension contiguous, base addresses 16-byte aligned.
 *   - Activations and weights are stored as `dtype` (LIME_F32 or LIME_BF16); logits are always fp32;
 *     ids / lengths / offsets are int32 (addresses are formed in 64 bits).
 *   - Projections act on the right: X~ = X W, W stored [d_in x d_out].  Heads are H contiguous chunks of
 *     d_h = d / H features.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL = the legacy default stream).
 *     No entry point synchronises the device, allocates device memory (except lime_create /
 *     lime_set_weights, which are set-up calls) or launches from more than one stream.
 *   - Every function returns a lime_status; nothing throws, aborts or traps on the device.  Arguments are
 *     validated on the host before any launch; a failed validation launches nothing.
 *   - The caller provides scratch memory ("workspace") sized by lime_workspace_bytes(); its contents are
 *     undefined between calls.  Two calls that overlap on the GPU must not share a workspace.
 */
#ifndef LIME_B200_H
#define LIME_B200_H

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define LIME_API __attribute__((visibility("default")))
#else
#define LIME_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum lime_status {
  LIME_OK = 0,
  LIME_INVALID_ARG = 1,         /* NULL where a pointer is required, negative size, misaligned pointer   */
  LIME_UNSUPPORTED_SHAPE = 2,   /* d, H, ell, d_ff outside what the kernels are built for                */
  LIME_WORKSPACE_TOO_SMALL = 3,
  LIME_CUDA_ERROR = 4,          /* a CUDA runtime/driver call failed; see lime_last_cuda_error()         */
  LIME_NOT_READY = 5,           /* weights not set                                                        */
  LIME_DEVICE_TIMEOUT = 6,      /* a bounded wait inside a kernel gave up; outputs of that call are invalid */
  LIME_EXCEEDS_STATIC_SCRATCH = 7 /* shape too large for the fixed scratch of an allocation-free entry point    */
} lime_status;

typedef enum lime_dtype { LIME_F32 = 0, LIME_BF16 = 1 } lime_dtype;
typedef enum lime_phi { LIME_PHI_SOFTMAX = 0, LIME_PHI_SILU = 1 } lime_phi;

#define LIME_MAX_LAYERS 16

/* Model shape (notation of the paper's App. A): d embedding dim, H heads, ell links, n_layers XOR layers. */
typedef struct lime_config {
  int32_t d;            /* multiple of 8, <= 1024; d % H == 0; d_h = d / H <= 128;
                           8*ell*(d+1) + 16*d <= 204800 (a user's link keys and values stay in shared memory) */
  int32_t H;
  int32_t ell;          /* 1..256                                                                         */
  int32_t n_layers;     /* 1..LIME_MAX_LAYERS                                                             */
  int32_t d_ff;         /* GatedMLP width; 0 means d                                                      */
  int32_t dtype;        /* lime_dtype: storage type of embeddings, weights, link states, cached weights   */
  int32_t phi;          /* lime_phi: attention activation of the XOR layers (candidate side is softmax)   */
  int32_t ln;           /* 1: non-affine LayerNorm before the Q/K/V projections (App. C)                  */
  int32_t gated_mlp;    /* 1: GatedMLP after the attention (Eq. 5 / Eq. 8); 0: identity                   */
  float attn_scale;     /* softmax scale of the XOR layers; 0 means 1/sqrt(d_h)                           */
  float cand_scale;     /* softmax scale of the candidate->link attention; 0 means 1/sqrt(d)              */
  float ln_eps;         /* 0 means 1e-5                                                                   */
  int32_t cand_heads;   /* candidate side (Eq. 4): 0 or 1 = one weight row per candidate over the full width,
                           scale 1/sqrt(d); H = Eq. 1 applied head by head: one weight row per (candidate, head),
                           scale 1/sqrt(d_h), each head mixing its own d_h columns of the link states.  With H the
                           cached weights have ell_c = H*ell columns (head-major) and a user's link states ell_c
                           rows (row h*ell + l = link l on head h's columns, zero elsewhere); H*ell <= 256.       */
} lime_config;

/* Device pointers to the parameters theta, eta of Eq. 1 / Eq. 5 / Eq. 8, all stored as config.dtype. */
typedef struct lime_weights {
  const void* links;                    /* L   [ell x d]                                                   */
  const void* Wq[LIME_MAX_LAYERS];      /* W_Q [d x d] per layer; NULL = identity                          */
  const void* Wk[LIME_MAX_LAYERS];      /* W_K [d x d]                                                     */
  const void* Wv[LIME_MAX_LAYERS];      /* W_V [d x d]                                                     */
  const void* Wg[LIME_MAX_LAYERS];      /* GatedMLP gate  [d x d_ff]   (required when gated_mlp = 1)       */
  const void* Wu[LIME_MAX_LAYERS];      /* GatedMLP up    [d x d_ff]                                       */
  const void* Wo[LIME_MAX_LAYERS];      /* GatedMLP down  [d_ff x d]                                       */
  const void* cand_Wq;                  /* candidate-side W_Q [d x d] of Eq. 4, NULL = identity            */
  const void* cand_Wk;                  /* candidate-side W_K [d x d] (applied to the raw links L)         */
  const void* cand_Wv;                  /* candidate-side W_V [d x d] (applied to L^P -> link states)      */
} lime_weights;

typedef struct lime_ctx lime_ctx;       /* opaque; holds the config, borrowed weight pointers and a few KB
                                           of derived device data */

/* Set-up.  lime_create validates the shape and allocates the context (host) plus a small device buffer for
 * weight-derived data; call it with the target device current.  lime_destroy frees both (NULL is a no-op). */
LIME_API lime_status lime_create(const lime_config* cfg, lime_ctx** out);
LIME_API lime_status lime_destroy(lime_ctx* ctx);

/* Borrow the parameter pointers (host struct of device pointers).  Launches, on `stream`, the tiny
 * weight-only preparation the candidate side needs (the effective link keys (L W_K^c) W_Q^c^T of Eq. 4,
 * so that the cached weights are phi(T K_eff^T) whatever projections are present). */
LIME_API lime_status lime_set_weights(lime_ctx* ctx, const lime_weights* w, void* stream);

/* Bytes of scratch lime_xor_layer / lime_encode_user need for a batch of B users holding total_tokens
 * history items in all.  0 on invalid arguments. */
LIME_API size_t lime_workspace_bytes(const lime_ctx* ctx, int32_t B, int64_t total_tokens);

/* Ragged bookkeeping (Sec. 3: each user U has N(U) history items): exclusive prefix sum
 * off[0] = 0, off[b+1] = off[b] + len[b].  len [B], off [B+1] device int32.  Lengths must be >= 0 and sum
 * below 2^31; negative lengths are treated as 0. B = 0 writes off[0] = 0. */
LIME_API lime_status lime_lengths_to_offsets(lime_ctx* ctx, const int32_t* len, int32_t B, int32_t* off, void* stream);

/* History embedding lookup (Sec. 3, stand-in for the attribute-embedding pipeline): out[t,:] = table[ids[t],:].
 * table [V x d], ids [total_tokens], out [total_tokens x d].  An id outside [0, V) writes a zero row and, if
 * dev_flag is not NULL, atomically lowers *dev_flag (device int32, caller initialises it to INT32_MAX) to the
 * smallest offending position.  Exact byte copy otherwise. */
LIME_API lime_status lime_gather_history(lime_ctx* ctx, const void* table, int64_t V, const int32_t* ids,
                                int64_t total_tokens, void* out, int32_t* dev_flag, void* stream);

/* The same lookup with the LayerNorm of the first XOR layer applied on the way:
 *   out[t,:] = LN(table[ids[t],:])   (non-affine, eps of the config, rounded to config.dtype).
 * The XOR layers read the history only through the LayerNorm that precedes their Q/K/V projections (App. C, Eq. 1 /
 * Eq. 7), so nothing downstream needs the raw rows; normalising them here, while a row sits in registers, spares both
 * attention directions of the first layer the per-token statistics.  Pass the result to lime_encode_user_normalized.
 * Same arguments, layouts and treatment of bad ids as lime_gather_history; with config.ln = 0 it is that call. */
LIME_API lime_status lime_gather_history_normalized(lime_ctx* ctx, const void* table, int64_t V, const int32_t* ids,
                                           int64_t total_tokens, void* out, int32_t* dev_flag, void* stream);

/* Offline item-side stage (Eq. 4, Sec. 3.3 "pre-computed and cached"): out_w[c,:] = softmax over the ell
 * links of (T_c W_Q^c)(L W_K^c)^T * cand_scale.  cand_emb [M x d], out_w [M x ell_c] stored as config.dtype
 * (ell_c = ell, or H*ell with cand_heads = H: per head the softmax over that head's scores). */
LIME_API lime_status lime_precompute_candidate_links(lime_ctx* ctx, const void* cand_emb, int64_t M, void* out_w,
                                            void* stream);

/* One XOR layer (Eq. 6-7 with the GatedMLP of Eq. 5 on both partitions):
 *   O[T] = phi(Q[T] K[S]^T) V[S]   links attend over the user's history     -> links_out = GatedMLP(O[T])
 *   O[S] = phi(Q[S] K[T]^T) V[T]   history attends back over the links      -> hist_out  = GatedMLP(O[S])
 * hist_in [total_tokens x d] (config.dtype), off [B+1] device int32, links_in fp32 [B x ell x d] or, with
 * links_shared != 0, one [ell x d] block used for every user.  links_out fp32 [B x ell x d].  hist_out
 * (config.dtype) may be NULL (the last layer's history update is never used, Eq. 8) and may alias hist_in.
 * A user with an empty history gets O[T] = 0.  `layer` selects the weights. */
LIME_API lime_status lime_xor_layer(lime_ctx* ctx, int32_t layer, const void* hist_in, const int32_t* off, int32_t B,
                           int64_t total_tokens, const float* links_in, int32_t links_shared, void* hist_out,
                           float* links_out, void* ws, size_t ws_bytes, void* stream);

/* Online user-side stage (Eq. 8): runs the n_layers stacked XOR layers on hist [total_tokens x d] and writes
 * the link states V~ = L^P W_V^c (Eq. 4's values) as config.dtype into link_states [B x ell_c x d].
 * link_ctx: optional per-user contextualised links L^C (Eq. 2) as fp32 [B x ell x d]; NULL uses the shared L.
 * hist is not modified. */
LIME_API lime_status lime_encode_user(lime_ctx* ctx, const void* hist, const int32_t* off, int32_t B,
                             int64_t total_tokens, const float* link_ctx, void* link_states, void* ws,
                             size_t ws_bytes, void* stream);

/* lime_encode_user for history rows that are LayerNorm-ed already (as lime_gather_history_normalized leaves them):
 * the first layer then skips its LayerNorm of the history.  Same arguments, ownership and errors.  The result equals
 * lime_encode_user on the raw rows up to the rounding of the normalised rows to config.dtype.  With config.ln = 0 the
 * two calls are the same. */
LIME_API lime_status lime_encode_user_normalized(lime_ctx* ctx, const void* hist_normalized, const int32_t* off, int32_t B,
                                        int64_t total_tokens, const float* link_ctx, void* link_states, void* ws,
                                        size_t ws_bytes, void* stream);

/* Per-candidate stage (Eq. 4 and Sec. 3.3 "lightweight user-item interaction"):
 *   logits[i] = < sum_l cand_w[i,l] * link_states[b(i),l,:] , cand_emb[i,:] >   for every candidate slot i.
 * Candidates are per user: user b owns slots cand_off[b] .. cand_off[b+1]-1 of cand_w [total_cands x ell_c],
 * cand_emb [total_cands x d] and logits [total_cands]; cand_off is a DEVICE int32 array [B+1], non-decreasing,
 * cand_off[0] = 0, cand_off[B] = total_cands.  With cand_off = NULL every user owns C slots (slot b*C + c) and
 * total_cands must equal B*C.  cand_ids (device int32 [total_cands], nullable): when given, cand_w and
 * cand_emb are corpus-level caches (Sec. 3.3 "QK cache") of corpus_rows rows each (1 <= corpus_rows < 2^31) and row
 * cand_ids[i] is read for slot i.  An id outside [0, corpus_rows) reads nothing: that slot's logit is 0 and, if
 * dev_flag is not NULL, *dev_flag (device int32, caller initialises it to INT32_MAX) is atomically lowered to the
 * smallest offending slot, as in lime_gather_history.  Without cand_ids both arguments are ignored.
 * link_states [B x ell_c x d] as written by lime_encode_user. */
LIME_API lime_status lime_score_candidates(lime_ctx* ctx, const void* link_states, int32_t B, const void* cand_w,
                                  const void* cand_emb, const int32_t* cand_off, int32_t C, int64_t total_cands,
                                  const int32_t* cand_ids, int64_t corpus_rows, int32_t* dev_flag, float* logits,
                                  void* stream);

/* Corpus caches as one record per item (Sec. 3.3: the cached weights sit beside the item embedding): packed [corpus_rows x
 * (d + ell_c)] in config.dtype, record v = [ cand_emb[v, 0..d) | cand_w[v, 0..ell_c) ].  lime_pack_corpus_cache builds it
 * from the two separate caches (offline, whenever they change).  lime_score_candidates_packed is lime_score_candidates
 * with cand_ids over such records: a candidate's embedding and weights then come from one place in memory instead of
 * two.  Same logits, same treatment of ids outside [0, corpus_rows), same meaning of cand_off / C / total_cands. */
LIME_API lime_status lime_pack_corpus_cache(lime_ctx* ctx, const void* cand_emb, const void* cand_w, int64_t corpus_rows,
                                   void* packed, void* stream);
LIME_API lime_status lime_score_candidates_packed(lime_ctx* ctx, const void* link_states, int32_t B, const void* packed,
                                         int64_t corpus_rows, const int32_t* cand_ids, const int32_t* cand_off, int32_t C,
                                         int64_t total_cands, int32_t* dev_flag, float* logits, void* stream);

/* The two small feed-forward networks the paper names without a formula.  Both are read as x <- ReLU(x W_i + b_i)
 * for each of n_hidden hidden layers followed by one linear layer; W[i] is [in_i x out_i] row-major in config.dtype,
 * b[i] fp32 [out_i] or NULL (no bias); all are device pointers, borrowed until replaced or lime_destroy. */
#define LIME_FFN_MAX_HIDDEN 3
typedef struct lime_ffn {
  int32_t n_hidden;                          /* hidden layers: 0..3 (the interaction network needs at least 1)        */
  int32_t widths[LIME_FFN_MAX_HIDDEN];       /* their widths, each 1..1024                                             */
  const void* W[LIME_FFN_MAX_HIDDEN + 1];    /* n_hidden + 1 weight matrices                                           */
  const float* b[LIME_FFN_MAX_HIDDEN + 1];   /* n_hidden + 1 bias vectors (nullable)                                   */
} lime_ffn;

/* Link contextualisation (Eq. 2): L^C_b = MLP(L (+) E^C_b).  Every link row L_l [d] is followed by the user's context
 * features E^C_b [d_c]; the network maps the (d + d_c)-wide rows to d: in_0 = d + d_c (rows 0..d-1 of W[0] act on the
 * link, rows d.. on the context), out of the last layer = d.  lime_set_context_mlp is a set-up call (it allocates a
 * few KB and launches the weights-only part of the first layer on `stream`); call it after lime_set_weights, and again
 * after the links change.  lime_contextualize_links writes link_ctx fp32 [B x ell x d], the `link_ctx` argument of
 * lime_encode_user; user_ctx [B x d_c] in config.dtype.  LIME_NOT_READY without a network. */
LIME_API lime_status lime_set_context_mlp(lime_ctx* ctx, int32_t d_c, const lime_ffn* mlp, void* stream);
LIME_API lime_status lime_contextualize_links(lime_ctx* ctx, const void* user_ctx, int32_t B, float* link_ctx, void* stream);

/* Interaction network on the LIME embedding (Sec. 3.3 "Lightweight User-Item Interaction"; hidden widths as the
 * "Interaction MLP" row of App. C's table, e.g. one 96-wide layer):
 *   logits[i] = FFN( [O_i | T_i] ),  O_i = sum_l cand_w[i,l] * link_states[b(i),l,:],  T_i = cand_emb[i,:]
 * in_0 = 2d (rows 0..d-1 of W[0] act on O, rows d..2d-1 on T), out of the last layer = 1, n_hidden >= 1.
 * lime_set_head is a set-up call (allocates copies of two small operands).  lime_score_candidates_head takes the
 * arguments of lime_score_candidates plus scratch of lime_head_workspace_bytes(ctx, B) bytes (the per-user product
 * link_states . W[0][:d], so that O is never formed).  LIME_NOT_READY without a network. */
LIME_API lime_status lime_set_head(lime_ctx* ctx, const lime_ffn* head, void* stream);
LIME_API size_t lime_head_workspace_bytes(const lime_ctx* ctx, int32_t B);
LIME_API lime_status lime_score_candidates_head(lime_ctx* ctx, const void* link_states, int32_t B, const void* cand_w,
                                       const void* cand_emb, const int32_t* cand_off, int32_t C, int64_t total_cands,
                                       const int32_t* cand_ids, int64_t corpus_rows, int32_t* dev_flag, float* logits,
                                       void* ws, size_t ws_bytes, void* stream);

/* Allocation-free precompute (the paper has no counterpart: this exists for hosts that must not allocate).
 * Same result as lime_create + lime_set_weights + lime_precompute_candidate_links, for callers that cannot call
 * cudaMalloc at this point - a serving process whose device memory pool is frozen after start-up, or code running
 * inside a framework that owns the allocator - and therefore cannot create a context.  It takes the shape and the
 * weight pointers directly (dtype, d, ell, cand_scale as in lime_config; links [ell x d]; cand_Wq / cand_Wk [d x d]
 * or NULL; cand_emb [M x d]; out_w [M x ell]; all device pointers of `dtype`, 16-byte aligned) and calls no
 * cudaMalloc, cudaFree or other allocating routine.  Its scratch (the effective link keys and one intermediate,
 * 2 * ell * d floats) lives in a fixed device array inside the library, 2 * LIME_NOALLOC_MAX_LINK_ELEMS floats
 * (128 KB) that every GPU loading the library holds until the process exits.
 *   - ell * d > LIME_NOALLOC_MAX_LINK_ELEMS returns LIME_EXCEEDS_STATIC_SCRATCH (and sets the error text); nothing
 *     is launched.
 *   - The first call on each device looks up the array's device address (with that device current); make that
 *     first call before starting any stream capture.
 *   - All calls share the one array, which keeps the previous call's contents; every call rewrites all of the part
 *     it uses before reading it, so nothing needs clearing.  Two calls that overlap on the GPU (different streams,
 *     or different threads) race on it: serialise them. */
#define LIME_NOALLOC_MAX_LINK_ELEMS 16384
LIME_API lime_status lime_precompute_candidate_links_noalloc(int32_t dtype, int32_t d, int32_t ell, float cand_scale,
                                                             const void* links, const void* cand_Wq,
                                                             const void* cand_Wk, const void* cand_emb, int64_t M,
                                                             void* out_w, void* stream);

/* Health check.  The tensor-core kernels synchronise their warps through mbarriers with bounded waits (2 s); a wait
 * that gives up records a non-zero code in a device word of the context and the kernel exits cleanly (no trap, no
 * hang) with its outputs undefined.  lime_device_status SYNCHRONISES the device (a blocking copy of that word),
 * writes the code to *code (host), clears it, and returns LIME_DEVICE_TIMEOUT if it was set, else LIME_OK.
 * The paper has no counterpart; codes: 1 producer, 2-3 MMA issuer, 4 epilogue waits of the scorer. */
LIME_API lime_status lime_device_status(lime_ctx* ctx, int32_t* code);

/* Self-test of that mechanism (the paper has no counterpart): launches one thread that waits, for at most limit_us
 * microseconds (1 .. 1,000,000), on a barrier nothing ever arrives at.  The wait gives up, the kernel returns, and the
 * next lime_device_status reports LIME_DEVICE_TIMEOUT with code LIME_SELFTEST_WAIT_CODE; the context stays usable.
 * Nothing faults, traps or spins without a bound. */
#define LIME_SELFTEST_WAIT_CODE 200
LIME_API lime_status lime_selftest_wait_expiry(lime_ctx* ctx, int32_t limit_us, void* stream);

/* Per-kernel timing for benchmarks (the paper reports latency only end to end, App. F; this breaks a call down).
 * Between lime_profile_start(capacity) and lime_profile_stop every kernel this library launches is bracketed by two
 * CUDA events on its stream, up to `capacity` launches (later ones are counted but not timed).  lime_profile_stop
 * waits for the recorded events, writes the launch durations in milliseconds to ms[0..min(count, ms_capacity))
 * (host), the kernel names, newline-separated in launch order, to names (host, names_bytes long, truncated if
 * short), the number of launches seen to *count, and frees the events.  Process-wide, not thread-safe; both are
 * set-up calls (they create and destroy events) and must not be used during stream capture. */
LIME_API lime_status lime_profile_start(int32_t capacity);
LIME_API lime_status lime_profile_stop(char* names, size_t names_bytes, float* ms, int32_t ms_capacity, int32_t* count);

/* Text of the last CUDA error seen by this library on the calling thread ("" if none). Host pointer, static. */
LIME_API const char* lime_last_cuda_error(void);

/* Library version and the SM architecture it was compiled for (e.g. "lime-b200 0.1 sm_100a"). Host pointer. */
LIME_API const char* lime_version(void);

#ifdef __cplusplus
}
#endif
#endif /* LIME_B200_H */
