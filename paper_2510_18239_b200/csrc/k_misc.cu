// Ragged bookkeeping, the history-embedding gather and small elementwise helpers.
#include "lime_common.cuh"

namespace lime {

// ----------------------------------------------------------------------------- block-wide exclusive scan
// One block of 1024 threads walks the array in slabs of 1024 with a running carry. B is at most a few
// thousand users per batch, so a single block is latency-optimal (one launch, no inter-block traffic).
template <typename F>
__device__ __forceinline__ void block_exclusive_scan(int n, int32_t* out, F value_at) {
  __shared__ int32_t warp_tot[32];
  __shared__ int32_t carry_s;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  if (threadIdx.x == 0) carry_s = 0;
  __syncthreads();
  for (int base = 0; base < n; base += blockDim.x) {
    const int i = base + threadIdx.x;
    const int32_t v = (i < n) ? value_at(i) : 0;
    int32_t incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int32_t t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    if (lane == 31) warp_tot[wid] = incl;
    __syncthreads();
    if (wid == 0) {
      int32_t w = (lane < (int)(blockDim.x >> 5)) ? warp_tot[lane] : 0;
      int32_t wi = w;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int32_t t = __shfl_up_sync(0xffffffffu, wi, o);
        if (lane >= o) wi += t;
      }
      warp_tot[lane] = wi - w;  // exclusive prefix of warp totals
    }
    __syncthreads();
    const int32_t carry = carry_s;
    if (i < n) out[i] = carry + warp_tot[wid] + incl - v;
    __syncthreads();
    if (threadIdx.x == blockDim.x - 1) carry_s = carry + warp_tot[wid] + incl;  // last thread holds the slab total
    __syncthreads();
  }
  if (threadIdx.x == 0) out[n] = carry_s;
}

__global__ void __launch_bounds__(1024) k_offsets(const int32_t* __restrict__ len, int B, int32_t* __restrict__ off) {
  pdl_launch_dependents();     // simple kernel: the next one may set itself up beside it
  pdl_wait();                  // nothing is read or written before the previous kernel is complete
  block_exclusive_scan(B, off, [&](int i) { return max(len[i], 0); });
}

// Deal the (user, chunk) items of the links<-history attention to `G` groups of CTAs so that the groups' token tiles
// come out even.  Items are sorted by size (a counting sort over their tile counts, largest first) and handed out in
// rounds of G: within a round the group with the least work so far takes the largest item, the next group the next
// one, and so on.  Ragged histories dealt round-robin leave the busiest group 16 % above the mean (1024 users of
// 1024..4096 tokens over 37 groups); this order leaves it under 1 %.  One block; a round is one rank computation over
// the G loads in shared memory and one barrier.
// group_start[G+1], group_items[items]: the items of group j in the order it takes them.  scratch: 4 x items ints.
__device__ void balance_groups(const int32_t* __restrict__ off, int chunk, const int32_t* __restrict__ chunk_start,
                               const int32_t* __restrict__ chunk_user, int n_items, int G, int att_tile,
                               int32_t* __restrict__ group_start, int32_t* __restrict__ group_items, int32_t* __restrict__ scratch) {
  constexpr int KEYS = 256, GMAX = 160, KCAP = 16384;
  __shared__ int32_t hist[KEYS];
  __shared__ int32_t load[GMAX], cnt[GMAX];
  __shared__ uint8_t skey[KCAP];                   // sizes in sorted order (the first KCAP items; the rest are read from global)
  int32_t* sorted = scratch;
  int32_t* key_of = scratch + n_items;             // by item, then (after the sort) by sorted position
  int32_t* group_of = scratch + 2 * (size_t)n_items;
  int32_t* slot_of = scratch + 3 * (size_t)n_items;
  for (int i = threadIdx.x; i < KEYS; i += blockDim.x) hist[i] = 0;
  for (int i = threadIdx.x; i < GMAX; i += blockDim.x) { load[i] = 0; cnt[i] = 0; }
  __syncthreads();
  for (int i = threadIdx.x; i < n_items; i += blockDim.x) {
    const int b = chunk_user[i];
    const int tok = min(chunk, off[b + 1] - off[b] - (i - chunk_start[b]) * chunk);
    const int key = min(KEYS - 1, (tok + att_tile - 1) / att_tile);
    group_of[i] = key;                             // parked here until the scatter below
    atomicAdd(&hist[KEYS - 1 - key], 1);           // bucket 0 holds the largest items
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int run = 0;
    for (int k = 0; k < KEYS; ++k) { const int c = hist[k]; hist[k] = run; run += c; }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < n_items; i += blockDim.x) {
    const int key = group_of[i];
    const int at = atomicAdd(&hist[KEYS - 1 - key], 1);
    sorted[at] = i;
    key_of[at] = key;
    if (at < KCAP) skey[at] = (uint8_t)key;
  }
  __syncthreads();
  for (int r0 = 0; r0 < n_items; r0 += G) {
    const int j = threadIdx.x;
    int rank = 0, mine = 0;
    if (j < G) {
      mine = load[j];
      for (int o = 0; o < G; ++o) {
        const int lo = load[o];
        rank += (lo < mine || (lo == mine && o < j)) ? 1 : 0;
      }
    }
    __syncthreads();                               // every rank is taken before a load changes
    if (j < G && r0 + rank < n_items) {
      const int at = r0 + rank;
      const int key = at < KCAP ? (int)skey[at] : key_of[at];
      group_of[at] = j;                             // by sorted position: no dependent read inside a round
      slot_of[at] = cnt[j]++;
      load[j] = mine + key;
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    int run = 0;
    for (int j = 0; j < G; ++j) { group_start[j] = run; run += cnt[j]; }
    group_start[G] = run;
  }
  __syncthreads();
  for (int at = threadIdx.x; at < n_items; at += blockDim.x) group_items[group_start[group_of[at]] + slot_of[at]] = sorted[at];
}

// both work lists of the XOR layers in one launch: chunks of the links<-history attention, tiles of the history update
__global__ void __launch_bounds__(1024)
k_layer_schedules(const int32_t* __restrict__ off, int B, int chunk, int32_t* __restrict__ chunk_start, int tile,
                  int32_t* __restrict__ tile_start, int32_t* __restrict__ chunk_user, int32_t* __restrict__ merge_needed,
                  int G, int att_tile, int32_t* __restrict__ group_start, int32_t* __restrict__ group_items,
                  int32_t* __restrict__ scratch) {
  pdl_launch_dependents();     // simple kernel: the next one may set itself up beside it
  pdl_wait();                  // nothing is read or written before the previous kernel is complete
  // does any user's attention output need the merge step (several chunks to combine, or no history: a zero row)?
  __shared__ int any_merge;
  if (threadIdx.x == 0) any_merge = 0;
  __syncthreads();
  for (int b = threadIdx.x; b < B; b += blockDim.x)
    if (off[b + 1] - off[b] <= 0 || off[b + 1] - off[b] > chunk) any_merge = 1;
  __syncthreads();
  if (threadIdx.x == 0 && merge_needed != nullptr) *merge_needed = any_merge;
  block_exclusive_scan(B, chunk_start, [&](int i) {
    int n = off[i + 1] - off[i];
    return n > 0 ? (n + chunk - 1) / chunk : 0;
  });
  __syncthreads();
  block_exclusive_scan(B, tile_start, [&](int i) {
    int n = off[i + 1] - off[i];
    return n > 0 ? (n + tile - 1) / tile : 0;
  });
  // inverse map (chunk item -> user): the attention kernel strides through the items, and one read of this table
  // replaces a search over chunk_start per item
  __syncthreads();
  if (chunk_user != nullptr)
    for (int b = threadIdx.x; b < B; b += blockDim.x)
      for (int i = chunk_start[b]; i < chunk_start[b + 1]; ++i) chunk_user[i] = b;
  if (group_start != nullptr && chunk_user != nullptr) {
    __syncthreads();
    balance_groups(off, chunk, chunk_start, chunk_user, chunk_start[B], G, att_tile, group_start, group_items, scratch);
  }
}

lime_status launch_layer_schedules(const int32_t* off, int B, int chunk, int32_t* chunk_start, int tile, int32_t* tile_start,
                                   int32_t* chunk_user, int32_t* merge_needed, const GroupSchedule& gs, cudaStream_t st) {
  if (gs.group_start != nullptr && (gs.n_groups < 1 || gs.n_groups > 160 || gs.att_tile < 1)) return LIME_INVALID_ARG;
  ProfScope _p("k_layer_schedules", st);
  launch_pdl(k_layer_schedules, dim3(1), dim3(1024), 0, st, off, B, chunk, chunk_start, tile, tile_start, chunk_user, merge_needed,
             gs.n_groups, gs.att_tile, gs.group_start, gs.group_items, gs.scratch);
  LIME_LAUNCH_CHECK("k_layer_schedules");
  return LIME_OK;
}

lime_status launch_offsets(const int32_t* len, int B, int32_t* off, cudaStream_t st) {
  ProfScope _p("k_offsets", st);
  launch_pdl(k_offsets, dim3(1), dim3(1024), 0, st, len, B, off);
  LIME_LAUNCH_CHECK("k_offsets");
  return LIME_OK;
}

// ----------------------------------------------------------------------------- gather
// out[t, :] = table[ids[t], :].  Rows are 16-byte multiples (d % 8 == 0 for both dtypes), so a row moves as
// uint4 words: `LANES` consecutive threads own one row and each moves row_vec / LANES words, giving fully
// coalesced 128-bit loads and stores.  Reads of hot (Zipf head) rows hit L2; the stream is write-dominated.
template <int LANES>
__global__ void __launch_bounds__(256)
k_gather(const uint4* __restrict__ table, int64_t V, int row_vec, const int32_t* __restrict__ ids, int64_t total,
         uint4* __restrict__ out, int32_t* __restrict__ dev_flag) {
  const int rows_per_block = blockDim.x / LANES;
  const int sub = threadIdx.x % LANES;
  const int64_t stride = (int64_t)gridDim.x * rows_per_block;
  for (int64_t t = (int64_t)blockIdx.x * rows_per_block + threadIdx.x / LANES; t < total; t += stride) {
    const int32_t id = __ldg(ids + t);
    const bool ok = id >= 0 && (int64_t)id < V;
    uint4* dst = out + t * row_vec;
    if (ok) {
      const uint4* src = table + (int64_t)id * row_vec;
      for (int v = sub; v < row_vec; v += LANES) dst[v] = __ldg(src + v);
    } else {
      for (int v = sub; v < row_vec; v += LANES) dst[v] = make_uint4(0, 0, 0, 0);
      if (sub == 0 && dev_flag != nullptr) atomicMin(dev_flag, (int32_t)min(t, (int64_t)INT32_MAX));
    }
  }
}

// out[t, :] = LayerNorm(table[ids[t], :]) (non-affine), in the storage type (ids == NULL: the rows of `table` in order,
// i.e. a plain LayerNorm pass over V = total rows).  Same row-per-LANES mapping; a lane keeps
// its WORDS 16-byte words of the row in registers, the lanes of a row reduce the sum and then the squared
// deviations with shuffles (two passes: exact mean first), and the normalised row is written once.  The loop runs
// per warp-wide group of rows so that every lane takes part in the shuffles.
// a 16-byte word of the storage type <-> floats (bf16: two elements per 32-bit lane, widened with a shift / a mask
// and narrowed pairwise with one round-to-nearest conversion)
template <typename T> struct Word16;
template <> struct Word16<float> {
  static __device__ __forceinline__ void unpack(const uint4& w, float (&x)[4]) {
    x[0] = __uint_as_float(w.x); x[1] = __uint_as_float(w.y); x[2] = __uint_as_float(w.z); x[3] = __uint_as_float(w.w);
  }
  static __device__ __forceinline__ uint4 pack(const float (&x)[4]) {
    return make_uint4(__float_as_uint(x[0]), __float_as_uint(x[1]), __float_as_uint(x[2]), __float_as_uint(x[3]));
  }
};
template <> struct Word16<__nv_bfloat16> {
  static __device__ __forceinline__ void unpack(const uint4& w, float (&x)[8]) {
    const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) { x[2 * k] = __uint_as_float(u[k] << 16); x[2 * k + 1] = __uint_as_float(u[k] & 0xffff0000u); }
  }
  static __device__ __forceinline__ uint4 pack(const float (&x)[8]) {
    uint32_t u[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const __nv_bfloat162 p2 = __floats2bfloat162_rn(x[2 * k], x[2 * k + 1]);
      u[k] = *reinterpret_cast<const uint32_t*>(&p2);
    }
    return make_uint4(u[0], u[1], u[2], u[3]);
  }
};

template <typename T, int LANES, int WORDS>
__global__ void __launch_bounds__(256)
k_gather_ln(const uint4* __restrict__ table, int64_t V, int row_vec, int d, float eps, const int32_t* __restrict__ ids,
            int64_t total, uint4* __restrict__ out, int32_t* __restrict__ dev_flag) {
  pdl_launch_dependents();     // simple kernel: the next one may set itself up beside it
  pdl_wait();                  // nothing is read or written before the previous kernel is complete
  constexpr int PER = 16 / (int)sizeof(T);                 // elements per 16-byte word
  constexpr int ROWS = 1;   // rows per lane group and pass (more in flight measured slower: the grid already covers the latency)
  const int rows_per_block = blockDim.x / LANES;
  const int sub = threadIdx.x % LANES;
  const int64_t stride = (int64_t)gridDim.x * rows_per_block * ROWS;
  for (int64_t base = (int64_t)blockIdx.x * rows_per_block * ROWS; base < total; base += stride) {
    int64_t t[ROWS];
    bool live[ROWS], ok[ROWS];
    int32_t id[ROWS];
#pragma unroll
    for (int k = 0; k < ROWS; ++k) {
      t[k] = base + (int64_t)k * rows_per_block + threadIdx.x / LANES;
      live[k] = t[k] < total;
      id[k] = live[k] ? (ids != nullptr ? __ldg(ids + t[k]) : (int32_t)t[k]) : 0;   // no ids: row t of `table` itself
      ok[k] = live[k] && id[k] >= 0 && (int64_t)id[k] < V;
    }
    uint4 w[ROWS][WORDS];
#pragma unroll
    for (int k = 0; k < ROWS; ++k)
#pragma unroll
      for (int i = 0; i < WORDS; ++i) {
        const int v = sub + i * LANES;
        w[k][i] = (ok[k] && v < row_vec) ? __ldg(table + (int64_t)id[k] * row_vec + v) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
    for (int k = 0; k < ROWS; ++k) {
      float x[WORDS][PER];
      float sum = 0.f;
#pragma unroll
      for (int i = 0; i < WORDS; ++i) {
        Word16<T>::unpack(w[k][i], x[i]);
#pragma unroll
        for (int j = 0; j < PER; ++j) sum += x[i][j];
      }
#pragma unroll
      for (int o = LANES / 2; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      const float mu = sum / (float)d;
      float var = 0.f;
#pragma unroll
      for (int i = 0; i < WORDS; ++i) {
        if (sub + i * LANES < row_vec) {
#pragma unroll
          for (int j = 0; j < PER; ++j) { x[i][j] -= mu; var = fmaf(x[i][j], x[i][j], var); }
        }
      }
#pragma unroll
      for (int o = LANES / 2; o > 0; o >>= 1) var += __shfl_xor_sync(0xffffffffu, var, o);
      const float rstd = rsqrtf(var / (float)d + eps);
      if (live[k]) {
#pragma unroll
        for (int i = 0; i < WORDS; ++i) {
          const int v = sub + i * LANES;
          if (v < row_vec) {
            uint4 o4 = make_uint4(0, 0, 0, 0);              // an id outside [0, V) gives a zero row, as in k_gather
            if (ok[k]) {
#pragma unroll
              for (int j = 0; j < PER; ++j) x[i][j] *= rstd;
              o4 = Word16<T>::pack(x[i]);
            }
            out[t[k] * row_vec + v] = o4;
          }
        }
        if (!ok[k] && sub == 0 && dev_flag != nullptr) atomicMin(dev_flag, (int32_t)min(t[k], (int64_t)INT32_MAX));
      }
    }
  }
}

template <typename T, int WORDS>
static void launch_gather_ln_w(int lanes, int blocks, const uint4* tb, int64_t V, int row_vec, int d, float eps,
                               const int32_t* ids, int64_t total, uint4* o, int32_t* dev_flag, cudaStream_t st) {
  switch (lanes) {
    case 32: launch_pdl(k_gather_ln<T, 32, WORDS>, dim3((unsigned)blocks), dim3(256), 0, st, tb, V, row_vec, d, eps, ids, total, o, dev_flag); break;
    case 16: launch_pdl(k_gather_ln<T, 16, WORDS>, dim3((unsigned)blocks), dim3(256), 0, st, tb, V, row_vec, d, eps, ids, total, o, dev_flag); break;
    case 8:  launch_pdl(k_gather_ln<T, 8, WORDS>, dim3((unsigned)blocks), dim3(256), 0, st, tb, V, row_vec, d, eps, ids, total, o, dev_flag); break;
    default: launch_pdl(k_gather_ln<T, 4, WORDS>, dim3((unsigned)blocks), dim3(256), 0, st, tb, V, row_vec, d, eps, ids, total, o, dev_flag); break;
  }
}
template <typename T>
static lime_status launch_gather_ln_t(int lanes, int words, int blocks, const uint4* tb, int64_t V, int row_vec, int d, float eps,
                                      const int32_t* ids, int64_t total, uint4* o, int32_t* dev_flag, cudaStream_t st) {
  if (words <= 1) launch_gather_ln_w<T, 1>(lanes, blocks, tb, V, row_vec, d, eps, ids, total, o, dev_flag, st);
  else if (words <= 2) launch_gather_ln_w<T, 2>(lanes, blocks, tb, V, row_vec, d, eps, ids, total, o, dev_flag, st);
  else if (words <= 4) launch_gather_ln_w<T, 4>(lanes, blocks, tb, V, row_vec, d, eps, ids, total, o, dev_flag, st);
  else if (words <= 8) launch_gather_ln_w<T, 8>(lanes, blocks, tb, V, row_vec, d, eps, ids, total, o, dev_flag, st);
  else return LIME_UNSUPPORTED_SHAPE;                                  // d <= 1024 keeps a row within 32 lanes x 8 words
  return LIME_OK;
}

lime_status launch_gather_ln(int dtype, const void* table, int64_t V, int d, float eps, const int32_t* ids, int64_t total,
                             void* out, int32_t* dev_flag, cudaStream_t st) {
  if (total == 0) return LIME_OK;
  const int es = dtype == LIME_F32 ? 4 : 2;
  const int row_vec = d * es / 16;
  // two words per lane where the row allows: half the shuffle steps and two independent loads per thread
  int lanes = row_vec >= 64 ? 32 : (row_vec >= 32 ? 16 : (row_vec >= 16 ? 8 : 4));
  const int words = (row_vec + lanes - 1) / lanes;
  const int rows_per_block = 256 / lanes;
  int64_t blocks = (total + rows_per_block - 1) / rows_per_block;
  const int64_t cap = (int64_t)kSMs * 16;
  if (blocks > cap) blocks = cap;
  ProfScope _p("k_gather_ln", st);
  const lime_status s =
      dtype == LIME_F32
          ? launch_gather_ln_t<float>(lanes, words, (int)blocks, (const uint4*)table, V, row_vec, d, eps, ids, total, (uint4*)out, dev_flag, st)
          : launch_gather_ln_t<__nv_bfloat16>(lanes, words, (int)blocks, (const uint4*)table, V, row_vec, d, eps, ids, total, (uint4*)out,
                                              dev_flag, st);
  if (s != LIME_OK) return s;
  LIME_LAUNCH_CHECK("k_gather_ln");
  return LIME_OK;
}

lime_status launch_gather(int dtype, const void* table, int64_t V, int d, const int32_t* ids, int64_t total,
                          void* out, int32_t* dev_flag, cudaStream_t st) {
  if (total == 0) return LIME_OK;
  const int es = dtype == LIME_F32 ? 4 : 2;
  const int row_vec = d * es / 16;
  const int threads = 256;
  // enough lanes per row that each thread moves 1-2 words
  int lanes = row_vec >= 32 ? 32 : (row_vec >= 16 ? 16 : (row_vec >= 8 ? 8 : 4));
  const int rows_per_block = threads / lanes;
  int64_t blocks = (total + rows_per_block - 1) / rows_per_block;
  const int64_t cap = (int64_t)kSMs * 16;
  if (blocks > cap) blocks = cap;
  ProfScope _p("k_gather", st);
  const uint4* tb = (const uint4*)table;
  uint4* o = (uint4*)out;
  switch (lanes) {
    case 32: k_gather<32><<<(int)blocks, threads, 0, st>>>(tb, V, row_vec, ids, total, o, dev_flag); break;
    case 16: k_gather<16><<<(int)blocks, threads, 0, st>>>(tb, V, row_vec, ids, total, o, dev_flag); break;
    case 8:  k_gather<8><<<(int)blocks, threads, 0, st>>>(tb, V, row_vec, ids, total, o, dev_flag); break;
    default: k_gather<4><<<(int)blocks, threads, 0, st>>>(tb, V, row_vec, ids, total, o, dev_flag); break;
  }
  LIME_LAUNCH_CHECK("k_gather");
  return LIME_OK;
}

// ----------------------------------------------------------------------------- elementwise helpers
template <typename T>
__global__ void k_cast_rows(const float* __restrict__ in, int64_t n, T* __restrict__ out) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
    Store<T>::st(out + i, in[i]);
}
template <typename T>
__global__ void k_widen(const T* __restrict__ in, int64_t n, float* __restrict__ out) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
    out[i] = Store<T>::ld(in + i);
}
__global__ void k_axpy(const float* __restrict__ x, float* __restrict__ y, int64_t n, int zero_first) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
    y[i] = (zero_first ? 0.0f : y[i]) + x[i];
}

// Link states of the per-head candidate side (Eq. 1 applied to Eq. 4): row (h, l) of a user is L^P row l on head h's
// columns and zero elsewhere, so that the full-width dot <T_c, row (h, l)> is head h's dot product.
template <typename T>
__global__ void k_expand_heads(const float* __restrict__ src, int64_t n_out, int ell, int d, int heads, T* __restrict__ out) {
  const int dh = d / heads;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_out; i += (int64_t)gridDim.x * blockDim.x) {
    const int j = (int)(i % d);
    const int64_t row = i / d;                       // (user, head, link)
    const int l = (int)(row % ell), h = (int)((row / ell) % heads);
    const int64_t b = row / ((int64_t)ell * heads);
    Store<T>::st(out + i, j / dh == h ? src[(b * ell + l) * d + j] : 0.f);
  }
}

static inline int ew_blocks(int64_t n) {
  int64_t b = (n + 255) / 256;
  const int64_t cap = (int64_t)kSMs * 8;
  return (int)(b > cap ? cap : (b < 1 ? 1 : b));
}

lime_status launch_expand_heads(const float* src, int64_t rows_in, int ell, int d, int heads, void* out, int dtype,
                                cudaStream_t st) {
  const int64_t n_out = rows_in * heads * d;
  if (n_out == 0) return LIME_OK;
  ProfScope _p("k_expand_heads", st);
  if (dtype == LIME_F32) k_expand_heads<float><<<ew_blocks(n_out), 256, 0, st>>>(src, n_out, ell, d, heads, (float*)out);
  else k_expand_heads<__nv_bfloat16><<<ew_blocks(n_out), 256, 0, st>>>(src, n_out, ell, d, heads, (__nv_bfloat16*)out);
  LIME_LAUNCH_CHECK("k_expand_heads");
  return LIME_OK;
}

lime_status launch_cast_rows(const float* in, int64_t n, void* out, int dtype, cudaStream_t st) {
  if (n == 0) return LIME_OK;
  ProfScope _p("k_cast_rows", st);
  if (dtype == LIME_F32) k_cast_rows<float><<<ew_blocks(n), 256, 0, st>>>(in, n, (float*)out);
  else k_cast_rows<__nv_bfloat16><<<ew_blocks(n), 256, 0, st>>>(in, n, (__nv_bfloat16*)out);
  LIME_LAUNCH_CHECK("k_cast_rows");
  return LIME_OK;
}
lime_status launch_widen(const void* in, int dtype, float* out, int64_t n, cudaStream_t st) {
  if (n == 0) return LIME_OK;
  ProfScope _p("k_widen", st);
  if (dtype == LIME_F32) k_widen<float><<<ew_blocks(n), 256, 0, st>>>((const float*)in, n, out);
  else k_widen<__nv_bfloat16><<<ew_blocks(n), 256, 0, st>>>((const __nv_bfloat16*)in, n, out);
  LIME_LAUNCH_CHECK("k_widen");
  return LIME_OK;
}
lime_status launch_axpy(const float* x, float* y, int64_t n, int zero_first, cudaStream_t st) {
  if (n == 0) return LIME_OK;
  ProfScope _p("k_axpy", st);
  k_axpy<<<ew_blocks(n), 256, 0, st>>>(x, y, n, zero_first);
  LIME_LAUNCH_CHECK("k_axpy");
  return LIME_OK;
}

}  // namespace lime
