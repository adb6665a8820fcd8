// Allocation-free variant of the offline candidate->link precompute.
//
// Some hosts of this library may not allocate device memory once they are running: a serving process whose memory
// pool was sized and frozen at start-up, or code that runs under a framework that owns the allocator and forbids
// cudaMalloc outside it.  Such callers cannot use lime_create (it allocates the context's device buffers), so this
// entry point takes the model shape and the weight pointers directly and keeps its only scratch - the effective
// link keys (L W_K)(W_Q)^T of Eq. 4 and the intermediate L W_K - in a fixed array that is part of the library image.
#include "lime_common.cuh"

namespace lime {

// keff [ell x d] followed by the stage-1 intermediate [ell x d], fp32.  Every GPU that loads the library holds
// these 128 KB until the process exits.
static __device__ __align__(256) float g_noalloc_scratch[2 * LIME_NOALLOC_MAX_LINK_ELEMS];

constexpr int kMaxDevices = 64;
static float* g_scratch_ptr[kMaxDevices] = {nullptr};

// In host code `g_noalloc_scratch` is only a handle for the runtime, not an address a kernel may use: the device
// address is looked up once per device (with that device current) and cached.
static lime_status scratch_for_current_device(float** out) {
  int dev = -1;
  LIME_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return LIME_INVALID_ARG;
  if (g_scratch_ptr[dev] == nullptr) {
    float* p = nullptr;
    LIME_CUDA(cudaGetSymbolAddress((void**)&p, g_noalloc_scratch));
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return LIME_OK;
}

}  // namespace lime

using namespace lime;

extern "C" lime_status lime_precompute_candidate_links_noalloc(int32_t dtype, int32_t d, int32_t ell, float cand_scale,
                                                               const void* links, const void* cand_Wq,
                                                               const void* cand_Wk, const void* cand_emb, int64_t M,
                                                               void* out_w, void* stream) {
  if (dtype != LIME_F32 && dtype != LIME_BF16) return LIME_INVALID_ARG;
  if (d <= 0 || ell <= 0 || M < 0 || cand_scale < 0.f) return LIME_INVALID_ARG;
  if (d % 8 || ell > 256 || d > 1024) return LIME_UNSUPPORTED_SHAPE;
  if ((int64_t)ell * d > LIME_NOALLOC_MAX_LINK_ELEMS) {
    cuda_fail(cudaErrorInvalidValue, "lime_precompute_candidate_links_noalloc: ell*d exceeds LIME_NOALLOC_MAX_LINK_ELEMS");
    return LIME_EXCEEDS_STATIC_SCRATCH;
  }
  if (!links || (M > 0 && (!cand_emb || !out_w))) return LIME_INVALID_ARG;
  const void* ps[6] = {links, cand_Wq, cand_Wk, cand_emb, out_w, nullptr};
  for (const void* p : ps)
    if (reinterpret_cast<uintptr_t>(p) & 15u) return LIME_INVALID_ARG;
  float* scratch = nullptr;
  lime_status s = scratch_for_current_device(&scratch);
  if (s != LIME_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const float scale = cand_scale > 0.f ? cand_scale : 1.0f / sqrtf((float)d);
  // both halves of the scratch are fully rewritten before they are read, so nothing has to start at zero
  if ((s = launch_keff(dtype, links, cand_Wk, cand_Wq, ell, d, 1, scale, scratch, st)) != LIME_OK) return s;
  return launch_precompute(dtype, cand_emb, M, d, ell, ell, scratch, out_w, st);
}
