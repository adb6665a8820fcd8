// Host-side helpers of the tensor-core kernels: TMA tensor-map encoding through the driver entry point
// (resolved at run time, so the library does not link against libcuda).
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdlib>

#include "lime_common.cuh"
#include "tc_common.cuh"

namespace lime {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

bool make_tmap_bf16_sw128(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint64_t pitch_elems,
                          uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn || rows == 0 || cols < 64 || box_rows == 0 || box_rows > 256) return false;
  if ((reinterpret_cast<uintptr_t>(base) & 15u) || (pitch_elems * 2) % 16) return false;
  const cuuint64_t gdim[2] = {cols, rows};
  const cuuint64_t gstride[1] = {pitch_elems * 2};
  const cuuint32_t box[2] = {64, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_tmap_bf16_kmajor(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint64_t pitch_elems,
                           uint32_t box_rows, uint32_t box_cols) {
  EncodeTiledFn fn = encode_fn();
  if (!fn || rows == 0 || box_rows == 0 || box_rows > 256 || cols < box_cols) return false;
  if (box_cols != 64 && box_cols != 32 && box_cols != 16) return false;
  if ((reinterpret_cast<uintptr_t>(base) & 15u) || (pitch_elems * 2) % 16) return false;
  const cuuint64_t gdim[2] = {cols, rows};
  const cuuint64_t gstride[1] = {pitch_elems * 2};
  const cuuint32_t box[2] = {box_cols, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUtensorMapSwizzle sw = box_cols == 64 ? CU_TENSOR_MAP_SWIZZLE_128B
                                               : (box_cols == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
  return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool pdl_enabled() {
  static const bool on = [] {
    const char* e = std::getenv("LIME_PDL");
    return !(e != nullptr && e[0] == '0');
  }();
  return on;
}

lime_status ensure_dynamic_smem(const void* kernel, int bytes, bool (&done)[kMaxDeviceOrdinals]) {
  int dev = 0;
  LIME_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDeviceOrdinals) return LIME_INVALID_ARG;
  if (!done[dev]) {
    LIME_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    done[dev] = true;
  }
  return LIME_OK;
}

// Same matrix, box [box_rows x cols] covering whole rows, no swizzle (rows land back to back in shared memory).
bool make_tmap_bf16_plain(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint64_t pitch_elems,
                          uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn || rows == 0 || cols == 0 || cols > 256 || (cols * 2) % 16 || box_rows == 0 || box_rows > 256) return false;
  if ((reinterpret_cast<uintptr_t>(base) & 15u) || (pitch_elems * 2) % 16) return false;
  const cuuint64_t gdim[2] = {cols, rows};
  const cuuint64_t gstride[1] = {pitch_elems * 2};
  const cuuint32_t box[2] = {(cuuint32_t)cols, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Self-test of the bounded waits: one thread waits on an mbarrier that nothing ever arrives at; after `limit_ns` the
// wait gives up, records `code` in the status word and the kernel returns.
__global__ void k_wait_expiry(int* err, unsigned long long limit_ns, int code) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    tc::mbar_init(&bar, 1);
    tc::fence_barrier_init();
    tc::mbar_wait_limit(&bar, 0, err, code, limit_ns);
  }
}

lime_status launch_wait_expiry(int* err, uint64_t limit_ns, int code, cudaStream_t st) {
  ProfScope _p("k_wait_expiry", st);
  k_wait_expiry<<<1, 32, 0, st>>>(err, (unsigned long long)limit_ns, code);
  LIME_LAUNCH_CHECK("k_wait_expiry");
  return LIME_OK;
}

}  // namespace lime
