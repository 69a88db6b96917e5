// Device helpers shared by the forward and backward kernels: bounded mbarrier waits,
// host-side TMA descriptor encoding for the token-major [T][H][D] bf16 tensors.
#pragma once
#include <cuda.h>

#include "pp_internal.h"
#include "pp_ptx.cuh"

namespace pp {

constexpr uint32_t kSpinLimit = 1u << 21;  // polls of mbarrier.try_wait before giving up

// Waits for a phase of an mbarrier, but never forever: after kSpinLimit polls the CTA records
// the site in the plan's status word, raises its abort flag (which turns every later wait of
// this CTA into a no-op) and carries on to its normal exit path.
#if defined(PP_TIMING) || defined(PP_CYCLES)
// Developer switches.  -DPP_TIMING: cycles CTA 0 spends in each wait site, summed over lane 0
// of every warp that waits there (the waits lose their fast path, so totals are inflated);
// slot 127 holds CTA 0's total cycles.  -DPP_CYCLES: only the per-CTA total cycles, with the
// kernels otherwise unchanged.
#define PP_DEBUG_COUNTERS 1
static __device__ unsigned long long g_wait_cycles[128];
static __device__ unsigned long long g_cta_cycles[256];  // per-CTA busy cycles
#endif

__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                         int32_t* header, int site, uint32_t limit = kSpinLimit) {
#ifndef PP_TIMING
  if (mbar_try_wait(bar, parity)) return true;  // fast path: already complete
#endif
  if (*abort_flag) return false;
#ifdef PP_TIMING
  const long long t0 = clock64();
#endif
  for (uint32_t it = 0; it < limit; ++it) {
    if (mbar_try_wait(bar, parity)) {
#ifdef PP_TIMING
      if (blockIdx.x == 0 && (threadIdx.x & 31) == 0)
        atomicAdd(&g_wait_cycles[site & 127], (unsigned long long)(clock64() - t0));
#endif
      return true;
    }
    if ((it & 0xfff) == 0xfff && *abort_flag) return false;
  }
  if (atomicCAS(&header[0], kStatusOk, kStatusWaitExpired) == kStatusOk) header[1] = site;
  *abort_flag = 1;
  return false;
}

// ---------------------------------------------------------------- host: tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) !=
            cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// Tensor [T][H][D] bf16 viewed as 3-D (D, H, T); one box = 64 elements of D x 1 head x
// `rows` tokens, 128-byte swizzled: in shared memory row r sits at r * 128 bytes and its
// 16-byte chunks are XOR-ed with (r mod 8).
inline bool encode_thd(CUtensorMap* m, const void* base, int T, int H, int D, int rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {cuuint64_t(D), cuuint64_t(H), cuuint64_t(T)};
  cuuint64_t strides[2] = {cuuint64_t(D) * 2, cuuint64_t(H) * D * 2};
  cuuint32_t box[3] = {64, 1, cuuint32_t(rows)};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box,
            estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// fp32 tensor [T][H][D] for TMA reductions: one box = 32 floats x 1 head x 128 tokens,
// 128-byte swizzled (row r at r * 128 bytes, 16-byte chunks XOR-ed with r mod 8).
inline bool encode_thd_f32(CUtensorMap* m, const void* base, int T, int H, int D) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {cuuint64_t(D), cuuint64_t(H), cuuint64_t(T)};
  cuuint64_t strides[2] = {cuuint64_t(D) * 4, cuuint64_t(H) * D * 4};
  cuuint32_t box[3] = {32, 1, 128};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(base), dims, strides, box,
            estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr uint32_t kBoxBytes = 128 * 128;  // one {64 x 128 rows} bf16 box

// K-major operand descriptor for k-step `k16` (16 elements of the contraction = 32 bytes
// inside a 128-byte row; four steps per box).
__device__ __forceinline__ uint64_t kmajor_desc(uint32_t tile_base, int k16) {
  return make_sdesc(tile_base + (k16 >> 2) * kBoxBytes + (k16 & 3) * 32, 16, 1024);
}
// MN-major operand descriptor for k-step `k16` (16 rows = 2048 bytes); the next 64 elements
// of the M/N index live in the next box.
__device__ __forceinline__ uint64_t mnmajor_desc(uint32_t tile_base, int k16) {
  return make_sdesc(tile_base + k16 * 2048, kBoxBytes, 1024);
}

// Descriptor arithmetic for unrolled k-loops: a descriptor for k-step k16 is the tile's base
// descriptor plus a compile-time constant in its address field (shared-memory addresses stay
// below 2^18, so the 14-bit field cannot overflow).
__device__ __forceinline__ uint64_t kmajor_base(uint32_t tile_base) {
  return make_sdesc(tile_base, 16, 1024);
}
__device__ __forceinline__ uint64_t mnmajor_base(uint32_t tile_base) {
  return make_sdesc(tile_base, kBoxBytes, 1024);
}
__host__ __device__ constexpr uint64_t kmajor_off(int k16) {
  return uint64_t(((k16 >> 2) * kBoxBytes + (k16 & 3) * 32) >> 4);
}
__host__ __device__ constexpr uint64_t mnmajor_off(int k16) { return uint64_t((k16 * 2048) >> 4); }

}  // namespace pp
