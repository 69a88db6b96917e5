// Backward kernels: dQ, dK, dV of preference-packed attention.
//
//   preprocess : Delta_i = sum_d dO_id O_id and LSE * log2(e), per (query head, token)
//   main       : one CTA per (key tile, KV head).  K and V stay in shared memory; dK and dV
//                stay in tensor memory while the CTA walks over every query tile that sees
//                the key tile -- its own diagonal tile, then the contiguous range of later
//                queries (for prompt keys: the rest of the prompt and every response) -- and
//                over the query heads sharing the KV head.  So the prompt keys' gradients
//                gather all responses' contributions inside one accumulator, with no atomics.
//                Per query tile: S^T = K Q^T and dP^T = V dO^T (tensor memory), P^T =
//                exp2(S^T - LSE), dS^T = P^T (dP^T - Delta) in registers (thread = key row),
//                dV += P^T dO, dK += dS^T Q, dQ_tile = dS K.  Only dQ leaves the CTA per tile:
//                it is added into an fp32 accumulator with vector reductions.
//   finalize   : dQ = bf16(scale * accumulator)
#include <algorithm>
#include <mutex>

#include "pp_dev.cuh"

namespace pp {
namespace {

struct BwdParams {
  int32_t* header;
  const Tile* tiles;
  const int32_t* order;
  const float* delta;  // [Hq][T]
  const float* lse2;   // [Hq][T]  LSE * log2(e)
  float* dq_acc;       // [T][Hq][D] fp32
  __nv_bfloat16* dk;
  __nv_bfloat16* dv;
  int T, Hq, Hkv;
  float scale, scale_log2;
};

// ---------------------------------------------------------------- preprocess
template <int D>
__global__ void __launch_bounds__(256)
bwd_preprocess_kernel(const __nv_bfloat16* __restrict__ o, const __nv_bfloat16* __restrict__ d_o,
                      const float* __restrict__ lse, float* __restrict__ delta,
                      float* __restrict__ lse2, int T, int Hq) {
  const int lane = threadIdx.x & 31;
  const long long idx = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (idx >= (long long)T * Hq) return;
  const int t = int(idx / Hq), h = int(idx % Hq);
  constexpr int kPer = D / 32;  // elements per lane: 4 (D=128) or 2 (D=64)
  const __nv_bfloat16* po = o + idx * D + lane * kPer;
  const __nv_bfloat16* pd = d_o + idx * D + lane * kPer;
  float acc = 0.f;
#pragma unroll
  for (int i = 0; i < kPer; i += 2) {
    float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(po + i));
    float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(pd + i));
    acc += a.x * b.x + a.y * b.y;
  }
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, s);
  if (lane == 0) {
    delta[size_t(h) * T + t] = acc;
    lse2[size_t(h) * T + t] = lse[size_t(h) * T + t] * 1.4426950408889634f;
  }
}

// ---------------------------------------------------------------- finalize
__global__ void __launch_bounds__(256)
bwd_finalize_kernel(const float4* __restrict__ acc, uint2* __restrict__ dq, size_t n4, float scale) {
  size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x;
  const size_t stride = size_t(gridDim.x) * blockDim.x;
  for (; i < n4; i += stride) {
    float4 a = acc[i];
    uint2 w;
    w.x = pack_bf16(a.x * scale, a.y * scale);
    w.y = pack_bf16(a.z * scale, a.w * scale);
    dq[i] = w;
  }
}

// ---------------------------------------------------------------- main
constexpr int kBwdThreads = 128;
constexpr uint32_t kBwdTmemCols = 512;  // S^T/P^T [0,128) | dP^T/dQ [128,256) | dV [256,..) | dK [384,..)

template <int D>
struct BwdSmem {
  static constexpr int kTileBytes = 128 * D * 2;
  static constexpr int kK = 0, kV = kTileBytes, kQ = 2 * kTileBytes, kdO = 3 * kTileBytes,
                       kdS = 4 * kTileBytes, kLse = kdS + 128 * 128 * 2, kDelta = kLse + 512,
                       kBars = kDelta + 512;
  static constexpr int kTotal = kBars + 64 + 1024;
};

template <int D>
__global__ void __launch_bounds__(kBwdThreads)
bwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
           const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
           BwdParams prm) {
  using L = BwdSmem<D>;
  extern __shared__ uint8_t smem_raw[];
  const int tid = threadIdx.x, warp = tid >> 5;

  if (prm.header[0] != kStatusOk) return;
  const int ord = blockIdx.x / prm.Hkv, kvh = blockIdx.x % prm.Hkv;
  if (ord >= prm.header[2]) return;
  const Tile tile = prm.tiles[prm.order[ord]];
  const int r = prm.Hq / prm.Hkv;

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gbase = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sK = base + L::kK, sV = base + L::kV, sQ = base + L::kQ, sdO = base + L::kdO,
                 sdS = base + L::kdS;
  float* sLse = reinterpret_cast<float*>(gbase + L::kLse);
  float* sDelta = reinterpret_cast<float*>(gbase + L::kDelta);
  const uint32_t bar_kv = base + L::kBars, bar_ld = bar_kv + 8, bar_s = bar_kv + 16,
                 bar_d = bar_kv + 24, tmem_slot = bar_kv + 32;
  volatile uint32_t* tmem_slot_p = reinterpret_cast<volatile uint32_t*>(gbase + L::kBars + 32);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gbase + L::kBars + 40);

  if (tid == 0) {
    mbar_init(bar_kv, 1);
    mbar_init(bar_ld, 1);
    mbar_init(bar_s, 1);
    mbar_init(bar_d, 1);
    *abort_flag = 0;
    fence_mbar_init();
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_k);
    tma_prefetch_desc(&tm_v);
    tma_prefetch_desc(&tm_do);
  }
  if (warp == 0) {
    tmem_alloc(tmem_slot, kBwdTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot_p;
  const uint32_t lane_base = tmem + (uint32_t(warp * 32) << 16);
  constexpr uint32_t tS = 0, tP = 0, tdP = 128, tdQ = 128, tdV = 256, tdK = 384;

  constexpr uint32_t idesc_st = make_idesc(128, 128, 0, 0);  // S^T, dP^T : K-major x K-major
  constexpr uint32_t idesc_kv = make_idesc(128, D, 0, 1);    // dV, dK    : K-major A, MN-major B
  constexpr uint32_t idesc_dq = make_idesc(128, D, 1, 1);    // dQ        : MN-major A and B

  const int k_start = tile.start, k_len = tile.len;
  if (tid == 0) {
    mbar_expect_tx(bar_kv, 2 * L::kTileBytes);
    for (int b = 0; b < D / 64; ++b) {
      tma_load_3d(sK + b * kBoxBytes, &tm_k, b * 64, kvh, k_start, bar_kv);
      tma_load_3d(sV + b * kBoxBytes, &tm_v, b * 64, kvh, k_start, bar_kv);
    }
  }

  const int full_len = tile.vis_end - (k_start + k_len);
  const int nq = 1 + (full_len + kTile - 1) / kTile;
  const int lane = tid;  // TMEM lane = key row (S^T, dP^T, dK, dV) or query row (dQ)

  int it = 0;
  for (int hh = 0; hh < r; ++hh) {
    const int h = kvh * r + hh;
    for (int qt = 0; qt < nq; ++qt, ++it) {
      const bool diag = (qt == 0);
      const int q_start = diag ? k_start : k_start + k_len + (qt - 1) * kTile;
      const int q_len = diag ? k_len : min(kTile, tile.vis_end - q_start);
      const uint32_t par = it & 1;

      if (tid == 0) {
        mbar_expect_tx(bar_ld, 2 * L::kTileBytes);
        for (int b = 0; b < D / 64; ++b) {
          tma_load_3d(sQ + b * kBoxBytes, &tm_q, b * 64, h, q_start, bar_ld);
          tma_load_3d(sdO + b * kBoxBytes, &tm_do, b * 64, h, q_start, bar_ld);
        }
      }
      // per-query statistics of this tile; +inf LSE switches off queries past the tile's end
      sLse[tid] = tid < q_len ? prm.lse2[size_t(h) * prm.T + q_start + tid] : INFINITY;
      sDelta[tid] = tid < q_len ? prm.delta[size_t(h) * prm.T + q_start + tid] : 0.f;

      if (tid == 0) {
        if (it == 0) wait_bar(bar_kv, 0, abort_flag, prm.header, 11);
        wait_bar(bar_ld, par, abort_flag, prm.header, 12);
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < D / 16; ++k)
          mma_ss(tmem + tS, kmajor_desc(sK, k), kmajor_desc(sQ, k), idesc_st, k > 0);
#pragma unroll
        for (int k = 0; k < D / 16; ++k)
          mma_ss(tmem + tdP, kmajor_desc(sV, k), kmajor_desc(sdO, k), idesc_st, k > 0);
        mma_commit(bar_s);
      }
      __syncthreads();  // sLse / sDelta visible
      wait_bar(bar_s, par, abort_flag, prm.header, 13);
      tc_fence_after();

      const bool row_ok = lane < k_len;
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        uint32_t v[32];
        float p[32];
        tmem_ld32(lane_base + tS + c * 32, v);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int col = c * 32 + i;
          float e = ex2(__uint_as_float(v[i]) * prm.scale_log2 - sLse[col]);
          const bool vis = row_ok && (!diag || col >= lane);
          p[i] = vis ? e : 0.f;
        }
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) pk[i] = pack_bf16(p[2 * i], p[2 * i + 1]);
        tmem_st16(lane_base + tP + c * 16, pk);

        tmem_ld32(lane_base + tdP + c * 32, v);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int col = c * 32 + 2 * i;
          float d0 = p[2 * i] * (__uint_as_float(v[2 * i]) - sDelta[col]);
          float d1 = p[2 * i + 1] * (__uint_as_float(v[2 * i + 1]) - sDelta[col + 1]);
          pk[i] = pack_bf16(d0, d1);
        }
        // dS^T row `lane`, columns [32c, 32c+32): box c/2, 16-byte chunks (c%2)*4 .. +3, swizzled
        const uint32_t row_addr = sdS + (c >> 1) * kBoxBytes + lane * 128;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint32_t chunk = uint32_t((c & 1) * 4 + i) ^ uint32_t(lane & 7);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row_addr + chunk * 16),
                       "r"(pk[4 * i]), "r"(pk[4 * i + 1]), "r"(pk[4 * i + 2]), "r"(pk[4 * i + 3])
                       : "memory");
        }
      }
      tmem_wait_st();
      fence_proxy_async_smem();
      tc_fence_before();
      __syncthreads();

      if (tid == 0) {
        tc_fence_after();
        const int qsteps = (q_len + 15) / 16, ksteps = (k_len + 15) / 16;
        for (int k = 0; k < qsteps; ++k)
          mma_ts(tmem + tdV, tmem + tP + k * 8, mnmajor_desc(sdO, k), idesc_kv, (it > 0) || (k > 0));
        for (int k = 0; k < qsteps; ++k)
          mma_ss(tmem + tdK, kmajor_desc(sdS, k), mnmajor_desc(sQ, k), idesc_kv, (it > 0) || (k > 0));
        for (int k = 0; k < ksteps; ++k)
          mma_ss(tmem + tdQ, mnmajor_desc(sdS, k), mnmajor_desc(sK, k), idesc_dq, k > 0);
        mma_commit(bar_d);
      }
      wait_bar(bar_d, par, abort_flag, prm.header, 14);
      tc_fence_after();

      // dQ tile: lane = query row; add into the fp32 accumulator
#pragma unroll 1
      for (int c = 0; c < D / 32; ++c) {
        uint32_t v[32];
        tmem_ld32(lane_base + tdQ + c * 32, v);
        tmem_wait_ld();
        if (lane < q_len) {
          float* dst = prm.dq_acc + ((size_t(q_start) + lane) * prm.Hq + h) * D + c * 32;
#pragma unroll
          for (int i = 0; i < 8; ++i)
            red_add_v4(dst + 4 * i, __uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1]),
                       __uint_as_float(v[4 * i + 2]), __uint_as_float(v[4 * i + 3]));
        }
      }
      tc_fence_before();
      __syncthreads();
    }
  }

  // ---- epilogue: dK (scaled), dV -> bf16
  tc_fence_after();
#pragma unroll 1
  for (int which = 0; which < 2; ++which) {
    const uint32_t tsrc = which ? tdK : tdV;
    __nv_bfloat16* out = which ? prm.dk : prm.dv;
    const float f = which ? prm.scale : 1.f;
#pragma unroll 1
    for (int c = 0; c < D / 32; ++c) {
      uint32_t v[32];
      tmem_ld32(lane_base + tsrc + c * 32, v);
      tmem_wait_ld();
      if (lane < k_len) {
        uint4* dst = reinterpret_cast<uint4*>(out + ((size_t(k_start) + lane) * prm.Hkv + kvh) * D + c * 32);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          uint4 w;
          w.x = pack_bf16(__uint_as_float(v[8 * i + 0]) * f, __uint_as_float(v[8 * i + 1]) * f);
          w.y = pack_bf16(__uint_as_float(v[8 * i + 2]) * f, __uint_as_float(v[8 * i + 3]) * f);
          w.z = pack_bf16(__uint_as_float(v[8 * i + 4]) * f, __uint_as_float(v[8 * i + 5]) * f);
          w.w = pack_bf16(__uint_as_float(v[8 * i + 6]) * f, __uint_as_float(v[8 * i + 7]) * f);
          dst[i] = w;
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kBwdTmemCols);
}

template <int D>
cudaError_t launch_bwd_t(const pp_plan* plan, const void* o, const float* lse, const void* d_o,
                         void* dq, const CUtensorMap& tq, const CUtensorMap& tk,
                         const CUtensorMap& tv, const CUtensorMap& tdo, const BwdParams& prm,
                         cudaStream_t stream, int* launches) {
  static bool configured = false;
  auto kern = bwd_kernel<D>;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         BwdSmem<D>::kTotal);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  const pp_problem& pb = plan->prob;
  const size_t T = pb.total_tokens, Hq = pb.num_q_heads;
  cudaError_t e = cudaMemsetAsync(prm.dq_acc, 0, 4 * T * Hq * D, stream);
  if (e != cudaSuccess) return e;
  const long long pairs = (long long)T * Hq;
  bwd_preprocess_kernel<D><<<unsigned((pairs + 7) / 8), 256, 0, stream>>>(
      static_cast<const __nv_bfloat16*>(o), static_cast<const __nv_bfloat16*>(d_o), lse,
      const_cast<float*>(prm.delta), const_cast<float*>(prm.lse2), int(T), int(Hq));
  dim3 grid(unsigned(plan->max_tiles) * unsigned(pb.num_kv_heads));
  ProfileEvents& ev = profile_events();
  if (ev.on) cudaEventRecord(ev.bwd0, stream);
  kern<<<grid, kBwdThreads, BwdSmem<D>::kTotal, stream>>>(tq, tk, tv, tdo, prm);
  if (ev.on) {
    cudaEventRecord(ev.bwd1, stream);
    ev.bwd_valid = true;
  }
  const size_t n4 = T * Hq * D / 4;
  unsigned fb = unsigned(std::min<size_t>((n4 + 255) / 256, 148 * 16));
  bwd_finalize_kernel<<<fb, 256, 0, stream>>>(reinterpret_cast<const float4*>(prm.dq_acc),
                                              static_cast<uint2*>(dq), n4, prm.scale);
  if (launches) *launches += 3;
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_bwd(const pp_plan* plan, const void* q, const void* k, const void* v,
                       const void* o, const float* lse, const void* d_o, float scale, void* dq,
                       void* dk, void* dv, void* scratch, cudaStream_t stream, int* launches) {
  const pp_problem& pb = plan->prob;
  CUtensorMap tq, tk, tv, tdo;
  if (!encode_thd(&tq, q, pb.total_tokens, pb.num_q_heads, pb.head_dim, kTile) ||
      !encode_thd(&tk, k, pb.total_tokens, pb.num_kv_heads, pb.head_dim, kTile) ||
      !encode_thd(&tv, v, pb.total_tokens, pb.num_kv_heads, pb.head_dim, kTile) ||
      !encode_thd(&tdo, d_o, pb.total_tokens, pb.num_q_heads, pb.head_dim, kTile))
    return cudaErrorNotSupported;
  BwdScratch sl = bwd_scratch_layout(pb);
  char* sc = static_cast<char*>(scratch);
  BwdParams prm;
  prm.header = reinterpret_cast<int32_t*>(plan->ws + plan->lay.header);
  prm.tiles = reinterpret_cast<const Tile*>(plan->ws + plan->lay.tiles);
  prm.order = reinterpret_cast<const int32_t*>(plan->ws + plan->lay.bwd_order);
  prm.delta = reinterpret_cast<float*>(sc + sl.delta);
  prm.lse2 = reinterpret_cast<float*>(sc + sl.lse2);
  prm.dq_acc = reinterpret_cast<float*>(sc + sl.dq_acc);
  prm.dk = static_cast<__nv_bfloat16*>(dk);
  prm.dv = static_cast<__nv_bfloat16*>(dv);
  prm.T = pb.total_tokens;
  prm.Hq = pb.num_q_heads;
  prm.Hkv = pb.num_kv_heads;
  prm.scale = scale;
  prm.scale_log2 = scale * 1.4426950408889634f;
  return pb.head_dim == 128
             ? launch_bwd_t<128>(plan, o, lse, d_o, dq, tq, tk, tv, tdo, prm, stream, launches)
             : launch_bwd_t<64>(plan, o, lse, d_o, dq, tq, tk, tv, tdo, prm, stream, launches);
}

// ---------------------------------------------------------------- built-in scratch
// Backward scratch for callers that cannot allocate device memory (pp_attn_bwd_noalloc).
// The array is part of the library image: every device that loads the library holds
// kStaticScratchBytes until the process exits, and every call on a device shares it.
static __device__ __align__(256) unsigned char g_static_bwd_scratch[kStaticScratchBytes];

// In host code `g_static_bwd_scratch` is only a stand-in for the symbol, not a device
// address, so the address is looked up once per device (with that device current) and kept.
static cudaError_t static_scratch_address(void** out) {
  constexpr int kMaxDevices = 64;
  static std::mutex mu;
  static void* ptrs[kMaxDevices] = {};
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(mu);
  if (!ptrs[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_bwd_scratch);
    if (e != cudaSuccess) return e;
    if (!p) return cudaErrorInvalidSymbol;
    ptrs[dev] = p;
  }
  *out = ptrs[dev];
  return cudaSuccess;
}

cudaError_t launch_bwd_static(const pp_plan* plan, const void* q, const void* k, const void* v,
                              const void* o, const float* lse, const void* d_o, float scale,
                              void* dq, void* dk, void* dv, cudaStream_t stream, int* launches) {
  void* scratch = nullptr;
  cudaError_t e = static_scratch_address(&scratch);
  if (e != cudaSuccess) return e;
  // launch_bwd zeroes the fp32 dQ accumulator inside the scratch on every call and rewrites
  // Delta and the scaled LSE, so nothing of an earlier call's contents is read.
  return launch_bwd(plan, q, k, v, o, lse, d_o, scale, dq, dk, dv, scratch, stream, launches);
}

}  // namespace pp
