// Forward kernel: O = softmax(mask(scale Q K^T)) V and LSE over the plan's visible tiles.
//
// One CTA per (query tile, query head).  TMA stages Q once and K/V per key tile in 128-byte
// swizzled shared memory; tcgen05.mma accumulates S = Q K^T and O += P V in tensor memory
// (fp32); each of the 128 threads owns one query row (= one TMEM lane) for the online
// softmax, so row maxima and sums need no cross-thread traffic.  P is rounded to bf16 and
// written back into tensor memory, over the columns S occupied, where the second MMA reads
// it as its A operand.  Two CTAs fit per SM (256 TMEM columns, 96 KB shared memory each), so
// one CTA's softmax overlaps the other's MMAs.
#include "pp_dev.cuh"

namespace pp {
namespace {

struct FwdParams {
  int32_t* header;
  const Tile* tiles;
  const int32_t* order;
  __nv_bfloat16* o;
  float* lse;
  int T, Hq, Hkv;
  float scale_log2;  // softmax scale * log2(e)
};

constexpr int kFwdThreads = 128;
constexpr uint32_t kFwdTmemCols = 256;  // [0,128): S then P (bf16, 64 columns); [128, 128+D): O

template <int D>
struct FwdSmem {
  static constexpr int kTileBytes = 128 * D * 2;
  static constexpr int kQ = 0, kK = kTileBytes, kV = 2 * kTileBytes, kBars = 3 * kTileBytes;
  static constexpr int kTotal = kBars + 64 + 1024;  // + slack to align the base to 1024 B
};

template <int D>
__global__ void __launch_bounds__(kFwdThreads)
fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
           const __grid_constant__ CUtensorMap tm_v, FwdParams prm) {
  using L = FwdSmem<D>;
  extern __shared__ uint8_t smem_raw[];
  const int tid = threadIdx.x, warp = tid >> 5;

  if (prm.header[0] != kStatusOk) return;
  const int ord = blockIdx.x / prm.Hq, h = blockIdx.x % prm.Hq;
  if (ord >= prm.header[2]) return;
  const Tile tile = prm.tiles[prm.order[ord]];
  const int kvh = h / (prm.Hq / prm.Hkv);

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sQ = base + L::kQ, sK = base + L::kK, sV = base + L::kV;
  const uint32_t bar_q = base + L::kBars, bar_kv = bar_q + 8, bar_s = bar_q + 16,
                 bar_o = bar_q + 24, tmem_slot = bar_q + 32;
  uint8_t* gbase = smem_raw + (base - smem_u32(smem_raw));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gbase + L::kBars + 40);
  volatile uint32_t* tmem_slot_p = reinterpret_cast<volatile uint32_t*>(gbase + L::kBars + 32);

  if (tid == 0) {
    mbar_init(bar_q, 1);
    mbar_init(bar_kv, 1);
    mbar_init(bar_s, 1);
    mbar_init(bar_o, 1);
    *abort_flag = 0;
    fence_mbar_init();
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_k);
    tma_prefetch_desc(&tm_v);
  }
  if (warp == 0) {
    tmem_alloc(tmem_slot, kFwdTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot_p;
  const uint32_t lane_base = tmem + (uint32_t(warp * 32) << 16);
  const uint32_t tS = 0, tP = 0, tO = 128;

  constexpr uint32_t idesc_s = make_idesc(128, 128, 0, 0);
  constexpr uint32_t idesc_o = make_idesc(128, D, 0, 1);

  if (tid == 0) {
    mbar_expect_tx(bar_q, L::kTileBytes);
    for (int b = 0; b < D / 64; ++b) tma_load_3d(sQ + b * kBoxBytes, &tm_q, b * 64, h, tile.start, bar_q);
  }

  const int n0 = (tile.kv0_len + kTile - 1) / kTile, n1 = (tile.kv1_len + kTile - 1) / kTile;
  const int ntiles = n0 + n1 + 1;
  float m_run = -INFINITY, l_run = 0.f;
  const int row = tid;

  for (int j = 0; j < ntiles; ++j) {
    int k_start, k_len;
    const bool diag = (j == ntiles - 1);
    if (j < n0) {
      k_start = tile.kv0_start + j * kTile;
      k_len = min(kTile, tile.kv0_len - j * kTile);
    } else if (j < n0 + n1) {
      k_start = tile.kv1_start + (j - n0) * kTile;
      k_len = min(kTile, tile.kv1_len - (j - n0) * kTile);
    } else {
      k_start = tile.start;
      k_len = tile.len;
    }
    const uint32_t par = j & 1;

    if (tid == 0) {
      mbar_expect_tx(bar_kv, 2 * L::kTileBytes);
      for (int b = 0; b < D / 64; ++b) {
        tma_load_3d(sK + b * kBoxBytes, &tm_k, b * 64, kvh, k_start, bar_kv);
        tma_load_3d(sV + b * kBoxBytes, &tm_v, b * 64, kvh, k_start, bar_kv);
      }
      if (j == 0) wait_bar(bar_q, 0, abort_flag, prm.header, 1);
      wait_bar(bar_kv, par, abort_flag, prm.header, 2);
      tc_fence_after();
#pragma unroll
      for (int k = 0; k < D / 16; ++k)
        mma_ss(tmem + tS, kmajor_desc(sQ, k), kmajor_desc(sK, k), idesc_s, k > 0);
      mma_commit(bar_s);
    }
    wait_bar(bar_s, par, abort_flag, prm.header, 3);
    tc_fence_after();

    // ---- online softmax on this thread's row (base-2 exponentials)
    uint32_t v[32];
    float mx = m_run;
    const int col_lim = diag ? min(k_len, row + 1) : k_len;  // columns [0, col_lim) are visible
#pragma unroll 1
    for (int c = 0; c < 4; ++c) {
      tmem_ld32(lane_base + tS + c * 32, v);
      tmem_wait_ld();
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        float s = __uint_as_float(v[i]) * prm.scale_log2;
        if (c * 32 + i < col_lim) mx = fmaxf(mx, s);
      }
    }
    const float alpha = ex2(m_run - mx);
    float rs = 0.f;
#pragma unroll 1
    for (int c = 0; c < 4; ++c) {
      tmem_ld32(lane_base + tS + c * 32, v);
      tmem_wait_ld();
      uint32_t pk[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        int c0 = c * 32 + 2 * i;
        float p0 = ex2(__uint_as_float(v[2 * i]) * prm.scale_log2 - mx);
        float p1 = ex2(__uint_as_float(v[2 * i + 1]) * prm.scale_log2 - mx);
        p0 = (c0 < col_lim) ? p0 : 0.f;
        p1 = (c0 + 1 < col_lim) ? p1 : 0.f;
        rs += p0 + p1;
        pk[i] = pack_bf16(p0, p1);
      }
      tmem_st16(lane_base + tP + c * 16, pk);
    }
    l_run = l_run * alpha + rs;
    m_run = mx;
    if (j > 0) {
#pragma unroll 1
      for (int c = 0; c < D / 32; ++c) {
        tmem_ld32(lane_base + tO + c * 32, v);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * alpha);
        tmem_st32(lane_base + tO + c * 32, v);
      }
    }
    tmem_wait_st();
    tc_fence_before();
    __syncthreads();

    if (tid == 0) {
      tc_fence_after();
      const int ksteps = (k_len + 15) / 16;
      for (int k = 0; k < ksteps; ++k)
        mma_ts(tmem + tO, tmem + tP + k * 8, mnmajor_desc(sV, k), idesc_o, (j > 0) || (k > 0));
      mma_commit(bar_o);
    }
    wait_bar(bar_o, par, abort_flag, prm.header, 4);
    tc_fence_after();
  }

  // ---- epilogue: normalise, round to bf16, store this thread's row; LSE in natural log
  const float inv_l = 1.f / l_run;
  if (row < tile.len) {
    const size_t tok = size_t(tile.start) + row;
    prm.lse[size_t(h) * prm.T + tok] = (m_run + log2f(l_run)) * 0.69314718055994531f;
  }
#pragma unroll 1
  for (int c = 0; c < D / 32; ++c) {
    uint32_t v[32];
    tmem_ld32(lane_base + tO + c * 32, v);
    tmem_wait_ld();
    if (row < tile.len) {
      uint4* dst = reinterpret_cast<uint4*>(prm.o + ((size_t(tile.start) + row) * prm.Hq + h) * D + c * 32);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        uint4 w;
        w.x = pack_bf16(__uint_as_float(v[8 * i + 0]) * inv_l, __uint_as_float(v[8 * i + 1]) * inv_l);
        w.y = pack_bf16(__uint_as_float(v[8 * i + 2]) * inv_l, __uint_as_float(v[8 * i + 3]) * inv_l);
        w.z = pack_bf16(__uint_as_float(v[8 * i + 4]) * inv_l, __uint_as_float(v[8 * i + 5]) * inv_l);
        w.w = pack_bf16(__uint_as_float(v[8 * i + 6]) * inv_l, __uint_as_float(v[8 * i + 7]) * inv_l);
        dst[i] = w;
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kFwdTmemCols);
}

template <int D>
cudaError_t launch_fwd_t(const pp_plan* plan, const CUtensorMap& tq, const CUtensorMap& tk,
                         const CUtensorMap& tv, const FwdParams& prm, cudaStream_t stream) {
  static bool configured = false;
  auto kern = fwd_kernel<D>;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         FwdSmem<D>::kTotal);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  dim3 grid(unsigned(plan->max_tiles) * unsigned(plan->prob.num_q_heads));
  ProfileEvents& ev = profile_events();
  if (ev.on) cudaEventRecord(ev.fwd0, stream);
  kern<<<grid, kFwdThreads, FwdSmem<D>::kTotal, stream>>>(tq, tk, tv, prm);
  if (ev.on) {
    cudaEventRecord(ev.fwd1, stream);
    ev.fwd_valid = true;
  }
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_fwd(const pp_plan* plan, const void* q, const void* k, const void* v, float scale,
                       void* o, float* lse, cudaStream_t stream, int* launches) {
  const pp_problem& pb = plan->prob;
  CUtensorMap tq, tk, tv;
  if (!encode_thd(&tq, q, pb.total_tokens, pb.num_q_heads, pb.head_dim, kTile) ||
      !encode_thd(&tk, k, pb.total_tokens, pb.num_kv_heads, pb.head_dim, kTile) ||
      !encode_thd(&tv, v, pb.total_tokens, pb.num_kv_heads, pb.head_dim, kTile))
    return cudaErrorNotSupported;
  FwdParams prm;
  prm.header = reinterpret_cast<int32_t*>(plan->ws + plan->lay.header);
  prm.tiles = reinterpret_cast<const Tile*>(plan->ws + plan->lay.tiles);
  prm.order = reinterpret_cast<const int32_t*>(plan->ws + plan->lay.fwd_order);
  prm.o = static_cast<__nv_bfloat16*>(o);
  prm.lse = lse;
  prm.T = pb.total_tokens;
  prm.Hq = pb.num_q_heads;
  prm.Hkv = pb.num_kv_heads;
  prm.scale_log2 = scale * 1.4426950408889634f;
  cudaError_t e = pb.head_dim == 128 ? launch_fwd_t<128>(plan, tq, tk, tv, prm, stream)
                                     : launch_fwd_t<64>(plan, tq, tk, tv, prm, stream);
  if (e == cudaSuccess && launches) *launches += 1;
  return e;
}

}  // namespace pp
