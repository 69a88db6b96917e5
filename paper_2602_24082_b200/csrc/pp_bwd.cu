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

#include <type_traits>

#include "pp_dev.cuh"

namespace pp {
namespace {

struct BwdParams {
  int32_t* header;
  const BTile* tiles;       // the backward's key tiles (cut per group)
  const int32_t* order;
  const int32_t* key_end;   // [T] first query that cannot see key j
  const float* delta;  // [Hq][T]
  const float* lse2;   // [Hq][T]  LSE * log2(e)
  float* dq_acc;       // [T][Hq][D] fp32
  int32_t* dq_sem;     // deterministic variant: turn counters [backward tile][Hq]; else null
  __nv_bfloat16* dk;
  __nv_bfloat16* dv;
  int T, Hq, Hkv;
  float scale, scale_log2;
};

// ---------------------------------------------------------------- preprocess
// Delta = sum_d dO * O per (token, query head) row, the LSE in base-2 units, and the row of
// the fp32 dQ accumulator cleared (so no separate memset pass over it is needed) unless the
// forward has already cleared it (kClear = false).  D / 8 lanes per row with 16-byte loads,
// four row groups per warp in flight: the pass is a pure stream over O and dO.  The rows
// [T][Hq] and the statistics [Hq][T] are transposed to each other, so one side is strided:
// kTokenMajor walks memory order (contiguous O / dO, scattered 4-byte statistics), otherwise
// rows are walked head by head (contiguous statistics, one row per Hq * D * 2 bytes).  The
// second measured about 5 us faster where a token's heads span 8 KB (Hq = 32, D = 128,
// T = 9241), the first about 60 us faster at 16 KB (Hq = 64, T = 16384); the launcher picks by
// that size.
// lanes that share a row: D / 8 (16 bytes of bf16 per lane), rounded up to a power of two
__host__ __device__ constexpr int pre_lanes(int d) { return d == 96 ? 16 : d / 8; }

template <int D, bool kClear, bool kTokenMajor>
__global__ void __launch_bounds__(256)
bwd_preprocess_kernel(const __nv_bfloat16* __restrict__ o, const __nv_bfloat16* __restrict__ d_o,
                      const float* __restrict__ lse, float* __restrict__ delta,
                      float* __restrict__ lse2, float* __restrict__ dq_acc, int T, int Hq) {
  constexpr int kLanes = pre_lanes(D);    // lanes per row (D / 8 of them hold data)
  constexpr int kRows = 32 / kLanes;      // rows per warp and step
  constexpr int kUnroll = 4;
  const int lane = threadIdx.x & 31, sub = lane % kLanes, rin = lane / kLanes;
  const long long rows = (long long)T * Hq;
  const long long warp0 = ((long long)blockIdx.x * 8 + (threadIdx.x >> 5)) * (kRows * kUnroll);
  const long long stride = (long long)gridDim.x * 8 * (kRows * kUnroll);
  for (long long base = warp0; base < rows; base += stride) {
    uint4 a[kUnroll], b[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      // rows are walked head by head, tokens fastest: the per-row statistics [Hq][T] are then
      // written to consecutive addresses (each O / dO row is one contiguous piece anyway)
      const long long idx = base + u * kRows + rin;
      a[u] = b[u] = make_uint4(0u, 0u, 0u, 0u);
      if (idx < rows && sub < D / 8) {
        long long row = idx;
        if (!kTokenMajor) {
          const int h = int(idx / T), t = int(idx - (long long)h * T);
          row = (long long)t * Hq + h;
        }
        a[u] = reinterpret_cast<const uint4*>(o + row * D)[sub];
        b[u] = reinterpret_cast<const uint4*>(d_o + row * D)[sub];
      }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const long long idx = base + u * kRows + rin;
      const uint32_t aw[4] = {a[u].x, a[u].y, a[u].z, a[u].w}, bw[4] = {b[u].x, b[u].y, b[u].z, b[u].w};
      float acc = 0.f;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 x = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&aw[i]));
        const float2 y = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&bw[i]));
        acc = fmaf(x.x, y.x, fmaf(x.y, y.y, acc));
      }
#pragma unroll
      for (int sft = kLanes / 2; sft > 0; sft >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, sft);
      if (idx < rows) {
        long long row = idx, stat = idx;  // position in [T][Hq] and in [Hq][T]
        if (kTokenMajor) {
          const int t = int(idx / Hq), h = int(idx - (long long)t * Hq);
          stat = (long long)h * T + t;
        } else {
          const int h = int(idx / T), t = int(idx - (long long)h * T);
          row = (long long)t * Hq + h;
        }
        if (kClear && sub < D / 8) {
          float4* z = reinterpret_cast<float4*>(dq_acc + row * D + sub * 8);
          z[0] = make_float4(0.f, 0.f, 0.f, 0.f);
          z[1] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        if (sub == 0) {
          delta[stat] = acc;
          lse2[stat] = lse[stat] * 1.4426950408889634f;
        }
      }
    }
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
// Persistent, warp-specialised CTA (one per SM), 448 threads:
//   warp 0       producer: K, V once per unit; per query tile Q and dO by TMA (two-stage rings)
//                and the tile's LSE*log2(e) / Delta into shared memory
//   warp 1       MMA issuer (one thread)
//   warps 2-5    compute warpgroup 0: thread = key row, query columns 0..63 of the tile
//   warps 6-9    compute warpgroup 1: query columns 64..127
//   warps 10-13  dQ warpgroup: thread = query row; moves each dQ tile from tensor memory
//                through a swizzled shared-memory staging buffer into the fp32 accumulator
//                with TMA reduce-add (whole 128-byte lines per row instead of per-thread
//                16-byte reductions, which saturate the L2 atomic units)
// Tensor-memory map (columns): [0,128) S^T, overwritten by P^T (bf16: columns [0,32) and
// [64,96), each warpgroup inside the columns it has read itself); [128,256) dP^T, then the
// dQ tile; [256,256+D) dV; [384,384+D) dK.
// MMA order per query tile i:  dP(i)  dV(i)  S(i+1)  dQ(i)  dK(i).  The exponentials of tile
// i+1 run under dQ(i), dK(i), dP(i+1); dS(i) is computed under dV(i), S(i+1); the dQ tile is
// drained under dK(i), so the dP/dQ columns are free again when dP(i+1) is issued.
constexpr int kBwdThreads = 448;
constexpr uint32_t kBwdTmemCols = 512;

enum BwdBar : int {
  kKvFull = 0,
  kKvEmpty,
  kQFullB,       // [2]   33 arrivals: TMA transaction + 32 producer lanes (LSE / Delta)
  kQEmptyB = 4,  // [2]
  kDoFull = 6,   // dO is single-buffered: free after dV(i), needed again at dP(i+1)
  kDoEmpty = 8,
  kSFullB = 10,
  kPReady,       // 256
  kDpFull,
  kDsReady,      // 256
  kDqFull,
  kDqDrained,    // 128
  kDkvFull,
  kDkvFree,      // 256
  kSchedFull,    // [2]  unit ids handed from the producer warp to the other roles
  kSchedEmpty = kSchedFull + 2,  // [2]  13 arrivals: MMA thread + 8 compute warps + 4 dQ warps
  kNumBwdBars = kSchedEmpty + 2
};

template <int D>
struct BwdSmem {
  static constexpr int kTileBytes = 128 * D * 2;
  static constexpr int kStageBytes = 128 * 128;  // one {32 floats x 128 rows} box of a dQ tile
  static constexpr int kK = 0, kV = kTileBytes, kQ = 2 * kTileBytes, kdO = 4 * kTileBytes,
                       kStg = 5 * kTileBytes, kdS = kStg + 2 * kStageBytes,
                       kStats = kdS + 128 * 128 * 2, kBars = kStats + 2 * 256 * 4;
  static constexpr int kUsed = kBars + 8 * kNumBwdBars + 32;
  // The declared 1024-byte alignment of the dynamic shared memory leaves no slack to spend at
  // D = 128 (227 KB limit); the kernel checks the base and reports if it is not aligned.
  static constexpr int kTotal = kUsed + (kUsed + 1024 <= 232448 ? 1024 : 0);
};

struct BwdUnit {
  BTile tile;
  int kvh, nq, n_it, tidx;
};

// Units are handed out dynamically: the producer warp draws the next index of the plan's
// longest-work-first order from a global counter whenever the CTA is ready for more (list
// scheduling), and passes it to the other roles through a two-entry shared-memory ring.
// header[5] is that counter, header[7] counts finished CTAs; the last one resets both, so a
// plan can be used by any number of launches without a memset in between.
constexpr int kHdrBwdNext = 5, kHdrBwdDone = 7;

__device__ __forceinline__ bool get_bwd_unit(const BwdParams& prm, int u, int ntiles_total,
                                             BwdUnit& un) {
  if (u < 0 || u >= ntiles_total * prm.Hkv) return false;
  const int packed = prm.order[u];  // (kv head << 24) | backward tile
  un.kvh = packed >> 24;
  un.tidx = packed & 0xffffff;
  un.tile = prm.tiles[un.tidx];
  un.nq = un.tile.work;
  un.n_it = un.nq * (prm.Hq / prm.Hkv);
  return true;
}

// Query tile qt of a unit: tile qt of the group's 128-token grid counted from the key tile
// itself.  Key j of the unit sees query i iff j <= i < key_end[j].
struct QTile {
  int h, start, len;
};

// (query tile, head) position inside a unit, advanced without divisions.  Order: query tiles
// from the key tile itself upwards, and for each query tile all query heads of the KV head
// (the other three combinations of ascending / descending tiles and inner / outer head loop
// measured within 2 % of this one).
struct QIter {
  int hh = 0, qt = 0;
};
__device__ __forceinline__ void q_advance(QIter& s, int heads) {
  if (++s.hh == heads) {
    s.hh = 0;
    ++s.qt;
  }
}
__device__ __forceinline__ QTile q_tile_at(const BwdParams& prm, const BwdUnit& un, const QIter& s) {
  QTile q;
  q.h = un.kvh * (prm.Hq / prm.Hkv) + s.hh;
  q.start = un.tile.start + s.qt * kTile;
  q.len = min(kTile, un.tile.grp_end - q.start);
  return q;
}

// D: head dimension of the shared-memory tiles; DV <= D: head dimension of the tensors in
// global memory (96 in tiles of 128: the TMA loads zero-fill the columns past DV, so only the
// loops over the head dimension, the N of dV / dK / dQ and global addressing know about DV).
template <int D, bool kDet, int DV = D>
__global__ void __launch_bounds__(kBwdThreads, 1)
bwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
           const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
           const __grid_constant__ CUtensorMap tm_dq, BwdParams prm) {
  using L = BwdSmem<D>;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (prm.header[0] != kStatusOk) return;
  const int ntiles_total = prm.header[kHdrNumBTiles];
#ifdef PP_DEBUG_COUNTERS
  const long long t_kernel0 = clock64();
#endif

  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  if (base - raw + L::kUsed > L::kTotal) {  // cannot happen with an aligned base
    if (tid == 0 && atomicCAS(&prm.header[0], kStatusOk, kStatusWaitExpired) == kStatusOk)
      prm.header[1] = 99;
    return;
  }
  uint8_t* gbase = smem_raw + (base - raw);
  const uint32_t sK = base + L::kK, sV = base + L::kV, sQ = base + L::kQ, sdO = base + L::kdO,
                 sdS = base + L::kdS;
  float* stats = reinterpret_cast<float*>(gbase + L::kStats);  // [stage][lse2 128 | delta 128]
  const uint32_t bars = base + L::kBars;
  auto bar = [&](int i) { return bars + 8u * uint32_t(i); };
  const uint32_t tmem_slot = bars + 8 * kNumBwdBars;
  volatile uint32_t* tmem_slot_p = reinterpret_cast<volatile uint32_t*>(gbase + L::kBars + 8 * kNumBwdBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gbase + L::kBars + 8 * kNumBwdBars + 8);

  if (tid == 0) {
    for (int i = 0; i < kNumBwdBars; ++i) {
      uint32_t cnt = 1;
      if (i == kQFullB || i == kQFullB + 1) cnt = 33;
      if (i == kPReady || i == kDsReady || i == kDkvFree) cnt = 256;
      if (i == kDqDrained) cnt = 128;
      if (i == kSchedEmpty || i == kSchedEmpty + 1) cnt = 13;
      mbar_init(bar(i), cnt);
    }
    *abort_flag = 0;
    fence_mbar_init();
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_k);
    tma_prefetch_desc(&tm_v);
    tma_prefetch_desc(&tm_do);
    tma_prefetch_desc(&tm_dq);
  }
  if (warp == 0) {
    tmem_alloc(tmem_slot, kBwdTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot_p;
  constexpr uint32_t tS = 0, tdP = 128, tdV = 256, tdK = 384;
  volatile int* sched = reinterpret_cast<volatile int*>(gbase + L::kBars + 8 * kNumBwdBars + 16);
  // producer warp (all lanes): draw the n-th unit of this CTA and publish it
  auto fetch_unit = [&](uint32_t n) -> int {
    int u = 0;
    if (lane == 0) {
      wait_bar(bar(kSchedEmpty + (n & 1)), ((n >> 1) & 1) ^ 1, abort_flag, prm.header, 90);
      // after a wait has given up, no more work is drawn: an out-of-range id ends every role
      u = *abort_flag ? 0x7fffffff : atomicAdd(&prm.header[kHdrBwdNext], 1);
      sched[n & 1] = u;
      mbar_arrive(bar(kSchedFull + (n & 1)));
    }
    return __shfl_sync(0xffffffffu, u, 0);
  };
  // other roles: read the n-th unit; `whole_warp` = all 32 lanes are calling
  auto take_unit = [&](uint32_t n, bool whole_warp) -> int {
    const bool ok = wait_bar(bar(kSchedFull + (n & 1)), (n >> 1) & 1, abort_flag, prm.header, 91);
    const int u = ok ? sched[n & 1] : 0x7fffffff;
    if (whole_warp) {
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(kSchedEmpty + (n & 1)));
    } else {
      mbar_arrive(bar(kSchedEmpty + (n & 1)));
    }
    return u;
  };

  if (warp == 0) {
    // ------------------------------------------------------------ producer
    uint32_t qc = 0, ucnt = 0;
    BwdUnit un;
    for (; get_bwd_unit(prm, fetch_unit(ucnt), ntiles_total, un); ++ucnt) {
      if (lane == 0) {
        wait_bar(bar(kKvEmpty), (ucnt & 1) ^ 1, abort_flag, prm.header, 50);
        mbar_expect_tx(bar(kKvFull), 2 * L::kTileBytes);
        for (int b = 0; b < D / 64; ++b) {
          tma_load_3d(sK + b * kBoxBytes, &tm_k, b * 64, un.kvh, un.tile.start, bar(kKvFull));
          tma_load_3d(sV + b * kBoxBytes, &tm_v, b * 64, un.kvh, un.tile.start, bar(kKvFull));
        }
      }
      QIter qi;
      for (int it = 0; it < un.n_it && !*abort_flag; ++it, ++qc, q_advance(qi, prm.Hq / prm.Hkv)) {
        const QTile qt = q_tile_at(prm, un, qi);
        const uint32_t st = qc & 1, par = ((qc >> 1) & 1) ^ 1;
        // per-query statistics, fetched before the stage is known to be free and handed on
        // NEGATED (the compute warps add them in packed two-lane instructions);
        // +inf LSE and zero Delta switch off columns past the tile's end
        const size_t row0 = size_t(qt.h) * prm.T + qt.start;
        float r_lse[4], r_del[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int c = lane + 32 * i;
          r_lse[i] = c < qt.len ? prm.lse2[row0 + c] : INFINITY;
          r_del[i] = c < qt.len ? prm.delta[row0 + c] : 0.f;
        }
        wait_bar(bar(kQEmptyB + st), par, abort_flag, prm.header, 51);
        if (lane == 0) {
          mbar_expect_tx(bar(kQFullB + st), L::kTileBytes);
          for (int b = 0; b < D / 64; ++b)
            tma_load_3d(sQ + st * L::kTileBytes + b * kBoxBytes, &tm_q, b * 64, qt.h, qt.start,
                        bar(kQFullB + st));
        }
        float* sl = stats + st * 256;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          sl[lane + 32 * i] = -r_lse[i];
          sl[128 + lane + 32 * i] = -r_del[i];
        }
        mbar_arrive(bar(kQFullB + st));
        if (lane == 0) {
          wait_bar(bar(kDoEmpty), (qc & 1) ^ 1, abort_flag, prm.header, 52);
          mbar_expect_tx(bar(kDoFull), L::kTileBytes);
          for (int b = 0; b < D / 64; ++b)
            tma_load_3d(sdO + b * kBoxBytes, &tm_do, b * 64, qt.h, qt.start, bar(kDoFull));
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t gc = 0, ucnt = 0;
      constexpr uint32_t idesc_kv = make_idesc(128, DV, 0, 1);  // dV, dK : K-major A, MN-major B
      constexpr uint32_t idesc_dq = make_idesc(128, DV, 1, 1);  // dQ     : MN-major A and B
      BwdUnit un;
      const uint64_t dK_k = kmajor_base(sK), dV_k = kmajor_base(sV), dK_mn = mnmajor_base(sK);
      const uint64_t dS_k = kmajor_base(sdS), dS_mn = mnmajor_base(sdS);
      constexpr uint64_t kStageStep = uint64_t(L::kTileBytes >> 4);
      auto issue_s = [&](uint32_t st, int q_len) {
        const uint32_t idesc = make_idesc(128, ((q_len + 15) >> 4) << 4, 0, 0);
        const uint64_t dq_k = kmajor_base(sQ) + st * kStageStep;
#pragma unroll
        for (int k = 0; k < DV / 16; ++k)
          mma_ss(tmem + tS, dK_k + kmajor_off(k), dq_k + kmajor_off(k), idesc, k > 0);
        mma_commit(bar(kSFullB));
      };
      for (; get_bwd_unit(prm, take_unit(ucnt, false), ntiles_total, un); ++ucnt) {
        const int ksteps = (un.tile.len + 15) >> 4;
        wait_bar(bar(kKvFull), ucnt & 1, abort_flag, prm.header, 60);
        QIter qi;
        QTile qt = q_tile_at(prm, un, qi);
        wait_bar(bar(kQFullB + (gc & 1)), (gc >> 1) & 1, abort_flag, prm.header, 61);
        tc_fence_after();
        issue_s(gc & 1, qt.len);
        for (int it = 0; it < un.n_it; ++it) {
          const uint32_t g = gc + it, st = g & 1, par = g & 1;
          const int qsteps = (qt.len + 15) >> 4;
          const uint64_t dq_mn = mnmajor_base(sQ) + st * kStageStep;
          const uint64_t ddo_k = kmajor_base(sdO), ddo_mn = mnmajor_base(sdO);
          // dP^T(it) = V dO^T
          wait_bar(bar(kDoFull), par, abort_flag, prm.header, 62);
          if (g > 0) wait_bar(bar(kDqDrained), (g - 1) & 1, abort_flag, prm.header, 63);
          tc_fence_after();
          {
            const uint32_t idesc = make_idesc(128, qsteps << 4, 0, 0);
#pragma unroll
            for (int k = 0; k < DV / 16; ++k)
              mma_ss(tmem + tdP, dV_k + kmajor_off(k), ddo_k + kmajor_off(k), idesc, k > 0);
            mma_commit(bar(kDpFull));
          }
          // (the next tile's coordinates and descriptors are worked out here, while the pipe is
          // still busy with dP, not between dV and S)
          QTile nx = qt;
          const bool has_next = it + 1 < un.n_it;
          if (has_next) {
            q_advance(qi, prm.Hq / prm.Hkv);
            nx = q_tile_at(prm, un, qi);
          }
          const uint32_t idesc_s_next = make_idesc(128, ((nx.len + 15) >> 4) << 4, 0, 0);
          const uint64_t dq_k_next = kmajor_base(sQ) + ((g + 1) & 1) * kStageStep;
          // dV += P^T dO
          wait_bar(bar(kPReady), par, abort_flag, prm.header, 64);
          if (it == 0) wait_bar(bar(kDkvFree), (ucnt & 1) ^ 1, abort_flag, prm.header, 65);
          tc_fence_after();
          // (the k-step count and the accumulate flag are decided once per group: a branch or
          // a run-time predicate in front of every MMA costs the issuing thread more than the
          // MMA takes)
          auto issue_dv = [&](auto full_c, auto acc_c) {
#pragma unroll
            for (int k = 0; k < 8; ++k)
              if (decltype(full_c)::value || k < qsteps)
                mma_ts(tmem + tdV, tmem + tS + (k < 4 ? k * 8 : 64 + (k - 4) * 8),
                       ddo_mn + mnmajor_off(k), idesc_kv, (decltype(acc_c)::value || k > 0) ? 1u : 0u);
          };
          if (qsteps == 8) {
            if (it > 0) issue_dv(std::true_type{}, std::true_type{});
            else issue_dv(std::true_type{}, std::false_type{});
          } else {
            if (it > 0) issue_dv(std::false_type{}, std::true_type{});
            else issue_dv(std::false_type{}, std::false_type{});
          }
          mma_commit(bar(kDoEmpty));
          // S^T(it+1) = K Q^T
          if (has_next) {
            const uint32_t g1 = g + 1;
            wait_bar(bar(kQFullB + (g1 & 1)), (g1 >> 1) & 1, abort_flag, prm.header, 66);
            tc_fence_after();
#pragma unroll
            for (int k = 0; k < DV / 16; ++k)
              mma_ss(tmem + tS, dK_k + kmajor_off(k), dq_k_next + kmajor_off(k), idesc_s_next, k > 0);
            mma_commit(bar(kSFullB));
          }
          // dQ(it) = dS K, then dK += dS^T Q
          wait_bar(bar(kDsReady), par, abort_flag, prm.header, 67);
          tc_fence_after();
          if (ksteps == 8) {
#pragma unroll
            for (int k = 0; k < 8; ++k)
              mma_ss(tmem + tdP, dS_mn + mnmajor_off(k), dK_mn + mnmajor_off(k), idesc_dq, k > 0);
          } else {
#pragma unroll
            for (int k = 0; k < 8; ++k)
              if (k < ksteps)
                mma_ss(tmem + tdP, dS_mn + mnmajor_off(k), dK_mn + mnmajor_off(k), idesc_dq, k > 0);
          }
          mma_commit(bar(kDqFull));
          auto issue_dk = [&](auto full_c, auto acc_c) {
#pragma unroll
            for (int k = 0; k < 8; ++k)
              if (decltype(full_c)::value || k < qsteps)
                mma_ss(tmem + tdK, dS_k + kmajor_off(k), dq_mn + mnmajor_off(k), idesc_kv,
                       (decltype(acc_c)::value || k > 0) ? 1u : 0u);
          };
          if (qsteps == 8) {
            if (it > 0) issue_dk(std::true_type{}, std::true_type{});
            else issue_dk(std::true_type{}, std::false_type{});
          } else {
            if (it > 0) issue_dk(std::false_type{}, std::true_type{});
            else issue_dk(std::false_type{}, std::false_type{});
          }
          mma_commit(bar(kQEmptyB + st));
          qt = nx;
        }
        mma_commit(bar(kDkvFull));
        mma_commit(bar(kKvEmpty));
        gc += un.n_it;
      }
    }
  } else if (warp < 10) {
    // ------------------------------------------------------------ compute warpgroups
    const int wg = (warp - 2) >> 2;       // column half
    const int row = 32 * (warp & 3) + lane;
    const uint32_t lane_base = tmem + (uint32_t(32 * (warp & 3)) << 16);
    const int cb = 64 * wg;
    uint32_t gc = 0, ucnt = 0;
    BwdUnit un;
    for (; get_bwd_unit(prm, take_unit(ucnt, true), ntiles_total, un); ++ucnt) {
      const bool row_ok = row < un.tile.len;
      // my key j = tile.start + row is seen by the queries [j, key_end[j])
      const int key_lo = un.tile.start + row;
      const int key_hi = row_ok ? prm.key_end[key_lo] : key_lo;
      QIter qi;
      for (int it = 0; it < un.n_it; ++it, q_advance(qi, prm.Hq / prm.Hkv)) {
        const QTile qt = q_tile_at(prm, un, qi);
        const uint32_t g = gc + it, st = g & 1, par = g & 1;
        const float* sl = stats + st * 256 + cb;
        // Fast path: both tiles complete and every key row of this warp sees either the whole
        // query tile or none of it -- true for all query tiles behind the key tile except
        // where a segment ends inside them, also when the key tile itself straddles segments
        // (its prompt / earlier-response keys then see everything, the others nothing).  The
        // unmasked arithmetic runs and an unseen row's P (hence dS) is set to zero afterwards.
        const int lo = key_lo - qt.start, hi = key_hi - qt.start;
        const bool row_all = lo <= 0 && hi >= kTile, row_none = hi <= 0 || lo >= kTile;
        const bool full = qt.len == kTile && un.tile.len == kTile &&
                          __all_sync(0xffffffffu, row_all || row_none);
        wait_bar(bar(kQFullB + st), (g >> 1) & 1, abort_flag, prm.header, 70);
        wait_bar(bar(kSFullB), par, abort_flag, prm.header, 71);
        tc_fence_after();
        uint32_t v[64];
        tmem_ld32(lane_base + tS + cb, *reinterpret_cast<uint32_t(*)[32]>(&v[0]));
        tmem_ld32(lane_base + tS + cb + 32, *reinterpret_cast<uint32_t(*)[32]>(&v[32]));
        tmem_wait_ld();
        uint32_t pk[32];
        const float4* sl4 = reinterpret_cast<const float4*>(sl);
        const uint64_t sc2 = pack2(prm.scale_log2, prm.scale_log2);
        if (full) {
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float4 l = sl4[i];   // -LSE * log2(e)
            float x0, x1, x2, x3;
            unpack2(fma2(pack2(__uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1])), sc2,
                         pack2(l.x, l.y)), x0, x1);
            unpack2(fma2(pack2(__uint_as_float(v[4 * i + 2]), __uint_as_float(v[4 * i + 3])), sc2,
                         pack2(l.z, l.w)), x2, x3);
            pk[2 * i] = pack_bf16(ex2(x0), ex2(x1));
            pk[2 * i + 1] = pack_bf16(ex2(x2), ex2(x3));
          }
          if (!row_all) {
#pragma unroll
            for (int i = 0; i < 32; ++i) pk[i] = 0u;
          }
        } else {
          // query column c is visible iff key_lo <= qt.start + c < key_hi (an absent key row
          // has an empty range; key_hi never exceeds the group's end, so c < qt.len follows)
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const int c0 = cb + 2 * i;
            float p0 = ex2(fmaf(__uint_as_float(v[2 * i]), prm.scale_log2, sl[2 * i]));
            float p1 = ex2(fmaf(__uint_as_float(v[2 * i + 1]), prm.scale_log2, sl[2 * i + 1]));
            p0 = (c0 >= lo && c0 < hi) ? p0 : 0.f;
            p1 = (c0 + 1 >= lo && c0 + 1 < hi) ? p1 : 0.f;
            pk[i] = pack_bf16(p0, p1);
          }
        }
        tmem_st32(lane_base + tS + cb, pk);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar(kPReady));

        wait_bar(bar(kDpFull), par, abort_flag, prm.header, 72);
        tc_fence_after();
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          uint32_t d[32];
          tmem_ld32(lane_base + tdP + cb + 32 * half, d);
          tmem_wait_ld();
          uint32_t ds[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const uint32_t pp = pk[16 * half + i];
            const float p0 = __uint_as_float(pp << 16), p1 = __uint_as_float(pp & 0xffff0000u);
            const float2 dl = reinterpret_cast<const float2*>(sl + 128 + 32 * half)[i];   // -Delta
            float d0, d1;
            unpack2(fma2(pack2(p0, p1),
                         add2(pack2(__uint_as_float(d[2 * i]), __uint_as_float(d[2 * i + 1])),
                              pack2(dl.x, dl.y)),
                         pack2(0.f, 0.f)),
                    d0, d1);
            if (!full) {  // stale tensor-memory columns may hold anything
              d0 = (pp & 0xffffu) ? d0 : 0.f;
              d1 = (pp & 0xffff0000u) ? d1 : 0.f;
            }
            ds[i] = pack_bf16(d0, d1);
          }
          // dS^T row `row`, columns [cb + 32 half, +32): box wg, 16-byte chunks 4 half .. +3
          const uint32_t row_addr = sdS + wg * kBoxBytes + row * 128;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const uint32_t chunk = uint32_t(half * 4 + i) ^ uint32_t(row & 7);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row_addr + chunk * 16),
                         "r"(ds[4 * i]), "r"(ds[4 * i + 1]), "r"(ds[4 * i + 2]), "r"(ds[4 * i + 3])
                         : "memory");
          }
        }
        fence_proxy_async_smem();
        mbar_arrive(bar(kDsReady));
      }
      gc += un.n_it;
      // ---- unit epilogue: warpgroup 0 stores dV, warpgroup 1 stores scale * dK
      wait_bar(bar(kDkvFull), ucnt & 1, abort_flag, prm.header, 73);
      tc_fence_after();
      const uint32_t tsrc = wg ? tdK : tdV;
      const float f = wg ? prm.scale : 1.f;
      uint32_t ob[D / 2];
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t w[32];
        if (DV == D || c * 32 < DV) {
          tmem_ld32(lane_base + tsrc + c * 32, w);
          tmem_wait_ld();
        } else {  // columns past DV hold nothing and are not stored
#pragma unroll
          for (int i = 0; i < 32; ++i) w[i] = 0u;
        }
#pragma unroll
        for (int i = 0; i < 16; ++i)
          ob[c * 16 + i] = pack_bf16(__uint_as_float(w[2 * i]) * f, __uint_as_float(w[2 * i + 1]) * f);
      }
      tc_fence_before();
      mbar_arrive(bar(kDkvFree));
      // A thread holds one row as 16-byte chunks; transposing each group of eight chunks
      // (128 bytes) inside groups of eight lanes gives every lane the same chunk of eight
      // consecutive rows, so that one store instruction of the warp writes four whole
      // 128-byte lines instead of 32 scattered 16-byte pieces (which kept the SM's memory
      // pipe busy for thousands of cycles at every unit boundary).
#pragma unroll
      for (int hb = 0; hb < D / 64; ++hb) {
        uint32_t* x = ob + 32 * hb;
        auto exchange = [&](auto dist) {
          constexpr int d = decltype(dist)::value;
          const bool hi = (lane & d) != 0;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            if ((i & d) == 0) {
#pragma unroll
              for (int c = 0; c < 4; ++c) {
                const uint32_t send = hi ? x[4 * i + c] : x[4 * (i | d) + c];
                const uint32_t recv = __shfl_xor_sync(0xffffffffu, send, d);
                if (hi) x[4 * i + c] = recv; else x[4 * (i | d) + c] = recv;
              }
            }
          }
        };
        exchange(std::integral_constant<int, 4>{});
        exchange(std::integral_constant<int, 2>{});
        exchange(std::integral_constant<int, 1>{});
      }
      {
        __nv_bfloat16* out = wg ? prm.dk : prm.dv;
        const int grp = lane >> 3, chunk = lane & 7;
#pragma unroll
        for (int hb = 0; hb < D / 64; ++hb) {
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int r = 32 * (warp & 3) + grp * 8 + i;
            if (r < un.tile.len && (DV == D || hb * 64 + chunk * 8 < DV)) {
              uint4* dst = reinterpret_cast<uint4*>(
                  out + ((size_t(un.tile.start) + r) * prm.Hkv + un.kvh) * DV + hb * 64 + chunk * 8);
              *dst = make_uint4(ob[32 * hb + 4 * i], ob[32 * hb + 4 * i + 1], ob[32 * hb + 4 * i + 2],
                                ob[32 * hb + 4 * i + 3]);
            }
          }
        }
      }
    }
  } else {
    // ------------------------------------------------------------ dQ warpgroup
    const int row = 32 * (warp & 3) + lane;
    const bool leader = (warp == 10 && lane == 0);
    const uint32_t lane_base = tmem + (uint32_t(32 * (warp & 3)) << 16);
    const uint32_t stg = base + L::kStg;
    uint32_t gc = 0, chunk = 0, ucnt = 0;
    BwdUnit un;
    for (; get_bwd_unit(prm, take_unit(ucnt, true), ntiles_total, un); ++ucnt) {
      QIter qi;
      // Deterministic variant: the key tiles that add to a (query tile, head) do so in
      // DESCENDING tile order: the query tile's own key tile first, then the tiles below it
      // down to dep_lo of the query tile, then the prompt tiles from npc - 1 down to 0.  With
      // every unit walking its query tiles upwards from its own tile, that is the order in
      // which the units reach a query tile anyway (tile k gets there one query tile's worth
      // of iterations after tile k + 1), so in the steady state nobody waits.  The counter of
      // the pair holds 1 + the group-relative index of the last key tile that has added (0:
      // none yet).  Units are handed out set by set and inside a set in descending tile order
      // (the plan's second unit list), so the tile waited for is always running or done and
      // the waits cannot lock up.
      const int k_rel = (un.tile.start - un.tile.grp_start) / kTile;
      int dep_lo = 0;
      // Passing the turn on needs the reductions of the tile to be complete (a wait of a
      // microsecond or two), so it is deferred: the counter of iteration i is published after
      // the reductions of iteration i + 1 have been issued -- the next key tile gets to the
      // same query tile a whole query tile's worth of iterations later -- or at once whenever
      // this unit finds that it has to wait for its own turn.
      int32_t* pend = nullptr;
      auto publish = [&](int32_t* p) {   // (the release store orders it behind the completed adds)
        const int mine = k_rel + 1;
        asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(mine) : "memory");
      };
      for (int it = 0; it < un.n_it; ++it, q_advance(qi, prm.Hq / prm.Hkv)) {
        const QTile qt = q_tile_at(prm, un, qi);
        const uint32_t g = gc + it;
        int32_t* sem = nullptr;
        int seen_early = -1;
        if (kDet && leader) {
          sem = prm.dq_sem + size_t(un.tidx + qi.qt) * prm.Hq + qt.h;
          // the last prompt tile follows the lowest response tile that adds to this query tile
          if (qi.hh == 0 && qi.qt > 0 && k_rel == un.tile.npc - 1 && k_rel + qi.qt >= un.tile.npc)
            dep_lo = prm.tiles[un.tidx + qi.qt].dep_lo;
          // read the counter now: the answer (normally already the expected one) is back by the
          // time the first box of the tile is staged
          asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen_early) : "l"(sem) : "memory");
        }
        wait_bar(bar(kDqFull), g & 1, abort_flag, prm.header, 80);
        tc_fence_after();
        // Two halves of D/2 columns.  The second half is read out of tensor memory (and the
        // dP/dQ columns handed back to the MMA warp) before any wait on the reductions issued
        // for the first half, so the MMA pipeline never waits for TMA reads of the staging.
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          uint32_t w[D / 2];
#pragma unroll
          for (int c = 0; c < D / 64; ++c) {
            if (DV == D || half * (D / 2) + c * 32 < DV) {
              tmem_ld32(lane_base + tdP + half * (D / 2) + c * 32,
                        *reinterpret_cast<uint32_t(*)[32]>(&w[c * 32]));
            } else {  // no such columns in global memory: the box is not reduced either
#pragma unroll
              for (int i = 0; i < 32; ++i) w[c * 32 + i] = 0u;
            }
          }
          tmem_wait_ld();
          if (half == 1) {
            tc_fence_before();
            mbar_arrive(bar(kDqDrained));
          }
          if (row >= qt.len) {  // rows past the tile's end belong to other tokens: add zero
#pragma unroll
            for (int i = 0; i < D / 2; ++i) w[i] = 0u;
          }
#pragma unroll
          for (int c = 0; c < D / 64; ++c, ++chunk) {
            const uint32_t buf = stg + (chunk & 1) * L::kStageBytes;
            // the reduce issued two chunks ago must have finished reading this buffer
            if (leader) bulk_wait_group_read<1>();
            named_barrier_sync(1, 128);
            const uint32_t row_addr = buf + row * 128;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const uint32_t ch = uint32_t(i) ^ uint32_t(row & 7);
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row_addr + ch * 16),
                           "r"(w[c * 32 + 4 * i]), "r"(w[c * 32 + 4 * i + 1]),
                           "r"(w[c * 32 + 4 * i + 2]), "r"(w[c * 32 + 4 * i + 3])
                           : "memory");
            }
            fence_proxy_async_smem();
            named_barrier_sync(1, 128);
            if (leader) {
              if (kDet && sem && half == 0 && c == 0) {  // wait for this unit's turn (bounded)
                const int expect =
                    qi.qt == 0 ? 0
                               : ((k_rel == un.tile.npc - 1 && k_rel + qi.qt >= un.tile.npc) ? dep_lo + 1
                                                                                            : k_rel + 2);
                bool ok = seen_early == expect;
                for (uint32_t spin = 0; !ok && spin < (1u << 22); ++spin) {
                  int seen;
                  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(sem) : "memory");
                  if (seen == expect) {
                    ok = true;
                    break;
                  }
                  if (pend) {  // about to wait: do not keep the unit below waiting for us
                    bulk_wait_group<0>();
                    publish(pend);
                    pend = nullptr;
                  }
                  if ((spin & 0xff) == 0xff && *abort_flag) break;
                  __nanosleep(20);
                }
                if (!ok && !*abort_flag) {
                  if (atomicCAS(&prm.header[0], kStatusOk, kStatusWaitExpired) == kStatusOk)
                    prm.header[1] = 81;
                  *abort_flag = 1;
                }
              }
              if (DV == D || half * (D / 2) + c * 32 < DV)
                tma_reduce_add_3d(&tm_dq, buf, half * (D / 2) + c * 32, qt.h, qt.start);
              bulk_commit_group();
            }
          }
        }
        if (kDet && sem) {
          if (pend) {  // the previous tile's boxes (all but this tile's D / 32 groups) have landed
            bulk_wait_group<D / 32>();
            publish(pend);
          }
          pend = sem;
        }
      }
      if (kDet && pend) {
        bulk_wait_group<0>();
        publish(pend);
      }
      gc += un.n_it;
    }
    if (leader) bulk_wait_group<0>();
  }

  tc_fence_before();
  __syncthreads();
  // After a wait that gave up, copies, reductions and MMAs issued without their barriers may
  // still be in flight: give them time to land before shared and tensor memory are released.
  if (*abort_flag)
    for (int i = 0; i < 50; ++i) __nanosleep(1000);
  if (warp == 0) tmem_dealloc(tmem, kBwdTmemCols);
  if (tid == 0) {  // the last CTA to finish re-arms the unit counter for the next launch
    __threadfence();
    if (atomicAdd(&prm.header[kHdrBwdDone], 1) == int(gridDim.x) - 1) {
      prm.header[kHdrBwdNext] = 0;
      prm.header[kHdrBwdDone] = 0;
    }
  }
#ifdef PP_DEBUG_COUNTERS
  if (blockIdx.x == 0 && tid == 0) g_wait_cycles[127] = (unsigned long long)(clock64() - t_kernel0);
  if (tid == 0) g_cta_cycles[blockIdx.x & 255] = (unsigned long long)(clock64() - t_kernel0);
#endif
}

#ifdef PP_DEBUG_COUNTERS
}  // namespace
}  // namespace pp
extern "C" int pp_debug_bwd_cta_cycles(unsigned long long* out) {
  return cudaMemcpyFromSymbol(out, pp::g_cta_cycles, sizeof(unsigned long long) * 256) == cudaSuccess ? 0 : -5;
}
extern "C" int pp_debug_bwd_wait_cycles(unsigned long long* out, int reset) {
  if (out && cudaMemcpyFromSymbol(out, pp::g_wait_cycles, sizeof(unsigned long long) * 128) != cudaSuccess)
    return -5;
  if (reset) {
    static unsigned long long zeros[128] = {};
    if (cudaMemcpyToSymbol(pp::g_wait_cycles, zeros, sizeof zeros) != cudaSuccess) return -5;
  }
  return 0;
}
namespace pp {
namespace {
#endif

template <int D, int DV = D>
cudaError_t launch_bwd_t(const pp_plan* plan, const void* o, const float* lse, const void* d_o,
                         void* dq, const CUtensorMap& tq, const CUtensorMap& tk,
                         const CUtensorMap& tv, const CUtensorMap& tdo, const CUtensorMap& tdq,
                         const BwdParams& prm, bool dq_cleared, cudaStream_t stream,
                         int* launches) {
  static DeviceSetup setup[kMaxDevices];
  DeviceSetup* dev = device_setup(setup);
  if (!dev) return cudaErrorInvalidDevice;
  if (dev->cc_major != 10) return cudaErrorNotSupported;
  auto kern = prm.dq_sem ? bwd_kernel<D, true, DV> : bwd_kernel<D, false, DV>;
  if (!dev->configured) {
    cudaError_t e = cudaFuncSetAttribute(bwd_kernel<D, false, DV>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         BwdSmem<D>::kTotal);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(bwd_kernel<D, true, DV>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               BwdSmem<D>::kTotal);
    if (e != cudaSuccess) return e;
    dev->configured = true;
  }
  const pp_problem& pb = plan->prob;
  const size_t T = pb.total_tokens, Hq = pb.num_q_heads;
  const long long pairs = (long long)T * Hq;
  const int num_sms = dev->num_sms;
  constexpr int kRowsPerBlock = 8 * (32 / pre_lanes(DV)) * 4;  // warps x rows per warp x unroll
  const unsigned pre_blocks = unsigned(
      std::min<long long>((pairs + kRowsPerBlock - 1) / kRowsPerBlock, (long long)num_sms * 16));
  auto pre = [&](auto clear, auto token_major) {
    bwd_preprocess_kernel<DV, decltype(clear)::value, decltype(token_major)::value>
        <<<pre_blocks, 256, 0, stream>>>(
            static_cast<const __nv_bfloat16*>(o), static_cast<const __nv_bfloat16*>(d_o), lse,
            const_cast<float*>(prm.delta), const_cast<float*>(prm.lse2), prm.dq_acc, int(T), int(Hq));
  };
  const bool token_major = Hq * DV * 2 >= 16384;
  if (dq_cleared) {
    if (token_major) pre(std::false_type{}, std::true_type{});
    else pre(std::false_type{}, std::false_type{});
  } else {
    if (token_major) pre(std::true_type{}, std::true_type{});
    else pre(std::true_type{}, std::false_type{});
  }
  const long long units = (long long)plan->max_tiles * pb.num_kv_heads;
  dim3 grid(unsigned(std::min<long long>(units, num_sms)));
  ProfileEvents& ev = profile_events();
  const int slot = int(ev.bwd_count % kProfileRing);
  if (ev.on) profile_record(ev.bwd0[slot], stream);
  kern<<<grid, kBwdThreads, BwdSmem<D>::kTotal, stream>>>(tq, tk, tv, tdo, tdq, prm);
  if (ev.on) {
    profile_record(ev.bwd1[slot], stream);
    ++ev.bwd_count;
  }
  const size_t n4 = T * Hq * DV / 4;
  unsigned fb = unsigned(std::min<size_t>((n4 + 255) / 256, size_t(num_sms) * 16));
  bwd_finalize_kernel<<<fb, 256, 0, stream>>>(reinterpret_cast<const float4*>(prm.dq_acc),
                                              static_cast<uint2*>(dq), n4, prm.scale);
  if (launches) *launches += 3;
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_bwd(const pp_plan* plan, const void* q, const void* k, const void* v,
                       const void* o, const float* lse, const void* d_o, float scale, void* dq,
                       void* dk, void* dv, void* scratch, bool dq_cleared, bool deterministic,
                       cudaStream_t stream, int* launches) {
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
  prm.tiles = reinterpret_cast<const BTile*>(plan->ws + plan->lay.btiles);
  prm.order = reinterpret_cast<const int32_t*>(
      plan->ws + (deterministic ? plan->lay.bwd_units_det : plan->lay.bwd_units));
  prm.key_end = reinterpret_cast<const int32_t*>(plan->ws + plan->lay.key_end);
  prm.delta = reinterpret_cast<float*>(sc + sl.delta);
  prm.lse2 = reinterpret_cast<float*>(sc + sl.lse2);
  prm.dq_acc = reinterpret_cast<float*>(sc + sl.dq_acc);
  prm.dq_sem = nullptr;
  if (deterministic) {
    prm.dq_sem = reinterpret_cast<int32_t*>(sc + sl.sem);
    cudaError_t me = cudaMemsetAsync(prm.dq_sem, 0, sl.sem_bytes, stream);
    if (me != cudaSuccess) return me;
  }
  prm.dk = static_cast<__nv_bfloat16*>(dk);
  prm.dv = static_cast<__nv_bfloat16*>(dv);
  prm.T = pb.total_tokens;
  prm.Hq = pb.num_q_heads;
  prm.Hkv = pb.num_kv_heads;
  prm.scale = scale;
  prm.scale_log2 = scale * 1.4426950408889634f;
  CUtensorMap tdq;
  if (!encode_thd_f32(&tdq, prm.dq_acc, pb.total_tokens, pb.num_q_heads, pb.head_dim))
    return cudaErrorNotSupported;
  if (pb.head_dim == 128)
    return launch_bwd_t<128>(plan, o, lse, d_o, dq, tq, tk, tv, tdo, tdq, prm, dq_cleared, stream,
                             launches);
  if (pb.head_dim == 96)
    return launch_bwd_t<128, 96>(plan, o, lse, d_o, dq, tq, tk, tv, tdo, tdq, prm, dq_cleared,
                                 stream, launches);
  return launch_bwd_t<64>(plan, o, lse, d_o, dq, tq, tk, tv, tdo, tdq, prm, dq_cleared, stream,
                          launches);
}

// ---------------------------------------------------------------- built-in scratch
// Backward scratch for callers that cannot allocate device memory (pp_attn_bwd_noalloc).
// The array is part of the library image: every device that loads the library holds
// kStaticScratchBytes until the process exits, and every call on a device shares it.
static __device__ __align__(256) unsigned char g_static_bwd_scratch[kStaticScratchBytes];

// In host code `g_static_bwd_scratch` is only a stand-in for the symbol, not a device
// address, so the address is looked up once per device (with that device current) and kept.
// The array used must be the one on the device that holds the plan (and so the tensors): the
// current device has to be that device, otherwise the call is refused instead of handing the
// kernels another GPU's array.
static cudaError_t static_scratch_address(const pp_plan* plan, void** out) {
  static std::mutex mu;
  static void* ptrs[kMaxDevices] = {};
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  cudaPointerAttributes attr;
  e = cudaPointerGetAttributes(&attr, plan->ws);
  if (e != cudaSuccess) return e;
  if (attr.type != cudaMemoryTypeDevice || attr.device != dev) return cudaErrorInvalidDevice;
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
  cudaError_t e = static_scratch_address(plan, &scratch);
  if (e != cudaSuccess) return e;
  // launch_bwd zeroes the fp32 dQ accumulator inside the scratch on every call and rewrites
  // Delta and the scaled LSE, so nothing of an earlier call's contents is read.
  return launch_bwd(plan, q, k, v, o, lse, d_o, scale, dq, dk, dv, scratch, false, false, stream,
                    launches);
}

}  // namespace pp
