// Forward kernel: O = softmax(mask(scale Q K^T)) V and LSE over the plan's visible tiles.
//
// Persistent, warp-specialised CTA (one per SM):
//   warp 0      TMA producer: draws and decodes the work units (the only reader of the plan's
//               tile list; the other roles get a decoded record through shared memory), loads
//               the Q tiles of the unit's two query heads, then the K / V tiles of every
//               visible key tile in two-deep stages {V(j), K(j + 1)} (one barrier pair each)
//   warp 1      MMA issuer (one thread): S = Q K^T and O += P V with tcgen05.mma, fp32 in TMEM
//   warps 2-9   softmax warps of slot 0: two threads per query row (= TMEM lane), 64 key
//               columns each
//   warps 10-17 softmax warps of slot 1
//   warps 18-19 optional: clear the backward's fp32 dQ accumulator for the unit's rows
// A work unit is (query tile, KV head, pair of query heads of that KV head): both slots see
// the same keys and the same mask, so every K / V tile staged in shared memory feeds two
// S tiles.  While one slot's warpgroup does its exponentials the tensor core works on the
// other slot (order: PV_0(j), QK_0(j+1), PV_1(j), QK_1(j+1), ...).  P (bf16) overwrites columns
// [0,32) and [64,96) of its S tile in tensor memory (each half-row thread inside the columns it
// has read itself) and is the A operand of the second MMA; V is
// its MN-major B operand straight from the TMA layout.  O is rescaled lazily: only when a
// row's running maximum grew by more than 2^8 since the value used for scaling.
// TMEM: S0 | S1 | O0 | O1, 128 columns each.
#include <algorithm>
#include <type_traits>

#include "pp_dev.cuh"

namespace pp {
namespace {

struct FwdParams {
  int32_t* header;
  const Tile* tiles;
  const int32_t* order;
  __nv_bfloat16* o;
  float* lse;
  float* dq_clear;  // optional: the backward's fp32 dQ accumulator [T][Hq][D], cleared here
  int T, Hq, Hkv;
  float scale_log2;  // softmax scale * log2(e)
};

constexpr int kFwdThreads = 640;
constexpr uint32_t kFwdTmemCols = 512;
constexpr float kRescaleThreshold = 8.f;  // log2 units

enum FwdBar : int {
  kQFull = 0,   // [2] per slot
  kQEmpty = 2,  // [2]
  kKFull = 4,   // [2] per K / V stage: full
  kKEmpty = 6,  // [2]                 empty
  kVFull = 8,   // (unused)
  kVEmpty = 10,
  kSFull = 12,  // [2] per slot
  kPFull = 14,
  kODone = 16,
  kOFree = 18,
  kSchedFullF = 20,   // [2] unit ids handed from the producer to the other roles
  kSchedEmptyF = 22,  // [2] 17 arrivals: MMA thread + 16 softmax warps
  kNumFwdBars = 24
};

template <int D>
struct FwdSmem {
  static constexpr int kTileBytes = 128 * D * 2;
  static constexpr int kQ = 0, kK = 2 * kTileBytes, kV = 4 * kTileBytes, kBars = 6 * kTileBytes;
  static constexpr int kSched = kBars + 256;          // two decoded unit records of 8 ints
  static constexpr int kXch = kSched + 64;            // float [2 slots][2 buffers][128 rows][2 halves]
  static constexpr int kTotal = kXch + 4096 + 1024;   // + slack to align the base to 1024 B
};

struct KvTile {
  int start, len;
  bool diag;
};

__device__ __forceinline__ KvTile kv_tile_of(const Tile& t, int j, int n0, int n1) {
  KvTile k;
  if (j < n0) {
    k.start = t.kv0_start + j * kTile;
    k.len = min(kTile, t.kv0_len - j * kTile);
    k.diag = false;
  } else if (j < n0 + n1) {
    k.start = t.kv1_start + (j - n0) * kTile;
    k.len = min(kTile, t.kv1_len - (j - n0) * kTile);
    k.diag = false;
  } else {
    k.start = t.start;
    k.len = t.len;
    k.diag = true;
  }
  return k;
}

struct Unit {
  Tile tile;
  int h0, kvh, nslots, n0, n1, ntiles;
};

// Units are handed out dynamically in the plan's longest-work-first order: the producer
// draws the next index from a global counter (header[4]) when the CTA is ready for more and
// passes it on through a two-entry shared-memory ring; header[6] counts finished CTAs and the
// last one resets both counters for the next launch.
constexpr int kHdrFwdNext = 4, kHdrFwdDone = 6;

__device__ __forceinline__ bool get_unit(const FwdParams& prm, int u, int ntiles_total, Unit& un) {
  const int r = prm.Hq / prm.Hkv, npairs = (r + 1) >> 1, per_tile = prm.Hkv * npairs;
  const int ord = u / per_tile;
  if (ord >= ntiles_total) return false;
  const int rem = u - ord * per_tile;
  un.kvh = rem / npairs;
  const int pair = rem - un.kvh * npairs;
  un.h0 = un.kvh * r + 2 * pair;
  un.nslots = (2 * pair + 1 < r) ? 2 : 1;
  un.tile = prm.tiles[prm.order[ord]];
  un.n0 = (un.tile.kv0_len + kTile - 1) / kTile;
  un.n1 = (un.tile.kv1_len + kTile - 1) / kTile;
  un.ntiles = un.n0 + un.n1 + 1;
  return true;
}

// D: head dimension of the shared-memory tiles (64 or 128); DV <= D: head dimension of the
// tensors in global memory.  For DV < D (96 in tiles of 128) the TMA loads fill the columns
// past DV with zeros, so only the loops over the head dimension, the N of the second GEMM and
// everything that addresses global memory know about DV.
template <int D, int DV = D>
__global__ void __launch_bounds__(kFwdThreads, 1)
fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
           const __grid_constant__ CUtensorMap tm_v, FwdParams prm) {
  using L = FwdSmem<D>;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (prm.header[0] != kStatusOk) return;
  const int ntiles_total = prm.header[2];
#ifdef PP_DEBUG_COUNTERS
  const long long t_kernel0 = clock64();
#endif

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gbase = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sQ = base + L::kQ, sK = base + L::kK, sV = base + L::kV;
  const uint32_t bars = base + L::kBars;
  auto bar = [&](int i) { return bars + 8u * uint32_t(i); };
  const uint32_t tmem_slot = bars + 8 * kNumFwdBars;
  volatile uint32_t* tmem_slot_p = reinterpret_cast<volatile uint32_t*>(gbase + L::kBars + 8 * kNumFwdBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gbase + L::kBars + 8 * kNumFwdBars + 8);

  if (tid == 0) {
    for (int i = 0; i < kNumFwdBars; ++i) {
      const bool wg_count = (i >= kPFull && i < kPFull + 2) || (i >= kOFree && i < kOFree + 2);
      const bool sched_empty = (i >= kSchedEmptyF && i < kSchedEmptyF + 2);
      // unit records are released by the MMA thread, the 16 softmax warps and, when the dQ
      // accumulator is cleared here, the two clearing warps
      mbar_init(bar(i), wg_count ? 256 : (sched_empty ? (prm.dq_clear ? 19 : 17) : 1));
    }
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
  // Ring of two decoded unit records (producer -> MMA thread and softmax warps): the producer
  // alone reads the plan's tile list; the other roles get what they need from shared memory.
  volatile int* sched = reinterpret_cast<volatile int*>(gbase + L::kSched);
  auto fetch_unit = [&](uint32_t n, Unit& un) -> bool {  // producer thread
    wait_bar(bar(kSchedEmptyF + (n & 1)), ((n >> 1) & 1) ^ 1, abort_flag, prm.header, 90);
    // after a wait has given up, no more work is drawn: the end marker goes out instead
    const int u = *abort_flag ? 0x7fffffff : atomicAdd(&prm.header[kHdrFwdNext], 1);
    const bool ok = get_unit(prm, u, ntiles_total, un);
    volatile int* e = sched + (n & 1) * 8;
    e[0] = un.tile.start;
    e[1] = un.tile.len;
    e[2] = un.h0;
    e[3] = ok ? un.nslots : 0;  // 0 slots marks the end of the work list
    e[4] = un.n0;
    e[5] = un.n1;
    e[6] = un.tile.kv0_len - (un.n0 - 1) * kTile;
    e[7] = un.tile.kv1_len - (un.n1 - 1) * kTile;
    mbar_arrive(bar(kSchedFullF + (n & 1)));
    return ok;
  };
  // Consumers: read the record into plain scalars (kept in registers) and release the entry.
#define PP_TAKE_UNIT(n, whole_warp)                                                              \
  const bool u_ok = wait_bar(bar(kSchedFullF + ((n) & 1)), ((n) >> 1) & 1, abort_flag, prm.header, 91); \
  const volatile int* u_e = sched + ((n) & 1) * 8;                                               \
  const int u_start = u_e[0], u_len = u_e[1], u_h0 = u_e[2], u_nslots = u_ok ? u_e[3] : 0;       \
  const int u_n0 = u_e[4], u_n1 = u_e[5], u_last0 = u_e[6], u_last1 = u_e[7];                    \
  const int u_ntiles = u_n0 + u_n1 + 1;                                                          \
  if (whole_warp) {                                                                              \
    __syncwarp();                                                                                \
    if (lane == 0) mbar_arrive(bar(kSchedEmptyF + ((n) & 1)));                                   \
  } else {                                                                                       \
    mbar_arrive(bar(kSchedEmptyF + ((n) & 1)));                                                  \
  }                                                                                              \
  (void)u_start, (void)u_len, (void)u_h0;                                                        \
  /* keys of visible key tile j: only the last tile of a full range and the diagonal tile */    \
  /* can be shorter than 128 */                                                                  \
  auto u_klen = [=](int j) -> int {                                                              \
    return (j + 1 == u_n0) ? u_last0 : (j + 1 == u_n0 + u_n1) ? u_last1 : (j + 1 == u_ntiles) ? u_len : kTile; \
  };

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t kc = 0, qc[2] = {0, 0};
      Unit un;
      for (uint32_t un_i = 0; fetch_unit(un_i, un); ++un_i) {
        for (int s = 0; s < un.nslots; ++s) {
          wait_bar(bar(kQEmpty + s), (qc[s] & 1) ^ 1, abort_flag, prm.header, 20 + s);
          mbar_expect_tx(bar(kQFull + s), L::kTileBytes);
          for (int b = 0; b < D / 64; ++b)
            tma_load_3d(sQ + s * L::kTileBytes + b * kBoxBytes, &tm_q, b * 64, un.h0 + s,
                        un.tile.start, bar(kQFull + s));
          ++qc[s];
        }
        // K and V travel in stages {V(j), K(j + 1)} -- what one period of the MMA thread
        // consumes -- with ONE full / empty barrier pair per stage (the first stage of a unit
        // holds only K(0), the last only V(last)): every barrier operation costs the MMA
        // thread 100 - 150 cycles of tensor-pipe time, so it gets one wait and one commit per
        // period instead of two of each.  Stage n uses the K and V buffers n & 1.
        auto load_stage = [&](int jv, int jk) {   // key tile of V and of K in this stage, or -1
          const uint32_t st = kc & 1;
          wait_bar(bar(kKEmpty + st), ((kc >> 1) & 1) ^ 1, abort_flag, prm.header, 22);
          mbar_expect_tx(bar(kKFull + st), (jv >= 0 && jk >= 0 ? 2 : 1) * L::kTileBytes);
          if (jk >= 0) {
            const KvTile kt = kv_tile_of(un.tile, jk, un.n0, un.n1);
            for (int b = 0; b < D / 64; ++b)
              tma_load_3d(sK + st * L::kTileBytes + b * kBoxBytes, &tm_k, b * 64, un.kvh, kt.start,
                          bar(kKFull + st));
          }
          if (jv >= 0) {
            const KvTile kt = kv_tile_of(un.tile, jv, un.n0, un.n1);
            for (int b = 0; b < D / 64; ++b)
              tma_load_3d(sV + st * L::kTileBytes + b * kBoxBytes, &tm_v, b * 64, un.kvh, kt.start,
                          bar(kKFull + st));
          }
          ++kc;
        };
        load_stage(-1, 0);
        for (int j = 0; j < un.ntiles && !*abort_flag; ++j)
          load_stage(j, j + 1 < un.ntiles ? j + 1 : -1);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    // tcgen05.mma issue blocks this thread for about one MMA duration, so the tensor pipe is
    // idle whenever the thread executes anything else for longer than that: the loop below
    // keeps the work between two groups of MMAs to a minimum (descriptors and instruction
    // descriptors precomputed, barrier addresses and parities kept in registers, one branch
    // for the common case of full 128-key tiles).
    if (lane == 0) {
      uint32_t kc = 0, tc0 = 0, tc1 = 0, uc0 = 0, uc1 = 0;
      constexpr uint32_t idesc_o = make_idesc(128, DV, 0, 1);
      constexpr uint32_t idesc_full = make_idesc(128, 128, 0, 0);
      constexpr uint64_t kStageStep = uint64_t(L::kTileBytes >> 4);
      const uint64_t dq0 = kmajor_base(sQ), dk0 = kmajor_base(sK), dv0 = mnmajor_base(sV);
      // length of key tile j of a unit: only the last tile of each visible range and the
      // diagonal tile can be shorter than 128
      auto issue_qk = [&](int s, uint32_t kstage, int k_len) {
        const uint64_t a = dq0 + s * kStageStep, b = dk0 + kstage * kStageStep;
        const uint32_t tS = tmem + s * 128;
        if (k_len == kTile) {
#pragma unroll
          for (int kk = 0; kk < DV / 16; ++kk)
            mma_ss(tS, a + kmajor_off(kk), b + kmajor_off(kk), idesc_full, kk > 0);
        } else {
          const uint32_t idesc_s = make_idesc(128, 0, 0, 0) | (uint32_t(((k_len + 15) >> 4) << 1) << 17);
#pragma unroll
          for (int kk = 0; kk < DV / 16; ++kk)
            mma_ss(tS, a + kmajor_off(kk), b + kmajor_off(kk), idesc_s, kk > 0);
        }
        mma_commit(bar(kSFull + s));
      };
      auto issue_pv = [&](int s, uint32_t vstage, int k_len, bool first, bool last) {
        const uint64_t b = dv0 + vstage * kStageStep;
        const uint32_t tS = tmem + s * 128, tO = tmem + 256 + s * 128;
        if (k_len == kTile && !first) {
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            mma_ts(tO, tS + (kk < 4 ? kk * 8 : 64 + (kk - 4) * 8), b + mnmajor_off(kk), idesc_o, 1);
        } else {
          const int ksteps = (k_len + 15) >> 4;
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            if (kk < ksteps)
              mma_ts(tO, tS + (kk < 4 ? kk * 8 : 64 + (kk - 4) * 8), b + mnmajor_off(kk), idesc_o,
                     !first || (kk > 0));
        }
        // the accumulator is only waited for after the unit's last PV (the lazy rescale, rare,
        // runs after S of the next tile is complete, whose commit covers this PV as well)
        if (last) mma_commit(bar(kODone + s));
      };
      for (uint32_t un_i = 0;; ++un_i) {
        PP_TAKE_UNIT(un_i, false)
        if (u_nslots == 0) break;
        const bool two = u_nslots == 2;
        wait_bar(bar(kQFull + 0), uc0 & 1, abort_flag, prm.header, 30);
        if (two) wait_bar(bar(kQFull + 1), uc1 & 1, abort_flag, prm.header, 31);
        int cur_len = u_klen(0);
        wait_bar(bar(kKFull + (kc & 1)), (kc >> 1) & 1, abort_flag, prm.header, 32);
        tc_fence_after();
        issue_qk(0, kc & 1, cur_len);
        if (u_ntiles == 1) mma_commit(bar(kQEmpty + 0));
        if (two) {
          issue_qk(1, kc & 1, cur_len);
          if (u_ntiles == 1) mma_commit(bar(kQEmpty + 1));
        }
        mma_commit(bar(kKEmpty + (kc & 1)));
        ++kc;
        for (int j = 0; j < u_ntiles; ++j) {
          const bool has_next = j + 1 < u_ntiles;
          const int nx_len = has_next ? u_klen(j + 1) : 0;
          const uint32_t vst = kc & 1, kst = kc & 1;   // stage {V(j), K(j + 1)}
          wait_bar(bar(kKFull + kst), (kc >> 1) & 1, abort_flag, prm.header, 33);
          // slot 0
          wait_bar(bar(kPFull + 0), tc0 & 1, abort_flag, prm.header, 35);
          if (j == 0) wait_bar(bar(kOFree + 0), (uc0 & 1) ^ 1, abort_flag, prm.header, 37);
          tc_fence_after();
          issue_pv(0, vst, cur_len, j == 0, !has_next);
          ++tc0;
          if (has_next) {
            issue_qk(0, kst, nx_len);
            if (j + 2 == u_ntiles) mma_commit(bar(kQEmpty + 0));
          }
          if (two) {
            wait_bar(bar(kPFull + 1), tc1 & 1, abort_flag, prm.header, 36);
            if (j == 0) wait_bar(bar(kOFree + 1), (uc1 & 1) ^ 1, abort_flag, prm.header, 38);
            tc_fence_after();
            issue_pv(1, vst, cur_len, j == 0, !has_next);
            ++tc1;
            if (has_next) {
              issue_qk(1, kst, nx_len);
              if (j + 2 == u_ntiles) mma_commit(bar(kQEmpty + 1));
            }
          }
          mma_commit(bar(kKEmpty + kst));
          ++kc;
          cur_len = nx_len;
        }
        ++uc0;
        if (two) ++uc1;
      }
    }
  } else if (warp >= 18) {
    // ------------------------------------------------------------ clearing warps (optional)
    // The kernel is compute-bound and leaves most of the memory bandwidth idle: when the
    // caller passes the backward's scratch, these two warps write zeros over the rows of the
    // fp32 dQ accumulator that belong to the unit's query tile and heads, so that the
    // backward needs no clearing pass.  Every (token, query head) row belongs to exactly one
    // unit and slot.
    if (prm.dq_clear) {
      const int cl = (warp - 18) * 32 + lane;  // 0..63
      for (uint32_t un_i = 0;; ++un_i) {
        PP_TAKE_UNIT(un_i, true)
        if (u_nslots == 0) break;
        constexpr int kChunks = DV / 4;  // 16-byte chunks per row
        const int total = u_len * kChunks;
        for (int sl = 0; sl < u_nslots; ++sl) {
          float* base = prm.dq_clear + (size_t(u_start) * prm.Hq + (u_h0 + sl)) * DV;
          for (int c = cl; c < total; c += 64) {
            const int r = c / kChunks, col = c - r * kChunks;
            *reinterpret_cast<float4*>(base + size_t(r) * prm.Hq * DV + col * 4) =
                make_float4(0.f, 0.f, 0.f, 0.f);
          }
        }
      }
    }
  } else {
    // ------------------------------------------------------------ softmax warps
    // Eight warps per slot: two threads share a query row (= TMEM lane), each owning 64 of
    // the tile's 128 key columns and D/2 of the output columns.  Halving the work per thread
    // keeps one slot's softmax shorter than the other slot's MMA phase, so the two slots'
    // exponentials do not pile up on the same MUFU at the same time.  The two halves of a row
    // exchange their partial maxima (every tile) and sums (once per unit) through shared
    // memory, guarded by a 64-thread named barrier per (slot, lane quarter).
    const int lw = warp - 2;                  // 0..15
    const int s = lw >> 3;                    // slot
    const int half = (lw >> 2) & 1;           // column half of the row
    const int qd = warp & 3;                  // lane quarter this warp may touch
    const int row = 32 * qd + lane;
    const int bar_id = 1 + s * 4 + qd;        // named barrier shared with the partner warp
    const uint32_t lane_base = tmem + (uint32_t(32 * qd) << 16);
    const uint32_t tS = lane_base + s * 128 + half * 64;   // my S columns; P goes to their start
    const uint32_t tO = lane_base + 256 + s * 128 + half * (D / 2);
    float* xch = reinterpret_cast<float*>(gbase + L::kXch) + s * 512;  // [2 buffers][128 rows][2]
    uint32_t tcS = 0, ucS = 0;
    for (uint32_t un_i = 0;; ++un_i) {
      PP_TAKE_UNIT(un_i, true)
      if (u_nslots == 0) break;
      if (s >= u_nslots) continue;
      float m_used = -INFINITY, l_part = 0.f;
      for (int j = 0; j < u_ntiles; ++j) {
        KvTile kt;
        kt.len = u_klen(j);
        kt.diag = j + 1 == u_ntiles;
        wait_bar(bar(kSFull + s), tcS & 1, abort_flag, prm.header, 40 + s);
        tc_fence_after();
        const bool full = !kt.diag && kt.len == kTile;
        // visible columns of this half: [0, col_lim) in the half's own numbering
        const int col_lim = (kt.diag ? min(kt.len, row + 1) : kt.len) - 64 * half;
        float* xb = xch + (tcS & 1) * 256 + row * 2;
        // The 64 scores of this thread are handled as two chunks of 32 (fewer live registers).
        // max over the visible scores of one chunk
        auto chunk_max = [&](const uint32_t (&w)[32], int c, float m) -> float {
          if (full) {
            float m1 = -INFINITY;
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
              m = max3(m, __uint_as_float(w[i]), __uint_as_float(w[i + 1]));
              m1 = max3(m1, __uint_as_float(w[i + 2]), __uint_as_float(w[i + 3]));
            }
            return fmaxf(m, m1);
          }
#pragma unroll
          for (int i = 0; i < 32; ++i) m = fmaxf(m, 32 * c + i < col_lim ? __uint_as_float(w[i]) : -INFINITY);
          return m;
        };
        float mx = -INFINITY;
        bool settled = (j == 0);
        if (settled) {
          // first tile of the unit: the reference maximum is needed before the exponentials
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            uint32_t w[32];
            tmem_ld32(tS + 32 * c, w);
            tmem_wait_ld();
            mx = chunk_max(w, c, mx);
          }
          xb[half] = mx;
          named_barrier_sync(bar_id, 64);
          m_used = fmaxf(mx, xb[half ^ 1]) * prm.scale_log2;
        }
        // Later tiles: the exponentials use the reference maximum of the previous tiles while
        // the half-row maxima are exchanged; only if the new maximum exceeds the reference by
        // more than the rescale threshold (rare) is the accumulator rescaled and the tile redone
        // from the S values, which stay in tensor memory until P is stored.
        uint32_t pk[32];
        float rs = 0.f;
        bool done = false;
        if (j > 0) {
          // Common path (every tile but a unit's first, whose exact row maximum is formed first
          // below -- with a guessed reference the largest P of a row would not be exactly 1,
          // and rows that see one or two keys would lose the exact cancellation in dP - Delta): the 64 scores go through in four pieces of 16, the tensor-memory load
          // of the next piece in flight under the exponentials of this one, and no maximum is
          // formed from the scores: the largest exponential tells as well whether the row has
          // outgrown its reference maximum by more than the rescale threshold
          // (p > 2^threshold), and its max3 rides in the MUFU-bound loop for free.  (Measured:
          // loads and the two maxima were 430 of a tile's 1850 softmax cycles, none of it
          // overlapped with the exponentials.)
          const float neg_m = -m_used;
          const uint64_t sc2 = pack2(prm.scale_log2, prm.scale_log2), nm2 = pack2(neg_m, neg_m);
          uint64_t sum2 = pack2(0.f, 0.f);
          float pm0 = 0.f, pm1 = 0.f;
          uint32_t wa[16], wb[16];
          auto exp16 = [&](const uint32_t (&w)[16], int piece, auto masked_c) {
            constexpr bool kMasked = decltype(masked_c)::value;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              float x0, x1;
              unpack2(fma2(pack2(__uint_as_float(w[2 * i]), __uint_as_float(w[2 * i + 1])), sc2, nm2), x0, x1);
              float p0 = ex2(x0), p1 = ex2(x1);
              if (kMasked) {   // columns at and past col_lim are not visible
                p0 = (16 * piece + 2 * i < col_lim) ? p0 : 0.f;
                p1 = (16 * piece + 2 * i + 1 < col_lim) ? p1 : 0.f;
              }
              sum2 = add2(sum2, pack2(p0, p1));
              if (i & 1) pm1 = max3(pm1, p0, p1); else pm0 = max3(pm0, p0, p1);
              pk[8 * piece + i] = pack_bf16(p0, p1);
            }
          };
          auto pieces = [&](auto masked_c) {
            tmem_ld16(tS, wa);
            tmem_wait_ld();
            tmem_ld16(tS + 16, wb);
            exp16(wa, 0, masked_c);
            tmem_wait_ld();
            tmem_ld16(tS + 32, wa);
            exp16(wb, 1, masked_c);
            tmem_wait_ld();
            tmem_ld16(tS + 48, wb);
            exp16(wa, 2, masked_c);
            tmem_wait_ld();
            exp16(wb, 3, masked_c);
          };
          if (full) pieces(std::false_type{}); else pieces(std::true_type{});
          float s0, s1;
          unpack2(sum2, s0, s1);
          rs = s0 + s1;
          const float pmax = fmaxf(pm0, pm1);
          xb[half] = pmax;
          named_barrier_sync(bar_id, 64);
          const float hi = fmaxf(pmax, xb[half ^ 1]);
          // (rows past the tile's end must not steer the warp-wide decision)
          const bool need = row < u_len && !(hi <= exp2f(kRescaleThreshold));
          if (!__any_sync(0xffffffffu, need)) done = true;   // same rows and values in the partner warp
          else xb = xch + ((tcS & 1) ^ 1) * 256 + row * 2;   // rare: the exact path below, which
                                                            // exchanges again, in the other buffer
        }
        if (!done)
        for (;;) {
          const float neg_m = -m_used;
          const uint64_t sc2 = pack2(prm.scale_log2, prm.scale_log2), nm2 = pack2(neg_m, neg_m);
          uint64_t sum2 = pack2(0.f, 0.f);
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            uint32_t w[32];
            tmem_ld32(tS + 32 * c, w);
            tmem_wait_ld();
            if (!settled) mx = chunk_max(w, c, mx);
            if (full) {
#pragma unroll
              for (int i = 0; i < 16; ++i) {
                float x0, x1;
                unpack2(fma2(pack2(__uint_as_float(w[2 * i]), __uint_as_float(w[2 * i + 1])), sc2, nm2), x0, x1);
                const float p0 = ex2(x0), p1 = ex2(x1);
                sum2 = add2(sum2, pack2(p0, p1));
                pk[16 * c + i] = pack_bf16(p0, p1);
              }
            } else {
#pragma unroll
              for (int i = 0; i < 16; ++i) {
                float p0 = ex2(fmaf(__uint_as_float(w[2 * i]), prm.scale_log2, neg_m));
                float p1 = ex2(fmaf(__uint_as_float(w[2 * i + 1]), prm.scale_log2, neg_m));
                p0 = (32 * c + 2 * i < col_lim) ? p0 : 0.f;
                p1 = (32 * c + 2 * i + 1 < col_lim) ? p1 : 0.f;
                sum2 = add2(sum2, pack2(p0, p1));
                pk[16 * c + i] = pack_bf16(p0, p1);
              }
            }
          }
          float s0, s1;
          unpack2(sum2, s0, s1);
          rs = s0 + s1;
          if (settled) break;
          xb[half] = mx;
          named_barrier_sync(bar_id, 64);
          const float m_new = fmaxf(m_used, fmaxf(mx, xb[half ^ 1]) * prm.scale_log2);
          // Rows past the tile's end hold whatever follows in memory: they must not steer the
          // warp-wide decision, or a row's rounding would depend on its neighbours' data.
          const bool need = row < u_len && (m_new - m_used) > kRescaleThreshold;
          if (!__any_sync(0xffffffffu, need)) break;  // same rows, same values in the partner warp
          const float alpha = ex2(m_used - m_new);
          // PV of the previous tile is complete: the commit that announced this tile's S was
          // issued after it and covers every earlier MMA of the issuing thread
#pragma unroll 1
          for (int c = 0; c < D / 16; ++c) {  // eight columns at a time
            uint32_t w[8];
            tmem_ld8(tO + c * 8, w);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 8; ++i) w[i] = __float_as_uint(__uint_as_float(w[i]) * alpha);
            tmem_st8(tO + c * 8, w);
          }
          l_part *= alpha;
          m_used = m_new;
          settled = true;
        }
        l_part += rs;
        tmem_st32(tS, pk);  // P over the first half of my own S columns
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar(kPFull + s));
        ++tcS;
      }
      // ---- epilogue: row sum from both halves, O / l -> bf16, release the accumulator, store
      float* xb = xch + (tcS & 1) * 256 + row * 2;
      xb[half] = l_part;
      named_barrier_sync(bar_id, 64);
      const float l_run = l_part + xb[half ^ 1];
      wait_bar(bar(kODone + s), ucS & 1, abort_flag, prm.header, 44 + s);
      ++ucS;
      tc_fence_after();
      const float inv_l = 1.f / l_run;
      uint32_t ob[D / 4];
#pragma unroll
      for (int c = 0; c < D / 64; ++c) {
        uint32_t w[32];
        // (columns at and past DV hold nothing and are not stored: the zeros only fill ob)
        if (DV == D || half * (D / 2) + c * 32 < DV) {
          tmem_ld32(tO + c * 32, w);
          tmem_wait_ld();
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) w[i] = 0u;
        }
#pragma unroll
        for (int i = 0; i < 16; ++i)
          ob[c * 16 + i] = pack_bf16(__uint_as_float(w[2 * i]) * inv_l, __uint_as_float(w[2 * i + 1]) * inv_l);
      }
      tc_fence_before();
      mbar_arrive(bar(kOFree + s));
      // the exchange buffer of parity (tcS & 1) is written again two uses later, after another
      // barrier: no further synchronisation needed here
      const int h = u_h0 + s;
      if (half == 0 && row < u_len)
        prm.lse[size_t(h) * prm.T + u_start + row] = (m_used + log2f(l_run)) * 0.69314718055994531f;
      // A thread holds kCh 16-byte chunks of one row; transposing them inside groups of kCh
      // lanes gives every lane the same chunk of kCh consecutive rows, so that one store
      // instruction of the warp writes whole contiguous half-rows instead of 32 scattered
      // 16-byte pieces.
      constexpr int kCh = D / 16;
      auto exchange = [&](auto dist) {
        constexpr int d = decltype(dist)::value;
        if constexpr (d < kCh) {
          const bool hi = (lane & d) != 0;
#pragma unroll
          for (int i = 0; i < kCh; ++i) {
            if ((i & d) == 0) {
#pragma unroll
              for (int c = 0; c < 4; ++c) {
                const uint32_t send = hi ? ob[4 * i + c] : ob[4 * (i | d) + c];
                const uint32_t recv = __shfl_xor_sync(0xffffffffu, send, d);
                if (hi) ob[4 * i + c] = recv; else ob[4 * (i | d) + c] = recv;
              }
            }
          }
        }
      };
      exchange(std::integral_constant<int, 4>{});
      exchange(std::integral_constant<int, 2>{});
      exchange(std::integral_constant<int, 1>{});
      {
        const int grp = lane / kCh, chunk = lane % kCh;
#pragma unroll
        for (int i = 0; i < kCh; ++i) {
          const int r = 32 * qd + grp * kCh + i;
          if (r < u_len && (DV == D || half * (D / 2) + chunk * 8 < DV)) {
            uint4* dst = reinterpret_cast<uint4*>(
                prm.o + ((size_t(u_start) + r) * prm.Hq + h) * DV + half * (D / 2) + chunk * 8);
            *dst = make_uint4(ob[4 * i], ob[4 * i + 1], ob[4 * i + 2], ob[4 * i + 3]);
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  // After a wait that gave up, copies and MMAs issued without their barriers may still be in
  // flight: give them time to land before the CTA's shared and tensor memory are released.
  if (*abort_flag)
    for (int i = 0; i < 50; ++i) __nanosleep(1000);
  if (warp == 0) tmem_dealloc(tmem, kFwdTmemCols);
  if (tid == 0) {  // the last CTA to finish re-arms the unit counter for the next launch
    __threadfence();
    if (atomicAdd(&prm.header[kHdrFwdDone], 1) == int(gridDim.x) - 1) {
      prm.header[kHdrFwdNext] = 0;
      prm.header[kHdrFwdDone] = 0;
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
extern "C" int pp_debug_fwd_cta_cycles(unsigned long long* out) {
  return cudaMemcpyFromSymbol(out, pp::g_cta_cycles, sizeof(unsigned long long) * 256) == cudaSuccess ? 0 : -5;
}
extern "C" int pp_debug_fwd_wait_cycles(unsigned long long* out, int reset) {
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
cudaError_t launch_fwd_t(const pp_plan* plan, const CUtensorMap& tq, const CUtensorMap& tk,
                         const CUtensorMap& tv, const FwdParams& prm, cudaStream_t stream) {
  static DeviceSetup setup[kMaxDevices];
  DeviceSetup* dev = device_setup(setup);
  if (!dev) return cudaErrorInvalidDevice;
  if (dev->cc_major != 10) return cudaErrorNotSupported;
  auto kern = fwd_kernel<D, DV>;
  if (!dev->configured) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         FwdSmem<D>::kTotal);
    if (e != cudaSuccess) return e;
    dev->configured = true;
  }
  const int num_sms = dev->num_sms;
  const pp_problem& pb = plan->prob;
  const int r = pb.num_q_heads / pb.num_kv_heads;
  const long long units = (long long)plan->max_tiles * pb.num_kv_heads * ((r + 1) / 2);
  dim3 grid(unsigned(std::min<long long>(units, num_sms)));
  ProfileEvents& ev = profile_events();
  const int slot = int(ev.fwd_count % kProfileRing);
  if (ev.on && ev.fwd_on) profile_record(ev.fwd0[slot], stream);
  kern<<<grid, kFwdThreads, FwdSmem<D>::kTotal, stream>>>(tq, tk, tv, prm);
  if (ev.on && ev.fwd_on) {
    profile_record(ev.fwd1[slot], stream);
    ++ev.fwd_count;
  }
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_fwd(const pp_plan* plan, const void* q, const void* k, const void* v, float scale,
                       void* o, float* lse, float* dq_clear, cudaStream_t stream, int* launches) {
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
  prm.dq_clear = dq_clear;
  prm.T = pb.total_tokens;
  prm.Hq = pb.num_q_heads;
  prm.Hkv = pb.num_kv_heads;
  prm.scale_log2 = scale * 1.4426950408889634f;
  cudaError_t e = pb.head_dim == 128  ? launch_fwd_t<128>(plan, tq, tk, tv, prm, stream)
                  : pb.head_dim == 96 ? launch_fwd_t<128, 96>(plan, tq, tk, tv, prm, stream)
                                      : launch_fwd_t<64>(plan, tq, tk, tv, prm, stream);
  if (e == cudaSuccess && launches) *launches += 1;
  return e;
}

}  // namespace pp
