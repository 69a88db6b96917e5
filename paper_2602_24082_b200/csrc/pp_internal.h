// Internal definitions shared by the plan builder, the kernels and the C ABI.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/pp_attn.h"

namespace pp {

constexpr int kTile = 128;  // query-tile and key-tile length in tokens

// One tile of a segment (prompt or response).  Read as a query tile it lists the keys it
// sees; read as a key tile it lists the queries that see it.
struct Tile {
  int32_t start;      // first token
  int32_t len;        // 1..128 tokens
  int32_t kv0_start;  // FULL range 0: prompt keys visible to every row of the tile
  int32_t kv0_len;    //   (for a prompt tile: the prompt keys before the tile)
  int32_t kv1_start;  // FULL range 1: own-response keys before the tile (0 for prompt tiles)
  int32_t kv1_len;
  int32_t vis_end;    // queries [start, vis_end) see this tile's keys (causally inside the tile)
  int32_t work;       // forward work estimate in key tiles (backward: derived)
};
static_assert(sizeof(Tile) == 32, "tile record is 32 bytes");

// One key tile of the backward pass.  The backward cuts each GROUP (prompt and responses as one
// token range) into tiles of 128 tokens from the group's start, so a tile may straddle segment
// boundaries: short segments then leave no ragged tile each, only the group's last tile is
// short.  Key j of the tile is seen by the queries [j, key_end[j]); the query tiles of the unit
// are the tiles of the same grid from this one on, up to vis_end.
struct BTile {
  int32_t start;      // first token
  int32_t len;        // 1..128 tokens
  int32_t vis_end;    // largest key_end of the tile's keys: queries [start, vis_end) see some key
  int32_t dep_lo;     // read as a query tile: besides the prompt tiles [0, npc), the key tiles
                      //   [dep_lo, own index] of the group's grid add to its dQ
  int32_t grp_start;  // first token of the group (also the group's identity)
  int32_t grp_end;    // one past the last token of the group
  int32_t work;       // number of query tiles: 1 + ceil((vis_end - start - len) / 128)
  int32_t npc;        // tiles of the group that hold prompt keys: ceil(prompt length / 128)
};
static_assert(sizeof(BTile) == 32, "backward tile record is 32 bytes");

// Words of the plan header (int32[16]).
constexpr int kHdrStatus = 0, kHdrDetail = 1, kHdrNumTiles = 2, kHdrNumSegments = 3,
              kHdrNumBTiles = 8;

// Status word values written by device code.
enum : int32_t {
  kStatusOk = 0,
  kStatusBadDescriptor = 1,  // detail = index of the offending group / response
  kStatusTokenMismatch = 2,  // detail = token count found
  kStatusWaitExpired = 3,    // detail = site id
};

// Device part of a plan: offsets (bytes) into the caller's workspace.
struct PlanLayout {
  size_t header;     // int32[16]: status, detail, num_tiles, num_segments, counters, num_btiles
  size_t desc;       // device copy of the descriptor arrays (when given on host)
  size_t seg_start;  // int32[nseg + 1]
  size_t seg_tile0;  // int32[nseg + 1]  first tile of each segment
  size_t tiles;      // Tile[max_tiles]
  size_t fwd_order;  // int32[max_tiles]
  size_t grp_btile0; // int32[G + 1]  first backward tile of each group
  size_t btiles;     // BTile[max_tiles]  (at most T / 128 + G of them)
  size_t bwd_order;  // int32[max_tiles]  backward tiles, longest work first
  size_t tile_gwork; // int32[max_tiles]  backward work of the backward tile's whole group
  size_t tile_sgroup; // int32[max_tiles] super-group (block of consecutive groups)
  size_t bwd_units;  // int32[max_tiles * Hkv]  (kv head << 24) | backward tile, processing order
  size_t bwd_units_det;  // the same units, one (group, KV head) set after the other and inside a
                         //   set by descending tile index: the order of the deterministic backward
  size_t key_end;    // int32[T]
  size_t total;
};

}  // namespace pp

struct pp_plan {
  pp_problem prob;  // descriptor pointers are rewritten to the copies in the workspace
  // Descriptors given on the device: the caller's arrays, which the first plan kernel copies
  // into the workspace (null when the host path has staged them already).
  const int32_t* src_desc[4] = {nullptr, nullptr, nullptr, nullptr};
  int nseg;
  int max_tiles;
  char* ws;
  pp::PlanLayout lay;
  // scratch sizes
  size_t fwd_scratch, bwd_scratch;
  // backward scratch whose dQ accumulator the latest forward on this plan has cleared
  mutable const void* cleared_scratch = nullptr;
};

namespace pp {

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

inline int max_tiles_of(const pp_problem& p) {
  // sum over segments of ceil(len / 128) <= T / 128 + number of segments
  return p.total_tokens / kTile + p.num_groups + p.num_responses;
}

inline PlanLayout plan_layout(const pp_problem& p) {
  PlanLayout l{};
  int nseg = p.num_groups + p.num_responses;
  int mt = max_tiles_of(p);
  size_t off = 0;
  l.header = off;    off = align_up(off + 64, 256);
  l.desc = off;
  off = align_up(off + sizeof(int32_t) * (size_t(p.num_rows) + 1 + p.num_groups +
                                           (p.num_groups + 1) + p.num_responses), 256);
  l.seg_start = off; off = align_up(off + sizeof(int32_t) * (nseg + 1), 256);
  l.seg_tile0 = off; off = align_up(off + sizeof(int32_t) * (nseg + 1), 256);
  l.tiles = off;     off = align_up(off + sizeof(Tile) * size_t(mt), 256);
  l.fwd_order = off; off = align_up(off + sizeof(int32_t) * size_t(mt), 256);
  l.grp_btile0 = off; off = align_up(off + sizeof(int32_t) * (size_t(p.num_groups) + 1), 256);
  l.btiles = off;    off = align_up(off + sizeof(BTile) * size_t(mt), 256);
  l.bwd_order = off; off = align_up(off + sizeof(int32_t) * size_t(mt), 256);
  l.tile_gwork = off; off = align_up(off + sizeof(int32_t) * size_t(mt), 256);
  l.tile_sgroup = off; off = align_up(off + sizeof(int32_t) * size_t(mt), 256);
  l.bwd_units = off; off = align_up(off + sizeof(int32_t) * size_t(mt) * size_t(p.num_kv_heads), 256);
  l.bwd_units_det = off;
  off = align_up(off + sizeof(int32_t) * size_t(mt) * size_t(p.num_kv_heads), 256);
  l.key_end = off;   off = align_up(off + sizeof(int32_t) * size_t(p.total_tokens), 256);
  l.total = off;
  return l;
}

// Backward scratch: fp32 dQ accumulator [T][Hq][D], Delta [Hq][T], LSE*log2(e) [Hq][T], and
// the turn counters of the deterministic variant, one per (query tile of the backward grid,
// query head)
struct BwdScratch {
  size_t dq_acc, delta, lse2, sem, sem_bytes, total;
};
inline BwdScratch bwd_scratch_layout(const pp_problem& p) {
  BwdScratch s{};
  size_t T = p.total_tokens, Hq = p.num_q_heads, D = p.head_dim;
  size_t off = 0;
  s.dq_acc = off; off = align_up(off + 4 * T * Hq * D, 256);
  s.delta = off;  off = align_up(off + 4 * T * Hq, 256);
  s.lse2 = off;   off = align_up(off + 4 * T * Hq, 256);
  s.sem = off;
  s.sem_bytes = 4 * size_t(max_tiles_of(p)) * Hq;
  off = align_up(off + s.sem_bytes, 256);
  s.total = off;
  return s;
}

// Device arena of pp_attn_step_host: inputs, outputs, plan workspace, backward scratch.  The
// step is cut into at most kStepChunks runs of whole groups, each with its own plan, scratch and
// LSE block inside the shared regions; the regions carry the alignment slack that costs.
constexpr int kStepChunks = 8;
struct StepArena {
  size_t q, k, v, d_o, o, lse, dq, dk, dv, plan, scratch, total;
};
inline StepArena step_arena_layout(const pp_problem& p) {
  StepArena a{};
  const size_t T = p.total_tokens, D = p.head_dim;
  const size_t qb = T * p.num_q_heads * D * 2, kb = T * p.num_kv_heads * D * 2;
  size_t off = 0;
  auto take = [&](size_t n) { size_t o = off; off = align_up(off + n, 256); return o; };
  a.q = take(qb); a.k = take(kb); a.v = take(kb); a.d_o = take(qb);
  a.o = take(qb); a.lse = take(T * p.num_q_heads * 4 + 256 * kStepChunks);
  a.dq = take(qb); a.dk = take(kb); a.dv = take(kb);
  a.plan = take(plan_layout(p).total + size_t(16384) * kStepChunks);
  a.scratch = take(bwd_scratch_layout(p).total + size_t(4096) * kStepChunks);
  a.total = off;
  return a;
}

// Per-device launch state of a kernel family: the opt-in to large dynamic shared memory is a
// per-device function attribute, and the SM count differs between devices, so a process that
// drives several GPUs must set up each of them.
constexpr int kMaxDevices = 64;
struct DeviceSetup {
  bool configured = false;
  int num_sms = 0;
  int cc_major = 0;
};
// Entry for the current device in `table` (kMaxDevices entries), or null.
inline DeviceSetup* device_setup(DeviceSetup* table) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  DeviceSetup* d = table + dev;
  if (!d->num_sms &&
      (cudaDeviceGetAttribute(&d->cc_major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
       cudaDeviceGetAttribute(&d->num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess))
    return nullptr;
  return d;
}
// The kernels are sm_100a code (tcgen05, tensor memory): any other device is refused before a
// launch is attempted.  Checked once per device.
inline bool device_is_sm100() {
  static DeviceSetup probe[kMaxDevices];
  DeviceSetup* d = device_setup(probe);
  return d && d->cc_major == 10;
}

// Optional event pairs around the forward kernel and the backward main kernel.
// A ring of pairs per kernel, so that a benchmark can time many steps and read the durations
// afterwards instead of synchronising after every step.
constexpr int kProfileRing = 64;
struct ProfileEvents {
  bool on = false;
  bool fwd_on = false;  // forward events wanted too (mode 1); mode 2 times the backward only
  cudaEvent_t fwd0[kProfileRing] = {}, fwd1[kProfileRing] = {}, bwd0[kProfileRing] = {},
              bwd1[kProfileRing] = {};
  long long fwd_count = 0, bwd_count = 0;   // launches recorded since the events were enabled
};
ProfileEvents& profile_events();
// Records a profiling event.  On a capturing stream the record becomes a node of the graph
// that marks the event at every replay (an ordinary record would only order the capture).
inline void profile_record(cudaEvent_t ev, cudaStream_t stream) {
  cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(stream, &st) == cudaSuccess && st == cudaStreamCaptureStatusActive)
    cudaEventRecordWithFlags(ev, stream, cudaEventRecordExternal);
  else
    cudaEventRecord(ev, stream);
}
bool profile_enable(int mode);
bool profile_read(float* fwd_ms, float* bwd_ms);
bool profile_read_all(float* fwd_ms, float* bwd_ms, int capacity, int* n_fwd, int* n_bwd);

// launchers (defined in the .cu files); all return a cudaError_t
cudaError_t launch_plan(const pp_plan* plan, cudaStream_t stream, int* launches);
cudaError_t launch_fwd(const pp_plan* plan, const void* q, const void* k, const void* v, float scale,
                       void* o, float* lse, float* dq_clear, cudaStream_t stream, int* launches);
cudaError_t launch_bwd(const pp_plan* plan, const void* q, const void* k, const void* v,
                       const void* o, const float* lse, const void* d_o, float scale, void* dq,
                       void* dk, void* dv, void* scratch, bool dq_cleared, bool deterministic,
                       cudaStream_t stream, int* launches);

// Row builder (csrc/pp_rows.cu).
size_t rows_workspace_bytes(int num_groups);
cudaError_t launch_build_rows(int G, int N, const int32_t* prompt_len, const int32_t* resp_off,
                              const int32_t* resp_len, int capacity, void* ws, int32_t* order,
                              int32_t* row_group_off, int32_t* num_rows, long long* row_tokens,
                              long long* row_cost, int32_t* out_prompt_len, int32_t* out_resp_off,
                              int32_t* out_resp_len, int32_t* status, cudaStream_t stream,
                              int* launches);

cudaError_t launch_assign_rows(int R, const long long* row_cost, int ranks, int32_t* order,
                               int32_t* rank_of_row, long long* rank_cost, cudaStream_t stream,
                               int* launches);

// Size of the scratch array built into the library image for pp_attn_bwd_noalloc.
constexpr size_t kStaticScratchBytes = size_t(32) << 20;
cudaError_t launch_bwd_static(const pp_plan* plan, const void* q, const void* k, const void* v,
                              const void* o, const float* lse, const void* d_o, float scale,
                              void* dq, void* dk, void* dv, cudaStream_t stream, int* launches);

cudaError_t launch_position_ids(const pp_plan* plan, int32_t* pos, cudaStream_t stream);
cudaError_t launch_rope(const pp_plan* plan, void* q, void* k, float base, cudaStream_t stream);

cudaError_t launch_preference_loss(const pp_plan* plan, const float* logp, const float* ref,
                                   float beta, float* resp_logp, float* resp_reward,
                                   float* grp_loss, float* d_logp, cudaStream_t stream);

}  // namespace pp
