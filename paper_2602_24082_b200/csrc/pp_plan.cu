// Device-side plan builder: segment descriptors -> tiles, visible key/query ranges, orders.
//
// The packing mask (paper Sec. 3.2) has a simple structure once tokens are grouped by
// segment: a key j is seen by the contiguous queries [j, end_j) where end_j is the end of
// j's group for a prompt key and the end of j's own response otherwise; a query sees at
// most two contiguous key ranges (its group's prompt, and its own segment up to itself).
// Forward tiles are cut per segment (aligned to the segment start), so a tile never straddles
// two segments and only its own diagonal block needs element-wise causal masking.  The
// backward has its own key tiles, cut per group (see BTile): its masks are two comparisons per
// element with per-key bounds, so straddling costs nothing there and short segments leave no
// ragged tiles.
#include <algorithm>

#include "pp_internal.h"

namespace pp {
namespace {

struct PlanPtrs {
  int32_t* header;
  // descriptors given on the device: the caller's arrays (null otherwise) and the workspace
  // block they are copied into, which is what row_group_off .. resp_len below point at
  const int32_t* src_desc[4];
  int32_t* desc_copy;
  const int32_t* row_group_off;
  const int32_t* grp_prompt_len;
  const int32_t* grp_resp_off;
  const int32_t* resp_len;
  int32_t* seg_start;
  int32_t* seg_tile0;
  Tile* tiles;
  int32_t* grp_btile0;
  BTile* btiles;
  int32_t* fwd_order;
  int32_t* bwd_order;
  int32_t* tile_gwork;
  int32_t* tile_sgroup;
  int32_t* bwd_units;
  int32_t* bwd_units_det;
  int Hkv;
  int32_t* key_end;
  int det_asc_max;  // deterministic order: sets of at most this many tiles are handed out longest first
  int num_rows, G, N, T, nseg, max_tiles;
};

__device__ __forceinline__ void set_status(int32_t* header, int32_t status, int32_t detail) {
  if (atomicCAS(&header[0], kStatusOk, status) == kStatusOk) header[1] = detail;
}

// Segment order: group 0 prompt, group 0 responses, group 1 prompt, ...  so the prompt of
// group g is segment g + resp_off[g] and response x (global index) of group g is g + 1 + x.

// One block of 1024 threads.  Validates, writes segment lengths, scans them into seg_start /
// seg_tile0.  Returns (uniformly) whether the descriptors were accepted.
__device__ __forceinline__ bool plan_scan_body(const PlanPtrs& p) {
  __shared__ int32_t s_tok[1024];
  __shared__ int32_t s_til[1024];
  __shared__ int32_t s_carry[2];
  const int tid = threadIdx.x;

  // Descriptors handed over on the device are copied into the workspace first: everything
  // after this call -- the later plan kernels, position ids, rotary embedding, the loss -- reads
  // the copy, so the caller's arrays are free again once this kernel has run.
  if (p.src_desc[0]) {
    const int n[4] = {p.num_rows + 1, p.G, p.G + 1, p.N};
    int32_t* dst = p.desc_copy;
    for (int a = 0; a < 4; ++a) {
      for (int i = tid; i < n[a]; i += blockDim.x) dst[i] = p.src_desc[a][i];
      dst += n[a];
    }
    __syncthreads();
  }
  if (tid == 0) {
    p.header[0] = kStatusOk;
    p.header[1] = 0;
    p.header[2] = 0;
    p.header[3] = p.nseg;
    for (int i = 4; i < 16; ++i) p.header[i] = 0;  // [4,8): dynamic-scheduling counters
    if (p.row_group_off[0] != 0 || p.row_group_off[p.num_rows] != p.G)
      set_status(p.header, kStatusBadDescriptor, -1);
    if (p.grp_resp_off[0] != 0 || p.grp_resp_off[p.G] != p.N)
      set_status(p.header, kStatusBadDescriptor, -2);
    s_carry[0] = 0;
    s_carry[1] = 0;
  }
  __syncthreads();
  for (int r = tid; r < p.num_rows; r += blockDim.x)
    if (p.row_group_off[r + 1] < p.row_group_off[r]) set_status(p.header, kStatusBadDescriptor, r);
  // segment lengths (stored in seg_start, scanned in place below)
  for (int g = tid; g < p.G; g += blockDim.x) {
    int lo = p.grp_resp_off[g], hi = p.grp_resp_off[g + 1];
    bool ok = p.grp_prompt_len[g] >= 1 && hi > lo && lo >= 0 && hi <= p.N;
    if (!ok) {
      set_status(p.header, kStatusBadDescriptor, g);
      continue;
    }
    p.seg_start[g + lo] = p.grp_prompt_len[g];
    for (int x = lo; x < hi; ++x) {
      int len = p.resp_len[x];
      if (len < 1) set_status(p.header, kStatusBadDescriptor, p.G + x);
      p.seg_start[g + 1 + x] = len;
    }
  }
  __syncthreads();
  if (p.header[0] != kStatusOk) return false;

  // chunked exclusive scan of lengths and tile counts
  for (int base = 0; base < p.nseg; base += blockDim.x) {
    int s = base + tid;
    int len = s < p.nseg ? p.seg_start[s] : 0;
    // guard against overflow from absurd lengths
    if (len > p.T) len = p.T + 1;
    int til = (len + kTile - 1) / kTile;
    s_tok[tid] = len;
    s_til[tid] = til;
    __syncthreads();
    for (int d = 1; d < (int)blockDim.x; d <<= 1) {
      int a = tid >= d ? s_tok[tid - d] : 0;
      int b = tid >= d ? s_til[tid - d] : 0;
      __syncthreads();
      // saturate so a corrupted descriptor cannot wrap around
      s_tok[tid] = min(s_tok[tid] + a, 0x3fffffff);
      s_til[tid] += b;
      __syncthreads();
    }
    if (s < p.nseg) {
      p.seg_start[s] = s_carry[0] + s_tok[tid] - len;
      p.seg_tile0[s] = s_carry[1] + s_til[tid] - til;
    }
    __syncthreads();
    if (tid == blockDim.x - 1) {
      s_carry[0] = min(s_carry[0] + s_tok[tid], 0x3fffffff);
      s_carry[1] += s_til[tid];
    }
    __syncthreads();
  }
  if (tid == 0) {
    p.seg_start[p.nseg] = s_carry[0];
    p.seg_tile0[p.nseg] = s_carry[1];
    if (s_carry[0] != p.T) {
      set_status(p.header, kStatusTokenMismatch, s_carry[0]);
    } else {
      p.header[2] = s_carry[1];  // number of tiles
    }
  }
  __syncthreads();
  if (p.header[0] != kStatusOk) return false;

  // backward tiles: ceil(group length / 128) per group, exclusive scan over the groups
  if (tid == 0) s_carry[1] = 0;
  __syncthreads();
  for (int base = 0; base < p.G; base += blockDim.x) {
    const int g = base + tid;
    int til = 0;
    if (g < p.G) {
      const int gs = p.seg_start[g + p.grp_resp_off[g]];
      const int ge = p.seg_start[(g + 1) + p.grp_resp_off[g + 1]];
      til = (ge - gs + kTile - 1) / kTile;
    }
    s_til[tid] = til;
    __syncthreads();
    for (int d = 1; d < (int)blockDim.x; d <<= 1) {
      int b = tid >= d ? s_til[tid - d] : 0;
      __syncthreads();
      s_til[tid] += b;
      __syncthreads();
    }
    if (g < p.G) p.grp_btile0[g] = s_carry[1] + s_til[tid] - til;
    __syncthreads();
    if (tid == blockDim.x - 1) s_carry[1] += s_til[tid];
    __syncthreads();
  }
  if (tid == 0) {
    p.grp_btile0[p.G] = s_carry[1];
    p.header[kHdrNumBTiles] = s_carry[1];
  }
  __syncthreads();
  return true;
}

__global__ void __launch_bounds__(1024) plan_scan_kernel(PlanPtrs p) { plan_scan_body(p); }

// largest s in [0, n) with a[s] <= x  (a is non-decreasing, a[0] <= x)
__device__ __forceinline__ int upper_segment(const int32_t* a, int n, int x) {
  int lo = 0, hi = n;
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (a[mid] <= x) lo = mid; else hi = mid;
  }
  return lo;
}

// group of segment s: the largest g with g + resp_off[g] <= s
__device__ __forceinline__ int group_of_segment(const PlanPtrs& p, int s) {
  int lo = 0, hi = p.G;
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (mid + p.grp_resp_off[mid] <= s) lo = mid; else hi = mid;
  }
  return lo;
}

__device__ __forceinline__ void plan_tile_body(const PlanPtrs& p, int t) {
  int s = upper_segment(p.seg_tile0, p.nseg, t);
  // segments with zero tiles cannot exist (len >= 1), so seg_tile0 is strictly increasing
  int g = group_of_segment(p, s);
  int sp = g + p.grp_resp_off[g];             // the group's prompt segment
  int gs = p.seg_start[sp];
  int P = p.grp_prompt_len[g];
  int gend = p.seg_start[(g + 1) + p.grp_resp_off[g + 1]];  // next group's prompt (or T)
  int ss = p.seg_start[s], se = p.seg_start[s + 1];
  int start = ss + (t - p.seg_tile0[s]) * kTile;
  Tile tl;
  tl.start = start;
  tl.len = min(kTile, se - start);
  if (s == sp) {
    tl.kv0_start = gs;  tl.kv0_len = start - gs;
    tl.kv1_start = start; tl.kv1_len = 0;
    tl.vis_end = gend;
  } else {
    tl.kv0_start = gs;  tl.kv0_len = P;
    tl.kv1_start = ss;  tl.kv1_len = start - ss;
    tl.vis_end = se;
  }
  tl.work = (tl.kv0_len + kTile - 1) / kTile + (tl.kv1_len + kTile - 1) / kTile + 1;
  p.tiles[t] = tl;
}

__global__ void plan_tiles_kernel(PlanPtrs p) {
  if (p.header[0] != kStatusOk) return;
  int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t < p.header[2]) plan_tile_body(p, t);
}

__device__ __forceinline__ void plan_key_end_body(const PlanPtrs& p, int j) {
  int s = upper_segment(p.seg_start, p.nseg, j);
  int g = group_of_segment(p, s);
  bool prompt = (s == g + p.grp_resp_off[g]);
  p.key_end[j] = prompt ? p.seg_start[(g + 1) + p.grp_resp_off[g + 1]] : p.seg_start[s + 1];
}

__global__ void plan_key_end_kernel(PlanPtrs p) {
  if (p.header[0] != kStatusOk) return;
  int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j < p.T) plan_key_end_body(p, j);
}

// Backward tile t: tile k of its group's 128-token grid.
__device__ __forceinline__ void plan_btile_body(const PlanPtrs& p, int t) {
  const int g = upper_segment(p.grp_btile0, p.G, t);
  const int sp = g + p.grp_resp_off[g];  // the group's prompt segment
  const int gs = p.seg_start[sp];
  const int pe = p.seg_start[sp + 1];    // end of the prompt
  const int ge = p.seg_start[(g + 1) + p.grp_resp_off[g + 1]];
  BTile b;
  b.start = gs + (t - p.grp_btile0[g]) * kTile;
  b.len = min(kTile, ge - b.start);
  b.grp_start = gs;
  b.grp_end = ge;
  // segments of the first and of the last key
  const int s_first = upper_segment(p.seg_start, p.nseg, b.start);
  const int s_last = upper_segment(p.seg_start, p.nseg, b.start + b.len - 1);
  // key_end is the group's end for prompt keys and the own response's end otherwise; along
  // the tile it is: (group end for the prompt part,) then increasing response ends
  b.vis_end = (s_first == sp) ? ge : p.seg_start[s_last + 1];
  b.work = 1 + (b.vis_end - (b.start + b.len) + kTile - 1) / kTile;
  b.npc = (pe - gs + kTile - 1) / kTile;
  // Read as a QUERY tile: the key tiles that add to its dQ are the prompt tiles [0, npc) and
  // the tiles [dep_lo, own index] -- from the one holding the start of the first row's own
  // response on (earlier tiles past the prompt hold only earlier responses' keys).
  const int k_rel = (b.start - gs) / kTile;
  b.dep_lo = k_rel;
  if (b.start >= pe) b.dep_lo = max(b.npc, (p.seg_start[s_first] - gs) / kTile);
  p.btiles[t] = b;
}

__global__ void plan_btiles_kernel(PlanPtrs p) {
  if (p.header[0] != kStatusOk) return;
  int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t < p.header[kHdrNumBTiles]) plan_btile_body(p, t);
}

// Longest-work-first orders by rank counting (tile counts are small: T/128 + segments).
__device__ __forceinline__ void plan_fwd_order_body(const PlanPtrs& p, int t, int n) {
  const int wf = p.tiles[t].work;
  int rf = 0;
  for (int u = 0; u < n; ++u) {
    const int of = p.tiles[u].work;
    rf += (of > wf) || (of == wf && u < t);
  }
  p.fwd_order[rf] = t;
}

__global__ void plan_fwd_order_kernel(PlanPtrs p) {
  if (p.header[0] != kStatusOk) return;
  const int n = p.header[kHdrNumTiles];
  int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t < n) plan_fwd_order_body(p, t, n);
}

// Backward processing order, built for L2 reuse and balance.  Key tiles of one group stream
// the same Q / dO tiles, so groups are taken in order of decreasing work and consecutive
// groups are merged into super-groups of about kSuperGroupUnits units (cut from the end of
// the list, so the last block is a full one); inside a super-group
// units are ordered longest first (all KV heads of a tile adjacent).  Small problems collapse
// into one super-group, i.e. a plain longest-first list; large ones keep the working set of the
// concurrently running units near one group's Q / dO.  Dynamic scheduling in the kernel does
// the balancing.  A tile's group is identified by the group's first token.
constexpr int kSuperGroupUnits = 600;

// bwd_order (plain longest-first list of the backward tiles) and each tile's group work
__device__ __forceinline__ void plan_gwork_body(const PlanPtrs& p, int t, int n) {
  const BTile me = p.btiles[t];
  int gw = 0, rb = 0;
  for (int u = 0; u < n; ++u) {
    const BTile o = p.btiles[u];
    gw += (o.grp_start == me.grp_start) ? o.work : 0;
    rb += (o.work > me.work) || (o.work == me.work && u < t);
  }
  p.tile_gwork[t] = gw;
  p.bwd_order[rb] = t;
}

__device__ __forceinline__ void plan_sgroup_body(const PlanPtrs& p, int t, int n) {
  const int gs = p.btiles[t].grp_start, gw = p.tile_gwork[t];
  int rest = 0;  // tiles of this group and of the groups that come later
  for (int u = 0; u < n; ++u) {
    const int ogs = p.btiles[u].grp_start, ow = p.tile_gwork[u];
    rest += (ogs == gs) || (ow < gw) || (ow == gw && ogs > gs);
  }
  // counted from the END of the list, so the last block is never a small leftover whose
  // long units would start late: blocks are processed in decreasing index
  p.tile_sgroup[t] = (p.Hkv * rest - 1) / kSuperGroupUnits;
}

__device__ __forceinline__ void plan_units_body(const PlanPtrs& p, int t, int n) {
  const int sg = p.tile_sgroup[t], wb = p.btiles[t].work;
  int pos = 0;
  for (int u = 0; u < n; ++u) {
    const int osg = p.tile_sgroup[u], ob = p.btiles[u].work;
    pos += (osg > sg) || (osg == sg && ((ob > wb) || (ob == wb && u < t)));
  }
  for (int kvh = 0; kvh < p.Hkv; ++kvh) p.bwd_units[p.Hkv * pos + kvh] = (kvh << 24) | t;
  // Deterministic order: one (group, KV head) set after the other, groups by decreasing work.
  // The tiles add to a query tile's dQ in descending order, so a unit waits for the unit of the
  // next tile.  Inside a set the units go out in ascending tile order (longest first, as in the
  // default order) when the set is small against the grid: only the one set at the frontier of
  // the list can have units waiting for a unit that has not been handed out yet, so fewer than
  // det_asc_max CTAs can be held up that way and the others keep drawing.  Larger sets go out
  // in DESCENDING tile order, where every unit follows the units it waits for.
  const int gs = p.btiles[t].grp_start, gw = p.tile_gwork[t];
  int before = 0, ng = 0;  // tiles of groups ranked earlier; tiles of this group
  for (int u = 0; u < n; ++u) {
    const int ogs = p.btiles[u].grp_start, ow = p.tile_gwork[u];
    before += (ow > gw) || (ow == gw && ogs < gs);
    ng += (ogs == gs);
  }
  const int k_rel = (p.btiles[t].start - gs) / kTile;
  const int slot = ng <= p.det_asc_max ? k_rel : ng - 1 - k_rel;
  for (int kvh = 0; kvh < p.Hkv; ++kvh)
    p.bwd_units_det[p.Hkv * before + kvh * ng + slot] = (kvh << 24) | t;
}

__global__ void plan_gwork_kernel(PlanPtrs p) {
  if (p.header[0] != kStatusOk) return;
  const int n = p.header[kHdrNumBTiles];
  int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t < n) plan_gwork_body(p, t, n);
}

__global__ void plan_sgroup_kernel(PlanPtrs p) {
  if (p.header[0] != kStatusOk) return;
  const int n = p.header[kHdrNumBTiles];
  int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t < n) plan_sgroup_body(p, t, n);
}

__global__ void plan_units_kernel(PlanPtrs p) {
  if (p.header[0] != kStatusOk) return;
  const int n = p.header[kHdrNumBTiles];
  int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t < n) plan_units_body(p, t, n);
}

// The whole plan in one block: used when the problem is small enough that one block's
// latency beats eight dependent launches (every stage only needs block-level ordering).  The
// per-tile keys of the rank-counting stages are kept in shared memory, so that the O(n^2)
// loops do not go through global memory, and key_end is filled tile by tile (every key of a
// forward tile ends its visibility at the tile's vis_end) instead of by a search per token.
constexpr int kFusedMaxTiles = 2048;

__global__ void __launch_bounds__(1024) plan_fused_kernel(PlanPtrs p) {
  __shared__ uint16_t s_wf[kFusedMaxTiles];   // forward work of the forward tiles
  __shared__ uint16_t s_wb[kFusedMaxTiles];   // work of the backward tiles
  __shared__ int32_t s_gs[kFusedMaxTiles];    // group id of the backward tiles
  __shared__ int32_t s_gw[kFusedMaxTiles];    // backward work of the tile's whole group
  __shared__ uint16_t s_sg[kFusedMaxTiles];   // super-group
  if (!plan_scan_body(p)) return;
  const int n = p.header[kHdrNumTiles], nb = p.header[kHdrNumBTiles];
  const int tid = threadIdx.x, nthr = blockDim.x;
  for (int t = tid; t < n; t += nthr) {
    plan_tile_body(p, t);
    s_wf[t] = uint16_t(p.tiles[t].work);  // own write
  }
  for (int t = tid; t < nb; t += nthr) {
    plan_btile_body(p, t);
    const BTile b = p.btiles[t];  // own write
    s_wb[t] = uint16_t(b.work);
    s_gs[t] = b.grp_start;
  }
  __syncthreads();
  // key_end: one warp per forward tile, coalesced
  for (int t = tid >> 5; t < n; t += nthr >> 5) {
    const Tile tl = p.tiles[t];
    for (int i = tid & 31; i < tl.len; i += 32) p.key_end[tl.start + i] = tl.vis_end;
  }
  // Longest-work-first orders by rank counting, and the work of each backward tile's group.
  // One warp per tile: the lanes stride over the other tiles and the partial counts are
  // summed with shuffles (a thread per tile would walk the whole list alone, a few
  // microseconds of dependent shared-memory reads per pass on a 100-tile plan).
  const int lane = tid & 31, wid = tid >> 5, nwarp = nthr >> 5;
  auto warp_sum = [](int x) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) x += __shfl_xor_sync(0xffffffffu, x, d);
    return x;
  };
  for (int t = wid; t < n; t += nwarp) {
    const int wf = s_wf[t];
    int rf = 0;
    for (int u = lane; u < n; u += 32) {
      const int of = s_wf[u];
      rf += (of > wf) || (of == wf && u < t);
    }
    rf = warp_sum(rf);
    if (lane == 0) p.fwd_order[rf] = t;
  }
  for (int t = wid; t < nb; t += nwarp) {
    const int wb = s_wb[t], gs = s_gs[t];
    int rb = 0, gw = 0;
    for (int u = lane; u < nb; u += 32) {
      const int ob = s_wb[u];
      rb += (ob > wb) || (ob == wb && u < t);
      gw += (s_gs[u] == gs) ? ob : 0;
    }
    rb = warp_sum(rb);
    gw = warp_sum(gw);
    if (lane == 0) {
      p.bwd_order[rb] = t;
      p.tile_gwork[t] = gw;
      s_gw[t] = gw;
    }
  }
  __syncthreads();
  for (int t = wid; t < nb; t += nwarp) {
    const int gs = s_gs[t], gw = s_gw[t];
    int rest = 0;  // tiles of this group and of the groups that come later
    for (int u = lane; u < nb; u += 32) {
      const int ogs = s_gs[u], ow = s_gw[u];
      rest += (ogs == gs) || (ow < gw) || (ow == gw && ogs > gs);
    }
    rest = warp_sum(rest);
    if (lane == 0) {
      const int sg = (p.Hkv * rest - 1) / kSuperGroupUnits;
      p.tile_sgroup[t] = sg;
      s_sg[t] = uint16_t(sg);
    }
  }
  __syncthreads();
  for (int t = wid; t < nb; t += nwarp) {
    const int sg = s_sg[t], wb = s_wb[t], gs = s_gs[t], gw = s_gw[t];
    int pos = 0, before = 0, ng = 0, k_rel = 0;
    for (int u = lane; u < nb; u += 32) {
      const int osg = s_sg[u], ob = s_wb[u], ogs = s_gs[u], ow = s_gw[u];
      pos += (osg > sg) || (osg == sg && ((ob > wb) || (ob == wb && u < t)));
      before += (ow > gw) || (ow == gw && ogs < gs);
      ng += (ogs == gs);
      k_rel += (ogs == gs && u < t);   // tiles of a group are consecutive
    }
    pos = warp_sum(pos);
    before = warp_sum(before);
    ng = warp_sum(ng);
    k_rel = warp_sum(k_rel);
    // deterministic backward: set after set (see plan_units_body)
    const int slot = ng <= p.det_asc_max ? k_rel : ng - 1 - k_rel;
    for (int kvh = lane; kvh < p.Hkv; kvh += 32) {
      p.bwd_units[p.Hkv * pos + kvh] = (kvh << 24) | t;
      p.bwd_units_det[p.Hkv * before + kvh * ng + slot] = (kvh << 24) | t;
    }
  }
}

}  // namespace

ProfileEvents& profile_events() {
  static ProfileEvents ev;
  return ev;
}

bool profile_enable(int mode) {
  ProfileEvents& ev = profile_events();
  const bool on = mode != 0;
  if (on && ev.on) {  // already on: the choice of kernels can change, and the counts restart
    ev.fwd_on = mode == 1;
    ev.fwd_count = ev.bwd_count = 0;
    return true;
  }
  if (on == ev.on) return true;
  if (on) {
    bool ok = true;
    for (int i = 0; i < kProfileRing && ok; ++i)
      ok = cudaEventCreate(&ev.fwd0[i]) == cudaSuccess && cudaEventCreate(&ev.fwd1[i]) == cudaSuccess &&
           cudaEventCreate(&ev.bwd0[i]) == cudaSuccess && cudaEventCreate(&ev.bwd1[i]) == cudaSuccess;
    ev.on = ok;
    ev.fwd_on = mode == 1;
    ev.fwd_count = ev.bwd_count = 0;
    return ok;
  }
  for (int i = 0; i < kProfileRing; ++i) {
    cudaEventDestroy(ev.fwd0[i]); cudaEventDestroy(ev.fwd1[i]);
    cudaEventDestroy(ev.bwd0[i]); cudaEventDestroy(ev.bwd1[i]);
  }
  ev = ProfileEvents();
  return true;
}

// Durations of the most recent launches, oldest first (at most kProfileRing are kept).
bool profile_read_all(float* fwd_ms, float* bwd_ms, int capacity, int* n_fwd, int* n_bwd) {
  ProfileEvents& ev = profile_events();
  if (!ev.on || capacity < 0) return false;
  bool ok = true;
  auto dump = [&](float* out, int* n_out, long long count, cudaEvent_t* e0, cudaEvent_t* e1) {
    const int n = int(std::min<long long>(std::min<long long>(count, kProfileRing), capacity));
    if (n_out) *n_out = n;
    if (!out) return;
    for (int i = 0; i < n; ++i) {
      const long long idx = count - n + i;
      ok = ok && cudaEventElapsedTime(&out[i], e0[idx % kProfileRing], e1[idx % kProfileRing]) == cudaSuccess;
    }
  };
  dump(fwd_ms, n_fwd, ev.fwd_count, ev.fwd0, ev.fwd1);
  dump(bwd_ms, n_bwd, ev.bwd_count, ev.bwd0, ev.bwd1);
  return ok;
}

bool profile_read(float* fwd_ms, float* bwd_ms) {
  ProfileEvents& ev = profile_events();
  if (!ev.on) return false;
  bool ok = true;
  if (fwd_ms) {
    const long long i = (ev.fwd_count - 1) % kProfileRing;
    ok = ok && ev.fwd_count > 0 && cudaEventElapsedTime(fwd_ms, ev.fwd0[i], ev.fwd1[i]) == cudaSuccess;
  }
  if (bwd_ms) {
    const long long i = (ev.bwd_count - 1) % kProfileRing;
    ok = ok && ev.bwd_count > 0 && cudaEventElapsedTime(bwd_ms, ev.bwd0[i], ev.bwd1[i]) == cudaSuccess;
  }
  return ok;
}

cudaError_t launch_plan(const pp_plan* plan, cudaStream_t stream, int* launches) {
  PlanPtrs p;
  char* ws = plan->ws;
  const PlanLayout& l = plan->lay;
  p.header = reinterpret_cast<int32_t*>(ws + l.header);
  for (int a = 0; a < 4; ++a) p.src_desc[a] = plan->src_desc[a];
  p.desc_copy = reinterpret_cast<int32_t*>(ws + l.desc);
  p.row_group_off = plan->prob.row_group_off;
  p.grp_prompt_len = plan->prob.grp_prompt_len;
  p.grp_resp_off = plan->prob.grp_resp_off;
  p.resp_len = plan->prob.resp_len;
  p.seg_start = reinterpret_cast<int32_t*>(ws + l.seg_start);
  p.seg_tile0 = reinterpret_cast<int32_t*>(ws + l.seg_tile0);
  p.tiles = reinterpret_cast<Tile*>(ws + l.tiles);
  p.grp_btile0 = reinterpret_cast<int32_t*>(ws + l.grp_btile0);
  p.btiles = reinterpret_cast<BTile*>(ws + l.btiles);
  p.fwd_order = reinterpret_cast<int32_t*>(ws + l.fwd_order);
  p.bwd_order = reinterpret_cast<int32_t*>(ws + l.bwd_order);
  p.tile_gwork = reinterpret_cast<int32_t*>(ws + l.tile_gwork);
  p.tile_sgroup = reinterpret_cast<int32_t*>(ws + l.tile_sgroup);
  p.bwd_units = reinterpret_cast<int32_t*>(ws + l.bwd_units);
  p.bwd_units_det = reinterpret_cast<int32_t*>(ws + l.bwd_units_det);
  p.Hkv = plan->prob.num_kv_heads;
  p.key_end = reinterpret_cast<int32_t*>(ws + l.key_end);
  {
    // a third of the SMs (the backward runs one CTA per SM), at most 48 tiles = 6144 tokens
    static DeviceSetup setup[kMaxDevices];
    DeviceSetup* dev = device_setup(setup);
    p.det_asc_max = dev ? std::min(48, dev->num_sms / 3) : 0;
  }
  p.num_rows = plan->prob.num_rows;
  p.G = plan->prob.num_groups;
  p.N = plan->prob.num_responses;
  p.T = plan->prob.total_tokens;
  p.nseg = plan->nseg;
  p.max_tiles = plan->max_tiles;

  int mt = plan->max_tiles;
  if (mt <= kFusedMaxTiles && p.T <= (1 << 18)) {
    plan_fused_kernel<<<1, 1024, 0, stream>>>(p);
    if (launches) *launches = 1;
    return cudaGetLastError();
  }
  plan_scan_kernel<<<1, 1024, 0, stream>>>(p);
  plan_tiles_kernel<<<(mt + 255) / 256, 256, 0, stream>>>(p);
  plan_key_end_kernel<<<(p.T + 255) / 256, 256, 0, stream>>>(p);
  plan_btiles_kernel<<<(mt + 255) / 256, 256, 0, stream>>>(p);
  plan_fwd_order_kernel<<<(mt + 127) / 128, 128, 0, stream>>>(p);
  plan_gwork_kernel<<<(mt + 127) / 128, 128, 0, stream>>>(p);
  plan_sgroup_kernel<<<(mt + 127) / 128, 128, 0, stream>>>(p);
  plan_units_kernel<<<(mt + 127) / 128, 128, 0, stream>>>(p);
  if (launches) *launches = 8;
  return cudaGetLastError();
}

}  // namespace pp
