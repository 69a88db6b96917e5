// Row builder: the step before the attention path (paper Sec. 2.2, used with preference
// packing in Sec. 5.2).  Preference groups [prompt | responses] of varying length are ordered by
// total length, longest first with ties in their original order (batch sorting: samples of
// similar length end up together), and consecutive groups of that order are concatenated into
// rows of at most `capacity` tokens (batch packing: next fit).  The outputs are
// the order, the rows, each row's tokens and visible query-key pairs (the attention cost of
// Sec. 3.2.1, for balancing data-parallel ranks) and the descriptor arrays in row order, ready
// for pp_build_plan with descriptors on the device.  Integer work only; microseconds.
#include "pp_internal.h"

namespace pp {
namespace {

enum : int32_t { kRowsOk = 0, kRowsBadGroup = 1, kRowsTooLong = 2 };

struct RowsPtrs {
  int G, N, capacity;
  const int32_t* prompt_len;
  const int32_t* resp_off;
  const int32_t* resp_len;
  long long* tok;    // [G] tokens per group
  long long* cost;   // [G] visible pairs per group
  long long* pre;    // [G] inclusive prefix sums of the sorted groups' tokens
  int32_t* nxt;      // [G] end of the row that would start at each sorted position
  int32_t* jump_a;   // [G] pointer-doubling buffers
  int32_t* jump_b;   // [G]
  int32_t* mark;     // [G] 1 = a row starts here
  int32_t* order;
  int32_t* row_group_off;
  int32_t* num_rows;
  long long* row_tokens;
  long long* row_cost;
  int32_t* out_prompt_len;
  int32_t* out_resp_off;
  int32_t* out_resp_len;
  int32_t* status;   // [2]: code, detail
};

__device__ __forceinline__ void rows_fail(int32_t* status, int32_t code, int32_t detail) {
  if (atomicCAS(&status[0], kRowsOk, code) == kRowsOk) status[1] = detail;
}

// tokens and visible pairs of every group: P (P + 1) / 2 for the causal prompt, and
// R P + R (R + 1) / 2 for a response that sees the whole prompt and itself causally
__global__ void rows_measure_kernel(RowsPtrs p) {
  const int g = blockIdx.x * blockDim.x + threadIdx.x;
  if (g >= p.G) return;
  const long long P = p.prompt_len[g];
  const int x0 = p.resp_off[g], x1 = p.resp_off[g + 1];
  if (P < 1 || x1 <= x0 || x0 < 0 || x1 > p.N) {
    rows_fail(p.status, kRowsBadGroup, g);
    p.tok[g] = 0;
    p.cost[g] = 0;
    return;
  }
  long long t = P, u = P * (P + 1) / 2;
  for (int x = x0; x < x1; ++x) {
    const long long R = p.resp_len[x];
    if (R < 1) rows_fail(p.status, kRowsBadGroup, g);
    t += R;
    u += R * P + R * (R + 1) / 2;
  }
  if (t > p.capacity) rows_fail(p.status, kRowsTooLong, g);
  p.tok[g] = t;
  p.cost[g] = u;
}

// position of every group in the order "longest first, ties by original index": rank counting
// against all groups, staged through shared memory
__global__ void __launch_bounds__(256) rows_rank_kernel(RowsPtrs p) {
  __shared__ long long s_tok[256];
  const int g = blockIdx.x * blockDim.x + threadIdx.x;
  const long long mine = g < p.G ? p.tok[g] : 0;
  int rank = 0;
  for (int base = 0; base < p.G; base += 256) {
    const int u = base + threadIdx.x;
    s_tok[threadIdx.x] = u < p.G ? p.tok[u] : -1;
    __syncthreads();
    const int lim = min(256, p.G - base);
    for (int i = 0; i < lim; ++i) {
      const long long o = s_tok[i];
      rank += (o > mine) || (o == mine && base + i < g);
    }
    __syncthreads();
  }
  if (g < p.G) p.order[rank] = g;
}

// one block: prefix sums over the sorted groups, next-fit rows, row costs, reordered
// descriptors
__global__ void __launch_bounds__(1024) rows_pack_kernel(RowsPtrs p) {
  __shared__ long long s_a[1024];
  __shared__ int32_t s_b[1024];
  __shared__ long long s_carry;
  __shared__ int32_t s_carry_b;
  __shared__ int32_t s_rows;
  const int tid = threadIdx.x, nthr = blockDim.x;
  if (p.status[0] != kRowsOk) {
    if (tid == 0) *p.num_rows = 0;
    return;
  }
  if (tid == 0) {
    s_carry = 0;
    s_carry_b = 0;
  }
  __syncthreads();
  // inclusive scan of tokens and exclusive scan of response counts, both in sorted order
  for (int base = 0; base < p.G; base += nthr) {
    const int i = base + tid;
    long long a = 0;
    int32_t b = 0;
    if (i < p.G) {
      const int g = p.order[i];
      a = p.tok[g];
      b = p.resp_off[g + 1] - p.resp_off[g];
      p.out_prompt_len[i] = p.prompt_len[g];
    }
    s_a[tid] = a;
    s_b[tid] = b;
    __syncthreads();
    for (int d = 1; d < nthr; d <<= 1) {
      const long long xa = tid >= d ? s_a[tid - d] : 0;
      const int32_t xb = tid >= d ? s_b[tid - d] : 0;
      __syncthreads();
      s_a[tid] += xa;
      s_b[tid] += xb;
      __syncthreads();
    }
    if (i < p.G) {
      p.pre[i] = s_carry + s_a[tid];
      p.out_resp_off[i] = s_carry_b + s_b[tid] - b;
    }
    __syncthreads();
    if (tid == nthr - 1) {
      s_carry += s_a[tid];
      s_carry_b += s_b[tid];
    }
    __syncthreads();
  }
  if (tid == 0) p.out_resp_off[p.G] = s_carry_b;
  __syncthreads();
  // Next fit in parallel.  nxt[s] = where the row that starts at sorted position s ends: the
  // largest e whose tokens still fit (every group fits alone, so e > s).  The row starts are
  // the positions reachable from 0 through nxt; they are marked by pointer doubling (after
  // round r every start within 2^r hops is marked), then numbered by a prefix count.
  for (int s = tid; s < p.G; s += nthr) {
    const long long base = s ? p.pre[s - 1] : 0;
    int lo = s + 1, hi = p.G;
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (p.pre[mid - 1] - base <= p.capacity) lo = mid; else hi = mid - 1;
    }
    p.nxt[s] = lo;
    p.jump_a[s] = lo;
    p.mark[s] = (s == 0);
  }
  int32_t* ja = p.jump_a;
  int32_t* jb = p.jump_b;
  for (int hop = 1; hop < p.G; hop <<= 1) {
    __syncthreads();
    for (int s = tid; s < p.G; s += nthr)
      if (p.mark[s] && ja[s] < p.G) p.mark[ja[s]] = 1;
    for (int s = tid; s < p.G; s += nthr) jb[s] = ja[s] < p.G ? ja[ja[s]] : p.G;
    __syncthreads();
    int32_t* t = ja;
    ja = jb;
    jb = t;
  }
  __syncthreads();
  // number the marked positions (exclusive scan of the marks) and emit the rows
  if (tid == 0) s_carry_b = 0;
  __syncthreads();
  for (int base = 0; base < p.G; base += nthr) {
    const int i = base + tid;
    const int32_t m = i < p.G ? p.mark[i] : 0;
    s_b[tid] = m;
    __syncthreads();
    for (int d = 1; d < nthr; d <<= 1) {
      const int32_t xb = tid >= d ? s_b[tid - d] : 0;
      __syncthreads();
      s_b[tid] += xb;
      __syncthreads();
    }
    if (m) {
      const int r = s_carry_b + s_b[tid] - 1;
      p.row_group_off[r] = i;
      p.row_tokens[r] = p.pre[p.nxt[i] - 1] - (i ? p.pre[i - 1] : 0);
    }
    __syncthreads();
    if (tid == nthr - 1) s_carry_b += s_b[tid];
    __syncthreads();
  }
  if (tid == 0) {
    p.row_group_off[s_carry_b] = p.G;
    *p.num_rows = s_carry_b;
    s_rows = s_carry_b;
  }
  __syncthreads();
  for (int r = tid; r < s_rows; r += nthr) {
    long long c = 0;
    for (int i = p.row_group_off[r]; i < p.row_group_off[r + 1]; ++i) c += p.cost[p.order[i]];
    p.row_cost[r] = c;
  }
  for (int i = tid; i < p.G; i += nthr) {
    const int g = p.order[i];
    const int x0 = p.resp_off[g], n = p.resp_off[g + 1] - x0, y0 = p.out_resp_off[i];
    for (int x = 0; x < n; ++x) p.out_resp_len[y0 + x] = p.resp_len[x0 + x];
  }
}

// ---------------------------------------------------------------- rows -> data-parallel ranks
// Longest-processing-time assignment: rows in order of decreasing cost (ties by index), each to
// the rank with the least cost so far (ties to the lowest rank).  The order comes from rank
// counting over all rows; the greedy pass is sequential by nature and runs in one warp, the
// lanes sharing the search for the least-loaded rank.
__global__ void __launch_bounds__(256)
assign_rank_kernel(int R, const long long* __restrict__ cost, int32_t* __restrict__ order) {
  __shared__ long long s_c[256];
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  const long long mine = r < R ? cost[r] : 0;
  int rank = 0;
  for (int base = 0; base < R; base += 256) {
    const int u = base + threadIdx.x;
    s_c[threadIdx.x] = u < R ? cost[u] : -1;
    __syncthreads();
    const int lim = min(256, R - base);
    for (int i = 0; i < lim; ++i) {
      const long long o = s_c[i];
      rank += (o > mine) || (o == mine && base + i < r);
    }
    __syncthreads();
  }
  if (r < R) order[rank] = r;
}

constexpr int kMaxAssignRanks = 1024;

__global__ void __launch_bounds__(32)
assign_greedy_kernel(int R, int ranks, const long long* __restrict__ cost,
                     const int32_t* __restrict__ order, int32_t* __restrict__ rank_of_row,
                     long long* __restrict__ rank_cost) {
  __shared__ long long s_load[kMaxAssignRanks];
  const int lane = threadIdx.x;
  for (int k = lane; k < ranks; k += 32) s_load[k] = 0;
  __syncwarp();
  for (int i = 0; i < R; ++i) {
    long long best = 0x7fffffffffffffffLL;
    int best_k = ranks;
    for (int k = lane; k < ranks; k += 32) {   // ascending k: the first minimum is kept
      const long long l = s_load[k];
      if (l < best) {
        best = l;
        best_k = k;
      }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
      const long long ob = __shfl_xor_sync(0xffffffffu, best, d);
      const int ok = __shfl_xor_sync(0xffffffffu, best_k, d);
      if (ob < best || (ob == best && ok < best_k)) {
        best = ob;
        best_k = ok;
      }
    }
    if (lane == 0) {
      const int row = order[i];
      rank_of_row[row] = best_k;
      s_load[best_k] = best + cost[row];
    }
    __syncwarp();
  }
  for (int k = lane; k < ranks; k += 32) rank_cost[k] = s_load[k];
}

}  // namespace

cudaError_t launch_assign_rows(int R, const long long* row_cost, int ranks, int32_t* order,
                               int32_t* rank_of_row, long long* rank_cost, cudaStream_t stream,
                               int* launches) {
  assign_rank_kernel<<<(R + 255) / 256, 256, 0, stream>>>(R, row_cost, order);
  assign_greedy_kernel<<<1, 32, 0, stream>>>(R, ranks, row_cost, order, rank_of_row, rank_cost);
  if (launches) *launches = 2;
  return cudaGetLastError();
}

size_t rows_workspace_bytes(int G) {
  return align_up(size_t(8) * G, 256) * 3 + align_up(size_t(4) * G, 256) * 4;
}

cudaError_t launch_build_rows(int G, int N, const int32_t* prompt_len, const int32_t* resp_off,
                              const int32_t* resp_len, int capacity, void* ws, int32_t* order,
                              int32_t* row_group_off, int32_t* num_rows, long long* row_tokens,
                              long long* row_cost, int32_t* out_prompt_len, int32_t* out_resp_off,
                              int32_t* out_resp_len, int32_t* status, cudaStream_t stream,
                              int* launches) {
  RowsPtrs p;
  p.G = G;
  p.N = N;
  p.capacity = capacity;
  p.prompt_len = prompt_len;
  p.resp_off = resp_off;
  p.resp_len = resp_len;
  char* w = static_cast<char*>(ws);
  const size_t a8 = align_up(size_t(8) * G, 256);
  p.tok = reinterpret_cast<long long*>(w);
  p.cost = reinterpret_cast<long long*>(w + a8);
  p.pre = reinterpret_cast<long long*>(w + 2 * a8);
  const size_t a4 = align_up(size_t(4) * G, 256);
  p.nxt = reinterpret_cast<int32_t*>(w + 3 * a8);
  p.jump_a = reinterpret_cast<int32_t*>(w + 3 * a8 + a4);
  p.jump_b = reinterpret_cast<int32_t*>(w + 3 * a8 + 2 * a4);
  p.mark = reinterpret_cast<int32_t*>(w + 3 * a8 + 3 * a4);
  p.order = order;
  p.row_group_off = row_group_off;
  p.num_rows = num_rows;
  p.row_tokens = row_tokens;
  p.row_cost = row_cost;
  p.out_prompt_len = out_prompt_len;
  p.out_resp_off = out_resp_off;
  p.out_resp_len = out_resp_len;
  p.status = status;
  cudaError_t e = cudaMemsetAsync(status, 0, 8, stream);
  if (e != cudaSuccess) return e;
  rows_measure_kernel<<<(G + 255) / 256, 256, 0, stream>>>(p);
  rows_rank_kernel<<<(G + 255) / 256, 256, 0, stream>>>(p);
  rows_pack_kernel<<<1, 1024, 0, stream>>>(p);
  if (launches) *launches = 3;
  return cudaGetLastError();
}

}  // namespace pp
