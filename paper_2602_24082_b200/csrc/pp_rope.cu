// Packed position ids and rotary embedding on Q / K (the step right before attention).
//
// Paper Sec. 3.2: in the packed sequence every response keeps the positions it would have
// in its own (x, y^k) sequence, i.e. positions restart right after the prompt for every
// response.  Position of token t: (t - group start) inside the prompt, P + (t - response
// start) inside a response.  The rotary embedding itself is the usual rotate-half form used
// by the models the paper trains (Llama / Qwen): for i < D/2 and angle a = pos * base^(-2i/D)
//   x'[i]       = x[i] cos a - x[i + D/2] sin a
//   x'[i + D/2] = x[i + D/2] cos a + x[i] sin a
// Both kernels are HBM-bound: one pass over Q and K (read + write, bf16), 4 bytes per token
// for the ids.
#include "pp_internal.h"
#include "pp_ptx.cuh"

namespace pp {
namespace {

struct SegPtrs {
  const int32_t* header;
  const int32_t* seg_start;     // [nseg + 1]
  const int32_t* grp_resp_off;  // [G + 1]
  const int32_t* grp_prompt_len;
  int nseg, G, T;
};

__device__ __forceinline__ int position_of(const SegPtrs& p, int t) {
  // segment of t: largest s with seg_start[s] <= t
  int lo = 0, hi = p.nseg;
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (p.seg_start[mid] <= t) lo = mid; else hi = mid;
  }
  const int s = lo;
  // group of s: largest g with g + resp_off[g] <= s  (segment order: prompt, its responses, ...)
  lo = 0, hi = p.G;
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (mid + p.grp_resp_off[mid] <= s) lo = mid; else hi = mid;
  }
  const int g = lo;
  const bool prompt = (s == g + p.grp_resp_off[g]);
  const int in_seg = t - p.seg_start[s];
  return prompt ? in_seg : p.grp_prompt_len[g] + in_seg;
}

__global__ void position_ids_kernel(SegPtrs p, int32_t* __restrict__ pos) {
  if (p.header[0] != kStatusOk) return;
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t < p.T) pos[t] = position_of(p, t);
}

// One warp per token: for D = 128 lane i owns the frequency pair (2i, 2i+1), so every access
// is a 4-byte bf16x2 and a warp touches 128 contiguous bytes; the sines / cosines are computed
// once per token and reused for every Q and K head.
template <int D>
__global__ void __launch_bounds__(256)
rope_kernel(SegPtrs p, __nv_bfloat16* __restrict__ q, __nv_bfloat16* __restrict__ k, int Hq,
            int Hkv, float log2_base) {
  if (p.header[0] != kStatusOk) return;
  const int lane = threadIdx.x & 31;
  const int t = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (t >= p.T) return;
  const float pos = float(position_of(p, t));
  constexpr int kHalf = D / 2;
  if (D != 64) {   // two frequencies per lane: lanes 0 .. D / 4 - 1 cover the D / 2 pairs
    float c0, s0, c1, s1;
    sincosf(pos * exp2f(-log2_base * (2.f * float(2 * lane) / float(D))), &s0, &c0);
    sincosf(pos * exp2f(-log2_base * (2.f * float(2 * lane + 1) / float(D))), &s1, &c1);
    auto rotate = [&](__nv_bfloat16* x) {
      if (lane >= D / 4) return;
      __nv_bfloat162* lo = reinterpret_cast<__nv_bfloat162*>(x) + lane;
      __nv_bfloat162* hi = reinterpret_cast<__nv_bfloat162*>(x + kHalf) + lane;
      const float2 a = __bfloat1622float2(*lo), b = __bfloat1622float2(*hi);
      *lo = __floats2bfloat162_rn(a.x * c0 - b.x * s0, a.y * c1 - b.y * s1);
      *hi = __floats2bfloat162_rn(b.x * c0 + a.x * s0, b.y * c1 + a.y * s1);
    };
    for (int h = 0; h < Hq; ++h) rotate(q + (size_t(t) * Hq + h) * D);
    for (int h = 0; h < Hkv; ++h) rotate(k + (size_t(t) * Hkv + h) * D);
  } else {
    float c0, s0;
    sincosf(pos * exp2f(-log2_base * (2.f * float(lane) / float(D))), &s0, &c0);
    auto rotate = [&](__nv_bfloat16* x) {
      const float a = __bfloat162float(x[lane]), b = __bfloat162float(x[lane + kHalf]);
      x[lane] = __float2bfloat16_rn(a * c0 - b * s0);
      x[lane + kHalf] = __float2bfloat16_rn(b * c0 + a * s0);
    };
    for (int h = 0; h < Hq; ++h) rotate(q + (size_t(t) * Hq + h) * D);
    for (int h = 0; h < Hkv; ++h) rotate(k + (size_t(t) * Hkv + h) * D);
  }
}

SegPtrs seg_ptrs(const pp_plan* plan) {
  SegPtrs p;
  p.header = reinterpret_cast<const int32_t*>(plan->ws + plan->lay.header);
  p.seg_start = reinterpret_cast<const int32_t*>(plan->ws + plan->lay.seg_start);
  p.grp_resp_off = plan->prob.grp_resp_off;
  p.grp_prompt_len = plan->prob.grp_prompt_len;
  p.nseg = plan->nseg;
  p.G = plan->prob.num_groups;
  p.T = plan->prob.total_tokens;
  return p;
}

}  // namespace

cudaError_t launch_position_ids(const pp_plan* plan, int32_t* pos, cudaStream_t stream) {
  SegPtrs p = seg_ptrs(plan);
  position_ids_kernel<<<(p.T + 255) / 256, 256, 0, stream>>>(p, pos);
  return cudaGetLastError();
}

cudaError_t launch_rope(const pp_plan* plan, void* q, void* k, float base, cudaStream_t stream) {
  SegPtrs p = seg_ptrs(plan);
  const pp_problem& pb = plan->prob;
  const float log2_base = log2f(base);
  const unsigned blocks = unsigned((p.T + 7) / 8);
  if (pb.head_dim == 128)
    rope_kernel<128><<<blocks, 256, 0, stream>>>(p, static_cast<__nv_bfloat16*>(q),
                                                 static_cast<__nv_bfloat16*>(k), pb.num_q_heads,
                                                 pb.num_kv_heads, log2_base);
  else if (pb.head_dim == 96)
    rope_kernel<96><<<blocks, 256, 0, stream>>>(p, static_cast<__nv_bfloat16*>(q),
                                                static_cast<__nv_bfloat16*>(k), pb.num_q_heads,
                                                pb.num_kv_heads, log2_base);
  else
    rope_kernel<64><<<blocks, 256, 0, stream>>>(p, static_cast<__nv_bfloat16*>(q),
                                                static_cast<__nv_bfloat16*>(k), pb.num_q_heads,
                                                pb.num_kv_heads, log2_base);
  return cudaGetLastError();
}

}  // namespace pp
