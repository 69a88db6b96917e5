// Loss-side consumer on the packed layout (paper Sec. 2.1): per-response sequence
// log-probabilities and the pairwise preference loss over the ranked responses of a group.
//
// The packed row is split back into its responses here: s_k = sum of the token log-probs of
// response k (prompt tokens do not count).  Reward r_k = beta * (s_k - s_k_ref) (DPO; the
// paper prints the ratio without the logarithm -- the log-ratio of Rafailov et al. is used),
// or beta * s_k when no reference is given.  Responses are ranked as in the paper's Sec. 3.1:
// response a is preferred over response b for a > b.  Group loss = mean over the pairs a > b
// of -log sigmoid(r_a - r_b) (the paper's Bradley-Terry expression with the usual minus sign);
// the optional gradient is d(sum of group losses) / d token_logp.
// One warp per group; HBM-bound: 4 bytes per token read per log-prob array, 4 written for
// the gradient.
#include "pp_internal.h"

namespace pp {
namespace {

struct LossPtrs {
  const int32_t* header;
  const int32_t* seg_start;
  const int32_t* grp_resp_off;
  int G;
};

__device__ __forceinline__ float log_sigmoid(float x) {
  return fminf(x, 0.f) - log1pf(expf(-fabsf(x)));
}
__device__ __forceinline__ float sigmoid(float x) { return 1.f / (1.f + expf(-x)); }

__global__ void __launch_bounds__(256)
preference_loss_kernel(LossPtrs p, const float* __restrict__ logp, const float* __restrict__ ref,
                       float beta, float* __restrict__ resp_logp, float* __restrict__ resp_reward,
                       float* __restrict__ grp_loss, float* __restrict__ d_logp) {
  if (p.header[0] != kStatusOk) return;
  const int lane = threadIdx.x & 31;
  const int g = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (g >= p.G) return;
  const int x0 = p.grp_resp_off[g], x1 = p.grp_resp_off[g + 1], n = x1 - x0;
  const int sp = g + x0;  // the group's prompt segment; response x is segment g + 1 + x
  // 1. sequence log-probs and rewards
  for (int x = x0; x < x1; ++x) {
    const int a = p.seg_start[g + 1 + x], b = p.seg_start[g + 2 + x];
    float s = 0.f, sr = 0.f;
    for (int t = a + lane; t < b; t += 32) {
      s += logp[t];
      if (ref) sr += ref[t];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      s += __shfl_xor_sync(0xffffffffu, s, o);
      sr += __shfl_xor_sync(0xffffffffu, sr, o);
    }
    if (lane == 0) {
      resp_logp[x] = s;
      resp_reward[x] = beta * (s - sr);
    }
  }
  __syncwarp();
  // 2. pairwise loss over ranked pairs (a preferred over b for a > b) and d loss / d reward
  const int npairs = n * (n - 1) / 2;
  float loss = 0.f;
  for (int a = 1 + lane; a < n; a += 32)
    for (int b = 0; b < a; ++b) loss -= log_sigmoid(resp_reward[x0 + a] - resp_reward[x0 + b]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) loss += __shfl_xor_sync(0xffffffffu, loss, o);
  const float inv = npairs > 0 ? 1.f / float(npairs) : 0.f;
  if (lane == 0) grp_loss[g] = loss * inv;
  if (!d_logp) return;
  // 3. gradient: prompt tokens get 0; tokens of response k get beta * dL/dr_k
  for (int t = p.seg_start[sp] + lane; t < p.seg_start[sp + 1]; t += 32) d_logp[t] = 0.f;
  for (int k = 0; k < n; ++k) {
    const float rk = resp_reward[x0 + k];
    float gk = 0.f;
    for (int j = lane; j < n; j += 32) {
      if (j == k) continue;
      const float rj = resp_reward[x0 + j];
      // k preferred over j (k > j): d/dr_k of -log sig(r_k - r_j) = -sig(r_j - r_k)
      // j preferred over k (j > k): d/dr_k of -log sig(r_j - r_k) = +sig(r_k - r_j)
      gk += (k > j) ? -sigmoid(rj - rk) : sigmoid(rk - rj);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) gk += __shfl_xor_sync(0xffffffffu, gk, o);
    const float gt = beta * gk * inv;
    const int a = p.seg_start[g + 1 + x0 + k], b = p.seg_start[g + 2 + x0 + k];
    for (int t = a + lane; t < b; t += 32) d_logp[t] = gt;
  }
}

}  // namespace

cudaError_t launch_preference_loss(const pp_plan* plan, const float* logp, const float* ref,
                                   float beta, float* resp_logp, float* resp_reward,
                                   float* grp_loss, float* d_logp, cudaStream_t stream) {
  LossPtrs p;
  p.header = reinterpret_cast<const int32_t*>(plan->ws + plan->lay.header);
  p.seg_start = reinterpret_cast<const int32_t*>(plan->ws + plan->lay.seg_start);
  p.grp_resp_off = plan->prob.grp_resp_off;
  p.G = plan->prob.num_groups;
  preference_loss_kernel<<<(p.G + 7) / 8, 256, 0, stream>>>(p, logp, ref, beta, resp_logp,
                                                            resp_reward, grp_loss, d_logp);
  return cudaGetLastError();
}

}  // namespace pp
