// C ABI of the preference-packed attention library: argument checking, plan handle,
// workspace bookkeeping.  Apart from the kernel that stages host descriptors, all device work
// is enqueued by the launchers in the other files.
#include <new>
#include <string.h>

#include <algorithm>
#include <mutex>
#include <vector>

#include "pp_dev.cuh"

namespace {

// Test hook: one thread waits on an mbarrier that nobody ever arrives at, with a poll limit of
// a few thousand instead of the kernels' two million.  No copy and no MMA is in flight, so the
// give-up path of the bounded wait -- status word, site id, abort flag, return -- can be
// exercised on a GPU without hanging or faulting anything.
__global__ void expire_wait_kernel(int32_t* header, int site) {
  __shared__ __align__(8) unsigned long long bar_storage;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    const uint32_t bar = pp::smem_u32(&bar_storage);
    pp::mbar_init(bar, 1);
    abort_flag = 0;
    pp::fence_mbar_init();
    const bool done = pp::wait_bar(bar, 0, &abort_flag, header, site, 4096);
    // a second wait after the give-up returns at once
    const bool again = pp::wait_bar(bar, 0, &abort_flag, header, site + 1, 4096);
    if (done || again || !abort_flag) header[1] = -1;
  }
}

thread_local int g_last_launches = 0;

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// Host descriptors handed to the device as a kernel argument (no copy engine, no host-side
// wait): two sizes so that small batches do not pay for a large argument block.
constexpr size_t kDescSmall = 960, kDescLarge = 7168;
template <size_t N>
struct DescBlock {
  int32_t v[N];
};
template <size_t N>
__global__ void stage_desc_kernel(const __grid_constant__ DescBlock<N> blk, int n, int32_t* dst) {
  for (int i = threadIdx.x; i < n; i += blockDim.x) dst[i] = blk.v[i];
}
template <size_t N>
cudaError_t stage_descriptors(const int32_t* const (&src)[4], const size_t (&n)[4], int32_t* dst,
                              cudaStream_t s) {
  DescBlock<N> blk;
  size_t at = 0;
  for (int i = 0; i < 4; ++i) {
    memcpy(blk.v + at, src[i], n[i] * sizeof(int32_t));
    at += n[i];
  }
  stage_desc_kernel<N><<<1, 256, 0, s>>>(blk, int(at), dst);
  return cudaGetLastError();
}

int check_problem_shape(const pp_problem* p) {
  if (!p) return PP_ERR_INVALID_ARG;
  if (p->num_rows < 1 || p->num_groups < 1 || p->num_responses < 1 || p->total_tokens < 1)
    return PP_ERR_INVALID_ARG;
  if (p->num_groups < p->num_rows || p->num_responses < p->num_groups) return PP_ERR_INVALID_ARG;
  if (p->num_q_heads < 1 || p->num_kv_heads < 1 || p->num_q_heads % p->num_kv_heads != 0)
    return PP_ERR_INVALID_ARG;
  if (p->head_dim != 64 && p->head_dim != 96 && p->head_dim != 128) return PP_ERR_UNSUPPORTED;
  // unit records pack (kv head << 24) | tile
  if (p->num_kv_heads > 127 || p->total_tokens / 128 + p->num_groups + p->num_responses >= (1 << 24))
    return PP_ERR_UNSUPPORTED;
  return PP_OK;
}

// Complete validation of host-side descriptors.
int check_host_descriptors(const pp_problem* p) {
  if (!p->row_group_off || !p->grp_prompt_len || !p->grp_resp_off || !p->resp_len)
    return PP_ERR_INVALID_ARG;
  if (p->row_group_off[0] != 0 || p->row_group_off[p->num_rows] != p->num_groups)
    return PP_ERR_INVALID_ARG;
  for (int r = 0; r < p->num_rows; ++r)
    if (p->row_group_off[r + 1] <= p->row_group_off[r]) return PP_ERR_INVALID_ARG;
  if (p->grp_resp_off[0] != 0 || p->grp_resp_off[p->num_groups] != p->num_responses)
    return PP_ERR_INVALID_ARG;
  long long total = 0;
  for (int g = 0; g < p->num_groups; ++g) {
    if (p->grp_prompt_len[g] < 1) return PP_ERR_INVALID_ARG;
    if (p->grp_resp_off[g + 1] <= p->grp_resp_off[g]) return PP_ERR_INVALID_ARG;
    total += p->grp_prompt_len[g];
  }
  for (int x = 0; x < p->num_responses; ++x) {
    if (p->resp_len[x] < 1) return PP_ERR_INVALID_ARG;
    total += p->resp_len[x];
  }
  if (total != p->total_tokens) return PP_ERR_INVALID_ARG;
  return PP_OK;
}

}  // namespace

extern "C" {

int pp_plan_workspace_bytes(const pp_problem* problem, size_t* plan_bytes,
                            size_t* fwd_scratch_bytes, size_t* bwd_scratch_bytes) {
  int rc = check_problem_shape(problem);
  if (rc) return rc;
  if (plan_bytes) *plan_bytes = pp::plan_layout(*problem).total;
  if (fwd_scratch_bytes) *fwd_scratch_bytes = 0;
  if (bwd_scratch_bytes) *bwd_scratch_bytes = pp::bwd_scratch_layout(*problem).total;
  return PP_OK;
}

int pp_build_plan(const pp_problem* problem, void* d_workspace, size_t workspace_bytes,
                  pp_stream_t stream, pp_plan** out_plan) {
  if (!out_plan) return PP_ERR_INVALID_ARG;
  *out_plan = nullptr;
  int rc = check_problem_shape(problem);
  if (rc) return rc;
  if (!d_workspace) return PP_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(d_workspace) & 255) return PP_ERR_ALIGNMENT;
  if (!problem->row_group_off || !problem->grp_prompt_len || !problem->grp_resp_off ||
      !problem->resp_len)
    return PP_ERR_INVALID_ARG;
  pp::PlanLayout lay = pp::plan_layout(*problem);
  if (workspace_bytes < lay.total) return PP_ERR_WORKSPACE_TOO_SMALL;
  if (!problem->desc_on_device) {
    rc = check_host_descriptors(problem);
    if (rc) return rc;
  }
  // first call that touches a device: everything above is host-side validation
  if (!pp::device_is_sm100()) return PP_ERR_UNSUPPORTED;
  pp_plan* plan = new (std::nothrow) pp_plan;
  if (!plan) return PP_ERR_CUDA;
  plan->prob = *problem;
  plan->nseg = problem->num_groups + problem->num_responses;
  plan->max_tiles = pp::max_tiles_of(*problem);
  plan->ws = static_cast<char*>(d_workspace);
  plan->lay = lay;
  plan->fwd_scratch = 0;
  plan->bwd_scratch = pp::bwd_scratch_layout(*problem).total;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);

  g_last_launches = 0;
  if (!problem->desc_on_device) {
    // Stage the four arrays, back to back, in the workspace; the plan kernels read them from
    // there.  Up to kDescLarge entries travel as the argument of a small kernel, which keeps
    // the call asynchronous (a cudaMemcpyAsync from pageable host memory would first wait on
    // the host for everything already in the stream); longer descriptor sets are copied.
    int32_t* d = reinterpret_cast<int32_t*>(plan->ws + lay.desc);
    const int32_t* src[4] = {problem->row_group_off, problem->grp_prompt_len,
                             problem->grp_resp_off, problem->resp_len};
    const size_t n[4] = {size_t(problem->num_rows) + 1, size_t(problem->num_groups),
                         size_t(problem->num_groups) + 1, size_t(problem->num_responses)};
    const size_t n_all = n[0] + n[1] + n[2] + n[3];
    cudaError_t e = cudaSuccess;
    if (n_all <= kDescSmall) {
      e = stage_descriptors<kDescSmall>(src, n, d, s);
      g_last_launches = 1;
    } else if (n_all <= kDescLarge) {
      e = stage_descriptors<kDescLarge>(src, n, d, s);
      g_last_launches = 1;
    } else {
      int32_t* at = d;
      for (int i = 0; i < 4 && e == cudaSuccess; ++i) {
        e = cudaMemcpyAsync(at, src[i], n[i] * sizeof(int32_t), cudaMemcpyHostToDevice, s);
        at += n[i];
      }
    }
    if (e != cudaSuccess) {
      delete plan;
      return PP_ERR_CUDA;
    }
    plan->prob.row_group_off = d;
    plan->prob.grp_prompt_len = d + n[0];
    plan->prob.grp_resp_off = d + n[0] + n[1];
    plan->prob.resp_len = d + n[0] + n[1] + n[2];
  } else {
    // Device descriptors: the first plan kernel copies them into the same block of the
    // workspace, and the plan (plan kernels, position ids, rotary embedding, loss) reads the
    // copy -- the caller's arrays are only needed until that kernel has run.
    int32_t* d = reinterpret_cast<int32_t*>(plan->ws + lay.desc);
    const size_t n0 = size_t(problem->num_rows) + 1, n1 = size_t(problem->num_groups);
    plan->src_desc[0] = problem->row_group_off;
    plan->src_desc[1] = problem->grp_prompt_len;
    plan->src_desc[2] = problem->grp_resp_off;
    plan->src_desc[3] = problem->resp_len;
    plan->prob.row_group_off = d;
    plan->prob.grp_prompt_len = d + n0;
    plan->prob.grp_resp_off = d + n0 + n1;
    plan->prob.resp_len = d + n0 + n1 + n1 + 1;
  }
  if (pp::launch_plan(plan, s, &g_last_launches) != cudaSuccess) {
    delete plan;
    return PP_ERR_CUDA;
  }
  *out_plan = plan;
  return PP_OK;
}

int pp_plan_status(const pp_plan* plan, pp_stream_t stream, int32_t* status, int32_t* detail) {
  if (!plan) return PP_ERR_INVALID_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  int32_t h[2] = {0, 0};
  if (cudaMemcpyAsync(h, plan->ws + plan->lay.header, sizeof h, cudaMemcpyDeviceToHost, s) !=
          cudaSuccess ||
      cudaStreamSynchronize(s) != cudaSuccess)
    return PP_ERR_CUDA;
  if (status) *status = h[0];
  if (detail) *detail = h[1];
  return h[0] == 0 ? PP_OK : PP_ERR_PLAN_STATUS;
}

int pp_destroy_plan(pp_plan* plan) {
  delete plan;
  return PP_OK;
}

int pp_plan_max_tiles(const pp_plan* plan) { return plan ? plan->max_tiles : PP_ERR_INVALID_ARG; }

int pp_plan_read_bwd_units(const pp_plan* plan, pp_stream_t stream, int32_t* units) {
  if (!plan || !units) return PP_ERR_INVALID_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  const size_t n = size_t(plan->max_tiles) * plan->prob.num_kv_heads;
  if (cudaMemcpyAsync(units, plan->ws + plan->lay.bwd_units, n * 4, cudaMemcpyDeviceToHost, s) !=
          cudaSuccess ||
      cudaStreamSynchronize(s) != cudaSuccess)
    return PP_ERR_CUDA;
  return PP_OK;
}

int pp_plan_read_bwd_tiles(const pp_plan* plan, pp_stream_t stream, int32_t* num_tiles,
                           int32_t* btiles) {
  if (!plan) return PP_ERR_INVALID_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  int32_t h[16] = {};
  bool ok = cudaMemcpyAsync(h, plan->ws + plan->lay.header, sizeof h, cudaMemcpyDeviceToHost, s) ==
            cudaSuccess;
  if (ok && btiles)
    ok = cudaMemcpyAsync(btiles, plan->ws + plan->lay.btiles,
                         size_t(plan->max_tiles) * sizeof(pp::BTile), cudaMemcpyDeviceToHost,
                         s) == cudaSuccess;
  if (!ok || cudaStreamSynchronize(s) != cudaSuccess) return PP_ERR_CUDA;
  if (num_tiles) *num_tiles = h[pp::kHdrNumBTiles];
  return h[0] == 0 ? PP_OK : PP_ERR_PLAN_STATUS;
}

int pp_plan_read(const pp_plan* plan, pp_stream_t stream, int32_t* num_tiles, int32_t* tiles,
                 int32_t* fwd_order, int32_t* bwd_order, int32_t* key_end) {
  if (!plan) return PP_ERR_INVALID_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  int32_t h[4] = {0, 0, 0, 0};
  bool ok = cudaMemcpyAsync(h, plan->ws + plan->lay.header, sizeof h, cudaMemcpyDeviceToHost, s) ==
            cudaSuccess;
  size_t mt = size_t(plan->max_tiles);
  if (ok && tiles)
    ok = cudaMemcpyAsync(tiles, plan->ws + plan->lay.tiles, mt * sizeof(pp::Tile),
                         cudaMemcpyDeviceToHost, s) == cudaSuccess;
  if (ok && fwd_order)
    ok = cudaMemcpyAsync(fwd_order, plan->ws + plan->lay.fwd_order, mt * 4, cudaMemcpyDeviceToHost,
                         s) == cudaSuccess;
  if (ok && bwd_order)
    ok = cudaMemcpyAsync(bwd_order, plan->ws + plan->lay.bwd_order, mt * 4, cudaMemcpyDeviceToHost,
                         s) == cudaSuccess;
  if (ok && key_end)
    ok = cudaMemcpyAsync(key_end, plan->ws + plan->lay.key_end,
                         size_t(plan->prob.total_tokens) * 4, cudaMemcpyDeviceToHost, s) ==
         cudaSuccess;
  if (!ok || cudaStreamSynchronize(s) != cudaSuccess) return PP_ERR_CUDA;
  if (num_tiles) *num_tiles = h[2];
  return h[0] == 0 ? PP_OK : PP_ERR_PLAN_STATUS;
}

int pp_attn_fwd(const pp_plan* plan, const void* q, const void* k, const void* v,
                float softmax_scale, void* o, float* lse, void* d_scratch, size_t scratch_bytes,
                pp_stream_t stream) {
  g_last_launches = 0;
  if (!plan || !q || !k || !v || !o || !lse) return PP_ERR_INVALID_ARG;
  if (!(softmax_scale > 0.f) || softmax_scale > 1e30f) return PP_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(lse))
    return PP_ERR_ALIGNMENT;
  // Optional: the buffer the caller will hand to pp_attn_bwd as scratch.  The forward then
  // also clears the fp32 dQ accumulator inside it (the kernel is compute-bound and has memory
  // bandwidth to spare), and the backward's preprocess pass skips its own clearing.
  // Measured: it pays while the accumulator is a few hundred MB (0.15-0.3 GB: step -4..5 %,
  // 0.54 GB: -1.5..4 %); at 1 GB the extra stores slow the forward's loads and the zeros have
  // left L2 long before the backward adds to them (step +2 %), so larger accumulators are left
  // to the backward.
  constexpr size_t kFwdClearMaxBytes = size_t(640) << 20;
  float* dq_clear = nullptr;
  plan->cleared_scratch = nullptr;
  if (d_scratch) {
    if (scratch_bytes < plan->bwd_scratch) return PP_ERR_WORKSPACE_TOO_SMALL;
    if (reinterpret_cast<uintptr_t>(d_scratch) & 255) return PP_ERR_ALIGNMENT;
    const pp_problem& pb = plan->prob;
    if (size_t(4) * pb.total_tokens * pb.num_q_heads * pb.head_dim <= kFwdClearMaxBytes)
      dq_clear = reinterpret_cast<float*>(static_cast<char*>(d_scratch) +
                                          pp::bwd_scratch_layout(pb).dq_acc);
  }
  cudaError_t e = pp::launch_fwd(plan, q, k, v, softmax_scale, o, lse, dq_clear,
                                 reinterpret_cast<cudaStream_t>(stream), &g_last_launches);
  if (e == cudaSuccess && dq_clear) plan->cleared_scratch = d_scratch;
  return e == cudaSuccess ? PP_OK : (e == cudaErrorNotSupported ? PP_ERR_UNSUPPORTED : PP_ERR_CUDA);
}

static int attn_bwd_common(const pp_plan* plan, const void* q, const void* k, const void* v,
                           const void* o, const float* lse, const void* d_o, float softmax_scale,
                           void* d_q, void* d_k, void* d_v, void* d_scratch, size_t scratch_bytes,
                           pp_stream_t stream, bool deterministic) {
  g_last_launches = 0;
  if (!plan || !q || !k || !v || !o || !lse || !d_o || !d_q || !d_k || !d_v || !d_scratch)
    return PP_ERR_INVALID_ARG;
  if (!(softmax_scale > 0.f) || softmax_scale > 1e30f) return PP_ERR_INVALID_ARG;
  if (scratch_bytes < plan->bwd_scratch) return PP_ERR_WORKSPACE_TOO_SMALL;
  const void* ptrs[] = {q, k, v, o, lse, d_o, d_q, d_k, d_v};
  for (const void* p : ptrs)
    if (!aligned16(p)) return PP_ERR_ALIGNMENT;
  if (reinterpret_cast<uintptr_t>(d_scratch) & 255) return PP_ERR_ALIGNMENT;
  // cleared by the latest forward on this plan (which must precede this call on the stream)?
  const bool dq_cleared = plan->cleared_scratch == d_scratch;
  plan->cleared_scratch = nullptr;
  cudaError_t e = pp::launch_bwd(plan, q, k, v, o, lse, d_o, softmax_scale, d_q, d_k, d_v,
                                 d_scratch, dq_cleared, deterministic,
                                 reinterpret_cast<cudaStream_t>(stream), &g_last_launches);
  return e == cudaSuccess ? PP_OK : (e == cudaErrorNotSupported ? PP_ERR_UNSUPPORTED : PP_ERR_CUDA);
}

int pp_attn_bwd(const pp_plan* plan, const void* q, const void* k, const void* v, const void* o,
                const float* lse, const void* d_o, float softmax_scale, void* d_q, void* d_k,
                void* d_v, void* d_scratch, size_t scratch_bytes, pp_stream_t stream) {
  return attn_bwd_common(plan, q, k, v, o, lse, d_o, softmax_scale, d_q, d_k, d_v, d_scratch,
                         scratch_bytes, stream, false);
}

int pp_attn_bwd_deterministic(const pp_plan* plan, const void* q, const void* k, const void* v,
                              const void* o, const float* lse, const void* d_o,
                              float softmax_scale, void* d_q, void* d_k, void* d_v,
                              void* d_scratch, size_t scratch_bytes, pp_stream_t stream) {
  return attn_bwd_common(plan, q, k, v, o, lse, d_o, softmax_scale, d_q, d_k, d_v, d_scratch,
                         scratch_bytes, stream, true);
}

int pp_attn_bwd_noalloc_max_bytes(size_t* bytes) {
  if (!bytes) return PP_ERR_INVALID_ARG;
  *bytes = pp::kStaticScratchBytes;
  return PP_OK;
}

int pp_attn_bwd_noalloc(const pp_plan* plan, const void* q, const void* k, const void* v,
                        const void* o, const float* lse, const void* d_o, float softmax_scale,
                        void* d_q, void* d_k, void* d_v, pp_stream_t stream) {
  g_last_launches = 0;
  if (!plan || !q || !k || !v || !o || !lse || !d_o || !d_q || !d_k || !d_v)
    return PP_ERR_INVALID_ARG;
  if (!(softmax_scale > 0.f) || softmax_scale > 1e30f) return PP_ERR_INVALID_ARG;
  if (plan->bwd_scratch > pp::kStaticScratchBytes) return PP_ERR_STATIC_SCRATCH_LIMIT;
  const void* ptrs[] = {q, k, v, o, lse, d_o, d_q, d_k, d_v};
  for (const void* p : ptrs)
    if (!aligned16(p)) return PP_ERR_ALIGNMENT;
  cudaError_t e = pp::launch_bwd_static(plan, q, k, v, o, lse, d_o, softmax_scale, d_q, d_k, d_v,
                                        reinterpret_cast<cudaStream_t>(stream), &g_last_launches);
  if (e == cudaErrorInvalidDevice) return PP_ERR_INVALID_ARG;  // the plan's device is not current
  return e == cudaSuccess ? PP_OK : (e == cudaErrorNotSupported ? PP_ERR_UNSUPPORTED : PP_ERR_CUDA);
}

int pp_debug_expire_wait(const pp_plan* plan, int32_t site, pp_stream_t stream) {
  if (!plan || site < 1) return PP_ERR_INVALID_ARG;
  expire_wait_kernel<<<1, 32, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
      reinterpret_cast<int32_t*>(plan->ws + plan->lay.header), site);
  return cudaGetLastError() == cudaSuccess ? PP_OK : PP_ERR_CUDA;
}

int pp_position_ids(const pp_plan* plan, int32_t* position_ids, pp_stream_t stream) {
  g_last_launches = 0;
  if (!plan || !position_ids) return PP_ERR_INVALID_ARG;
  if (pp::launch_position_ids(plan, position_ids, reinterpret_cast<cudaStream_t>(stream)) !=
      cudaSuccess)
    return PP_ERR_CUDA;
  g_last_launches = 1;
  return PP_OK;
}

int pp_rope_qk(const pp_plan* plan, void* q, void* k, float rope_base, pp_stream_t stream) {
  g_last_launches = 0;
  if (!plan || !q || !k) return PP_ERR_INVALID_ARG;
  if (!(rope_base > 1.f) || rope_base > 1e12f) return PP_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k)) return PP_ERR_ALIGNMENT;
  if (pp::launch_rope(plan, q, k, rope_base, reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess)
    return PP_ERR_CUDA;
  g_last_launches = 1;
  return PP_OK;
}

int pp_preference_loss(const pp_plan* plan, const float* token_logp, const float* ref_token_logp,
                       float beta, float* resp_logp, float* resp_reward, float* grp_loss,
                       float* d_token_logp, pp_stream_t stream) {
  g_last_launches = 0;
  if (!plan || !token_logp || !resp_logp || !resp_reward || !grp_loss) return PP_ERR_INVALID_ARG;
  if (!(beta > 0.f) || beta > 1e30f) return PP_ERR_INVALID_ARG;
  if (pp::launch_preference_loss(plan, token_logp, ref_token_logp, beta, resp_logp, resp_reward,
                                 grp_loss, d_token_logp,
                                 reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess)
    return PP_ERR_CUDA;
  g_last_launches = 1;
  return PP_OK;
}

int pp_last_launch_count(void) { return g_last_launches; }

int pp_step_host_arena_bytes(const pp_problem* problem, size_t* arena_bytes) {
  int rc = check_problem_shape(problem);
  if (rc) return rc;
  if (!arena_bytes) return PP_ERR_INVALID_ARG;
  *arena_bytes = pp::step_arena_layout(*problem).total;
  return PP_OK;
}

namespace {
// Side streams and events of pp_attn_step_host, created once per device on first use.
struct StepStreams {
  cudaStream_t up = nullptr, down = nullptr;
  cudaEvent_t e_start = nullptr, e_end = nullptr;
  cudaEvent_t e_qkv[pp::kStepChunks] = {}, e_do[pp::kStepChunks] = {}, e_fwd[pp::kStepChunks] = {},
              e_bwd[pp::kStepChunks] = {};
};
StepStreams* step_streams() {
  static std::mutex mu;
  static StepStreams per_device[pp::kMaxDevices];
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= pp::kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  StepStreams& st = per_device[dev];
  if (!st.up) {
    auto ev = [](cudaEvent_t* e) {
      return cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess;
    };
    bool ok = cudaStreamCreateWithFlags(&st.up, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&st.down, cudaStreamNonBlocking) == cudaSuccess &&
              ev(&st.e_start) && ev(&st.e_end);
    for (int c = 0; ok && c < pp::kStepChunks; ++c)
      ok = ev(&st.e_qkv[c]) && ev(&st.e_do[c]) && ev(&st.e_fwd[c]) && ev(&st.e_bwd[c]);
    if (!ok) {
      st = StepStreams();
      return nullptr;
    }
  }
  return &st;
}

// One run of whole rows of a step: its descriptors (rebased to start at zero), its token range
// and where its private blocks sit in the arena.
struct StepChunk {
  std::vector<int32_t> row_group_off, grp_resp_off;
  pp_problem prob{};
  size_t t0 = 0, plan_off = 0, plan_bytes = 0, scratch_off = 0, scratch_bytes = 0, lse_off = 0;
};

// Cuts `p` (host descriptors, already validated) into at most `want` runs of whole groups with
// about equal token counts.  Groups never interact, so a row that is cut becomes two rows.
std::vector<StepChunk> cut_step(const pp_problem& p, int want) {
  std::vector<size_t> grp_end(p.num_groups);
  size_t t = 0;
  for (int g = 0; g < p.num_groups; ++g) {
    t += p.grp_prompt_len[g];
    for (int i = p.grp_resp_off[g]; i < p.grp_resp_off[g + 1]; ++i) t += p.resp_len[i];
    grp_end[g] = t;
  }
  const int n = std::max(1, std::min(want, p.num_groups));
  std::vector<StepChunk> out;
  int g0 = 0, r = 0;
  for (int c = 0; c < n && g0 < p.num_groups; ++c) {
    int g1 = g0 + 1;
    const size_t target = t * size_t(c + 1) / size_t(n);
    // leave at least one group for every later run
    while (g1 < p.num_groups - (n - 1 - c) && grp_end[g1 - 1] < target) ++g1;
    if (c == n - 1) g1 = p.num_groups;
    StepChunk ch;
    const int i0 = p.grp_resp_off[g0], i1 = p.grp_resp_off[g1];
    ch.row_group_off.push_back(0);
    while (p.row_group_off[r + 1] <= g0) ++r;
    for (int rr = r; rr < p.num_rows && p.row_group_off[rr] < g1; ++rr)
      ch.row_group_off.push_back(std::min(p.row_group_off[rr + 1], g1) - g0);
    for (int g = g0; g <= g1; ++g) ch.grp_resp_off.push_back(p.grp_resp_off[g] - i0);
    ch.t0 = g0 ? grp_end[g0 - 1] : 0;
    ch.prob = p;
    ch.prob.num_rows = int32_t(ch.row_group_off.size()) - 1;
    ch.prob.num_groups = g1 - g0;
    ch.prob.num_responses = i1 - i0;
    ch.prob.total_tokens = int32_t(grp_end[g1 - 1] - ch.t0);
    ch.prob.grp_prompt_len = p.grp_prompt_len + g0;
    ch.prob.resp_len = p.resp_len + i0;
    out.push_back(std::move(ch));
    g0 = g1;
  }
  for (StepChunk& ch : out) {   // the vectors no longer move
    ch.prob.row_group_off = ch.row_group_off.data();
    ch.prob.grp_resp_off = ch.grp_resp_off.data();
  }
  return out;
}

// A run below a quarter MiB of input is all launch overhead: fewer runs then.
int step_runs_wanted(const pp_problem& p) {
  const size_t in_bytes = size_t(p.total_tokens) * (p.num_q_heads + p.num_kv_heads) * p.head_dim * 4;
  return int(std::min<size_t>(pp::kStepChunks, std::max<size_t>(1, in_bytes >> 18)));
}

// Places the chunks' private blocks; false if they do not fit the arena's regions.
bool place_step(std::vector<StepChunk>& chunks, const pp::StepArena& a, size_t heads_q) {
  size_t po = a.plan, so = a.scratch, lo = a.lse;
  for (StepChunk& ch : chunks) {
    ch.plan_off = po;
    ch.plan_bytes = pp::plan_layout(ch.prob).total;
    po += pp::align_up(ch.plan_bytes, 256);
    ch.scratch_off = so;
    ch.scratch_bytes = pp::bwd_scratch_layout(ch.prob).total;
    so += pp::align_up(ch.scratch_bytes, 256);
    ch.lse_off = lo;
    lo += pp::align_up(size_t(ch.prob.total_tokens) * heads_q * 4, 256);
  }
  return po <= a.scratch && so <= a.total && lo <= a.dq;
}
}  // namespace

int pp_step_host_runs(const pp_problem* problem, int32_t* num_runs, int32_t* group_begin,
                      int32_t* token_begin) {
  int rc = check_problem_shape(problem);
  if (rc) return rc;
  if (problem->desc_on_device || !num_runs || !group_begin || !token_begin)
    return PP_ERR_INVALID_ARG;
  if (!problem->row_group_off || !problem->grp_prompt_len || !problem->grp_resp_off ||
      !problem->resp_len)
    return PP_ERR_INVALID_ARG;
  rc = check_host_descriptors(problem);
  if (rc) return rc;
  const std::vector<StepChunk> chunks = cut_step(*problem, step_runs_wanted(*problem));
  int g = 0;
  for (size_t c = 0; c < chunks.size(); ++c) {
    group_begin[c] = g;
    token_begin[c] = int32_t(chunks[c].t0);
    g += chunks[c].prob.num_groups;
  }
  group_begin[chunks.size()] = g;
  token_begin[chunks.size()] = problem->total_tokens;
  *num_runs = int32_t(chunks.size());
  return PP_OK;
}

int pp_attn_step_host(const pp_problem* problem, const void* h_q, const void* h_k, const void* h_v,
                      const void* h_do, float softmax_scale, void* h_o, float* h_lse, void* h_dq,
                      void* h_dk, void* h_dv, void* d_arena, size_t arena_bytes,
                      pp_stream_t stream) {
  g_last_launches = 0;
  int rc = check_problem_shape(problem);
  if (rc) return rc;
  if (problem->desc_on_device) return PP_ERR_INVALID_ARG;
  if (!h_q || !h_k || !h_v || !h_do || !h_o || !h_lse || !h_dq || !h_dk || !h_dv || !d_arena)
    return PP_ERR_INVALID_ARG;
  if (!problem->row_group_off || !problem->grp_prompt_len || !problem->grp_resp_off ||
      !problem->resp_len)
    return PP_ERR_INVALID_ARG;
  rc = check_host_descriptors(problem);
  if (rc) return rc;
  if (reinterpret_cast<uintptr_t>(d_arena) & 255) return PP_ERR_ALIGNMENT;
  const pp::StepArena a = pp::step_arena_layout(*problem);
  if (arena_bytes < a.total) return PP_ERR_WORKSPACE_TOO_SMALL;
  StepStreams* ss = step_streams();
  if (!ss) return PP_ERR_CUDA;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  char* base = static_cast<char*>(d_arena);
  const size_t T = problem->total_tokens, D = problem->head_dim;
  const size_t Hq = problem->num_q_heads, Hkv = problem->num_kv_heads;

  // Groups are independent, so the step runs as a short pipeline over runs of whole groups: the
  // inputs of run c+1 go up and the results of run c-1 come down (two copy engines, opposite
  // directions) while the kernels of run c execute.  Inside a run dO still goes up behind
  // the forward and O / LSE come down behind the backward.
  std::vector<StepChunk> chunks = cut_step(*problem, step_runs_wanted(*problem));
  if (!place_step(chunks, a, Hq)) {
    chunks = cut_step(*problem, 1);
    if (!place_step(chunks, a, Hq)) return PP_ERR_WORKSPACE_TOO_SMALL;
  }
  auto ok = [](cudaError_t e) { return e == cudaSuccess; };
  if (!ok(cudaEventRecord(ss->e_start, s)) || !ok(cudaStreamWaitEvent(ss->up, ss->e_start, 0)) ||
      !ok(cudaStreamWaitEvent(ss->down, ss->e_start, 0)))
    return PP_ERR_CUDA;  // nothing has been given to the side streams yet
  int launches = 0;
  const char* hq = static_cast<const char*>(h_q);
  const char* hk = static_cast<const char*>(h_k);
  const char* hv = static_cast<const char*>(h_v);
  const char* hdo = static_cast<const char*>(h_do);
  for (size_t c = 0; c < chunks.size() && rc == PP_OK; ++c) {  // all uploads, in order, on `up`
    const StepChunk& ch = chunks[c];
    const size_t tc = ch.prob.total_tokens;
    const size_t qo = ch.t0 * Hq * D * 2, ko = ch.t0 * Hkv * D * 2;
    const size_t qb = tc * Hq * D * 2, kb = tc * Hkv * D * 2;
    if (!ok(cudaMemcpyAsync(base + a.q + qo, hq + qo, qb, cudaMemcpyHostToDevice, ss->up)) ||
        !ok(cudaMemcpyAsync(base + a.k + ko, hk + ko, kb, cudaMemcpyHostToDevice, ss->up)) ||
        !ok(cudaMemcpyAsync(base + a.v + ko, hv + ko, kb, cudaMemcpyHostToDevice, ss->up)) ||
        !ok(cudaEventRecord(ss->e_qkv[c], ss->up)) ||
        !ok(cudaMemcpyAsync(base + a.d_o + qo, hdo + qo, qb, cudaMemcpyHostToDevice, ss->up)) ||
        !ok(cudaEventRecord(ss->e_do[c], ss->up)))
      rc = PP_ERR_CUDA;  // fall through to the join below: copies may already be in flight
  }
  for (size_t c = 0; c < chunks.size() && rc == PP_OK; ++c) {
    const StepChunk& ch = chunks[c];
    const size_t tc = ch.prob.total_tokens;
    const size_t qo = ch.t0 * Hq * D * 2, ko = ch.t0 * Hkv * D * 2;
    const size_t qb = tc * Hq * D * 2, kb = tc * Hkv * D * 2;
    float* d_lse = reinterpret_cast<float*>(base + ch.lse_off);
    pp_plan* plan = nullptr;
    rc = pp_build_plan(&ch.prob, base + ch.plan_off, ch.plan_bytes, stream, &plan);
    if (rc) break;
    launches += g_last_launches;
    if (!ok(cudaStreamWaitEvent(s, ss->e_qkv[c], 0))) rc = PP_ERR_CUDA;
    if (rc == PP_OK) {
      rc = pp_attn_fwd(plan, base + a.q + qo, base + a.k + ko, base + a.v + ko, softmax_scale,
                       base + a.o + qo, d_lse, base + ch.scratch_off, ch.scratch_bytes, stream);
      launches += g_last_launches;
    }
    if (rc == PP_OK) {
      // LSE is [Hq][tokens of the run] on the device and [Hq][T] on the host
      bool good =
          ok(cudaEventRecord(ss->e_fwd[c], s)) && ok(cudaStreamWaitEvent(ss->down, ss->e_fwd[c], 0)) &&
          ok(cudaMemcpyAsync(static_cast<char*>(h_o) + qo, base + a.o + qo, qb,
                             cudaMemcpyDeviceToHost, ss->down)) &&
          ok(cudaMemcpy2DAsync(h_lse + ch.t0, T * 4, d_lse, tc * 4, tc * 4, Hq,
                               cudaMemcpyDeviceToHost, ss->down)) &&
          ok(cudaStreamWaitEvent(s, ss->e_do[c], 0));
      if (!good) rc = PP_ERR_CUDA;
    }
    if (rc == PP_OK) {
      rc = pp_attn_bwd(plan, base + a.q + qo, base + a.k + ko, base + a.v + ko, base + a.o + qo,
                       d_lse, base + a.d_o + qo, softmax_scale, base + a.dq + qo, base + a.dk + ko,
                       base + a.dv + ko, base + ch.scratch_off, ch.scratch_bytes, stream);
      launches += g_last_launches;
    }
    pp_destroy_plan(plan);
    if (rc == PP_OK) {
      bool good =
          ok(cudaEventRecord(ss->e_bwd[c], s)) && ok(cudaStreamWaitEvent(ss->down, ss->e_bwd[c], 0)) &&
          ok(cudaMemcpyAsync(static_cast<char*>(h_dq) + qo, base + a.dq + qo, qb,
                             cudaMemcpyDeviceToHost, ss->down)) &&
          ok(cudaMemcpyAsync(static_cast<char*>(h_dk) + ko, base + a.dk + ko, kb,
                             cudaMemcpyDeviceToHost, ss->down)) &&
          ok(cudaMemcpyAsync(static_cast<char*>(h_dv) + ko, base + a.dv + ko, kb,
                             cudaMemcpyDeviceToHost, ss->down));
      if (!good) rc = PP_ERR_CUDA;
    }
  }
  // the caller's stream ends behind everything the side streams were given, also on failure
  bool joined = ok(cudaEventRecord(ss->e_end, ss->down)) && ok(cudaStreamWaitEvent(s, ss->e_end, 0)) &&
                ok(cudaEventRecord(ss->e_end, ss->up)) && ok(cudaStreamWaitEvent(s, ss->e_end, 0));
  g_last_launches = launches;
  if (rc) return rc;
  return joined ? PP_OK : PP_ERR_CUDA;
}

int pp_profile_enable(int on) {
  if (on < 0 || on > 2) return PP_ERR_INVALID_ARG;
  return pp::profile_enable(on) ? PP_OK : PP_ERR_CUDA;
}

int pp_profile_read(float* fwd_kernel_ms, float* bwd_main_kernel_ms) {
  return pp::profile_read(fwd_kernel_ms, bwd_main_kernel_ms) ? PP_OK : PP_ERR_CUDA;
}

int pp_profile_read_all(float* fwd_kernel_ms, float* bwd_main_kernel_ms, int32_t capacity,
                        int32_t* num_fwd, int32_t* num_bwd) {
  if (capacity < 0) return PP_ERR_INVALID_ARG;
  int nf = 0, nb = 0;
  const bool ok = pp::profile_read_all(fwd_kernel_ms, bwd_main_kernel_ms, capacity, &nf, &nb);
  if (num_fwd) *num_fwd = nf;
  if (num_bwd) *num_bwd = nb;
  return ok ? PP_OK : PP_ERR_CUDA;
}

int pp_build_rows_workspace_bytes(int32_t num_groups, size_t* bytes) {
  if (num_groups < 1 || !bytes) return PP_ERR_INVALID_ARG;
  *bytes = pp::rows_workspace_bytes(num_groups);
  return PP_OK;
}

int pp_build_rows(int32_t num_groups, int32_t num_responses, const int32_t* grp_prompt_len,
                  const int32_t* grp_resp_off, const int32_t* resp_len, int32_t row_capacity,
                  void* d_workspace, size_t workspace_bytes, int32_t* order,
                  int32_t* row_group_off, int32_t* num_rows, int64_t* row_tokens,
                  int64_t* row_cost, int32_t* out_prompt_len, int32_t* out_resp_off,
                  int32_t* out_resp_len, int32_t* status, pp_stream_t stream) {
  g_last_launches = 0;
  if (num_groups < 1 || num_responses < num_groups || row_capacity < 1 || !grp_prompt_len ||
      !grp_resp_off || !resp_len || !d_workspace || !order || !row_group_off || !num_rows ||
      !row_tokens || !row_cost || !out_prompt_len || !out_resp_off || !out_resp_len || !status)
    return PP_ERR_INVALID_ARG;
  if (num_groups > 65536) return PP_ERR_UNSUPPORTED;
  if (workspace_bytes < pp::rows_workspace_bytes(num_groups)) return PP_ERR_WORKSPACE_TOO_SMALL;
  if (reinterpret_cast<uintptr_t>(d_workspace) & 255) return PP_ERR_ALIGNMENT;
  cudaError_t e = pp::launch_build_rows(
      num_groups, num_responses, grp_prompt_len, grp_resp_off, resp_len, row_capacity, d_workspace,
      order, row_group_off, num_rows, reinterpret_cast<long long*>(row_tokens),
      reinterpret_cast<long long*>(row_cost), out_prompt_len, out_resp_off, out_resp_len, status,
      reinterpret_cast<cudaStream_t>(stream), &g_last_launches);
  return e == cudaSuccess ? PP_OK : PP_ERR_CUDA;
}

int pp_assign_rows(int32_t num_rows, const int64_t* row_cost, int32_t num_ranks, int32_t* order,
                   int32_t* rank_of_row, int64_t* rank_cost, pp_stream_t stream) {
  g_last_launches = 0;
  if (num_rows < 1 || num_ranks < 1 || !row_cost || !order || !rank_of_row || !rank_cost)
    return PP_ERR_INVALID_ARG;
  if (num_rows > 65536 || num_ranks > 1024) return PP_ERR_UNSUPPORTED;
  cudaError_t e = pp::launch_assign_rows(
      num_rows, reinterpret_cast<const long long*>(row_cost), num_ranks, order, rank_of_row,
      reinterpret_cast<long long*>(rank_cost), reinterpret_cast<cudaStream_t>(stream),
      &g_last_launches);
  return e == cudaSuccess ? PP_OK : PP_ERR_CUDA;
}

const char* pp_error_string(int code) {
  switch (code) {
    case PP_OK: return "ok";
    case PP_ERR_INVALID_ARG: return "invalid argument";
    case PP_ERR_UNSUPPORTED: return "unsupported head_dim or device";
    case PP_ERR_WORKSPACE_TOO_SMALL: return "workspace or scratch too small";
    case PP_ERR_ALIGNMENT: return "pointer not sufficiently aligned";
    case PP_ERR_CUDA: return "CUDA call failed";
    case PP_ERR_PLAN_STATUS: return "device-side validation failed or a bounded wait expired";
    case PP_ERR_STATIC_SCRATCH_LIMIT:
      return "problem needs more backward scratch than the 32 MiB built into the library; "
             "use pp_attn_bwd with caller-provided scratch";
    default: return "unknown error";
  }
}

}  // extern "C"
