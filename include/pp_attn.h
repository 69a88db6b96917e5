/*
 * pp_attn.h -- C ABI of the preference-packed attention library for B200 (sm_100a).
 *
 * Operation (paper Sec. 3.2, "Preference packing"): one preference sample
 * (x, y^1 .. y^K) is laid out as a single sequence [x | y^1 | ... | y^K].  The
 * attention mask makes the result identical to running the K sequences (x, y^k)
 * separately: prompt tokens attend causally among themselves, a response token
 * attends to the whole prompt and causally inside its own response, and never to
 * another response.  Several such groups may follow each other in one row (batch
 * packing, Sec. 2.2); attention never crosses a group boundary.  The library
 * computes that masked softmax attention, forward and backward, touching only the
 * (query, key) tiles the mask leaves visible.
 *
 * Data layout (all device memory, owned by the caller, never freed or allocated here):
 *   tokens of all rows are concatenated; T = total tokens; no padding tokens exist.
 *   Q, O, dO, dQ : bf16 [T][Hq][D]        K, V, dK, dV : bf16 [T][Hkv][D]
 *   LSE          : fp32 [Hq][T], natural log of sum_j exp(scale * q_i . k_j) over visible j
 *   query head h reads KV head h / (Hq / Hkv).
 *   Base pointers must be 16-byte aligned.  Inputs must be finite.
 *
 * All functions return 0 (PP_OK) or a negative pp_status; they never throw, exit or print.
 * Work is enqueued on the caller's stream; only pp_plan_status and the pp_plan_read* test
 * accessors synchronise it.
 */
#ifndef PP_ATTN_H_
#define PP_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st* pp_stream_t; /* a cudaStream_t */
typedef struct pp_plan pp_plan;          /* opaque host handle; device part lives in caller memory */

enum pp_status {
  PP_OK = 0,
  PP_ERR_INVALID_ARG = -1,         /* null pointer, non-positive length, non-monotone offsets,
                                      total_tokens mismatch, Hq % Hkv != 0 */
  PP_ERR_UNSUPPORTED = -2,         /* head_dim not in {64, 96, 128}; device is not compute capability 10.x */
  PP_ERR_WORKSPACE_TOO_SMALL = -3, /* plan workspace or scratch smaller than the size query says */
  PP_ERR_ALIGNMENT = -4,           /* a tensor base pointer is not 16-byte aligned */
  PP_ERR_CUDA = -5,                /* a CUDA runtime / driver call failed */
  PP_ERR_PLAN_STATUS = -6,         /* device-side validation failed or a bounded wait expired */
  PP_ERR_STATIC_SCRATCH_LIMIT = -7 /* pp_attn_bwd_noalloc: problem larger than its built-in scratch */
};

/*
 * Problem statement, in the paper's terms (Sec. 3.1 symbols): per group g one prompt of
 * length P_g (l_in) and n_g >= 1 responses of lengths R_{g,1..n_g} (l_resp^k).
 * Descriptor arrays are int32 and are read by pp_build_plan only: host arrays during the call,
 * device arrays by the first plan kernel it enqueues, which copies them into the workspace
 * (keep them unchanged until that kernel has run; everything later -- the other plan kernels,
 * pp_position_ids, pp_rope_qk, pp_preference_loss -- reads the copy).
 */
typedef struct {
  int32_t num_rows;
  const int32_t* row_group_off;  /* [num_rows + 1]  groups of row r = [off[r], off[r+1])      */
  const int32_t* grp_prompt_len; /* [G]             P_g >= 1                                  */
  const int32_t* grp_resp_off;   /* [G + 1]         responses of group g = [off[g], off[g+1]) */
  const int32_t* resp_len;       /* [N]             R >= 1                                    */
  int32_t num_groups;            /* G = row_group_off[num_rows]                               */
  int32_t num_responses;         /* N = grp_resp_off[G]                                       */
  int32_t desc_on_device;        /* 0: host arrays (validated and copied by the library);
                                    1: device arrays (validated by the plan kernel)          */
  int32_t num_q_heads;           /* Hq                                                        */
  int32_t num_kv_heads;          /* Hkv, divides Hq                                           */
  int32_t head_dim;              /* D: 64, 96 or 128                                          */
  int32_t total_tokens;          /* T = sum of every prompt and response length (checked)     */
} pp_problem;

/* Bytes the caller must provide: plan workspace (device, 256-byte aligned), scratch for
 * pp_attn_fwd (may be 0) and for pp_attn_bwd (fp32 dQ accumulator, Delta, scaled LSE). */
int pp_plan_workspace_bytes(const pp_problem* problem, size_t* plan_bytes,
                            size_t* fwd_scratch_bytes, size_t* bwd_scratch_bytes);

/*
 * Plan builder (device side, stream ordered, no host synchronisation).  Turns the segment
 * descriptors into query/key tiles of 128 tokens aligned to segment starts, each with the
 * key ranges it must visit -- the prompt range and the part of its own segment before it
 * (class FULL: no masking), then its own diagonal tile (class DIAG: causal masking) --
 * while tiles of sibling responses are never listed (class SKIP is implicit).  The same
 * tiles, read as key tiles, carry the contiguous query range [start, vis_end) that sees
 * them, for the backward pass.  Tiles are ordered longest-work-first for the forward pass;
 * the backward pass processes (tile, KV head) units group by group (largest group first,
 * longest tile first inside a group) so that concurrently running units share Q / dO in L2.
 * Both kernels draw units dynamically, so the order is a priority list, not an assignment.
 * Host descriptors (desc_on_device == 0) are validated on the host and staged in the
 * workspace: up to 7168 entries over the four arrays travel as the argument of a small kernel,
 * so the call never waits on the host for work already in `stream`; longer ones are copied
 * with cudaMemcpyAsync, which for pageable host memory does wait for the stream first.  The
 * host arrays may be changed or freed as soon as the call returns -- except page-locked arrays
 * of more than 7168 entries, which the copy reads asynchronously: keep those unchanged until
 * `stream` has reached the plan kernels.
 * d_workspace must stay alive and untouched while the plan is used.  The plan's tables are
 * fixed once built and serve any number of pp_attn_fwd / pp_attn_bwd calls whose tensors have
 * the shapes stated in `problem`, with two pieces of mutable state to respect:
 *  - the workspace holds the work counters the kernels draw their units from (re-armed by the
 *    last CTA of each launch), so two forwards, or two backwards, on ONE plan must not overlap
 *    on the GPU: order them on one stream (or by events); overlapping launches would each
 *    process part of the work and leave outputs partly unwritten.  Build one plan per stream
 *    for concurrent use.  A forward and a backward never share a counter.
 *  - the host handle remembers which scratch buffer the latest pp_attn_fwd cleared for the next
 *    pp_attn_bwd (see pp_attn_fwd): calls on one plan must come from one host thread at a time.
 * Returns PP_ERR_UNSUPPORTED when the current device is not compute capability 10.x.
 */
int pp_build_plan(const pp_problem* problem, void* d_workspace, size_t workspace_bytes,
                  pp_stream_t stream, pp_plan** out_plan);

/* Synchronises `stream`, then reports the device status word (0 = fine) and a detail word
 * (site of a failed validation or of an expired wait).  Returns PP_ERR_PLAN_STATUS if the
 * status is non-zero. */
int pp_plan_status(const pp_plan* plan, pp_stream_t stream, int32_t* status, int32_t* detail);

/* Frees the host handle only. */
int pp_destroy_plan(pp_plan* plan);

/* Debug / test access: copies the forward tile table to host memory after synchronising
 * `stream`.  Each tile is 8 int32: {start, len, kv0_start, kv0_len, kv1_start, kv1_len, vis_end,
 * work}; forward tiles are cut per segment.  fwd_order receives the forward processing order
 * (tile indices); bwd_order the backward tiles (indices into the backward tile table, below)
 * longest work first.  key_end receives, per token j, the first query index that can NOT see
 * key j.  Any pointer may be NULL.  *num_tiles receives the forward tile count; arrays must
 * hold pp_plan_max_tiles entries. */
int pp_plan_max_tiles(const pp_plan* plan);
/* The backward's key tiles: each GROUP (prompt and responses as one token range) cut into
 * tiles of 128 tokens from the group's start, so a tile may straddle segments.  Each record is
 * 8 int32: {start, len, vis_end, dep_lo, grp_start, grp_end, work, npc}: queries
 * [start, vis_end) see at least one key of the tile, work = number of 128-token query tiles
 * from `start` that reach vis_end, npc = number of tiles of the group that hold prompt keys;
 * read as a query tile, the key tiles that add to its dQ are the group's tiles [0, npc) and
 * [dep_lo, own index] (group-relative indices).
 * *num_tiles receives their count (at most pp_plan_max_tiles).  Synchronises `stream`. */
int pp_plan_read_bwd_tiles(const pp_plan* plan, pp_stream_t stream, int32_t* num_tiles,
                           int32_t* btiles);
/* Backward processing order: max_tiles * Hkv records (kv_head << 24) | backward tile, of which
 * the first num_bwd_tiles * Hkv are valid.  Units of one group are adjacent (they stream the
 * same Q / dO tiles through L2), groups with the most work first.  Synchronises `stream`. */
int pp_plan_read_bwd_units(const pp_plan* plan, pp_stream_t stream, int32_t* units);
int pp_plan_read(const pp_plan* plan, pp_stream_t stream, int32_t* num_tiles, int32_t* tiles,
                 int32_t* fwd_order, int32_t* bwd_order, int32_t* key_end);

/*
 * Forward (Sec. 3.2): O = softmax(mask(scale * Q K^T)) V and LSE, per row and query head.
 * q, k, v, o: bf16 device pointers; lse: fp32 device pointer.  The forward itself needs no
 * scratch: d_scratch may be NULL.  Training callers may pass the buffer they are going to give
 * pp_attn_bwd as its scratch (256-byte aligned, at least the backward size reported by
 * pp_plan_workspace_bytes; PP_ERR_WORKSPACE_TOO_SMALL / PP_ERR_ALIGNMENT otherwise): the
 * forward then also clears the fp32 dQ accumulator inside it (when that accumulator,
 * 4 * T * Hq * D bytes, is at most 640 MiB -- beyond that the library leaves the clearing to
 * the backward, which measured faster), and the next pp_attn_bwd on this plan with the same
 * buffer (later on the same stream) skips its own clearing pass.  The buffer must not be used
 * for anything else in between.
 */
int pp_attn_fwd(const pp_plan* plan, const void* q, const void* k, const void* v,
                float softmax_scale, void* o, float* lse, void* d_scratch, size_t scratch_bytes,
                pp_stream_t stream);

/*
 * Backward of the same operation (training is the paper's use case, Sec. 4-5): given dO,
 * the forward's O and LSE, writes dQ, dK, dV (bf16).  Prompt keys receive contributions from
 * the prompt's own queries and from every response's queries; dK and dV are summed over the
 * query heads that share a KV head.  dQ is accumulated in fp32 inside d_scratch and rounded
 * once at the end.
 */
int pp_attn_bwd(const pp_plan* plan, const void* q, const void* k, const void* v, const void* o,
                const float* lse, const void* d_o, float softmax_scale, void* d_q, void* d_k,
                void* d_v, void* d_scratch, size_t scratch_bytes, pp_stream_t stream);

/*
 * The same backward with a bit-reproducible dQ (the paper does not discuss reproducibility;
 * Sec. 3.2's equivalence to unpacked training is what a reproducible gradient lets a user
 * verify run against run).  pp_attn_bwd adds the per-key-tile contributions to a query tile's
 * dQ in whatever order the CTAs reach it, so dQ can differ in the last bits between runs; here
 * the key tiles of a group take turns in descending tile order -- the order in which the units,
 * each walking its query tiles upwards from its own tile, reach a query tile anyway -- (one
 * counter per query tile and head inside d_scratch; units handed out one (group, KV head) set
 * after the other and in descending tile order inside a set, so that no CTA waits for work
 * that has not started).  dK, dV and the forward are reproducible in both variants.
 * Same arguments, sizes and errors as pp_attn_bwd; a turn that does not come within a bounded
 * number of polls sets the plan's status word (PP_ERR_PLAN_STATUS from pp_plan_status).
 */
int pp_attn_bwd_deterministic(const pp_plan* plan, const void* q, const void* k, const void* v,
                              const void* o, const float* lse, const void* d_o,
                              float softmax_scale, void* d_q, void* d_k, void* d_v,
                              void* d_scratch, size_t scratch_bytes, pp_stream_t stream);

/*
 * The step right before attention (Sec. 3.2: every token keeps the position it has in its own
 * unpacked sequence).  pp_position_ids writes, per token, the position it would have
 * in its own unpacked sequence (x, y^k): index inside the prompt for prompt tokens, P + index
 * inside the response for response tokens -- positions restart after the prompt for every
 * response.  pp_rope_qk applies the rotary embedding (rotate-half form, angle = position *
 * rope_base^(-2i/D)) with those positions to Q [T][Hq][D] and K [T][Hkv][D] in place (bf16
 * device pointers); V is untouched.  Both need only the plan (any plan built for the same
 * descriptors) and run on `stream`.  position_ids: int32 device pointer, [T].
 */
int pp_position_ids(const pp_plan* plan, int32_t* position_ids, pp_stream_t stream);
int pp_rope_qk(const pp_plan* plan, void* q, void* k, float rope_base, pp_stream_t stream);

/*
 * The step right after the model forward (Sec. 2.1): splits the packed rows back into their
 * responses and evaluates the preference loss.  token_logp [T] (fp32, device) holds the
 * log-probability of each token under the policy; prompt entries are ignored.  Per response
 * k: resp_logp = sum of its tokens' log-probs; resp_reward = beta * (resp_logp - the same sum
 * of ref_token_logp), or beta * resp_logp when ref_token_logp is NULL.  Responses are ranked as
 * in Sec. 3.1 (response a preferred over b for a > b); grp_loss[g] = mean over the pairs a > b
 * of -log sigmoid(r_a - r_b) (0 for a single-response group).  d_token_logp [T] (may be NULL)
 * receives d(sum_g grp_loss[g]) / d token_logp.  resp_logp, resp_reward: [N]; grp_loss: [G].
 */
int pp_preference_loss(const pp_plan* plan, const float* token_logp, const float* ref_token_logp,
                       float beta, float* resp_logp, float* resp_reward, float* grp_loss,
                       float* d_token_logp, pp_stream_t stream);

/*
 * pp_attn_bwd for callers that cannot allocate device memory.  (The paper has no counterpart:
 * this is a packaging variant of the backward above, not a different computation.)
 *
 * Some callers have no way to hand the library a scratch buffer: an extension loaded into a
 * host application that owns the whole device heap and gives plug-ins none of it, a step
 * running after every byte has been committed to other tenants, or a latency-critical loop
 * in which cudaMalloc / cudaFree are forbidden because they may synchronise the device.  For
 * them the backward's scratch (fp32 dQ accumulator, Delta, scaled LSE) lives in an array that
 * is part of the library image.  This entry point calls no cudaMalloc, cudaFree or other
 * allocating routine; the caller still passes every input and output tensor.
 *
 *  - Limit: the scratch pp_plan_workspace_bytes reports for the plan's problem must not exceed
 *    pp_attn_bwd_noalloc_max_bytes (32 MiB, i.e. about T * Hq * D <= 8.2 M elements);
 *    larger problems are rejected with PP_ERR_STATIC_SCRATCH_LIMIT and nothing is launched.
 *  - Cost: every GPU on which the library is loaded holds those 32 MiB until the process exits.
 *  - The array used is the one on the device that holds the plan's workspace, and that device
 *    must be the current device at the call (PP_ERR_INVALID_ARG otherwise: another device's
 *    array is never handed to the kernels).  The first call on each device looks up the
 *    array's device address.  Make that first call before any stream capture begins.
 *  - All calls on a device share the one array, and it keeps the previous call's contents.
 *    Each call clears the part that must start at zero (the dQ accumulator) and rewrites
 *    the rest, so back-to-back calls on ONE stream are safe; calls that can overlap on the
 *    GPU (different streams, different host threads without ordering) race on it and give
 *    wrong gradients.
 * Results, layouts and the other errors are those of pp_attn_bwd.
 */
int pp_attn_bwd_noalloc_max_bytes(size_t* bytes);
int pp_attn_bwd_noalloc(const pp_plan* plan, const void* q, const void* k, const void* v,
                        const void* o, const float* lse, const void* d_o, float softmax_scale,
                        void* d_q, void* d_k, void* d_v, pp_stream_t stream);

/* Kernel launches enqueued by the last pp_build_plan / pp_attn_fwd / pp_attn_bwd /
 * pp_attn_bwd_noalloc / pp_attn_step_host call of this thread. */
int pp_last_launch_count(void);

/*
 * One whole pass of the hot path on HOST buffers: copies Q, K, V, dO to the device, builds
 * the plan from the host descriptors, runs forward and backward, and copies O, LSE, dQ, dK,
 * dV back; the caller synchronises `stream` before reading the outputs.  Groups never interact
 * (paper section 3), so the pass is cut into up to eight runs of whole groups with about equal
 * token counts (fewer when a run would hold under a quarter MiB of input), each with its own plan, and pipelined: the kernels run on `stream`, all
 * uploads on one side stream of the library and all downloads on another (both created once
 * per device), so that the inputs of the next run go up and the results of the previous run
 * come down, in opposite directions, while the kernels of the current run execute.  `stream`
 * is made to wait for both side streams: once `stream` has completed, everything has.  The
 * results are those of one pp_attn_fwd + pp_attn_bwd over the whole problem (dK, dV, O and
 * LSE bit for bit).  Host buffers should be page-locked for the copies to be asynchronous.
 * d_arena is caller-owned device memory of at least pp_step_host_arena_bytes (256-byte
 * aligned); it holds the device copies, the plan workspaces and the backward scratch.
 * `problem` must have desc_on_device == 0; its descriptors are validated on the host first.
 * All calls on one device share the two side streams and their events: make them from one
 * host thread at a time.  Same layouts and errors as the calls above.
 */
int pp_step_host_arena_bytes(const pp_problem* problem, size_t* arena_bytes);
/* The runs pp_attn_step_host cuts `problem` into (host only, no device work): run c holds
 * groups [group_begin[c], group_begin[c+1]) = tokens [token_begin[c], token_begin[c+1]).
 * Both arrays must hold 9 entries. */
int pp_step_host_runs(const pp_problem* problem, int32_t* num_runs, int32_t* group_begin,
                      int32_t* token_begin);
int pp_attn_step_host(const pp_problem* problem, const void* h_q, const void* h_k, const void* h_v,
                      const void* h_do, float softmax_scale, void* h_o, float* h_lse, void* h_dq,
                      void* h_dk, void* h_dv, void* d_arena, size_t arena_bytes,
                      pp_stream_t stream);

/*
 * Kernel timing for benchmarks.  pp_profile_enable(1) makes pp_attn_fwd / pp_attn_bwd record
 * CUDA events on the caller's stream directly around the forward kernel and around the
 * backward main kernel; pp_profile_enable(2) only around the backward main kernel (every
 * event between two kernels keeps the second from being queued behind the first, about 5 us
 * each on a sub-millisecond step).  pp_profile_read returns the durations (ms) of the most
 * recent calls once that stream has been synchronised by the caller (PP_ERR_CUDA otherwise;
 * pass NULL for a duration that is not being recorded).  On a capturing stream the records
 * become nodes of the graph and mark the events at every replay.
 * pp_profile_enable(0) releases the events.  One set of events per process, created on the
 * device that is current at pp_profile_enable(1): profile one device at a time.
 */
int pp_profile_enable(int on);
int pp_profile_read(float* fwd_kernel_ms, float* bwd_main_kernel_ms);
/*
 * The same for many calls at once: the event pairs form a ring of 64 per kernel, so a benchmark
 * can run its timed steps without a synchronisation in between and read the durations (ms,
 * oldest first, at most `capacity` and at most 64 of the most recent launches since the last
 * pp_profile_enable) after synchronising the stream once.  HOST arrays; either may be NULL;
 * *num_fwd / *num_bwd receive how many entries were written.  PP_ERR_CUDA if profiling is off
 * or an event has not completed.  Calling pp_profile_enable again while profiling is on
 * restarts the counts.
 */
int pp_profile_read_all(float* fwd_kernel_ms, float* bwd_main_kernel_ms, int32_t capacity,
                        int32_t* num_fwd, int32_t* num_bwd);

/*
 * Row builder: the step before the attention path (batch sorting and batch packing, Sec. 2.2;
 * applied together with preference packing in Sec. 5.2, Table 2).  Groups [prompt | responses]
 * are ordered by total length, longest first and ties in their original order (batch sorting),
 * and consecutive groups of that order are concatenated into rows of at most row_capacity
 * tokens (batch packing; next fit).  All pointers are DEVICE pointers; everything runs on
 * `stream`.
 *   in : grp_prompt_len [G], grp_resp_off [G + 1], resp_len [N]        (int32, as in pp_problem)
 *   out: order [G]            original index of the group at each position of the new order
 *        row_group_off [G + 1], num_rows [1]   positions [off[r], off[r + 1]) form row r
 *        row_tokens [G], row_cost [G]          (int64) tokens and visible query-key pairs per
 *                                              row (Sec. 3.2.1's attention cost)
 *        out_prompt_len [G], out_resp_off [G + 1], out_resp_len [N]   descriptors in row order:
 *                                              with row_group_off they are a pp_problem
 *        status [2]            0 = fine; 1 = malformed group, 2 = a group alone exceeds the
 *                              capacity (then num_rows = 0); status[1] = the group
 * d_workspace: pp_build_rows_workspace_bytes(G) bytes, 256-byte aligned.  G <= 65536.
 * Errors: PP_ERR_INVALID_ARG, PP_ERR_UNSUPPORTED (G too large), PP_ERR_WORKSPACE_TOO_SMALL,
 * PP_ERR_ALIGNMENT, PP_ERR_CUDA; the device status is for the caller to read.
 */
int pp_build_rows_workspace_bytes(int32_t num_groups, size_t* bytes);
int pp_build_rows(int32_t num_groups, int32_t num_responses, const int32_t* grp_prompt_len,
                  const int32_t* grp_resp_off, const int32_t* resp_len, int32_t row_capacity,
                  void* d_workspace, size_t workspace_bytes, int32_t* order,
                  int32_t* row_group_off, int32_t* num_rows, int64_t* row_tokens,
                  int64_t* row_cost, int32_t* out_prompt_len, int32_t* out_resp_off,
                  int32_t* out_resp_len, int32_t* status, pp_stream_t stream);

/*
 * Rows -> data-parallel ranks (Sec. 2.2: batch sorting exists so that no rank waits for the
 * one with the longest sequences; Sec. 5.2, Table 2, the run with sorting and packing both).
 * Longest-processing-time assignment by attention cost: rows are taken in order of decreasing
 * row_cost (ties: lower index first) and each goes to the rank whose cost so far is least
 * (ties: lowest rank).  Every rank's total then stays within (mean + largest row cost).
 * All pointers are DEVICE pointers; two small kernels on `stream`; nothing is allocated.
 *   in : row_cost [num_rows] (int64; pp_build_rows' row_cost, or any non-negative cost)
 *   out: order [num_rows]        rows in the order they were assigned
 *        rank_of_row [num_rows]  rank that processes each row
 *        rank_cost [num_ranks]   (int64) total cost per rank
 * num_rows <= 65536, num_ranks <= 1024 (PP_ERR_UNSUPPORTED beyond); PP_ERR_INVALID_ARG,
 * PP_ERR_CUDA.  The ranks themselves exchange nothing: each computes the same assignment from
 * the same costs and processes its own rows.
 */
int pp_assign_rows(int32_t num_rows, const int64_t* row_cost, int32_t num_ranks, int32_t* order,
                   int32_t* rank_of_row, int64_t* rank_cost, pp_stream_t stream);

/*
 * Test hook for the bounded waits (no counterpart in the paper).  Every wait inside the
 * kernels polls a bounded number of times and then records kStatusWaitExpired (3) with the
 * wait's site id in the plan's status word instead of spinning on.  This call runs that same
 * wait routine in a one-thread kernel on a barrier nobody arrives at, with a limit of 4096
 * polls and with no copy or MMA in flight, so the give-up path can be checked on a GPU without
 * hanging anything: afterwards pp_plan_status reports status 3 / detail `site`, and the
 * kernels of later calls on this plan return at once.  site >= 1.
 */
int pp_debug_expire_wait(const pp_plan* plan, int32_t site, pp_stream_t stream);

const char* pp_error_string(int code);

#ifdef __cplusplus
}
#endif
#endif /* PP_ATTN_H_ */
