/*
 * d3tom.h -- C ABI of the D3ToM merge-layer library for NVIDIA B200 (sm_100a).
 *
 * The library implements the merge-layer work of ONE denoising step of a
 * diffusion multimodal LLM with decider-guided token merging:
 *
 *   d3tom_attn_importance   bidirectional self-attention at the merge layer l*
 *                           + the decider->visual importance map, one pass
 *   d3tom_select            keep / merge partition by rank of the importance
 *   d3tom_merge             nearest-kept-neighbour routing by cosine similarity,
 *                           aggregation, physical removal of the merged rows
 *   d3tom_attn_varlen       bidirectional attention over the shortened sequences
 *   d3tom_merge_kv          the same routing applied to a cached K/V prefix
 *   d3tom_proj_qkv          (supporting) Q,K,V projection of a post-merge layer
 *   d3tom_linear, d3tom_ffn (supporting) output projection and gated feed-forward
 *                           network of a post-merge block
 *
 * Conventions shared by every call
 * --------------------------------
 *  - A batch holds B requests packed back to back.  Request b is the
 *    concatenation [visual | prompt | response] (Algorithm 1, Embed(Concat(V,P,X)))
 *    and occupies packed rows [cu_seqlens[b], cu_seqlens[b+1]); its first
 *    n_visual[b] rows are the visual tokens.
 *  - Activations are row-major [rows, H, dh] == [rows, D], D = H*dh, in the
 *    storage type `dt` (bf16 or fp32).
 *  - Unless a parameter says "host", every pointer is DEVICE memory owned by
 *    the caller and valid on the context's device.  The library never
 *    allocates, frees or resizes caller buffers, never synchronises the
 *    stream and never changes the current device; all work is enqueued on
 *    `stream` and is complete when the stream reaches that point.
 *  - Scratch memory lives in the context and is sized once, at
 *    d3tom_create, from d3tom_limits.  A call that needs more returns
 *    D3TOM_ERR_WORKSPACE; nothing is reallocated.  Two calls on the same
 *    context must not overlap on the GPU (use one context per stream).
 *  - Every function returns a status: D3TOM_OK (0) or a negative error.  No
 *    exceptions, no abort, nothing printed (unless the environment variable
 *    D3TOM_LOG is set to something other than 0: then d3tom_create and the four
 *    calls of the path write one line per call, sizes and status, to stderr).  Argument errors are detected on
 *    the host before anything is launched.  Problems only the device can see
 *    (a bounded wait that ran out) are recorded in a status word read by
 *    d3tom_device_status.
 *  - bf16 runs on the tcgen05 tensor-core kernels and needs head_dim 64 or
 *    128; fp32 runs on plain CUDA-core kernels (any head_dim that is a
 *    multiple of 4 up to 128).  There is no CPU fallback.
 */
#ifndef D3TOM_H_
#define D3TOM_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct d3tom_ctx d3tom_ctx;          /* opaque; owns scratch only */
typedef void* d3tom_stream;                  /* a cudaStream_t */

typedef enum { D3TOM_BF16 = 0, D3TOM_FP32 = 1 } d3tom_dtype;
typedef enum { D3TOM_AGG_SUM = 0, D3TOM_AGG_MEAN = 1 } d3tom_agg;

enum {
  D3TOM_OK = 0,
  D3TOM_ERR_INVALID_ARG = -1,   /* null pointer, negative size, inconsistent sizes */
  D3TOM_ERR_UNSUPPORTED = -2,   /* dtype / head_dim / device architecture not supported */
  D3TOM_ERR_WORKSPACE   = -3,   /* request exceeds the limits given at d3tom_create */
  D3TOM_ERR_CUDA        = -4,   /* a CUDA runtime / driver call failed (see d3tom_last_cuda_error) */
  D3TOM_ERR_TIMEOUT     = -5    /* device status: a bounded wait inside a kernel ran out */
};

typedef struct {
  int max_total_tokens;        /* packed rows over the whole batch */
  int max_batch;               /* requests per call */
  int heads;                   /* H */
  int head_dim;                /* dh */
  int max_deciders;            /* decider tokens over the whole batch */
  int max_visual_per_request;  /* largest n_visual[b] */
} d3tom_limits;

/* Create a context on CUDA device `device` (must be sm_100) and allocate its
 * scratch.  Returns D3TOM_ERR_UNSUPPORTED on any other architecture. */
int d3tom_create(d3tom_ctx** out, int device, const d3tom_limits* lim);
int d3tom_destroy(d3tom_ctx* ctx);
const char* d3tom_status_string(int status);
/* cudaError_t / CUresult of the last failing CUDA call on this context (0 if none). */
int d3tom_last_cuda_error(const d3tom_ctx* ctx);
/* Copies the device-side status word to *status_out (host).  Synchronises the
 * device; call it after the stream work of interest has been waited for. */
int d3tom_device_status(d3tom_ctx* ctx, int* status_out);
/* Sets the device-side status word back to 0 (synchronises the device first) and
 * returns the counters and flags that kernels leave at zero between launches to that
 * state: call it after D3TOM_ERR_TIMEOUT was reported, before the context is used again. */
int d3tom_reset_device_status(d3tom_ctx* ctx);
/* Self-test of the bounded waits.  Every wait inside the library's kernels (on a
 * barrier that a copy, the tensor pipe or another warp completes) gives up after a
 * time limit, records D3TOM_ERR_TIMEOUT in the status word and lets the kernel release
 * what it holds and return, so that a wait that cannot end costs that limit and not a
 * hung GPU.  This call enqueues a one-block kernel that waits, with the same routine
 * and a limit of `limit_ns` (1 .. 10^9), on a barrier that nothing completes: after the
 * stream has been waited for, d3tom_device_status reports D3TOM_ERR_TIMEOUT and the
 * context is usable as before (clear the word with d3tom_reset_device_status).
 * The kernel issues no copy and no tensor-core instruction and faults nothing. */
int d3tom_selftest_wait_timeout(d3tom_ctx* ctx, int64_t limit_ns, d3tom_stream stream);
/* Bytes of scratch the context holds (host query). */
int64_t d3tom_workspace_bytes(const d3tom_ctx* ctx);

/* Debugging aid: with on != 0, bf16 calls also run on the plain CUDA-core
 * kernels that serve fp32 (slow; lets the two code paths be compared on the GPU). */
int d3tom_set_reference_kernels(d3tom_ctx* ctx, int on);

/* Profiling aid, process-wide.  By default every kernel of the library is launched so
 * that its thread blocks may become resident while the kernel before it in the stream
 * drains (programmatic dependent launch; each kernel still waits for its predecessor's
 * results before it reads them).  A profiler then attributes that waiting to the later
 * kernel.  With on == 0 kernels start only after their predecessor has finished, so
 * per-kernel device times are separable (and a step is a little slower); results are
 * the same either way.  Not thread-safe against concurrent launches. */
int d3tom_set_launch_overlap(int on);

/* Tile shape of the dense layers (d3tom_proj_qkv, d3tom_linear, d3tom_ffn; Sec. 3.2.1 "Q = H W_Q", Algorithm 1
 * FFN_l): -1 (default) lets the library choose per shape (pairs from about two thousand rows on), 0 keeps single-CTA
 * tiles, 256 forces tiles of 256 x 256 computed by a pair of CTAs (cta_group::2) wherever the number of output columns
 * is a multiple of 256.  Results do not depend on the choice: every output is one fp32 accumulator over K in
 * ascending order, rounded once.  Process-wide; not thread-safe against concurrent launches.
 * Returns D3TOM_ERR_INVALID_ARG for other values. */
int d3tom_set_pair_tiles(int width);

/* Which tensor-core attention kernel serves d3tom_attn_varlen / d3tom_attn_importance (Sec. 3.2.1): -1 (default) the
 * library's choice per launch, 0 the kernels with two query tiles per CTA, 1 the kernel with one query tile per CTA and
 * three score buffers wherever it supports the launch (bf16, head_dim 128, no importance side-work).  Results agree
 * within the attention tolerance (different summation orders of the row sum).  Process-wide; not thread-safe against
 * concurrent launches.  Returns D3TOM_ERR_INVALID_ARG for other values. */
int d3tom_set_single_tile_attention(int mode);

/* Sec. 3.2.1, "Rank(S_j) <= (1-alpha)|V|": number of kept tokens for keep
 * ratio r = 1-alpha.  Host arithmetic: clamp(floor(r*n_visual + 1e-9), 1, n_visual). */
int d3tom_keep_count(int n_visual, double keep_ratio);

/* Sec. 3.2.3, linear schedule: alpha at decode-order step `step` in 0..T-1 is
 * a_min + (a_max - a_min) * step/(T-1) (smallest at the beginning of decoding);
 * `reversed` != 0 gives the high->low ablation.  Host arithmetic. */
int d3tom_schedule_alpha(int step, int T, double a_min, double a_max, int reversed, double* alpha_out);

/* Sec. 3.2.1 (self-attention matrix A and decider score S_j); Algorithm 1,
 * SelfAttn_l and the line S_j <- sum_{i in D} A_ij.
 *
 * Per request and head: O = softmax(Q K^T * softmax_scale) V over ALL keys of
 * the request (no mask).  In the same pass, for every visual key j,
 *   importance[cu_vis[b] + j] = sum over heads, sum over decider rows i of A_ij.
 *
 *  q, k, v       [total, H, dh] storage type
 *  cu_seqlens    [B+1] int32, n_visual [B] int32
 *  decider_pos   [cu_deciders[B]] int32: decider rows relative to the request
 *                start, strictly ascending per request
 *  cu_deciders   [B+1] int32.  A request with no deciders gets importance 0.
 *  n_deciders_total  == cu_deciders[B] (host copy, sizes the scratch use)
 *  total_tokens  == cu_seqlens[B]; max_seqlen >= every request length;
 *  max_visual >= every n_visual[b] (host copies)
 *  attn_out      [total, H*dh] storage type (the post-attention states H~)
 *  importance    [cu_vis[B]] fp32, cu_vis [B+1] int32
 * The importance is reduced in a fixed order: results are run-to-run identical. */
int d3tom_attn_importance(d3tom_ctx* ctx, d3tom_dtype dt,
                          const void* q, const void* k, const void* v,
                          const int32_t* cu_seqlens, const int32_t* n_visual,
                          const int32_t* decider_pos, const int32_t* cu_deciders,
                          int B, int total_tokens, int max_seqlen, int max_visual, int n_deciders_total,
                          float softmax_scale,
                          void* attn_out, float* importance, const int32_t* cu_vis,
                          d3tom_stream stream);

/* Allocation-free variant of d3tom_attn_importance.  The paper has no
 * counterpart: this exists for hosts that must not allocate device memory
 * (a process whose memory pool owns the whole device, a sandbox that registers
 * every allocation up front, a latency-critical loop that must stay off the
 * allocator's device-wide lock) and therefore cannot call d3tom_create.
 *
 * It needs no context.  The scratch that the context would own lives in a
 * fixed array inside the library image: about 10.1 MiB that every GPU
 * loading the library holds until the process exits.  That array bounds the
 * problem size; a call beyond any of
 *     heads * max(1, n_deciders_total)                       <= D3TOM_STATIC_MAX_LSE_PAIRS
 *     heads * total_tokens                                   <= D3TOM_STATIC_MAX_PARTIAL_FLOATS
 *     heads * max(1, n_deciders_total) * round_up(max_visual, 4) <= D3TOM_STATIC_MAX_SCORE_FLOATS
 * (or with B * ceil(max_visual / 256) > 4096) returns D3TOM_ERR_WORKSPACE and
 * launches nothing (e.g. 32 heads x 16 deciders x 4096 visual tokens, 16384
 * packed tokens, fits exactly).
 *
 * heads, head_dim replace the context's limits; every other argument is as in
 * d3tom_attn_importance.  The results are those of d3tom_attn_importance to
 * rounding: bit for bit where that call runs the same whole-item kernel, within
 * the tolerances of the parity tests where it balances a single request's work
 * items over the SMs (that path keeps partial tiles in context scratch, which
 * this entry point does not have).  The work
 * runs on the CURRENT device, which must be the one `stream` and the buffers
 * belong to.  device_status_out (device, nullable) receives the kernels'
 * status word at the end of the call (0, or D3TOM_ERR_TIMEOUT if a bounded
 * wait ran out); read it after the stream has been waited for.
 *
 * The first call on each device looks up the array's device address; make
 * that first call outside of any stream capture.  No call allocates or frees.
 * All calls on a device share the one array, and it keeps what the previous
 * call left there (this function clears the few words that have to start at
 * zero): two calls that overlap on the GPU race with each other, so keep all
 * calls of a device on one stream or order them with events. */
#define D3TOM_STATIC_MAX_LSE_PAIRS      (1 << 14)
#define D3TOM_STATIC_MAX_PARTIAL_FLOATS (1 << 19)
#define D3TOM_STATIC_MAX_SCORE_FLOATS   (1 << 21)
int d3tom_attn_importance_static(d3tom_dtype dt, int heads, int head_dim,
                                 const void* q, const void* k, const void* v,
                                 const int32_t* cu_seqlens, const int32_t* n_visual,
                                 const int32_t* decider_pos, const int32_t* cu_deciders,
                                 int B, int total_tokens, int max_seqlen, int max_visual, int n_deciders_total,
                                 float softmax_scale,
                                 void* attn_out, float* importance, const int32_t* cu_vis,
                                 int32_t* device_status_out, d3tom_stream stream);

/* Sec. 3.2.1, the partition V_kept / V_merge; Algorithm 1, TopK.
 *
 * Per request: the keep_count[b] visual tokens of highest importance, ordered by
 * (score descending, index ascending) on the fp32 bit pattern, emitted
 * ASCENDING by position.
 *  importance  [cu_vis[B]] fp32 (finite, >= 0)
 *  keep_count  [B] int32, 1 <= keep_count[b] <= n_visual[b]
 *  cu_kept     [B+1] int32, prefix sum of keep_count
 *  kept_idx    [cu_kept[B]] int32 out: positions relative to the request start
 *  keep_mask   [cu_vis[B]] uint8 out: 1 = kept, 0 = merged away
 *  max_visual  host: >= every n_visual[b] */
int d3tom_select(d3tom_ctx* ctx, const float* importance, const int32_t* cu_vis,
                 const int32_t* keep_count, const int32_t* cu_kept, int B, int max_visual,
                 int32_t* kept_idx, uint8_t* keep_mask, d3tom_stream stream);

/* Sec. 3.2.2 (similarity-based merging); Algorithm 1, the loop over V_merge
 * and the removal of the merged positions.
 *
 * For every pruned visual token m: k* = argmax over the request's kept tokens
 * of cos(h~_m, h~_k), cosines taken on the PRE-merge states in fp32
 * (dot * (1/|h_m|) * (1/|h_k|), zero-norm rows give 0), ties to the lowest kept
 * position.  Then out_k = h~_k + sum of its members (SUM, the paper's
 * equation) or that divided by 1 + members (MEAN), accumulated in fp32 in
 * ascending member order and rounded once.  The output sequence of request b
 * is [merged kept visual rows, ascending position | prompt | response].
 *
 *  hidden          [total_tokens, D] storage type
 *  kept_idx/cu_kept  from d3tom_select
 *  total_out       host: sum over b of N_b - n_visual[b] + k_b  (== cu_seqlens_out[B])
 *  max_visual, max_kept  host: >= every n_visual[b] / keep count
 *  hidden_out      [total_out, D] out
 *  cu_seqlens_out  [B+1] int32 in: prefix sum of the shortened lengths (host-computed by the caller)
 *  assign          [cu_vis[B]] int32 out: destination slot (rank in the kept list) of every visual token
 *  member_count    [cu_kept[B]] int32 out: pruned tokens routed to each kept token
 *  src_of_dst      [total_out] int32 out: original packed row of every output row
 *  sim_debug       nullable; [cu_vis[B], max_kept] fp32 out: entry (cu_vis[b]+m, s) is the
 *                  cosine of pruned token m with the kept token of slot s, exactly the
 *                  value the argmax compared; rows of kept tokens are not written */
int d3tom_merge(d3tom_ctx* ctx, d3tom_dtype dt, d3tom_agg mode,
                const void* hidden, const int32_t* cu_seqlens, const int32_t* n_visual, const int32_t* cu_vis,
                const int32_t* kept_idx, const int32_t* cu_kept,
                int B, int D, int total_tokens, int total_out, int max_visual, int max_kept,
                void* hidden_out, const int32_t* cu_seqlens_out,
                int32_t* assign, int32_t* member_count, int32_t* src_of_dst,
                float* sim_debug, d3tom_stream stream);

/* Sec. 4.4 (Compatibility with KV-Cache): the same merge applied to a cached prefix.
 *
 * k_cache, v_cache [total_tokens, D] hold, per request, the cached keys and values of its
 * [visual | prompt] prefix (cu_seqlens gives the prefix lengths, n_visual the visual part).
 * With the kept set K from d3tom_select and its complement M: every m in M is routed to
 * pi(m) = argmax over k in K of cos(K_m, K_k) (full-width rows, pre-merge values, ties to
 * the lowest kept position); then K_pi(m) += K_m and V_pi(m) += V_m (SUM, the paper's
 * equations; MEAN divides both by 1 + members, one reading of "renormalise"), and the
 * positions in M are dropped: k_out, v_out [total_out, D] are the shorter caches, rows
 * ordered as in d3tom_merge.  Every other argument is as in d3tom_merge; assign,
 * member_count and src_of_dst describe the routing shared by both tensors. */
int d3tom_merge_kv(d3tom_ctx* ctx, d3tom_dtype dt, d3tom_agg mode,
                   const void* k_cache, const void* v_cache,
                   const int32_t* cu_seqlens, const int32_t* n_visual, const int32_t* cu_vis,
                   const int32_t* kept_idx, const int32_t* cu_kept,
                   int B, int D, int total_tokens, int total_out, int max_visual, int max_kept,
                   void* k_out, void* v_out, const int32_t* cu_seqlens_out,
                   int32_t* assign, int32_t* member_count, int32_t* src_of_dst,
                   float* sim_debug, d3tom_stream stream);

/* Sec. 3.2.2, last paragraph: the layers after l* run on the shortened tensor.
 * Same attention as d3tom_attn_importance, over packed ragged sequences, with
 * no importance output. */
int d3tom_attn_varlen(d3tom_ctx* ctx, d3tom_dtype dt,
                      const void* q, const void* k, const void* v,
                      const int32_t* cu_seqlens, int B, int total_tokens, int max_seqlen,
                      float softmax_scale, void* out, d3tom_stream stream);

/* Sec. 3.2.1, Q = H W_Q, K = H W_K (and V): the projection feeding a
 * post-merge layer.  x [total, D]; w_qkv [3D, D] row-major, row o holds the
 * weights of output feature o (rows 0..D-1 -> Q, D..2D-1 -> K, 2D..3D-1 -> V);
 * q, k, v [total, D] out, fp32 accumulation, one rounding to the storage type. */
int d3tom_proj_qkv(d3tom_ctx* ctx, d3tom_dtype dt, const void* x, const void* w_qkv,
                   int total, int D, void* q, void* k, void* v, d3tom_stream stream);

/* Algorithm 1, H <- FFN_l(H^), and the layer-cost equation of the FLOPs appendix
 * (4 n d^2 for four d x d projections, 3 n d m for the feed-forward network): the
 * rest of a Transformer block, run on the shortened sequence after the merge.
 * The paper does not write the block out; this library takes the gated form the
 * three d x m matrices imply and no normalisation layers.
 *
 * d3tom_linear: out = residual + x w^T, fp32 accumulation, one rounding to the
 * storage type.  x [rows, K]; w [N, K] row-major, row o holds the weights of
 * output feature o; residual [rows, N] or NULL; out [rows, N].  With K = N = D
 * this is the attention output projection.  out may be the residual buffer itself
 * (in-place add) but not x.  All pointers are device memory, caller-owned.
 * bf16 on the tensor-core path needs K % 64 == 0 and N % 128 == 0
 * (D3TOM_ERR_UNSUPPORTED otherwise); fp32 has no such limit. */
int d3tom_linear(d3tom_ctx* ctx, d3tom_dtype dt, const void* x, const void* w, const void* residual,
                 int rows, int K, int N, void* out, d3tom_stream stream);

/* d3tom_ffn: act = silu(x Wg^T) * (x Wu^T), rounded to the storage type, then
 * out = residual + act Wd^T.  x [rows, D]; w_gate_up [2m, D]: rows 0..m-1 are
 * Wg, rows m..2m-1 are Wu; w_down [D, m]; residual [rows, D] or NULL;
 * act [rows, m] is scratch the caller provides (device memory; holds the
 * activation afterwards); out [rows, D], may be the residual buffer.  Two kernel
 * launches: the gate and up products share one pass whose epilogue applies
 * silu(gate) * up, so neither product is written out.  bf16 on the tensor-core
 * path needs D % 128 == 0 and m % 128 == 0. */
int d3tom_ffn(d3tom_ctx* ctx, d3tom_dtype dt, const void* x, const void* w_gate_up, const void* w_down,
              const void* residual, int rows, int D, int m, void* act, void* out, d3tom_stream stream);

#ifdef __cplusplus
}
#endif
#endif /* D3TOM_H_ */
