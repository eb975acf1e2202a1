// C ABI of the D3ToM merge-layer library: context, host helpers, argument
// validation and dispatch to the kernels.  See include/d3tom.h for the contract.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <new>

#include "common.cuh"

int g_d3tom_launch_overlap = 1;
int g_d3tom_pair_tiles = -1;
int g_d3tom_single_tile_attention = -1;

namespace {

// D3TOM_LOG=1 in the environment: one line per call on stderr (sizes and the status returned).  Read once.
bool log_enabled() {
  static const int on = [] { const char* e = getenv("D3TOM_LOG"); return (e != nullptr && e[0] != '\0' && e[0] != '0') ? 1 : 0; }();
  return on != 0;
}
int logged(int status, const char* fmt, ...) {
  if (log_enabled()) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof(buf), fmt, ap);
    va_end(ap);
    fprintf(stderr, "[d3tom] %s -> %d (%s)\n", buf, status, d3tom_status_string(status));
  }
  return status;
}

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
  }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

template <typename T>
int alloc(d3tom_ctx* ctx, T** p, size_t count) {
  const size_t bytes = (count > 0 ? count : 1) * sizeof(T);
  D3TOM_CUDA_TRY(ctx, cudaMalloc(reinterpret_cast<void**>(p), bytes));
  ctx->bytes += (int64_t)bytes;
  return D3TOM_OK;
}

void free_all(d3tom_ctx* c) {
  cudaFree(c->score_scratch); cudaFree(c->lse_scratch); cudaFree(c->imp_partial); cudaFree(c->imp_counters);
  cudaFree(c->inv_norm);
  cudaFree(c->inv_norm_kept); cudaFree(c->kept_rows); cudaFree(c->best); cudaFree(c->member_off);
  cudaFree(c->member_cursor); cudaFree(c->member_list); cudaFree(c->heavy_slots); cudaFree(c->n_heavy); cudaFree(c->row_desc); cudaFree(c->agg_counter);
  cudaFree(c->gemm_split_ws); cudaFree(c->gemm_split_counters); cudaFree(c->dev_status);
  cudaFree(c->attn_part_ws); cudaFree(c->attn_part_flags);
}

bool dtype_ok(d3tom_dtype dt) { return dt == D3TOM_BF16 || dt == D3TOM_FP32; }

// bf16 on tensor cores needs dh in {64, 128}; the CUDA-core kernels take dh % 4 == 0, dh <= 128
int check_head_dim(const d3tom_ctx* ctx, d3tom_dtype dt) {
  const int dh = ctx->lim.head_dim;
  if (dt == D3TOM_BF16 && !ctx->reference_kernels) return (dh == 64 || dh == 128) ? D3TOM_OK : D3TOM_ERR_UNSUPPORTED;
  return (dh % 4 == 0 && dh >= 4 && dh <= 128) ? D3TOM_OK : D3TOM_ERR_UNSUPPORTED;
}

}  // namespace

extern "C" {

static int create_impl(d3tom_ctx** out, int device, const d3tom_limits* lim);

int d3tom_create(d3tom_ctx** out, int device, const d3tom_limits* lim) {
  const int st = create_impl(out, device, lim);
  if (lim == nullptr) return logged(st, "d3tom_create device %d", device);
  return logged(st, "d3tom_create device %d: tokens %d batch %d heads %d x %d deciders %d visual %d, scratch %lld bytes", device,
                lim->max_total_tokens, lim->max_batch, lim->heads, lim->head_dim, lim->max_deciders,
                lim->max_visual_per_request, (long long)((st == D3TOM_OK && out && *out) ? (*out)->bytes : 0));
}

static int create_impl(d3tom_ctx** out, int device, const d3tom_limits* lim) {
  if (out == nullptr || lim == nullptr) return D3TOM_ERR_INVALID_ARG;
  *out = nullptr;
  if (lim->max_total_tokens <= 0 || lim->max_batch <= 0 || lim->heads <= 0 || lim->head_dim <= 0 ||
      lim->max_deciders < 0 || lim->max_visual_per_request <= 0)
    return D3TOM_ERR_INVALID_ARG;
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || device < 0 || device >= n_dev) return D3TOM_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return D3TOM_ERR_CUDA;
  if (prop.major != 10) return D3TOM_ERR_UNSUPPORTED;     // kernels are built for sm_100a only
  DeviceGuard guard(device);
  if (!guard.ok) return D3TOM_ERR_CUDA;
  d3tom_ctx* c = new (std::nothrow) d3tom_ctx();
  if (c == nullptr) return D3TOM_ERR_INVALID_ARG;
  c->device = device;
  c->lim = *lim;
  c->sm_count = prop.multiProcessorCount;
  c->vis_stride = (lim->max_visual_per_request + 3) & ~3;
  const size_t T = (size_t)lim->max_total_tokens, H = (size_t)lim->heads, D = H * lim->head_dim;
  const size_t nd = (size_t)(lim->max_deciders > 0 ? lim->max_deciders : 1);
  int st = D3TOM_OK;
  if (st == D3TOM_OK) st = alloc(c, &c->score_scratch, H * nd * c->vis_stride);
  if (st == D3TOM_OK) st = alloc(c, &c->lse_scratch, H * nd);
  if (st == D3TOM_OK) st = alloc(c, &c->imp_partial, H * T);
  const size_t n_ctr = (size_t)lim->max_batch * (((size_t)lim->max_visual_per_request + 255) / 256);
  if (st == D3TOM_OK) st = alloc(c, &c->imp_counters, n_ctr);
  if (st == D3TOM_OK && cudaMemset(c->imp_counters, 0, n_ctr * sizeof(int)) != cudaSuccess) st = D3TOM_ERR_CUDA;
  if (st == D3TOM_OK) st = alloc(c, &c->inv_norm, T);
  if (st == D3TOM_OK) st = alloc(c, &c->inv_norm_kept, T);
  if (st == D3TOM_OK) st = alloc(c, reinterpret_cast<char**>(&c->kept_rows), T * D * sizeof(float));
  if (st == D3TOM_OK) st = alloc(c, &c->best, T);
  if (st == D3TOM_OK) st = alloc(c, &c->member_off, T + 1);
  if (st == D3TOM_OK) st = alloc(c, &c->member_cursor, T);
  if (st == D3TOM_OK) st = alloc(c, &c->member_list, T);
  if (st == D3TOM_OK) st = alloc(c, &c->heavy_slots, T / 32 + 1);
  if (st == D3TOM_OK) st = alloc(c, &c->n_heavy, 1);
  if (st == D3TOM_OK) st = alloc(c, &c->row_desc, T);
  if (st == D3TOM_OK) st = alloc(c, &c->agg_counter, 2);
  if (st == D3TOM_OK && cudaMemset(c->agg_counter, 0, 2 * sizeof(int)) != cudaSuccess) st = D3TOM_ERR_CUDA;
  if (st == D3TOM_OK) st = alloc(c, &c->gemm_split_ws, (size_t)2 * c->sm_count * 128 * 256);
  if (st == D3TOM_OK) st = alloc(c, &c->gemm_split_counters, (size_t)2 * c->sm_count);
  if (st == D3TOM_OK && cudaMemset(c->gemm_split_counters, 0, 2 * c->sm_count * sizeof(int)) != cudaSuccess) st = D3TOM_ERR_CUDA;
  if (st == D3TOM_OK) st = alloc(c, &c->attn_part_ws, (size_t)c->sm_count * 2 * (128 + 2) * 128);
  if (st == D3TOM_OK) st = alloc(c, &c->attn_part_flags, (size_t)c->sm_count * 8);
  if (st == D3TOM_OK && cudaMemset(c->attn_part_flags, 0, (size_t)c->sm_count * 8 * sizeof(int)) != cudaSuccess) st = D3TOM_ERR_CUDA;
  if (st == D3TOM_OK) st = alloc(c, &c->dev_status, 1);
  if (st == D3TOM_OK && cudaMemset(c->dev_status, 0, sizeof(int)) != cudaSuccess) st = D3TOM_ERR_CUDA;
  if (st != D3TOM_OK) { free_all(c); delete c; return st; }
  *out = c;
  return D3TOM_OK;
}

int d3tom_destroy(d3tom_ctx* ctx) {
  if (ctx == nullptr) return D3TOM_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  free_all(ctx);
  delete ctx;
  return D3TOM_OK;
}

const char* d3tom_status_string(int status) {
  switch (status) {
    case D3TOM_OK: return "ok";
    case D3TOM_ERR_INVALID_ARG: return "invalid argument";
    case D3TOM_ERR_UNSUPPORTED: return "unsupported dtype, head_dim, size or device";
    case D3TOM_ERR_WORKSPACE: return "request exceeds the limits the context was created with";
    case D3TOM_ERR_CUDA: return "CUDA call failed";
    case D3TOM_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out";
    default: return "unknown status";
  }
}

int d3tom_last_cuda_error(const d3tom_ctx* ctx) { return ctx ? ctx->last_cuda_error : 0; }

int d3tom_device_status(d3tom_ctx* ctx, int* status_out) {
  if (ctx == nullptr || status_out == nullptr) return D3TOM_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  D3TOM_CUDA_TRY(ctx, cudaDeviceSynchronize());
  D3TOM_CUDA_TRY(ctx, cudaMemcpy(status_out, ctx->dev_status, sizeof(int), cudaMemcpyDeviceToHost));
  return D3TOM_OK;
}

int d3tom_reset_device_status(d3tom_ctx* ctx) {
  if (ctx == nullptr) return D3TOM_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  D3TOM_CUDA_TRY(ctx, cudaDeviceSynchronize());
  D3TOM_CUDA_TRY(ctx, cudaMemset(ctx->dev_status, 0, sizeof(int)));
  // a kernel that gave up may have left its self-cleaning counters and flags behind: back to their resting state
  const size_t n_ctr = (size_t)ctx->lim.max_batch * (((size_t)ctx->lim.max_visual_per_request + 255) / 256);
  D3TOM_CUDA_TRY(ctx, cudaMemset(ctx->imp_counters, 0, n_ctr * sizeof(int)));
  D3TOM_CUDA_TRY(ctx, cudaMemset(ctx->agg_counter, 0, 2 * sizeof(int)));
  D3TOM_CUDA_TRY(ctx, cudaMemset(ctx->gemm_split_counters, 0, (size_t)2 * ctx->sm_count * sizeof(int)));
  D3TOM_CUDA_TRY(ctx, cudaMemset(ctx->attn_part_flags, 0, (size_t)ctx->sm_count * 8 * sizeof(int)));
  return D3TOM_OK;
}

int d3tom_selftest_wait_timeout(d3tom_ctx* ctx, int64_t limit_ns, d3tom_stream stream) {
  if (ctx == nullptr || limit_ns <= 0 || limit_ns > 1000000000ll) return D3TOM_ERR_INVALID_ARG;   // at most one second
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return D3TOM_ERR_CUDA;
  return launch_wait_timeout_selftest(ctx, (long long)limit_ns, static_cast<cudaStream_t>(stream));
}

int64_t d3tom_workspace_bytes(const d3tom_ctx* ctx) { return ctx ? ctx->bytes : 0; }

int d3tom_set_reference_kernels(d3tom_ctx* ctx, int on) {
  if (ctx == nullptr) return D3TOM_ERR_INVALID_ARG;
  ctx->reference_kernels = on ? 1 : 0;
  return D3TOM_OK;
}

int d3tom_set_launch_overlap(int on) {
  g_d3tom_launch_overlap = on ? 1 : 0;
  return D3TOM_OK;
}

int d3tom_set_single_tile_attention(int mode) {
  if (mode < -1 || mode > 1) return D3TOM_ERR_INVALID_ARG;
  g_d3tom_single_tile_attention = mode;
  return D3TOM_OK;
}

int d3tom_set_pair_tiles(int width) {
  if (width != -1 && width != 0 && width != 256) return D3TOM_ERR_INVALID_ARG;
  g_d3tom_pair_tiles = width;
  return D3TOM_OK;
}

int d3tom_keep_count(int n_visual, double keep_ratio) {
  if (n_visual <= 0) return 0;
  double k = floor(keep_ratio * (double)n_visual + 1e-9);
  if (k < 1.0) k = 1.0;
  if (k > (double)n_visual) k = (double)n_visual;
  return (int)k;
}

int d3tom_schedule_alpha(int step, int T, double a_min, double a_max, int reversed, double* alpha_out) {
  if (alpha_out == nullptr || T <= 0 || step < 0 || step >= T) return D3TOM_ERR_INVALID_ARG;
  double frac = 0.0;            // a single step runs at a_min in either direction
  if (T > 1) {
    frac = (double)step / (double)(T - 1);
    if (reversed) frac = 1.0 - frac;
  }
  *alpha_out = a_min + (a_max - a_min) * frac;
  return D3TOM_OK;
}

static int attn_common(d3tom_ctx* ctx, d3tom_dtype dt, const void* q, const void* k, const void* v,
                       const int32_t* cu_seqlens, const int32_t* n_visual, const int32_t* decider_pos,
                       const int32_t* cu_deciders, int B, int total_tokens, int max_seqlen, int max_visual,
                       int n_deciders_total, float softmax_scale, void* out, float* importance,
                       const int32_t* cu_vis, bool with_importance, cudaStream_t stream) {
  if (ctx == nullptr) return D3TOM_ERR_INVALID_ARG;
  if (!dtype_ok(dt)) return D3TOM_ERR_UNSUPPORTED;
  if (q == nullptr || k == nullptr || v == nullptr || cu_seqlens == nullptr || out == nullptr) return D3TOM_ERR_INVALID_ARG;
  if (B <= 0 || total_tokens < 0 || max_seqlen < 0 || max_seqlen > total_tokens || !(softmax_scale > 0.f))
    return D3TOM_ERR_INVALID_ARG;
  if (with_importance) {
    if (n_visual == nullptr || cu_deciders == nullptr || importance == nullptr || cu_vis == nullptr ||
        n_deciders_total < 0 || max_visual < 0 || max_visual > max_seqlen)
      return D3TOM_ERR_INVALID_ARG;
    if (n_deciders_total > 0 && decider_pos == nullptr) return D3TOM_ERR_INVALID_ARG;
    if (n_deciders_total > ctx->lim.max_deciders || max_visual > ctx->lim.max_visual_per_request)
      return D3TOM_ERR_WORKSPACE;
  }
  if (B > ctx->lim.max_batch || total_tokens > ctx->lim.max_total_tokens) return D3TOM_ERR_WORKSPACE;
  int st = check_head_dim(ctx, dt);
  if (st != D3TOM_OK) return st;
  if (total_tokens == 0 || max_seqlen == 0) return D3TOM_OK;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return D3TOM_ERR_CUDA;
  AttnArgs a;
  a.q = q; a.k = k; a.v = v; a.out = out;
  a.cu_seqlens = cu_seqlens; a.n_visual = n_visual;
  a.decider_pos = with_importance ? decider_pos : nullptr;
  a.cu_deciders = with_importance ? cu_deciders : nullptr;
  if (with_importance && n_deciders_total == 0) a.decider_pos = nullptr;
  a.B = B; a.H = ctx->lim.heads; a.dh = ctx->lim.head_dim; a.total_tokens = total_tokens; a.max_seqlen = max_seqlen;
  a.scale_log2 = softmax_scale * 1.4426950408889634f;
  a.score_scratch = ctx->score_scratch; a.lse_scratch = ctx->lse_scratch;
  a.max_deciders = ctx->lim.max_deciders > 0 ? ctx->lim.max_deciders : 1; a.vis_stride = ctx->vis_stride;
  a.dev_status = ctx->dev_status;
  if (dt == D3TOM_BF16 && !ctx->reference_kernels) {
    st = D3TOM_ERR_UNSUPPORTED;
    if (g_d3tom_single_tile_attention == 1) st = launch_attn_one(ctx, a, stream);   // one query tile per CTA
    if (st == D3TOM_ERR_UNSUPPORTED) st = launch_attn_sk(ctx, a, stream);   // one request whose items do not fill whole rounds of SMs
    if (st == D3TOM_ERR_UNSUPPORTED) st = launch_attn_tc(ctx, a, stream);
  } else {
    st = launch_attn_simt(ctx, dt, a, stream);
  }
  if (st != D3TOM_OK) return st;
  if (with_importance) {
    a.cu_deciders = cu_deciders;
    st = launch_importance_finish(ctx, a, max_visual, importance, cu_vis, stream);
  }
  return st;
}

int d3tom_attn_importance(d3tom_ctx* ctx, d3tom_dtype dt, const void* q, const void* k, const void* v,
                          const int32_t* cu_seqlens, const int32_t* n_visual, const int32_t* decider_pos,
                          const int32_t* cu_deciders, int B, int total_tokens, int max_seqlen, int max_visual,
                          int n_deciders_total, float softmax_scale, void* attn_out, float* importance,
                          const int32_t* cu_vis, d3tom_stream stream) {
  return logged(attn_common(ctx, dt, q, k, v, cu_seqlens, n_visual, decider_pos, cu_deciders, B, total_tokens, max_seqlen,
                            max_visual, n_deciders_total, softmax_scale, attn_out, importance, cu_vis, true,
                            static_cast<cudaStream_t>(stream)),
                "d3tom_attn_importance dt %d B %d tokens %d max_seqlen %d max_visual %d deciders %d", (int)dt, B, total_tokens,
                max_seqlen, max_visual, n_deciders_total);
}

int d3tom_attn_varlen(d3tom_ctx* ctx, d3tom_dtype dt, const void* q, const void* k, const void* v,
                      const int32_t* cu_seqlens, int B, int total_tokens, int max_seqlen, float softmax_scale,
                      void* out, d3tom_stream stream) {
  return logged(attn_common(ctx, dt, q, k, v, cu_seqlens, nullptr, nullptr, nullptr, B, total_tokens, max_seqlen, 0, 0,
                            softmax_scale, out, nullptr, nullptr, false, static_cast<cudaStream_t>(stream)),
                "d3tom_attn_varlen dt %d B %d tokens %d max_seqlen %d", (int)dt, B, total_tokens, max_seqlen);
}

static int select_impl(d3tom_ctx* ctx, const float* importance, const int32_t* cu_vis, const int32_t* keep_count,
                       const int32_t* cu_kept, int B, int max_visual, int32_t* kept_idx, uint8_t* keep_mask,
                       d3tom_stream stream);

int d3tom_select(d3tom_ctx* ctx, const float* importance, const int32_t* cu_vis, const int32_t* keep_count,
                 const int32_t* cu_kept, int B, int max_visual, int32_t* kept_idx, uint8_t* keep_mask,
                 d3tom_stream stream) {
  return logged(select_impl(ctx, importance, cu_vis, keep_count, cu_kept, B, max_visual, kept_idx, keep_mask, stream),
                "d3tom_select B %d max_visual %d", B, max_visual);
}

static int select_impl(d3tom_ctx* ctx, const float* importance, const int32_t* cu_vis, const int32_t* keep_count,
                       const int32_t* cu_kept, int B, int max_visual, int32_t* kept_idx, uint8_t* keep_mask,
                       d3tom_stream stream) {
  if (ctx == nullptr || importance == nullptr || cu_vis == nullptr || keep_count == nullptr || cu_kept == nullptr ||
      kept_idx == nullptr || keep_mask == nullptr || B <= 0 || max_visual < 0)
    return D3TOM_ERR_INVALID_ARG;
  if (B > ctx->lim.max_batch || max_visual > ctx->lim.max_total_tokens) return D3TOM_ERR_WORKSPACE;
  if (max_visual == 0) return D3TOM_OK;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return D3TOM_ERR_CUDA;
  return launch_select(ctx, importance, cu_vis, keep_count, cu_kept, B, max_visual, kept_idx, keep_mask,
                       static_cast<cudaStream_t>(stream));
}

static int merge_common(d3tom_ctx* ctx, d3tom_dtype dt, d3tom_agg mode, const void* hidden, const void* second,
                        const int32_t* cu_seqlens, const int32_t* n_visual, const int32_t* cu_vis,
                        const int32_t* kept_idx, const int32_t* cu_kept, int B, int D, int total_tokens, int total_out,
                        int max_visual, int max_kept, void* hidden_out, void* second_out,
                        const int32_t* cu_seqlens_out, int32_t* assign, int32_t* member_count, int32_t* src_of_dst,
                        float* sim_debug, cudaStream_t s) {
  if (ctx == nullptr) return D3TOM_ERR_INVALID_ARG;
  if (!dtype_ok(dt)) return D3TOM_ERR_UNSUPPORTED;
  if (mode != D3TOM_AGG_SUM && mode != D3TOM_AGG_MEAN) return D3TOM_ERR_INVALID_ARG;
  if (hidden == nullptr || cu_seqlens == nullptr || n_visual == nullptr || cu_vis == nullptr || kept_idx == nullptr ||
      cu_kept == nullptr || hidden_out == nullptr || cu_seqlens_out == nullptr || assign == nullptr ||
      member_count == nullptr || src_of_dst == nullptr || (second == nullptr) != (second_out == nullptr))
    return D3TOM_ERR_INVALID_ARG;
  if (B <= 0 || D <= 0 || total_tokens < 0 || total_out < 0 || total_out > total_tokens || max_visual < 0 ||
      max_kept < 0 || max_kept > max_visual || max_visual > total_tokens)
    return D3TOM_ERR_INVALID_ARG;
  if (D != ctx->lim.heads * ctx->lim.head_dim) return D3TOM_ERR_INVALID_ARG;
  if (D % 8 != 0) return D3TOM_ERR_UNSUPPORTED;
  if (B > ctx->lim.max_batch || total_tokens > ctx->lim.max_total_tokens) return D3TOM_ERR_WORKSPACE;
  if (total_tokens == 0) return D3TOM_OK;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return D3TOM_ERR_CUDA;
  MergeArgs a;
  a.dt = dt; a.mode = mode; a.hidden = hidden; a.cu_seqlens = cu_seqlens; a.n_visual = n_visual; a.cu_vis = cu_vis;
  a.kept_idx = kept_idx; a.cu_kept = cu_kept; a.B = B; a.D = D; a.total_tokens = total_tokens; a.total_out = total_out;
  a.max_visual = max_visual; a.max_kept = max_kept; a.hidden_out = hidden_out; a.cu_seqlens_out = cu_seqlens_out;
  a.assign = assign; a.member_count = member_count; a.src_of_dst = src_of_dst; a.sim_debug = sim_debug;
  int st = D3TOM_OK;
  if (max_visual > 0) {
    st = launch_merge_prepare(ctx, a, s);
    if (st != D3TOM_OK) return st;
    if (total_out < total_tokens) {   // otherwise nothing is pruned anywhere
      if (dt == D3TOM_BF16 && !ctx->reference_kernels) st = launch_sim_tc(ctx, a, s);
      else st = launch_sim_simt(ctx, a, s);
      if (st != D3TOM_OK) return st;
    }
  }
  st = launch_merge_finish(ctx, a, s);
  if (st != D3TOM_OK || second == nullptr) return st;
  a.hidden = second; a.hidden_out = second_out;       // same routing, second payload
  return launch_merge_aggregate(ctx, a, s);
}

int d3tom_merge(d3tom_ctx* ctx, d3tom_dtype dt, d3tom_agg mode, const void* hidden, const int32_t* cu_seqlens,
                const int32_t* n_visual, const int32_t* cu_vis, const int32_t* kept_idx, const int32_t* cu_kept,
                int B, int D, int total_tokens, int total_out, int max_visual, int max_kept, void* hidden_out,
                const int32_t* cu_seqlens_out, int32_t* assign, int32_t* member_count, int32_t* src_of_dst,
                float* sim_debug, d3tom_stream stream) {
  return logged(merge_common(ctx, dt, mode, hidden, nullptr, cu_seqlens, n_visual, cu_vis, kept_idx, cu_kept, B, D,
                             total_tokens, total_out, max_visual, max_kept, hidden_out, nullptr, cu_seqlens_out, assign,
                             member_count, src_of_dst, sim_debug, static_cast<cudaStream_t>(stream)),
                "d3tom_merge dt %d mode %d B %d D %d tokens %d -> %d max_visual %d max_kept %d", (int)dt, (int)mode, B, D,
                total_tokens, total_out, max_visual, max_kept);
}

int d3tom_merge_kv(d3tom_ctx* ctx, d3tom_dtype dt, d3tom_agg mode, const void* k_cache, const void* v_cache,
                   const int32_t* cu_seqlens, const int32_t* n_visual, const int32_t* cu_vis, const int32_t* kept_idx,
                   const int32_t* cu_kept, int B, int D, int total_tokens, int total_out, int max_visual, int max_kept,
                   void* k_out, void* v_out, const int32_t* cu_seqlens_out, int32_t* assign, int32_t* member_count,
                   int32_t* src_of_dst, float* sim_debug, d3tom_stream stream) {
  if (v_cache == nullptr || v_out == nullptr) return D3TOM_ERR_INVALID_ARG;
  return merge_common(ctx, dt, mode, k_cache, v_cache, cu_seqlens, n_visual, cu_vis, kept_idx, cu_kept, B, D,
                      total_tokens, total_out, max_visual, max_kept, k_out, v_out, cu_seqlens_out, assign,
                      member_count, src_of_dst, sim_debug, static_cast<cudaStream_t>(stream));
}

int d3tom_proj_qkv(d3tom_ctx* ctx, d3tom_dtype dt, const void* x, const void* w_qkv, int total, int D, void* q,
                   void* k, void* v, d3tom_stream stream) {
  if (ctx == nullptr) return D3TOM_ERR_INVALID_ARG;
  if (!dtype_ok(dt)) return D3TOM_ERR_UNSUPPORTED;
  if (x == nullptr || w_qkv == nullptr || q == nullptr || k == nullptr || v == nullptr || total < 0 || D <= 0)
    return D3TOM_ERR_INVALID_ARG;
  if (total > ctx->lim.max_total_tokens) return D3TOM_ERR_WORKSPACE;
  if (total == 0) return D3TOM_OK;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return D3TOM_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (dt == D3TOM_BF16 && !ctx->reference_kernels) {
    if (D % 64 != 0) return D3TOM_ERR_UNSUPPORTED;
    return launch_proj_tc(ctx, x, w_qkv, total, D, q, k, v, s);
  }
  return launch_proj_simt(ctx, dt, x, w_qkv, total, D, q, k, v, s);
}

int d3tom_linear(d3tom_ctx* ctx, d3tom_dtype dt, const void* x, const void* w, const void* residual, int rows, int K,
                 int N, void* out, d3tom_stream stream) {
  if (ctx == nullptr) return D3TOM_ERR_INVALID_ARG;
  if (dt != D3TOM_FP32 && dt != D3TOM_BF16) return D3TOM_ERR_UNSUPPORTED;
  if (x == nullptr || w == nullptr || out == nullptr || rows < 0 || K <= 0 || N <= 0 || x == out)
    return D3TOM_ERR_INVALID_ARG;
  if (rows == 0) return D3TOM_OK;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return D3TOM_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (dt == D3TOM_BF16 && !ctx->reference_kernels) return launch_linear_tc(ctx, x, w, residual, rows, K, N, out, s);
  return launch_linear_simt(ctx, dt, x, w, residual, rows, K, N, out, s);
}

int d3tom_ffn(d3tom_ctx* ctx, d3tom_dtype dt, const void* x, const void* w_gate_up, const void* w_down,
              const void* residual, int rows, int D, int m, void* act, void* out, d3tom_stream stream) {
  if (ctx == nullptr) return D3TOM_ERR_INVALID_ARG;
  if (dt != D3TOM_FP32 && dt != D3TOM_BF16) return D3TOM_ERR_UNSUPPORTED;
  if (x == nullptr || w_gate_up == nullptr || w_down == nullptr || act == nullptr || out == nullptr || rows < 0 ||
      D <= 0 || m <= 0 || act == out || act == x || act == residual)
    return D3TOM_ERR_INVALID_ARG;
  if (rows == 0) return D3TOM_OK;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return D3TOM_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (dt == D3TOM_BF16 && !ctx->reference_kernels) {
    if (D % 128 != 0 || m % 128 != 0) return D3TOM_ERR_UNSUPPORTED;   // checked before anything is launched
    const int st = launch_gate_up_tc(ctx, x, w_gate_up, rows, D, m, act, s);
    if (st != D3TOM_OK) return st;
    return launch_linear_tc(ctx, act, w_down, residual, rows, m, D, out, s);
  }
  const int st = launch_gate_up_simt(ctx, dt, x, w_gate_up, rows, D, m, act, s);
  if (st != D3TOM_OK) return st;
  return launch_linear_simt(ctx, dt, act, w_down, residual, rows, m, D, out, s);
}

}  // extern "C"
