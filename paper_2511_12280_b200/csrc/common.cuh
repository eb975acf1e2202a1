// Shared declarations of the D3ToM merge-layer library (host + device).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/d3tom.h"

struct d3tom_ctx {
  int device;
  d3tom_limits lim;
  int sm_count;
  int last_cuda_error;
  int reference_kernels;        // 1: bf16 also runs on the CUDA-core kernels (debugging aid)
  int64_t bytes;
  // ---- scratch (device), sized at create ----
  float* score_scratch;         // [H][max_deciders][vis_stride] raw q.k of decider rows x visual keys
  float2* lse_scratch;          // [H][max_deciders] (M, l): l = sum_j exp2(s_j*c - M)
  float* imp_partial;           // [H][max_total_tokens] per-head importance
  int* imp_counters;            // [max_batch][ceil(max_visual / 256)] blocks done per key range; zero between calls
  float* inv_norm;              // [max_total_tokens] 1/|h| of visual rows (packed by cu_vis)
  float* inv_norm_kept;         // [max_total_tokens] the same for kept rows, packed by cu_kept
  void* kept_rows;              // [max_total_tokens, D] gathered kept rows (B operand of the similarity GEMM)
  unsigned long long* best;     // [max_total_tokens] packed (similarity, ~slot) running maximum
  int32_t* member_off;          // [max_total_tokens + 1] start of each kept slot's member list
  int32_t* member_cursor;       // [max_total_tokens]
  int32_t* member_list;         // [max_total_tokens] pruned positions grouped by destination slot
  int32_t* heavy_slots;         // [max_total_tokens / 32 + 1] kept tokens with 32 members or more
  int* n_heavy;                 // how many of them
  int* agg_counter;             // [2] work and exit counters of the streaming aggregation; the kernel leaves them at zero
  int4* row_desc;               // [max_total_tokens] per output row: {source row, members or -1, list offset, request start}
  float* gemm_split_ws;         // [2 * sm_count][256][128] fp32 partial similarity tiles (K slices of a tile)
  int* gemm_split_counters;     // [2 * sm_count] slices done per tile; zero between launches
  float* attn_part_ws;          // [sm_count][2][128 + 2][128] fp32: O tile and (m, l) of an attention item's later key tiles
  int* attn_part_flags;         // [sm_count][2][4] one word per (CTA, query tile, warp); zero between launches
  int* dev_status;              // device status word
  int vis_stride;               // row stride of score_scratch (floats)
};

#define D3TOM_CUDA_TRY(ctx, expr)                      \
  do {                                                 \
    cudaError_t e__ = (expr);                          \
    if (e__ != cudaSuccess) {                          \
      (ctx)->last_cuda_error = (int)e__;               \
      return D3TOM_ERR_CUDA;                           \
    }                                                  \
  } while (0)

#define D3TOM_LAUNCH_CHECK(ctx) D3TOM_CUDA_TRY(ctx, cudaGetLastError())

static inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// ------------------------------------------------------------------ device helpers
#ifdef __CUDACC__

// Every kernel of the library is launched with programmatic stream serialization: its CTAs may become resident while
// the kernel before it in the stream is still draining, which hides the launch latency between the many short
// kernels of a step.  A kernel therefore opens with grid_dependency_enter(), BEFORE it touches global memory: it waits
// until every earlier kernel has completed and its writes are visible, and only then lets the next kernel's CTAs be
// scheduled (releasing before the wait let several kernels ahead pile up as waiting CTAs; measured no faster).
// A kernel with on-chip set-up that needs no global memory does that set-up before the wait.
__device__ __forceinline__ void grid_dependency_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_enter() {
  grid_dependency_wait();
  grid_dependency_release();
}

// Process-wide switch behind d3tom_set_launch_overlap (1 = overlap, the default).
extern int g_d3tom_launch_overlap;
extern int g_d3tom_single_tile_attention;   // -1 chosen per launch, 0 never, 1 wherever the kernel supports the launch
extern int g_d3tom_pair_tiles;      // dense layers on CTA pairs: -1 chosen per shape, 0 never, 256 wherever the shape allows

template <typename... Params, typename... Args>
inline cudaError_t launch_serialized(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                     Args&&... args) {
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = g_d3tom_launch_overlap ? 1 : 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<Params>(args)...);
}

// largest b in [0, B) with cu[b] <= idx  (cu ascending, cu[0] = 0)
__device__ __forceinline__ int find_segment(const int32_t* __restrict__ cu, int B, int idx) {
  int lo = 0, hi = B;   // invariant: cu[lo] <= idx < cu[hi]
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (cu[mid] <= idx) lo = mid; else hi = mid;
  }
  return lo;
}

// total order on floats as unsigned integers (larger float -> larger key)
__device__ __forceinline__ uint32_t ordered_key(float f) {
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

template <typename T> struct Storage;
template <> struct Storage<float> {
  static constexpr int kVec = 4;   // elements per 16 bytes
  __device__ static __forceinline__ void load(const float* p, float (&f)[4]) {
    float4 v = *reinterpret_cast<const float4*>(p);
    f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
  }
  __device__ static __forceinline__ void store(float* p, const float (&f)[4]) {
    *reinterpret_cast<float4*>(p) = make_float4(f[0], f[1], f[2], f[3]);
  }
  __device__ static __forceinline__ float to_float(float x) { return x; }
  __device__ static __forceinline__ float from_float(float x) { return x; }
};
template <> struct Storage<__nv_bfloat16> {
  static constexpr int kVec = 8;
  __device__ static __forceinline__ void load(const __nv_bfloat16* p, float (&f)[8]) {
    uint4 v = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  __device__ static __forceinline__ void store(__nv_bfloat16* p, const float (&f)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
      w[i] = *reinterpret_cast<uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
  }
  __device__ static __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
  __device__ static __forceinline__ __nv_bfloat16 from_float(float x) { return __float2bfloat16_rn(x); }
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
#endif  // __CUDACC__

// ------------------------------------------------------------------ launchers (defined in the .cu files)
struct AttnArgs {
  const void* q; const void* k; const void* v; void* out;
  const int32_t* cu_seqlens; const int32_t* n_visual;
  const int32_t* decider_pos; const int32_t* cu_deciders;   // null when no importance is wanted
  int B, H, dh, total_tokens, max_seqlen;
  float scale_log2;             // softmax_scale * log2(e)
  float* score_scratch; float2* lse_scratch; int max_deciders; int vis_stride;
  int* dev_status;
  int nqb, split_from;          // tensor-core kernel only, set by its launcher: 256-row blocks per request, first cut item
};

int launch_attn_simt(d3tom_ctx* ctx, d3tom_dtype dt, const AttnArgs& a, cudaStream_t s);
int launch_attn_tc(d3tom_ctx* ctx, const AttnArgs& a, cudaStream_t s);
int launch_attn_sk(d3tom_ctx* ctx, const AttnArgs& a, cudaStream_t s);      // one request, work balanced over the SMs
int launch_attn_one(d3tom_ctx* ctx, const AttnArgs& a, cudaStream_t s);     // one query tile per CTA, three score buffers
int launch_importance_finish(d3tom_ctx* ctx, const AttnArgs& a, int max_visual, float* importance,
                             const int32_t* cu_vis, cudaStream_t s);
int launch_select(d3tom_ctx* ctx, const float* importance, const int32_t* cu_vis, const int32_t* keep_count,
                  const int32_t* cu_kept, int B, int max_visual, int32_t* kept_idx, uint8_t* keep_mask,
                  cudaStream_t s);

struct MergeArgs {
  d3tom_dtype dt; d3tom_agg mode;
  const void* hidden; const int32_t* cu_seqlens; const int32_t* n_visual; const int32_t* cu_vis;
  const int32_t* kept_idx; const int32_t* cu_kept;
  int B, D, total_tokens, total_out, max_visual, max_kept;
  void* hidden_out; const int32_t* cu_seqlens_out;
  int32_t* assign; int32_t* member_count; int32_t* src_of_dst; float* sim_debug;
};
int launch_merge_prepare(d3tom_ctx* ctx, const MergeArgs& a, cudaStream_t s);     // slots, norms, kept-row gather
int launch_sim_simt(d3tom_ctx* ctx, const MergeArgs& a, cudaStream_t s);          // similarity + argmax, CUDA cores
int launch_sim_tc(d3tom_ctx* ctx, const MergeArgs& a, cudaStream_t s);            // similarity + argmax, tcgen05
int launch_merge_finish(d3tom_ctx* ctx, const MergeArgs& a, cudaStream_t s);      // members, aggregate, compact
int launch_merge_aggregate(d3tom_ctx* ctx, const MergeArgs& a, cudaStream_t s);   // aggregate, compact (lists already built)
int launch_merge_aggregate_stream(d3tom_ctx* ctx, const MergeArgs& a, cudaStream_t s);   // the same as a bulk-copy pipeline

int launch_wait_timeout_selftest(d3tom_ctx* ctx, long long limit_ns, cudaStream_t s);   // a wait that cannot end

int launch_proj_simt(d3tom_ctx* ctx, d3tom_dtype dt, const void* x, const void* w, int total, int D,
                     void* q, void* k, void* v, cudaStream_t s);
int launch_proj_tc(d3tom_ctx* ctx, const void* x, const void* w, int total, int D,
                   void* q, void* k, void* v, cudaStream_t s);
// y = residual + x w^T and act = silu(x Wg^T) * (x Wu^T): the rest of a block (output projection, feed-forward network)
int launch_linear_tc(d3tom_ctx* ctx, const void* x, const void* w, const void* residual, int rows, int K, int N,
                     void* out, cudaStream_t s);
int launch_gate_up_tc(d3tom_ctx* ctx, const void* x, const void* w_gate_up, int rows, int D, int m, void* act,
                      cudaStream_t s);
int launch_linear_simt(d3tom_ctx* ctx, d3tom_dtype dt, const void* x, const void* w, const void* residual, int rows,
                       int K, int N, void* out, cudaStream_t s);
int launch_gate_up_simt(d3tom_ctx* ctx, d3tom_dtype dt, const void* x, const void* w_gate_up, int rows, int D, int m,
                        void* act, cudaStream_t s);
