// Similarity-based merging (Sec. 3.2.2; Algorithm 1, the loop over V_merge and
// the removal of the merged positions), everything except the tensor-core
// similarity kernel:
//
//   prepare   slot of every kept token, 1/|h| of every visual row, and a packed
//             copy of the kept rows (the second operand of the similarity)
//   sim_simt  cosine + arg-max on CUDA cores (fp32 storage, debugging aid)
//   finish    destination slots, per-slot member lists, aggregation in
//             ascending member order and compaction into the shortened sequence
//
// The arg-max is a 64-bit maximum over (order-preserving similarity bits << 32
// | ~slot): the largest similarity wins and, among equals, the lowest slot, no
// matter in which order candidates arrive.
#include "common.cuh"

namespace {

// ---------------------------------------------------------------- prepare
__global__ void __launch_bounds__(256)
init_slots_kernel(const int32_t* __restrict__ cu_vis, int B, int32_t* __restrict__ assign,
                  unsigned long long* __restrict__ best) {
  const int g = blockIdx.x * blockDim.x + threadIdx.x;
  if (g >= cu_vis[B]) return;
  assign[g] = -1;
  best[g] = 0ull;
}

__global__ void __launch_bounds__(256)
scatter_slots_kernel(const int32_t* __restrict__ kept_idx, const int32_t* __restrict__ cu_kept,
                     const int32_t* __restrict__ cu_vis, int B, int32_t* __restrict__ assign) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= cu_kept[B]) return;
  const int b = find_segment(cu_kept, B, i);
  assign[cu_vis[b] + kept_idx[i]] = i - cu_kept[b];
}

// one block per visual row: inverse norm; kept rows are also copied to their slot
template <typename T>
__global__ void __launch_bounds__(128)
rownorm_gather_kernel(const T* __restrict__ hidden, const int32_t* __restrict__ cu_seqlens,
                      const int32_t* __restrict__ cu_vis, const int32_t* __restrict__ cu_kept,
                      const int32_t* __restrict__ assign, int D, float* __restrict__ inv_norm,
                      float* __restrict__ inv_norm_kept, T* __restrict__ kept_rows) {
  constexpr int kVec = Storage<T>::kVec;
  const int b = blockIdx.y, m = blockIdx.x;
  const int v0 = cu_vis[b];
  if (m >= cu_vis[b + 1] - v0) return;
  const int g = v0 + m;
  const T* src = hidden + (size_t)(cu_seqlens[b] + m) * D;
  const int slot = assign[g];
  T* dst = slot >= 0 ? kept_rows + (size_t)(cu_kept[b] + slot) * D : nullptr;
  float ss = 0.f;
  for (int c = threadIdx.x * kVec; c < D; c += blockDim.x * kVec) {
    float f[kVec];
    Storage<T>::load(src + c, f);
#pragma unroll
    for (int i = 0; i < kVec; ++i) ss = fmaf(f[i], f[i], ss);
    if (dst != nullptr) Storage<T>::store(dst + c, f);
  }
  __shared__ float red[4];
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  if (threadIdx.x == 0) {
    const float tot = (red[0] + red[1]) + (red[2] + red[3]);
    const float inv = tot > 0.f ? 1.0f / sqrtf(tot) : 0.f;
    inv_norm[g] = inv;
    if (slot >= 0) inv_norm_kept[cu_kept[b] + slot] = inv;
  }
}

// ---------------------------------------------------------------- similarity on CUDA cores
// one block per pruned row; warp w scores slots w, w+8, ...
template <typename T>
__global__ void __launch_bounds__(256)
sim_simt_kernel(const T* __restrict__ hidden, const T* __restrict__ kept_rows,
                const int32_t* __restrict__ cu_seqlens, const int32_t* __restrict__ cu_vis,
                const int32_t* __restrict__ cu_kept, const int32_t* __restrict__ assign,
                const float* __restrict__ inv_norm, const float* __restrict__ inv_norm_kept,
                int D, int max_kept, unsigned long long* __restrict__ best, float* __restrict__ sim_debug) {
  constexpr int kVec = Storage<T>::kVec;
  const int b = blockIdx.y, m = blockIdx.x;
  const int v0 = cu_vis[b];
  if (m >= cu_vis[b + 1] - v0) return;
  const int g = v0 + m;
  if (assign[g] >= 0) return;                      // kept token
  const int k0 = cu_kept[b], kb = cu_kept[b + 1] - k0;
  const T* hm = hidden + (size_t)(cu_seqlens[b] + m) * D;
  const float inm = inv_norm[g];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  unsigned long long mine = 0ull;
  for (int s = warp; s < kb; s += 8) {
    const T* hk = kept_rows + (size_t)(k0 + s) * D;
    float acc = 0.f;
    for (int c = lane * kVec; c < D; c += 32 * kVec) {
      float x[kVec], y[kVec];
      Storage<T>::load(hm + c, x);
      Storage<T>::load(hk + c, y);
#pragma unroll
      for (int i = 0; i < kVec; ++i) acc = fmaf(x[i], y[i], acc);
    }
    acc = warp_sum(acc);
    const float sim = (acc * inm) * inv_norm_kept[k0 + s];   // the value the arg-max compares
    if (lane == 0) {
      const unsigned long long packed = ((unsigned long long)ordered_key(sim) << 32) | (0xffffffffu - (unsigned)s);
      mine = packed > mine ? packed : mine;
      if (sim_debug != nullptr) sim_debug[(size_t)g * max_kept + s] = sim;
    }
  }
  __shared__ unsigned long long red[8];
  if (lane == 0) red[warp] = mine;
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long r = red[0];
#pragma unroll
    for (int w = 1; w < 8; ++w) r = red[w] > r ? red[w] : r;
    best[g] = r;
  }
}

// ---------------------------------------------------------------- finish
constexpr int kMemberThreads = 1024;

// One block per request: destination slots, member counts, list offsets and the
// member lists (each list is put in ascending order by the aggregation kernel).
__global__ void __launch_bounds__(kMemberThreads)
members_kernel(const int32_t* __restrict__ cu_vis, const int32_t* __restrict__ cu_kept,
               const unsigned long long* __restrict__ best, int32_t* __restrict__ assign,
               int32_t* __restrict__ member_count, int32_t* __restrict__ member_off,
               int32_t* __restrict__ cursor, int32_t* __restrict__ member_list) {
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int v0 = cu_vis[b], V = cu_vis[b + 1] - v0;
  const int k0 = cu_kept[b], kb = cu_kept[b + 1] - k0;
  const int pruned_base = v0 - k0;                 // pruned tokens of earlier requests
  __shared__ int warp_tot[32];
  __shared__ int carry;
  for (int s = tid; s < kb; s += kMemberThreads) cursor[k0 + s] = 0;
  __syncthreads();
  for (int m = tid; m < V; m += kMemberThreads) {
    const int g = v0 + m;
    if (assign[g] < 0) {
      const int slot = (int)(0xffffffffu - (unsigned)(best[g] & 0xffffffffull));
      assign[g] = slot;
      atomicAdd(&cursor[k0 + slot], 1);
    }
  }
  if (tid == 0) carry = 0;
  __syncthreads();
  for (int base = 0; base < kb; base += kMemberThreads) {
    const int s = base + tid;
    const int c = s < kb ? cursor[k0 + s] : 0;
    int incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    int chunk_total = 0;
    if (warp == 0) {
      const int w = warp_tot[lane];
      int winc = w;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, winc, o);
        if (lane >= o) winc += t;
      }
      warp_tot[lane] = winc - w;
      chunk_total = __shfl_sync(0xffffffffu, winc, 31);
    }
    __syncthreads();
    const int excl = carry + warp_tot[warp] + incl - c;
    if (s < kb) {
      member_count[k0 + s] = c;
      member_off[k0 + s] = pruned_base + excl;
      cursor[k0 + s] = pruned_base + excl;
    }
    __syncthreads();
    if (tid == 0) carry += chunk_total;
    __syncthreads();
  }
  for (int m = tid; m < V; m += kMemberThreads) {
    const int g = v0 + m;
    const int slot = assign[g];
    // a kept token holds its own slot: tell it apart by asking whether it heads that slot
    // (kept tokens were given their slot before this kernel and have best == 0)
    if (best[g] != 0ull) member_list[atomicAdd(&cursor[k0 + slot], 1)] = m;
  }
}

constexpr int kAggThreads = 256;
// kAggMaxVec: 16-byte vectors per thread, D <= 256 * kAggMaxVec * kVec

template <typename T, int kAggMaxVec>
__device__ __forceinline__ void add_rows(const T* __restrict__ base, size_t row_stride, const int* list, int n,
                                         int D, float (&acc)[kAggMaxVec][Storage<T>::kVec]) {
  constexpr int kVec = Storage<T>::kVec;
  int i = 0;
  for (; i + 4 <= n; i += 4) {      // four rows in flight, added in list order
    float f[4][kAggMaxVec][kVec];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const T* src = base + (size_t)list[i + r] * row_stride;
#pragma unroll
      for (int v = 0; v < kAggMaxVec; ++v) {
        const int c = (threadIdx.x + v * kAggThreads) * kVec;
        if (c < D) Storage<T>::load(src + c, f[r][v]);
      }
    }
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int v = 0; v < kAggMaxVec; ++v) {
        const int c = (threadIdx.x + v * kAggThreads) * kVec;
        if (c < D) {
#pragma unroll
          for (int e = 0; e < kVec; ++e) acc[v][e] += f[r][v][e];
        }
      }
  }
  for (; i < n; ++i) {
    const T* src = base + (size_t)list[i] * row_stride;
#pragma unroll
    for (int v = 0; v < kAggMaxVec; ++v) {
      const int c = (threadIdx.x + v * kAggThreads) * kVec;
      if (c < D) {
        float f[kVec];
        Storage<T>::load(src + c, f);
#pragma unroll
        for (int e = 0; e < kVec; ++e) acc[v][e] += f[e];
      }
    }
  }
}

// One block per OUTPUT row.  Rows [0, k_b) of a request are the merged kept
// visual tokens, the rest are the prompt and response rows, copied.
template <typename T, int kAggMaxVec>
__global__ void __launch_bounds__(kAggThreads)
aggregate_compact_kernel(const T* __restrict__ hidden, const int32_t* __restrict__ cu_seqlens,
                         const int32_t* __restrict__ n_visual, const int32_t* __restrict__ cu_vis,
                         const int32_t* __restrict__ kept_idx, const int32_t* __restrict__ cu_kept,
                         const int32_t* __restrict__ cu_seqlens_out, int B, int D, int mean,
                         const int32_t* __restrict__ assign, const int32_t* __restrict__ member_count,
                         const int32_t* __restrict__ member_off, const int32_t* __restrict__ member_list,
                         T* __restrict__ hidden_out, int32_t* __restrict__ src_of_dst) {
  constexpr int kVec = Storage<T>::kVec;
  const int row = blockIdx.x;
  if (row >= cu_seqlens_out[B]) return;
  const int b = find_segment(cu_seqlens_out, B, row);
  const int r = row - cu_seqlens_out[b];
  const int k0 = cu_kept[b], kb = cu_kept[b + 1] - k0;
  const int lo = cu_seqlens[b], Vb = n_visual[b];
  T* dst = hidden_out + (size_t)row * D;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  if (r >= kb) {                                    // prompt / response row: copy
    const int src_row = lo + Vb + (r - kb);
    const T* src = hidden + (size_t)src_row * D;
    for (int c = tid * kVec; c < D; c += kAggThreads * kVec)
      *reinterpret_cast<uint4*>(dst + c) = *reinterpret_cast<const uint4*>(src + c);
    if (tid == 0) src_of_dst[row] = src_row;
    return;
  }

  const int pos = kept_idx[k0 + r];
  const int cnt = member_count[k0 + r];
  const T* req = hidden + (size_t)lo * D;
  float acc[kAggMaxVec][kVec];
  {
    const T* src = req + (size_t)pos * D;
#pragma unroll
    for (int v = 0; v < kAggMaxVec; ++v) {
      const int c = (tid + v * kAggThreads) * kVec;
      if (c < D) Storage<T>::load(src + c, acc[v]);
      else {
#pragma unroll
        for (int e = 0; e < kVec; ++e) acc[v][e] = 0.f;
      }
    }
  }
  __shared__ int list[kAggThreads];
  if (cnt > 0 && cnt <= 32) {
    // small list: rank-sort it inside one warp (members are distinct positions)
    if (warp == 0) {
      const int mine = lane < cnt ? member_list[member_off[k0 + r] + lane] : 0x7fffffff;
      int rank = 0;
      for (int j = 0; j < cnt; ++j) rank += __shfl_sync(0xffffffffu, mine, j) < mine ? 1 : 0;
      if (lane < cnt) list[rank] = mine;
    }
    __syncthreads();
    add_rows<T, kAggMaxVec>(req, (size_t)D, list, cnt, D, acc);
  } else if (cnt > 32) {
    // long list: walk the request's assignment array in position order, 256
    // positions at a time, compacting the members of this slot in order
    __shared__ int warp_tot[kAggThreads / 32];
    const int32_t* as = assign + cu_vis[b];
    for (int base = 0; base < Vb; base += kAggThreads) {
      const int m = base + tid;
      // a member is a position routed to this slot that is not the kept token itself
      const bool hit = m < Vb && as[m] == r && m != pos;
      const unsigned bal = __ballot_sync(0xffffffffu, hit);
      if (lane == 0) warp_tot[warp] = __popc(bal);
      __syncthreads();
      int before = 0, total = 0;
#pragma unroll
      for (int w = 0; w < kAggThreads / 32; ++w) {
        const int t = warp_tot[w];
        if (w < warp) before += t;
        total += t;
      }
      if (hit) list[before + __popc(bal & ((1u << lane) - 1u))] = m;
      __syncthreads();
      add_rows<T, kAggMaxVec>(req, (size_t)D, list, total, D, acc);
      __syncthreads();
    }
  }
  const float denom = mean ? (float)(1 + cnt) : 1.f;
#pragma unroll
  for (int v = 0; v < kAggMaxVec; ++v) {
    const int c = (tid + v * kAggThreads) * kVec;
    if (c < D) {
      float f[kVec];
#pragma unroll
      for (int e = 0; e < kVec; ++e) f[e] = acc[v][e] / denom;
      Storage<T>::store(dst + c, f);
    }
  }
  if (tid == 0) src_of_dst[row] = lo + pos;
}

}  // namespace

int launch_merge_prepare(d3tom_ctx* ctx, const MergeArgs& a, cudaStream_t s) {
  const int vis_bound = a.total_tokens < a.B * a.max_visual ? a.total_tokens : a.B * a.max_visual;
  const int kept_bound = a.total_tokens < a.B * a.max_kept ? a.total_tokens : a.B * a.max_kept;
  init_slots_kernel<<<ceil_div(vis_bound, 256), 256, 0, s>>>(a.cu_vis, a.B, a.assign, ctx->best);
  D3TOM_LAUNCH_CHECK(ctx);
  scatter_slots_kernel<<<ceil_div(kept_bound, 256), 256, 0, s>>>(a.kept_idx, a.cu_kept, a.cu_vis, a.B, a.assign);
  D3TOM_LAUNCH_CHECK(ctx);
  dim3 grid(a.max_visual, a.B);
  if (a.dt == D3TOM_FP32)
    rownorm_gather_kernel<float><<<grid, 128, 0, s>>>(static_cast<const float*>(a.hidden), a.cu_seqlens, a.cu_vis,
                                                      a.cu_kept, a.assign, a.D, ctx->inv_norm, ctx->inv_norm_kept,
                                                      static_cast<float*>(ctx->kept_rows));
  else
    rownorm_gather_kernel<__nv_bfloat16><<<grid, 128, 0, s>>>(static_cast<const __nv_bfloat16*>(a.hidden),
                                                              a.cu_seqlens, a.cu_vis, a.cu_kept, a.assign, a.D,
                                                              ctx->inv_norm, ctx->inv_norm_kept,
                                                              static_cast<__nv_bfloat16*>(ctx->kept_rows));
  D3TOM_LAUNCH_CHECK(ctx);
  return D3TOM_OK;
}

int launch_sim_simt(d3tom_ctx* ctx, const MergeArgs& a, cudaStream_t s) {
  dim3 grid(a.max_visual, a.B);
  if (a.dt == D3TOM_FP32)
    sim_simt_kernel<float><<<grid, 256, 0, s>>>(static_cast<const float*>(a.hidden),
                                                static_cast<const float*>(ctx->kept_rows), a.cu_seqlens, a.cu_vis,
                                                a.cu_kept, a.assign, ctx->inv_norm, ctx->inv_norm_kept, a.D,
                                                a.max_kept, ctx->best, a.sim_debug);
  else
    sim_simt_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(a.hidden),
                                                        static_cast<const __nv_bfloat16*>(ctx->kept_rows),
                                                        a.cu_seqlens, a.cu_vis, a.cu_kept, a.assign, ctx->inv_norm,
                                                        ctx->inv_norm_kept, a.D, a.max_kept, ctx->best, a.sim_debug);
  D3TOM_LAUNCH_CHECK(ctx);
  return D3TOM_OK;
}

int launch_merge_finish(d3tom_ctx* ctx, const MergeArgs& a, cudaStream_t s) {
  members_kernel<<<a.B, kMemberThreads, 0, s>>>(a.cu_vis, a.cu_kept, ctx->best, a.assign, a.member_count,
                                                ctx->member_off, ctx->member_cursor, ctx->member_list);
  D3TOM_LAUNCH_CHECK(ctx);
  const int mean = a.mode == D3TOM_AGG_MEAN ? 1 : 0;
  if (a.total_out <= 0) return D3TOM_OK;
#define D3TOM_AGG_LAUNCH(T, NV)                                                                              \
  aggregate_compact_kernel<T, NV><<<a.total_out, kAggThreads, 0, s>>>(                                       \
      static_cast<const T*>(a.hidden), a.cu_seqlens, a.n_visual, a.cu_vis, a.kept_idx, a.cu_kept,            \
      a.cu_seqlens_out, a.B, a.D, mean, a.assign, a.member_count, ctx->member_off, ctx->member_list,         \
      static_cast<T*>(a.hidden_out), a.src_of_dst)
  if (a.dt == D3TOM_FP32) {
    const int nv = ceil_div(a.D, kAggThreads * 4);
    if (nv <= 1) D3TOM_AGG_LAUNCH(float, 1);
    else if (nv <= 2) D3TOM_AGG_LAUNCH(float, 2);
    else if (nv <= 4) D3TOM_AGG_LAUNCH(float, 4);
    else return D3TOM_ERR_UNSUPPORTED;
  } else {
    const int nv = ceil_div(a.D, kAggThreads * 8);
    if (nv <= 1) D3TOM_AGG_LAUNCH(__nv_bfloat16, 1);
    else if (nv <= 2) D3TOM_AGG_LAUNCH(__nv_bfloat16, 2);
    else if (nv <= 4) D3TOM_AGG_LAUNCH(__nv_bfloat16, 4);
    else return D3TOM_ERR_UNSUPPORTED;
  }
#undef D3TOM_AGG_LAUNCH
  D3TOM_LAUNCH_CHECK(ctx);
  return D3TOM_OK;
}
