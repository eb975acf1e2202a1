// Bidirectional attention on CUDA cores (fp32 arithmetic) and the importance
// finishing kernels shared with the tensor-core attention.
//
// One warp owns one (query row, head).  Keys are visited 32 at a time: every
// lane scores one key (Sec. 3.2.1, A = softmax(QK^T * scale)), the warp keeps
// the running maximum and sum (online softmax in the log2 domain) and the
// output accumulators, lane c owning channels c, c+32, ...
//
// Decider rows additionally write their raw q.k scores over the visual keys to
// the score scratch and their final (M, l) pair to the lse scratch; the
// finishing kernel turns those into S_j = sum_h sum_{i in D} A_ij.
#include "common.cuh"

namespace {

constexpr int kRowsPerBlock = 8;   // warps per block

template <typename T>
__global__ void __launch_bounds__(kRowsPerBlock * 32)
attn_simt_kernel(AttnArgs a) {
  grid_dependency_enter();
  const int b = blockIdx.z, h = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int lo = a.cu_seqlens[b], n = a.cu_seqlens[b + 1] - lo;
  const int row = blockIdx.x * kRowsPerBlock + warp;
  __shared__ float q_s[kRowsPerBlock][128];
  if (row >= n) return;   // whole warp leaves together (row is per warp)
  const int H = a.H, dh = a.dh;
  const T* q = static_cast<const T*>(a.q) + ((size_t)(lo + row) * H + h) * dh;
  const T* kbase = static_cast<const T*>(a.k) + ((size_t)lo * H + h) * dh;
  const T* vbase = static_cast<const T*>(a.v) + ((size_t)lo * H + h) * dh;
  for (int c = lane; c < dh; c += 32) q_s[warp][c] = Storage<T>::to_float(q[c]);
  __syncwarp();

  // is this row a decider?  (strictly ascending list -> binary search)
  int dec_slot = -1, n_vis = 0;
  if (a.decider_pos != nullptr) {
    n_vis = a.n_visual[b];
    int d0 = a.cu_deciders[b], d1 = a.cu_deciders[b + 1];
    int l = d0, r = d1;
    while (l < r) {
      int mid = (l + r) >> 1;
      int p = a.decider_pos[mid];
      if (p == row) { dec_slot = mid; break; }
      if (p < row) l = mid + 1; else r = mid;
    }
  }
  float* score_row = dec_slot >= 0
      ? a.score_scratch + ((size_t)h * a.max_deciders + dec_slot) * a.vis_stride : nullptr;

  float m = -INFINITY, l = 0.f;
  float o[4] = {0.f, 0.f, 0.f, 0.f};
  for (int j0 = 0; j0 < n; j0 += 32) {
    const int j = j0 + lane;
    float s = -INFINITY;
    if (j < n) {
      const T* kr = kbase + (size_t)j * H * dh;
      float acc = 0.f;
      for (int c = 0; c < dh; ++c) acc = fmaf(q_s[warp][c], Storage<T>::to_float(kr[c]), acc);
      if (score_row != nullptr && j < n_vis) score_row[j] = acc;
      s = acc * a.scale_log2;
    }
    const float m_new = fmaxf(m, warp_max(s));
    const float corr = exp2f(m - m_new);           // first chunk: exp2(-inf) = 0
    const float p = (j < n) ? exp2f(s - m_new) : 0.f;
    l = l * corr + warp_sum(p);
#pragma unroll
    for (int i = 0; i < 4; ++i) o[i] *= corr;
    const int cnt = min(32, n - j0);
    for (int jj = 0; jj < cnt; ++jj) {
      const float pj = __shfl_sync(0xffffffffu, p, jj);
      const T* vr = vbase + (size_t)(j0 + jj) * H * dh;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int c = lane + 32 * i;
        if (c < dh) o[i] = fmaf(pj, Storage<T>::to_float(vr[c]), o[i]);
      }
    }
    m = m_new;
  }
  T* out = static_cast<T*>(a.out) + ((size_t)(lo + row) * H + h) * dh;
  const float inv_l = 1.f / l;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int c = lane + 32 * i;
    if (c < dh) out[c] = Storage<T>::from_float(o[i] * inv_l);
  }
  if (dec_slot >= 0 && lane == 0) a.lse_scratch[(size_t)h * a.max_deciders + dec_slot] = make_float2(m, l);
}

// One block = (256 visual keys, head, request).
//   partial[h][cu_vis[b] + j] = sum over the request's deciders (ascending) of exp2(score * c - M) / l
// The last of the H blocks of a key range to finish (a counter per range, left at zero again
// afterwards) adds the H partials in ascending head order:
//   importance[g] = sum over heads of partial[h][g]
// so the result does not depend on which block that is: no float atomics, reproducible.
constexpr int kImpThreads = 256;
constexpr int kImpDecChunk = 128;

__global__ void __launch_bounds__(kImpThreads)
importance_finish_kernel(const float* __restrict__ score, const float2* __restrict__ lse,
                         const int32_t* __restrict__ n_visual, const int32_t* __restrict__ cu_deciders,
                         const int32_t* __restrict__ cu_vis, int max_deciders, int vis_stride, float scale_log2,
                         float* __restrict__ partial, int partial_stride, int H, int* __restrict__ counters,
                         float* __restrict__ importance) {
  grid_dependency_enter();
  const int b = blockIdx.z, h = blockIdx.y;
  const int Vb = n_visual[b];
  if ((int)blockIdx.x * kImpThreads >= Vb) return;              // uniform: no key of this request in the range
  const int j = blockIdx.x * kImpThreads + threadIdx.x;
  const int d0 = cu_deciders[b], d1 = cu_deciders[b + 1];
  __shared__ float neg_m[kImpDecChunk], inv_l[kImpDecChunk];
  __shared__ int is_last;
  const int jj = j < Vb ? j : Vb - 1;                           // threads past the end read a valid column, write nothing
  float acc = 0.f;
  for (int dc = d0; dc < d1; dc += kImpDecChunk) {
    const int nd = min(kImpDecChunk, d1 - dc);
    __syncthreads();
    if (threadIdx.x < nd) {
      const float2 ml = lse[(size_t)h * max_deciders + dc + threadIdx.x];
      neg_m[threadIdx.x] = -ml.x;
      inv_l[threadIdx.x] = 1.0f / ml.y;
    }
    __syncthreads();
    const float* col = score + ((size_t)h * max_deciders + dc) * vis_stride + jj;
    // (the loads of 16 deciders are in flight together; the sum still runs in ascending decider order)
#pragma unroll 16
    for (int d = 0; d < nd; ++d)
      acc = fmaf(exp2f(fmaf(col[(size_t)d * vis_stride], scale_log2, neg_m[d])), inv_l[d], acc);
  }
  const int g0 = cu_vis[b];
  if (j < Vb) partial[(size_t)h * partial_stride + g0 + j] = acc;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    int* ctr = counters + (size_t)b * gridDim.x + blockIdx.x;
    const int prev = atomicAdd(ctr, 1);
    is_last = prev == H - 1;
    if (is_last) *ctr = 0;                                      // ready for the next call
  }
  __syncthreads();
  if (is_last && j < Vb) {
    __threadfence();
    float tot = 0.f;
#pragma unroll 8
    for (int hh = 0; hh < H; ++hh) tot += __ldcg(partial + (size_t)hh * partial_stride + g0 + j);
    importance[g0 + j] = tot;
  }
}

}  // namespace

int launch_attn_simt(d3tom_ctx* ctx, d3tom_dtype dt, const AttnArgs& a, cudaStream_t s) {
  dim3 grid(ceil_div(a.max_seqlen, kRowsPerBlock), a.H, a.B);
  if (dt == D3TOM_FP32) D3TOM_CUDA_TRY(ctx, launch_serialized(attn_simt_kernel<float>, grid, kRowsPerBlock * 32, 0, s, a));
  else D3TOM_CUDA_TRY(ctx, launch_serialized(attn_simt_kernel<__nv_bfloat16>, grid, kRowsPerBlock * 32, 0, s, a));
  return D3TOM_OK;
}

int launch_importance_finish(d3tom_ctx* ctx, const AttnArgs& a, int max_visual, float* importance,
                             const int32_t* cu_vis, cudaStream_t s) {
  if (max_visual <= 0) return D3TOM_OK;
  dim3 grid(ceil_div(max_visual, kImpThreads), a.H, a.B);
  D3TOM_CUDA_TRY(ctx, launch_serialized(importance_finish_kernel, grid, kImpThreads, 0, s, a.score_scratch, a.lse_scratch,
                                        a.n_visual, a.cu_deciders, cu_vis, a.max_deciders, a.vis_stride, a.scale_log2,
                                        ctx->imp_partial, ctx->lim.max_total_tokens, a.H, ctx->imp_counters, importance));
  return D3TOM_OK;
}
