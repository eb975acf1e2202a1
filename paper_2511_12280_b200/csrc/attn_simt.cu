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
// finishing kernels turn those into S_j = sum_h sum_{i in D} A_ij.
#include "common.cuh"

namespace {

constexpr int kRowsPerBlock = 8;   // warps per block

template <typename T>
__global__ void __launch_bounds__(kRowsPerBlock * 32)
attn_simt_kernel(AttnArgs a) {
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

// partial[h][cu_vis[b] + j] = sum over the request's deciders (ascending) of
// exp2(score * c - M) / l
__global__ void __launch_bounds__(256)
importance_partial_kernel(const float* __restrict__ score, const float2* __restrict__ lse,
                          const int32_t* __restrict__ n_visual, const int32_t* __restrict__ cu_deciders,
                          const int32_t* __restrict__ cu_vis, int max_deciders, int vis_stride,
                          float scale_log2, float* __restrict__ partial, int partial_stride) {
  const int b = blockIdx.z, h = blockIdx.y;
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= n_visual[b]) return;
  const int d0 = cu_deciders[b], d1 = cu_deciders[b + 1];
  float acc = 0.f;
  for (int d = d0; d < d1; ++d) {
    const size_t r = (size_t)h * max_deciders + d;
    const float2 ml = lse[r];
    acc += exp2f(fmaf(score[r * vis_stride + j], scale_log2, -ml.x)) / ml.y;
  }
  partial[(size_t)h * partial_stride + cu_vis[b] + j] = acc;
}

// importance[g] = sum over heads (ascending) of partial[h][g]
__global__ void __launch_bounds__(256)
importance_reduce_kernel(const float* __restrict__ partial, int partial_stride, int H,
                         const int32_t* __restrict__ cu_vis, int B, float* __restrict__ importance) {
  const int g = blockIdx.x * blockDim.x + threadIdx.x;
  if (g >= cu_vis[B]) return;
  float acc = 0.f;
  for (int h = 0; h < H; ++h) acc += partial[(size_t)h * partial_stride + g];
  importance[g] = acc;
}

}  // namespace

int launch_attn_simt(d3tom_ctx* ctx, d3tom_dtype dt, const AttnArgs& a, cudaStream_t s) {
  dim3 grid(ceil_div(a.max_seqlen, kRowsPerBlock), a.H, a.B);
  if (dt == D3TOM_FP32) attn_simt_kernel<float><<<grid, kRowsPerBlock * 32, 0, s>>>(a);
  else attn_simt_kernel<__nv_bfloat16><<<grid, kRowsPerBlock * 32, 0, s>>>(a);
  D3TOM_LAUNCH_CHECK(ctx);
  return D3TOM_OK;
}

int launch_importance_finish(d3tom_ctx* ctx, const AttnArgs& a, int max_visual, float* importance,
                             const int32_t* cu_vis, cudaStream_t s) {
  if (max_visual <= 0) return D3TOM_OK;
  dim3 grid(ceil_div(max_visual, 256), a.H, a.B);
  importance_partial_kernel<<<grid, 256, 0, s>>>(a.score_scratch, a.lse_scratch, a.n_visual, a.cu_deciders, cu_vis,
                                                 a.max_deciders, a.vis_stride, a.scale_log2, ctx->imp_partial,
                                                 ctx->lim.max_total_tokens);
  D3TOM_LAUNCH_CHECK(ctx);
  // the visual total is cu_vis[B] on the device; the grid is sized by its host bound
  const int total_vis_bound = min(a.total_tokens, a.B * max_visual);
  importance_reduce_kernel<<<ceil_div(total_vis_bound, 256), 256, 0, s>>>(ctx->imp_partial, ctx->lim.max_total_tokens,
                                                                          a.H, cu_vis, a.B, importance);
  D3TOM_LAUNCH_CHECK(ctx);
  return D3TOM_OK;
}
