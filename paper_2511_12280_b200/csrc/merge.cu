// Similarity-based merging (Sec. 3.2.2; Algorithm 1, the loop over V_merge and
// the removal of the merged positions), everything except the tensor-core
// similarity kernel:
//
//   prepare   slot of every visual token in the kept list (-1 = pruned), 1/|h| of
//             every visual row, and a packed copy of the kept rows (the second
//             operand of the similarity)
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
// One block per visual row: its slot in the kept list (binary search of the ascending
// list; -1 for a pruned row), a cleared arg-max word, the inverse norm, and, for kept
// rows, a copy into the packed second operand of the similarity.
constexpr int kPrepThreads = 128;
constexpr int kPrepVec = 4;          // 16-byte vectors per thread and pass

template <typename T>
__global__ void __launch_bounds__(kPrepThreads)
prepare_rows_kernel(const T* __restrict__ hidden, const int32_t* __restrict__ cu_seqlens,
                    const int32_t* __restrict__ cu_vis, const int32_t* __restrict__ kept_idx,
                    const int32_t* __restrict__ cu_kept, int D, int32_t* __restrict__ assign,
                    unsigned long long* __restrict__ best, float* __restrict__ inv_norm,
                    float* __restrict__ inv_norm_kept, T* __restrict__ kept_rows) {
  constexpr int kVec = Storage<T>::kVec;
  const int b = blockIdx.y, m = blockIdx.x;
  const int v0 = cu_vis[b];
  if (m >= cu_vis[b + 1] - v0) return;
  const int g = v0 + m;
  const int k0 = cu_kept[b], kb = cu_kept[b + 1] - k0;
  int lo = 0, hi = kb;                                   // first kept position >= m
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (kept_idx[k0 + mid] < m) lo = mid + 1; else hi = mid;
  }
  const int slot = (lo < kb && kept_idx[k0 + lo] == m) ? lo : -1;
  const T* src = hidden + (size_t)(cu_seqlens[b] + m) * D;
  T* dst = slot >= 0 ? kept_rows + (size_t)(k0 + slot) * D : nullptr;
  float ss = 0.f;
  for (int c0 = threadIdx.x * kVec; c0 < D; c0 += kPrepThreads * kVec * kPrepVec) {
    float f[kPrepVec][kVec];
#pragma unroll
    for (int v = 0; v < kPrepVec; ++v) {                 // all loads of the pass are issued before any is used
      const int c = c0 + v * kPrepThreads * kVec;
      if (c < D) Storage<T>::load(src + c, f[v]);
    }
#pragma unroll
    for (int v = 0; v < kPrepVec; ++v) {
      const int c = c0 + v * kPrepThreads * kVec;
      if (c < D) {
#pragma unroll
        for (int i = 0; i < kVec; ++i) ss = fmaf(f[v][i], f[v][i], ss);
        if (dst != nullptr) Storage<T>::store(dst + c, f[v]);
      }
    }
  }
  __shared__ float red[kPrepThreads / 32];
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  if (threadIdx.x == 0) {
    const float tot = (red[0] + red[1]) + (red[2] + red[3]);
    const float inv = tot > 0.f ? 1.0f / sqrtf(tot) : 0.f;
    inv_norm[g] = inv;
    assign[g] = slot;
    best[g] = 0ull;
    if (slot >= 0) inv_norm_kept[k0 + slot] = inv;
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
    const float sim = (acc * inm) * inv_norm_kept[k0 + s] + 0.0f;   // the value the arg-max compares (never -0)
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
constexpr int kMemberSmemSlots = 12 * 1024;        // kept counts up to this keep their counters in shared memory

// One block per request: destination slots, member counts, list offsets and the
// member lists (each list is put in ascending order by the aggregation kernel).
// Counters live in shared memory when the kept count allows, else in `cursor`.
__global__ void __launch_bounds__(kMemberThreads)
members_kernel(const int32_t* __restrict__ cu_vis, const int32_t* __restrict__ cu_kept,
               const unsigned long long* __restrict__ best, int32_t* __restrict__ assign,
               int32_t* __restrict__ member_count, int32_t* __restrict__ member_off,
               int32_t* __restrict__ cursor, int32_t* __restrict__ member_list) {
  extern __shared__ int ctr_s[];
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int v0 = cu_vis[b], V = cu_vis[b + 1] - v0;
  const int k0 = cu_kept[b], kb = cu_kept[b + 1] - k0;
  const int pruned_base = v0 - k0;                 // pruned tokens of earlier requests
  int* ctr = kb <= kMemberSmemSlots ? ctr_s : cursor + k0;
  __shared__ int warp_tot[32];
  __shared__ int carry;
  for (int s = tid; s < kb; s += kMemberThreads) ctr[s] = 0;
  __syncthreads();
  for (int m = tid; m < V; m += kMemberThreads) {
    const int g = v0 + m;
    const unsigned long long w = best[g];
    if (w != 0ull) {                               // a pruned token (kept tokens keep best == 0)
      const int slot = (int)(0xffffffffu - (unsigned)(w & 0xffffffffull));
      assign[g] = slot;
      atomicAdd(&ctr[slot], 1);
    }
  }
  if (tid == 0) carry = 0;
  __syncthreads();
  for (int base = 0; base < kb; base += kMemberThreads) {
    const int s = base + tid;
    const int c = s < kb ? ctr[s] : 0;
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
      ctr[s] = pruned_base + excl;
    }
    __syncthreads();
    if (tid == 0) carry += chunk_total;
    __syncthreads();
  }
  for (int m = tid; m < V; m += kMemberThreads) {
    const int g = v0 + m;
    if (best[g] != 0ull) member_list[atomicAdd(&ctr[assign[g]], 1)] = m;
  }
}

__device__ __forceinline__ int ceil_div_dev(int a, int b) { return (a + b - 1) / b; }

// acc += the 16 bytes of storage in `raw`, element by element
template <typename T> __device__ __forceinline__ void add_raw(float (&acc)[Storage<T>::kVec], uint4 raw);
template <> __device__ __forceinline__ void add_raw<float>(float (&acc)[4], uint4 raw) {
  acc[0] += __uint_as_float(raw.x); acc[1] += __uint_as_float(raw.y);
  acc[2] += __uint_as_float(raw.z); acc[3] += __uint_as_float(raw.w);
}
template <> __device__ __forceinline__ void add_raw<__nv_bfloat16>(float (&acc)[8], uint4 raw) {
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    acc[2 * i] += __uint_as_float(w[i] << 16);
    acc[2 * i + 1] += __uint_as_float(w[i] & 0xffff0000u);
  }
}

constexpr int kAggMaxThreads = 512;
constexpr int kAggUnroll = 8;            // member rows in flight per thread

// One block per OUTPUT row, one 16-byte vector of the row per thread and pass.  Rows
// [0, k_b) of a request are the merged kept visual tokens, the rest are the prompt and
// response rows, copied.  Members are added in ascending position, kAggUnroll rows in
// flight, fp32 accumulation, one rounding.
template <typename T>
__global__ void __launch_bounds__(kAggMaxThreads)
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
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nthreads = blockDim.x, nwarps = nthreads >> 5;

  if (r >= kb) {                                    // prompt / response row: copy
    const int src_row = lo + Vb + (r - kb);
    const T* src = hidden + (size_t)src_row * D;
    for (int c = tid * kVec; c < D; c += nthreads * kVec)
      *reinterpret_cast<uint4*>(dst + c) = *reinterpret_cast<const uint4*>(src + c);
    if (tid == 0) src_of_dst[row] = src_row;
    return;
  }

  const int pos = kept_idx[k0 + r];
  const int cnt = member_count[k0 + r];
  const int off = member_off[k0 + r];
  const T* req = hidden + (size_t)lo * D;
  __shared__ int list[kAggMaxThreads];
  __shared__ int warp_tot[kAggMaxThreads / 32];
  const float inv_denom = mean ? 1.0f / (float)(1 + cnt) : 1.f;
  if (cnt > 0 && cnt <= 32) {
    // small list: rank-sort it inside one warp (members are distinct positions)
    if (warp == 0) {
      const int mine = lane < cnt ? member_list[off + lane] : 0x7fffffff;
      int rank = 0;
      for (int j = 0; j < cnt; ++j) rank += __shfl_sync(0xffffffffu, mine, j) < mine ? 1 : 0;
      if (lane < cnt) list[rank] = mine;
    }
    __syncthreads();
  }
  const int passes = ceil_div_dev(D, nthreads * kVec);            // uniform over the block
  for (int p = 0; p < passes; ++p) {
    const int c = (p * nthreads + tid) * kVec;
    const bool live = c < D;
    const T* col = req + (live ? c : 0);                        // threads past the row end read column 0, write nothing
    float acc[kVec];
    Storage<T>::load(col + (size_t)pos * D, acc);
    auto add_list = [&](int n) {
      int i = 0;
      for (; i + kAggUnroll <= n; i += kAggUnroll) {
        uint4 raw[kAggUnroll];
#pragma unroll
        for (int u = 0; u < kAggUnroll; ++u) raw[u] = *reinterpret_cast<const uint4*>(col + (size_t)list[i + u] * D);
#pragma unroll
        for (int u = 0; u < kAggUnroll; ++u) add_raw<T>(acc, raw[u]);
      }
      for (; i < n; ++i) add_raw<T>(acc, *reinterpret_cast<const uint4*>(col + (size_t)list[i] * D));
    };
    if (cnt <= 32) {
      add_list(cnt);
    } else {
      // long list: walk the request's assignment array in position order, one block-width of
      // positions at a time, compacting the members of this slot in order
      const int32_t* as = assign + cu_vis[b];
      for (int base = 0; base < Vb; base += nthreads) {
        const int m = base + tid;
        const bool hit = m < Vb && as[m] == r && m != pos;     // routed here and not the kept token itself
        const unsigned bal = __ballot_sync(0xffffffffu, hit);
        if (lane == 0) warp_tot[warp] = __popc(bal);
        __syncthreads();
        int before = 0, total = 0;
        for (int w = 0; w < nwarps; ++w) {
          const int t = warp_tot[w];
          if (w < warp) before += t;
          total += t;
        }
        if (hit) list[before + __popc(bal & ((1u << lane) - 1u))] = m;
        __syncthreads();
        add_list(total);
        __syncthreads();
      }
    }
    if (live) {
#pragma unroll
      for (int e = 0; e < kVec; ++e) acc[e] *= inv_denom;
      Storage<T>::store(dst + c, acc);
    }
  }
  if (tid == 0) src_of_dst[row] = lo + pos;
}

}  // namespace

int launch_merge_prepare(d3tom_ctx* ctx, const MergeArgs& a, cudaStream_t s) {
  dim3 grid(a.max_visual, a.B);
  if (a.dt == D3TOM_FP32)
    prepare_rows_kernel<float><<<grid, kPrepThreads, 0, s>>>(static_cast<const float*>(a.hidden), a.cu_seqlens, a.cu_vis,
                                                            a.kept_idx, a.cu_kept, a.D, a.assign, ctx->best,
                                                            ctx->inv_norm, ctx->inv_norm_kept,
                                                            static_cast<float*>(ctx->kept_rows));
  else
    prepare_rows_kernel<__nv_bfloat16><<<grid, kPrepThreads, 0, s>>>(static_cast<const __nv_bfloat16*>(a.hidden),
                                                                    a.cu_seqlens, a.cu_vis, a.kept_idx, a.cu_kept, a.D,
                                                                    a.assign, ctx->best, ctx->inv_norm,
                                                                    ctx->inv_norm_kept,
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
  static bool attr_set = false;
  if (!attr_set) {
    D3TOM_CUDA_TRY(ctx, cudaFuncSetAttribute(members_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             kMemberSmemSlots * (int)sizeof(int)));
    attr_set = true;
  }
  const size_t ctr_bytes = (size_t)(a.max_kept <= kMemberSmemSlots ? a.max_kept : 0) * sizeof(int);
  members_kernel<<<a.B, kMemberThreads, ctr_bytes, s>>>(a.cu_vis, a.cu_kept, ctx->best, a.assign, a.member_count,
                                                        ctx->member_off, ctx->member_cursor, ctx->member_list);
  D3TOM_LAUNCH_CHECK(ctx);
  const int mean = a.mode == D3TOM_AGG_MEAN ? 1 : 0;
  if (a.total_out <= 0) return D3TOM_OK;
  const int vec = a.dt == D3TOM_FP32 ? 4 : 8;
  int threads = ceil_div(ceil_div(a.D, vec), 32) * 32;             // one 16-byte vector per thread when the row allows
  if (threads > kAggMaxThreads) threads = kAggMaxThreads;
  if (a.dt == D3TOM_FP32)
    aggregate_compact_kernel<float><<<a.total_out, threads, 0, s>>>(
        static_cast<const float*>(a.hidden), a.cu_seqlens, a.n_visual, a.cu_vis, a.kept_idx, a.cu_kept, a.cu_seqlens_out,
        a.B, a.D, mean, a.assign, a.member_count, ctx->member_off, ctx->member_list, static_cast<float*>(a.hidden_out),
        a.src_of_dst);
  else
    aggregate_compact_kernel<__nv_bfloat16><<<a.total_out, threads, 0, s>>>(
        static_cast<const __nv_bfloat16*>(a.hidden), a.cu_seqlens, a.n_visual, a.cu_vis, a.kept_idx, a.cu_kept,
        a.cu_seqlens_out, a.B, a.D, mean, a.assign, a.member_count, ctx->member_off, ctx->member_list,
        static_cast<__nv_bfloat16*>(a.hidden_out), a.src_of_dst);
  D3TOM_LAUNCH_CHECK(ctx);
  return D3TOM_OK;
}
