// Similarity-based merging (Sec. 3.2.2; Algorithm 1, the loop over V_merge and
// the removal of the merged positions), everything except the tensor-core
// similarity kernel:
//
//   prepare   slot of every visual token in the kept list (-1 = pruned), 1/|h| of
//             every visual row, and a packed copy of the kept rows (the second
//             operand of the similarity)
//   sim_simt  cosine + arg-max on CUDA cores (fp32 storage, debugging aid)
//   finish    destination slots, per-slot member lists, aggregation in a fixed
//             order and compaction into the shortened sequence
//
// The arg-max is a 64-bit maximum over (order-preserving similarity bits << 32
// | ~slot): the largest similarity wins and, among equals, the lowest slot, no
// matter in which order candidates arrive.
#include "common.cuh"

namespace {

// ---------------------------------------------------------------- prepare
// sum of squares of the 16 bytes of storage in `raw`
template <typename T> __device__ __forceinline__ float sq_raw(uint4 raw);
template <> __device__ __forceinline__ float sq_raw<float>(uint4 raw) {
  const float a = __uint_as_float(raw.x), b = __uint_as_float(raw.y), c = __uint_as_float(raw.z), d = __uint_as_float(raw.w);
  return fmaf(a, a, fmaf(b, b, fmaf(c, c, d * d)));
}
template <> __device__ __forceinline__ float sq_raw<__nv_bfloat16>(uint4 raw) {
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float lo = __uint_as_float(w[i] << 16), hi = __uint_as_float(w[i] & 0xffff0000u);
    s = fmaf(lo, lo, fmaf(hi, hi, s));
  }
  return s;
}

// One WARP per visual row (no block-wide synchronisation, so many rows are in flight per
// SM): its slot in the kept list (-1 for a pruned row), a cleared arg-max word, the
// inverse norm and, for kept rows, a copy into the packed second operand of the similarity.
constexpr int kPrepWarps = 8;
constexpr int kPrepInFlight = 8;       // 16-byte loads in flight per lane

template <typename T>
__global__ void __launch_bounds__(kPrepWarps * 32)
prepare_rows_kernel(const T* __restrict__ hidden, const int32_t* __restrict__ cu_seqlens,
                    const int32_t* __restrict__ cu_vis, const int32_t* __restrict__ kept_idx,
                    const int32_t* __restrict__ cu_kept, int D, int32_t* __restrict__ assign,
                    unsigned long long* __restrict__ best, float* __restrict__ inv_norm,
                    float* __restrict__ inv_norm_kept, T* __restrict__ kept_rows, int* __restrict__ n_heavy) {
  constexpr int kVec = Storage<T>::kVec;
  grid_dependency_enter();
  if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) *n_heavy = 0;   // counted by the members kernel, two launches on
  const int b = blockIdx.y, lane = threadIdx.x & 31;
  const int m = blockIdx.x * kPrepWarps + (threadIdx.x >> 5);
  const int v0 = cu_vis[b];
  if (m >= cu_vis[b + 1] - v0) return;                       // whole warp
  const int g = v0 + m;
  const int k0 = cu_kept[b], kb = cu_kept[b + 1] - k0;
  const uint4* src = reinterpret_cast<const uint4*>(hidden + (size_t)(cu_seqlens[b] + m) * D);
  const int n_vec = D / kVec;                                 // 16-byte vectors of the row
  // the first batch of row loads goes out before the slot search so that the two latencies overlap
  uint4 raw[kPrepInFlight];
#pragma unroll
  for (int u = 0; u < kPrepInFlight; ++u) {
    const int vi = lane + u * 32;
    if (vi < n_vec) raw[u] = src[vi];
  }
  // slot of position m in the ascending kept list: a 32-way search (each step narrows the range
  // 32-fold with one load per lane and a ballot)
  int lo = 0, len = kb;
  while (len > 32) {
    const int stride = (len + 31) >> 5;
    const int idx = lo + lane * stride;
    const bool le = idx < lo + len && kept_idx[k0 + idx] <= m;
    const int n_le = __popc(__ballot_sync(0xffffffffu, le));   // lanes are ascending: the `le` lanes form a prefix
    if (n_le == 0) { len = 0; break; }                          // every kept position is larger than m
    const int new_lo = lo + (n_le - 1) * stride;
    len = min(stride, lo + len - new_lo);
    lo = new_lo;
  }
  const bool eq = lane < len && kept_idx[k0 + lo + lane] == m;
  const unsigned eqb = __ballot_sync(0xffffffffu, eq);
  const int slot = eqb ? lo + __ffs(eqb) - 1 : -1;
  uint4* dst = slot >= 0 ? reinterpret_cast<uint4*>(kept_rows + (size_t)(k0 + slot) * D) : nullptr;
  float ss = 0.f;
  for (int base = 0; base < n_vec; base += kPrepInFlight * 32) {
    if (base > 0) {
#pragma unroll
      for (int u = 0; u < kPrepInFlight; ++u) {
        const int vi = base + lane + u * 32;
        if (vi < n_vec) raw[u] = src[vi];
      }
    }
#pragma unroll
    for (int u = 0; u < kPrepInFlight; ++u) {
      const int vi = base + lane + u * 32;
      if (vi < n_vec) {
        ss += sq_raw<T>(raw[u]);
        if (dst != nullptr) dst[vi] = raw[u];
      }
    }
  }
  ss = warp_sum(ss);
  if (lane == 0) {
    const float inv = ss > 0.f ? 1.0f / sqrtf(ss) : 0.f;
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
  grid_dependency_enter();
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
constexpr int kBitmapBytes = 64 * 1024;            // shared memory for the per-warp position bitmaps
constexpr int kHeavy = 32;                         // a kept token with this many members or more is "heavy"

// One block per request: destination slots, member counts, list offsets and the member
// lists.  Lists of fewer than kHeavy members are left in arrival order (the aggregation
// kernel orders them inside a warp).  Heavy lists are rewritten in ascending position
// here, by marking the members in a bitmap over the request's positions and reading the
// bits back in order, and their slots are appended to `heavy_slots`.
// Dynamic shared memory: [counters (kb ints, when kb <= kMemberSmemSlots)] [bitmaps].
__global__ void __launch_bounds__(kMemberThreads)
members_kernel(const int32_t* __restrict__ cu_vis, const int32_t* __restrict__ cu_kept,
               const unsigned long long* __restrict__ best, int32_t* __restrict__ assign,
               int32_t* __restrict__ member_count, int32_t* __restrict__ member_off,
               int32_t* __restrict__ cursor, int32_t* __restrict__ member_list,
               int32_t* __restrict__ heavy_slots, int* __restrict__ n_heavy, int ctr_ints, int bitmap_warps,
               const int32_t* __restrict__ cu_seqlens, const int32_t* __restrict__ cu_seqlens_out,
               const int32_t* __restrict__ kept_idx, int4* __restrict__ row_desc) {
  extern __shared__ int dyn_s[];
  grid_dependency_enter();
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int v0 = cu_vis[b], V = cu_vis[b + 1] - v0;
  const int k0 = cu_kept[b], kb = cu_kept[b + 1] - k0;
  const int pruned_base = v0 - k0;                 // pruned tokens of earlier requests
  const int lo = cu_seqlens[b], out0 = cu_seqlens_out[b], n_out = cu_seqlens_out[b + 1] - out0;
  // prompt / response rows are copied: member count -1 marks them
  for (int r = kb + tid; r < n_out; r += kMemberThreads) row_desc[out0 + r] = make_int4(lo + V + (r - kb), -1, 0, lo);
  int* ctr = kb <= ctr_ints ? dyn_s : cursor + k0;
  unsigned* bitmaps = reinterpret_cast<unsigned*>(dyn_s + ctr_ints);
  __shared__ int warp_tot[32];
  __shared__ int carry;
  // the request's heavy kept tokens, so that the sorting warps below need not walk over all kept tokens
  constexpr int kHeavyLocal = 2048;
  __shared__ int heavy_local[kHeavyLocal];
  __shared__ int n_heavy_local;
  if (tid == 0) n_heavy_local = 0;
  for (int s = tid; s < kb; s += kMemberThreads) ctr[s] = 0;
  __syncthreads();
  // requests of up to kSlotRegs x 1024 visual tokens keep every token's slot in a register between the counting
  // pass and the filling pass (one round trip to global memory less); -1: a kept token
  constexpr int kSlotRegs = 8;
  const bool in_regs = V <= kSlotRegs * kMemberThreads;
  int my_slot[kSlotRegs];
#pragma unroll
  for (int i = 0; i < kSlotRegs; ++i) {
    my_slot[i] = -1;
    const int m = tid + i * kMemberThreads;
    if (in_regs && m < V) {
      const unsigned long long w = best[v0 + m];
      if (w != 0ull) my_slot[i] = (int)(0xffffffffu - (unsigned)(w & 0xffffffffull));   // a pruned token (kept tokens keep best == 0)
    }
  }
#pragma unroll
  for (int i = 0; i < kSlotRegs; ++i)
    if (my_slot[i] >= 0) {
      assign[v0 + tid + i * kMemberThreads] = my_slot[i];
      atomicAdd(&ctr[my_slot[i]], 1);
    }
  for (int m = tid; m < V && !in_regs; m += kMemberThreads) {
    const int g = v0 + m;
    const unsigned long long w = best[g];
    if (w != 0ull) {
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
      if (c >= kHeavy) {
        heavy_slots[atomicAdd(n_heavy, 1)] = k0 + s;
        const int li = atomicAdd(&n_heavy_local, 1);
        if (li < kHeavyLocal) heavy_local[li] = s;
      }
      // what the aggregation needs to know about this output row, in one 16-byte record
      row_desc[out0 + s] = make_int4(lo + kept_idx[k0 + s], c, pruned_base + excl, lo);
    }
    __syncthreads();
    if (tid == 0) carry += chunk_total;
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < kSlotRegs; ++i)
    if (my_slot[i] >= 0) member_list[atomicAdd(&ctr[my_slot[i]], 1)] = tid + i * kMemberThreads;
  for (int m = tid; m < V && !in_regs; m += kMemberThreads) {
    const int g = v0 + m;
    if (best[g] != 0ull) member_list[atomicAdd(&ctr[assign[g]], 1)] = m;
  }
  __syncthreads();
  // ---- heavy lists into ascending order (one warp per list, bitmap_warps warps take part)
  if (warp < bitmap_warps) {
    const int words = (V + 31) >> 5;
    unsigned* bm = bitmaps + (size_t)warp * words;
    const int nh = n_heavy_local;
    const bool listed = nh <= kHeavyLocal;         // else (more heavy tokens than the list holds): walk over all kept tokens
    for (int h = warp; h < (listed ? nh : kb); h += bitmap_warps) {
      const int s = listed ? heavy_local[h] : h;
      const int cnt = member_count[k0 + s];
      if (cnt < kHeavy) continue;                  // uniform over the warp
      const int off = member_off[k0 + s];
      for (int w = lane; w < words; w += 32) bm[w] = 0u;
      __syncwarp();
      for (int i = lane; i < cnt; i += 32) {
        const int m = member_list[off + i];
        atomicOr(&bm[m >> 5], 1u << (m & 31));
      }
      __syncwarp();
      int written = 0;
      for (int w0 = 0; w0 < words; w0 += 32) {     // 32 words = 1024 positions per pass, in order
        const int w = w0 + lane;
        unsigned bits = w < words ? bm[w] : 0u;
        const int n = __popc(bits);
        int incl = n;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          int t = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += t;
        }
        int dst = off + written + incl - n;
        while (bits) {
          member_list[dst++] = (w << 5) + __ffs(bits) - 1;
          bits &= bits - 1;
        }
        written += __shfl_sync(0xffffffffu, incl, 31);
      }
      __syncwarp();
    }
  }
}

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

constexpr int kAggWarps = 8;
constexpr int kAggUnroll = 4;            // rows in flight per lane
constexpr int kAggCpw = 4;               // 512-byte chunks of a row handled by one warp of a light row

// acc += rows[0..n) of `req` (row indices held one per lane in `rows`), in that order,
// kAggUnroll loads in flight
template <typename T>
__device__ __forceinline__ void add_rows(float (&acc)[Storage<T>::kVec], const T* req, int D, int rows, int n) {
  for (int i = 0; i < n; i += kAggUnroll) {
    uint4 raw[kAggUnroll];
#pragma unroll
    for (int u = 0; u < kAggUnroll; ++u) {
      const int rr = __shfl_sync(0xffffffffu, rows, (i + u) & 31);
      if (i + u < n) raw[u] = *reinterpret_cast<const uint4*>(req + (size_t)rr * D);
    }
#pragma unroll
    for (int u = 0; u < kAggUnroll; ++u)
      if (i + u < n) add_raw<T>(acc, raw[u]);
  }
}

// Aggregation and compaction.  Blocks [heavy_blocks, ...): one WARP per (output row, group of
// kAggCpw 512-byte chunks of the row), one 16-byte vector per lane and chunk, so that one chain
// of index loads is followed by up to kAggUnroll x kAggCpw row loads in flight.  Rows [0, k_b) of a request are the
// merged kept visual tokens, the rest are the prompt and response rows, copied.  The kept
// row comes first, then its members in ascending position, fp32 accumulation, one rounding;
// the (short) member list is ordered with shuffles inside the warp.
// Blocks [0, heavy_blocks): one BLOCK per (heavy kept token, chunk); beyond the actual number they leave at once.  Its list is already
// ascending; warp w adds the kept row (w = 0) and the 32-member segments w, w + 8, ...,
// and the eight partial sums are added in warp order.  Every order is a fixed function of
// the sorted list, so results do not depend on scheduling.
template <typename T>
__global__ void __launch_bounds__(kAggWarps * 32)
aggregate_compact_kernel(const T* __restrict__ hidden, const int32_t* __restrict__ cu_seqlens,
                         const int32_t* __restrict__ n_visual, const int32_t* __restrict__ kept_idx,
                         const int32_t* __restrict__ cu_kept, const int32_t* __restrict__ cu_seqlens_out, int B, int D,
                         int chunks, int total_out, int heavy_blocks, int mean,
                         const int32_t* __restrict__ member_count, const int32_t* __restrict__ member_off,
                         const int32_t* __restrict__ member_list, const int32_t* __restrict__ heavy_slots,
                         const int* __restrict__ n_heavy, const int4* __restrict__ row_desc, T* __restrict__ hidden_out,
                         int32_t* __restrict__ src_of_dst) {
  constexpr int kVec = Storage<T>::kVec;
  grid_dependency_enter();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float acc[kVec];
#pragma unroll
  for (int e = 0; e < kVec; ++e) acc[e] = 0.f;

  if ((int)blockIdx.x < heavy_blocks) {
    // ------------------------------------------------------------ a heavy kept token (these blocks take the longest: first in the grid)
    // (the host cannot know how many kept tokens are heavy: a fixed number of blocks walks over them)
    const int n_items = *n_heavy * chunks;
    for (int item = (int)blockIdx.x; item < n_items; item += heavy_blocks) {
    const int hi = item / chunks, ch = item - hi * chunks;
#pragma unroll
    for (int e = 0; e < kVec; ++e) acc[e] = 0.f;
    const int ks = heavy_slots[hi];                              // slot in the packed kept list
    const int b = find_segment(cu_kept, B, ks);
    const int r = ks - cu_kept[b];
    const int lo = cu_seqlens[b];
    const int row = cu_seqlens_out[b] + r;
    const int c = (ch * 32 + lane) * kVec;
    const bool live = c < D;
    const T* req = hidden + (size_t)lo * D + (live ? c : 0);
    const int pos = kept_idx[ks], cnt = member_count[ks], off = member_off[ks];
    if (warp == 0) add_raw<T>(acc, *reinterpret_cast<const uint4*>(req + (size_t)pos * D));
    for (int seg = warp; seg * 32 < cnt; seg += kAggWarps) {
      const int n = min(32, cnt - seg * 32);
      const int mine = lane < n ? member_list[off + seg * 32 + lane] : 0;
      add_rows<T>(acc, req, D, mine, n);
    }
    __shared__ float part[kAggWarps][32][Storage<T>::kVec + 1];
#pragma unroll
    for (int e = 0; e < kVec; ++e) part[warp][lane][e] = acc[e];
    __syncthreads();
    if (warp == 0 && live) {
      for (int w = 1; w < kAggWarps; ++w)
#pragma unroll
        for (int e = 0; e < kVec; ++e) acc[e] += part[w][lane][e];
      const float inv_denom = mean ? 1.0f / (float)(1 + cnt) : 1.f;
#pragma unroll
      for (int e = 0; e < kVec; ++e) acc[e] *= inv_denom;
      Storage<T>::store(hidden_out + (size_t)row * D + c, acc);
    }
    if (ch == 0 && threadIdx.x == 0) src_of_dst[row] = lo + pos;
    __syncthreads();                                            // `part` is reused by the next item
    }
    return;
  }

  // ------------------------------------------------------------ light rows: one warp per (row, group of kAggCpw chunks)
  const int groups = (chunks + kAggCpw - 1) / kAggCpw;
  const int gw = ((int)blockIdx.x - heavy_blocks) * kAggWarps + warp;
  const int row = gw / groups, cg = gw - row * groups;
  if (row >= total_out) return;                                 // whole warp
  const int4 desc = row_desc[row];                             // {source row, members (-1: copy), list offset, request's first row}
  const int cnt = desc.y, off = desc.z, lo = desc.w;
  const int pos = desc.x - lo;                                  // position in the request
  int col[kAggCpw];
  bool live[kAggCpw];
#pragma unroll
  for (int j = 0; j < kAggCpw; ++j) {
    col[j] = ((cg * kAggCpw + j) * 32 + lane) * kVec;
    live[j] = col[j] < D;
    if (!live[j]) col[j] = 0;                                   // lanes past the row end read column 0, write nothing
  }
  const T* req = hidden + (size_t)lo * D;
  T* dst = hidden_out + (size_t)row * D;
  if (cg == 0 && lane == 0) src_of_dst[row] = desc.x;

  if (cnt < 0) {                                                // prompt / response row: copy
    uint4 raw[kAggCpw];
#pragma unroll
    for (int j = 0; j < kAggCpw; ++j) raw[j] = *reinterpret_cast<const uint4*>(req + (size_t)pos * D + col[j]);
#pragma unroll
    for (int j = 0; j < kAggCpw; ++j) if (live[j]) *reinterpret_cast<uint4*>(dst + col[j]) = raw[j];
    return;
  }
  if (cnt >= kHeavy) return;                                    // a heavy block does this row
  // lane t ends up holding the t-th row to add: the kept row, then the members by ascending
  // position (distinct values, ranked by counting the smaller ones)
  const int mine = lane < cnt ? member_list[off + lane] : 0x7fffffff;
  int rank = 0;
  for (int j = 0; j < cnt; ++j) rank += __shfl_sync(0xffffffffu, mine, j) < mine ? 1 : 0;
  int ordered = pos;
  for (int j = 0; j < cnt; ++j) {
    const int v = __shfl_sync(0xffffffffu, mine, j), rj = __shfl_sync(0xffffffffu, rank, j);
    if (lane == rj + 1) ordered = v;
  }
  float accs[kAggCpw][kVec];
#pragma unroll
  for (int j = 0; j < kAggCpw; ++j)
#pragma unroll
    for (int e = 0; e < kVec; ++e) accs[j][e] = 0.f;
  const int n = cnt + 1;
  for (int i = 0; i < n; i += kAggUnroll) {                     // kAggUnroll rows x kAggCpw chunks in flight
    uint4 raw[kAggUnroll][kAggCpw];
#pragma unroll
    for (int u = 0; u < kAggUnroll; ++u) {
      const int rr = __shfl_sync(0xffffffffu, ordered, (i + u) & 31);
      if (i + u < n) {
#pragma unroll
        for (int j = 0; j < kAggCpw; ++j) raw[u][j] = *reinterpret_cast<const uint4*>(req + (size_t)rr * D + col[j]);
      }
    }
#pragma unroll
    for (int u = 0; u < kAggUnroll; ++u)
      if (i + u < n) {
#pragma unroll
        for (int j = 0; j < kAggCpw; ++j) add_raw<T>(accs[j], raw[u][j]);
      }
  }
  const float inv_denom = mean ? 1.0f / (float)(1 + cnt) : 1.f;
#pragma unroll
  for (int j = 0; j < kAggCpw; ++j)
    if (live[j]) {
#pragma unroll
      for (int e = 0; e < kVec; ++e) accs[j][e] *= inv_denom;
      Storage<T>::store(dst + col[j], accs[j]);
    }
}

}  // namespace

int launch_merge_prepare(d3tom_ctx* ctx, const MergeArgs& a, cudaStream_t s) {
  dim3 grid(ceil_div(a.max_visual, kPrepWarps), a.B);
  if (a.dt == D3TOM_FP32)
    D3TOM_CUDA_TRY(ctx, launch_serialized(prepare_rows_kernel<float>, grid, kPrepWarps * 32, 0, s,
                                          static_cast<const float*>(a.hidden), a.cu_seqlens, a.cu_vis, a.kept_idx,
                                          a.cu_kept, a.D, a.assign, ctx->best, ctx->inv_norm, ctx->inv_norm_kept,
                                          static_cast<float*>(ctx->kept_rows), ctx->n_heavy));
  else
    D3TOM_CUDA_TRY(ctx, launch_serialized(prepare_rows_kernel<__nv_bfloat16>, grid, kPrepWarps * 32, 0, s,
                                          static_cast<const __nv_bfloat16*>(a.hidden), a.cu_seqlens, a.cu_vis,
                                          a.kept_idx, a.cu_kept, a.D, a.assign, ctx->best, ctx->inv_norm,
                                          ctx->inv_norm_kept, static_cast<__nv_bfloat16*>(ctx->kept_rows), ctx->n_heavy));
  return D3TOM_OK;
}

int launch_sim_simt(d3tom_ctx* ctx, const MergeArgs& a, cudaStream_t s) {
  dim3 grid(a.max_visual, a.B);
  if (a.dt == D3TOM_FP32)
    D3TOM_CUDA_TRY(ctx, launch_serialized(sim_simt_kernel<float>, grid, 256, 0, s, static_cast<const float*>(a.hidden),
                                          static_cast<const float*>(ctx->kept_rows), a.cu_seqlens, a.cu_vis, a.cu_kept,
                                          a.assign, ctx->inv_norm, ctx->inv_norm_kept, a.D, a.max_kept, ctx->best,
                                          a.sim_debug));
  else
    D3TOM_CUDA_TRY(ctx, launch_serialized(sim_simt_kernel<__nv_bfloat16>, grid, 256, 0, s,
                                          static_cast<const __nv_bfloat16*>(a.hidden),
                                          static_cast<const __nv_bfloat16*>(ctx->kept_rows), a.cu_seqlens, a.cu_vis,
                                          a.cu_kept, a.assign, ctx->inv_norm, ctx->inv_norm_kept, a.D, a.max_kept,
                                          ctx->best, a.sim_debug));
  return D3TOM_OK;
}

int launch_merge_finish(d3tom_ctx* ctx, const MergeArgs& a, cudaStream_t s) {
  // (the attribute belongs to the current device: set on every call, a process may drive several GPUs)
  D3TOM_CUDA_TRY(ctx, cudaFuncSetAttribute(members_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           kMemberSmemSlots * (int)sizeof(int) + kBitmapBytes));
  // shared memory of the members kernel: counters when they fit, then one position bitmap per sorting warp
  const int ctr_ints = a.max_kept <= kMemberSmemSlots ? a.max_kept : 0;
  const int words = ceil_div(a.max_visual > 0 ? a.max_visual : 1, 32);
  int bitmap_warps = kBitmapBytes / (words * 4);
  if (bitmap_warps > kMemberThreads / 32) bitmap_warps = kMemberThreads / 32;
  if (bitmap_warps < 1) return D3TOM_ERR_UNSUPPORTED;              // more than 512 Ki visual tokens in one request
  const size_t smem = (size_t)ctr_ints * sizeof(int) + (size_t)bitmap_warps * words * 4;
  // the count of heavy kept tokens is zeroed by the prepare kernel, which runs whenever there are visual tokens
  if (a.max_visual <= 0) D3TOM_CUDA_TRY(ctx, cudaMemsetAsync(ctx->n_heavy, 0, sizeof(int), s));
  D3TOM_CUDA_TRY(ctx, launch_serialized(members_kernel, a.B, kMemberThreads, smem, s, a.cu_vis, a.cu_kept, ctx->best, a.assign,
                                        a.member_count, ctx->member_off, ctx->member_cursor, ctx->member_list,
                                        ctx->heavy_slots, ctx->n_heavy, ctr_ints, bitmap_warps, a.cu_seqlens,
                                        a.cu_seqlens_out, a.kept_idx, ctx->row_desc));
  return launch_merge_aggregate(ctx, a, s);
}

// aggregation + compaction of a.hidden into a.hidden_out with the member lists the context holds
// (may run again on another tensor of the same rows: the V cache after the K cache)
int launch_merge_aggregate(d3tom_ctx* ctx, const MergeArgs& a, cudaStream_t s) {
  const int mean = a.mode == D3TOM_AGG_MEAN ? 1 : 0;
  if (a.total_out <= 0) return D3TOM_OK;
  {   // the streaming pipeline takes every row size it supports; the kernel below is the general one
    const int st = launch_merge_aggregate_stream(ctx, a, s);
    if (st != D3TOM_ERR_UNSUPPORTED) return st;
  }
  const int vec = a.dt == D3TOM_FP32 ? 4 : 8;
  const int chunks = ceil_div(a.D, 32 * vec);                       // 512-byte chunks per row
  const long long warps = (long long)a.total_out * ceil_div(chunks, kAggCpw);
  const int light_blocks = (int)((warps + kAggWarps - 1) / kAggWarps);
  // at most (pruned tokens) / kHeavy kept tokens can be heavy; the blocks beyond the actual number leave at once
  const int max_heavy = (a.total_tokens - a.total_out) / kHeavy;
  int heavy_blocks = max_heavy * chunks;
  if (heavy_blocks > ctx->sm_count) heavy_blocks = ctx->sm_count;
  const int blocks = light_blocks + heavy_blocks;
  if (a.dt == D3TOM_FP32)
    D3TOM_CUDA_TRY(ctx, launch_serialized(aggregate_compact_kernel<float>, blocks, kAggWarps * 32, 0, s,
        static_cast<const float*>(a.hidden), a.cu_seqlens, a.n_visual, a.kept_idx, a.cu_kept, a.cu_seqlens_out, a.B, a.D,
        chunks, a.total_out, heavy_blocks, mean, a.member_count, ctx->member_off, ctx->member_list, ctx->heavy_slots,
        ctx->n_heavy, ctx->row_desc, static_cast<float*>(a.hidden_out), a.src_of_dst));
  else
    D3TOM_CUDA_TRY(ctx, launch_serialized(aggregate_compact_kernel<__nv_bfloat16>, blocks, kAggWarps * 32, 0, s,
        static_cast<const __nv_bfloat16*>(a.hidden), a.cu_seqlens, a.n_visual, a.kept_idx, a.cu_kept, a.cu_seqlens_out,
        a.B, a.D, chunks, a.total_out, heavy_blocks, mean, a.member_count, ctx->member_off, ctx->member_list,
        ctx->heavy_slots, ctx->n_heavy, ctx->row_desc, static_cast<__nv_bfloat16*>(a.hidden_out), a.src_of_dst));
  return D3TOM_OK;
}
