// Keep / merge partition (Sec. 3.2.1; Algorithm 1, TopK): per request the k
// visual tokens of highest importance under the total order (score descending,
// index ascending), emitted ascending by position.
//
// One CTA per request.  Requests of up to 8192 visual tokens keep their keys in
// registers (select_reg_kernel, below); longer ones use select_kernel: the scores
// are mapped to order-preserving 32-bit keys and staged in shared memory.  A most-significant-digit radix select (4 passes
// of 8 bits, warp-aggregated histogram updates) finds the key T of rank k and
// how many keys equal to T still belong to the kept set; the equal keys of
// lowest index are taken.  A final ordered pass writes the mask and the
// ascending index list with a block-wide prefix sum, so the result does not
// depend on thread scheduling: it is bit-exact and reproducible.
#include "common.cuh"

namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;

struct SelectShared {
  unsigned hist[256];
  unsigned warp_tot[kWarps];
  unsigned prefix, remaining, carry;
};

template <bool kKeysInSmem>
__global__ void __launch_bounds__(kThreads)
select_kernel(const float* __restrict__ importance, const int32_t* __restrict__ cu_vis,
              const int32_t* __restrict__ keep_count, const int32_t* __restrict__ cu_kept,
              int32_t* __restrict__ kept_idx, uint8_t* __restrict__ keep_mask) {
  extern __shared__ uint32_t keys_s[];
  __shared__ SelectShared sh;
  grid_dependency_enter();
  const int b = blockIdx.x;
  const int v0 = cu_vis[b], V = cu_vis[b + 1] - v0;
  const float* sc = importance + v0;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (V <= 0) return;
  int k = keep_count[b];
  k = k < 0 ? 0 : (k > V ? V : k);          // as select_reg_kernel: a count outside [0, V] cannot leave the segment

  if (kKeysInSmem) {
    for (int j = tid; j < V; j += kThreads) keys_s[j] = ordered_key(sc[j]);
  }
  auto key_at = [&](int j) -> uint32_t { return kKeysInSmem ? keys_s[j] : ordered_key(sc[j]); };
  if (tid == 0) { sh.prefix = 0u; sh.remaining = (unsigned)k; }
  __syncthreads();

  // ---- radix select of the k-th largest key ----
  uint32_t mask = 0u;
  const int v_round = ((V + 31) / 32) * 32;
  for (int pass = 0; pass < (k > 0 ? 4 : 0); ++pass) {   // k = 0: nothing is kept, there is no key of rank k
    const int shift = 24 - 8 * pass;
    for (int d = tid; d < 256; d += kThreads) sh.hist[d] = 0u;
    __syncthreads();
    const uint32_t prefix = sh.prefix;
    for (int j = tid; j < v_round; j += kThreads) {   // whole warps iterate together
      uint32_t digit = 0xffffffffu;
      if (j < V) {
        const uint32_t key = key_at(j);
        if ((key & mask) == prefix) digit = (key >> shift) & 255u;
      }
      const unsigned peers = __match_any_sync(0xffffffffu, digit);
      if (digit != 0xffffffffu && lane == __ffs(peers) - 1) atomicAdd(&sh.hist[digit], __popc(peers));
    }
    __syncthreads();
    if (warp == 0) {
      // lane owns digits 255-8*lane .. 248-8*lane (descending); find where the
      // running count from the top reaches `remaining`
      unsigned cnt[8], mine = 0u;
#pragma unroll
      for (int i = 0; i < 8; ++i) { cnt[i] = sh.hist[255 - (lane * 8 + i)]; mine += cnt[i]; }
      unsigned incl = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        unsigned t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
      }
      const unsigned excl = incl - mine;
      const unsigned rem = sh.remaining;
      __syncwarp();
      if (excl < rem && rem <= incl) {          // exactly one lane
        unsigned run = excl;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (run < rem && rem <= run + cnt[i]) {
            sh.prefix = prefix | ((uint32_t)(255 - (lane * 8 + i)) << shift);
            sh.remaining = rem - run;
          }
          run += cnt[i];
        }
      }
    }
    mask |= 255u << shift;
    __syncthreads();
  }
  const uint32_t T = sh.prefix;          // key of rank k
  const unsigned need_eq = k > 0 ? sh.remaining : 0u; // how many keys == T are kept (lowest indices first)

  // ---- ordered output pass ----
  if (tid == 0) sh.carry = 0u;           // packed running totals: (greater << 16 | equal) per chunk, 32-bit each below
  __shared__ unsigned run_gt, run_eq;
  if (tid == 0) { run_gt = 0u; run_eq = 0u; }
  __syncthreads();
  int32_t* out = kept_idx + cu_kept[b];
  uint8_t* mk = keep_mask + v0;
  for (int base = 0; base < V; base += kThreads) {
    const int j = base + tid;
    uint32_t key = 0u;
    bool gt = false, eq = false;
    if (j < V && k > 0) { key = key_at(j); gt = key > T; eq = key == T; }
    // packed per-thread counts: high 16 bits greater, low 16 bits equal (chunk <= 1024)
    unsigned val = (gt ? 0x10000u : 0u) | (eq ? 1u : 0u);
    unsigned incl = val;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      unsigned t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    if (lane == 31) sh.warp_tot[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      unsigned w = sh.warp_tot[lane];
      unsigned winc = w;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        unsigned t = __shfl_up_sync(0xffffffffu, winc, o);
        if (lane >= o) winc += t;
      }
      sh.warp_tot[lane] = winc - w;       // exclusive over warps
      if (lane == 31) sh.carry = winc;    // chunk total
    }
    __syncthreads();
    const unsigned excl = sh.warp_tot[warp] + incl - val;
    const unsigned gt_before = run_gt + (excl >> 16);
    const unsigned eq_before = run_eq + (excl & 0xffffu);
    if (j < V) {
      const bool keep = gt || (eq && eq_before < need_eq);
      mk[j] = keep ? 1 : 0;
      if (keep) out[gt_before + min(eq_before, need_eq)] = j;
    }
    __syncthreads();
    if (tid == 0) { run_gt += sh.carry >> 16; run_eq += sh.carry & 0xffffu; }
    __syncthreads();
  }
}

// Requests of up to 1024 x IPT visual tokens: every thread keeps IPT CONSECUTIVE keys in registers, so the ordered
// output needs a single block-wide prefix sum and the keys are read once.  The radix select takes three passes of
// 12, 10 and 10 bits; the wide first digit (sign, exponent, three mantissa bits) spreads scores that share their
// leading bits over many bins, after which few keys remain candidates.  A thread owns the same bins in every pass
// and clears them as it reads them, which saves the barrier of a separate clearing phase.
constexpr int kRegBinsMax = 4096;

template <int IPT>
__global__ void __launch_bounds__(kThreads)
select_reg_kernel(const float* __restrict__ importance, const int32_t* __restrict__ cu_vis,
                  const int32_t* __restrict__ keep_count, const int32_t* __restrict__ cu_kept,
                  int32_t* __restrict__ kept_idx, uint8_t* __restrict__ keep_mask) {
  __shared__ unsigned hist[kRegBinsMax];
  __shared__ unsigned warp_tot[kWarps];
  __shared__ unsigned sh_prefix, sh_remaining;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int d = tid; d < kRegBinsMax; d += kThreads) hist[d] = 0u;      // on-chip only: before the dependency wait
  grid_dependency_enter();
  const int b = blockIdx.x;
  const int v0 = cu_vis[b], V = cu_vis[b + 1] - v0;
  if (V <= 0) return;
  int k = keep_count[b];
  k = k < 0 ? 0 : (k > V ? V : k);
  const float* sc = importance + v0;
  const int j0 = tid * IPT;
  uint32_t key[IPT];
#pragma unroll
  for (int i = 0; i < IPT; ++i) key[i] = (j0 + i < V) ? ordered_key(sc[j0 + i]) : 0u;
  if (tid == 0) { sh_prefix = 0u; sh_remaining = (unsigned)k; }
  __syncthreads();

  // inclusive prefix sum of `val` over the block in thread order; every warp scans the 32 warp totals itself
  auto block_scan = [&](unsigned val, unsigned& total) -> unsigned {
    unsigned incl = val;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    unsigned w = warp_tot[lane], winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned t = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += t;
    }
    total = __shfl_sync(0xffffffffu, winc, 31);
    const unsigned before = __shfl_sync(0xffffffffu, winc - w, warp);
    return incl + before;
  };

  uint32_t mask = 0u;
  if (k > 0) {
#pragma unroll
    for (int pass = 0; pass < 3; ++pass) {
      const int bits = pass == 0 ? 12 : 10;
      const int shift = pass == 0 ? 20 : (pass == 1 ? 10 : 0);
      const int bpt = (1 << bits) / kThreads;              // bins per thread: 4, 1, 1
      const uint32_t prefix = sh_prefix;
      const unsigned rem = sh_remaining;
#pragma unroll
      for (int i = 0; i < IPT; ++i)
        if (j0 + i < V && (key[i] & mask) == prefix) atomicAdd(&hist[(key[i] >> shift) & ((1u << bits) - 1u)], 1u);
      __syncthreads();
      // thread t owns the bins (bins - 1 - bpt * t) downwards: the running count from the top digit
      const int top = (1 << bits) - 1 - bpt * tid;
      unsigned cnt[4], mine = 0u;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        cnt[i] = 0u;
        if (i < bpt) { cnt[i] = hist[top - i]; mine += cnt[i]; }
      }
      if (pass == 0) {                                      // the 4096 bins are clear again for the next passes
#pragma unroll
        for (int i = 0; i < 4; ++i) hist[top - i] = 0u;
      } else {
        hist[top] = 0u;
      }
      unsigned total;
      const unsigned incl = block_scan(mine, total);
      const unsigned excl = incl - mine;
      if (excl < rem && rem <= incl) {                      // exactly one thread: the digit of the key of rank k
        unsigned run = excl;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          if (i < bpt && run < rem && rem <= run + cnt[i]) {
            sh_prefix = prefix | ((uint32_t)(top - i) << shift);
            sh_remaining = rem - run;
          }
          run += cnt[i];
        }
      }
      mask |= ((1u << bits) - 1u) << shift;
      __syncthreads();
    }
  }
  const uint32_t T = sh_prefix;            // key of rank k
  const unsigned need_eq = k > 0 ? sh_remaining : 0u;    // keys equal to T that are kept: the lowest positions

  // ---- ordered output: one prefix sum over the per-thread counts (greater << 16 | equal)
  unsigned val = 0u;
  if (k > 0) {
#pragma unroll
    for (int i = 0; i < IPT; ++i)
      if (j0 + i < V) val += (key[i] > T ? 0x10000u : 0u) + (key[i] == T ? 1u : 0u);
  }
  __syncthreads();                          // warp_tot is reused
  unsigned total;
  const unsigned incl = block_scan(val, total);
  unsigned gt_before = (incl - val) >> 16, eq_before = (incl - val) & 0xffffu;
  int32_t* out = kept_idx + cu_kept[b];
  uint8_t* mk = keep_mask + v0;
#pragma unroll
  for (int i = 0; i < IPT; ++i) {
    const int j = j0 + i;
    if (j < V) {
      const bool gt = k > 0 && key[i] > T, eq = k > 0 && key[i] == T;
      const bool keep = gt || (eq && eq_before < need_eq);
      mk[j] = keep ? 1 : 0;
      if (keep) out[gt_before + min(eq_before, need_eq)] = j;
      gt_before += gt ? 1u : 0u;
      eq_before += eq ? 1u : 0u;
    }
  }
}

}  // namespace

int launch_select(d3tom_ctx* ctx, const float* importance, const int32_t* cu_vis, const int32_t* keep_count,
                  const int32_t* cu_kept, int B, int max_visual, int32_t* kept_idx, uint8_t* keep_mask,
                  cudaStream_t s) {
  const size_t smem = (size_t)max_visual * sizeof(uint32_t);
  if (max_visual <= 8 * kThreads) {           // keys in registers
    if (max_visual <= kThreads) D3TOM_CUDA_TRY(ctx, launch_serialized(select_reg_kernel<1>, B, kThreads, 0, s, importance, cu_vis, keep_count, cu_kept, kept_idx, keep_mask));
    else if (max_visual <= 2 * kThreads) D3TOM_CUDA_TRY(ctx, launch_serialized(select_reg_kernel<2>, B, kThreads, 0, s, importance, cu_vis, keep_count, cu_kept, kept_idx, keep_mask));
    else if (max_visual <= 4 * kThreads) D3TOM_CUDA_TRY(ctx, launch_serialized(select_reg_kernel<4>, B, kThreads, 0, s, importance, cu_vis, keep_count, cu_kept, kept_idx, keep_mask));
    else D3TOM_CUDA_TRY(ctx, launch_serialized(select_reg_kernel<8>, B, kThreads, 0, s, importance, cu_vis, keep_count, cu_kept, kept_idx, keep_mask));
  } else if (smem <= 160 * 1024) {
    // (the attribute belongs to the current device: set on every call, a process may drive several GPUs)
    D3TOM_CUDA_TRY(ctx, cudaFuncSetAttribute(select_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024));
    D3TOM_CUDA_TRY(ctx, launch_serialized(select_kernel<true>, B, kThreads, smem, s, importance, cu_vis, keep_count, cu_kept, kept_idx, keep_mask));
  } else {
    D3TOM_CUDA_TRY(ctx, launch_serialized(select_kernel<false>, B, kThreads, 0, s, importance, cu_vis, keep_count, cu_kept, kept_idx, keep_mask));
  }
  D3TOM_LAUNCH_CHECK(ctx);
  return D3TOM_OK;
}
