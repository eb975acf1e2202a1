// Keep / merge partition (Sec. 3.2.1; Algorithm 1, TopK): per request the k
// visual tokens of highest importance under the total order (score descending,
// index ascending), emitted ascending by position.
//
// One CTA per request.  The scores are mapped to order-preserving 32-bit keys
// and staged in shared memory.  A most-significant-digit radix select (4 passes
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
  const int k = keep_count[b];
  const float* sc = importance + v0;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (V <= 0) return;

  if (kKeysInSmem) {
    for (int j = tid; j < V; j += kThreads) keys_s[j] = ordered_key(sc[j]);
  }
  auto key_at = [&](int j) -> uint32_t { return kKeysInSmem ? keys_s[j] : ordered_key(sc[j]); };
  if (tid == 0) { sh.prefix = 0u; sh.remaining = (unsigned)k; }
  __syncthreads();

  // ---- radix select of the k-th largest key ----
  uint32_t mask = 0u;
  const int v_round = ((V + 31) / 32) * 32;
  for (int pass = 0; pass < 4; ++pass) {
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
  const unsigned need_eq = sh.remaining; // how many keys == T are kept (lowest indices first)

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
    if (j < V) { key = key_at(j); gt = key > T; eq = key == T; }
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

}  // namespace

int launch_select(d3tom_ctx* ctx, const float* importance, const int32_t* cu_vis, const int32_t* keep_count,
                  const int32_t* cu_kept, int B, int max_visual, int32_t* kept_idx, uint8_t* keep_mask,
                  cudaStream_t s) {
  const size_t smem = (size_t)max_visual * sizeof(uint32_t);
  if (smem <= 160 * 1024) {
    // (the attribute belongs to the current device: set on every call, a process may drive several GPUs)
    D3TOM_CUDA_TRY(ctx, cudaFuncSetAttribute(select_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024));
    D3TOM_CUDA_TRY(ctx, launch_serialized(select_kernel<true>, B, kThreads, smem, s, importance, cu_vis, keep_count, cu_kept, kept_idx, keep_mask));
  } else {
    D3TOM_CUDA_TRY(ctx, launch_serialized(select_kernel<false>, B, kThreads, 0, s, importance, cu_vis, keep_count, cu_kept, kept_idx, keep_mask));
  }
  D3TOM_LAUNCH_CHECK(ctx);
  return D3TOM_OK;
}
