// bf16 x bf16 -> fp32 "NT" GEMM on tcgen05 tensor cores, C[m, n] = sum_k A[m, k] B[n, k],
// with four fused epilogues:
//
//   kEpiProj  the Q,K,V projection of a post-merge layer (Sec. 3.2.1, Q = H W_Q,
//             K = H W_K): rounds to bf16 and writes the tile into q, k or v.
//   kEpiSim   the similarity step of the merge (Sec. 3.2.2, arg max of the cosine
//             over the kept set): scales the dot products by the two inverse norms
//             and folds every pruned row's candidates into its packed 64-bit
//             running maximum, so the (V x k) similarity matrix never reaches HBM.
//   kEpiLinear  y = residual + x W^T rounded to bf16: the attention output projection and the
//             down projection of the feed-forward network (Algorithm 1, FFN_l; the fourth
//             d x d matrix of the 4nd^2 term and the third d x m matrix of the 3ndm term).
//   kEpiGateUp  the first two d x m matrices of the feed-forward network in one pass: a 256-wide
//             tile is 128 gate rows and the 128 up rows of the same features, and the epilogue
//             writes act = silu(gate) * up, so neither product reaches HBM.
//
// Persistent CTAs (one per SM) walk over the 128 x BN output tiles, M fastest so that the
// BN x K operand stays hot in L2 while the M tiles that share it are computed.  Warps 0
// and 6 stream 128x64 / BNx64 operand tiles with TMA into a ring of 128-byte-swizzled
// stages and keep streaming across tile boundaries; one thread of warp 1 issues tcgen05.mma
// (M = 128, N = BN, K = 16) into one of TWO TMEM accumulators; warps 2..5 read the other
// accumulator back with tcgen05.ld (one row per thread) and run the epilogue meanwhile.
#include "common.cuh"
#include "ptx.cuh"

namespace {

constexpr int kBM = 128, kBK = 64;
constexpr int kGemmThreads = 224;      // warps: 0 A loads, 1 MMA, 2..5 epilogue, 6 B loads

enum { kEpiProj = 0, kEpiSim = 1, kEpiLinear = 2, kEpiGateUp = 3 };
constexpr int kMaxKSplits = 4;        // K slices per tile at most when the last slice to arrive adds them all
constexpr int kCoopSlices = 16;       // K slices per similarity tile at most when every slice adds its own share of the columns (8 or 16)

struct GemmParams {
  int num_k_blocks;           // K / 64
  int m_tiles, n_tiles, batch;   // tile grid (per request for the similarity); tiles outside a request are skipped
  int k_splits;               // tiles from `full_tiles` on have their K range cut into this many work units
  int full_tiles;             // the first tiles of the walk are whole work units (0: every tile is cut)
  float* split_ws;            // [(tiles - full_tiles) * k_splits][BN][128] fp32 partial tiles (column-major: coalesced per warp)
  int* split_counters;        // [tiles] parts done; zero between launches
  int coop;                   // similarity, few tiles: 8 or 16 slices per tile, all resident; each reduces BN / k_splits columns
  // projection
  __nv_bfloat16* out[3];      // q, k, v
  int out_rows;               // total tokens
  int out_cols;               // D
  // linear / gate-up: rows are out_rows
  __nv_bfloat16* lin_out;     // [out_rows, ld_out]
  const __nv_bfloat16* residual;   // [out_rows, ld_out] or null (linear only; may be lin_out itself)
  int ld_out;                 // N of the linear layer; m for the gate-up pass
  int up_row_offset;          // gate-up: row of the weight matrix where the up matrix starts (m)
  // similarity
  const int32_t* cu_seqlens; const int32_t* cu_vis; const int32_t* cu_kept; const int32_t* assign;
  const float* inv_norm; const float* inv_norm_kept;
  unsigned long long* best; float* sim_debug; int max_kept;
  int* dev_status;
};

// Work unit u of the walk: tile t, K slice sp of nsp.  Whole tiles come first, so the cut tiles are the last
// (incomplete) round over the SMs: its few tiles are spread over all SMs instead of occupying a full tile time.
struct Unit {
  int t, sp, nsp, kb0, kb1;
  __device__ __forceinline__ void set(const GemmParams& p, int u) {
    if (u < p.full_tiles) { t = u; sp = 0; nsp = 1; }
    else { const int r = u - p.full_tiles; t = p.full_tiles + r / p.k_splits; sp = r - (t - p.full_tiles) * p.k_splits; nsp = p.k_splits; }
    kb0 = sp * p.num_k_blocks / nsp; kb1 = (sp + 1) * p.num_k_blocks / nsp;
  }
};

// MT = 1: a CTA tile is 128 x BN with two accumulators (the epilogue of a tile overlaps the main loop of the next).
// MT = 2: a CTA tile is 256 x BN: two 128-row A tiles share every B tile in shared memory, so a k-block moves
//         32 + 32 KB for 1024 tensor cycles (62 B/clk) where the 128 x 256 tile moves 16 + 32 KB for 512 (96 B/clk);
//         the dense layers are bound by what the SMs can pull out of L2, so this is the faster shape whenever there
//         are enough rows.  Both accumulators belong to the one tile (no overlap of epilogue and main loop).
template <int BN, int MT = 1> struct GemmSmem {
  static constexpr int kABytes = MT * kBM * kBK * 2, kBBytes = BN * kBK * 2;
  static constexpr int kStages = (MT == 2) ? 3 : (BN == 256 ? 4 : (BN == 192 ? 5 : 6));   // as many as fit in 227 KB
  static constexpr int kAccStride = BN <= 128 ? 128 : 256;              // TMEM columns between the two accumulators
  static constexpr int kBytes = kStages * (kABytes + kBBytes) + 1024 /*alignment slack*/ + 256 /*barriers*/ + BN * 4;
};

// Where tile `t` of the walk lies: rows of A, rows of B, and for the similarity the request
// it belongs to.  Returns false for a tile of the bounding grid that a request does not reach.
template <int BN, int EPI, int MT = 1>
struct TileCoord {
  int m0, n0, a_row, b_row, b, Vb, kb, v0, k0;
  const int* prefix;      // similarity with a ragged batch: tiles before request b (shared memory), or null
  __device__ __forceinline__ bool set(const GemmParams& p, int t) {
    int mi, ni;
    if (EPI == kEpiSim && prefix != nullptr) {
      // only the tiles that exist are numbered: request b owns [prefix[b], prefix[b + 1]), M fastest
      b = 0;
      while (prefix[b + 1] <= t) ++b;
      const int local = t - prefix[b];
      v0 = p.cu_vis[b]; Vb = p.cu_vis[b + 1] - v0;
      k0 = p.cu_kept[b]; kb = p.cu_kept[b + 1] - k0;
      const int mt = (Vb + kBM - 1) / kBM;
      mi = local % mt; ni = local / mt;
      m0 = mi * kBM; n0 = ni * BN;
      a_row = p.cu_seqlens[b] + m0;
      b_row = k0 + n0;
      return true;
    }
    mi = t % p.m_tiles;
    const int rest = t / p.m_tiles;
    ni = rest % p.n_tiles;
    b = rest / p.n_tiles;
    // (a gate-up tile covers BN / 2 output features: its B rows are 128 gate rows and 128 up rows)
    m0 = mi * (MT * kBM); n0 = ni * (EPI == kEpiGateUp ? BN / 2 : BN); a_row = m0; b_row = n0;
    Vb = kb = v0 = k0 = 0;
    if (EPI == kEpiSim) {
      v0 = p.cu_vis[b]; Vb = p.cu_vis[b + 1] - v0;
      k0 = p.cu_kept[b]; kb = p.cu_kept[b + 1] - k0;
      if (m0 >= Vb || n0 >= kb || kb >= Vb) return false;   // nothing pruned in this request, or outside it
      a_row = p.cu_seqlens[b] + m0;
      b_row = k0 + n0;
    }
    return true;
  }
};

constexpr int kMaxPrefixBatch = 64;     // ragged batches up to this many requests number only the tiles that exist

template <int BN, int EPI, int MT = 1>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b, GemmParams p) {
  static_assert(MT == 1 || (BN >= 224 && BN % 32 == 0 && EPI != kEpiSim), "the 256-row tile serves the dense layers at 224 or 256 columns");
  using S = GemmSmem<BN, MT>;
  constexpr int kStages = S::kStages;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* a_s = smem;
  uint8_t* b_s = smem + kStages * S::kABytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kStages * (S::kABytes + S::kBBytes));
  uint64_t* empty = full + kStages;
  uint64_t* acc_full = empty + kStages;       // [2]
  uint64_t* acc_empty = acc_full + 2;         // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* ink_s = reinterpret_cast<float*>(smem + kStages * (S::kABytes + S::kBBytes) + 256);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // barriers and tensor memory first (on-chip only), then wait for the kernels before this one
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { ptx::mbar_init(&full[s], 2); ptx::mbar_init(&empty[s], 1); }   // A and B loaders
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(&acc_full[i], 1); ptx::mbar_init(&acc_empty[i], 4); }   // one arrival per epilogue warp
    *abort_flag = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 2) { ptx::tmem_alloc(tmem_slot, 2 * S::kAccStride); ptx::tmem_relinquish(); }
  grid_dependency_wait();
  grid_dependency_release();
  int total_units = p.full_tiles + (p.m_tiles * p.n_tiles * p.batch - p.full_tiles) * p.k_splits;   // a unit = one tile, or one K slice of a tile
  // A batch of requests of different sizes: the bounding grid (batch x largest request) is mostly holes, and
  // walking it leaves the SMs unevenly loaded.  Every CTA numbers the tiles that exist (a prefix over requests).
  __shared__ int tile_prefix[kMaxPrefixBatch + 1];
  const bool use_prefix = EPI == kEpiSim && p.batch > 1 && p.batch <= kMaxPrefixBatch;
  if (use_prefix) {
    if (threadIdx.x == 0) {
      int run = 0;
      for (int b = 0; b < p.batch; ++b) {
        tile_prefix[b] = run;
        const int Vb = p.cu_vis[b + 1] - p.cu_vis[b], kb = p.cu_kept[b + 1] - p.cu_kept[b];
        if (kb < Vb) run += ((Vb + kBM - 1) / kBM) * ((kb + BN - 1) / BN);
      }
      tile_prefix[p.batch] = run;
    }
  }

  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  if (use_prefix) total_units = tile_prefix[p.batch] * p.k_splits;      // (the similarity cuts every tile or none)
  const uint32_t tmem_base = *tmem_slot;
  TileCoord<BN, EPI, MT> tc;
  tc.prefix = use_prefix ? tile_prefix : nullptr;

  if (warp == 0 || warp == 6) {
    // ------------------------------------------------------------ TMA producers: warp 0 streams A, warp 6 streams B
    // (issuing a load and its barrier traffic costs the issuing thread a few hundred cycles per
    // k-block; two threads keep ahead of 128 x 192 tiles, one does not)
    if (lane == 0) {
      const bool is_a = warp == 0;
      const CUtensorMap* tm = is_a ? &tmap_a : &tmap_b;
      uint8_t* ring = is_a ? a_s : b_s;
      const int stage_bytes = is_a ? S::kABytes : S::kBBytes;
      ptx::prefetch_tensormap(tm);
      int it = 0;                                   // k-blocks loaded so far, over all tiles
      bool ok = true;
      Unit un;
      for (int u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
        un.set(p, u);
        if (!tc.set(p, un.t)) continue;
        const int row0 = is_a ? tc.a_row : tc.b_row;
        for (int kbk = un.kb0; kbk < un.kb1; ++kbk, ++it) {
          const int s = it % kStages;
          ok = ptx::mbar_wait(&empty[s], ((it / kStages) & 1) ^ 1, abort_flag, p.dev_status);
          if (!ok) break;
          ptx::mbar_arrive_expect_tx(&full[s], stage_bytes);
          if (EPI == kEpiGateUp && !is_a) {        // two boxes of BN / 2 rows: gate rows, then the up rows of the same features
            ptx::tma_load_2d(ring + s * stage_bytes, tm, &full[s], kbk * kBK, row0);
            ptx::tma_load_2d(ring + s * stage_bytes + stage_bytes / 2, tm, &full[s], kbk * kBK, p.up_row_offset + row0);
          } else {
            ptx::tma_load_2d(ring + s * stage_bytes, tm, &full[s], kbk * kBK, row0);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = ptx::idesc_bf16_f32(kBM, BN, 0, 0);
      const ptx::SmemDesc a_desc0 = ptx::smem_desc_kmajor_sw128(ptx::smem_u32(a_s));
      const ptx::SmemDesc b_desc0 = ptx::smem_desc_kmajor_sw128(ptx::smem_u32(b_s));
      int it = 0, lt = 0;                           // k-blocks and tiles consumed so far
      bool ok = true;
      Unit un;
      for (int u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
        un.set(p, u);
        if (!tc.set(p, un.t)) continue;
        const int kb0 = un.kb0, kb1 = un.kb1;
        const int buf = MT == 2 ? 0 : (lt & 1);               // (a 256-row tile owns both accumulators)
        const uint32_t acc_use = MT == 2 ? (uint32_t)lt : (uint32_t)(lt >> 1);   // how often this buffer has been used
        ok = ptx::mbar_wait(&acc_empty[buf], (acc_use & 1) ^ 1, abort_flag, p.dev_status);   // epilogue done with it
        if (!ok) break;
        ptx::tc_fence_after_sync();
        const uint32_t tmem_acc = tmem_base + (uint32_t)buf * S::kAccStride;
        for (int kbk = kb0; kbk < kb1; ++kbk, ++it) {
          const int s = it % kStages;
          ok = ptx::mbar_wait(&full[s], (it / kStages) & 1, abort_flag, p.dev_status);
          if (!ok) break;
          ptx::tc_fence_after_sync();
          const ptx::SmemDesc ad = ptx::smem_desc_advance(a_desc0, s * S::kABytes), bd = ptx::smem_desc_advance(b_desc0, s * S::kBBytes);
#pragma unroll
          for (int kk = 0; kk < kBK / 16; ++kk) {
            ptx::mma_ss(tmem_acc, ptx::smem_desc_advance(ad, kk * 32), ptx::smem_desc_advance(bd, kk * 32), idesc,
                        (kbk > kb0 || kk > 0) ? 1u : 0u);
            if (MT == 2)   // rows 128..255 of the A stage against the same B tile, into the second accumulator
              ptx::mma_ss(tmem_acc + S::kAccStride, ptx::smem_desc_advance(ad, kBM * kBK * 2 + kk * 32),
                          ptx::smem_desc_advance(bd, kk * 32), idesc, (kbk > kb0 || kk > 0) ? 1u : 0u);
          }
          ptx::mma_commit(&empty[s]);     // frees the stage once these MMAs have read it
        }
        if (ok) ptx::mma_commit(&acc_full[buf]);
        ++lt;
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue: warp w may touch TMEM lanes 32*(w%4) .. +31
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;           // row of the tile owned by this thread
    const int et = threadIdx.x - 64;               // 0..127 among the epilogue threads
    int lt = 0;
    __shared__ int s_prev;
    Unit un;
    for (int u = blockIdx.x; u < total_units; u += gridDim.x) {
      un.set(p, u);
      const int t = un.t, sp = un.sp;
      if (!tc.set(p, t)) continue;
      const int buf = MT == 2 ? 0 : (lt & 1);
      const uint32_t acc_use = MT == 2 ? (uint32_t)lt : (uint32_t)(lt >> 1);
      if (EPI == kEpiSim) {
        // inverse norms of this tile's kept rows; the four epilogue warps share them (named barrier 1)
        asm volatile("bar.sync 1, 128;" ::: "memory");          // everyone is done with the previous tile's values
        for (int j = et; j < BN; j += 128) ink_s[j] = (tc.n0 + j < tc.kb) ? p.inv_norm_kept[tc.k0 + tc.n0 + j] : 0.f;
        asm volatile("bar.sync 1, 128;" ::: "memory");
      }
      const bool ok = __all_sync(0xffffffffu, ptx::mbar_wait(&acc_full[buf], acc_use & 1, abort_flag, p.dev_status));
      if (!ok) break;
      ptx::tc_fence_after_sync();
      uint32_t t_row = tmem_base + (uint32_t)buf * S::kAccStride + ((uint32_t)(quarter * 32) << 16);
      int m_base = tc.m0;                                       // first row of the 128-row half in hand
      // A tile whose K range is cut into slices on different SMs: every unit writes its partial sums out
      // (column-major, so a warp's 32 rows are one 128-byte line); the unit that completes the tile (a
      // counter, left at zero again) adds the parts in the order of the K slices and runs the epilogue on
      // the sums: same values whichever unit comes last.
      const bool split = un.nsp > 1;
      const bool coop = EPI == kEpiSim && p.coop != 0;
      const int ws_tile = t - p.full_tiles;                     // cut tiles are numbered from zero in the workspace
      bool last = true;
      if (split) {
        float* part = p.split_ws + (size_t)(ws_tile * un.nsp + sp) * BN * kBM;
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
          uint32_t r[32];
          ptx::tmem_ld32(t_row + c, r);
          ptx::tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) part[(size_t)(c + i) * kBM + row] = __uint_as_float(r[i]);
        }
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&acc_empty[buf]);          // the accumulator is free again
        __threadfence();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (et == 0) s_prev = atomicAdd(p.split_counters + ws_tile, 1);
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (!coop) {
          last = s_prev == un.nsp - 1;
          if (last) {
            if (et == 0) p.split_counters[ws_tile] = 0;
            __threadfence();
          }
        } else {
          // every slice of the tile is a CTA of its own and all of them are resident: wait (bounded) until all have
          // written, then each adds up its own share of the columns
          if (et == 0) {
            const volatile int* ctr = p.split_counters + ws_tile;
            const uint64_t t0 = ptx::globaltimer_ns();
            uint32_t polls = 0;
            s_prev = 1;
            while (*ctr < un.nsp) {
              if ((++polls & 0xffu) == 0u && (*abort_flag || ptx::globaltimer_ns() - t0 > ptx::kWaitLimitNs)) {
                *abort_flag = 1;
                atomicExch(p.dev_status, -5);
                s_prev = 0;
                break;
              }
            }
          }
          asm volatile("bar.sync 1, 128;" ::: "memory");
          if (s_prev == 0) break;
          __threadfence();
        }
      }
      // 32 accumulator columns of this thread's row: from tensor memory, or the sum of the slices
      auto load32 = [&](int c, float (&acc)[32]) {
        if (!split) {
          uint32_t r[32];
          ptx::tmem_ld32(t_row + c, r);
          ptx::tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) acc[i] = __uint_as_float(r[i]);
        } else {
          // all slices of the 32 columns are requested before any is added (one round trip, not one per slice)
          float part[kMaxKSplits][32];
#pragma unroll
          for (int q = 0; q < kMaxKSplits; ++q) {
            const float* src = p.split_ws + ((size_t)(ws_tile * un.nsp + q) * BN + c) * kBM + row;
            if (q < un.nsp) {
#pragma unroll
              for (int i = 0; i < 32; ++i) part[q][i] = __ldcg(src + (size_t)i * kBM);
            }
          }
#pragma unroll
          for (int i = 0; i < 32; ++i) acc[i] = 0.f;
#pragma unroll
          for (int q = 0; q < kMaxKSplits; ++q)
            if (q < un.nsp) {
#pragma unroll
              for (int i = 0; i < 32; ++i) acc[i] += part[q][i];
            }
        }
      };
      if (!last) { ++lt; continue; }
      if (EPI == kEpiSim && coop) {
        // this slice's share of the tile's columns, eight at a time: the sums over all slices (ascending slice
        // order), then the arg-max over those columns; the 64-bit maximum over slices and tiles is order-independent
        const int nsp = un.nsp;                                  // 8 or 16
        const int cw = BN / nsp;
        const int cb = sp * cw;
        const int m = m_base + row;
        const int g = tc.v0 + m;
        const bool active = m < tc.Vb && p.assign[g] < 0;
        const float inm = active ? p.inv_norm[g] : 0.f;
        float best_sim = -INFINITY;
        int best_slot = 0;
        float* dbg = (p.sim_debug != nullptr && active) ? p.sim_debug + (size_t)g * p.max_kept + tc.n0 : nullptr;
#pragma unroll 1
        for (int c8 = cb; c8 < cb + cw; c8 += 8) {
          float dot[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) dot[i] = 0.f;
#pragma unroll 1
          for (int q0 = 0; q0 < nsp; q0 += 8) {                  // eight slices' loads in flight at a time
            float part[8][8];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              const float* src = p.split_ws + ((size_t)(ws_tile * nsp + q0 + q) * BN + c8) * kBM + row;
#pragma unroll
              for (int i = 0; i < 8; ++i) part[q][i] = __ldcg(src + (size_t)i * kBM);
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
#pragma unroll
              for (int q = 0; q < 8; ++q) dot[i] += part[q][i];
            }
          }
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int sidx = tc.n0 + c8 + i;
            if (active && sidx < tc.kb) {
              const float sim = (dot[i] * inm) * ink_s[c8 + i] + 0.0f;
              if (sim > best_sim) { best_sim = sim; best_slot = sidx; }
              if (dbg != nullptr) dbg[c8 + i] = sim;
            }
          }
        }
        if (active && tc.n0 + cb < tc.kb) {
          const unsigned long long mine =
              ((unsigned long long)ordered_key(best_sim) << 32) | (0xffffffffu - (unsigned)best_slot);
          atomicMax(p.best + g, mine);
        }
        // the counter goes on to twice the slices as they finish reading; the last one leaves it at zero
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (et == 0 && atomicAdd(p.split_counters + ws_tile, 1) == 2 * nsp - 1) p.split_counters[ws_tile] = 0;
        ++lt;
        continue;
      }
      // (a 256-row tile: the same epilogue once per 128-row half, each half in its own accumulator)
#pragma unroll 1
      for (int mh = 0; mh < MT; ++mh, t_row += S::kAccStride, m_base += kBM) {
      if (EPI == kEpiProj) {
        const int grow = m_base + row;
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
          float r[32];
          load32(c, r);
          // 32 divides D, so a 32-column piece lies in one of q, k, v even when the tile straddles two of them
          const int gcol = tc.n0 + c, which = gcol / p.out_cols;
          __nv_bfloat16* dst = p.out[which] + (size_t)grow * p.out_cols + (gcol - which * p.out_cols) - c;
          if (grow < p.out_rows && which < 3) {      // (a tile width that does not divide 3 D: the last tile hangs over)
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
              uint32_t w[4];
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                __nv_bfloat162 h2 = __floats2bfloat162_rn(r[i + 2 * j], r[i + 2 * j + 1]);
                w[j] = *reinterpret_cast<uint32_t*>(&h2);
              }
              *reinterpret_cast<uint4*>(dst + c + i) = make_uint4(w[0], w[1], w[2], w[3]);
            }
          }
        }
      } else if (EPI == kEpiLinear) {
        const int grow = m_base + row;
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
          float r[32];
          load32(c, r);
          if (grow < p.out_rows && tc.n0 + c < p.ld_out) {
            const size_t off = (size_t)grow * p.ld_out + tc.n0 + c;
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
              uint32_t w[4] = {0u, 0u, 0u, 0u};
              if (p.residual != nullptr) {
                const uint4 rr = *reinterpret_cast<const uint4*>(p.residual + off + i);
                w[0] = rr.x; w[1] = rr.y; w[2] = rr.z; w[3] = rr.w;
              }
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const float lo = r[i + 2 * j] + __uint_as_float(w[j] << 16);
                const float hi = r[i + 2 * j + 1] + __uint_as_float(w[j] & 0xffff0000u);
                __nv_bfloat162 h2 = __floats2bfloat162_rn(lo, hi);
                w[j] = *reinterpret_cast<uint32_t*>(&h2);
              }
              *reinterpret_cast<uint4*>(p.lin_out + off + i) = make_uint4(w[0], w[1], w[2], w[3]);
            }
          }
        }
      } else if (EPI == kEpiGateUp) {
        const int grow = m_base + row;
#pragma unroll 1
        for (int c = 0; c < BN / 2; c += 32) {
          float g[32], up[32];
          load32(c, g);
          load32(BN / 2 + c, up);
          if (grow < p.out_rows) {
            __nv_bfloat16* dst = p.lin_out + (size_t)grow * p.ld_out + tc.n0 + c;
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
              uint32_t w[4];
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const float g0 = g[i + 2 * j], g1 = g[i + 2 * j + 1];
                // silu(g) = g / (1 + exp(-g)); for very negative g the divisor is inf and the quotient 0
                const float a0 = __fdividef(g0, 1.f + __expf(-g0)) * up[i + 2 * j];
                const float a1 = __fdividef(g1, 1.f + __expf(-g1)) * up[i + 2 * j + 1];
                __nv_bfloat162 h2 = __floats2bfloat162_rn(a0, a1);
                w[j] = *reinterpret_cast<uint32_t*>(&h2);
              }
              *reinterpret_cast<uint4*>(dst + i) = make_uint4(w[0], w[1], w[2], w[3]);
            }
          }
        }
      } else {
        const int m = m_base + row;
        const int g = tc.v0 + m;
        const bool active = m < tc.Vb && p.assign[g] < 0;     // a pruned token of this request
        const float inm = active ? p.inv_norm[g] : 0.f;
        float best_sim = -INFINITY;                        // strict > below: the lowest slot wins a tie
        int best_slot = 0;
        float* dbg = (p.sim_debug != nullptr && active) ? p.sim_debug + (size_t)g * p.max_kept + tc.n0 : nullptr;
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
          float dot[32];
          load32(c, dot);
          if (active) {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const int sidx = tc.n0 + c + i;
              if (sidx < tc.kb) {
                // the value the arg-max compares; + 0 turns a negative zero into the positive one
                const float sim = (dot[i] * inm) * ink_s[c + i] + 0.0f;
                if (sim > best_sim) { best_sim = sim; best_slot = sidx; }
                if (dbg != nullptr) dbg[c + i] = sim;
              }
            }
          }
        }
        if (active) {
          const unsigned long long mine =
              ((unsigned long long)ordered_key(best_sim) << 32) | (0xffffffffu - (unsigned)best_slot);
          atomicMax(p.best + g, mine);
        }
      }
      }
      if (split) { ++lt; continue; }                      // (its accumulator was released when the partial went out)
      // the accumulator may be overwritten once all four warps have read it
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&acc_empty[buf]);
      ++lt;
    }
    ptx::tc_fence_before_sync();
  }
  __syncthreads();
  if (warp == 2) ptx::tmem_dealloc(tmem_base, 2 * S::kAccStride);
}

// ---------------------------------------------------------------- CTA pairs
// Two CTAs of a cluster (ranks 0 and 1, neighbouring SMs) compute one 256 x BN tile with `cta_group::2` MMAs: each CTA
// holds its own 128 rows of A and HALF of the B tile (BN / 2 rows) in shared memory, the tensor cores of both read both
// halves, and each CTA's 128 x BN accumulator lands in its own tensor memory.  Per k-block a CTA pulls 16 + BN / 4 KB out
// of L2 instead of 16 + BN / 2 KB: 32 KB for 512 tensor cycles at BN = 256, where the single-CTA 128 x 256 tile needs 48 KB
// and is bound by what an SM can pull out of L2 (about 56 B per cycle).
//   * both CTAs run the same warp roles; each loader thread waits on its OWN `empty` barrier and loads its own boxes, whose
//     bytes are counted on rank 0's `full` barrier (rank 0's loader threads expect the bytes of both CTAs);
//   * one thread of rank 0 issues every MMA and commits to the `empty` / `acc_full` barriers of BOTH CTAs;
//   * the epilogue warps of both CTAs arrive on rank 0's `acc_empty` barrier (8 arrivals);
//   * before a CTA leaves, its loaders have seen every commit aimed at it, rank 0 has seen every epilogue arrival, and
//     the two CTAs meet in a cluster barrier; tensor memory is allocated and freed by warp 2 of both CTAs together.
// Whole tiles only (no K split); every mbarrier wait is bounded as elsewhere.
template <int BN> struct PairSmem {
  static constexpr int kABytes = kBM * kBK * 2, kBBytes = (BN / 2) * kBK * 2;
  static constexpr int kStages = 6;
  static constexpr int kBytes = kStages * (kABytes + kBBytes) + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

template <int BN, int EPI>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b, GemmParams p) {
  static_assert(BN % 32 == 0 && BN <= 256 && (BN / 2) % 8 == 0, "half of the B tile is a whole number of 8-row swizzle groups");
  static_assert(EPI != kEpiSim, "the dense layers only");
  using S = PairSmem<BN>;
  constexpr int kStages = S::kStages;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* a_s = smem;
  uint8_t* b_s = smem + kStages * S::kABytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kStages * (S::kABytes + S::kBBytes));
  uint64_t* empty = full + kStages;
  uint64_t* acc_full = empty + kStages;       // [2]
  uint64_t* acc_empty = acc_full + 2;         // [2] (rank 0's are the ones in use)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();
  const bool leader = rank == 0;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { ptx::mbar_init(&full[s], 2); ptx::mbar_init(&empty[s], 1); }   // A and B loaders of rank 0; one commit
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(&acc_full[i], 1); ptx::mbar_init(&acc_empty[i], 8); }   // four epilogue warps in each CTA
    *abort_flag = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 2) { ptx::tmem_alloc_pair(tmem_slot, 512); ptx::tmem_relinquish_pair(); }
  grid_dependency_wait();
  grid_dependency_release();
  ptx::tc_fence_before_sync();
  ptx::cluster_sync();                     // the peer's barriers exist before anything arrives on them
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const int tiles = p.m_tiles * p.n_tiles;
  const int n_pairs = gridDim.x >> 1, pair = blockIdx.x >> 1;
  // tile t: M fastest, so that the pairs of a round share their B tiles in L2
  auto tile_m0 = [&](int t) { return (t % p.m_tiles) * (2 * kBM); };
  auto tile_n0 = [&](int t) { return (t / p.m_tiles) * (EPI == kEpiGateUp ? BN / 2 : BN); };

  if (warp == 0 || warp == 6) {
    // ------------------------------------------------------------ TMA producers: warp 0 streams A, warp 6 streams B
    if (lane == 0) {
      const bool is_a = warp == 0;
      const CUtensorMap* tm = is_a ? &tmap_a : &tmap_b;
      uint8_t* ring = is_a ? a_s : b_s;
      const int stage_bytes = is_a ? S::kABytes : S::kBBytes;
      ptx::prefetch_tensormap(tm);
      int it = 0;
      bool ok = true;
      for (int t = pair; t < tiles && ok; t += n_pairs) {
        const int n0 = tile_n0(t);
        // this CTA's rows: its half of the 256 rows of A; its half of the B tile (gate rows for rank 0, up rows for rank 1)
        const int row0 = is_a ? tile_m0(t) + (int)rank * kBM
                              : (EPI == kEpiGateUp ? (leader ? n0 : p.up_row_offset + n0) : n0 + (int)rank * (BN / 2));
        for (int kbk = 0; kbk < p.num_k_blocks; ++kbk, ++it) {
          const int s = it % kStages;
          ok = ptx::mbar_wait(&empty[s], ((it / kStages) & 1) ^ 1, abort_flag, p.dev_status);
          if (!ok) break;
          if (leader) ptx::mbar_arrive_expect_tx(&full[s], 2 * stage_bytes);     // this operand's boxes of both CTAs
          ptx::tma_load_2d_pair(ring + s * stage_bytes, tm, &full[s], kbk * kBK, row0);
        }
      }
      // every commit aimed at this CTA's `empty` barriers has landed before the CTA may leave
      for (int j = it > kStages ? it - kStages : 0; j < it && ok; ++j)
        ok = ptx::mbar_wait(&empty[j % kStages], (j / kStages) & 1, abort_flag, p.dev_status);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (rank 0 only)
    if (lane == 0 && leader) {
      constexpr uint32_t idesc = ptx::idesc_bf16_f32(2 * kBM, BN, 0, 0);
      const ptx::SmemDesc a_desc0 = ptx::smem_desc_kmajor_sw128(ptx::smem_u32(a_s));
      const ptx::SmemDesc b_desc0 = ptx::smem_desc_kmajor_sw128(ptx::smem_u32(b_s));
      int it = 0, lt = 0;
      bool ok = true;
      for (int t = pair; t < tiles && ok; t += n_pairs, ++lt) {
        const int buf = lt & 1;
        ok = ptx::mbar_wait(&acc_empty[buf], ((lt >> 1) & 1) ^ 1, abort_flag, p.dev_status);   // both epilogues done with it
        if (!ok) break;
        ptx::tc_fence_after_sync();
        const uint32_t tmem_acc = tmem_base + (uint32_t)buf * 256u;
        for (int kbk = 0; kbk < p.num_k_blocks; ++kbk, ++it) {
          const int s = it % kStages;
          ok = ptx::mbar_wait(&full[s], (it / kStages) & 1, abort_flag, p.dev_status);
          if (!ok) break;
          ptx::tc_fence_after_sync();
          const ptx::SmemDesc ad = ptx::smem_desc_advance(a_desc0, s * S::kABytes), bd = ptx::smem_desc_advance(b_desc0, s * S::kBBytes);
#pragma unroll
          for (int kk = 0; kk < kBK / 16; ++kk)
            ptx::mma_ss_pair(tmem_acc, ptx::smem_desc_advance(ad, kk * 32), ptx::smem_desc_advance(bd, kk * 32), idesc,
                             (kbk > 0 || kk > 0) ? 1u : 0u);
          ptx::mma_commit_pair(&empty[s], 3);      // frees the stage in both CTAs once these MMAs have read it
        }
        if (ok) ptx::mma_commit_pair(&acc_full[buf], 3);
      }
      // the peer's epilogue arrivals for the last tiles have landed before this CTA may leave
      for (int j = lt > 2 ? lt - 2 : 0; j < lt && ok; ++j)
        ok = ptx::mbar_wait(&acc_empty[j & 1], (j >> 1) & 1, abort_flag, p.dev_status);
    }
  } else {
    // ------------------------------------------------------------ epilogue: warp w may touch TMEM lanes 32*(w%4) .. +31
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    int lt = 0;
    for (int t = pair; t < tiles; t += n_pairs, ++lt) {
      const int buf = lt & 1;
      const bool ok = __all_sync(0xffffffffu, ptx::mbar_wait(&acc_full[buf], (lt >> 1) & 1, abort_flag, p.dev_status));
      if (!ok) break;
      ptx::tc_fence_after_sync();
      const uint32_t t_row = tmem_base + (uint32_t)buf * 256u + ((uint32_t)(quarter * 32) << 16);
      const int grow = tile_m0(t) + (int)rank * kBM + row;
      const int n0 = tile_n0(t);
      if (EPI == kEpiProj) {
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
          uint32_t r[32];
          ptx::tmem_ld32(t_row + c, r);
          ptx::tmem_wait_ld();
          const int gcol = n0 + c, which = gcol / p.out_cols;
          if (grow < p.out_rows && which < 3) {
            __nv_bfloat16* dst = p.out[which] + (size_t)grow * p.out_cols + (gcol - which * p.out_cols);
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
              uint32_t w[4];
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(r[i + 2 * j]), __uint_as_float(r[i + 2 * j + 1]));
                w[j] = *reinterpret_cast<uint32_t*>(&h2);
              }
              *reinterpret_cast<uint4*>(dst + i) = make_uint4(w[0], w[1], w[2], w[3]);
            }
          }
        }
      } else if (EPI == kEpiLinear) {
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
          uint32_t r[32];
          ptx::tmem_ld32(t_row + c, r);
          ptx::tmem_wait_ld();
          if (grow < p.out_rows && n0 + c < p.ld_out) {
            const size_t off = (size_t)grow * p.ld_out + n0 + c;
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
              uint32_t w[4] = {0u, 0u, 0u, 0u};
              if (p.residual != nullptr) {
                const uint4 rr = *reinterpret_cast<const uint4*>(p.residual + off + i);
                w[0] = rr.x; w[1] = rr.y; w[2] = rr.z; w[3] = rr.w;
              }
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const float lo = __uint_as_float(r[i + 2 * j]) + __uint_as_float(w[j] << 16);
                const float hi = __uint_as_float(r[i + 2 * j + 1]) + __uint_as_float(w[j] & 0xffff0000u);
                __nv_bfloat162 h2 = __floats2bfloat162_rn(lo, hi);
                w[j] = *reinterpret_cast<uint32_t*>(&h2);
              }
              *reinterpret_cast<uint4*>(p.lin_out + off + i) = make_uint4(w[0], w[1], w[2], w[3]);
            }
          }
        }
      } else {
#pragma unroll 1
        for (int c = 0; c < BN / 2; c += 32) {
          uint32_t g[32], up[32];
          ptx::tmem_ld32(t_row + c, g);
          ptx::tmem_ld32(t_row + BN / 2 + c, up);
          ptx::tmem_wait_ld();
          if (grow < p.out_rows) {
            __nv_bfloat16* dst = p.lin_out + (size_t)grow * p.ld_out + n0 + c;
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
              uint32_t w[4];
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const float g0 = __uint_as_float(g[i + 2 * j]), g1 = __uint_as_float(g[i + 2 * j + 1]);
                const float a0 = __fdividef(g0, 1.f + __expf(-g0)) * __uint_as_float(up[i + 2 * j]);
                const float a1 = __fdividef(g1, 1.f + __expf(-g1)) * __uint_as_float(up[i + 2 * j + 1]);
                __nv_bfloat162 h2 = __floats2bfloat162_rn(a0, a1);
                w[j] = *reinterpret_cast<uint32_t*>(&h2);
              }
              *reinterpret_cast<uint4*>(dst + i) = make_uint4(w[0], w[1], w[2], w[3]);
            }
          }
        }
      }
      // the accumulator may be overwritten once the four warps of both CTAs have read it: tell rank 0
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) {
        if (leader) ptx::mbar_arrive(&acc_empty[buf]);
        else ptx::mbar_arrive_cluster(&acc_empty[buf], 0);
      }
    }
  }
  __syncwarp();                            // (the lanes that ran a role's loop rejoin their warp before the aligned barrier)
  ptx::tc_fence_before_sync();
  ptx::cluster_sync();                     // neither CTA frees tensor memory or leaves while the other may still reach it
  if (warp == 2) ptx::tmem_dealloc_pair(tmem_base, 512);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// The dense layers walk whole tiles; when the last round over the SMs is incomplete, its tiles are cut into K
// slices so that the round costs a fraction of a tile time plus the exchange of partial sums.  Costs in units of
// one k-block of main loop (about 0.35 us): a cut round costs about 30 + 5 per slice on top of its k-blocks (measured:
// 15 - 18 us; reading the slices back through bulk copies instead of register loads did not change it, so it is the
// cold start of the short main loops and the fence / counter round trips rather than the read-back), so cutting
// pays for long K only: the down projection of the feed-forward network, not the 64-k-block projections.
void plan_tail_split(const d3tom_ctx* ctx, GemmParams& p) {
  const int tiles = p.m_tiles * p.n_tiles * p.batch, sms = ctx->sm_count;
  p.k_splits = 1; p.full_tiles = tiles;
  const int rem = tiles % sms;
  if (rem == 0 || p.split_ws == nullptr) return;
  int best = p.num_k_blocks, best_s = 1;
  for (int sp = 2; sp <= kMaxKSplits; ++sp) {
    if (p.num_k_blocks / sp < 8 || rem * sp > 2 * sms) break;      // slices too short / more parts than the workspace holds
    const int rounds = (rem * sp + sms - 1) / sms;
    const int cost = rounds * ((p.num_k_blocks + sp - 1) / sp) + 30 + 5 * sp;
    if (cost < best) { best = cost; best_s = sp; }
  }
  if (best_s > 1) { p.k_splits = best_s; p.full_tiles = tiles - rem; }
}

// Which tile shape finishes a dense layer sooner, from measured main-loop cycles per 64 of K (projection timings at
// 128 .. 7600 rows).  128 x 256 tiles: 850 per full round over the SMs (48 KB of operands per k-block: what the SMs
// together can pull out of L2), and 150 + 3.9 r for a last round of r tiles, which runs faster per tile because
// fewer SMs share L2.  256 x 256 tiles: 1450 per full round (64 KB per k-block in three 64 KB stages: bound by the
// load latency of one SM, so a round of few tiles is no cheaper), 900 + 3.5 r for the last round; 256 x 224 tiles
// cost 0.89 of that per round and sometimes need a round less, or fill the last one better (1216 rows x 12288
// columns: 275 tiles in two rounds, 93 us against 99 us for the 240 tiles of 256 x 256).
// Returns the width of the 256-row tile to use (256 or 224), or 0 for 128-row tiles.
int two_m_tile_width(const d3tom_ctx* ctx, int rows, int ncols, bool allow_224) {
  const int sms = ctx->sm_count;
  const long long t1 = (long long)ceil_div(rows, kBM) * ceil_div(ncols, 256);
  const double r1 = (double)(t1 % sms);
  const double cost1 = 850.0 * (double)(t1 / sms) + (r1 > 0 ? 150.0 + 3.9 * r1 : 0.0);
  auto cost2 = [&](int width, double scale) {
    const long long t2 = (long long)ceil_div(rows, 2 * kBM) * ceil_div(ncols, width);
    const double r2 = (double)(t2 % sms);
    return scale * (1450.0 * (double)(t2 / sms) + (r2 > 0 ? 900.0 + 3.5 * r2 : 0.0));
  };
  const double c256 = ncols % 256 == 0 ? cost2(256, 1.0) : 1e30, c224 = allow_224 ? cost2(224, 0.89) : 1e30;
  if (c224 < 0.97 * c256 && c224 < 0.97 * cost1) return 224;
  return c256 < 0.97 * cost1 ? 256 : 0;
}

template <int BN, int EPI, int MT = 1>
int launch_gemm(d3tom_ctx* ctx, const CUtensorMap& ta, const CUtensorMap& tb, GemmParams p, cudaStream_t s) {
  if (EPI != kEpiSim && MT == 1) {
    p.split_ws = ctx->gemm_split_ws; p.split_counters = ctx->gemm_split_counters;
    plan_tail_split(ctx, p);
  }
  if (MT == 2) { p.k_splits = 1; p.full_tiles = p.m_tiles * p.n_tiles * p.batch; }   // whole tiles only
  const long long tiles = (long long)p.m_tiles * p.n_tiles * p.batch;
  const long long units = p.full_tiles + (tiles - p.full_tiles) * p.k_splits;
  if (units <= 0) return D3TOM_OK;
  const int grid = (int)(units < ctx->sm_count ? units : ctx->sm_count);          // persistent: one CTA per SM
  D3TOM_CUDA_TRY(ctx, cudaFuncSetAttribute(gemm_tc_kernel<BN, EPI, MT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           GemmSmem<BN, MT>::kBytes));
  D3TOM_CUDA_TRY(ctx, launch_serialized(gemm_tc_kernel<BN, EPI, MT>, grid, kGemmThreads, GemmSmem<BN, MT>::kBytes, s, ta, tb, p));
  return D3TOM_OK;
}

// How many CTA pairs of this kernel the device holds at once (asked once per device; 0 = clusters of two cannot be
// launched here, and the caller keeps single-CTA tiles).
template <int BN, int EPI>
int resident_pairs(d3tom_ctx* ctx) {
  static int cached[64] = {};
  int& pairs = cached[ctx->device & 63];
  if (pairs == 0) {
    auto kernel = gemm_pair_kernel<BN, EPI>;
    pairs = -1;
    if (ctx->sm_count >= 2 &&
        cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, PairSmem<BN>::kBytes) == cudaSuccess) {
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3((unsigned)(ctx->sm_count & ~1)); cfg.blockDim = dim3(kGemmThreads);
      cfg.dynamicSmemBytes = PairSmem<BN>::kBytes; cfg.attrs = attr; cfg.numAttrs = 1;
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) == cudaSuccess && n > 0)
        pairs = n < ctx->sm_count / 2 ? n : ctx->sm_count / 2;
    }
    if (pairs < 0) (void)cudaGetLastError();     // (the refusal is not an error of the call in hand)
  }
  return pairs > 0 ? pairs : 0;
}

template <int BN, int EPI>
int launch_gemm_pair(d3tom_ctx* ctx, const CUtensorMap& ta, const CUtensorMap& tb, GemmParams p, cudaStream_t s) {
  const long long tiles = (long long)p.m_tiles * p.n_tiles;
  if (tiles <= 0) return D3TOM_OK;
  const int pairs = resident_pairs<BN, EPI>(ctx);
  if (pairs <= 0) return D3TOM_ERR_UNSUPPORTED;
  auto kernel = gemm_pair_kernel<BN, EPI>;
  // (the attribute belongs to the current device: set on every call, a process may drive several GPUs)
  D3TOM_CUDA_TRY(ctx, cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, PairSmem<BN>::kBytes));
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = g_d3tom_launch_overlap ? 1 : 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(2 * (tiles < pairs ? tiles : pairs))); cfg.blockDim = dim3(kGemmThreads);
  cfg.dynamicSmemBytes = PairSmem<BN>::kBytes; cfg.stream = s; cfg.attrs = attr; cfg.numAttrs = 2;
  D3TOM_CUDA_TRY(ctx, cudaLaunchKernelEx(&cfg, kernel, ta, tb, p));
  return D3TOM_OK;
}

// Whether a dense layer of `rows` x `ncols` outputs runs as 256 x 256 tiles on CTA pairs.  Measured against the
// single-CTA shapes, alternating the two in one process (projection / output projection / feed-forward network at
// D = 4096, m = 12288, us): 1216 rows 94 / 51 / 294 against 92 / 56 / 303, 1152 rows 98 / 59 / 297 against
// 87 / 39 / 257, 2176 rows 147 / 56 / 453 against 156 / 62 / 480, 4288 rows 281 / 105 / 914 against 303 / 132 / 1076,
// 7800 rows 543 / 212 / 1715 against 583 / 290 / 1988.  A round of 74 pair tiles costs what a round of 148 tiles of
// 256 x 256 costs per flop (both run at the tensor rate the board's power limit allows), so short layers, which are
// decided by how the tiles fill the last round, keep their shapes; from about two thousand rows on the pairs win on
// every layer: half the operand traffic per SM leaves more of the power budget to the tensor cores.
bool use_pair_tiles(const d3tom_ctx* ctx, int rows, int ncols) {
  if (ncols % 256 != 0 || ctx->sm_count < 2) return false;
  if (g_d3tom_pair_tiles == 0) return false;
  if (g_d3tom_pair_tiles == 256) return true;
  return rows >= 2048;
}

}  // namespace

int make_tmap_bf16_2d(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint64_t pitch_elems,
                      uint32_t box_rows, uint32_t box_cols) {
  EncodeTiledFn fn = get_encode_fn();
  if (fn == nullptr) return -1;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {pitch_elems * 2};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : (int)r;
}

int launch_proj_tc(d3tom_ctx* ctx, const void* x, const void* w, int total, int D, void* q, void* k, void* v,
                   cudaStream_t s) {
  if (D % 128 != 0) return D3TOM_ERR_UNSUPPORTED;
  CUtensorMap ta, tb;
  int r = make_tmap_bf16_2d(&ta, x, (uint64_t)total, (uint64_t)D, (uint64_t)D, kBM);
  if (r != 0) { ctx->last_cuda_error = r; return D3TOM_ERR_CUDA; }
  GemmParams p = {};
  p.num_k_blocks = D / kBK;
  p.out[0] = static_cast<__nv_bfloat16*>(q); p.out[1] = static_cast<__nv_bfloat16*>(k); p.out[2] = static_cast<__nv_bfloat16*>(v);
  p.out_rows = total; p.out_cols = D; p.dev_status = ctx->dev_status;
  p.m_tiles = ceil_div(total, kBM); p.batch = 1; p.k_splits = 1;
  // Tile width: fewest (rounds of tiles over the SMs) x (measured cycles per 64-deep k-block at that
  // width: 667 / 633 / 600 for 256 / 192 / 128 columns; narrow tiles pay the per-k-block barrier
  // traffic of the issuing thread more often per unit of work).  192 divides 3 D whenever 64 divides D.
  int bn = 128;
  double best_cost = 1e30;
  for (int cand : {256, 192, 128}) {
    if ((3 * D) % cand != 0) continue;
    const long long tiles = (long long)p.m_tiles * (3 * D / cand);
    const double rounds = (double)((tiles + ctx->sm_count - 1) / ctx->sm_count);
    const double cost = rounds * (cand == 256 ? 667.0 : cand == 192 ? 633.0 : 600.0);
    if (cost < best_cost) { best_cost = cost; bn = cand; }
  }
  if (use_pair_tiles(ctx, total, 3 * D) && resident_pairs<256, kEpiProj>(ctx) > 0) {
    r = make_tmap_bf16_2d(&tb, w, (uint64_t)3 * D, (uint64_t)D, (uint64_t)D, 128);       // a CTA's half of the weight tile
    if (r != 0) { ctx->last_cuda_error = r; return D3TOM_ERR_CUDA; }
    p.m_tiles = ceil_div(total, 2 * kBM); p.n_tiles = 3 * D / 256;
    return launch_gemm_pair<256, kEpiProj>(ctx, ta, tb, p, s);
  }
  if (const int w2 = two_m_tile_width(ctx, total, 3 * D, D % 32 == 0)) {
    r = make_tmap_bf16_2d(&ta, x, (uint64_t)total, (uint64_t)D, (uint64_t)D, 2 * kBM);
    if (r == 0) r = make_tmap_bf16_2d(&tb, w, (uint64_t)3 * D, (uint64_t)D, (uint64_t)D, (uint32_t)w2);
    if (r != 0) { ctx->last_cuda_error = r; return D3TOM_ERR_CUDA; }
    p.m_tiles = ceil_div(total, 2 * kBM); p.n_tiles = ceil_div(3 * D, w2);
    if (w2 == 224) return launch_gemm<224, kEpiProj, 2>(ctx, ta, tb, p, s);
    return launch_gemm<256, kEpiProj, 2>(ctx, ta, tb, p, s);
  }
  r = make_tmap_bf16_2d(&tb, w, (uint64_t)3 * D, (uint64_t)D, (uint64_t)D, (uint32_t)bn);
  if (r != 0) { ctx->last_cuda_error = r; return D3TOM_ERR_CUDA; }
  p.n_tiles = 3 * D / bn;
  if (bn == 256) return launch_gemm<256, kEpiProj>(ctx, ta, tb, p, s);
  if (bn == 192) return launch_gemm<192, kEpiProj>(ctx, ta, tb, p, s);
  return launch_gemm<128, kEpiProj>(ctx, ta, tb, p, s);
}

int launch_linear_tc(d3tom_ctx* ctx, const void* x, const void* w, const void* residual, int rows, int K, int N,
                     void* out, cudaStream_t s) {
  if (K % kBK != 0 || N % 128 != 0) return D3TOM_ERR_UNSUPPORTED;
  CUtensorMap ta, tb;
  int r = make_tmap_bf16_2d(&ta, x, (uint64_t)rows, (uint64_t)K, (uint64_t)K, kBM);
  if (r != 0) { ctx->last_cuda_error = r; return D3TOM_ERR_CUDA; }
  GemmParams p = {};
  p.num_k_blocks = K / kBK;
  p.lin_out = static_cast<__nv_bfloat16*>(out); p.residual = static_cast<const __nv_bfloat16*>(residual);
  p.ld_out = N; p.out_rows = rows; p.dev_status = ctx->dev_status;
  p.m_tiles = ceil_div(rows, kBM); p.batch = 1; p.k_splits = 1;
  // tile width as for the Q,K,V projection: fewest rounds of tiles over the SMs, weighted by the cycles per k-block
  int bn = 128;
  double best_cost = 1e30;
  for (int cand : {256, 192, 128}) {
    if (N % cand != 0) continue;
    const long long tiles = (long long)p.m_tiles * (N / cand);
    const double rounds = (double)((tiles + ctx->sm_count - 1) / ctx->sm_count);
    const double cost = rounds * (cand == 256 ? 667.0 : cand == 192 ? 633.0 : 600.0);
    if (cost < best_cost) { best_cost = cost; bn = cand; }
  }
  if (use_pair_tiles(ctx, rows, N) && resident_pairs<256, kEpiLinear>(ctx) > 0) {
    r = make_tmap_bf16_2d(&tb, w, (uint64_t)N, (uint64_t)K, (uint64_t)K, 128);
    if (r != 0) { ctx->last_cuda_error = r; return D3TOM_ERR_CUDA; }
    p.m_tiles = ceil_div(rows, 2 * kBM); p.n_tiles = N / 256;
    return launch_gemm_pair<256, kEpiLinear>(ctx, ta, tb, p, s);
  }
  if (const int w2 = two_m_tile_width(ctx, rows, N, true)) {
    r = make_tmap_bf16_2d(&ta, x, (uint64_t)rows, (uint64_t)K, (uint64_t)K, 2 * kBM);
    if (r == 0) r = make_tmap_bf16_2d(&tb, w, (uint64_t)N, (uint64_t)K, (uint64_t)K, (uint32_t)w2);
    if (r != 0) { ctx->last_cuda_error = r; return D3TOM_ERR_CUDA; }
    p.m_tiles = ceil_div(rows, 2 * kBM); p.n_tiles = ceil_div(N, w2);
    if (w2 == 224) return launch_gemm<224, kEpiLinear, 2>(ctx, ta, tb, p, s);
    return launch_gemm<256, kEpiLinear, 2>(ctx, ta, tb, p, s);
  }
  r = make_tmap_bf16_2d(&tb, w, (uint64_t)N, (uint64_t)K, (uint64_t)K, (uint32_t)bn);
  if (r != 0) { ctx->last_cuda_error = r; return D3TOM_ERR_CUDA; }
  p.n_tiles = N / bn;
  if (bn == 256) return launch_gemm<256, kEpiLinear>(ctx, ta, tb, p, s);
  if (bn == 192) return launch_gemm<192, kEpiLinear>(ctx, ta, tb, p, s);
  return launch_gemm<128, kEpiLinear>(ctx, ta, tb, p, s);
}

int launch_gate_up_tc(d3tom_ctx* ctx, const void* x, const void* w_gate_up, int rows, int D, int m, void* act,
                      cudaStream_t s) {
  if (D % kBK != 0 || m % 128 != 0) return D3TOM_ERR_UNSUPPORTED;
  CUtensorMap ta, tb;
  int r = make_tmap_bf16_2d(&ta, x, (uint64_t)rows, (uint64_t)D, (uint64_t)D, kBM);
  if (r == 0) r = make_tmap_bf16_2d(&tb, w_gate_up, (uint64_t)2 * m, (uint64_t)D, (uint64_t)D, 128);
  if (r != 0) { ctx->last_cuda_error = r; return D3TOM_ERR_CUDA; }
  GemmParams p = {};
  p.num_k_blocks = D / kBK;
  p.lin_out = static_cast<__nv_bfloat16*>(act); p.ld_out = m; p.up_row_offset = m; p.out_rows = rows;
  p.dev_status = ctx->dev_status;
  p.m_tiles = ceil_div(rows, kBM); p.n_tiles = m / 128; p.batch = 1; p.k_splits = 1;
  if (use_pair_tiles(ctx, rows, 2 * m) && resident_pairs<256, kEpiGateUp>(ctx) > 0) {       // (the B map's box is already 128 rows: one CTA's half)
    p.m_tiles = ceil_div(rows, 2 * kBM);
    return launch_gemm_pair<256, kEpiGateUp>(ctx, ta, tb, p, s);
  }
  {
    if (two_m_tile_width(ctx, rows, 2 * m, false) == 256) {
      r = make_tmap_bf16_2d(&ta, x, (uint64_t)rows, (uint64_t)D, (uint64_t)D, 2 * kBM);
      if (r != 0) { ctx->last_cuda_error = r; return D3TOM_ERR_CUDA; }
      p.m_tiles = ceil_div(rows, 2 * kBM);
      return launch_gemm<256, kEpiGateUp, 2>(ctx, ta, tb, p, s);
    }
  }
  return launch_gemm<256, kEpiGateUp>(ctx, ta, tb, p, s);
}

int launch_sim_tc(d3tom_ctx* ctx, const MergeArgs& a, cudaStream_t s) {
  if (a.D % kBK != 0) return D3TOM_ERR_UNSUPPORTED;
  CUtensorMap ta, tb;
  int r = make_tmap_bf16_2d(&ta, a.hidden, (uint64_t)a.total_tokens, (uint64_t)a.D, (uint64_t)a.D, kBM);
  if (r != 0) { ctx->last_cuda_error = r; return D3TOM_ERR_CUDA; }
  const int kept_rows_bound = a.total_tokens;    // rows the kept-row scratch can hold
  r = make_tmap_bf16_2d(&tb, ctx->kept_rows, (uint64_t)kept_rows_bound, (uint64_t)a.D, (uint64_t)a.D, 128);
  if (r != 0) { ctx->last_cuda_error = r; return D3TOM_ERR_CUDA; }
  GemmParams p = {};
  p.num_k_blocks = a.D / kBK;
  p.cu_seqlens = a.cu_seqlens; p.cu_vis = a.cu_vis; p.cu_kept = a.cu_kept; p.assign = a.assign;
  p.inv_norm = ctx->inv_norm; p.inv_norm_kept = ctx->inv_norm_kept; p.best = ctx->best; p.sim_debug = a.sim_debug;
  p.max_kept = a.max_kept; p.dev_status = ctx->dev_status;
  p.m_tiles = ceil_div(a.max_visual, kBM); p.batch = a.B;
  // Few tiles (short requests, small kept sets): a tile is 64 k-blocks of serial work on one SM while
  // most SMs idle, so each tile's K range is cut into slices for different SMs (see the epilogue).
  {
    const int bn = a.max_kept > 128 ? 256 : 128;
    const long long tiles = (long long)p.m_tiles * ceil_div(a.max_kept, bn) * p.batch;
    int splits = (int)(ctx->sm_count / (tiles > 0 ? tiles : 1));
    if (splits > kMaxKSplits) splits = kMaxKSplits;
    if (splits > p.num_k_blocks) splits = p.num_k_blocks;
    if (splits < 2 || tiles * splits > 2LL * ctx->sm_count) splits = 1;
    // very few tiles (a small kept set, one short request): eight or sixteen slices per tile, each a CTA of its
    // own, and every slice adds up its share of the tile's columns itself instead of the last one adding all
    for (int c = kCoopSlices; c >= 8; c /= 2) {
      if (tiles * c <= ctx->sm_count && p.num_k_blocks >= 2 * c) {
        splits = c;
        p.coop = 1;
        break;
      }
    }
    p.k_splits = splits;
    p.full_tiles = 0;                                   // every tile is cut (or none: one slice)
    p.split_ws = ctx->gemm_split_ws; p.split_counters = ctx->gemm_split_counters;
  }
  if (a.max_kept > 128) {      // 256-wide tiles: the A tile is streamed once per 256 kept rows and each MMA covers twice the work
    r = make_tmap_bf16_2d(&tb, ctx->kept_rows, (uint64_t)kept_rows_bound, (uint64_t)a.D, (uint64_t)a.D, 256);
    if (r != 0) { ctx->last_cuda_error = r; return D3TOM_ERR_CUDA; }
    p.n_tiles = ceil_div(a.max_kept, 256);
    return launch_gemm<256, kEpiSim>(ctx, ta, tb, p, s);
  }
  p.n_tiles = ceil_div(a.max_kept, 128);
  return launch_gemm<128, kEpiSim>(ctx, ta, tb, p, s);
}
