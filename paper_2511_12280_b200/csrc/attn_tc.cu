// Bidirectional (unmasked) flash attention for packed ragged sequences on the
// sm_100a tensor cores, bf16 in / fp32 accumulate (Sec. 3.2.1, A = softmax(QK^T *
// scale); Algorithm 1, SelfAttn_l; the layers after l* reuse it on the shortened
// sequences).  The decider -> visual importance map (Sec. 3.2.1, S_j) is fed from
// the SAME score tiles: decider rows spill their raw q.k scores over the visual
// keys plus their final softmax statistics, and a small finishing kernel turns
// those into S_j.  There is no second QK^T.
//
// One CTA = one (request, head, 256 query rows): two 128-row query tiles that
// ping-pong on the tensor pipe.
//   warps 0-3   softmax of query tile 0 (one row per thread = one TMEM lane)
//   warps 4-7   softmax of query tile 1
//   warp  8     TMA producer: Q tiles once, then stages {K_t, V_(t-1)}, two in flight
//   warp  9     one thread issues every tcgen05.mma
//   warps 10-11 idle (they complete the third warpgroup so that registers can be
//               moved from it to the softmax warpgroups with setmaxnreg)
// TMEM (512 columns): S0 | S1 (128 fp32 columns each; the bf16 P tile overwrites
// the first 64 columns of its S tile) | O0 | O1 (head_dim fp32 columns each).
// Per key tile j and query tile i:  S_i = Q_i K_j^T  ->  softmax warps read S_i,
// write P_i in two halves  ->  O_i += P_i V_j, the first half of the keys while
// the second half is still being exponentiated.  The running maximum is only
// raised when the new one exceeds it by more than 2^8 (the O tile is then
// rescaled in place by its own softmax warps); sums and outputs are exact for
// any reference maximum.  CTAs are issued from the END of each request towards
// its beginning: the response rows (where the decider rows live and spill their
// scores) are at the end, and the CTAs with extra work should not run last.
#include "common.cuh"
#include "ptx.cuh"

namespace {

constexpr int kTile = 128;            // query rows per tile and keys per tile
constexpr int kAttnThreads = 384;
constexpr int kSoftmaxRegs = 216, kOtherRegs = 64;   // 256 * 216 + 128 * 64 <= 384 * 168
constexpr int kKvSlots = 4;
constexpr float kRescaleThreshold = 8.0f;

template <int DH> struct AttnSmem {
  static constexpr int kTileBytes = kTile * DH * 2;
  static constexpr int kBytes = 2 * kTileBytes + kKvSlots * kTileBytes + 1024 + 256;
};

__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
// 32 lanes x 16 columns: the 16-register form of tcgen05.st
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}

// kImp: the launch also feeds the importance map (decider rows look themselves up and store their scores); the
// plain instance carries none of that code, which keeps its softmax loop at the registers and schedule it had.
template <int DH, bool kImp>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
               const __grid_constant__ CUtensorMap tmap_v, AttnArgs a) {
  using S = AttnSmem<DH>;
  constexpr int kTileBytes = S::kTileBytes;
  constexpr int kHalfBytes = kTile * 128;               // one 64-column sub-tile: 128 rows x 128 bytes
  constexpr int kHalves = DH / 64;
  // CTAs are dispatched in the order of their index.  Requests of a batch go longest first (below).  Per request: the first H work items take the
  // LAST 256-row query block of every head (the response rows live there and decider rows do extra
  // work, so those CTAs must not end up in the last wave); the remaining items walk head by head
  // (one head's K/V stay hot in L2), query blocks from the end.  Items from `split_from` on are cut
  // into two CTAs of one 128-row tile each: the host does that to the items of an incomplete last
  // wave, which then costs the time of a single tile instead of a pair.
  grid_dependency_enter();
  const int items = a.H * a.nqb, per_req = items + (items - a.split_from);
  int b = (int)blockIdx.x / per_req;
  const int lin = (int)blockIdx.x - b * per_req;
  if (a.B > 1 && a.B <= 32) {
    // Requests are dispatched longest first (a work item's time grows with its request's length, and the last wave
    // should hold short items): the group of CTAs number b takes the request of rank b by descending length,
    // ties by index.  Every warp works the ranks out for itself (one load per lane, B shuffles).
    const int lane_ = threadIdx.x & 31;
    const int nl = lane_ < a.B ? a.cu_seqlens[lane_ + 1] - a.cu_seqlens[lane_] : -1;
    int rank = 0;
    for (int o = 0; o < a.B; ++o) {
      const int no = __shfl_sync(0xffffffffu, nl, o);
      rank += (no > nl || (no == nl && o < lane_)) ? 1 : 0;
    }
    b = __ffs(__ballot_sync(0xffffffffu, lane_ < a.B && rank == b)) - 1;
  }
  int item = lin, half = -1;
  if (lin >= a.split_from) { item = a.split_from + ((lin - a.split_from) >> 1); half = (lin - a.split_from) & 1; }
  int h, qb;
  if (item < a.H) { h = item; qb = a.nqb - 1; }
  else { const int r = item - a.H; h = r / (a.nqb - 1); qb = a.nqb - 2 - r % (a.nqb - 1); }
  const int lo = a.cu_seqlens[b], n = a.cu_seqlens[b + 1] - lo;
  const int q0 = qb * 2 * kTile + (half > 0 ? kTile : 0);
  if (q0 >= n) return;                                  // uniform; nothing allocated yet
  const int n_qt = (half < 0 && n - q0 > kTile) ? 2 : 1;
  const int n_kv = (n + kTile - 1) / kTile;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_s = smem;                                  // 2 tiles
  uint8_t* kv_s = smem + 2 * kTileBytes;                // two stages of {K tile, V tile}
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (2 + kKvSlots) * kTileBytes);
  uint64_t* q_full = bars;                              // [2]
  uint64_t* kv_full = bars + 2;                         // [2] (of 4 reserved)
  uint64_t* kv_empty = bars + 6;                        // [2] (of 4 reserved)
  uint64_t* s_full = bars + 10;                         // [2]
  uint64_t* p_lo = bars + 12;                           // [2]  P columns of keys 0..63 written (and O consistent)
  uint64_t* p_hi = bars + 14;                           // [2]  P columns of keys 64..127 written
  uint64_t* o_final = bars + 16;                        // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 18);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&q_full[i], 1); ptx::mbar_init(&s_full[i], 1);
      ptx::mbar_init(&p_lo[i], 4); ptx::mbar_init(&p_hi[i], 4);      // one arrival per softmax warp
      ptx::mbar_init(&o_final[i], 1);
    }
    for (int s = 0; s < kKvSlots; ++s) { ptx::mbar_init(&kv_full[s], 1); ptx::mbar_init(&kv_empty[s], 4 * n_qt); }   // freed by the softmax warps
    *abort_flag = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 0) { ptx::tmem_alloc(tmem_slot, 512); ptx::tmem_relinquish(); }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;
  auto col_s = [](int i) -> uint32_t { return (uint32_t)i * 128u; };          // S_i (and P_i) columns
  auto col_o = [](int i) -> uint32_t { return 256u + (uint32_t)i * 128u; };   // O_i columns

  if (warp >= 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kOtherRegs));
    if (warp == 8) {
      // ------------------------------------------------------------ TMA producer
      if (lane == 0) {
        ptx::prefetch_tensormap(&tmap_q); ptx::prefetch_tensormap(&tmap_k); ptx::prefetch_tensormap(&tmap_v);
        for (int i = 0; i < n_qt; ++i) {
          ptx::mbar_arrive_expect_tx(&q_full[i], kTileBytes);
          for (int hf = 0; hf < kHalves; ++hf)
            ptx::tma_load_2d(q_s + i * kTileBytes + hf * kHalfBytes, &tmap_q, &q_full[i], h * DH + hf * 64,
                             lo + q0 + i * kTile);
        }
        // stage t = {K_t, V_(t-1)}: what key tile t-1's PV and key tile t's QK^T need; two stages in flight
        for (int t = 0; t <= n_kv; ++t) {
          const int st = t & 1;
          if (t >= 2 && !ptx::mbar_wait(&kv_empty[st], ((t >> 1) & 1) ^ 1, abort_flag, a.dev_status)) break;
          const bool has_k = t < n_kv, has_v = t > 0;
          ptx::mbar_arrive_expect_tx(&kv_full[st], (has_k ? kTileBytes : 0) + (has_v ? kTileBytes : 0));
          for (int hf = 0; hf < kHalves; ++hf) {
            if (has_v) ptx::tma_load_2d(kv_s + (2 * st + 1) * kTileBytes + hf * kHalfBytes, &tmap_v, &kv_full[st],
                                        h * DH + hf * 64, lo + (t - 1) * kTile);
            if (has_k) ptx::tma_load_2d(kv_s + (2 * st) * kTileBytes + hf * kHalfBytes, &tmap_k, &kv_full[st],
                                        h * DH + hf * 64, lo + t * kTile);
          }
        }
      }
    } else if (warp == 9) {
      // ------------------------------------------------------------ MMA issuer
      // tcgen05.mma issue blocks once about two instructions are queued, so whatever this thread
      // does between two MMAs is idle time of the tensor pipe: descriptors are built once and
      // only advanced by one 32-bit add per instruction.
      if (lane == 0) {
        constexpr uint32_t idesc_qk = ptx::idesc_bf16_f32(kTile, kTile, 0, 0);   // S = Q K^T, both K-major
        constexpr uint32_t idesc_pv = ptx::idesc_bf16_f32(kTile, DH, 0, 1);      // O += P V, V is MN-major
        const ptx::SmemDesc q_desc[2] = {ptx::smem_desc_kmajor_sw128(ptx::smem_u32(q_s)),
                                         ptx::smem_desc_kmajor_sw128(ptx::smem_u32(q_s + kTileBytes))};
        const ptx::SmemDesc k_desc0 = ptx::smem_desc_kmajor_sw128(ptx::smem_u32(kv_s));
        const ptx::SmemDesc v_desc0 = ptx::smem_desc_mnmajor_sw128(ptx::smem_u32(kv_s), kHalfBytes);
        auto issue_qk = [&](int i, int slot) {
          const ptx::SmemDesc qd = q_desc[i], kd = ptx::smem_desc_advance(k_desc0, slot * kTileBytes);
#pragma unroll
          for (int kk = 0; kk < DH / 16; ++kk) {
            const uint32_t off = (kk / 4) * kHalfBytes + (kk % 4) * 32;
            ptx::mma_ss(tmem + col_s(i), ptx::smem_desc_advance(qd, off), ptx::smem_desc_advance(kd, off), idesc_qk,
                        kk > 0 ? 1u : 0u);
          }
        };
        // keys 64*half .. 64*half+63 of the tile: P columns 32*half .., V rows 64*half ..
        auto issue_pv_half = [&](int i, int slot, int half, bool accumulate) {
          const ptx::SmemDesc vd = ptx::smem_desc_advance(v_desc0, slot * kTileBytes + half * 4 * 2048);
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4) {                       // 16 keys per instruction
            ptx::mma_ts(tmem + col_o(i), tmem + col_s(i) + (half * 4 + k4) * 8, ptx::smem_desc_advance(vd, k4 * 2048),
                        idesc_pv, (accumulate || half > 0 || k4 > 0) ? 1u : 0u);
          }
        };
        bool ok = true;
        for (int i = 0; i < n_qt && ok; ++i) ok = ptx::mbar_wait(&q_full[i], 0, abort_flag, a.dev_status);
        if (ok) ok = ptx::mbar_wait(&kv_full[0], 0, abort_flag, a.dev_status);     // stage 0 = K_0
        if (ok) {
          ptx::tc_fence_after_sync();
          for (int i = 0; i < n_qt; ++i) { issue_qk(i, 0); ptx::mma_commit(&s_full[i]); }
        }
        // Key tile j needs stage j+1 (V_j and K_(j+1)).  The softmax warps wait for that stage
        // before they announce P_j, so this thread has no load barrier of its own to check: every
        // barrier check between two MMAs costs the tensor pipe more than an instruction slot.
        for (int j = 0; j < n_kv && ok; ++j) {
          const int st = (j + 1) & 1;
          const bool more = j + 1 < n_kv;
          for (int i = 0; i < n_qt && ok; ++i) {
            ok = ptx::mbar_wait(&p_lo[i], j & 1, abort_flag, a.dev_status);          // first half of P_j(i), O_i consistent
            if (!ok) break;
            ptx::tc_fence_after_sync();
            issue_pv_half(i, 2 * st + 1, 0, j > 0);
            ok = ptx::mbar_wait(&p_hi[i], j & 1, abort_flag, a.dev_status);
            if (!ok) break;
            ptx::tc_fence_after_sync();
            issue_pv_half(i, 2 * st + 1, 1, true);
            if (more) {
              issue_qk(i, 2 * st);
              ptx::mma_commit(&s_full[i]);
            } else {
              ptx::mma_commit(&o_final[i]);
            }
          }
        }
      }
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kSoftmaxRegs));
    // ------------------------------------------------------------ softmax + epilogue
    const int i = warp >> 2;                       // query tile of this warpgroup
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;           // row in the tile == TMEM lane
    const int q_row = q0 + i * kTile + row;        // row in the request
    const bool valid_row = q_row < n;
    if (i < n_qt) {
      const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
      const uint32_t t_s = tmem + lane_addr + col_s(i);
      const uint32_t t_o = tmem + lane_addr + col_o(i);
      // is this row a decider of the request?
      // (deciders are response rows: a row below the visual count cannot be one and skips the look-up)
      int dec_slot = -1, n_vis = 0;
      if ((kImp && a.decider_pos != nullptr)) n_vis = a.n_visual[b];
      if ((kImp && a.decider_pos != nullptr) && valid_row && q_row >= n_vis) {
        int l = a.cu_deciders[b], r = a.cu_deciders[b + 1];
        while (l < r) {
          const int mid = (l + r) >> 1, pos = a.decider_pos[mid];
          if (pos == q_row) { dec_slot = mid; break; }
          if (pos < q_row) l = mid + 1; else r = mid;
        }
      }
      float* score_row = dec_slot >= 0 ? a.score_scratch + ((size_t)h * a.max_deciders + dec_slot) * a.vis_stride : nullptr;

      float m_used = -INFINITY;
      float2 l2 = make_float2(0.f, 0.f);           // the row sum, kept as two partial sums
      const float c = a.scale_log2;
      const float2 c2 = make_float2(c, c);
      bool ok = true;
      for (int j = 0; j < n_kv; ++j) {
        ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_full[i], j & 1, abort_flag, a.dev_status));
        if (!ok) break;
        ptx::tc_fence_after_sync();
        // S_j of this tile is complete, so its QK^T has read K_j and, issued before it, the PV of the
        // previous key tile has read V_(j-1): stage j is free once every softmax warp has seen that
        // (a commit by the MMA thread would cost the tensor pipe an issue gap)
        if (lane == 0) ptx::mbar_arrive(&kv_empty[j & 1]);
        // ---- the whole score row of this tile: 128 fp32 values, one TMEM lane
        uint32_t sr[kTile];
        ptx::tmem_ld32(t_s, sr);
        ptx::tmem_ld32(t_s + 32, sr + 32);
        ptx::tmem_ld32(t_s + 64, sr + 64);
        ptx::tmem_ld32(t_s + 96, sr + 96);
        ptx::tmem_wait_ld();
        const int n_valid = n - j * kTile;                  // keys of this tile that belong to the request
        if (n_valid < kTile) {                              // ragged last tile: keys past the end score -inf
#pragma unroll
          for (int e = 0; e < kTile; ++e) if (e >= n_valid) sr[e] = 0xff800000u;
        }
        // ---- p = exp2(s*c - m) in four chunks of 32 keys.  The first two chunks are computed
        //      against the maximum known BEFORE this tile, while the tile's own maximum is still being
        //      reduced: any reference within 2^8 of the true maximum is exact after the final division,
        //      so the result stands unless the maximum grew by more than that (then it is redone).
        uint32_t pk[2][16];
        float2 l_tile = make_float2(0.f, 0.f);
        auto exp_chunk = [&](int ch, float m_ref, uint32_t (&out)[16], float2& lsum) {
          const float2 nm2 = make_float2(-m_ref, -m_ref);
          float2 t2[16];
#pragma unroll
          for (int e = 0; e < 16; ++e)
            t2[e] = __ffma2_rn(make_float2(__uint_as_float(sr[ch * 32 + 2 * e]), __uint_as_float(sr[ch * 32 + 2 * e + 1])),
                               c2, nm2);
#pragma unroll
          for (int e = 0; e < 16; ++e) { t2[e].x = ptx::ex2(t2[e].x); t2[e].y = ptx::ex2(t2[e].y); }
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            out[e] = pack_bf16x2(t2[e].x, t2[e].y);
            lsum = __fadd2_rn(lsum, t2[e]);
          }
        };
        exp_chunk(0, m_used, pk[0], l_tile);                // (first tile: against -inf, always redone below)
        exp_chunk(1, m_used, pk[1], l_tile);
        // ---- row maximum: 8 independent chains of three-input maxima
        float mx[8];
#pragma unroll
        for (int t = 0; t < 8; ++t) mx[t] = fmaxf(__uint_as_float(sr[2 * t]), __uint_as_float(sr[2 * t + 1]));
#pragma unroll
        for (int e = 16; e < kTile; e += 16)
#pragma unroll
          for (int t = 0; t < 8; ++t)
            mx[t] = max3(mx[t], __uint_as_float(sr[e + 2 * t]), __uint_as_float(sr[e + 2 * t + 1]));
        const float mxa = max3(max3(mx[0], mx[1], mx[2]), max3(mx[3], mx[4], mx[5]), fmaxf(mx[6], mx[7]));
        const float m_new = fmaxf(m_used, mxa * c);
        const bool need = (m_new - m_used) > kRescaleThreshold;   // first tile: inf > threshold
        if (__any_sync(0xffffffffu, need)) {
          const float alpha = need ? exp2f(m_used - m_new) : 1.f;
          if (j > 0) {
#pragma unroll 1
            for (int c0 = 0; c0 < DH; c0 += 32) {
              uint32_t r[32];
              ptx::tmem_ld32(t_o + c0, r);
              ptx::tmem_wait_ld();
#pragma unroll
              for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
              ptx::tmem_st32(t_o + c0, r);
            }
            ptx::tmem_wait_st();
          }
          l2.x *= alpha; l2.y *= alpha;
          if (need) m_used = m_new;
          l_tile = make_float2(0.f, 0.f);                   // the speculative half is redone against the new maximum
          exp_chunk(0, m_used, pk[0], l_tile);
          exp_chunk(1, m_used, pk[1], l_tile);
        }
        // ---- the bf16 P tile goes into the first 64 columns of the S tile; the tensor pipe is told after each half
        tmem_st16(t_s, pk[0]);                             // keys 32*ch .. +31 -> P columns 16*ch .. +15
        tmem_st16(t_s + 16, pk[1]);
        exp_chunk(2, m_used, pk[0], l_tile);
        ptx::tmem_wait_st();
        ptx::tc_fence_before_sync();
        // V_j and K_(j+1) must have landed before the tensor pipe is sent on (it does not check)
        ok = __all_sync(0xffffffffu, ptx::mbar_wait(&kv_full[(j + 1) & 1], ((j + 1) >> 1) & 1, abort_flag, a.dev_status));
        if (!ok) break;
        if (lane == 0) ptx::mbar_arrive(&p_lo[i]);
        tmem_st16(t_s + 32, pk[0]);
        exp_chunk(3, m_used, pk[1], l_tile);
        tmem_st16(t_s + 48, pk[1]);
        l2 = __fadd2_rn(l2, l_tile);
        ptx::tmem_wait_st();
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&p_hi[i]);
        // Decider rows: the raw scores over the visual keys go out AFTER P has been announced: the stores (one row per
        // lane, 512 bytes each, uncoalesced) then run while the tensor pipe works on this tile instead of delaying it
        // (the score registers stay live until the next key tile's load).
        if (kImp && score_row != nullptr && j * kTile < n_vis) {
          const int key0 = j * kTile;
#pragma unroll
          for (int e = 0; e < kTile; e += 4) {
            if (key0 + e + 3 < n_vis) {
              *reinterpret_cast<float4*>(score_row + key0 + e) =
                  make_float4(__uint_as_float(sr[e]), __uint_as_float(sr[e + 1]), __uint_as_float(sr[e + 2]),
                              __uint_as_float(sr[e + 3]));
            } else {
#pragma unroll
              for (int t = 0; t < 4; ++t) if (key0 + e + t < n_vis) score_row[key0 + e + t] = __uint_as_float(sr[e + t]);
            }
          }
        }
      }
      // ---- epilogue: O / l -> bf16 -> global
      if (ok) ok = __all_sync(0xffffffffu, ptx::mbar_wait(&o_final[i], 0, abort_flag, a.dev_status));
      ptx::tc_fence_after_sync();
      if (ok) {
        const float l_sum = l2.x + l2.y;
        const float inv_l = 1.f / l_sum;
        __nv_bfloat16* dst = static_cast<__nv_bfloat16*>(a.out) + ((size_t)(lo + q_row) * a.H + h) * DH;
#pragma unroll 1
        for (int c0 = 0; c0 < DH; c0 += 32) {
          uint32_t r[32];
          ptx::tmem_ld32(t_o + c0, r);
          ptx::tmem_wait_ld();
          if (valid_row) {
#pragma unroll
            for (int e = 0; e < 32; e += 8) {
              uint32_t w[4];
#pragma unroll
              for (int t = 0; t < 4; ++t)
                w[t] = pack_bf16x2(__uint_as_float(r[e + 2 * t]) * inv_l, __uint_as_float(r[e + 2 * t + 1]) * inv_l);
              *reinterpret_cast<uint4*>(dst + c0 + e) = make_uint4(w[0], w[1], w[2], w[3]);
            }
          }
        }
        if (dec_slot >= 0) a.lse_scratch[(size_t)h * a.max_deciders + dec_slot] = make_float2(m_used, l_sum);
      }
    }
    ptx::tc_fence_before_sync();
  }
  __syncthreads();
  if (warp == 0) ptx::tmem_dealloc(tmem, 512);
}

template <int DH>
int launch(d3tom_ctx* ctx, const AttnArgs& a, cudaStream_t s) {
  CUtensorMap tq, tk, tv;
  const uint64_t rows = (uint64_t)a.total_tokens, cols = (uint64_t)a.H * DH;
  int r = make_tmap_bf16_2d(&tq, a.q, rows, cols, cols, kTile);
  if (r == 0) r = make_tmap_bf16_2d(&tk, a.k, rows, cols, cols, kTile);
  if (r == 0) r = make_tmap_bf16_2d(&tv, a.v, rows, cols, cols, kTile);
  if (r != 0) { ctx->last_cuda_error = r; return D3TOM_ERR_CUDA; }
  auto kernel = a.decider_pos != nullptr ? attn_tc_kernel<DH, true> : attn_tc_kernel<DH, false>;
  D3TOM_CUDA_TRY(ctx, cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnSmem<DH>::kBytes));
  AttnArgs k = a;
  k.nqb = ceil_div(a.max_seqlen, 2 * kTile);
  const int items = a.H * k.nqb, sms = ctx->sm_count > 0 ? ctx->sm_count : 1;
  k.split_from = items;
  if (a.B == 1) {                                   // (with one request the row count is known here)
    const int rest = items % sms;
    if (2 * items <= sms) k.split_from = 0;                                   // tiny: single tiles reach more SMs
    else if (items > sms && rest > 0 && 2 * rest <= sms) k.split_from = items - rest;   // incomplete last wave
  }
  const int grid = a.B * (items + (items - k.split_from));
  D3TOM_CUDA_TRY(ctx, launch_serialized(kernel, grid, kAttnThreads, AttnSmem<DH>::kBytes, s, tq, tk, tv, k));
  D3TOM_LAUNCH_CHECK(ctx);
  return D3TOM_OK;
}

}  // namespace

int launch_attn_tc(d3tom_ctx* ctx, const AttnArgs& a, cudaStream_t s) {
  if (a.dh == 128) return launch<128>(ctx, a, s);
  if (a.dh == 64) return launch<64>(ctx, a, s);
  return D3TOM_ERR_UNSUPPORTED;
}
