// The attention kernel of attn_tc.cu for ONE request, with the work balanced over the SMs
// (Sec. 3.2.1, A = softmax(QK^T * scale); Algorithm 1, SelfAttn_l; the layers after l*).
//
// A work item is (head, 256 query rows) and costs one step per 128-key tile.  With whole items
// per CTA the SMs are loaded unevenly whenever the items are not a multiple of the SM count:
// 160 items of 10 steps on 148 SMs cost two waves, 544 items of 34 steps cost four rounds for
// 3.68 rounds of work.  Here the (item, key tile) steps are numbered in one line and every CTA
// (one per SM, all resident at once) takes an equal, contiguous share of it.  A share is at
// least one item long, so an item is cut at most once: its tail (the later key tiles) is the
// FIRST thing the next CTA does, its head the LAST thing this CTA does.  The CTA with the tail
// writes its unnormalised O tile and softmax statistics (m, l) to a per-CTA slot in global
// memory; the CTA with the head, which finishes later, adds them to its own
// (O = O1 2^(m1-m) + O2 2^(m2-m), l likewise) and writes the rows.  The order of the two terms
// is fixed, so results do not depend on timing.
//
// Inside a CTA everything is as in attn_tc.cu (two 128-row query tiles ping-pong on the tensor
// pipe, S/P/O in TMEM, {K_t, V_(t-1)} stages, P in two halves, lazy rescaling, decider rows
// spill their raw scores); the barriers simply keep counting across the CTA's segments.
#include "common.cuh"
#include "ptx.cuh"

namespace {

constexpr int kTile = 128;
constexpr int kAttnThreads = 384;
constexpr int kSoftmaxRegs = 216, kOtherRegs = 64;
constexpr int kKvSlots = 4;
constexpr float kRescaleThreshold = 8.0f;

template <int DH> struct SkSmem {
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
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}

// A bounded wait for a word in global memory that another CTA of this (fully resident) grid sets.
__device__ __forceinline__ bool flag_wait(const int* flag, int want, volatile int* abort_flag, int* dev_status) {
  const volatile int* f = flag;
  if (*f == want) return true;
  const uint64_t t0 = ptx::globaltimer_ns();
  uint32_t polls = 0;
  while (*f != want) {
    if ((++polls & 0xffu) == 0u) {
      if (*abort_flag) return false;
      if (ptx::globaltimer_ns() - t0 > ptx::kWaitLimitNs) {
        *abort_flag = 1;
        atomicExch(dev_status, -5);
        return false;
      }
    }
  }
  return true;
}

// The CTA's walk over its share [pos, hi) of the step line: one segment = (item, key tiles [j0, j1)).
// The line holds, head by head, the n_kv steps of each of the head's nqb items and then `pad` empty positions:
// the head's last item carries the response rows, and when those spill their scores for the importance map its
// steps cost about a quarter more; the empty positions charge that to the share that gets them.
struct Walk {
  int pos, hi, n_kv, nqb, n, pad;
  int t, j0, j1, h, q0, n_qt;
  __device__ __forceinline__ bool next() {
    const int head_len = nqb * n_kv + pad;
    while (pos < hi) {
      h = pos / head_len;
      const int r = pos - h * head_len, qb = r / n_kv;
      if (qb >= nqb) { pos += min(head_len - r, hi - pos); continue; }      // empty positions: nothing to do
      j0 = r - qb * n_kv;
      j1 = min(n_kv, j0 + (hi - pos));
      t = h * nqb + qb;
      q0 = qb * 2 * kTile;
      n_qt = (n - q0 > kTile) ? 2 : 1;
      pos += j1 - j0;
      return true;
    }
    return false;
  }
};

// kImp: the launch also feeds the importance map (decider rows look themselves up and store their scores); the
// plain instance carries none of that code, which keeps its softmax loop at the registers and schedule it had.
template <int DH, bool kImp>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_sk_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
               const __grid_constant__ CUtensorMap tmap_v, AttnArgs a, float* __restrict__ part_ws,
               int* __restrict__ part_flags) {
  using S = SkSmem<DH>;
  constexpr int kTileBytes = S::kTileBytes;
  constexpr int kHalfBytes = kTile * 128;
  constexpr int kHalves = DH / 64;
  constexpr int kSlotFloats = 2 * (128 + 2) * kTile;     // per CTA: two tiles of [128 columns][128 rows] + (m, l) per row
  grid_dependency_enter();
  const int lo = a.cu_seqlens[0], n = a.cu_seqlens[1] - lo;
  // deciders are response rows: rows below the visual count cannot be any, and their segments skip the look-up
  const int n_vis = (kImp && a.decider_pos != nullptr) ? a.n_visual[0] : 0;
  const int dec_lo = (kImp && a.decider_pos != nullptr) ? a.cu_deciders[0] : 0, dec_hi = (kImp && a.decider_pos != nullptr) ? a.cu_deciders[1] : 0;
  const int nqb = (n + 2 * kTile - 1) / (2 * kTile), n_kv = (n + kTile - 1) / kTile;
  const int pad = (kImp && a.decider_pos != nullptr) ? (n_kv + 2) / 4 : 0;
  const long long W = (long long)a.H * (nqb * n_kv + pad);
  // a share must be at least one item (and its empty positions) long, so that an item is cut at most once
  const int G = (int)min((long long)gridDim.x, W / (n_kv + pad));
  const int cta = (int)blockIdx.x;
  if (cta >= G || n <= 0) return;                        // uniform; nothing allocated yet
  Walk walk0;
  walk0.pos = (int)((long long)cta * W / G); walk0.hi = (int)((long long)(cta + 1) * W / G);
  walk0.n_kv = n_kv; walk0.nqb = nqb; walk0.n = n; walk0.pad = pad;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_s = smem;
  uint8_t* kv_s = smem + 2 * kTileBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (2 + kKvSlots) * kTileBytes);
  uint64_t* q_full = bars;            // [2] Q tile of slot i has landed
  uint64_t* q_empty = bars + 2;       // [2] every QK^T of the segment in slot i has been computed
  uint64_t* kv_full = bars + 4;       // [2]
  uint64_t* kv_empty = bars + 6;      // [2]
  uint64_t* s_full = bars + 8;        // [2]
  uint64_t* p_lo = bars + 10;         // [2]
  uint64_t* p_hi = bars + 12;         // [2]
  uint64_t* o_final = bars + 14;      // [2]
  uint64_t* o_empty = bars + 16;      // [2] the O tile of slot i has been read out
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 18);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&q_full[i], 1); ptx::mbar_init(&q_empty[i], 4);
      ptx::mbar_init(&kv_full[i], 1); ptx::mbar_init(&kv_empty[i], 4);   // freed by the warps of the segment's last tile
      ptx::mbar_init(&s_full[i], 1);
      ptx::mbar_init(&p_lo[i], 4); ptx::mbar_init(&p_hi[i], 4);
      ptx::mbar_init(&o_final[i], 1); ptx::mbar_init(&o_empty[i], 4);
    }
    *abort_flag = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 0) { ptx::tmem_alloc(tmem_slot, 512); ptx::tmem_relinquish(); }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;
  auto col_s = [](int i) -> uint32_t { return (uint32_t)i * 128u; };
  auto col_o = [](int i) -> uint32_t { return 256u + (uint32_t)i * 128u; };

  if (warp >= 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kOtherRegs));
    if (warp == 8) {
      // ------------------------------------------------------------ TMA producer
      if (lane == 0) {
        ptx::prefetch_tensormap(&tmap_q); ptx::prefetch_tensormap(&tmap_k); ptx::prefetch_tensormap(&tmap_v);
        Walk w = walk0;
        int g = 0, segs[2] = {0, 0};
        bool ok = true;
        while (ok && w.next()) {
          const int ns = w.j1 - w.j0;
          for (int i = 0; i < w.n_qt && ok; ++i) {
            if (segs[i] > 0) ok = ptx::mbar_wait(&q_empty[i], (segs[i] - 1) & 1, abort_flag, a.dev_status);
            if (!ok) break;
            ptx::mbar_arrive_expect_tx(&q_full[i], kTileBytes);
            for (int hf = 0; hf < kHalves; ++hf)
              ptx::tma_load_2d(q_s + i * kTileBytes + hf * kHalfBytes, &tmap_q, &q_full[i], w.h * DH + hf * 64,
                               lo + w.q0 + i * kTile);
            ++segs[i];
          }
          // stage s of the segment = {K of key tile j0 + s, V of key tile j0 + s - 1}; stages are numbered through
          for (int s = 0; s <= ns && ok; ++s) {
            const int gs = g + s, st = gs & 1;
            if (gs >= 2) ok = ptx::mbar_wait(&kv_empty[st], ((gs >> 1) & 1) ^ 1, abort_flag, a.dev_status);
            if (!ok) break;
            const bool has_k = s < ns, has_v = s > 0;
            ptx::mbar_arrive_expect_tx(&kv_full[st], (has_k ? kTileBytes : 0) + (has_v ? kTileBytes : 0));
            for (int hf = 0; hf < kHalves; ++hf) {
              if (has_v) ptx::tma_load_2d(kv_s + (2 * st + 1) * kTileBytes + hf * kHalfBytes, &tmap_v, &kv_full[st],
                                          w.h * DH + hf * 64, lo + (w.j0 + s - 1) * kTile);
              if (has_k) ptx::tma_load_2d(kv_s + (2 * st) * kTileBytes + hf * kHalfBytes, &tmap_k, &kv_full[st],
                                          w.h * DH + hf * 64, lo + (w.j0 + s) * kTile);
            }
          }
          g += ns + 1;
        }
      }
    } else if (warp == 9) {
      // ------------------------------------------------------------ MMA issuer
      if (lane == 0) {
        constexpr uint32_t idesc_qk = ptx::idesc_bf16_f32(kTile, kTile, 0, 0);
        constexpr uint32_t idesc_pv = ptx::idesc_bf16_f32(kTile, DH, 0, 1);
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
        auto issue_pv_half = [&](int i, int slot, int half, bool accumulate) {
          const ptx::SmemDesc vd = ptx::smem_desc_advance(v_desc0, slot * kTileBytes + half * 4 * 2048);
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4) {
            ptx::mma_ts(tmem + col_o(i), tmem + col_s(i) + (half * 4 + k4) * 8, ptx::smem_desc_advance(vd, k4 * 2048),
                        idesc_pv, (accumulate || half > 0 || k4 > 0) ? 1u : 0u);
          }
        };
        Walk w = walk0;
        int g = 0, segs[2] = {0, 0}, cnt[2] = {0, 0};
        bool ok = true;
        while (ok && w.next()) {
          const int ns = w.j1 - w.j0;
          for (int i = 0; i < w.n_qt && ok; ++i) ok = ptx::mbar_wait(&q_full[i], segs[i] & 1, abort_flag, a.dev_status);
          if (ok) ok = ptx::mbar_wait(&kv_full[g & 1], (g >> 1) & 1, abort_flag, a.dev_status);    // first stage: K only
          if (!ok) break;
          ptx::tc_fence_after_sync();
          for (int i = 0; i < w.n_qt; ++i) { issue_qk(i, 2 * (g & 1)); ptx::mma_commit(&s_full[i]); }
          for (int jj = 0; jj < ns && ok; ++jj) {
            const int st = (g + jj + 1) & 1;
            const bool more = jj + 1 < ns;
            for (int i = 0; i < w.n_qt && ok; ++i) {
              const uint32_t ph = (uint32_t)(cnt[i] + jj) & 1u;
              ok = ptx::mbar_wait(&p_lo[i], ph, abort_flag, a.dev_status);
              // the first PV of a segment overwrites the O tile: the segment before must have been read out
              if (ok && jj == 0 && segs[i] > 0) ok = ptx::mbar_wait(&o_empty[i], (segs[i] - 1) & 1, abort_flag, a.dev_status);
              if (!ok) break;
              ptx::tc_fence_after_sync();
              issue_pv_half(i, 2 * st + 1, 0, jj > 0);
              ok = ptx::mbar_wait(&p_hi[i], ph, abort_flag, a.dev_status);
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
          for (int i = 0; i < w.n_qt; ++i) { cnt[i] += ns; ++segs[i]; }
          g += ns + 1;
        }
      }
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kSoftmaxRegs));
    // ------------------------------------------------------------ softmax + epilogue
    const int i = warp >> 2;
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const uint32_t t_s = tmem + lane_addr + col_s(i);
    const uint32_t t_o = tmem + lane_addr + col_o(i);
    const float c = a.scale_log2;
    const float2 c2 = make_float2(c, c);
    Walk w = walk0;
    int g = 0, seg_i = 0, cnt_i = 0;
    bool ok = true;
    while (ok && w.next()) {
      const int ns = w.j1 - w.j0;
      if (i >= w.n_qt) { g += ns + 1; continue; }              // this slot is idle in a one-tile segment
      const bool last_tile = i == w.n_qt - 1;                  // its warps release the K/V stages
      const int q_row = w.q0 + i * kTile + row;
      const bool valid_row = q_row < n;
      int dec_slot = -1;
      if ((kImp && a.decider_pos != nullptr) && valid_row && q_row >= n_vis) {
        int l = dec_lo, r = dec_hi;
        while (l < r) {
          const int mid = (l + r) >> 1, pos = a.decider_pos[mid];
          if (pos == q_row) { dec_slot = mid; break; }
          if (pos < q_row) l = mid + 1; else r = mid;
        }
      }
      float* score_row = dec_slot >= 0 ? a.score_scratch + ((size_t)w.h * a.max_deciders + dec_slot) * a.vis_stride : nullptr;

      float m_used = -INFINITY;
      float2 l2 = make_float2(0.f, 0.f);
      for (int jj = 0; jj < ns; ++jj) {
        const int j = w.j0 + jj;                               // key tile of the request
        const uint32_t ph = (uint32_t)(cnt_i + jj) & 1u;
        ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_full[i], ph, abort_flag, a.dev_status));
        if (!ok) break;
        ptx::tc_fence_after_sync();
        // S of this step is complete: its QK^T has read the stage's K and, issued before it, the PV of the step before
        // has read the stage's V, for this tile and for every tile issued before it
        if (last_tile && lane == 0) ptx::mbar_arrive(&kv_empty[(g + jj) & 1]);
        if (jj == ns - 1 && lane == 0) ptx::mbar_arrive(&q_empty[i]);     // the segment's last QK^T of this tile: Q is free
        uint32_t sr[kTile];
        ptx::tmem_ld32(t_s, sr);
        ptx::tmem_ld32(t_s + 32, sr + 32);
        ptx::tmem_ld32(t_s + 64, sr + 64);
        ptx::tmem_ld32(t_s + 96, sr + 96);
        ptx::tmem_wait_ld();
        const int n_valid = n - j * kTile;
        if (n_valid < kTile) {
#pragma unroll
          for (int e = 0; e < kTile; ++e) if (e >= n_valid) sr[e] = 0xff800000u;
        }
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
        exp_chunk(0, m_used, pk[0], l_tile);
        exp_chunk(1, m_used, pk[1], l_tile);
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
        const bool need = (m_new - m_used) > kRescaleThreshold;
        if (__any_sync(0xffffffffu, need)) {
          const float alpha = need ? exp2f(m_used - m_new) : 1.f;
          if (jj > 0) {                                        // (the O tile of this segment starts at its first step)
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
          l_tile = make_float2(0.f, 0.f);
          exp_chunk(0, m_used, pk[0], l_tile);
          exp_chunk(1, m_used, pk[1], l_tile);
        }
        tmem_st16(t_s, pk[0]);
        tmem_st16(t_s + 16, pk[1]);
        exp_chunk(2, m_used, pk[0], l_tile);
        ptx::tmem_wait_st();
        ptx::tc_fence_before_sync();
        {
          const int gs = g + jj + 1;                           // the stage with this step's V and the next step's K
          ok = __all_sync(0xffffffffu, ptx::mbar_wait(&kv_full[gs & 1], (gs >> 1) & 1, abort_flag, a.dev_status));
        }
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
      // ---- end of the segment
      if (ok) ok = __all_sync(0xffffffffu, ptx::mbar_wait(&o_final[i], seg_i & 1, abort_flag, a.dev_status));
      if (!ok) break;
      ptx::tc_fence_after_sync();
      if (last_tile && lane == 0) ptx::mbar_arrive(&kv_empty[(g + ns) & 1]);      // the segment's last stage (V only)
      const bool is_tail = w.j0 > 0, is_head = w.j1 < n_kv;    // (a share is at least one item long: never both)
      float l_sum = l2.x + l2.y;
      if (is_tail) {
        // the unnormalised O rows and (m, l) go to this CTA's slot; the CTA before this one picks them up
        float* slot = part_ws + (size_t)cta * kSlotFloats + (size_t)i * (128 + 2) * kTile;
#pragma unroll 1
        for (int c0 = 0; c0 < DH; c0 += 32) {
          uint32_t r[32];
          ptx::tmem_ld32(t_o + c0, r);
          ptx::tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) slot[(size_t)(c0 + e) * kTile + row] = __uint_as_float(r[e]);
        }
        slot[(size_t)128 * kTile + row] = m_used;
        slot[(size_t)129 * kTile + row] = l_sum;
        __threadfence();
        __syncwarp();
        if (lane == 0) atomicExch(part_flags + (cta * 2 + i) * 4 + quarter, 1);
      } else {
        float a1 = 1.f, a2 = 0.f;
        const float* other = part_ws + (size_t)(cta + 1) * kSlotFloats + (size_t)i * (128 + 2) * kTile;
        if (is_head) {
          int* flag = part_flags + ((cta + 1) * 2 + i) * 4 + quarter;     // set by the warp that owns the same 32 rows
          ok = __all_sync(0xffffffffu, flag_wait(flag, 1, abort_flag, a.dev_status));
          if (!ok) break;
          __threadfence();
          const float m2 = __ldcg(other + (size_t)128 * kTile + row), lb = __ldcg(other + (size_t)129 * kTile + row);
          const float m = fmaxf(m_used, m2);
          a1 = exp2f(m_used - m); a2 = exp2f(m2 - m);
          l_sum = l_sum * a1 + lb * a2;
          m_used = m;
        }
        const float inv_l = 1.f / l_sum;
        __nv_bfloat16* dst = static_cast<__nv_bfloat16*>(a.out) + ((size_t)(lo + q_row) * a.H + w.h) * DH;
#pragma unroll 1
        for (int c0 = 0; c0 < DH; c0 += 32) {
          uint32_t r[32];
          ptx::tmem_ld32(t_o + c0, r);
          ptx::tmem_wait_ld();
          if (is_head) {
#pragma unroll
            for (int e = 0; e < 32; ++e)
              r[e] = __float_as_uint(__uint_as_float(r[e]) * a1 + __ldcg(other + (size_t)(c0 + e) * kTile + row) * a2);
          }
          if (valid_row) {
#pragma unroll
            for (int e = 0; e < 32; e += 8) {
              uint32_t wv[4];
#pragma unroll
              for (int t = 0; t < 4; ++t)
                wv[t] = pack_bf16x2(__uint_as_float(r[e + 2 * t]) * inv_l, __uint_as_float(r[e + 2 * t + 1]) * inv_l);
              *reinterpret_cast<uint4*>(dst + c0 + e) = make_uint4(wv[0], wv[1], wv[2], wv[3]);
            }
          }
        }
        if (dec_slot >= 0) a.lse_scratch[(size_t)w.h * a.max_deciders + dec_slot] = make_float2(m_used, l_sum);
        if (is_head) {                                         // the slot's flag goes back to zero for the next launch
          __syncwarp();
          if (lane == 0) atomicExch(part_flags + ((cta + 1) * 2 + i) * 4 + quarter, 0);
        }
      }
      // the O tile has been read: the next segment's first PV may overwrite it
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&o_empty[i]);
      cnt_i += ns; ++seg_i;
      g += ns + 1;
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
  auto kernel = a.decider_pos != nullptr ? attn_sk_kernel<DH, true> : attn_sk_kernel<DH, false>;
  D3TOM_CUDA_TRY(ctx, cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SkSmem<DH>::kBytes));
  D3TOM_CUDA_TRY(ctx, launch_serialized(kernel, ctx->sm_count, kAttnThreads, SkSmem<DH>::kBytes, s, tq, tk, tv, a,
                                        ctx->attn_part_ws, ctx->attn_part_flags));
  D3TOM_LAUNCH_CHECK(ctx);
  return D3TOM_OK;
}

}  // namespace

// One request, more work items than SMs and not a whole number of rounds of them: the balanced walk.  Returns
// D3TOM_ERR_UNSUPPORTED when the whole-item kernel of attn_tc.cu should run instead.
int launch_attn_sk(d3tom_ctx* ctx, const AttnArgs& a, cudaStream_t s) {
  if (a.B != 1 || ctx->attn_part_ws == nullptr || ctx->sm_count <= 0) return D3TOM_ERR_UNSUPPORTED;
  const int items = a.H * ceil_div(a.max_seqlen, 2 * kTile), sms = ctx->sm_count;
  if (items <= sms) return D3TOM_ERR_UNSUPPORTED;
  // Whole items cost ceil(items / SMs) rounds.  The balanced walk pays a partial tile per CTA and an epilogue per
  // segment, so it is taken where more than a twentieth of those rounds would be idle.  Measured in one process,
  // alternating (32 heads x 128, us, balanced / whole items): 1216 rows (1.08 rounds) 37.8 / 43.6, 1600 (1.51)
  // 57.7 / 59.1, 2176 (1.95) 81.8 / 72.3, 2500 (2.16) 105.7 / 116.5, 3500 (3.03) 185 / 211, 4288 (3.68) 270 / 283,
  // 6000 (5.19) 533 / 569, 8192 (6.92) 941 / 1026 (noisy under the power cap).
  const int rounds = ceil_div(items, sms);
  if ((long long)(rounds * sms - items) * 20 <= (long long)rounds * sms) return D3TOM_ERR_UNSUPPORTED;
  if (a.dh == 128) return launch<128>(ctx, a, s);
  if (a.dh == 64) return launch<64>(ctx, a, s);
  return D3TOM_ERR_UNSUPPORTED;
}
