// Bidirectional attention, one 128-row query tile per CTA (Sec. 3.2.1, A = softmax(QK^T * scale); the
// post-merge layers of Sec. 3.2.2 run the same kernel on the shortened sequence), head_dim 128, bf16.
//
// The kernel with two query tiles per CTA (attn_tc.cu) is bound by a dependency chain: the scores of
// a tile's next key block can only be computed once the PV product of the current one has consumed
// P, because P lives in the columns of S and tensor memory (512 columns) holds just S and O of two
// tiles.  Here a CTA has ONE query tile, so tensor memory holds THREE score buffers beside O:
//
//   columns   0..127  S buffer 0      key block j uses buffer j % 3; its bf16 P overwrites the first
//           128..255  S buffer 1      64 columns of the buffer and feeds the PV product from there
//           256..383  S buffer 2
//           384..511  O
//
// and QK^T runs three key blocks ahead of PV: the softmax of a key block never waits for the tensor
// pipe, and the pipe never waits for anything but P.  The two softmax warpgroups take the key blocks
// in turn (warps 0-3 the even ones, warps 4-7 the odd ones), each thread one query row, so that two
// warps per scheduler share the special-function unit.  There is one accumulator O, hence one
// reference maximum per row: the warpgroup of key block j takes the reference left by block j-1 from
// shared memory (an mbarrier orders the hand-over), raises it only when the block's maximum exceeds
// it by more than 2^8 (then O is rescaled, after the PV of block j-1 has completed), and passes it
// on.  Each warpgroup keeps its own partial row sum; they are brought to the final reference and
// added at the end.
//
//   warp 8   TMA producer: Q once, K three blocks ahead, V as PV needs it (rings of three 32 KB tiles)
//   warp 9   one thread issues every tcgen05.mma: PV_j (8 instructions), then QK^T_(j+3) into the
//            buffer PV_j has just read
//   warps 10-11 complete the third warpgroup so that registers can move to the softmax warps
//
// Every wait is bounded as everywhere in this library.
#include "common.cuh"
#include "ptx.cuh"

namespace {

constexpr int kTile = 128;
constexpr int kDH = 128;
constexpr int kOneThreads = 384;
constexpr int kSoftmaxRegs = 216, kOtherRegs = 64;
constexpr int kRing = 3;
constexpr float kRescaleThreshold = 8.0f;
constexpr int kTileBytes = kTile * kDH * 2;            // 32 KB
constexpr int kHalfBytes = kTile * 128;                // one 64-column sub-tile: 128 rows x 128 bytes
constexpr int kOneSmem = (1 + 2 * kRing) * kTileBytes + 1024 /*alignment*/ + 256 /*barriers*/ + 512 /*reference*/ + 1024 /*sums*/;

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
// a plain barrier of the 256 softmax threads (both warpgroups always reach it, also after a wait has run out)
__device__ __forceinline__ void bar_sync_softmax() { asm volatile("bar.sync 2, 256;" ::: "memory"); }

__global__ void __launch_bounds__(kOneThreads, 1)
attn_one_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                const __grid_constant__ CUtensorMap tmap_v, AttnArgs a) {
  grid_dependency_enter();
  // Work items: per request H x nqb query tiles (nqb = tiles of the longest request), heads outermost so that the
  // CTAs of a wave share a head's K and V in L2; requests of a batch longest first.
  const int per_req = a.H * a.nqb;
  int b = (int)blockIdx.x / per_req;
  const int lin = (int)blockIdx.x - b * per_req;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (a.B > 1 && a.B <= 32) {
    const int nl = lane < a.B ? a.cu_seqlens[lane + 1] - a.cu_seqlens[lane] : -1;
    int rank = 0;
    for (int o = 0; o < a.B; ++o) {
      const int no = __shfl_sync(0xffffffffu, nl, o);
      rank += (no > nl || (no == nl && o < lane)) ? 1 : 0;
    }
    b = __ffs(__ballot_sync(0xffffffffu, lane < a.B && rank == b)) - 1;
  }
  const int h = lin / a.nqb, qt = a.nqb - 1 - lin % a.nqb;
  const int lo = a.cu_seqlens[b], n = a.cu_seqlens[b + 1] - lo;
  const int q0 = qt * kTile;
  if (q0 >= n) return;                                  // uniform; nothing allocated yet
  const int n_kv = (n + kTile - 1) / kTile;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_s = smem;
  uint8_t* k_s = smem + kTileBytes;                     // ring of three K tiles
  uint8_t* v_s = k_s + kRing * kTileBytes;              // ring of three V tiles
  uint64_t* bars = reinterpret_cast<uint64_t*>(v_s + kRing * kTileBytes);
  uint64_t* q_full = bars;                              // [1]
  uint64_t* k_full = bars + 1;                          // [3]
  uint64_t* v_full = bars + 7;                          // [3]
  uint64_t* pv_done = bars + 10;                        // [3] PV_t has completed, for the last blocks, which no QK^T follows
  uint64_t* s_full = bars + 13;                         // [3]
  uint64_t* p_ready = bars + 16;                        // [3]
  uint64_t* o_final = bars + 19;                        // [1]
  uint64_t* m_pub = bars + 20;                          // [2] the reference for key block j is in shared memory (j & 1)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 22);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* m_sh = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(bars) + 256);      // [128] reference handed on
  float* l_sh = m_sh + 128;                                                          // [2][128] partial row sums

  if (threadIdx.x == 0) {
    ptx::mbar_init(q_full, 1); ptx::mbar_init(o_final, 1);
    ptx::mbar_init(&m_pub[0], 4); ptx::mbar_init(&m_pub[1], 4);      // one arrival per warp of the publishing warpgroup
    for (int s = 0; s < kRing; ++s) {
      ptx::mbar_init(&k_full[s], 1); ptx::mbar_init(&v_full[s], 1); ptx::mbar_init(&pv_done[s], 1);
      ptx::mbar_init(&s_full[s], 1); ptx::mbar_init(&p_ready[s], 4);
    }
    *abort_flag = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 0) { ptx::tmem_alloc(tmem_slot, 512); ptx::tmem_relinquish(); }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;
  constexpr uint32_t kColO = 384;

  if (warp >= 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kOtherRegs));
    if (warp == 8) {
      // ------------------------------------------------------------ TMA producer
      if (lane == 0) {
        ptx::prefetch_tensormap(&tmap_q); ptx::prefetch_tensormap(&tmap_k); ptx::prefetch_tensormap(&tmap_v);
        auto load_tile = [&](uint8_t* dst, const CUtensorMap* tm, uint64_t* bar, int row) {
          ptx::mbar_arrive_expect_tx(bar, kTileBytes);
          for (int hf = 0; hf < kDH / 64; ++hf) ptx::tma_load_2d(dst + hf * kHalfBytes, tm, bar, h * kDH + hf * 64, row);
        };
        load_tile(q_s, &tmap_q, q_full, lo + q0);
        bool ok = true;
        for (int t = 0; t < kRing && t < n_kv; ++t) load_tile(k_s + t * kTileBytes, &tmap_k, &k_full[t], lo + t * kTile);
        // Then, per key block j: V_j for its PV and K_(j+3) for the QK^T that follows it, both into slot j % 3.  The slot's
        // last readers were PV_(j-3) and QK^T_j, and the commit behind QK^T_j (s_full of block j) covers both, so this
        // thread watches that barrier and the issuing thread spends no commit of its own on the rings.
        for (int j = 0; j < n_kv && ok; ++j) {
          const int s = j % kRing, u = j / kRing;
          if (u == 0) load_tile(v_s + s * kTileBytes, &tmap_v, &v_full[s], lo + j * kTile);   // (a fresh V slot)
          ok = ptx::mbar_wait(&s_full[s], u & 1, abort_flag, a.dev_status);
          if (!ok) break;
          if (u > 0) load_tile(v_s + s * kTileBytes, &tmap_v, &v_full[s], lo + j * kTile);
          if (j + kRing < n_kv) load_tile(k_s + s * kTileBytes, &tmap_k, &k_full[s], lo + (j + kRing) * kTile);
        }
      }
    } else if (warp == 9) {
      // ------------------------------------------------------------ MMA issuer
      if (lane == 0) {
        constexpr uint32_t idesc_qk = ptx::idesc_bf16_f32(kTile, kTile, 0, 0);   // S = Q K^T, both K-major
        constexpr uint32_t idesc_pv = ptx::idesc_bf16_f32(kTile, kDH, 0, 1);     // O += P V, V is MN-major
        const ptx::SmemDesc q_desc = ptx::smem_desc_kmajor_sw128(ptx::smem_u32(q_s));
        const ptx::SmemDesc k_desc0 = ptx::smem_desc_kmajor_sw128(ptx::smem_u32(k_s));
        const ptx::SmemDesc v_desc0 = ptx::smem_desc_mnmajor_sw128(ptx::smem_u32(v_s), kHalfBytes);
        auto issue_qk = [&](int buf) {
          const ptx::SmemDesc kd = ptx::smem_desc_advance(k_desc0, buf * kTileBytes);
#pragma unroll
          for (int kk = 0; kk < kDH / 16; ++kk) {
            const uint32_t off = (kk / 4) * kHalfBytes + (kk % 4) * 32;
            ptx::mma_ss(tmem + (uint32_t)buf * 128u, ptx::smem_desc_advance(q_desc, off), ptx::smem_desc_advance(kd, off),
                        idesc_qk, kk > 0 ? 1u : 0u);
          }
        };
        auto issue_pv = [&](int buf, bool accumulate) {
          const ptx::SmemDesc vd = ptx::smem_desc_advance(v_desc0, buf * kTileBytes);
#pragma unroll
          for (int k8 = 0; k8 < 8; ++k8) {                        // 16 keys per instruction
            ptx::mma_ts(tmem + kColO, tmem + (uint32_t)buf * 128u + k8 * 8, ptx::smem_desc_advance(vd, k8 * 2048), idesc_pv,
                        (accumulate || k8 > 0) ? 1u : 0u);
          }
        };
        bool ok = ptx::mbar_wait(q_full, 0, abort_flag, a.dev_status);
        for (int t = 0; t < kRing && t < n_kv && ok; ++t) {
          ok = ptx::mbar_wait(&k_full[t], 0, abort_flag, a.dev_status);
          if (!ok) break;
          ptx::tc_fence_after_sync();
          issue_qk(t);
          ptx::mma_commit(&s_full[t]);
        }
        // Per key block: one barrier check (P_j; the softmax warps have also seen V_j and K_(j+3) land), sixteen
        // instructions, one commit.  Whatever this thread does between instructions is idle time of the tensor pipe.
        for (int j = 0; j < n_kv && ok; ++j) {
          const int buf = j % kRing, u = j / kRing;
          ok = ptx::mbar_wait(&p_ready[buf], u & 1, abort_flag, a.dev_status);
          if (!ok) break;
          ptx::tc_fence_after_sync();
          issue_pv(buf, j > 0);
          if (j + kRing < n_kv) {
            issue_qk(buf);                                          // into the buffer PV_j has just read (in issue order)
            ptx::mma_commit(&s_full[buf]);
          } else if (j == n_kv - 1) {
            ptx::mma_commit(o_final);
          } else {
            ptx::mma_commit(&pv_done[buf]);
          }
        }
      }
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kSoftmaxRegs));
    // ------------------------------------------------------------ softmax (key blocks in turn) + epilogue
    const int wg = warp >> 2;                      // 0: even key blocks, 1: odd key blocks
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;           // row of the tile == TMEM lane
    const int q_row = q0 + row;
    const bool valid_row = q_row < n;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const uint32_t t_o = tmem + lane_addr + kColO;
    const float c = a.scale_log2;
    const float2 c2 = make_float2(c, c);
    float m_mine = -INFINITY;                      // the reference my partial sum is expressed in
    float2 l2 = make_float2(0.f, 0.f);
    bool ok = true;
    for (int j = wg; j < n_kv; j += 2) {
      const int buf = j % kRing, u = j / kRing;
      const uint32_t t_s = tmem + lane_addr + (uint32_t)buf * 128u;
      ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_full[buf], u & 1, abort_flag, a.dev_status));
      if (!ok) break;
      ptx::tc_fence_after_sync();
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
      // ---- row maximum of the block
      float mx[8];
#pragma unroll
      for (int t = 0; t < 8; ++t) mx[t] = fmaxf(__uint_as_float(sr[2 * t]), __uint_as_float(sr[2 * t + 1]));
#pragma unroll
      for (int e = 16; e < kTile; e += 16)
#pragma unroll
        for (int t = 0; t < 8; ++t)
          mx[t] = max3(mx[t], __uint_as_float(sr[e + 2 * t]), __uint_as_float(sr[e + 2 * t + 1]));
      const float mxa = max3(max3(mx[0], mx[1], mx[2]), max3(mx[3], mx[4], mx[5]), fmaxf(mx[6], mx[7]));
      // ---- the reference left by key block j-1 (the other warpgroup), raised only when this block needs it
      float m_prev = -INFINITY;
      if (j > 0) {                                                     // (bounded like every wait; use (j - 1) / 2 of the barrier)
        ok = __all_sync(0xffffffffu, ptx::mbar_wait(&m_pub[j & 1], ((j - 1) >> 1) & 1, abort_flag, a.dev_status));
        if (!ok) break;
        m_prev = m_sh[row];
      }
      const float m_new = fmaxf(m_prev, mxa * c);
      const bool need = (m_new - m_prev) > kRescaleThreshold;        // first block: inf > threshold
      const float m_ref = need ? m_new : m_prev;
      if (j + 1 < n_kv) {                                              // hand it on before anything slow
        m_sh[row] = m_ref;
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&m_pub[(j + 1) & 1]);
      }
      if (__any_sync(0xffffffffu, need) && j > 0) {
        // O was accumulated against m_prev: PV_(j-1) must have completed before it is rescaled, and PV_j waits for
        // this warpgroup's announcement below
        // (PV_(j-1) is followed by QK^T_(j+2), whose commit covers it; the last blocks have a barrier of their own)
        if (j + 2 < n_kv) ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_full[(j + 2) % kRing], ((j + 2) / kRing) & 1, abort_flag, a.dev_status));
        else ok = __all_sync(0xffffffffu, ptx::mbar_wait(&pv_done[(j - 1) % kRing], 0, abort_flag, a.dev_status));
        if (!ok) break;
        ptx::tc_fence_after_sync();
        const float alpha = need ? exp2f(m_prev - m_new) : 1.f;
#pragma unroll 1
        for (int c0 = 0; c0 < kDH; c0 += 32) {
          uint32_t r[32];
          ptx::tmem_ld32(t_o + c0, r);
          ptx::tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
          ptx::tmem_st32(t_o + c0, r);
        }
        ptx::tmem_wait_st();
      }
      if (m_ref != m_mine) {                                           // my partial sum moves to the new reference
        const float beta = (l2.x + l2.y) > 0.f ? exp2f(m_mine - m_ref) : 0.f;
        l2.x *= beta; l2.y *= beta;
        m_mine = m_ref;
      }
      // ---- p = exp2(s*c - m_ref), bf16 P into the first 64 columns of the buffer
      const float2 nm2 = make_float2(-m_ref, -m_ref);
      float2 l_tile = make_float2(0.f, 0.f);
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        float2 t2[16];
        uint32_t pk[16];
#pragma unroll
        for (int e = 0; e < 16; ++e)
          t2[e] = __ffma2_rn(make_float2(__uint_as_float(sr[ch * 32 + 2 * e]), __uint_as_float(sr[ch * 32 + 2 * e + 1])), c2, nm2);
#pragma unroll
        for (int e = 0; e < 16; ++e) { t2[e].x = ptx::ex2(t2[e].x); t2[e].y = ptx::ex2(t2[e].y); }
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          pk[e] = pack_bf16x2(t2[e].x, t2[e].y);
          l_tile = __fadd2_rn(l_tile, t2[e]);
        }
        tmem_st16(t_s + ch * 16, pk);
      }
      l2 = __fadd2_rn(l2, l_tile);
      ptx::tmem_wait_st();
      ptx::tc_fence_before_sync();
      // V_j must have landed before the tensor pipe is sent on (the issuing thread does not check)
      ok = __all_sync(0xffffffffu, ptx::mbar_wait(&v_full[buf], u & 1, abort_flag, a.dev_status));
      if (ok && j + kRing < n_kv)                        // and K_(j+3), which the QK^T behind PV_j reads
        ok = __all_sync(0xffffffffu, ptx::mbar_wait(&k_full[buf], (u + 1) & 1, abort_flag, a.dev_status));
      if (!ok) break;
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&p_ready[buf]);
    }
    // ---- the two partial sums at the final reference (both warpgroups come here, also after an abort)
    const int g_last = (n_kv - 1) & 1;
    if (wg == g_last) m_sh[row] = m_mine;
    bar_sync_softmax();
    const float m_fin = m_sh[row];
    float l_part = l2.x + l2.y;
    if (m_mine != m_fin) l_part = l_part > 0.f ? l_part * exp2f(m_mine - m_fin) : 0.f;
    l_sh[wg * 128 + row] = l_part;
    bar_sync_softmax();
    const float l_sum = l_sh[row] + l_sh[128 + row];
    // ---- epilogue: O / l -> bf16 -> global; each warpgroup writes half of the columns
    if (ok) ok = __all_sync(0xffffffffu, ptx::mbar_wait(o_final, 0, abort_flag, a.dev_status));
    ptx::tc_fence_after_sync();
    if (ok) {
      const float inv_l = 1.f / l_sum;
      __nv_bfloat16* dst = static_cast<__nv_bfloat16*>(a.out) + ((size_t)(lo + q_row) * a.H + h) * kDH + wg * 64;
#pragma unroll 1
      for (int c0 = 0; c0 < 64; c0 += 32) {
        uint32_t r[32];
        ptx::tmem_ld32(t_o + wg * 64 + c0, r);
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
    }
    ptx::tc_fence_before_sync();
  }
  __syncthreads();
  if (warp == 0) ptx::tmem_dealloc(tmem, 512);
}

}  // namespace

// Plain attention (no importance side-work) at head_dim 128; D3TOM_ERR_UNSUPPORTED otherwise.
int launch_attn_one(d3tom_ctx* ctx, const AttnArgs& a, cudaStream_t s) {
  if (a.dh != kDH || a.decider_pos != nullptr) return D3TOM_ERR_UNSUPPORTED;
  CUtensorMap tq, tk, tv;
  const uint64_t rows = (uint64_t)a.total_tokens, cols = (uint64_t)a.H * kDH;
  int r = make_tmap_bf16_2d(&tq, a.q, rows, cols, cols, kTile);
  if (r == 0) r = make_tmap_bf16_2d(&tk, a.k, rows, cols, cols, kTile);
  if (r == 0) r = make_tmap_bf16_2d(&tv, a.v, rows, cols, cols, kTile);
  if (r != 0) { ctx->last_cuda_error = r; return D3TOM_ERR_CUDA; }
  D3TOM_CUDA_TRY(ctx, cudaFuncSetAttribute(attn_one_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kOneSmem));
  AttnArgs k = a;
  k.nqb = ceil_div(a.max_seqlen, kTile);
  const int grid = a.B * a.H * k.nqb;
  if (grid <= 0) return D3TOM_OK;
  D3TOM_CUDA_TRY(ctx, launch_serialized(attn_one_kernel, grid, kOneThreads, kOneSmem, s, tq, tk, tv, k));
  D3TOM_LAUNCH_CHECK(ctx);
  return D3TOM_OK;
}
