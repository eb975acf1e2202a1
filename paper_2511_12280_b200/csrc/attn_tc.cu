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
//   warp  8     TMA producer: Q tiles once, then K_j / V_j tiles through a ring
//   warp  9     one thread issues every tcgen05.mma
// TMEM (512 columns): S0 | S1 (128 fp32 columns each; the bf16 P tile overwrites
// the first 64 columns of its S tile) | O0 | O1 (head_dim fp32 columns each).
// Per key tile j and query tile i:  S_i = Q_i K_j^T  ->  softmax warps read S_i,
// write P_i  ->  O_i += P_i V_j.  The running maximum is only raised when the
// new one exceeds it by more than 2^8 (the O tile is then rescaled in place by
// its own softmax warps); sums and outputs are exact for any reference maximum.
#include "common.cuh"
#include "ptx.cuh"

namespace {

constexpr int kTile = 128;            // query rows per tile and keys per tile
constexpr int kAttnThreads = 320;
constexpr int kKvSlots = 4;
constexpr float kRescaleThreshold = 8.0f;

template <int DH> struct AttnSmem {
  static constexpr int kTileBytes = kTile * DH * 2;
  static constexpr int kBytes = 2 * kTileBytes + kKvSlots * kTileBytes + 1024 + 256;
};

template <int DH>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
               const __grid_constant__ CUtensorMap tmap_v, AttnArgs a) {
  using S = AttnSmem<DH>;
  constexpr int kTileBytes = S::kTileBytes;
  constexpr int kHalfBytes = kTile * 128;               // one 64-column sub-tile: 128 rows x 128 bytes
  constexpr int kHalves = DH / 64;
  const int b = blockIdx.z, h = blockIdx.y;
  const int lo = a.cu_seqlens[b], n = a.cu_seqlens[b + 1] - lo;
  const int q0 = blockIdx.x * 2 * kTile;
  if (q0 >= n) return;                                  // uniform; nothing allocated yet
  const int n_qt = (n - q0 > kTile) ? 2 : 1;
  const int n_kv = (n + kTile - 1) / kTile;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_s = smem;                                  // 2 tiles
  uint8_t* kv_s = smem + 2 * kTileBytes;                // ring: K_0, V_0, K_1, V_1, ...
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (2 + kKvSlots) * kTileBytes);
  uint64_t* q_full = bars;                              // [2]
  uint64_t* kv_full = bars + 2;                         // [4]
  uint64_t* kv_empty = bars + 6;                        // [4]
  uint64_t* s_full = bars + 10;                         // [2]
  uint64_t* p_full = bars + 12;                         // [2]
  uint64_t* o_final = bars + 14;                        // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 16);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&q_full[i], 1); ptx::mbar_init(&s_full[i], 1);
      ptx::mbar_init(&p_full[i], kTile); ptx::mbar_init(&o_final[i], 1);
    }
    for (int s = 0; s < kKvSlots; ++s) { ptx::mbar_init(&kv_full[s], 1); ptx::mbar_init(&kv_empty[s], 1); }
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
      for (int it = 0; it < 2 * n_kv; ++it) {             // it = 2j: K_j, it = 2j+1: V_j
        const int slot = it % kKvSlots, j = it >> 1;
        if (!ptx::mbar_wait(&kv_empty[slot], ((it / kKvSlots) & 1) ^ 1, abort_flag, a.dev_status)) break;
        ptx::mbar_arrive_expect_tx(&kv_full[slot], kTileBytes);
        const CUtensorMap* tm = (it & 1) ? &tmap_v : &tmap_k;
        for (int hf = 0; hf < kHalves; ++hf)
          ptx::tma_load_2d(kv_s + slot * kTileBytes + hf * kHalfBytes, tm, &kv_full[slot], h * DH + hf * 64,
                           lo + j * kTile);
      }
    }
  } else if (warp == 9) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_qk = ptx::idesc_bf16_f32(kTile, kTile, 0, 0);   // S = Q K^T, both K-major
      constexpr uint32_t idesc_pv = ptx::idesc_bf16_f32(kTile, DH, 0, 1);      // O += P V, V is MN-major
      auto issue_qk = [&](int i, int slot) {
        const uint32_t qa = ptx::smem_u32(q_s + i * kTileBytes), ka = ptx::smem_u32(kv_s + slot * kTileBytes);
#pragma unroll
        for (int kk = 0; kk < DH / 16; ++kk) {
          const uint32_t off = (kk / 4) * kHalfBytes + (kk % 4) * 32;
          ptx::mma_ss(tmem + col_s(i), ptx::smem_desc_kmajor_sw128(qa + off), ptx::smem_desc_kmajor_sw128(ka + off),
                      idesc_qk, kk > 0 ? 1u : 0u);
        }
      };
      auto issue_pv = [&](int i, int slot, bool accumulate) {
        const uint32_t va = ptx::smem_u32(kv_s + slot * kTileBytes);
#pragma unroll
        for (int kk = 0; kk < kTile / 16; ++kk) {            // 16 keys per instruction
          ptx::mma_ts(tmem + col_o(i), tmem + col_s(i) + kk * 8,
                      ptx::smem_desc_mnmajor_sw128(va + kk * 2048, kHalfBytes), idesc_pv,
                      (accumulate || kk > 0) ? 1u : 0u);
        }
      };
      bool ok = true;
      for (int i = 0; i < n_qt && ok; ++i) ok = ptx::mbar_wait(&q_full[i], 0, abort_flag, a.dev_status);
      if (ok) ok = ptx::mbar_wait(&kv_full[0], 0, abort_flag, a.dev_status);     // K_0
      if (ok) {
        ptx::tc_fence_after_sync();
        for (int i = 0; i < n_qt; ++i) { issue_qk(i, 0); ptx::mma_commit(&s_full[i]); }
        ptx::mma_commit(&kv_empty[0]);
      }
      for (int j = 0; j < n_kv && ok; ++j) {
        const int itv = 2 * j + 1, itk = 2 * j + 2;
        const int vslot = itv % kKvSlots, kslot = itk % kKvSlots;
        const bool more = j + 1 < n_kv;
        for (int i = 0; i < n_qt && ok; ++i) {
          ok = ptx::mbar_wait(&p_full[i], j & 1, abort_flag, a.dev_status);        // P_j(i) written, O_i consistent
          if (ok && i == 0) ok = ptx::mbar_wait(&kv_full[vslot], (itv / kKvSlots) & 1, abort_flag, a.dev_status);
          if (!ok) break;
          ptx::tc_fence_after_sync();
          issue_pv(i, vslot, j > 0);
          if (i == n_qt - 1) ptx::mma_commit(&kv_empty[vslot]);
          if (more) {
            if (i == 0) ok = ptx::mbar_wait(&kv_full[kslot], (itk / kKvSlots) & 1, abort_flag, a.dev_status);
            if (!ok) break;
            ptx::tc_fence_after_sync();
            issue_qk(i, kslot);
            ptx::mma_commit(&s_full[i]);
            if (i == n_qt - 1) ptx::mma_commit(&kv_empty[kslot]);
          } else {
            ptx::mma_commit(&o_final[i]);
          }
        }
      }
    }
  } else {
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
      int dec_slot = -1, n_vis = 0;
      if (a.decider_pos != nullptr && valid_row) {
        n_vis = a.n_visual[b];
        int l = a.cu_deciders[b], r = a.cu_deciders[b + 1];
        while (l < r) {
          const int mid = (l + r) >> 1, pos = a.decider_pos[mid];
          if (pos == q_row) { dec_slot = mid; break; }
          if (pos < q_row) l = mid + 1; else r = mid;
        }
      }
      float* score_row = dec_slot >= 0 ? a.score_scratch + ((size_t)h * a.max_deciders + dec_slot) * a.vis_stride : nullptr;

      float m_used = -INFINITY, l_sum = 0.f;
      const float c = a.scale_log2;
      bool ok = true;
      for (int j = 0; j < n_kv; ++j) {
        ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_full[i], j & 1, abort_flag, a.dev_status));
        if (!ok) break;
        ptx::tc_fence_after_sync();
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
        if (score_row != nullptr) {                         // decider row: raw scores over the visual keys
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
        float mx0 = __uint_as_float(sr[0]), mx1 = __uint_as_float(sr[1]), mx2 = __uint_as_float(sr[2]),
              mx3 = __uint_as_float(sr[3]);
#pragma unroll
        for (int e = 4; e < kTile; e += 4) {
          mx0 = fmaxf(mx0, __uint_as_float(sr[e]));     mx1 = fmaxf(mx1, __uint_as_float(sr[e + 1]));
          mx2 = fmaxf(mx2, __uint_as_float(sr[e + 2])); mx3 = fmaxf(mx3, __uint_as_float(sr[e + 3]));
        }
        const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
        const float m_new = fmaxf(m_used, mx * c);
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
          l_sum *= alpha;
          if (need) m_used = m_new;
        }
        // ---- p = exp2(s*c - m), row sum, bf16 P tile into the first 64 columns of the S tile
        const float neg_m = -m_used;
        float sum0 = 0.f, sum1 = 0.f, sum2 = 0.f, sum3 = 0.f;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          uint32_t pk[32];
#pragma unroll
          for (int e = 0; e < 64; e += 4) {
            const int x = half * 64 + e;
            const float p0 = ptx::ex2(fmaf(__uint_as_float(sr[x]), c, neg_m));
            const float p1 = ptx::ex2(fmaf(__uint_as_float(sr[x + 1]), c, neg_m));
            const float p2 = ptx::ex2(fmaf(__uint_as_float(sr[x + 2]), c, neg_m));
            const float p3 = ptx::ex2(fmaf(__uint_as_float(sr[x + 3]), c, neg_m));
            sum0 += p0; sum1 += p1; sum2 += p2; sum3 += p3;
            __nv_bfloat162 h01 = __floats2bfloat162_rn(p0, p1), h23 = __floats2bfloat162_rn(p2, p3);
            pk[e >> 1] = *reinterpret_cast<uint32_t*>(&h01);
            pk[(e >> 1) + 1] = *reinterpret_cast<uint32_t*>(&h23);
          }
          ptx::tmem_st32(t_s + half * 32, pk);             // keys 64*half .. +63 -> P columns 32*half .. +31
        }
        l_sum += (sum0 + sum1) + (sum2 + sum3);
        ptx::tmem_wait_st();
        ptx::tc_fence_before_sync();
        ptx::mbar_arrive(&p_full[i]);
      }
      // ---- epilogue: O / l -> bf16 -> global
      if (ok) ok = __all_sync(0xffffffffu, ptx::mbar_wait(&o_final[i], 0, abort_flag, a.dev_status));
      ptx::tc_fence_after_sync();
      if (ok) {
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
              for (int t = 0; t < 4; ++t) {
                __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(r[e + 2 * t]) * inv_l,
                                                          __uint_as_float(r[e + 2 * t + 1]) * inv_l);
                w[t] = *reinterpret_cast<uint32_t*>(&h2);
              }
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
  D3TOM_CUDA_TRY(ctx, cudaFuncSetAttribute(attn_tc_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           AttnSmem<DH>::kBytes));
  dim3 grid(ceil_div(a.max_seqlen, 2 * kTile), a.H, a.B);
  attn_tc_kernel<DH><<<grid, kAttnThreads, AttnSmem<DH>::kBytes, s>>>(tq, tk, tv, a);
  D3TOM_LAUNCH_CHECK(ctx);
  return D3TOM_OK;
}

}  // namespace

int launch_attn_tc(d3tom_ctx* ctx, const AttnArgs& a, cudaStream_t s) {
  if (a.dh == 128) return launch<128>(ctx, a, s);
  if (a.dh == 64) return launch<64>(ctx, a, s);
  return D3TOM_ERR_UNSUPPORTED;
}
