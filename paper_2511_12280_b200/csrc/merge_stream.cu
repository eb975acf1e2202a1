// Aggregation and compaction of the merge (Sec. 3.2.2, h_k* <- h_k* + h_m, and the
// physical removal of the merged positions) as a streaming pipeline.
//
// The work is HBM-bound: every input row is read once, every output row written
// once.  A work item is (output row, column segment).  In each CTA one producer
// warp takes items from a global counter, looks up the item's ordered source rows
// (the kept row, then its members in ascending position; one row for a copied
// prompt / response row) and streams their segments into a ring of shared-memory
// slots with bulk asynchronous copies; it runs ahead of the four consumer warps,
// across item boundaries, so the index lookups of later items are hidden behind
// the copies of earlier ones and the bytes in flight do not depend on registers.
// The consumers add the slots in ring order (fp32, so the order of addition is the
// sorted source order: reproducible), scale and round once, and store the row.
#include "common.cuh"
#include "ptx.cuh"

namespace {

constexpr int kConsumerWarps = 4;
constexpr int kStreamThreads = 32 * (1 + kConsumerWarps);
constexpr int kMaxSlots = 32;
constexpr int kRingBytes = 32 * 1024;
constexpr int kMaxVecPerThread = 4;        // 16-byte vectors of a segment per consumer thread
constexpr int kStreamMinRows = 4096;       // fewer output rows than this go to the plain kernel
constexpr int kHeavyList = 32;             // lists of this many members or more are already sorted in memory

__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(ptx::smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(ptx::smem_u32(bar))
               : "memory");
}

template <typename T> __device__ __forceinline__ void add_vec(float (&acc)[Storage<T>::kVec], uint4 raw);
template <> __device__ __forceinline__ void add_vec<float>(float (&acc)[4], uint4 raw) {
  acc[0] += __uint_as_float(raw.x); acc[1] += __uint_as_float(raw.y);
  acc[2] += __uint_as_float(raw.z); acc[3] += __uint_as_float(raw.w);
}
template <> __device__ __forceinline__ void add_vec<__nv_bfloat16>(float (&acc)[8], uint4 raw) {
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    acc[2 * i] += __uint_as_float(w[i] << 16);
    acc[2 * i + 1] += __uint_as_float(w[i] & 0xffff0000u);
  }
}

struct StreamParams {
  const void* hidden; void* hidden_out;
  const int4* row_desc;            // per output row: {source row, members or -1 (copy), list offset, request's first row}
  const int32_t* member_list;
  int32_t* src_of_dst;
  int* work_counter;               // [0] next work item, [1] CTAs done; both zero at launch, the last CTA zeroes them again
  int* dev_status;
  int total_out, D, col_splits, seg_bytes, slots, mean;
};

// slot header: x = output row (-1: no more work), y = bit 0 first source, bit 1 last source, bits 8.. column segment,
//              z = member count of the row, w = source row of the output row (for src_of_dst)
template <typename T>
__global__ void __launch_bounds__(kStreamThreads)
aggregate_stream_kernel(StreamParams p) {
  constexpr int kVec = Storage<T>::kVec;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
  __shared__ int4 header[kMaxSlots];
  __shared__ uint64_t full[kMaxSlots], empty[kMaxSlots];
  __shared__ int abort_word;
  volatile int* abort_flag = &abort_word;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int R = p.slots;
  if (threadIdx.x == 0) {
    for (int s = 0; s < R; ++s) { ptx::mbar_init(&full[s], 1); ptx::mbar_init(&empty[s], kConsumerWarps); }
    abort_word = 0;
    ptx::fence_mbar_init();
  }
  grid_dependency_wait();
  grid_dependency_release();
  __syncthreads();
  const int seg_elems = p.seg_bytes / (int)sizeof(T);
  const long long n_items = (long long)p.total_out * p.col_splits;

  if (warp == 0) {
    // ------------------------------------------------------------ producer warp
    const T* hidden = static_cast<const T*>(p.hidden);
    int it = 0;                                       // slots filled so far
    bool ok = true;
    // pushes one source segment; lane 0 does the waiting and the copy
    auto push = [&](int out_row, int src_row, int cq, int flags, int cnt, int src_of_row) {
      if (lane == 0 && ok) {
        const int s = it % R;
        ok = ptx::mbar_wait(&empty[s], ((it / R) & 1) ^ 1, abort_flag, p.dev_status);
        if (ok) {
          header[s] = make_int4(out_row, flags | (cq << 8), cnt, src_of_row);
          ptx::mbar_arrive_expect_tx(&full[s], (uint32_t)p.seg_bytes);
          bulk_load(ring + (size_t)s * p.seg_bytes, hidden + (size_t)src_row * p.D + (size_t)cq * seg_elems,
                    (uint32_t)p.seg_bytes, &full[s]);
        }
      }
      ++it;
    };
    while (true) {
      long long item = 0;
      if (lane == 0) item = atomicAdd(p.work_counter, 1);
      item = __shfl_sync(0xffffffffu, item, 0);
      ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
      if (item >= n_items || !ok) break;
      const int row = (int)(item / p.col_splits), cq = (int)(item - (long long)row * p.col_splits);
      const int4 d = p.row_desc[row];
      const int cnt = d.y < 0 ? 0 : d.y, lo = d.w;
      push(row, d.x, cq, 1 | (cnt == 0 ? 2 : 0), cnt, d.x);          // the kept (or copied) row itself comes first
      if (cnt == 0) continue;
      if (cnt < kHeavyList) {
        // short list, in arrival order in memory: rank it inside the warp (distinct positions)
        const int mine = lane < cnt ? p.member_list[d.z + lane] : 0x7fffffff;
        int rank = 0;
        for (int j = 0; j < cnt; ++j) rank += __shfl_sync(0xffffffffu, mine, j) < mine ? 1 : 0;
        int ordered = 0;
        for (int j = 0; j < cnt; ++j) {
          const int v = __shfl_sync(0xffffffffu, mine, j), rj = __shfl_sync(0xffffffffu, rank, j);
          if (lane == rj) ordered = v;
        }
        for (int i = 0; i < cnt; ++i)
          push(row, lo + __shfl_sync(0xffffffffu, ordered, i), cq, i == cnt - 1 ? 2 : 0, cnt, d.x);
      } else {
        // long list, already ascending in memory: 32 positions per load
        for (int base = 0; base < cnt; base += 32) {
          const int m = base + lane < cnt ? p.member_list[d.z + base + lane] : 0;
          const int n = min(32, cnt - base);
          for (int i = 0; i < n; ++i)
            push(row, lo + __shfl_sync(0xffffffffu, m, i), cq, base + i == cnt - 1 ? 2 : 0, cnt, d.x);
        }
      }
    }
    // tell the consumers that nothing follows
    if (lane == 0 && ok) {
      const int s = it % R;
      if (ptx::mbar_wait(&empty[s], ((it / R) & 1) ^ 1, abort_flag, p.dev_status)) {
        header[s] = make_int4(-1, 0, 0, 0);
        ptx::mbar_arrive(&full[s]);
      }
    }
    // this CTA takes no more work; the last CTA to say so leaves both counters at zero for the next launch
    if (lane == 0) {
      __threadfence();
      if (atomicAdd(p.work_counter + 1, 1) == (int)gridDim.x - 1) { p.work_counter[0] = 0; p.work_counter[1] = 0; }
    }
  } else {
    // ------------------------------------------------------------ consumer warps: 128 threads, 16 bytes per thread and pass
    const int ct = threadIdx.x - 32;
    T* out = static_cast<T*>(p.hidden_out);
    float acc[kMaxVecPerThread][kVec];
    for (int it = 0;; ++it) {
      const int s = it % R;
      if (!__all_sync(0xffffffffu, ptx::mbar_wait(&full[s], (it / R) & 1, abort_flag, p.dev_status))) break;
      const int4 h = header[s];
      if (h.x < 0) break;
      const uint8_t* seg = ring + (size_t)s * p.seg_bytes;
      const bool first = h.y & 1, last = h.y & 2;
#pragma unroll
      for (int v = 0; v < kMaxVecPerThread; ++v) {
        const int byte = (ct + v * 32 * kConsumerWarps) * 16;
        if (first) {
#pragma unroll
          for (int e = 0; e < kVec; ++e) acc[v][e] = 0.f;
        }
        if (byte < p.seg_bytes) add_vec<T>(acc[v], *reinterpret_cast<const uint4*>(seg + byte));
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&empty[s]);       // this warp has read the slot
      if (last) {
        const int cq = h.y >> 8;
        const float inv = (p.mean && h.z > 0) ? 1.0f / (float)(1 + h.z) : 1.f;
        T* dst = out + (size_t)h.x * p.D + (size_t)cq * seg_elems;
#pragma unroll
        for (int v = 0; v < kMaxVecPerThread; ++v) {
          const int byte = (ct + v * 32 * kConsumerWarps) * 16;
          if (byte < p.seg_bytes) {
#pragma unroll
            for (int e = 0; e < kVec; ++e) acc[v][e] *= inv;
            Storage<T>::store(dst + byte / (int)sizeof(T), acc[v]);
          }
        }
        if (ct == 0 && cq == 0) p.src_of_dst[h.x] = h.w;
      }
    }
  }
}

}  // namespace

// Returns D3TOM_ERR_UNSUPPORTED when the row size does not suit the pipeline (the caller then uses the plain kernel).
int launch_merge_aggregate_stream(d3tom_ctx* ctx, const MergeArgs& a, cudaStream_t s) {
  const int esize = a.dt == D3TOM_FP32 ? 4 : 2;
  const long long row_bytes = (long long)a.D * esize;
  if (row_bytes % 16 != 0) return D3TOM_ERR_UNSUPPORTED;
  // The pipeline pays off once every CTA streams many rows (measured: 68 against 87 us on 7.5 K output rows of
  // 8 KB, but 27 against 12 us on 1.2 K rows, where its start-up and the longest row of one CTA dominate).
  if (a.total_out < kStreamMinRows) return D3TOM_ERR_UNSUPPORTED;
  // column segments of at most 8 KB (128 consumer threads x 4 x 16 bytes); a power of two that divides the row into 16-byte multiples
  int splits = 1;
  while (row_bytes / splits > kMaxVecPerThread * 16 * 32 * kConsumerWarps && (row_bytes / (splits * 2)) % 16 == 0) splits *= 2;
  const long long seg = row_bytes / splits;
  if (seg > kMaxVecPerThread * 16 * 32 * kConsumerWarps || seg % 16 != 0) return D3TOM_ERR_UNSUPPORTED;
  int slots = (int)(kRingBytes / seg);
  if (slots > kMaxSlots) slots = kMaxSlots;
  if (slots < 4) return D3TOM_ERR_UNSUPPORTED;
  StreamParams p;
  p.hidden = a.hidden; p.hidden_out = a.hidden_out; p.row_desc = ctx->row_desc; p.member_list = ctx->member_list;
  p.src_of_dst = a.src_of_dst; p.work_counter = ctx->agg_counter; p.dev_status = ctx->dev_status;
  p.total_out = a.total_out; p.D = a.D; p.col_splits = splits; p.seg_bytes = (int)seg; p.slots = slots;
  p.mean = a.mode == D3TOM_AGG_MEAN ? 1 : 0;
  const size_t smem = (size_t)slots * seg + 128;
  const long long items = (long long)a.total_out * splits;
  long long grid = 6LL * ctx->sm_count;                 // six CTAs fit one SM (32 KB of ring each): what limits the
                                                        // pipeline is the rate at which one producer lane issues copies
  if (grid > items) grid = items;
  if (a.dt == D3TOM_FP32) {
    D3TOM_CUDA_TRY(ctx, cudaFuncSetAttribute(aggregate_stream_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, kRingBytes + 128));
    D3TOM_CUDA_TRY(ctx, launch_serialized(aggregate_stream_kernel<float>, (int)grid, kStreamThreads, smem, s, p));
  } else {
    D3TOM_CUDA_TRY(ctx, cudaFuncSetAttribute(aggregate_stream_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, kRingBytes + 128));
    D3TOM_CUDA_TRY(ctx, launch_serialized(aggregate_stream_kernel<__nv_bfloat16>, (int)grid, kStreamThreads, smem, s, p));
  }
  return D3TOM_OK;
}
