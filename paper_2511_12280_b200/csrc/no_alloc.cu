// d3tom_attn_importance_static: the merge-layer attention + importance map for
// callers that cannot allocate device memory.
//
// Some hosts of this library run where cudaMalloc is off limits: inside a
// memory pool that owns the whole device, under a sandbox that pre-registers
// every allocation, or in a serving loop that must not take the allocator's
// device-wide lock.  They cannot call d3tom_create (it allocates the scratch).
// This entry point runs the same kernels with the scratch placed in a fixed
// array that is part of the library image: every GPU that loads the library
// holds kStaticBytes of it until the process exits.
//
// The array's name is only a handle in host code, not a device address; the
// address is looked up once per device with cudaGetSymbolAddress while that
// device is current, and that pointer is what the kernels receive.
#include <mutex>

#include "common.cuh"

namespace {

// layout of the array (bytes): [status word + key-range counters | (M, l) pairs | per-head partials | raw decider scores]
constexpr size_t kCounterInts = 4096;     // batch * ceil(max_visual / 256) must stay below this
constexpr size_t kStatusBytes = 256 + kCounterInts * sizeof(int);
constexpr size_t kLseBytes = (size_t)D3TOM_STATIC_MAX_LSE_PAIRS * sizeof(float2);
constexpr size_t kPartialBytes = (size_t)D3TOM_STATIC_MAX_PARTIAL_FLOATS * sizeof(float);
constexpr size_t kScoreBytes = (size_t)D3TOM_STATIC_MAX_SCORE_FLOATS * sizeof(float);
constexpr size_t kStaticBytes = kStatusBytes + kLseBytes + kPartialBytes + kScoreBytes;
static_assert(kLseBytes % 256 == 0 && kPartialBytes % 256 == 0, "sections stay 256-byte aligned");

static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
unsigned char* g_base[kMaxDevices];      // device address of g_static_scratch on each device, once looked up
int g_major[kMaxDevices];
int g_sm_count[kMaxDevices];             // multiprocessors of each device (the attention launcher shapes its grid by it)

// Looks up (once per device) the device address of the array on the CURRENT device.
int static_scratch_base(int* device_out, unsigned char** base_out, int* sm_count_out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return D3TOM_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (g_base[dev] == nullptr) {
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return D3TOM_ERR_CUDA;
    g_major[dev] = major;
    if (major != 10) return D3TOM_ERR_UNSUPPORTED;
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) return D3TOM_ERR_CUDA;
    g_sm_count[dev] = sms;
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) {
      (void)cudaGetLastError();
      return D3TOM_ERR_CUDA;
    }
    g_base[dev] = static_cast<unsigned char*>(p);
  }
  if (g_major[dev] != 10) return D3TOM_ERR_UNSUPPORTED;
  *device_out = dev;
  *base_out = g_base[dev];
  *sm_count_out = g_sm_count[dev];
  return D3TOM_OK;
}

}  // namespace

extern "C" int d3tom_attn_importance_static(d3tom_dtype dt, int heads, int head_dim,
                                            const void* q, const void* k, const void* v,
                                            const int32_t* cu_seqlens, const int32_t* n_visual,
                                            const int32_t* decider_pos, const int32_t* cu_deciders,
                                            int B, int total_tokens, int max_seqlen, int max_visual,
                                            int n_deciders_total, float softmax_scale,
                                            void* attn_out, float* importance, const int32_t* cu_vis,
                                            int32_t* device_status_out, d3tom_stream stream) {
  if (dt != D3TOM_BF16 && dt != D3TOM_FP32) return D3TOM_ERR_UNSUPPORTED;
  if (q == nullptr || k == nullptr || v == nullptr || cu_seqlens == nullptr || attn_out == nullptr ||
      n_visual == nullptr || cu_deciders == nullptr || importance == nullptr || cu_vis == nullptr)
    return D3TOM_ERR_INVALID_ARG;
  if (heads <= 0 || head_dim <= 0 || B <= 0 || total_tokens < 0 || max_seqlen < 0 || max_seqlen > total_tokens ||
      n_deciders_total < 0 || max_visual < 0 || max_visual > max_seqlen || !(softmax_scale > 0.f))
    return D3TOM_ERR_INVALID_ARG;
  if (n_deciders_total > 0 && decider_pos == nullptr) return D3TOM_ERR_INVALID_ARG;
  if (dt == D3TOM_BF16 ? !(head_dim == 64 || head_dim == 128) : !(head_dim % 4 == 0 && head_dim <= 128))
    return D3TOM_ERR_UNSUPPORTED;
  // the fixed array bounds the problem size
  const size_t nd = (size_t)(n_deciders_total > 0 ? n_deciders_total : 1);
  const size_t vis_stride = ((size_t)max_visual + 3) & ~(size_t)3;
  if ((size_t)heads * nd > (size_t)D3TOM_STATIC_MAX_LSE_PAIRS ||
      (size_t)heads * (size_t)total_tokens > (size_t)D3TOM_STATIC_MAX_PARTIAL_FLOATS ||
      (size_t)heads * nd * vis_stride > (size_t)D3TOM_STATIC_MAX_SCORE_FLOATS ||
      (size_t)B * (((size_t)max_visual + 255) / 256) > kCounterInts)
    return D3TOM_ERR_WORKSPACE;
  if (total_tokens == 0 || max_seqlen == 0) return D3TOM_OK;

  int dev = -1, sms = 0;
  unsigned char* base = nullptr;
  int st = static_scratch_base(&dev, &base, &sms);
  if (st != D3TOM_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);

  // a context that lives on the host stack and only points into the array: nothing is allocated
  d3tom_ctx c = {};
  c.device = dev;
  c.sm_count = sms;
  c.lim.max_total_tokens = total_tokens; c.lim.max_batch = B; c.lim.heads = heads; c.lim.head_dim = head_dim;
  c.lim.max_deciders = (int)nd; c.lim.max_visual_per_request = max_visual;
  c.vis_stride = (int)vis_stride;
  c.dev_status = reinterpret_cast<int*>(base);
  c.imp_counters = reinterpret_cast<int*>(base + 256);
  c.lse_scratch = reinterpret_cast<float2*>(base + kStatusBytes);
  c.imp_partial = reinterpret_cast<float*>(base + kStatusBytes + kLseBytes);
  c.score_scratch = reinterpret_cast<float*>(base + kStatusBytes + kLseBytes + kPartialBytes);

  // the array keeps whatever the previous call left: the status word and the key-range counters must start at
  // zero (scores, (M, l) pairs and partials are fully rewritten before they are read)
  if (cudaMemsetAsync(base, 0, kStatusBytes, s) != cudaSuccess) return D3TOM_ERR_CUDA;

  AttnArgs a;
  a.q = q; a.k = k; a.v = v; a.out = attn_out;
  a.cu_seqlens = cu_seqlens; a.n_visual = n_visual;
  a.decider_pos = n_deciders_total > 0 ? decider_pos : nullptr;
  a.cu_deciders = cu_deciders;
  a.B = B; a.H = heads; a.dh = head_dim; a.total_tokens = total_tokens; a.max_seqlen = max_seqlen;
  a.scale_log2 = softmax_scale * 1.4426950408889634f;
  a.score_scratch = c.score_scratch; a.lse_scratch = c.lse_scratch;
  a.max_deciders = (int)nd; a.vis_stride = (int)vis_stride;
  a.dev_status = c.dev_status;
  st = dt == D3TOM_BF16 ? launch_attn_tc(&c, a, s) : launch_attn_simt(&c, dt, a, s);
  if (st != D3TOM_OK) return st;
  st = launch_importance_finish(&c, a, max_visual, importance, cu_vis, s);
  if (st != D3TOM_OK) return st;
  if (device_status_out != nullptr &&
      cudaMemcpyAsync(device_status_out, c.dev_status, sizeof(int), cudaMemcpyDeviceToDevice, s) != cudaSuccess)
    return D3TOM_ERR_CUDA;
  return D3TOM_OK;
}
