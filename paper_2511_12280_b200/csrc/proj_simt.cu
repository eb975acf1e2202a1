// Q,K,V projection and the other dense layers of a block on CUDA cores (Sec. 3.2.1,
// Q = H W_Q, K = H W_K; Algorithm 1, FFN_l): the fp32 storage path and a debugging aid for bf16.  C[n, 3D] = X[n, D] * W[3D, D]^T,
// fp32 accumulation, 32x32 output tile per block staged through shared memory.
#include "common.cuh"

namespace {

template <typename T>
__global__ void __launch_bounds__(1024)
proj_simt_kernel(const T* __restrict__ x, const T* __restrict__ w, int n, int D,
                 T* __restrict__ q, T* __restrict__ k, T* __restrict__ v) {
  __shared__ float xs[32][33];
  __shared__ float ws[32][33];
  grid_dependency_enter();
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int row = blockIdx.y * 32 + ty;       // token
  const int col = blockIdx.x * 32 + tx;       // output feature in [0, 3D)
  float acc = 0.f;
  for (int c0 = 0; c0 < D; c0 += 32) {
    const int xr = blockIdx.y * 32 + ty, wr = blockIdx.x * 32 + ty;
    xs[ty][tx] = (xr < n && c0 + tx < D) ? Storage<T>::to_float(x[(size_t)xr * D + c0 + tx]) : 0.f;
    ws[ty][tx] = (wr < 3 * D && c0 + tx < D) ? Storage<T>::to_float(w[(size_t)wr * D + c0 + tx]) : 0.f;
    __syncthreads();
#pragma unroll
    for (int c = 0; c < 32; ++c) acc = fmaf(xs[ty][c], ws[tx][c], acc);
    __syncthreads();
  }
  if (row < n && col < 3 * D) {
    T* dst = col < D ? q : (col < 2 * D ? k : v);
    dst[(size_t)row * D + (col % D)] = Storage<T>::from_float(acc);
  }
}

// y[n, N] = residual + x[n, K] w[N, K]^T (kGateUp == false), or the first half of the gated feed-forward network,
// act[n, m] = silu(x Wg^T) * (x Wu^T) with w = [Wg; Wu] of 2m rows (kGateUp == true, N = m): Algorithm 1, FFN_l.
template <typename T, bool kGateUp>
__global__ void __launch_bounds__(1024)
linear_simt_kernel(const T* __restrict__ x, const T* __restrict__ w, const T* residual, int n, int K, int N, T* out) {
  __shared__ float xs[32][33];
  __shared__ float ws[32][33];
  __shared__ float us[kGateUp ? 32 : 1][33];
  grid_dependency_enter();
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int row = blockIdx.y * 32 + ty;
  const int col = blockIdx.x * 32 + tx;
  float acc = 0.f, acc_u = 0.f;
  for (int c0 = 0; c0 < K; c0 += 32) {
    const int wr = blockIdx.x * 32 + ty;
    const bool in_k = c0 + tx < K;
    xs[ty][tx] = (row < n && in_k) ? Storage<T>::to_float(x[(size_t)row * K + c0 + tx]) : 0.f;
    ws[ty][tx] = (wr < N && in_k) ? Storage<T>::to_float(w[(size_t)wr * K + c0 + tx]) : 0.f;
    if (kGateUp) us[ty][tx] = (wr < N && in_k) ? Storage<T>::to_float(w[(size_t)(N + wr) * K + c0 + tx]) : 0.f;
    __syncthreads();
#pragma unroll
    for (int c = 0; c < 32; ++c) {
      acc = fmaf(xs[ty][c], ws[tx][c], acc);
      if (kGateUp) acc_u = fmaf(xs[ty][c], us[tx][c], acc_u);
    }
    __syncthreads();
  }
  if (row < n && col < N) {
    const size_t o = (size_t)row * N + col;
    if (kGateUp) out[o] = Storage<T>::from_float(acc / (1.f + expf(-acc)) * acc_u);
    else out[o] = Storage<T>::from_float(residual != nullptr ? acc + Storage<T>::to_float(residual[o]) : acc);
  }
}

template <typename T, bool kGateUp>
int launch_linear_simt_t(d3tom_ctx* ctx, const void* x, const void* w, const void* residual, int rows, int K, int N,
                         void* out, cudaStream_t s) {
  dim3 grid(ceil_div(N, 32), ceil_div(rows, 32));
  D3TOM_CUDA_TRY(ctx, launch_serialized(linear_simt_kernel<T, kGateUp>, grid, 1024, 0, s, static_cast<const T*>(x),
                                        static_cast<const T*>(w), static_cast<const T*>(residual), rows, K, N,
                                        static_cast<T*>(out)));
  return D3TOM_OK;
}

}  // namespace

int launch_linear_simt(d3tom_ctx* ctx, d3tom_dtype dt, const void* x, const void* w, const void* residual, int rows,
                       int K, int N, void* out, cudaStream_t s) {
  if (dt == D3TOM_FP32) return launch_linear_simt_t<float, false>(ctx, x, w, residual, rows, K, N, out, s);
  return launch_linear_simt_t<__nv_bfloat16, false>(ctx, x, w, residual, rows, K, N, out, s);
}

int launch_gate_up_simt(d3tom_ctx* ctx, d3tom_dtype dt, const void* x, const void* w_gate_up, int rows, int D, int m,
                        void* act, cudaStream_t s) {
  if (dt == D3TOM_FP32) return launch_linear_simt_t<float, true>(ctx, x, w_gate_up, nullptr, rows, D, m, act, s);
  return launch_linear_simt_t<__nv_bfloat16, true>(ctx, x, w_gate_up, nullptr, rows, D, m, act, s);
}

int launch_proj_simt(d3tom_ctx* ctx, d3tom_dtype dt, const void* x, const void* w, int total, int D,
                     void* q, void* k, void* v, cudaStream_t s) {
  dim3 grid(ceil_div(3 * D, 32), ceil_div(total, 32));
  if (dt == D3TOM_FP32)
    D3TOM_CUDA_TRY(ctx, launch_serialized(proj_simt_kernel<float>, grid, 1024, 0, s, static_cast<const float*>(x),
                                          static_cast<const float*>(w), total, D, static_cast<float*>(q),
                                          static_cast<float*>(k), static_cast<float*>(v)));
  else
    D3TOM_CUDA_TRY(ctx, launch_serialized(proj_simt_kernel<__nv_bfloat16>, grid, 1024, 0, s,
                                          static_cast<const __nv_bfloat16*>(x), static_cast<const __nv_bfloat16*>(w),
                                          total, D, static_cast<__nv_bfloat16*>(q), static_cast<__nv_bfloat16*>(k),
                                          static_cast<__nv_bfloat16*>(v)));
  return D3TOM_OK;
}
