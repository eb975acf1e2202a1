// Q,K,V projection on CUDA cores (Sec. 3.2.1, Q = H W_Q, K = H W_K): the fp32
// storage path and a debugging aid for bf16.  C[n, 3D] = X[n, D] * W[3D, D]^T,
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

}  // namespace

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
