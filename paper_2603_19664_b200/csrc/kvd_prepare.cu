// One-time weight preparation and the residual-checkpoint append (STORE_RESIDUAL of Algorithm 1).
#include "kvd_internal.h"
#include "kvd_ptx.cuh"

namespace kvd {

// wt[n][k] = bf16( gamma[k] * w[k][n] ): fold the RMSNorm scale of Eq. 1 into the projection of
// Eq. 13-14 and store the result K-major so that both GEMM operands are read along d_hidden.
__global__ void __launch_bounds__(256) kvd_prepare_weights_kernel(const __nv_bfloat16 *__restrict__ w,
                                                                  const __nv_bfloat16 *__restrict__ gamma,
                                                                  __nv_bfloat16 *__restrict__ wt, int d_hidden,
                                                                  int n_cols) {
  __shared__ float tile[32][33];
  const int k0 = blockIdx.y * 32, n0 = blockIdx.x * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;  // 32 x 8
  for (int r = ty; r < 32; r += 8) {
    const int k = k0 + r, n = n0 + tx;
    float v = 0.f;
    if (k < d_hidden && n < n_cols)
      v = __bfloat162float(gamma[k]) * __bfloat162float(w[static_cast<size_t>(k) * n_cols + n]);
    tile[r][tx] = v;
  }
  __syncthreads();
  for (int r = ty; r < 32; r += 8) {
    const int n = n0 + r, k = k0 + tx;
    if (k < d_hidden && n < n_cols) wt[static_cast<size_t>(n) * d_hidden + k] = __float2bfloat16_rn(tile[tx][r]);
  }
}

__global__ void kvd_convert_gamma_kernel(const __nv_bfloat16 *__restrict__ g, float *__restrict__ out, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = __bfloat162float(g[i]);
}

// Copy n rows of d_hidden bf16 (16 bytes per thread-iteration) and their positions into the store.
__global__ void __launch_bounds__(256) kvd_checkpoint_kernel(const uint4 *__restrict__ rows,
                                                             const int32_t *__restrict__ pos,
                                                             uint4 *__restrict__ dst_rows, int32_t *__restrict__ dst_pos,
                                                             long long n_vec, int n) {
  const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
  const long long tid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  grid_launch_dependents();  // the next kernel's set-up may overlap this copy
  for (long long i = tid; i < n_vec; i += stride) dst_rows[i] = rows[i];
  for (long long i = tid; i < n; i += stride) dst_pos[i] = pos[i];
}

// Self-test of the bounded wait: one thread waits on an mbarrier that nothing ever arrives on.  The
// wait gives up after `timeout_ns`, records STATUS_TIMEOUT and the kernel returns normally.
__global__ void kvd_selftest_timeout_kernel(int *status, unsigned long long timeout_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    fence_mbar_init();
    if (!mbar_wait(smem_u32(&bar), 0, &abort_flag, timeout_ns)) atomicOr(status, STATUS_TIMEOUT);
  }
}

kvd_status launch_selftest_timeout(kvd_ctx *ctx, unsigned long long timeout_ns, cudaStream_t stream) {
  kvd_selftest_timeout_kernel<<<1, 32, 0, stream>>>(ctx->d_status, timeout_ns);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "launch selftest");
  ctx->launches += 1;
  return KVD_OK;
}

kvd_status launch_prepare_weights(kvd_ctx *ctx, const __nv_bfloat16 *w, const __nv_bfloat16 *gamma, __nv_bfloat16 *wt,
                                  int d_hidden, int n_cols, cudaStream_t stream) {
  dim3 grid((n_cols + 31) / 32, (d_hidden + 31) / 32);
  kvd_prepare_weights_kernel<<<grid, 256, 0, stream>>>(w, gamma, wt, d_hidden, n_cols);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "launch prepare_weights");
  ctx->launches += 1;
  return KVD_OK;
}

kvd_status launch_convert_gamma(kvd_ctx *ctx, const __nv_bfloat16 *g, float *out, int n, cudaStream_t stream) {
  kvd_convert_gamma_kernel<<<(n + 127) / 128, 128, 0, stream>>>(g, out, n);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "launch convert_gamma");
  ctx->launches += 1;
  return KVD_OK;
}

kvd_status launch_checkpoint(kvd_ctx *ctx, const __nv_bfloat16 *rows, const int32_t *pos, __nv_bfloat16 *dst_rows,
                             int32_t *dst_pos, int n, int d_hidden, cudaStream_t stream) {
  const long long n_vec = static_cast<long long>(n) * d_hidden / 8;
  long long blocks = (n_vec + 255) / 256;
  const long long cap = static_cast<long long>(ctx->num_sms) * 8;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  kvd_checkpoint_kernel<<<static_cast<unsigned>(blocks), 256, 0, stream>>>(
      reinterpret_cast<const uint4 *>(rows), pos, reinterpret_cast<uint4 *>(dst_rows), dst_pos, n_vec, n);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "launch checkpoint");
  ctx->launches += 1;
  return KVD_OK;
}

}  // namespace kvd
