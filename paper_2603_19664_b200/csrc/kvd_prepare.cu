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

// Copy n rows of d_hidden bf16 and their positions into the store, one warp per row; the warp also
// takes the row's sum of squares (the RMSNorm statistic of Eq. 2), which the recompute kernel reads
// back instead of taking it again for every recomputation.
__global__ void __launch_bounds__(256) kvd_checkpoint_kernel(const uint4 *__restrict__ rows,
                                                             const int32_t *__restrict__ pos,
                                                             uint4 *__restrict__ dst_rows, int32_t *__restrict__ dst_pos,
                                                             float *__restrict__ dst_sumsq, int row_chunks, int n) {
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  grid_launch_dependents();  // the next kernel's set-up may overlap this copy
  for (int r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; r < n; r += warps) {
    const size_t off = static_cast<size_t>(r) * row_chunks;
    const uint4 *const src[1] = {rows + off};
    uint4 *const dst[1] = {dst_rows + off};
    float ss[1];
    warp_rows_sumsq<1, 10, true>(src, dst, row_chunks, lane, ss);  // all of a 2560-wide row in flight at once
    if (lane == 0) {
      dst_sumsq[r] = ss[0];
      dst_pos[r] = pos[r];
    }
  }
}

// Sums of squares of n caller rows (no copy), two rows per warp and pass: what kvd_recompute_kv takes
// ahead of the main kernel when the caller hands it more rows than that kernel's statistics warps
// can cover under the main loop.
__global__ void __launch_bounds__(256) kvd_rowstats_kernel(const uint4 *__restrict__ rows, float *__restrict__ sumsq,
                                                           int row_chunks, int n) {
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  grid_launch_dependents();
  for (int r = ((blockIdx.x * blockDim.x + threadIdx.x) >> 5) * 2; r < n; r += 2 * warps) {
    const int r1 = r + 1 < n ? r + 1 : r;
    const uint4 *const src[2] = {rows + static_cast<size_t>(r) * row_chunks, rows + static_cast<size_t>(r1) * row_chunks};
    uint4 *const none[2] = {nullptr, nullptr};
    float ss[2];
    warp_rows_sumsq<2, 8, false>(src, none, row_chunks, lane, ss);
    if (lane == 0) {
      sumsq[r] = ss[0];
      sumsq[r1] = ss[1];
    }
  }
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
                             int32_t *dst_pos, float *dst_sumsq, int n, int d_hidden, cudaStream_t stream) {
  long long blocks = (static_cast<long long>(n) + 7) / 8;  // eight warps, one row each per pass
  const long long cap = static_cast<long long>(ctx->num_sms) * 8;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  kvd_checkpoint_kernel<<<static_cast<unsigned>(blocks), 256, 0, stream>>>(
      reinterpret_cast<const uint4 *>(rows), pos, reinterpret_cast<uint4 *>(dst_rows), dst_pos, dst_sumsq, d_hidden / 8, n);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "launch checkpoint");
  ctx->launches += 1;
  return KVD_OK;
}

kvd_status launch_rowstats(kvd_ctx *ctx, const __nv_bfloat16 *rows, float *sumsq, int n, int d_hidden,
                           cudaStream_t stream) {
  long long blocks = (static_cast<long long>(n) + 15) / 16;  // eight warps, two rows each per pass
  const long long cap = static_cast<long long>(ctx->num_sms) * 8;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  kvd_rowstats_kernel<<<static_cast<unsigned>(blocks), 256, 0, stream>>>(reinterpret_cast<const uint4 *>(rows), sumsq,
                                                                         d_hidden / 8, n);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "launch rowstats");
  ctx->launches += 1;
  return KVD_OK;
}

}  // namespace kvd
