// One-time weight preparation and the residual-checkpoint append (STORE_RESIDUAL of Algorithm 1).
#include <cuda_fp8.h>

#include "kvd_internal.h"
#include "kvd_ptx.cuh"

namespace kvd {

// an element (bf16, fp16 or fp32 bits) as float, and back (round to nearest even)
template <int DT>
struct ElemBits {
  typedef uint16_t type;
};
template <>
struct ElemBits<2> {
  typedef uint32_t type;
};
template <int DT>
__device__ __forceinline__ float elem_to_float(typename ElemBits<DT>::type bits) {
  if constexpr (DT == 0) return __uint_as_float(static_cast<uint32_t>(bits) << 16);
  else if constexpr (DT == 1) return __half2float(__ushort_as_half(bits));
  else return __uint_as_float(bits);
}
template <int DT>
__device__ __forceinline__ typename ElemBits<DT>::type float_to_elem(float v) {
  if constexpr (DT == 0) return __bfloat16_as_ushort(__float2bfloat16_rn(v));
  else if constexpr (DT == 1) return __half_as_ushort(__float2half_rn(v));
  else return __float_as_uint(v);
}

// wt[n][k] = bf16( gamma[k] * w[k][n] ): fold the RMSNorm scale of Eq. 1 into the projection of
// Eq. 13-14 and store the result K-major so that both GEMM operands are read along d_hidden.
template <int DT>
__global__ void __launch_bounds__(256) kvd_prepare_weights_kernel(const typename ElemBits<DT>::type *__restrict__ w,
                                                                  const typename ElemBits<DT>::type *__restrict__ gamma,
                                                                  typename ElemBits<DT>::type *__restrict__ wt,
                                                                  int d_hidden, int n_cols) {
  __shared__ float tile[32][33];
  const int k0 = blockIdx.y * 32, n0 = blockIdx.x * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;  // 32 x 8
  for (int r = ty; r < 32; r += 8) {
    const int k = k0 + r, n = n0 + tx;
    float v = 0.f;
    if (k < d_hidden && n < n_cols)
      v = elem_to_float<DT>(gamma[k]) * elem_to_float<DT>(w[static_cast<size_t>(k) * n_cols + n]);
    tile[r][tx] = v;
  }
  __syncthreads();
  for (int r = ty; r < 32; r += 8) {
    const int n = n0 + r, k = k0 + tx;
    if (k < d_hidden && n < n_cols) wt[static_cast<size_t>(n) * d_hidden + k] = float_to_elem<DT>(tile[tx][r]);
  }
}

template <int DT>
__global__ void kvd_convert_gamma_kernel(const typename ElemBits<DT>::type *__restrict__ g, float *__restrict__ out, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = elem_to_float<DT>(g[i]);
}

// Copy n rows of d_hidden bf16 and their positions into the store, one warp per row; the warp also
// takes the row's sum of squares (the RMSNorm statistic of Eq. 2), which the recompute kernel reads
// back instead of taking it again for every recomputation.
template <int DT>
__global__ void __launch_bounds__(256) kvd_checkpoint_kernel(const uint4 *__restrict__ rows,
                                                             const int32_t *__restrict__ pos,
                                                             uint4 *__restrict__ dst_rows, int32_t *__restrict__ dst_pos,
                                                             float *__restrict__ dst_sumsq, int row_chunks, int n,
                                                             int capacity, int *status) {
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  grid_launch_dependents();  // the next kernel's set-up may overlap this copy
  for (int r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; r < n; r += warps) {
    if (!KVD_BOUNDS_OK(r < capacity, status)) continue;  // checking build: the row fits the sequence's slab
    const size_t off = static_cast<size_t>(r) * row_chunks;
    const uint4 *const src[1] = {rows + off};
    uint4 *const dst[1] = {dst_rows + off};
    float ss[1];
    warp_rows_sumsq<1, 10, true, DT>(src, dst, row_chunks, lane, ss);  // all of a 2560-wide row in flight at once
    if (lane == 0) {
      dst_sumsq[r] = ss[0];
      dst_pos[r] = pos[r];
    }
  }
}

// The same for one new row per sequence of a decode batch: row r goes to slot P.slot[r] of the store
// (rows, positions and statistics are indexed by slot), so that a whole batch is appended in one launch.
template <int DT>
__global__ void __launch_bounds__(256) kvd_checkpoint_scatter_kernel(const uint4 *__restrict__ rows,
                                                                     const int32_t *__restrict__ pos,
                                                                     uint4 *__restrict__ store_rows,
                                                                     int32_t *__restrict__ store_pos,
                                                                     float *__restrict__ store_sumsq, int row_chunks, int n,
                                                                     long long total_slots, int *status,
                                                                     const __grid_constant__ CkptSlots P) {
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  grid_launch_dependents();
  for (int r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; r < n; r += warps) {
    if (!KVD_BOUNDS_OK(P.slot[r] >= 0 && P.slot[r] < total_slots, status)) continue;  // checking build
    const size_t slot = static_cast<size_t>(P.slot[r]);
    const uint4 *const src[1] = {rows + static_cast<size_t>(r) * row_chunks};
    uint4 *const dst[1] = {store_rows + slot * row_chunks};
    float ss[1];
    warp_rows_sumsq<1, 10, true, DT>(src, dst, row_chunks, lane, ss);
    if (lane == 0) {
      store_sumsq[slot] = ss[0];
      store_pos[slot] = pos[r];
    }
  }
}

// Sums of squares of n caller rows (no copy), two rows per warp and pass: what kvd_recompute_kv takes
// ahead of the main kernel when the caller hands it more rows than that kernel's statistics warps
// can cover under the main loop.
template <int DT>
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
    warp_rows_sumsq<2, 8, false, DT>(src, none, row_chunks, lane, ss);
    if (lane == 0) {
      sumsq[r] = ss[0];
      sumsq[r1] = ss[1];
    }
  }
}

// ------------------------------------------------------------------------------ FP8 checkpoints
// The lower-precision variant (the paper's Section 6 names it as future work and fixes no format; the
// definition is in kvd.h): a row is stored as E4M3 codes with one fp32 scale, s = max|x| / 448,
// code = e4m3(x * (448 / max|x|)) rounded to nearest even and saturating, everything in IEEE fp32.  The row's
// sum of squares is taken from the ORIGINAL row with the shared function, so 1/rms is not affected.
__device__ __forceinline__ uint32_t e4m3x4(float a, float b, float c, float d) {
  const uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2(a, b), __NV_SATFINITE, __NV_E4M3);
  const uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2(c, d), __NV_SATFINITE, __NV_E4M3);
  return lo | (hi << 16);
}
// CPL > 0: rows of at most 32 * CPL chunks are held in registers (one pass over memory); CPL = 0: any
// width, the row is read three times (it sits in L1 / L2 after the first).  The arithmetic is the same.
template <int CPL>
__global__ void __launch_bounds__(256) kvd_checkpoint_fp8_kernel(const uint4 *__restrict__ rows,
                                                                 const int32_t *__restrict__ pos,
                                                                 uint2 *__restrict__ dst_codes,
                                                                 int32_t *__restrict__ dst_pos,
                                                                 float *__restrict__ dst_sumsq,
                                                                 float *__restrict__ dst_scale, int row_chunks, int n) {
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  grid_launch_dependents();
  auto chunk_amax = [](const uint4 &v, float amax) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) amax = fmaxf(amax, fmaxf(fabsf(bf16_lo(w[j])), fabsf(bf16_hi(w[j]))));
    return amax;
  };
  auto chunk_codes = [](const uint4 &v, float recip) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    float q[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      q[2 * j] = __fmul_rn(bf16_lo(w[j]), recip);
      q[2 * j + 1] = __fmul_rn(bf16_hi(w[j]), recip);
    }
    return make_uint2(e4m3x4(q[0], q[1], q[2], q[3]), e4m3x4(q[4], q[5], q[6], q[7]));
  };
  for (int r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; r < n; r += warps) {
    const size_t off = static_cast<size_t>(r) * row_chunks;
    float ss, amax = 0.f;
    if constexpr (CPL > 0) {
      uint4 v[CPL];
#pragma unroll
      for (int i = 0; i < CPL; ++i) {
        const int c = lane + 32 * i;
        v[i] = c < row_chunks ? __ldg(rows + off + c) : make_uint4(0u, 0u, 0u, 0u);
      }
      // the lane's chunks in ascending order, as warp_rows_sumsq takes them (absent chunks add exact zeros)
      uint64_t ps2[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
      for (int i = 0; i < CPL; ++i) {
        sumsq_chunk(ps2, v[i]);
        amax = chunk_amax(v[i], amax);
      }
      ss = sumsq_finish(ps2);
#pragma unroll
      for (int k = 16; k >= 1; k >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, k));
      amax = fmaxf(amax, 1e-30f);
      const float scale = __fdiv_rn(amax, 448.0f), recip = __fdiv_rn(448.0f, amax);
#pragma unroll
      for (int i = 0; i < CPL; ++i) {
        const int c = lane + 32 * i;
        if (c < row_chunks) dst_codes[off + c] = chunk_codes(v[i], recip);
      }
      if (lane == 0) dst_scale[r] = scale;
    } else {
      const uint4 *const src[1] = {rows + off};
      uint4 *const none[1] = {nullptr};
      float s1[1];
      warp_rows_sumsq<1, 10, false>(src, none, row_chunks, lane, s1);
      ss = s1[0];
      for (int c = lane; c < row_chunks; c += 32) amax = chunk_amax(__ldg(rows + off + c), amax);
#pragma unroll
      for (int k = 16; k >= 1; k >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, k));
      amax = fmaxf(amax, 1e-30f);
      const float scale = __fdiv_rn(amax, 448.0f), recip = __fdiv_rn(448.0f, amax);
      for (int c = lane; c < row_chunks; c += 32) dst_codes[off + c] = chunk_codes(__ldg(rows + off + c), recip);
      if (lane == 0) dst_scale[r] = scale;
    }
    if (lane == 0) {
      dst_sumsq[r] = ss;
      if (dst_pos != nullptr) dst_pos[r] = pos[r];  // (no positions when the rows are only quantised, not stored)
    }
  }
}

// W' = gamma (.) W in fp32 (exact for bf16 inputs): its largest magnitude, then the E4M3 codes of
// W' / s_w, s_w = max|W'| / 448, stored K-major like the bf16 copy.
__global__ void __launch_bounds__(256) kvd_weights_amax_kernel(const __nv_bfloat16 *__restrict__ w,
                                                               const __nv_bfloat16 *__restrict__ gamma, int d_hidden,
                                                               int n_cols, unsigned *__restrict__ amax_bits) {
  float m = 0.f;
  const size_t total = static_cast<size_t>(d_hidden) * n_cols;
  for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
       i += static_cast<size_t>(gridDim.x) * blockDim.x) {
    const int k = static_cast<int>(i / n_cols);
    m = fmaxf(m, fabsf(__bfloat162float(gamma[k]) * __bfloat162float(w[i])));
  }
#pragma unroll
  for (int k = 16; k >= 1; k >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, k));
  if ((threadIdx.x & 31) == 0) atomicMax(amax_bits, __float_as_uint(m));  // non-negative floats order like their bits
}
__global__ void __launch_bounds__(256) kvd_prepare_weights_fp8_kernel(const __nv_bfloat16 *__restrict__ w,
                                                                      const __nv_bfloat16 *__restrict__ gamma,
                                                                      uint8_t *__restrict__ wt8, int d_hidden, int n_cols,
                                                                      const unsigned *__restrict__ amax_bits,
                                                                      float *__restrict__ scale_out) {
  __shared__ float tile[32][33];
  const float amax = fmaxf(__uint_as_float(*amax_bits), 1e-30f);
  const float scale = __fdiv_rn(amax, 448.0f), recip = __fdiv_rn(448.0f, amax);
  if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) *scale_out = scale;
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
    if (k < d_hidden && n < n_cols) {
      const uint32_t c = __nv_cvt_float2_to_fp8x2(make_float2(__fmul_rn(tile[tx][r], recip), 0.f), __NV_SATFINITE, __NV_E4M3);
      wt8[static_cast<size_t>(n) * d_hidden + k] = static_cast<uint8_t>(c & 0xffu);
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

// Checking build: one index test that fails by construction (index 1 of a table of one entry); the access it
// guards is skipped, so nothing is read or written out of range.
__global__ void kvd_selftest_bounds_kernel(int *status, int *table) {
  const int idx = 1, entries = 1;
  if (KVD_BOUNDS_OK(idx < entries, status)) table[idx] = 0;
}
kvd_status launch_selftest_bounds(kvd_ctx *ctx, cudaStream_t stream) {
#ifdef KVD_CHECK
  kvd_selftest_bounds_kernel<<<1, 1, 0, stream>>>(ctx->d_status, ctx->d_status);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "launch selftest_bounds");
  ctx->launches += 1;
  return KVD_OK;
#else
  (void)ctx;
  (void)stream;
  return KVD_ERR_UNSUPPORTED;
#endif
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
  const uint16_t *w16 = reinterpret_cast<const uint16_t *>(w), *g16 = reinterpret_cast<const uint16_t *>(gamma);
  uint16_t *wt16 = reinterpret_cast<uint16_t *>(wt);
  if (ctx->dtype == 2)
    kvd_prepare_weights_kernel<2><<<grid, 256, 0, stream>>>(reinterpret_cast<const uint32_t *>(w), reinterpret_cast<const uint32_t *>(gamma),
                                                            reinterpret_cast<uint32_t *>(wt), d_hidden, n_cols);
  else if (ctx->dtype == 1) kvd_prepare_weights_kernel<1><<<grid, 256, 0, stream>>>(w16, g16, wt16, d_hidden, n_cols);
  else kvd_prepare_weights_kernel<0><<<grid, 256, 0, stream>>>(w16, g16, wt16, d_hidden, n_cols);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "launch prepare_weights");
  ctx->launches += 1;
  return KVD_OK;
}

kvd_status launch_convert_gamma(kvd_ctx *ctx, const __nv_bfloat16 *g, float *out, int n, cudaStream_t stream) {
  const uint16_t *g16 = reinterpret_cast<const uint16_t *>(g);
  if (ctx->dtype == 2) kvd_convert_gamma_kernel<2><<<(n + 127) / 128, 128, 0, stream>>>(reinterpret_cast<const uint32_t *>(g), out, n);
  else if (ctx->dtype == 1) kvd_convert_gamma_kernel<1><<<(n + 127) / 128, 128, 0, stream>>>(g16, out, n);
  else kvd_convert_gamma_kernel<0><<<(n + 127) / 128, 128, 0, stream>>>(g16, out, n);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "launch convert_gamma");
  ctx->launches += 1;
  return KVD_OK;
}

kvd_status launch_checkpoint(kvd_ctx *ctx, const __nv_bfloat16 *rows, const int32_t *pos, __nv_bfloat16 *dst_rows,
                             int32_t *dst_pos, float *dst_sumsq, int n, int d_hidden, cudaStream_t stream) {
  // rows left in the (layer, sequence) slab from dst on: what the checking build tests row indices against
  const long long slot = dst_pos - ctx->store_pos;
  const int capacity = ctx->desc.max_tokens_per_seq - static_cast<int>(slot % ctx->desc.max_tokens_per_seq);
  long long blocks = (static_cast<long long>(n) + 7) / 8;  // eight warps, one row each per pass
  const long long cap = static_cast<long long>(ctx->num_sms) * 8;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  if (ctx->dtype == 2)
    kvd_checkpoint_kernel<2><<<static_cast<unsigned>(blocks), 256, 0, stream>>>(
        reinterpret_cast<const uint4 *>(rows), pos, reinterpret_cast<uint4 *>(dst_rows), dst_pos, dst_sumsq, d_hidden / 4, n, capacity, ctx->d_status);
  else if (ctx->dtype == 1)
    kvd_checkpoint_kernel<1><<<static_cast<unsigned>(blocks), 256, 0, stream>>>(
        reinterpret_cast<const uint4 *>(rows), pos, reinterpret_cast<uint4 *>(dst_rows), dst_pos, dst_sumsq, d_hidden / 8, n, capacity, ctx->d_status);
  else
    kvd_checkpoint_kernel<0><<<static_cast<unsigned>(blocks), 256, 0, stream>>>(
        reinterpret_cast<const uint4 *>(rows), pos, reinterpret_cast<uint4 *>(dst_rows), dst_pos, dst_sumsq, d_hidden / 8, n, capacity, ctx->d_status);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "launch checkpoint");
  ctx->launches += 1;
  return KVD_OK;
}

kvd_status launch_checkpoint_scatter(kvd_ctx *ctx, const __nv_bfloat16 *rows, const int32_t *pos, const CkptSlots &slots,
                                     int n, int d_hidden, cudaStream_t stream) {
  const unsigned blocks = static_cast<unsigned>((n + 7) / 8);  // eight warps, one row each
  const uint4 *src = reinterpret_cast<const uint4 *>(rows);
  uint4 *dst = reinterpret_cast<uint4 *>(ctx->store_rows);
  const long long total = static_cast<long long>(ctx->layers_stored) * ctx->desc.max_seqs * ctx->desc.max_tokens_per_seq;
  if (ctx->dtype == 2)
    kvd_checkpoint_scatter_kernel<2><<<blocks, 256, 0, stream>>>(src, pos, dst, ctx->store_pos, ctx->store_sumsq, d_hidden / 4, n, total, ctx->d_status, slots);
  else if (ctx->dtype == 1)
    kvd_checkpoint_scatter_kernel<1><<<blocks, 256, 0, stream>>>(src, pos, dst, ctx->store_pos, ctx->store_sumsq, d_hidden / 8, n, total, ctx->d_status, slots);
  else
    kvd_checkpoint_scatter_kernel<0><<<blocks, 256, 0, stream>>>(src, pos, dst, ctx->store_pos, ctx->store_sumsq, d_hidden / 8, n, total, ctx->d_status, slots);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "launch checkpoint (batch)");
  ctx->launches += 1;
  return KVD_OK;
}

kvd_status launch_rowstats(kvd_ctx *ctx, const __nv_bfloat16 *rows, float *sumsq, int n, int d_hidden,
                           cudaStream_t stream) {
  long long blocks = (static_cast<long long>(n) + 15) / 16;  // eight warps, two rows each per pass
  const long long cap = static_cast<long long>(ctx->num_sms) * 8;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  if (ctx->dtype == 2)
    kvd_rowstats_kernel<2><<<static_cast<unsigned>(blocks), 256, 0, stream>>>(reinterpret_cast<const uint4 *>(rows), sumsq,
                                                                              d_hidden / 4, n);
  else if (ctx->dtype == 1)
    kvd_rowstats_kernel<1><<<static_cast<unsigned>(blocks), 256, 0, stream>>>(reinterpret_cast<const uint4 *>(rows), sumsq,
                                                                              d_hidden / 8, n);
  else
    kvd_rowstats_kernel<0><<<static_cast<unsigned>(blocks), 256, 0, stream>>>(reinterpret_cast<const uint4 *>(rows), sumsq,
                                                                              d_hidden / 8, n);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "launch rowstats");
  ctx->launches += 1;
  return KVD_OK;
}

kvd_status launch_checkpoint_fp8(kvd_ctx *ctx, const __nv_bfloat16 *rows, const int32_t *pos, uint8_t *dst_codes,
                                 int32_t *dst_pos, float *dst_sumsq, float *dst_scale, int n, int d_hidden,
                                 cudaStream_t stream) {
  long long blocks = (static_cast<long long>(n) + 7) / 8;
  const long long cap = static_cast<long long>(ctx->num_sms) * 8;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  const int row_chunks = d_hidden / 8;
  if (row_chunks <= 320)
    kvd_checkpoint_fp8_kernel<10><<<static_cast<unsigned>(blocks), 256, 0, stream>>>(
        reinterpret_cast<const uint4 *>(rows), pos, reinterpret_cast<uint2 *>(dst_codes), dst_pos, dst_sumsq, dst_scale,
        row_chunks, n);
  else
    kvd_checkpoint_fp8_kernel<0><<<static_cast<unsigned>(blocks), 256, 0, stream>>>(
        reinterpret_cast<const uint4 *>(rows), pos, reinterpret_cast<uint2 *>(dst_codes), dst_pos, dst_sumsq, dst_scale,
        row_chunks, n);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "launch checkpoint_fp8");
  ctx->launches += 1;
  return KVD_OK;
}

// amax_scratch: one zeroed unsigned on the device; scale_out: one float on the device
kvd_status launch_prepare_weights_fp8(kvd_ctx *ctx, const __nv_bfloat16 *w, const __nv_bfloat16 *gamma, uint8_t *wt8,
                                      int d_hidden, int n_cols, unsigned *amax_scratch, float *scale_out,
                                      cudaStream_t stream) {
  cudaError_t e = cudaMemsetAsync(amax_scratch, 0, sizeof(unsigned), stream);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "memset amax");
  kvd_weights_amax_kernel<<<ctx->num_sms * 4, 256, 0, stream>>>(w, gamma, d_hidden, n_cols, amax_scratch);
  dim3 grid((n_cols + 31) / 32, (d_hidden + 31) / 32);
  kvd_prepare_weights_fp8_kernel<<<grid, 256, 0, stream>>>(w, gamma, wt8, d_hidden, n_cols, amax_scratch, scale_out);
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "launch prepare_weights_fp8");
  ctx->launches += 2;
  return KVD_OK;
}

}  // namespace kvd
