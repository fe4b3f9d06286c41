// HBM-bound helpers around the GEMMs: the activation backward G = dY (.) act'(Z) for one slice
// of columns, and deterministic column sums (db).  Plain coalesced 16-byte accesses; these are
// not contractions, so no tensor cores.
#pragma once

#include "osdp_gemm.cuh"

namespace osdp {

constexpr int COLSUM_ROWS_PER_CHUNK = 1024;   // fixed, so that a column's summation order never depends on k

// g[m, j] = dy[m, c0 + j] * act'(z[m, c0 + j]),  j in [0, ncols), ncols % 8 == 0.
__global__ void __launch_bounds__(256) act_backward_kernel(const __nv_bfloat16 *__restrict__ dy, long long ld_dy,
                                                           const __nv_bfloat16 *__restrict__ z, long long ld_z,
                                                           __nv_bfloat16 *__restrict__ g, long long ld_g,
                                                           long long M, int c0, int ncols, int act) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");   // inputs may come from the previous kernel on the stream
  const int vec_per_row = ncols >> 3;
  const long long total = M * vec_per_row;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const long long m = i / vec_per_row;
    const int j = (int)(i - m * vec_per_row) << 3;
    float a[8], b[8];
    unpack_bf16x8(*reinterpret_cast<const uint4 *>(dy + m * ld_dy + c0 + j), a);
    unpack_bf16x8(*reinterpret_cast<const uint4 *>(z + m * ld_z + c0 + j), b);
    float grad[8];
    gelu_grad_array(b, grad, act);
#pragma unroll
    for (int t = 0; t < 8; ++t) a[t] *= grad[t];
    *reinterpret_cast<uint4 *>(g + m * ld_g + j) = pack_bf16x8(a);
  }
}

// partial[chunk, c] = sum over the chunk's rows of g[row, c0 + c]; 64 columns per block (c0, ncols
// multiples of 8, g 16-byte aligned).  A thread owns 8 adjacent columns (one 16-byte load per row) and
// every 32nd row of the chunk; row order inside a chunk: row lane ty sums rows ty, ty+32, ...; then the
// 32 row lanes are added in ascending order.  The order never depends on how the operator is split.
__global__ void __launch_bounds__(256) colsum_partial_kernel(const __nv_bfloat16 *__restrict__ g, long long ld,
                                                             long long M, int c0, int ncols,
                                                             float *__restrict__ partial, int ld_partial) {
  __shared__ float red[32][64 + 1];
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int tx = threadIdx.x & 7, ty = threadIdx.x >> 3;
  const int col = blockIdx.x * 64 + tx * 8;
  const long long r0 = (long long)blockIdx.y * COLSUM_ROWS_PER_CHUNK;
  const long long r1 = min(M, r0 + COLSUM_ROWS_PER_CHUNK);
  float acc[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) acc[j] = 0.f;
  if (col < ncols) {
    const __nv_bfloat16 *src = g + c0 + col;
    // A thread's rows are fetched 16 at a time (16 independent 16-byte loads in flight: the block's time is
    // a few memory latencies instead of one per four rows) and added in ascending row order as before.
    constexpr int BATCH = 16;
    for (long long rb = r0 + ty; rb < r1; rb += 32 * BATCH) {
      uint4 v[BATCH];
#pragma unroll
      for (int b = 0; b < BATCH; ++b) {
        const long long r = rb + 32ll * b;
        v[b] = (r < r1) ? *reinterpret_cast<const uint4 *>(src + r * ld) : make_uint4(0u, 0u, 0u, 0u);
      }
#pragma unroll
      for (int b = 0; b < BATCH; ++b) {
        if (rb + 32ll * b < r1) {
          float f[8];
          unpack_bf16x8(v[b], f);
#pragma unroll
          for (int j = 0; j < 8; ++j) acc[j] += f[j];
        }
      }
    }
  }
#pragma unroll
  for (int j = 0; j < 8; ++j) red[ty][tx * 8 + j] = acc[j];
  __syncthreads();
  if (threadIdx.x < 64) {
    const int c = blockIdx.x * 64 + threadIdx.x;
    if (c < ncols) {
      float s = red[0][threadIdx.x];
#pragma unroll
      for (int t = 1; t < 32; ++t) s += red[t][threadIdx.x];
      partial[(long long)blockIdx.y * ld_partial + c] = s;
    }
  }
}

// out[c0 + c] = sum over chunks (ascending) of partial[chunk, c].
__global__ void __launch_bounds__(256) colsum_final_kernel(const float *__restrict__ partial, int ld_partial,
                                                           int nchunks, int ncols, float *__restrict__ out) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= ncols) return;
  float s = 0.f;
  for (int k = 0; k < nchunks; ++k) s += partial[(long long)k * ld_partial + c];
  out[c] = s;
}

}  // namespace osdp
