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
#pragma unroll
    for (int t = 0; t < 8; ++t) a[t] *= gelu_grad_f(b[t], act);
    *reinterpret_cast<uint4 *>(g + m * ld_g + j) = pack_bf16x8(a);
  }
}

// partial[chunk, c] = sum over the chunk's rows of g[row, c0 + c]; 64 columns per block.
// Row order inside a chunk: lane ty sums rows ty, ty+8, ...; then lanes 0..7 are added in order.
__global__ void __launch_bounds__(256) colsum_partial_kernel(const __nv_bfloat16 *__restrict__ g, long long ld,
                                                             long long M, int c0, int ncols,
                                                             float *__restrict__ partial, int ld_partial) {
  __shared__ float2 red[8][32];
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int col = blockIdx.x * 64 + tx * 2;
  const long long r0 = (long long)blockIdx.y * COLSUM_ROWS_PER_CHUNK;
  const long long r1 = min(M, r0 + COLSUM_ROWS_PER_CHUNK);
  float2 acc = make_float2(0.f, 0.f);
  if (col < ncols) {
    const __nv_bfloat16 *src = g + c0 + col;
#pragma unroll 8
    for (long long r = r0 + ty; r < r1; r += 8) {
      const __nv_bfloat162 v = *reinterpret_cast<const __nv_bfloat162 *>(src + r * ld);
      const float2 f = __bfloat1622float2(v);
      acc.x += f.x;
      acc.y += f.y;
    }
  }
  red[ty][tx] = acc;
  __syncthreads();
  if (ty == 0 && col < ncols) {
    float2 s = red[0][tx];
#pragma unroll
    for (int t = 1; t < 8; ++t) {
      s.x += red[t][tx].x;
      s.y += red[t][tx].y;
    }
    partial[(long long)blockIdx.y * ld_partial + col] = s.x;
    partial[(long long)blockIdx.y * ld_partial + col + 1] = s.y;
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
