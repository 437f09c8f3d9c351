// Plain SIMT GEMM, C = A W^T (A [M,K] bf16, W [n_out,K] bf16, fp32 accumulate) with the same epilogues as
// the tensor-core kernel.  Used only by the HSD_FLAG_SIMT_DEBUG cross-check path and by hsd_debug_logits.
#include "hsd_kernels.h"

namespace hsd {

constexpr int ST = 64;    // tile M = N
constexpr int SK = 32;    // tile K

template <int MODE>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const bf16* __restrict__ A, const bf16* __restrict__ W, int M,
                                                        int n_cols, int K, GemmOut out) {
  __shared__ float sA[SK][ST + 1];
  __shared__ float sB[SK][ST + 1];
  __shared__ float sB2[MODE == GM_SWIGLU ? SK : 1][ST + 1];
  __shared__ float sC[MODE == GM_ARGMAX ? ST : 1][ST + 1];
  const int tid = threadIdx.x;
  const int m0 = blockIdx.y * ST, n0 = blockIdx.x * ST;
  const int tx = tid % 16, ty = tid / 16;
  float acc[4][4] = {}, acc2[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += SK) {
    for (int e = tid; e < ST * SK; e += 256) {
      const int r = e / SK, c = e % SK;
      sA[c][r] = (m0 + r < M) ? __bfloat162float(A[(size_t)(m0 + r) * K + k0 + c]) : 0.f;
      sB[c][r] = (n0 + r < n_cols) ? __bfloat162float(W[(size_t)(n0 + r) * K + k0 + c]) : 0.f;
      if (MODE == GM_SWIGLU)
        sB2[c][r] = (n0 + r < n_cols) ? __bfloat162float(W[(size_t)(n_cols + n0 + r) * K + k0 + c]) : 0.f;
    }
    __syncthreads();
#pragma unroll 8
    for (int k = 0; k < SK; ++k) {
      float a[4], b[4], b2[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        a[i] = sA[k][ty * 4 + i];
        b[i] = sB[k][tx * 4 + i];
        if (MODE == GM_SWIGLU) b2[i] = sB2[k][tx * 4 + i];
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[i][j] += a[i] * b[j];
          if (MODE == GM_SWIGLU) acc2[i][j] += a[i] * b2[j];
        }
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = m0 + ty * 4 + i;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = n0 + tx * 4 + j;
      float v = acc[i][j];
      if (MODE == GM_ARGMAX) {
        sC[ty * 4 + i][tx * 4 + j] = v;
        continue;
      }
      if (r >= M || c >= n_cols) continue;
      if (MODE == GM_STORE_BF16) reinterpret_cast<bf16*>(out.C)[(size_t)r * out.ldc + c] = __float2bfloat16(v);
      if (MODE == GM_STORE_F32) reinterpret_cast<float*>(out.C)[(size_t)r * out.ldc + c] = v;
      if (MODE == GM_ADD_F32) reinterpret_cast<float*>(out.C)[(size_t)r * out.ldc + c] += v;
      if (MODE == GM_SWIGLU) {
        const float g = v, u = acc2[i][j];
        reinterpret_cast<bf16*>(out.C)[(size_t)r * out.ldc + c] = __float2bfloat16(g / (1.f + __expf(-g)) * u);
      }
    }
  }
  if (MODE == GM_ARGMAX) {
    __syncthreads();
    if (tid < ST && m0 + tid < M) {
      const int r = m0 + tid;
      const int nxt = out.row_next ? out.row_next[r] : -1;
      unsigned long long best = 0ull;
      for (int j = 0; j < ST && n0 + j < n_cols; ++j) {
        const float v = sC[tid][j];
        const unsigned long long key = argmax_key(v, n0 + j);
        best = key > best ? key : best;
        if (n0 + j == nxt) out.zdraft[r] = v;
      }
      atomicMax(out.row_best + r, best);
    }
  }
}

void launch_gemm_simt(cudaStream_t st, const bf16* A, const bf16* W, int M, int n_out, int K, int mode,
                      const GemmOut& out) {
  if (M <= 0) return;
  const int n_cols = (mode == GM_SWIGLU) ? n_out / 2 : n_out;
  dim3 grid((n_cols + ST - 1) / ST, (M + ST - 1) / ST), block(256);
  switch (mode) {
    case GM_STORE_BF16: gemm_simt_kernel<GM_STORE_BF16><<<grid, block, 0, st>>>(A, W, M, n_cols, K, out); break;
    case GM_ADD_F32: gemm_simt_kernel<GM_ADD_F32><<<grid, block, 0, st>>>(A, W, M, n_cols, K, out); break;
    case GM_SWIGLU: gemm_simt_kernel<GM_SWIGLU><<<grid, block, 0, st>>>(A, W, M, n_cols, K, out); break;
    case GM_STORE_F32: gemm_simt_kernel<GM_STORE_F32><<<grid, block, 0, st>>>(A, W, M, n_cols, K, out); break;
    case GM_ARGMAX: gemm_simt_kernel<GM_ARGMAX><<<grid, block, 0, st>>>(A, W, M, n_cols, K, out); break;
    default: break;
  }
}

}  // namespace hsd
