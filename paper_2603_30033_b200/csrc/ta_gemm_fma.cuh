// Plain fp32 FMA building blocks shared by the shape-generic path and the HOSVD initialiser: typed loads /
// stores and a strided, batched GEMM.
#pragma once

#include "ta_common.cuh"

namespace ta {
namespace fma {

template <typename T> __device__ __forceinline__ float ld(const T* p);
template <> __device__ __forceinline__ float ld<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ld<bf16>(const bf16* p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ void st(T* p, float v);
template <> __device__ __forceinline__ void st<float>(float* p, float v) { *p = v; }
template <> __device__ __forceinline__ void st<bf16>(bf16* p, float v) { *p = __float2bfloat16_rn(v); }

// ---------------------------------------------------------------------------------------
// Generic strided, batched GEMM: C[m,n] = sum_k A[m,k] B[k,n], fp32 accumulation.
// Batch index z = blockIdx.z is split as (z / Z2, z % Z2) with separate strides.
// ---------------------------------------------------------------------------------------
struct GemmShape {
  int M, N, K, Z2;
  long sam, sak, sbk, sbn, scm, scn;
  long a1, a2, b1, b2, c1, c2;
};

template <typename TA, typename TB, typename TC>
__global__ void __launch_bounds__(256) k_gemm_generic(const TA* __restrict__ A, const TB* __restrict__ Bm,
                                                      TC* __restrict__ Cm, GemmShape g) {
  __shared__ float As[16][68];
  __shared__ float Bs[16][68];
  const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  const int z1 = blockIdx.z / g.Z2, z2 = blockIdx.z % g.Z2;
  A += z1 * g.a1 + z2 * g.a2;
  Bm += z1 * g.b1 + z2 * g.b2;
  Cm += z1 * g.c1 + z2 * g.c2;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  for (int k0 = 0; k0 < g.K; k0 += 16) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int idx = tid + i * 256;
      int m = idx / 16, k = idx % 16;
      float v = 0.f;
      if (m0 + m < g.M && k0 + k < g.K) v = ld(A + (long)(m0 + m) * g.sam + (long)(k0 + k) * g.sak);
      As[k][m] = v;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int idx = tid + i * 256;
      int k, n;
      if (g.sbn == 1) { k = idx / 64; n = idx % 64; } else { n = idx / 16; k = idx % 16; }
      float v = 0.f;
      if (n0 + n < g.N && k0 + k < g.K) v = ld(Bm + (long)(k0 + k) * g.sbk + (long)(n0 + n) * g.sbn);
      Bs[k][n] = v;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[k][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[k][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int m = m0 + ty * 4 + i;
    if (m >= g.M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int n = n0 + tx * 4 + j;
      if (n < g.N) st(Cm + (long)m * g.scm + (long)n * g.scn, acc[i][j]);
    }
  }
}

template <typename TA, typename TB, typename TC>
int gemm(Problem& p, const TA* A, const TB* Bm, TC* Cm, GemmShape g, int batches) {
  if (g.M <= 0 || g.N <= 0 || batches <= 0) return TA_OK;
  dim3 grid((g.N + 63) / 64, (g.M + 63) / 64, batches);
  k_gemm_generic<TA, TB, TC><<<grid, 256, 0, p.stream>>>(A, Bm, Cm, g);
  TA_LAUNCH_CHECK(p);
  return TA_OK;
}

static inline GemmShape plain(int M, int N, int K, long lda, long ldb_k, long ldb_n, long ldc) {
  GemmShape g;
  g.M = M; g.N = N; g.K = K; g.Z2 = 1;
  g.sam = lda; g.sak = 1; g.sbk = ldb_k; g.sbn = ldb_n; g.scm = ldc; g.scn = 1;
  g.a1 = g.a2 = g.b1 = g.b2 = g.c1 = g.c2 = 0;
  return g;
}

}  // namespace fma
}  // namespace ta
