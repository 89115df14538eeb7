// Weight packers: MHA, GQA / MQA and MLA written as Tucker attention (Sec. 2.2: Lemma 1 and
// Theorems 1-3 state that each is a special case; the constructions below are those of the proofs).
//
//   GQA with n_G key / value heads (n_G = n_H: MHA, n_G = 1: MQA), ranks (n_H, d, n_G d_H):
//     U1 = I, U2 = W^Q, U3 = [W^K_1 .. W^K_{n_G}],  C[i, n, m] = 1 iff n = i d_H + l and m = g(i) d_H + l
//     Ut1 = I, Ut2 = (W^O)^T, Ut3 = [W^V_1 .. W^V_{n_G}],  Ct = C         (g(i) = floor(i n_G / n_H))
//   MLA without RoPE, ranks (n_H, d_c^Q, d_c^K) and (n_H, d, d_c^K): the up-projections go into the cores
//     U2 = W^DQ, U3 = W^DKV, C[i] = W^UQ_i (W^UK_i)^T
//     Ut3 = W^DV (W^DKV again for a shared latent), Ut2 = I_d, Ct[i, o, c] = (W^UV_i W^O_i)[c, o]
//
// These run once per set of weights, not per token: plain kernels, one thread per output element
// (or per 32 x 32 tile for the transposes and the two small per-head products).
#include "ta_common.cuh"

namespace ta {
namespace {

template <typename T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ldf<bf16>(const bf16* p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ T cvt(float v);
template <> __device__ __forceinline__ float cvt<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 cvt<bf16>(float v) { return __float2bfloat16_rn(v); }

// dst[i] = src[i]; 16 bytes per thread where both pointers and the length allow it
template <typename T>
__global__ void k_copy(const T* __restrict__ src, T* __restrict__ dst, long n) {
  constexpr int VEC = 16 / (int)sizeof(T);
  const bool vec_ok = (n % VEC == 0) && ((uintptr_t)src % 16 == 0) && ((uintptr_t)dst % 16 == 0);
  if (vec_ok) {
    const uint4* s4 = reinterpret_cast<const uint4*>(src);
    uint4* d4 = reinterpret_cast<uint4*>(dst);
    for (long i = blockIdx.x * (long)blockDim.x + threadIdx.x; i < n / VEC; i += (long)gridDim.x * blockDim.x) d4[i] = s4[i];
  } else {
    for (long i = blockIdx.x * (long)blockDim.x + threadIdx.x; i < n; i += (long)gridDim.x * blockDim.x) dst[i] = src[i];
  }
}

// dst = I_n
template <typename T>
__global__ void k_identity(T* __restrict__ dst, int n) {
  for (long i = blockIdx.x * (long)blockDim.x + threadIdx.x; i < (long)n * n; i += (long)gridDim.x * blockDim.x)
    dst[i] = cvt<T>((i / n) == (i % n) ? 1.f : 0.f);
}

// dst[c, r] = src[r, c] for src [rows, cols]; 32 x 32 tiles through shared memory, block (32, 8)
template <typename T>
__global__ void k_transpose(const T* __restrict__ src, T* __restrict__ dst, int rows, int cols) {
  __shared__ float tile[32][33];
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  for (int k = threadIdx.y; k < 32; k += 8) {
    const int r = r0 + k, c = c0 + threadIdx.x;
    if (r < rows && c < cols) tile[k][threadIdx.x] = ldf(src + (long)r * cols + c);
  }
  __syncthreads();
  for (int k = threadIdx.y; k < 32; k += 8) {
    const int c = c0 + k, r = r0 + threadIdx.x;
    if (r < rows && c < cols) dst[(long)c * rows + r] = cvt<T>(tile[threadIdx.x][k]);
  }
}

// Selector core of Lemma 1 / Theorem 2, written to two tensors (pre- and post-softmax core are equal):
// C[i, n, m] over [n_H, d, n_G d_H].  A thread writes 16 bytes of a row at a time when the row width allows
// it (VEC elements; VEC = 1 otherwise); a row holds at most one 1.
template <typename T, int VEC>
__global__ void k_selector_core(T* __restrict__ C, T* __restrict__ Ct, int nH, int nG, int d, int dH) {
  const long w = (long)nG * dH, wv = w / VEC, total = (long)nH * d * wv;
  for (long idx = blockIdx.x * (long)blockDim.x + threadIdx.x; idx < total; idx += (long)gridDim.x * blockDim.x) {
    const int m0 = (int)(idx % wv) * VEC, n = (int)((idx / wv) % d), i = (int)(idx / (wv * d));
    const int g = (int)(((long)i * nG) / nH);
    const int m_one = (n / dH == i) ? g * dH + n % dH : -1;      // column of this row's 1, if the row has one
    T v[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) v[e] = cvt<T>(m0 + e == m_one ? 1.f : 0.f);
    const long off = ((long)i * d + n) * w + m0;
    if (VEC == 1) {
      C[off] = v[0];
      Ct[off] = v[0];
    } else {
      *reinterpret_cast<uint4*>(C + off) = *reinterpret_cast<const uint4*>(v);
      *reinterpret_cast<uint4*>(Ct + off) = *reinterpret_cast<const uint4*>(v);
    }
  }
}

// MLA pre-softmax core: C[i, q, k] = sum_l WUQ[q, i dH + l] WUK[k, i dH + l]   (WUQ [dcq, d], WUK [dck, d])
template <typename T>
__global__ void k_mla_core(const T* __restrict__ WUQ, const T* __restrict__ WUK, T* __restrict__ C, int nH, int dcq,
                           int dck, int d, int dH) {
  const long total = (long)nH * dcq * dck;
  for (long idx = blockIdx.x * (long)blockDim.x + threadIdx.x; idx < total; idx += (long)gridDim.x * blockDim.x) {
    const int k = (int)(idx % dck), q = (int)((idx / dck) % dcq), i = (int)(idx / ((long)dck * dcq));
    const T* a = WUQ + (long)q * d + (long)i * dH;
    const T* b = WUK + (long)k * d + (long)i * dH;
    float acc = 0.f;
    for (int l = 0; l < dH; ++l) acc = fmaf(ldf(a + l), ldf(b + l), acc);
    C[idx] = cvt<T>(acc);
  }
}

// MLA post-softmax core: Ct[i, o, c] = sum_l WUV[c, i dH + l] WO[i dH + l, o]   (WUV [dck, d], WO [d, d])
template <typename T>
__global__ void k_mla_core_out(const T* __restrict__ WUV, const T* __restrict__ WO, T* __restrict__ Ct, int nH, int dck,
                               int d, int dH) {
  const long total = (long)nH * d * dck;
  for (long idx = blockIdx.x * (long)blockDim.x + threadIdx.x; idx < total; idx += (long)gridDim.x * blockDim.x) {
    const int c = (int)(idx % dck), o = (int)((idx / dck) % d), i = (int)(idx / ((long)dck * d));
    const T* a = WUV + (long)c * d + (long)i * dH;
    const T* b = WO + (long)i * dH * d + o;
    float acc = 0.f;
    for (int l = 0; l < dH; ++l) acc = fmaf(ldf(a + l), ldf(b + (long)l * d), acc);
    Ct[idx] = cvt<T>(acc);
  }
}

int blocks_for(long n) {
  long g = (n + 255) / 256;
  if (g > 148L * 16) g = 148L * 16;
  return (int)(g < 1 ? 1 : g);
}

bool launch_ok() { return cudaGetLastError() == cudaSuccess; }

template <typename T>
int pack_gqa_t(int d, int nH, int nG, const void* WQ, const void* WKg, const void* WVg, const void* WO, void* C, void* U1,
               void* U2, void* U3, void* Ct, void* Ut1, void* Ut2, void* Ut3, cudaStream_t st) {
  const int dH = d / nH;
  const long w = (long)nG * dH;
  constexpr int VEC = 16 / (int)sizeof(T);
  const bool vec_ok = (w % VEC == 0) && ((uintptr_t)C % 16 == 0) && ((uintptr_t)Ct % 16 == 0);
  if (vec_ok) k_selector_core<T, VEC><<<blocks_for((long)nH * d * w / VEC), 256, 0, st>>>((T*)C, (T*)Ct, nH, nG, d, dH);
  else k_selector_core<T, 1><<<blocks_for((long)nH * d * w), 256, 0, st>>>((T*)C, (T*)Ct, nH, nG, d, dH);
  k_identity<T><<<blocks_for((long)nH * nH), 256, 0, st>>>((T*)U1, nH);
  k_identity<T><<<blocks_for((long)nH * nH), 256, 0, st>>>((T*)Ut1, nH);
  k_copy<T><<<blocks_for((long)d * d), 256, 0, st>>>((const T*)WQ, (T*)U2, (long)d * d);
  k_copy<T><<<blocks_for((long)d * w), 256, 0, st>>>((const T*)WKg, (T*)U3, (long)d * w);
  k_copy<T><<<blocks_for((long)d * w), 256, 0, st>>>((const T*)WVg, (T*)Ut3, (long)d * w);
  k_transpose<T><<<dim3((d + 31) / 32, (d + 31) / 32), dim3(32, 8), 0, st>>>((const T*)WO, (T*)Ut2, d, d);
  return launch_ok() ? TA_OK : TA_ERR_CUDA;
}

template <typename T>
int pack_mla_t(int d, int nH, int dcq, int dck, const void* WDQ, const void* WUQ, const void* WDKV, const void* WUK,
               const void* WDV, const void* WUV, const void* WO, void* C, void* U1, void* U2, void* U3, void* Ct,
               void* Ut1, void* Ut2, void* Ut3, cudaStream_t st) {
  const int dH = d / nH;
  k_mla_core<T><<<blocks_for((long)nH * dcq * dck), 256, 0, st>>>((const T*)WUQ, (const T*)WUK, (T*)C, nH, dcq, dck, d, dH);
  k_mla_core_out<T><<<blocks_for((long)nH * d * dck), 256, 0, st>>>((const T*)WUV, (const T*)WO, (T*)Ct, nH, dck, d, dH);
  k_identity<T><<<blocks_for((long)nH * nH), 256, 0, st>>>((T*)U1, nH);
  k_identity<T><<<blocks_for((long)nH * nH), 256, 0, st>>>((T*)Ut1, nH);
  k_identity<T><<<blocks_for((long)d * d), 256, 0, st>>>((T*)Ut2, d);
  k_copy<T><<<blocks_for((long)d * dcq), 256, 0, st>>>((const T*)WDQ, (T*)U2, (long)d * dcq);
  k_copy<T><<<blocks_for((long)d * dck), 256, 0, st>>>((const T*)WDKV, (T*)U3, (long)d * dck);
  k_copy<T><<<blocks_for((long)d * dck), 256, 0, st>>>((const T*)WDV, (T*)Ut3, (long)d * dck);
  return launch_ok() ? TA_OK : TA_ERR_CUDA;
}

}  // namespace
}  // namespace ta

extern "C" int tucker_pack_gqa(int32_t d_model, int32_t n_H, int32_t n_G, int32_t dtype, const void* WQ, const void* WKg,
                               const void* WVg, const void* WO, void* C, void* U1, void* U2, void* U3, void* Ct,
                               void* Ut1, void* Ut2, void* Ut3, void* cuda_stream) {
  if (d_model <= 0 || n_H <= 0 || n_G <= 0 || n_G > n_H || d_model % n_H) return TA_ERR_INVALID_ARG;
  if (!WQ || !WKg || !WVg || !WO || !C || !U1 || !U2 || !U3 || !Ct || !Ut1 || !Ut2 || !Ut3) return TA_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (dtype == TA_DTYPE_F32)
    return ta::pack_gqa_t<float>(d_model, n_H, n_G, WQ, WKg, WVg, WO, C, U1, U2, U3, Ct, Ut1, Ut2, Ut3, st);
  if (dtype == TA_DTYPE_BF16)
    return ta::pack_gqa_t<ta::bf16>(d_model, n_H, n_G, WQ, WKg, WVg, WO, C, U1, U2, U3, Ct, Ut1, Ut2, Ut3, st);
  return TA_ERR_INVALID_ARG;
}

extern "C" int tucker_pack_mha(int32_t d_model, int32_t n_H, int32_t dtype, const void* WQ, const void* WK, const void* WV,
                               const void* WO, void* C, void* U1, void* U2, void* U3, void* Ct, void* Ut1, void* Ut2,
                               void* Ut3, void* cuda_stream) {
  return tucker_pack_gqa(d_model, n_H, n_H, dtype, WQ, WK, WV, WO, C, U1, U2, U3, Ct, Ut1, Ut2, Ut3, cuda_stream);
}

extern "C" int tucker_pack_mla(int32_t d_model, int32_t n_H, int32_t dcq, int32_t dck, int32_t dtype, const void* WDQ,
                               const void* WUQ, const void* WDKV, const void* WUK, const void* WDV, const void* WUV,
                               const void* WO, void* C, void* U1, void* U2, void* U3, void* Ct, void* Ut1, void* Ut2,
                               void* Ut3, void* cuda_stream) {
  if (d_model <= 0 || n_H <= 0 || dcq <= 0 || dck <= 0 || d_model % n_H) return TA_ERR_INVALID_ARG;
  if (!WDQ || !WUQ || !WDKV || !WUK || !WDV || !WUV || !WO || !C || !U1 || !U2 || !U3 || !Ct || !Ut1 || !Ut2 || !Ut3)
    return TA_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (dtype == TA_DTYPE_F32)
    return ta::pack_mla_t<float>(d_model, n_H, dcq, dck, WDQ, WUQ, WDKV, WUK, WDV, WUV, WO, C, U1, U2, U3, Ct, Ut1, Ut2, Ut3, st);
  if (dtype == TA_DTYPE_BF16)
    return ta::pack_mla_t<ta::bf16>(d_model, n_H, dcq, dck, WDQ, WUQ, WDKV, WUK, WDV, WUV, WO, C, U1, U2, U3, Ct, Ut1, Ut2, Ut3, st);
  return TA_ERR_INVALID_ARG;
}
