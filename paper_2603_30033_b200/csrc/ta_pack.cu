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
// These run once per set of weights, not per token: plain kernels, one thread per output element or
// 16-byte vector (32 x 32 tiles for the transpose); the GQA / MHA packing is a single launch.
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

// One launch for the whole GQA / MHA packing: consecutive block ranges do the selector cores, the two
// identities, the three copies and the transpose (this runs once per set of weights, but seven launches
// of a few microseconds each were most of its time).
template <typename T>
struct GqaPack {
  const T *WQ, *WKg, *WVg, *WO;
  T *C, *U1, *U2, *U3, *Ct, *Ut1, *Ut2, *Ut3;
  int nH, nG, d, dH;
  int b_core, b_id, b_copy;      // blocks of the core part, of one identity, of one copy; then the transpose tiles
};

template <typename T, int VEC>
__device__ __forceinline__ void selector_core_part(T* __restrict__ C, T* __restrict__ Ct, int nH, int nG, int d, int dH,
                                                   int blk, int nblk) {
  const long w = (long)nG * dH, wv = w / VEC, total = (long)nH * d * wv;
  for (long idx = blk * (long)blockDim.x + threadIdx.x; idx < total; idx += (long)nblk * blockDim.x) {
    const int m0 = (int)(idx % wv) * VEC, n = (int)((idx / wv) % d), i = (int)(idx / (wv * d));
    const int g = (int)(((long)i * nG) / nH);
    const int m_one = (n / dH == i) ? g * dH + n % dH : -1;
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

template <typename T>
__device__ __forceinline__ void copy_part(const T* __restrict__ src, T* __restrict__ dst, long n, int blk, int nblk) {
  constexpr int VEC = 16 / (int)sizeof(T);
  const bool vec_ok = (n % VEC == 0) && ((uintptr_t)src % 16 == 0) && ((uintptr_t)dst % 16 == 0);
  if (vec_ok) {
    const uint4* s4 = reinterpret_cast<const uint4*>(src);
    uint4* d4 = reinterpret_cast<uint4*>(dst);
    for (long i = blk * (long)blockDim.x + threadIdx.x; i < n / VEC; i += (long)nblk * blockDim.x) d4[i] = s4[i];
  } else {
    for (long i = blk * (long)blockDim.x + threadIdx.x; i < n; i += (long)nblk * blockDim.x) dst[i] = src[i];
  }
}

template <typename T>
__device__ __forceinline__ void identity_part(T* __restrict__ dst, int n, int blk, int nblk) {
  for (long i = blk * (long)blockDim.x + threadIdx.x; i < (long)n * n; i += (long)nblk * blockDim.x)
    dst[i] = cvt<T>((i / n) == (i % n) ? 1.f : 0.f);
}

template <typename T, int VEC>
__global__ void __launch_bounds__(256) k_pack_gqa(const GqaPack<T> p) {
  __shared__ float tile[32][33];
  int blk = blockIdx.x;
  const long w = (long)p.nG * p.dH;
  if (blk < p.b_core) { selector_core_part<T, VEC>(p.C, p.Ct, p.nH, p.nG, p.d, p.dH, blk, p.b_core); return; }
  blk -= p.b_core;
  if (blk < 2 * p.b_id) { identity_part<T>(blk < p.b_id ? p.U1 : p.Ut1, p.nH, blk % p.b_id, p.b_id); return; }
  blk -= 2 * p.b_id;
  if (blk < 3 * p.b_copy) {
    const int which = blk / p.b_copy, b = blk % p.b_copy;
    if (which == 0) copy_part<T>(p.WQ, p.U2, (long)p.d * p.d, b, p.b_copy);
    else if (which == 1) copy_part<T>(p.WKg, p.U3, (long)p.d * w, b, p.b_copy);
    else copy_part<T>(p.WVg, p.Ut3, (long)p.d * w, b, p.b_copy);
    return;
  }
  blk -= 3 * p.b_copy;
  // Ut2 = WO^T: one 32 x 32 tile per block (thread (x, y) = (t % 32, t / 32), eight rows per pass)
  const int tiles_x = (p.d + 31) / 32;
  const int c0 = (blk % tiles_x) * 32, r0 = (blk / tiles_x) * 32;
  const int tx = threadIdx.x % 32, ty = threadIdx.x / 32;
  for (int k = ty; k < 32; k += 8) {
    const int r = r0 + k, c = c0 + tx;
    if (r < p.d && c < p.d) tile[k][tx] = ldf(p.WO + (long)r * p.d + c);
  }
  __syncthreads();
  for (int k = ty; k < 32; k += 8) {
    const int c = c0 + k, r = r0 + tx;
    if (r < p.d && c < p.d) p.Ut2[(long)c * p.d + r] = cvt<T>(tile[tx][k]);
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
  GqaPack<T> p;
  p.WQ = (const T*)WQ; p.WKg = (const T*)WKg; p.WVg = (const T*)WVg; p.WO = (const T*)WO;
  p.C = (T*)C; p.U1 = (T*)U1; p.U2 = (T*)U2; p.U3 = (T*)U3; p.Ct = (T*)Ct; p.Ut1 = (T*)Ut1; p.Ut2 = (T*)Ut2; p.Ut3 = (T*)Ut3;
  p.nH = nH; p.nG = nG; p.d = d; p.dH = dH;
  p.b_core = blocks_for((long)nH * d * w / (vec_ok ? VEC : 1));
  p.b_id = blocks_for((long)nH * nH);
  p.b_copy = blocks_for((long)d * d / VEC);
  const int tiles = ((d + 31) / 32) * ((d + 31) / 32);
  const int grid = p.b_core + 2 * p.b_id + 3 * p.b_copy + tiles;
  if (vec_ok) k_pack_gqa<T, VEC><<<grid, 256, 0, st>>>(p);
  else k_pack_gqa<T, 1><<<grid, 256, 0, st>>>(p);
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
