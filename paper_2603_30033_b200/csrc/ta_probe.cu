// Measurement probe for the core-factorised score form (Sec. 3.3, "Implementation": kernels that use the
// factorised core directly, S_h = sum_a U1[h, a] (Qt C_a K^T)): the step that form adds to the softmax warps.
// With the r1 plane tiles P_a = Qt C_a K^T of a [128 query x 128 key] tile at hand, every head's score tile is
// the mix sum_a U1[h, a] P_a: r1 fused multiply-adds per score and head, on the CUDA cores, by the thread that
// owns the score row.  This kernel does exactly that mixing and nothing else -- planes read from TMEM in
// 32-column chunks (where the plane MMAs would leave them), one warpgroup per head of a pair with thread =
// score row as in the attention kernel, packed f32x2 FMAs -- so that its cycles per tile can be set against the
// tensor-core cycles the form would save.
#include "ta_common.cuh"
#include "ta_sm100.cuh"

namespace ta {
namespace {

using namespace sm100;

constexpr int PM_THREADS = 256;     // two warpgroups: thread = one score row (TMEM lane) of one head of the pair
constexpr int PM_MAX_R1 = 16;

__global__ void __launch_bounds__(PM_THREADS, 1) k_probe_plane_mix(int tiles, int r1, const float* __restrict__ u1,
                                                                     long long* __restrict__ cycles, float* __restrict__ sink) {
  __shared__ uint32_t tmem_slot;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int head = threadIdx.x / 128;
  if (warp == 0) {
    tmem_alloc(&tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_slot;
  const uint32_t lane_addr = (uint32_t)((warp % 4) * 32) << 16;
  {
    // give the plane columns defined contents (four plane buffers of 128 columns; planes a and a + 4 share one)
    uint32_t z[32];
#pragma unroll
    for (int c = 0; c < 32; ++c) z[c] = __float_as_uint(1e-3f * (float)((lane + c) % 13));
    if (head == 0)
      for (int col = 0; col < 512; col += 32) tmem_st32(tmem + lane_addr + col, z);
    tmem_st_wait();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  float2 u[PM_MAX_R1];
#pragma unroll
  for (int a = 0; a < PM_MAX_R1; ++a) u[a] = a < r1 ? make_float2(u1[head * r1 + a], u1[head * r1 + a]) : make_float2(0.f, 0.f);
  float2 check = make_float2(0.f, 0.f);
  const long long t0 = clock64();
  for (int t = 0; t < tiles; ++t) {
#pragma unroll 1
    for (int ch = 0; ch < 4; ++ch) {                 // 4 chunks of 32 score columns
      float2 s[16];
#pragma unroll
      for (int c = 0; c < 16; ++c) s[c] = make_float2(0.f, 0.f);
#pragma unroll
      for (int a = 0; a < PM_MAX_R1; ++a) {
        if (a < r1) {
          uint32_t pr[32];
          tmem_ld32(tmem + lane_addr + (uint32_t)((a & 3) * 128 + ch * 32), pr);
          tmem_ld_wait();
#pragma unroll
          for (int c = 0; c < 16; ++c)
            s[c] = __ffma2_rn(u[a], make_float2(__uint_as_float(pr[2 * c]), __uint_as_float(pr[2 * c + 1])), s[c]);
        }
      }
#pragma unroll
      for (int c = 0; c < 16; ++c) check = __fadd2_rn(check, s[c]);
    }
  }
  const long long t1 = clock64();
  if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
  sink[blockIdx.x * PM_THREADS + threadIdx.x] = check.x + check.y;
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 512);
}

// Issue rate of tcgen05.mma (M = 128, K = 16, bf16 -> fp32) by operand source and layout: `iters` groups of
// eight dependent-accumulator MMAs issued back to back by one thread, one commit at the end.
//   mode 0  A and B in shared memory, both K-major       mode 1  A in TMEM, B K-major in shared memory
//   mode 2  A K-major, B MN-major in shared memory (a tile used where it lies with its N index contiguous)
__global__ void __launch_bounds__(128, 1) k_probe_mma_rate(int mode, int N, int iters, long long* __restrict__ cycles,
                                                            unsigned int* err) {
  extern __shared__ uint8_t pm_smem[];
  __shared__ uint64_t bar;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  const uint32_t base = (smem_u32(pm_smem) + 1023u) & ~1023u;
  uint8_t* tiles = pm_smem + (base - smem_u32(pm_smem));
  for (int i = threadIdx.x; i < 96 * 1024 / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(tiles)[i] = 0x3c003c00u;
  const int warp = threadIdx.x / 32;
  Abort ab{&abort_flag, err};
  if (threadIdx.x == 0) { abort_flag = 0; mbar_init(&bar, 1); fence_barrier_init(); }
  if (warp == 0) { tmem_alloc(&tmem_slot, 512); tmem_relinquish(); }
  fence_proxy_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_slot;
  if (warp == 1 && elect_one()) {
    const uint32_t idesc = umma_idesc_bf16(128, (uint32_t)N);
    const uint32_t a = smem_u32(tiles), b = smem_u32(tiles + 32 * 1024);
    const long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const uint32_t off = (uint32_t)(ks >> 2) * 16384u + (uint32_t)(ks & 3) * 32;
        if (mode == 0) umma_ss(tmem, umma_desc_kmajor_sw128(a + off), umma_desc_kmajor_sw128(b + off), idesc, 1);
        else if (mode == 1) umma_ts(tmem, tmem + 256 + ks * 8, umma_desc_kmajor_sw128(b + off), idesc, 1);
        else umma_ss(tmem, umma_desc_kmajor_sw128(a + off), umma_desc_mnmajor_sw128(b + ks * 2048, 16384), idesc | (1u << 16), 1);
      }
    }
    umma_commit(&bar);
    (void)mbar_wait(&bar, 0, ab);
    cycles[blockIdx.x] = clock64() - t0;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 512);
}

}  // namespace
}  // namespace ta

extern "C" int tucker_probe_plane_mix(int32_t tiles, int32_t r1, int32_t n_blocks, const float* u1, long long* cycles,
                                      float* sink, void* cuda_stream) {
  using namespace ta;
  if (tiles <= 0 || r1 <= 0 || r1 > PM_MAX_R1 || n_blocks <= 0 || !u1 || !cycles || !sink) return TA_ERR_INVALID_ARG;
  k_probe_plane_mix<<<n_blocks, PM_THREADS, 0, static_cast<cudaStream_t>(cuda_stream)>>>(tiles, r1, u1, cycles, sink);
  return cudaGetLastError() == cudaSuccess ? TA_OK : TA_ERR_CUDA;
}

extern "C" int tucker_probe_mma_rate(int32_t mode, int32_t N, int32_t iters, int32_t n_blocks, long long* cycles,
                                     void* cuda_stream) {
  using namespace ta;
  if (mode < 0 || mode > 2 || (N != 64 && N != 128 && N != 256) || iters <= 0 || iters > 4096 || n_blocks <= 0 || !cycles)
    return TA_ERR_INVALID_ARG;
  unsigned int* errp = device_error_word();
  if (!errp) return TA_ERR_CUDA;
  static PerDeviceFlag attr;
  TA_CUDA_TRY(ensure_dynamic_smem(attr, (const void*)k_probe_mma_rate, 100 * 1024));
  k_probe_mma_rate<<<n_blocks, 128, 100 * 1024, static_cast<cudaStream_t>(cuda_stream)>>>(mode, N, iters, cycles, errp);
  return cudaGetLastError() == cudaSuccess ? TA_OK : TA_ERR_CUDA;
}
