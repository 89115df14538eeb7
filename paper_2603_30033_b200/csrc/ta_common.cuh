// Shared declarations of the Tucker-attention CUDA library (internal; the public ABI is
// include/tucker_attn.h).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stddef.h>
#include <stdint.h>

#include <mutex>

#include "tucker_attn.h"

namespace ta {

typedef __nv_bfloat16 bf16;

// Device address of the current device's error word (nullptr if it cannot be resolved); ta_api.cu.
unsigned int* device_error_word();

// Everything a path needs to run one call; filled by the API layer after validation.
struct Problem {
  tucker_attn_desc d;
  float scale;              // resolved softmax scale
  const void *X, *C, *U1, *U2, *U3, *Ct, *Ut1, *Ut2, *Ut3;
  void* Y;
  void *Kc, *Vc;            // prefill: optional cache outputs; decode: caches
  int32_t Lmax;
  const int32_t* cache_len; // decode only (device)
  int32_t append;           // decode only
  int shared_kv;            // one latent cache / one projection serves keys and values (U3 == Ut3)
  int shared_rope;          // ... together with latent RoPE: the one cache holds UN-rotated latent rows
  char* ws;                 // workspace base (256-byte aligned)
  size_t ws_bytes;
  cudaStream_t stream;
  unsigned int* dev_err;    // device error word of the current device
  int launches;             // kernels launched so far by this call
  cudaEvent_t prof_start, prof_stop;  // optional: recorded around the dominant kernel
};

// Records the caller's profiling events (if registered) around the dominant kernel.
static inline void prof_begin(const Problem& p) { if (p.prof_start) (void)cudaEventRecord(p.prof_start, p.stream); }
static inline void prof_end(const Problem& p) { if (p.prof_stop) (void)cudaEventRecord(p.prof_stop, p.stream); }

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Carves consecutive 256-byte aligned regions out of the workspace; with base == nullptr it
// only measures.
struct Carver {
  char* base;
  size_t off;
  explicit Carver(char* b) : base(b), off(0) {}
  template <typename T>
  T* take(size_t count) {
    size_t o = off;
    off = align_up(off + count * sizeof(T), 256);
    return base ? reinterpret_cast<T*>(base + o) : nullptr;
  }
};

// shape-generic FMA path (ta_generic.cu)
size_t generic_fwd_workspace(const tucker_attn_desc& d);
size_t generic_decode_workspace(const tucker_attn_desc& d, int32_t Lmax);
int generic_fwd(Problem& p);
int generic_decode(Problem& p);

int simt_attention_bf16(Problem& p, const bf16* Qhat, const bf16* K, const bf16* V, bf16* O);

// tensor-core path (bf16 storage): returns false from *_supported when the shape is outside
// what the kernels were built for, in which case the generic path runs.
bool fast_fwd_supported(const tucker_attn_desc& d);
size_t fast_fwd_workspace(const tucker_attn_desc& d);
int fast_fwd(Problem& p);
bool fast_decode_supported(const tucker_attn_desc& d, int32_t Lmax);
size_t fast_decode_workspace(const tucker_attn_desc& d, int32_t Lmax);
int fast_decode(Problem& p);
int wait_selftest(unsigned int* dev_err, int budget_us, int* out_dev, cudaStream_t stream);

// Tensor-core GEMM with fp32 split-K partial outputs (ta_fast.cu): for z < splits,
//   out[z * split_stride + row * N + col] = sum over the z-th share of K of A[row, k] B[col, k],
// A [M, K] and B [N, K] bf16 with K contiguous (leading dimensions lda, ldb), K a multiple of 64 whose
// 64-blocks divide evenly by `splits`, N a multiple of 64; rows >= M of a 128-row tile are not written.
// Uses p.stream, p.dev_err, p.launches only.
int umma_gemm_f32_partials(Problem& p, const bf16* A, long lda, int M, const bf16* B, long ldb, int N, int K, int splits,
                           float* out, long split_stride);

// HOSVD initialiser (ta_hosvd.cu)
size_t hosvd_workspace(int n1, int n2, int n3, int r2, int r3);
int hosvd_run(Problem& p, int n1, int n2, int n3, int r1, int r2, int r3, const float* T, float* core, float* U1,
              float* U2, float* U3, float* spectra);
int mha_weight_tensors_run(Problem& p, int d, int nH, const float* WQ, const float* WK, const float* WV, const float* WO,
                           float* W, float* Wt);

// Layout of the prefill path's (cos, sin) table.  Its readers hold one position per thread and 32 consecutive
// positions per warp, so the table is stored in units of one float4 = two (cos, sin) pairs, with the 32 positions
// of a block of positions next to each other: unit u (0 .. r3/4 - 1) of position n lies at float4 index
//   ((n / 32) * units + u) * 32 + n % 32,
// and a warp's load of one unit for its 32 rows is one 512-byte segment.  (Stored position-major, every such load
// touched 32 different rows of the table: 2500 cycles per 32 columns in the attention kernel's query conversion.)
__host__ __device__ __forceinline__ long rope_unit_index(int n, int u, int units) {
  return ((long)(n >> 5) * units + u) * 32 + (n & 31);
}
static inline size_t rope_table_units(int n_pos, int r3) { return (size_t)((n_pos + 31) / 32) * 32 * (size_t)(r3 / 4); }

// Programmatic dependent launch.  Every kernel of the tensor-core paths starts with pdl_enter():
// it waits until the preceding kernels of the stream have completed and their writes are visible,
// and only then lets the next kernel of the stream be scheduled.  Launched through launch_pdl, a
// kernel's launch and block scheduling therefore overlap the tail of its predecessor, while nothing
// (global memory, TMEM) is touched before the predecessor is done.  Without the launch attribute
// both instructions are no-ops.
#if defined(__CUDACC__)
__device__ __forceinline__ void pdl_enter() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
#endif

template <typename... KArgs, typename... Args>
static inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                     Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Per-device one-time set-up.  A kernel's dynamic shared-memory limit and the device properties are per
// device, and one process may drive several GPUs, so each is recorded per device ordinal under a mutex.
constexpr int kMaxDevices = 64;
struct PerDeviceFlag {
  std::mutex m;
  bool done[kMaxDevices] = {};
};
// Raises `func`'s dynamic shared-memory limit to `bytes` on the current device, once per device.
static inline cudaError_t ensure_dynamic_smem(PerDeviceFlag& f, const void* func, int bytes) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(f.m);
  if (f.done[dev]) return cudaSuccess;
  e = cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) f.done[dev] = true;
  return e;
}

// Debug build (-DTA_BOUNDS_CHECK): every global index that the tensor-core kernels and the decode kernels
// form for a store, and for a load from the workspace, is compared with the extent of the tensor it
// addresses before it is used.  A failure sets TA_DEVERR_BAD_INDEX in the device error word and the access
// is skipped; nothing traps.  In the normal build the macro is the constant `true`.
#if defined(__CUDACC__) && defined(TA_BOUNDS_CHECK)
__device__ __forceinline__ bool index_in_bounds(unsigned int* err, long first, long count, long extent) {
  if (first >= 0 && count >= 0 && first + count <= extent) return true;
  if (err) atomicOr(err, (unsigned)TA_DEVERR_BAD_INDEX);
  return false;
}
#define TA_IDX_OK(err, first, count, extent) ::ta::index_in_bounds((err), (long)(first), (long)(count), (long)(extent))
#else
#define TA_IDX_OK(err, first, count, extent) true
#endif

#define TA_CUDA_TRY(expr)                          \
  do {                                             \
    cudaError_t _e = (expr);                       \
    if (_e != cudaSuccess) return TA_ERR_CUDA;     \
  } while (0)

#define TA_LAUNCH_CHECK(p)                                   \
  do {                                                       \
    (p).launches++;                                          \
    if (cudaPeekAtLastError() != cudaSuccess) {              \
      (void)cudaGetLastError();                              \
      return TA_ERR_CUDA;                                    \
    }                                                        \
  } while (0)

}  // namespace ta
