// tucker_attn_decode_static: the decode step for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc on the decode path at all: a serving
// loop whose device memory was handed out once at start-up to a pool owned by someone else,
// a plug-in that runs under a framework which forbids allocation outside its own allocator,
// or a latency-critical loop where the implicit device synchronisation of cudaMalloc /
// cudaFree is not acceptable.  Such callers have their inputs and outputs but no way to
// produce the scratch buffer tucker_attn_decode asks for.  For them the scratch lives
// here, in a file-scope device array that every GPU loading the library holds from load to
// exit (TA_STATIC_SCRATCH_BYTES of its memory).
//
// The array's name is only a handle on the host side; the device address is looked up once
// per device with cudaGetSymbolAddress (with that device current) and cached.  The lookup
// happens in the first call on a device.
#include "ta_common.cuh"

#include <mutex>

namespace ta {
namespace {

static __device__ __align__(256) unsigned char g_static_scratch[TA_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the scratch array on the current device (nullptr on failure).
void* static_scratch_for_current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_addr[dev]) {
    void* ptr = nullptr;
    const cudaError_t e = cudaGetSymbolAddress((void**)&ptr, g_static_scratch);
    if (e != cudaSuccess || !ptr) {
      (void)cudaGetLastError();
      return nullptr;
    }
    g_scratch_addr[dev] = ptr;
  }
  return g_scratch_addr[dev];
}

}  // namespace
}  // namespace ta

extern "C" int tucker_attn_decode_static(const tucker_attn_desc* desc, const void* x, const void* C, const void* U1,
                                         const void* U2, const void* U3, const void* Ct, const void* Ut1,
                                         const void* Ut2, const void* Ut3, void* Kcache, void* Vcache, int32_t Lmax,
                                         const int32_t* cache_len, int32_t append, void* y, void* cuda_stream) {
  const size_t need = tucker_attn_decode_workspace_bytes(desc, Lmax);
  if (need > (size_t)TA_STATIC_SCRATCH_BYTES) return TA_ERR_WORKSPACE_TOO_SMALL;   // problem too large for the array
  void* scratch = ta::static_scratch_for_current_device();
  if (!scratch) return TA_ERR_CUDA;
  // need == 0 (invalid descriptor or Lmax, or a shape no kernel covers): nothing will be launched; the decode
  // call's own validation below names the reason with the status a caller-supplied workspace would get.
  // Nothing in the decode scratch has to start at zero: every region is written by an
  // earlier kernel of the same call before a later one reads it, so stale contents of the
  // previous call are harmless.
  return tucker_attn_decode(desc, x, C, U1, U2, U3, Ct, Ut1, Ut2, Ut3, Kcache, Vcache, Lmax, cache_len, append, y,
                            scratch, (size_t)TA_STATIC_SCRATCH_BYTES, cuda_stream);
}
