// C ABI entry points: argument validation, path selection, workspace sizing, error word.
#include "ta_common.cuh"

#include <math.h>

namespace ta {

__device__ unsigned int g_device_error_word = 0;

static thread_local int tl_last_path = 0;
static thread_local int tl_last_launches = 0;
static thread_local cudaEvent_t tl_prof_start = nullptr;
static thread_local cudaEvent_t tl_prof_stop = nullptr;

static unsigned int* device_error_ptr() {
  // one address per device; looked up lazily, cached per device ordinal
  static unsigned int* cache[kMaxDevices] = {nullptr};
  static std::mutex m;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(m);
  if (!cache[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_device_error_word) != cudaSuccess) return nullptr;
    cache[dev] = static_cast<unsigned int*>(ptr);
  }
  return cache[dev];
}

unsigned int* device_error_word() { return device_error_ptr(); }

static bool desc_ok(const tucker_attn_desc* d, bool decode) {
  if (!d) return false;
  if (d->B <= 0 || d->d_model <= 0 || d->n_H <= 0) return false;
  if (!decode && d->N <= 0) return false;
  if (d->d_model % d->n_H) return false;
  if (d->r1 <= 0 || d->r2 <= 0 || d->r3 <= 0 || d->t1 <= 0 || d->t2 <= 0 || d->t3 <= 0) return false;
  if (d->rope && (d->r3 % 2)) return false;
  if (d->rope && !(d->rope_base > 0.f)) return false;
  if (d->dtype != TA_DTYPE_F32 && d->dtype != TA_DTYPE_BF16) return false;
  return true;
}

static float resolve_scale(const tucker_attn_desc& d) {
  return d.scale > 0.f ? d.scale : (float)(1.0 / sqrt((double)d.d_model / (double)d.n_H));
}

static bool use_fast_fwd(const tucker_attn_desc& d) {
  return d.dtype == TA_DTYPE_BF16 && !(d.flags & TA_FLAG_FORCE_GENERIC) && fast_fwd_supported(d);
}
static bool use_fast_decode(const tucker_attn_desc& d, int32_t Lmax) {
  return d.dtype == TA_DTYPE_BF16 && !(d.flags & TA_FLAG_FORCE_GENERIC) && fast_decode_supported(d, Lmax);
}

// Shared key / value projection (Sec. 3.1, L^KV = X U3): the caller passes the SAME factor for U3 and Ut3.
// Without RoPE the latent keys are then the latent values, so one projection and one cache serve both.
// With latent RoPE the one cache holds the un-rotated latent rows (the values); keys are rotated when used.
static bool shared_kv_weights(const tucker_attn_desc& d, const void* U3, const void* Ut3) {
  return U3 == Ut3 && d.r3 == d.t3;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace ta

using namespace ta;

extern "C" {

size_t tucker_attn_fwd_workspace_bytes(const tucker_attn_desc* desc) {
  if (!desc_ok(desc, false)) return 0;
  return use_fast_fwd(*desc) ? fast_fwd_workspace(*desc) : generic_fwd_workspace(*desc);
}

size_t tucker_attn_decode_workspace_bytes(const tucker_attn_desc* desc, int32_t Lmax) {
  if (!desc_ok(desc, true) || Lmax <= 0) return 0;
  return use_fast_decode(*desc, Lmax) ? fast_decode_workspace(*desc, Lmax) : generic_decode_workspace(*desc, Lmax);
}

int tucker_attn_fwd(const tucker_attn_desc* desc, const void* X, const void* C, const void* U1, const void* U2,
                    const void* U3, const void* Ct, const void* Ut1, const void* Ut2, const void* Ut3, void* Y,
                    void* Kcache_out, void* Vcache_out, int32_t Lmax, void* workspace, size_t workspace_bytes,
                    void* cuda_stream) {
  if (!desc_ok(desc, false)) return TA_ERR_INVALID_ARG;
  if (!X || !C || !U1 || !U2 || !U3 || !Ct || !Ut1 || !Ut2 || !Ut3 || !Y || !workspace) return TA_ERR_INVALID_ARG;
  if ((Kcache_out == nullptr) != (Vcache_out == nullptr)) return TA_ERR_INVALID_ARG;
  if (Kcache_out && Lmax < desc->N) return TA_ERR_INVALID_ARG;
  if (Kcache_out && Kcache_out == Vcache_out && !shared_kv_weights(*desc, U3, Ut3)) return TA_ERR_INVALID_ARG;
  const void* ptrs[] = {X, C, U1, U2, U3, Ct, Ut1, Ut2, Ut3, Y};
  for (const void* q : ptrs)
    if (!aligned16(q)) return TA_ERR_INVALID_ARG;
  if (Kcache_out && (!aligned16(Kcache_out) || !aligned16(Vcache_out))) return TA_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return TA_ERR_INVALID_ARG;
  const bool fast = use_fast_fwd(*desc);
  const size_t need = fast ? fast_fwd_workspace(*desc) : generic_fwd_workspace(*desc);
  if (need == 0) return TA_ERR_UNSUPPORTED_SHAPE;
  if (workspace_bytes < need) return TA_ERR_WORKSPACE_TOO_SMALL;
  Problem p;
  p.d = *desc;
  p.scale = resolve_scale(*desc);
  p.X = X; p.C = C; p.U1 = U1; p.U2 = U2; p.U3 = U3; p.Ct = Ct; p.Ut1 = Ut1; p.Ut2 = Ut2; p.Ut3 = Ut3;
  p.Y = Y; p.Kc = Kcache_out; p.Vc = Vcache_out; p.Lmax = Lmax;
  p.cache_len = nullptr; p.append = 0;
  const bool one_cache = shared_kv_weights(*desc, U3, Ut3) && Kcache_out == Vcache_out;
  p.shared_kv = (one_cache && !desc->rope) ? 1 : 0;                   // one projection serves keys and values
  p.shared_rope = (one_cache && desc->rope && Kcache_out) ? 1 : 0;    // rotated keys computed, un-rotated rows cached
  p.ws = static_cast<char*>(workspace); p.ws_bytes = workspace_bytes;
  p.stream = static_cast<cudaStream_t>(cuda_stream);
  p.dev_err = device_error_ptr();
  p.launches = 0;
  p.prof_start = tl_prof_start; p.prof_stop = tl_prof_stop;
  if (!p.dev_err) return TA_ERR_CUDA;
  const int rc = fast ? fast_fwd(p) : generic_fwd(p);
  tl_last_path = fast ? 2 : 1;
  tl_last_launches = p.launches;
  return rc;
}

int tucker_attn_decode(const tucker_attn_desc* desc, const void* x, const void* C, const void* U1, const void* U2,
                       const void* U3, const void* Ct, const void* Ut1, const void* Ut2, const void* Ut3,
                       void* Kcache, void* Vcache, int32_t Lmax, const int32_t* cache_len, int32_t append, void* y,
                       void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!desc_ok(desc, true)) return TA_ERR_INVALID_ARG;
  if (!x || !C || !U1 || !U2 || !U3 || !Ct || !Ut1 || !Ut2 || !Ut3 || !y || !workspace) return TA_ERR_INVALID_ARG;
  if (!Kcache || !Vcache || !cache_len || Lmax <= 0) return TA_ERR_INVALID_ARG;
  if (Kcache == Vcache && !shared_kv_weights(*desc, U3, Ut3)) return TA_ERR_INVALID_ARG;
  const void* ptrs[] = {x, C, U1, U2, U3, Ct, Ut1, Ut2, Ut3, y, Kcache, Vcache};
  for (const void* q : ptrs)
    if (!aligned16(q)) return TA_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return TA_ERR_INVALID_ARG;
  const bool fast = use_fast_decode(*desc, Lmax);
  const size_t need = fast ? fast_decode_workspace(*desc, Lmax) : generic_decode_workspace(*desc, Lmax);
  if (need == 0) return TA_ERR_UNSUPPORTED_SHAPE;
  if (workspace_bytes < need) return TA_ERR_WORKSPACE_TOO_SMALL;
  Problem p;
  p.d = *desc;
  p.scale = resolve_scale(*desc);
  p.X = x; p.C = C; p.U1 = U1; p.U2 = U2; p.U3 = U3; p.Ct = Ct; p.Ut1 = Ut1; p.Ut2 = Ut2; p.Ut3 = Ut3;
  p.Y = y; p.Kc = Kcache; p.Vc = Vcache; p.Lmax = Lmax;
  p.cache_len = cache_len; p.append = append ? 1 : 0;
  p.shared_kv = (Kcache == Vcache) ? 1 : 0;
  p.shared_rope = (p.shared_kv && desc->rope) ? 1 : 0;
  p.ws = static_cast<char*>(workspace); p.ws_bytes = workspace_bytes;
  p.stream = static_cast<cudaStream_t>(cuda_stream);
  p.dev_err = device_error_ptr();
  p.launches = 0;
  p.prof_start = tl_prof_start; p.prof_stop = tl_prof_stop;
  if (!p.dev_err) return TA_ERR_CUDA;
  const int rc = fast ? fast_decode(p) : generic_decode(p);
  tl_last_path = fast ? 2 : 1;
  tl_last_launches = p.launches;
  return rc;
}

const char* tucker_attn_status_string(int status) {
  switch (status) {
    case TA_OK: return "ok";
    case TA_ERR_INVALID_ARG: return "invalid argument";
    case TA_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case TA_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case TA_ERR_CUDA: return "CUDA error";
    case TA_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
  }
}

int tucker_attn_last_device_error(void* cuda_stream) {
  unsigned int* ptr = device_error_ptr();
  if (!ptr) return TA_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  unsigned int host = 0;
  if (cudaMemcpyAsync(&host, ptr, sizeof(host), cudaMemcpyDeviceToHost, s) != cudaSuccess) return TA_ERR_CUDA;
  if (cudaMemsetAsync(ptr, 0, sizeof(host), s) != cudaSuccess) return TA_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return TA_ERR_CUDA;
  return (int)host;
}

static bool hosvd_args_ok(int32_t d, int32_t nH, int32_t r1, int32_t r2, int32_t r3) {
  return d > 0 && d <= 8192 && nH > 0 && nH <= 64 && r1 >= 1 && r1 <= nH && r2 >= 1 && r2 <= d && r3 >= 1 && r3 <= d;
}

size_t tucker_hosvd_workspace_bytes(int32_t d_model, int32_t n_H, int32_t r2, int32_t r3) {
  if (!hosvd_args_ok(d_model, n_H, 1, r2, r3)) return 0;
  return hosvd_workspace(n_H, d_model, d_model, r2, r3);
}

int tucker_hosvd_init(int32_t d_model, int32_t n_H, int32_t r1, int32_t r2, int32_t r3, const float* W, float* C,
                      float* U1, float* U2, float* U3, float* spectra, void* workspace, size_t workspace_bytes,
                      void* cuda_stream) {
  if (!hosvd_args_ok(d_model, n_H, r1, r2, r3)) return TA_ERR_INVALID_ARG;
  if (!W || !C || !U1 || !U2 || !U3 || !workspace) return TA_ERR_INVALID_ARG;
  if (!aligned16(W) || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return TA_ERR_INVALID_ARG;
  if (workspace_bytes < hosvd_workspace(n_H, d_model, d_model, r2, r3)) return TA_ERR_WORKSPACE_TOO_SMALL;
  Problem p = {};
  p.ws = static_cast<char*>(workspace); p.ws_bytes = workspace_bytes;
  p.stream = static_cast<cudaStream_t>(cuda_stream);
  p.dev_err = device_error_ptr();
  p.prof_start = tl_prof_start; p.prof_stop = tl_prof_stop;
  if (!p.dev_err) return TA_ERR_CUDA;
  const int rc = hosvd_run(p, n_H, d_model, d_model, r1, r2, r3, W, C, U1, U2, U3, spectra);
  tl_last_path = 2;
  tl_last_launches = p.launches;
  return rc;
}

int tucker_mha_weight_tensors(int32_t d_model, int32_t n_H, const float* WQ, const float* WK, const float* WV,
                              const float* WO, float* W, float* Wt, void* cuda_stream) {
  if (d_model <= 0 || n_H <= 0 || d_model % n_H || !WQ || !WK || !WV || !WO || !W || !Wt) return TA_ERR_INVALID_ARG;
  Problem p = {};
  p.stream = static_cast<cudaStream_t>(cuda_stream);
  p.dev_err = device_error_ptr();
  if (!p.dev_err) return TA_ERR_CUDA;
  const int rc = mha_weight_tensors_run(p, d_model, n_H, WQ, WK, WV, WO, W, Wt);
  tl_last_launches = p.launches;
  return rc;
}

int tucker_attn_sync_status(void* cuda_stream) {
  const int word = tucker_attn_last_device_error(cuda_stream);
  if (word < 0) return word;
  if (word & TA_DEVERR_WAIT_TIMEOUT) return TA_ERR_DEVICE_TIMEOUT;
  if (word & TA_DEVERR_BAD_CACHE_LEN) return TA_ERR_INVALID_ARG;
  if (word & TA_DEVERR_BAD_INDEX) return TA_ERR_CUDA;
  return TA_OK;
}

int tucker_attn_bounds_checked(void) {
#ifdef TA_BOUNDS_CHECK
  return 1;
#else
  return 0;
#endif
}

int tucker_attn_selftest_wait_timeout(int32_t budget_us, int32_t* out, void* cuda_stream) {
  if (budget_us <= 0 || budget_us > 100000 || !out) return TA_ERR_INVALID_ARG;
  unsigned int* ptr = device_error_ptr();
  if (!ptr) return TA_ERR_CUDA;
  return wait_selftest(ptr, budget_us, out, static_cast<cudaStream_t>(cuda_stream));
}

int tucker_attn_set_profile_events(void* ev_start, void* ev_stop) {
  if ((ev_start == nullptr) != (ev_stop == nullptr)) return TA_ERR_INVALID_ARG;
  tl_prof_start = static_cast<cudaEvent_t>(ev_start);
  tl_prof_stop = static_cast<cudaEvent_t>(ev_stop);
  return TA_OK;
}

int tucker_attn_last_path(void) { return tl_last_path; }
int tucker_attn_last_launch_count(void) { return tl_last_launches; }

}  // extern "C"
