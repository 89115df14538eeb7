// Shape-generic FMA path: every step of the Tucker-attention forward as plain fp32 CUDA
// kernels, for fp32 storage (where tensor-core input rounding would break the 1e-4 bound)
// and for bf16 shapes the tensor-core kernels do not cover.  Intermediates are fp32.
//
// Steps follow Sec. 3 of the paper: latent projections (Sec. 3.1), head-mode core
// contraction and per-head queries (Definition 2), latent RoPE (Eq. 12), online-softmax
// attention with one shared latent K/V pair for all heads (Sec. 3.3), output-side factors
// (Eqs. 5-6), and the cached decode step (Eq. 9).
#include "ta_common.cuh"
#include "ta_gemm_fma.cuh"

namespace ta {
namespace {

using namespace fma;

// ---------------------------------------------------------------------------------------
// G[h,b,c] = mult * sum_a U1[h,a] C[a,b,c]   (C x_1 U1).  Output element (h,b,c) is stored at
// h*sh + b*sb + c (fp32), which lets the caller pick [h][b][c] or [b][h][c].
// ---------------------------------------------------------------------------------------
template <typename T>
__global__ void k_head_core(const T* __restrict__ C, const T* __restrict__ U1, float* __restrict__ G,
                            int nH, int r1, int rb, int rc, long sh, long sb, float mult) {
  long total = (long)nH * rb * rc;
  for (long i = blockIdx.x * (long)blockDim.x + threadIdx.x; i < total; i += (long)gridDim.x * blockDim.x) {
    int c = (int)(i % rc);
    int b = (int)((i / rc) % rb);
    int h = (int)(i / ((long)rc * rb));
    float acc = 0.f;
    for (int a = 0; a < r1; ++a) acc = fmaf(ld(U1 + (long)h * r1 + a), ld(C + ((long)a * rb + b) * rc + c), acc);
    G[h * sh + b * sb + c] = acc * mult;
  }
}

// ---------------------------------------------------------------------------------------
// RoPE.  Angles are formed in double precision (position * base^(-2i/r)) so that positions
// of tens of thousands keep full fp32 accuracy in cos / sin.
// ---------------------------------------------------------------------------------------
__global__ void k_rope_table(float2* __restrict__ tab, int n_pos, int half, int r, int pos0, double base) {
  long total = (long)n_pos * half;
  for (long i = blockIdx.x * (long)blockDim.x + threadIdx.x; i < total; i += (long)gridDim.x * blockDim.x) {
    int c = (int)(i % half);
    int n = (int)(i / half);
    double theta = pow(base, -2.0 * (double)c / (double)r);
    double s, co;
    sincos((double)(pos0 + n) * theta, &s, &co);
    tab[i] = make_float2((float)co, (float)s);
  }
}

// rows: [outer][n_pos][r] fp32, rotated in place; row position index = (row % n_pos).
__global__ void k_rope_apply(float* __restrict__ x, const float2* __restrict__ tab, long rows, int n_pos, int half) {
  long total = rows * half;
  for (long i = blockIdx.x * (long)blockDim.x + threadIdx.x; i < total; i += (long)gridDim.x * blockDim.x) {
    int c = (int)(i % half);
    long row = i / half;
    int n = (int)(row % n_pos);
    float2 cs = tab[(long)n * half + c];
    float* px = x + row * 2 * half + 2 * c;
    float xe = px[0], xo = px[1];
    px[0] = xe * cs.x - xo * cs.y;
    px[1] = xe * cs.y + xo * cs.x;
  }
}

// Decode: rotate the new key and every head's query at position cache_len[b]; store the
// new key / value (fp32 copies for the attention kernel, storage type into the cache when
// appending); flag cache lengths outside [0, Lmax).
template <typename T>
__global__ void k_decode_rope_append(float* __restrict__ knew, const float* __restrict__ vnew,
                                     float* __restrict__ qhat, T* __restrict__ Kc, T* __restrict__ Vc,
                                     const int32_t* __restrict__ cache_len, int B, int nH, int r3, int t3, int Lmax,
                                     int rope, double base, int append, int shared_rope, unsigned int* err) {
  const int b = blockIdx.x;
  int L = cache_len[b];
  if (L < 0 || L >= Lmax) {
    if (threadIdx.x == 0) atomicOr(err, (unsigned)TA_DEVERR_BAD_CACHE_LEN);
    L = L < 0 ? 0 : Lmax - 1;
  }
  if (rope) {
    const int half = r3 / 2;
    for (int i = threadIdx.x; i < half * (nH + 1); i += blockDim.x) {
      int c = i % half, which = i / half;             // which == nH -> the key row
      double theta = pow(base, -2.0 * (double)c / (double)r3);
      double s, co;
      sincos((double)L * theta, &s, &co);
      float* px = (which == nH ? knew + (long)b * r3 : qhat + ((long)b * nH + which) * r3) + 2 * c;
      float xe = px[0], xo = px[1];
      px[0] = xe * (float)co - xo * (float)s;
      px[1] = xe * (float)s + xo * (float)co;
    }
  }
  if (append) {
    __syncthreads();
    // one shared cache with latent RoPE holds un-rotated rows: the value row only
    if (!shared_rope)
      for (int c = threadIdx.x; c < r3; c += blockDim.x) st(Kc + ((long)b * Lmax + L) * r3 + c, knew[(long)b * r3 + c]);
    for (int c = threadIdx.x; c < t3; c += blockDim.x) st(Vc + ((long)b * Lmax + L) * t3 + c, vnew[(long)b * t3 + c]);
  }
}

// ---------------------------------------------------------------------------------------
// Online-softmax attention, one warp per query vector, 8 query vectors per block sharing
// each 32-key tile of the single latent K/V pair through shared memory.
//   prefill: block = 8 consecutive rows of one (b, h)
//   decode : block = 8 heads of one sequence b, keys = cache rows + the new token
// ---------------------------------------------------------------------------------------
constexpr int kMaxVRegs = 16;  // t3 <= 32 * kMaxVRegs

struct WarpState {
  float m, l;
  float o[kMaxVRegs];
};

// One 32-key tile for one warp.  `limit` = number of visible keys for this warp's query.
__device__ __forceinline__ void attend_tile(WarpState& st, const float* __restrict__ q, const float* __restrict__ Ks,
                                            const float* __restrict__ Vs, int k0, int limit, int r3, int t3,
                                            int lane) {
  float s = 0.f;
  const float* kr = Ks + lane * (r3 + 1);
  for (int c = 0; c < r3; ++c) s = fmaf(q[c], kr[c], s);
  const bool vis = (k0 + lane) < limit;
  s = vis ? s : -INFINITY;
  float tmax = s;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
  const float m_new = fmaxf(st.m, tmax);
  if (m_new == -INFINITY) return;  // nothing visible yet (warp-uniform)
  const float p = vis ? expf(s - m_new) : 0.f;
  const float corr = expf(st.m - m_new);  // exp(-inf) = 0 on the first visible tile
  float psum = p;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, o);
  st.l = st.l * corr + psum;
  st.m = m_new;
#pragma unroll
  for (int i = 0; i < kMaxVRegs; ++i) st.o[i] *= corr;
  for (int j = 0; j < 32; ++j) {
    const float pj = __shfl_sync(0xffffffffu, p, j);
    if (pj != 0.f) {
#pragma unroll
      for (int i = 0; i < kMaxVRegs; ++i) {
        int c = lane + 32 * i;
        if (c < t3) st.o[i] = fmaf(pj, Vs[j * t3 + c], st.o[i]);
      }
    }
  }
}

// Element (b, h, row, c) of Qhat is at b*q_b + h*q_h + row*q_n + c; K / V rows (b, n) start at
// b*kv_b + n*r3 (n*t3); O element (b, row, h, c) is at ((b*N + row)*nH + h)*t3 + c.
template <typename TI, typename TO>
__global__ void __launch_bounds__(256) k_attn_prefill_generic(const TI* __restrict__ Qhat, long q_b, long q_h, long q_n,
                                                              const TI* __restrict__ K, const TI* __restrict__ V,
                                                              long k_b, long v_b, TO* __restrict__ O, int N, int nH,
                                                              int r3, int t3, int causal) {
  extern __shared__ float smem[];
  float* qs = smem;                      // [8][r3]
  float* Ks = qs + 8 * r3;               // [32][r3+1]
  float* Vs = Ks + 32 * (r3 + 1);        // [32][t3]
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int row0 = blockIdx.x * 8, h = blockIdx.y, b = blockIdx.z;
  const int row = row0 + warp;
  const bool valid = row < N;
  const TI* qg = Qhat + (long)b * q_b + (long)h * q_h;
  for (int i = threadIdx.x; i < 8 * r3; i += 256) {
    int rr = i / r3, c = i % r3;
    qs[i] = (row0 + rr < N) ? ld(qg + (long)(row0 + rr) * q_n + c) : 0.f;
  }
  WarpState stt;
  stt.m = -INFINITY; stt.l = 0.f;
#pragma unroll
  for (int i = 0; i < kMaxVRegs; ++i) stt.o[i] = 0.f;
  const int kend = causal ? min(N, row0 + 8) : N;
  const int limit = causal ? min(row + 1, N) : N;
  const TI* Kb = K + (long)b * k_b;
  const TI* Vb = V + (long)b * v_b;
  for (int k0 = 0; k0 < kend; k0 += 32) {
    __syncthreads();
    for (int i = threadIdx.x; i < 32 * r3; i += 256) {
      int j = i / r3, c = i % r3;
      Ks[j * (r3 + 1) + c] = (k0 + j < N) ? ld(Kb + (long)(k0 + j) * r3 + c) : 0.f;
    }
    for (int i = threadIdx.x; i < 32 * t3; i += 256) {
      int j = i / t3;
      Vs[i] = (k0 + j < N) ? ld(Vb + (long)k0 * t3 + i) : 0.f;
    }
    __syncthreads();
    if (valid && k0 < limit) attend_tile(stt, qs + warp * r3, Ks, Vs, k0, limit, r3, t3, lane);
  }
  if (valid) {
    const float inv = 1.f / stt.l;
    TO* og = O + (((long)b * N + row) * nH + h) * t3;
#pragma unroll
    for (int i = 0; i < kMaxVRegs; ++i) {
      int c = lane + 32 * i;
      if (c < t3) st(og + c, stt.o[i] * inv);
    }
  }
}

template <typename T>
__global__ void __launch_bounds__(256) k_attn_decode_generic(const float* __restrict__ qhat,
                                                             const float* __restrict__ knew,
                                                             const float* __restrict__ vnew,
                                                             const T* __restrict__ Kc, const T* __restrict__ Vc,
                                                             const int32_t* __restrict__ cache_len,
                                                             float* __restrict__ o, int nH, int r3, int t3,
                                                             int Lmax, int rotate_keys, double base) {
  extern __shared__ float smem[];
  float* qs = smem;
  float* Ks = qs + 8 * r3;
  float* Vs = Ks + 32 * (r3 + 1);
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int h0 = blockIdx.x * 8, b = blockIdx.y;
  const int h = h0 + warp;
  const bool valid = h < nH;
  int L = cache_len[b];
  L = L < 0 ? 0 : (L >= Lmax ? Lmax - 1 : L);
  const float* qg = qhat + ((long)b * nH + h0) * r3;
  for (int i = threadIdx.x; i < 8 * r3; i += 256) qs[i] = (h0 + i / r3 < nH) ? qg[i] : 0.f;
  WarpState stt;
  stt.m = -INFINITY; stt.l = 0.f;
#pragma unroll
  for (int i = 0; i < kMaxVRegs; ++i) stt.o[i] = 0.f;
  const int limit = L + 1;  // cached keys 0..L-1 and the new token at index L
  const T* Kb = Kc + (long)b * Lmax * r3;
  const T* Vb = Vc + (long)b * Lmax * t3;
  for (int k0 = 0; k0 < limit; k0 += 32) {
    __syncthreads();
    for (int i = threadIdx.x; i < 32 * r3; i += 256) {
      int j = i / r3, c = i % r3;
      int kj = k0 + j;
      float v = 0.f;
      if (kj < L) {
        v = ld(Kb + (long)kj * r3 + c);
        if (rotate_keys) {
          // shared cache with latent RoPE: the cached row is un-rotated; its key is the row times R(kj, r3)
          const float other = ld(Kb + (long)kj * r3 + (c ^ 1));
          double sn, co;
          sincos((double)kj * pow(base, -2.0 * (double)(c >> 1) / (double)r3), &sn, &co);
          v = (c & 1) ? other * (float)sn + v * (float)co : v * (float)co - other * (float)sn;
        }
      } else if (kj == L) v = knew[(long)b * r3 + c];
      Ks[j * (r3 + 1) + c] = v;
    }
    for (int i = threadIdx.x; i < 32 * t3; i += 256) {
      int j = i / t3, c = i % t3;
      int kj = k0 + j;
      float v = 0.f;
      if (kj < L) v = ld(Vb + (long)kj * t3 + c);
      else if (kj == L) v = vnew[(long)b * t3 + c];
      Vs[i] = v;
    }
    __syncthreads();
    if (valid) attend_tile(stt, qs + warp * r3, Ks, Vs, k0, limit, r3, t3, lane);
  }
  if (valid) {
    const float inv = 1.f / stt.l;
    float* og = o + ((long)b * nH + h) * t3;
#pragma unroll
    for (int i = 0; i < kMaxVRegs; ++i) {
      int c = lane + 32 * i;
      if (c < t3) og[c] = stt.o[i] * inv;
    }
  }
}

// Copy fp32 latent K / V rows into the caller's cache (storage type T).
template <typename T>
__global__ void k_write_cache(const float* __restrict__ src, T* __restrict__ dst, int B, int N, int r, int Lmax) {
  long total = (long)B * N * r;
  for (long i = blockIdx.x * (long)blockDim.x + threadIdx.x; i < total; i += (long)gridDim.x * blockDim.x) {
    int c = (int)(i % r);
    long row = i / r;
    int n = (int)(row % N), b = (int)(row / N);
    st(dst + ((long)b * Lmax + n) * r + c, src[i]);
  }
}

static int grid_for(long total, int block = 256) {
  long g = (total + block - 1) / block;
  if (g > 148L * 16) g = 148L * 16;
  if (g < 1) g = 1;
  return (int)g;
}

struct FwdWs {
  float2* rope;
  float *G, *Gt, *Qt, *K, *V, *Qhat, *O, *Z;
};

static size_t carve_fwd(const tucker_attn_desc& d, char* base, FwdWs* w) {
  Carver c(base);
  const size_t T = (size_t)d.B * d.N;
  FwdWs t;
  t.rope = c.take<float2>(d.rope ? (size_t)d.N * (d.r3 / 2) : 0);
  t.G = c.take<float>((size_t)d.n_H * d.r2 * d.r3);
  t.Gt = c.take<float>((size_t)d.n_H * d.t2 * d.t3);
  t.Qt = c.take<float>(T * d.r2);
  t.K = c.take<float>(T * d.r3);
  t.V = c.take<float>(T * d.t3);
  t.Qhat = c.take<float>(T * d.n_H * d.r3);
  t.O = c.take<float>(T * d.n_H * d.t3);
  t.Z = c.take<float>(T * d.t2);
  if (w) *w = t;
  return c.off;
}

struct DecWs {
  float *G, *Gt, *qt, *knew, *vnew, *qhat, *o, *z;
};

static size_t carve_dec(const tucker_attn_desc& d, char* base, DecWs* w) {
  Carver c(base);
  DecWs t;
  t.G = c.take<float>((size_t)d.n_H * d.r2 * d.r3);
  t.Gt = c.take<float>((size_t)d.n_H * d.t2 * d.t3);
  t.qt = c.take<float>((size_t)d.B * d.r2);
  t.knew = c.take<float>((size_t)d.B * d.r3);
  t.vnew = c.take<float>((size_t)d.B * d.t3);
  t.qhat = c.take<float>((size_t)d.B * d.n_H * d.r3);
  t.o = c.take<float>((size_t)d.B * d.n_H * d.t3);
  t.z = c.take<float>((size_t)d.B * d.t2);
  if (w) *w = t;
  return c.off;
}

static size_t attn_smem(int r3, int t3) { return sizeof(float) * (8 * (size_t)r3 + 32 * (size_t)(r3 + 1) + 32 * (size_t)t3); }

template <typename T>
int fwd_typed(Problem& p) {
  const tucker_attn_desc& d = p.d;
  FwdWs w;
  carve_fwd(d, p.ws, &w);
  const int T_ = d.B * d.N;
  const T* X = (const T*)p.X;
  // head-mode core contraction; the softmax scale is folded into G, Gt is stored [t2][n_H][t3]
  k_head_core<T><<<grid_for((long)d.n_H * d.r2 * d.r3), 256, 0, p.stream>>>(
      (const T*)p.C, (const T*)p.U1, w.G, d.n_H, d.r1, d.r2, d.r3, (long)d.r2 * d.r3, d.r3, p.scale);
  TA_LAUNCH_CHECK(p);
  k_head_core<T><<<grid_for((long)d.n_H * d.t2 * d.t3), 256, 0, p.stream>>>(
      (const T*)p.Ct, (const T*)p.Ut1, w.Gt, d.n_H, d.t1, d.t2, d.t3, d.t3, (long)d.n_H * d.t3, 1.f);
  TA_LAUNCH_CHECK(p);
  // latent projections
  int rc;
  if ((rc = gemm(p, X, (const T*)p.U2, w.Qt, plain(T_, d.r2, d.d_model, d.d_model, d.r2, 1, d.r2), 1))) return rc;
  if ((rc = gemm(p, X, (const T*)p.U3, w.K, plain(T_, d.r3, d.d_model, d.d_model, d.r3, 1, d.r3), 1))) return rc;
  if ((rc = gemm(p, X, (const T*)p.Ut3, w.V, plain(T_, d.t3, d.d_model, d.d_model, d.t3, 1, d.t3), 1))) return rc;
  // per-head queries Qhat[b,h] = Qt[b] G_h
  {
    GemmShape g = plain(d.N, d.r3, d.r2, d.r2, d.r3, 1, d.r3);
    g.Z2 = d.n_H;
    g.a1 = (long)d.N * d.r2; g.a2 = 0;
    g.b1 = 0; g.b2 = (long)d.r2 * d.r3;
    g.c1 = (long)d.n_H * d.N * d.r3; g.c2 = (long)d.N * d.r3;
    if ((rc = gemm(p, w.Qt, w.G, w.Qhat, g, d.B * d.n_H))) return rc;
  }
  if (d.rope) {
    const int half = d.r3 / 2;
    k_rope_table<<<grid_for((long)d.N * half), 256, 0, p.stream>>>(w.rope, d.N, half, d.r3, d.pos0, (double)d.rope_base);
    TA_LAUNCH_CHECK(p);
    k_rope_apply<<<grid_for((long)T_ * half), 256, 0, p.stream>>>(w.K, w.rope, (long)T_, d.N, half);
    TA_LAUNCH_CHECK(p);
    k_rope_apply<<<grid_for((long)T_ * d.n_H * half), 256, 0, p.stream>>>(w.Qhat, w.rope, (long)T_ * d.n_H, d.N, half);
    TA_LAUNCH_CHECK(p);
  }
  if (p.Kc) {
    if (!p.shared_rope) {     // one shared cache with latent RoPE holds the un-rotated rows, i.e. V below
      k_write_cache<T><<<grid_for((long)T_ * d.r3), 256, 0, p.stream>>>(w.K, (T*)p.Kc, d.B, d.N, d.r3, p.Lmax);
      TA_LAUNCH_CHECK(p);
    }
    k_write_cache<T><<<grid_for((long)T_ * d.t3), 256, 0, p.stream>>>(w.V, (T*)p.Vc, d.B, d.N, d.t3, p.Lmax);
    TA_LAUNCH_CHECK(p);
  }
  // attention
  {
    size_t smem = attn_smem(d.r3, d.t3);
    TA_CUDA_TRY(cudaFuncSetAttribute(k_attn_prefill_generic<float, float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    dim3 grid((d.N + 7) / 8, d.n_H, d.B);
    prof_begin(p);
    k_attn_prefill_generic<float, float><<<grid, 256, smem, p.stream>>>(
        w.Qhat, (long)d.n_H * d.N * d.r3, (long)d.N * d.r3, (long)d.r3, w.K, w.V, (long)d.N * d.r3, (long)d.N * d.t3,
        w.O, d.N, d.n_H, d.r3, d.t3, d.causal);
    prof_end(p);
    TA_LAUNCH_CHECK(p);
  }
  // Z = sum_h O_h Gt_h^T  as one GEMM over (h, c); Y = Z Ut2^T
  if ((rc = gemm(p, w.O, w.Gt, w.Z, plain(T_, d.t2, d.n_H * d.t3, (long)d.n_H * d.t3, 1, (long)d.n_H * d.t3, d.t2), 1))) return rc;
  if ((rc = gemm(p, w.Z, (const T*)p.Ut2, (T*)p.Y, plain(T_, d.d_model, d.t2, d.t2, 1, d.t2, d.d_model), 1))) return rc;
  return TA_OK;
}

template <typename T>
int decode_typed(Problem& p) {
  const tucker_attn_desc& d = p.d;
  DecWs w;
  carve_dec(d, p.ws, &w);
  const T* x = (const T*)p.X;
  k_head_core<T><<<grid_for((long)d.n_H * d.r2 * d.r3), 256, 0, p.stream>>>(
      (const T*)p.C, (const T*)p.U1, w.G, d.n_H, d.r1, d.r2, d.r3, (long)d.r2 * d.r3, d.r3, p.scale);
  TA_LAUNCH_CHECK(p);
  k_head_core<T><<<grid_for((long)d.n_H * d.t2 * d.t3), 256, 0, p.stream>>>(
      (const T*)p.Ct, (const T*)p.Ut1, w.Gt, d.n_H, d.t1, d.t2, d.t3, d.t3, (long)d.n_H * d.t3, 1.f);
  TA_LAUNCH_CHECK(p);
  int rc;
  if ((rc = gemm(p, x, (const T*)p.U2, w.qt, plain(d.B, d.r2, d.d_model, d.d_model, d.r2, 1, d.r2), 1))) return rc;
  if ((rc = gemm(p, x, (const T*)p.U3, w.knew, plain(d.B, d.r3, d.d_model, d.d_model, d.r3, 1, d.r3), 1))) return rc;
  if ((rc = gemm(p, x, (const T*)p.Ut3, w.vnew, plain(d.B, d.t3, d.d_model, d.d_model, d.t3, 1, d.t3), 1))) return rc;
  {
    // qhat[b,h,:] = qt[b] G_h : batch over h, rows = sequences
    GemmShape g = plain(d.B, d.r3, d.r2, d.r2, d.r3, 1, (long)d.n_H * d.r3);
    g.Z2 = d.n_H;
    g.b2 = (long)d.r2 * d.r3;
    g.c2 = d.r3;
    if ((rc = gemm(p, w.qt, w.G, w.qhat, g, d.n_H))) return rc;
  }
  k_decode_rope_append<T><<<d.B, 128, 0, p.stream>>>(w.knew, w.vnew, w.qhat, (T*)p.Kc, (T*)p.Vc, p.cache_len, d.B,
                                                    d.n_H, d.r3, d.t3, p.Lmax, d.rope, (double)d.rope_base,
                                                    p.append, p.shared_rope, p.dev_err);
  TA_LAUNCH_CHECK(p);
  {
    size_t smem = attn_smem(d.r3, d.t3);
    TA_CUDA_TRY(cudaFuncSetAttribute(k_attn_decode_generic<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    dim3 grid((d.n_H + 7) / 8, d.B);
    prof_begin(p);
    k_attn_decode_generic<T><<<grid, 256, smem, p.stream>>>(w.qhat, w.knew, w.vnew, (const T*)p.Kc, (const T*)p.Vc,
                                                            p.cache_len, w.o, d.n_H, d.r3, d.t3, p.Lmax, p.shared_rope,
                                                            (double)d.rope_base);
    prof_end(p);
    TA_LAUNCH_CHECK(p);
  }
  if ((rc = gemm(p, w.o, w.Gt, w.z, plain(d.B, d.t2, d.n_H * d.t3, (long)d.n_H * d.t3, 1, (long)d.n_H * d.t3, d.t2), 1))) return rc;
  if ((rc = gemm(p, w.z, (const T*)p.Ut2, (T*)p.Y, plain(d.B, d.d_model, d.t2, d.t2, 1, d.t2, d.d_model), 1))) return rc;
  return TA_OK;
}

}  // namespace

// Attention on bf16 latent tensors laid out token-major (Qhat [T, n_H, r3], O [T, n_H, t3]); used by the
// tensor-core path for shapes its attention kernel does not cover.
int simt_attention_bf16(Problem& p, const bf16* Qhat, const bf16* K, const bf16* V, bf16* O) {
  const tucker_attn_desc& d = p.d;
  if (d.t3 > 32 * kMaxVRegs || attn_smem(d.r3, d.t3) > 200 * 1024) return TA_ERR_UNSUPPORTED_SHAPE;
  size_t smem = attn_smem(d.r3, d.t3);
  TA_CUDA_TRY(cudaFuncSetAttribute(k_attn_prefill_generic<bf16, bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  dim3 grid((d.N + 7) / 8, d.n_H, d.B);
  prof_begin(p);
  k_attn_prefill_generic<bf16, bf16><<<grid, 256, smem, p.stream>>>(
      Qhat, (long)d.N * d.n_H * d.r3, (long)d.r3, (long)d.n_H * d.r3, K, V, (long)d.N * d.r3, (long)d.N * d.t3, O, d.N,
      d.n_H, d.r3, d.t3, d.causal);
  prof_end(p);
  TA_LAUNCH_CHECK(p);
  return TA_OK;
}

static bool generic_shape_ok(const tucker_attn_desc& d) {
  return d.t3 <= 32 * kMaxVRegs && attn_smem(d.r3, d.t3) <= 200 * 1024;
}

size_t generic_fwd_workspace(const tucker_attn_desc& d) {
  if (!generic_shape_ok(d)) return 0;
  return carve_fwd(d, nullptr, nullptr);
}

size_t generic_decode_workspace(const tucker_attn_desc& d, int32_t) {
  if (!generic_shape_ok(d)) return 0;
  return carve_dec(d, nullptr, nullptr);
}

int generic_fwd(Problem& p) {
  if (!generic_shape_ok(p.d)) return TA_ERR_UNSUPPORTED_SHAPE;
  return p.d.dtype == TA_DTYPE_F32 ? fwd_typed<float>(p) : fwd_typed<bf16>(p);
}

int generic_decode(Problem& p) {
  if (!generic_shape_ok(p.d)) return TA_ERR_UNSUPPORTED_SHAPE;
  return p.d.dtype == TA_DTYPE_F32 ? decode_typed<float>(p) : decode_typed<bf16>(p);
}

}  // namespace ta
