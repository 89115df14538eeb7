// HOSVD initialiser: MHA weights -> Tucker-attention weights (App. C.1 "MHA to Tucker Attention") and the
// per-mode singular spectra that Sec. 2.1 ("Informed Compression Across All Modes") reads the ranks from.
//
// For a 3-way tensor T [n1, n2, n3] (here n_H x d x d, fp32) and ranks (r1, r2, r3):
//   G_j   = Mat_j(T) Mat_j(T)^T                       Gram matrix of the mode-j unfolding
//   U_j   = the r_j leading eigenvectors of G_j       (= leading left singular vectors of Mat_j(T))
//   s_j   = sqrt(eigenvalues of G_j), descending      (= singular values of Mat_j(T))
//   core  = T x_1 U1^T x_2 U2^T x_3 U3^T
// The Gram matrices of the two d-sized modes are dense contractions over n_H d^2 d elements and run on the
// tensor cores: the unfolding is written once as bf16 "high" and "low" halves (x = hi + lo up to 2^-16),
// concatenated along K as [hi | hi | lo] against [hi | lo | hi], so that ONE bf16 GEMM with fp32
// accumulation yields hi hi^T + hi lo^T + lo hi^T, i.e. the fp32 Gram matrix to about 2^-16 relative.
// Shapes that the tensor-core GEMM does not tile (mode sizes not multiples of 64) take an fp32 FMA route.
// The head-mode Gram matrix (n_H x n_H, one long dot product per entry) is a two-pass fp32 reduction.
// Eigenvectors come from a one-sided Jacobi iteration (Hestenes) on G in fp32, one launch per round of
// disjoint row pairs, a fixed number of sweeps with a device-side early exit: no host synchronisation.
#include "ta_common.cuh"
#include "ta_gemm_fma.cuh"

#include <algorithm>

namespace ta {
namespace {

using namespace fma;

constexpr int kSweeps = 14;
constexpr float kJacobiTol = 1e-6f;
constexpr int kG1Blocks = 512;

// ---- unfoldings as bf16 hi / lo, concatenated along K ------------------------------------------------
// mode 2: rows j, K index (a, k):  A[j, s K0 + a n3 + k], K0 = n1 n3, s = 0..2
__global__ void k_unfold2_split(const float* __restrict__ T, bf16* __restrict__ A, bf16* __restrict__ B, int n1, int n2,
                                int n3) {
  const long total = (long)n1 * n2 * n3, K0 = (long)n1 * n3;
  for (long i = blockIdx.x * (long)blockDim.x + threadIdx.x; i < total; i += (long)gridDim.x * blockDim.x) {
    const int k = (int)(i % n3), j = (int)((i / n3) % n2), a = (int)(i / ((long)n3 * n2));
    const float x = T[i];
    const bf16 hi = __float2bfloat16_rn(x);
    const bf16 lo = __float2bfloat16_rn(x - __bfloat162float(hi));
    const long o = (long)j * 3 * K0 + (long)a * n3 + k;
    A[o] = hi; A[o + K0] = hi; A[o + 2 * K0] = lo;
    B[o] = hi; B[o + K0] = lo; B[o + 2 * K0] = hi;
  }
}
// mode 3: rows k, K index (a, j): a 32 x 32 tile of (j, k) is transposed through shared memory
__global__ void k_unfold3_split(const float* __restrict__ T, bf16* __restrict__ A, bf16* __restrict__ B, int n1, int n2,
                                int n3) {
  __shared__ float tile[32][33];
  const int a = blockIdx.z, j0 = blockIdx.y * 32, k0 = blockIdx.x * 32;
  const int tx = threadIdx.x % 32, ty = threadIdx.x / 32;      // 256 threads: 8 rows per pass
  for (int r = ty; r < 32; r += 8) {
    const int j = j0 + r, k = k0 + tx;
    tile[r][tx] = (j < n2 && k < n3) ? T[((long)a * n2 + j) * n3 + k] : 0.f;
  }
  __syncthreads();
  const long K0 = (long)n1 * n2;
  for (int r = ty; r < 32; r += 8) {
    const int k = k0 + r, j = j0 + tx;
    if (k < n3 && j < n2) {
      const float x = tile[tx][r];
      const bf16 hi = __float2bfloat16_rn(x);
      const bf16 lo = __float2bfloat16_rn(x - __bfloat162float(hi));
      const long o = (long)k * 3 * K0 + (long)a * n2 + j;
      A[o] = hi; A[o + K0] = hi; A[o + 2 * K0] = lo;
      B[o] = hi; B[o + K0] = lo; B[o + 2 * K0] = hi;
    }
  }
}

// G = sum of the split-K partials, made exactly symmetric
__global__ void k_reduce_sym(const float* __restrict__ part, int splits, long stride, int ld, float* __restrict__ G, int n) {
  const long total = (long)n * n;
  for (long i = blockIdx.x * (long)blockDim.x + threadIdx.x; i < total; i += (long)gridDim.x * blockDim.x) {
    const int r = (int)(i / n), c = (int)(i % n);
    float s1 = 0.f, s2 = 0.f;
    for (int s = 0; s < splits; ++s) {
      s1 += part[s * stride + (long)r * ld + c];
      s2 += part[s * stride + (long)c * ld + r];
    }
    G[i] = 0.5f * (s1 + s2);
  }
}

// ---- head-mode Gram matrix: G1[a, b] = <T[a], T[b]> over n2 n3 elements, n1 <= 64 -----------------------
// pass 1: block x accumulates its slice of the element range for all pairs (thread = pair); pass 2 sums the blocks
__global__ void __launch_bounds__(256) k_gram1_partial(const float* __restrict__ T, int n1, long len, float* __restrict__ part) {
  extern __shared__ float xs[];                       // [n1][64] slice
  const long chunk = (len + gridDim.x - 1) / gridDim.x;
  const long beg = (long)blockIdx.x * chunk, end = min(len, beg + chunk);
  const int npair = n1 * n1;
  float acc[16];                                      // pairs p = threadIdx.x + 256 u, u < 16 (n1 <= 64)
#pragma unroll
  for (int u = 0; u < 16; ++u) acc[u] = 0.f;
  for (long e0 = beg; e0 < end; e0 += 64) {
    __syncthreads();
    for (int i = threadIdx.x; i < n1 * 64; i += 256) {
      const int a = i / 64, e = i % 64;
      xs[i] = (e0 + e < end) ? T[(long)a * len + e0 + e] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int u = 0; u < 16; ++u) {
      const int pr = threadIdx.x + 256 * u;
      if (pr < npair) {
        const float* xa = xs + (pr / n1) * 64;
        const float* xb = xs + (pr % n1) * 64;
        float s = 0.f;
#pragma unroll 8
        for (int e = 0; e < 64; ++e) s = fmaf(xa[e], xb[e], s);
        acc[u] += s;
      }
    }
  }
#pragma unroll
  for (int u = 0; u < 16; ++u) {
    const int pr = threadIdx.x + 256 * u;
    if (pr < npair) part[(long)blockIdx.x * npair + pr] = acc[u];
  }
}
__global__ void k_gram1_reduce(const float* __restrict__ part, int nblocks, int npair, float* __restrict__ G) {
  const int pr = blockIdx.x * blockDim.x + threadIdx.x;
  if (pr >= npair) return;
  float s = 0.f;
  for (int b = 0; b < nblocks; ++b) s += part[(long)b * npair + pr];
  G[pr] = s;
}

// ---- one-sided Jacobi on a symmetric positive semi-definite matrix ------------------------------------
// Bt holds the columns of B = G V as rows, Vt the columns of V as rows; initially Bt = G, Vt = I.  One
// launch = one round of the round-robin ordering: n / 2 disjoint row pairs (p, q), one CTA each:
//   alpha = |b_p|^2, beta = |b_q|^2, gamma = <b_p, b_q>; rotate (b_p, b_q) and (v_p, v_q) so that gamma -> 0.
// At convergence the rows of Bt are orthogonal with norms = eigenvalues and the rows of Vt are the eigenvectors.
struct JacobiCtl {
  unsigned int offmax;     // max over the sweep of |gamma| / sqrt(alpha beta), as float bits (non-negative)
  int done;                // set once a sweep stayed below the tolerance: later launches return at once
};

__global__ void k_jacobi_init(const float* __restrict__ G, float* __restrict__ Bt, float* __restrict__ Vt, int n,
                              JacobiCtl* ctl) {
  const long total = (long)n * n;
  for (long i = blockIdx.x * (long)blockDim.x + threadIdx.x; i < total; i += (long)gridDim.x * blockDim.x) {
    Bt[i] = G[i];
    Vt[i] = (i / n == i % n) ? 1.f : 0.f;
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) { ctl->offmax = 0u; ctl->done = 0; }
}

__device__ __forceinline__ float block_sum_128(float v, float* red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  return red[0] + red[1] + red[2] + red[3];
}

__global__ void __launch_bounds__(128) k_jacobi_round(float* __restrict__ Bt, float* __restrict__ Vt, int n, int round,
                                                      JacobiCtl* ctl) {
  if (ctl->done) return;
  __shared__ float red[4];
  const int m = n + (n & 1);                     // even number of players; index n (if present) is a bye
  const int k = blockIdx.x;                      // pair index 0 .. m/2 - 1
  int p, q;
  if (k == 0) { p = round % (m - 1); q = m - 1; }
  else { p = (round + k) % (m - 1); q = (round - k + (m - 1)) % (m - 1); }
  if (p >= n || q >= n) return;
  if (p > q) { const int t = p; p = q; q = t; }
  float* bp = Bt + (long)p * n;
  float* bq = Bt + (long)q * n;
  float a = 0.f, b = 0.f, g = 0.f;
  for (int i = threadIdx.x; i < n; i += 128) {
    const float x = bp[i], y = bq[i];
    a = fmaf(x, x, a); b = fmaf(y, y, b); g = fmaf(x, y, g);
  }
  a = block_sum_128(a, red);
  b = block_sum_128(b, red);
  g = block_sum_128(g, red);
  const float denom = sqrtf(a) * sqrtf(b);
  if (!(denom > 0.f) || !(fabsf(g) > 1e-30f)) return;      // a zero row, or already orthogonal
  const float off = fabsf(g) / denom;
  if (threadIdx.x == 0) atomicMax(&ctl->offmax, __float_as_uint(off));
  if (off <= kJacobiTol * 0.1f) return;
  // rotation that orthogonalises the pair
  const float zeta = (b - a) / (2.f * g);
  const float t = (zeta >= 0.f ? 1.f : -1.f) / (fabsf(zeta) + sqrtf(1.f + zeta * zeta));
  const float c = rsqrtf(1.f + t * t), s = c * t;
  float* vp = Vt + (long)p * n;
  float* vq = Vt + (long)q * n;
  for (int i = threadIdx.x; i < n; i += 128) {
    const float x = bp[i], y = bq[i];
    bp[i] = c * x - s * y; bq[i] = s * x + c * y;
    const float u = vp[i], w = vq[i];
    vp[i] = c * u - s * w; vq[i] = s * u + c * w;
  }
}

__global__ void k_jacobi_sweep_end(JacobiCtl* ctl) {
  if (ctl->done) return;
  if (__uint_as_float(ctl->offmax) <= kJacobiTol) ctl->done = 1;
  ctl->offmax = 0u;
}

// eigenvalue of row i = |Bt row i|; rank by counting (descending, ties by index); spectrum = sqrt; the first r
// eigenvectors become the columns of U [n, r], each with its largest component made positive
__global__ void __launch_bounds__(128) k_row_norms(const float* __restrict__ Bt, int n, float* __restrict__ lam) {
  __shared__ float red[4];
  const float* b = Bt + (long)blockIdx.x * n;
  float a = 0.f;
  for (int i = threadIdx.x; i < n; i += 128) a = fmaf(b[i], b[i], a);
  a = block_sum_128(a, red);
  if (threadIdx.x == 0) lam[blockIdx.x] = sqrtf(a);
}
__global__ void k_rank_and_emit(const float* __restrict__ lam, const float* __restrict__ Vt, int n, int r,
                                float* __restrict__ U, float* __restrict__ spectrum) {
  const int i = blockIdx.x;                      // one block per eigenpair
  __shared__ int rank_s;
  __shared__ float sign_s;
  __shared__ float bestv[128];
  __shared__ int cnt[128];
  const float li = lam[i];
  int c = 0;
  for (int j = threadIdx.x; j < n; j += 128) {
    const float lj = lam[j];
    c += (lj > li || (lj == li && j < i)) ? 1 : 0;
  }
  cnt[threadIdx.x] = c;
  const float* v = Vt + (long)i * n;
  float best = 0.f;
  for (int j = threadIdx.x; j < n; j += 128)
    if (fabsf(v[j]) > fabsf(best)) best = v[j];
  bestv[threadIdx.x] = best;
  __syncthreads();
  if (threadIdx.x == 0) {
    int tot = 0;
    float bb = 0.f;
    for (int t = 0; t < 128; ++t) {
      tot += cnt[t];
      if (fabsf(bestv[t]) > fabsf(bb)) bb = bestv[t];
    }
    rank_s = tot;
    sign_s = bb < 0.f ? -1.f : 1.f;
    if (spectrum) spectrum[tot] = sqrtf(fmaxf(li, 0.f));
  }
  __syncthreads();
  const int rk = rank_s;
  if (rk < r)
    for (int j = threadIdx.x; j < n; j += 128) U[(long)j * r + rk] = sign_s * v[j];
}

// ---- workspace -------------------------------------------------------------------------------------------
struct HosvdWs {
  bf16 *A, *B;          // unfolding halves [n, 3 K0]
  float* part;          // split-K partials of a Gram GEMM / per-slice Gram matrices / head-mode partials
  float *G, *Bt, *Vt, *lam;
  float *Y1, *Y2;
  JacobiCtl* ctl;
};

int gram_splits(int n) {
  const int tiles = ((n + 127) / 128) * ((n + 127) / 128);
  int s = (148 + tiles - 1) / tiles;
  return s < 1 ? 1 : (s > 16 ? 16 : s);
}
bool tensor_route(int n1, int n2, int n3) { return n2 % 64 == 0 && n3 % 64 == 0 && n2 >= 64 && n3 >= 64 && n1 >= 1; }

size_t carve_hosvd(int n1, int n2, int n3, int r2, int r3, char* base, HosvdWs* w) {
  Carver c(base);
  HosvdWs t;
  const size_t elems = (size_t)n1 * n2 * n3;
  const int nmax = n2 > n3 ? n2 : n3;
  const bool tc = tensor_route(n1, n2, n3);
  t.A = c.take<bf16>(tc ? 3 * elems : 0);
  t.B = c.take<bf16>(tc ? 3 * elems : 0);
  size_t part = (size_t)kG1Blocks * n1 * n1;
  if (tc) part = std::max(part, (size_t)16 * ((nmax + 127) / 128 * 128) * nmax);
  else part = std::max(part, (size_t)n1 * nmax * nmax);
  t.part = c.take<float>(part);
  t.G = c.take<float>((size_t)nmax * nmax);
  t.Bt = c.take<float>((size_t)nmax * nmax);
  t.Vt = c.take<float>((size_t)nmax * nmax);
  t.lam = c.take<float>(nmax);
  t.Y1 = c.take<float>((size_t)n1 * n2 * r3);
  t.Y2 = c.take<float>((size_t)n1 * r2 * r3);
  t.ctl = c.take<JacobiCtl>(1);
  if (w) *w = t;
  return c.off;
}

int grid_for(long total, int block = 256) {
  long g = (total + block - 1) / block;
  if (g > 148L * 16) g = 148L * 16;
  return (int)(g < 1 ? 1 : g);
}

// eigenvectors / spectrum of the n x n Gram matrix in w.G -> U [n, r] and spectrum [n]
int eig_and_emit(Problem& p, HosvdWs& w, int n, int r, float* U, float* spectrum) {
  k_jacobi_init<<<grid_for((long)n * n), 256, 0, p.stream>>>(w.G, w.Bt, w.Vt, n, w.ctl);
  TA_LAUNCH_CHECK(p);
  const int m = n + (n & 1);
  if (n > 1)
    for (int sweep = 0; sweep < kSweeps; ++sweep) {
      for (int round = 0; round < m - 1; ++round) {
        k_jacobi_round<<<m / 2, 128, 0, p.stream>>>(w.Bt, w.Vt, n, round, w.ctl);
        TA_LAUNCH_CHECK(p);
      }
      k_jacobi_sweep_end<<<1, 1, 0, p.stream>>>(w.ctl);
      TA_LAUNCH_CHECK(p);
    }
  k_row_norms<<<n, 128, 0, p.stream>>>(w.Bt, n, w.lam);
  TA_LAUNCH_CHECK(p);
  k_rank_and_emit<<<n, 128, 0, p.stream>>>(w.lam, w.Vt, n, r, U, spectrum);
  TA_LAUNCH_CHECK(p);
  return TA_OK;
}

}  // namespace

int hosvd_run(Problem& p, int n1, int n2, int n3, int r1, int r2, int r3, const float* T, float* core, float* U1,
              float* U2, float* U3, float* spectra) {
  HosvdWs w;
  carve_hosvd(n1, n2, n3, r2, r3, p.ws, &w);
  const long elems = (long)n1 * n2 * n3;
  const bool tc = tensor_route(n1, n2, n3);
  int rc;
  // ---- mode 1 (heads): two-pass fp32 reduction ----
  {
    k_gram1_partial<<<kG1Blocks, 256, (size_t)n1 * 64 * sizeof(float), p.stream>>>(T, n1, (long)n2 * n3, w.part);
    TA_LAUNCH_CHECK(p);
    k_gram1_reduce<<<(n1 * n1 + 127) / 128, 128, 0, p.stream>>>(w.part, kG1Blocks, n1 * n1, w.G);
    TA_LAUNCH_CHECK(p);
    if ((rc = eig_and_emit(p, w, n1, r1, U1, spectra))) return rc;
  }
  // ---- modes 2 and 3 ----
  for (int mode = 2; mode <= 3; ++mode) {
    const int n = mode == 2 ? n2 : n3;
    float* U = mode == 2 ? U2 : U3;
    const int r = mode == 2 ? r2 : r3;
    float* spec = spectra ? spectra + n1 + (mode == 3 ? n2 : 0) : nullptr;
    if (tc) {
      const long K0 = mode == 2 ? (long)n1 * n3 : (long)n1 * n2;
      if (mode == 2) {
        k_unfold2_split<<<grid_for(elems), 256, 0, p.stream>>>(T, w.A, w.B, n1, n2, n3);
      } else {
        dim3 g((n3 + 31) / 32, (n2 + 31) / 32, n1);
        k_unfold3_split<<<g, 256, 0, p.stream>>>(T, w.A, w.B, n1, n2, n3);
      }
      TA_LAUNCH_CHECK(p);
      const int splits_want = gram_splits(n);
      int splits = 1;                      // a divisor of the K-block count, as close to the wish as possible
      const long nkb = 3 * K0 / 64;
      for (int s = splits_want; s >= 1; --s)
        if (nkb % s == 0) { splits = s; break; }
      const int Mpad = (n + 127) / 128 * 128;
      const long stride = (long)Mpad * n;
      prof_begin(p);
      rc = umma_gemm_f32_partials(p, w.A, 3 * K0, n, w.B, 3 * K0, n, (int)(3 * K0), splits, w.part, stride);
      prof_end(p);
      if (rc) return rc;
      k_reduce_sym<<<grid_for((long)n * n), 256, 0, p.stream>>>(w.part, splits, stride, n, w.G, n);
      TA_LAUNCH_CHECK(p);
    } else {
      // fp32 route: per-slice Gram matrices T[a] T[a]^T (mode 2) or T[a]^T T[a] (mode 3), then their sum
      GemmShape g;
      g.M = n; g.N = n; g.Z2 = 1;
      g.K = mode == 2 ? n3 : n2;
      if (mode == 2) { g.sam = n3; g.sak = 1; g.sbk = 1; g.sbn = n3; }
      else { g.sam = 1; g.sak = n3; g.sbk = n3; g.sbn = 1; }
      g.scm = n; g.scn = 1;
      g.a1 = (long)n2 * n3; g.a2 = 0; g.b1 = (long)n2 * n3; g.b2 = 0; g.c1 = (long)n * n; g.c2 = 0;
      if ((rc = gemm(p, T, T, w.part, g, n1))) return rc;
      k_reduce_sym<<<grid_for((long)n * n), 256, 0, p.stream>>>(w.part, n1, (long)n * n, n, w.G, n);
      TA_LAUNCH_CHECK(p);
    }
    if ((rc = eig_and_emit(p, w, n, r, U, spec))) return rc;
  }
  // ---- core = T x_3 U3^T x_2 U2^T x_1 U1^T ----
  // Y1[(a, j), c] = sum_k T[a, j, k] U3[k, c]
  if ((rc = gemm(p, T, U3, w.Y1, plain(n1 * n2, r3, n3, n3, r3, 1, r3), 1))) return rc;
  {
    // Y2[a][b, c] = sum_j U2[j, b] Y1[a][j, c]
    GemmShape g = plain(r2, r3, n2, 1, r3, 1, r3);
    g.sam = 1; g.sak = r2;                      // A = U2^T: element (b, j) at U2[j, b]
    g.b1 = (long)n2 * r3; g.c1 = (long)r2 * r3;
    if ((rc = gemm(p, U2, w.Y1, w.Y2, g, n1))) return rc;
  }
  {
    // core[alpha, (b, c)] = sum_a U1[a, alpha] Y2[a, (b, c)]
    GemmShape g = plain(r1, r2 * r3, n1, 1, (long)r2 * r3, 1, (long)r2 * r3);
    g.sam = 1; g.sak = r1;
    if ((rc = gemm(p, U1, w.Y2, core, g, 1))) return rc;
  }
  return TA_OK;
}

size_t hosvd_workspace(int n1, int n2, int n3, int r2, int r3) { return carve_hosvd(n1, n2, n3, r2, r3, nullptr, nullptr); }

// W[i] = WQ_i WK_i^T  [d, d];  Wt[i] = (WV_i WO_i)^T, i.e. Wt[i][o, v] = sum_l WO[i d_H + l, o] WV[v, i d_H + l]
int mha_weight_tensors_run(Problem& p, int d, int nH, const float* WQ, const float* WK, const float* WV, const float* WO,
                           float* W, float* Wt) {
  const int dH = d / nH;
  int rc;
  GemmShape g;
  g.M = d; g.N = d; g.K = dH; g.Z2 = 1;
  g.sam = d; g.sak = 1;          // A = WQ[:, i dH + l]
  g.sbk = 1; g.sbn = d;          // B[l, k] = WK[k, i dH + l]
  g.scm = d; g.scn = 1;
  g.a1 = dH; g.a2 = 0; g.b1 = dH; g.b2 = 0; g.c1 = (long)d * d; g.c2 = 0;
  if ((rc = gemm(p, WQ, WK, W, g, nH))) return rc;
  g.sam = 1; g.sak = d;          // A[o, l] = WO[i dH + l, o]
  g.sbk = 1; g.sbn = d;          // B[l, v] = WV[v, i dH + l]
  g.a1 = (long)dH * d; g.b1 = dH;
  if ((rc = gemm(p, WO, WV, Wt, g, nH))) return rc;
  return TA_OK;
}

}  // namespace ta
