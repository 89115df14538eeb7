// Decode step over the latent KV cache (Eq. 9, "KV Caching"): the per-sequence kernels of the bf16 path --
// the query kernel k_dec_qhat and the output kernel k_dec_out -- and what they share with the
// cache-streaming kernel (ta_decode_umma.cuh): the tile split, the RoPE angle helpers, the partial format.
//
// The cache is cut into tiles of 128 keys; the flat list of tiles of all sequences is divided evenly
// over the CTAs of the streaming kernel (one per SM), so that the load is balanced for any mix of
// cache lengths.  Each of those CTAs keeps an online-softmax state per sequence segment and writes one
// partial (max, sum, unnormalised O for all heads) per segment; k_dec_out combines the partials of a
// sequence with log-sum-exp weights and applies the output-side core (Z = sum_h o_h Gt_h^T).
#pragma once

#include "ta_common.cuh"
#include "ta_sm100.cuh"

namespace ta {
namespace dec {

using namespace sm100;

constexpr int TK = 128;                 // keys per tile
constexpr int MAX_GRID = 160;           // partial weights table in the merge kernel

struct Params {
  int B, nH, Lmax, grid;
  int shared_kv;       // 1: the value cache IS the key cache (one latent cache L^KV, Sec. 3.1): each tile is loaded once
  const int32_t* cache_len;
  const bf16* qhat;    // [B, nH, R3] rotated, scaled by softmax scale * log2 e
  const bf16* knew;    // [B, R3] rotated new key
  const bf16* vnew;    // [B, T3] new value
  float* part_o;       // [grid + B][32][T3]
  float* part_ml;      // [grid + B][32][2]  (max in log2 units, sum)
  unsigned int* err;
};

__device__ __forceinline__ int clamp_len(int L, int Lmax) { return L < 0 ? 0 : (L >= Lmax ? Lmax - 1 : L); }
__device__ __forceinline__ int tiles_of(int L) { return L / TK + 1; }   // keys 0..L inclusive (L = the new token)

// First global tile of CTA i when `total` tiles are split over `grid` CTAs.
__device__ __forceinline__ long cta_first_tile(long i, long total, long grid) { return i * total / grid; }

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Block-wide scan over the tile counts of all sequences.  Thread t owns the sequences
// [lo, hi) = [t * chunk, (t + 1) * chunk); returns the total number of tiles and sets `excl` to the
// number of tiles before sequence `lo`.  wtot_s needs one slot per warp of the block; contains a
// __syncthreads.
__device__ __forceinline__ long block_tile_scan(const int32_t* __restrict__ cache_len, int B, int Lmax, int& lo,
                                                int& hi, long& excl, long long* wtot_s) {
  const int nthr = blockDim.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, nwarp = (nthr + 31) >> 5;
  const int chunk = (B + nthr - 1) / nthr;
  lo = min(B, tid * chunk);
  hi = min(B, lo + chunk);
  long long cnt = 0;
  for (int b = lo; b < hi; ++b) cnt += tiles_of(clamp_len(cache_len[b], Lmax));
  long long incl = cnt;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const long long v = __shfl_up_sync(0xffffffffu, incl, off);
    if (lane >= off) incl += v;
  }
  if (lane == 31) wtot_s[wid] = incl;
  __syncthreads();
  long long before = 0, total = 0;
  for (int w = 0; w < nwarp; ++w) {
    const long long v = wtot_s[w];
    if (w < wid) before += v;
    total += v;
  }
  excl = (long)(before + incl - cnt);
  return (long)total;
}

// (cos, sin) of pos * theta for a rotation frequency theta given in double precision: the angle is
// reduced to a fraction of a turn in double (positions of tens of thousands would lose ~1e-3 rad
// in fp32) and only then handed to the fp32 sincospi.
__device__ __forceinline__ float2 rope_cos_sin_theta(int pos, double theta) {
  double turns = (double)pos * theta * 0.15915494309189535;   // angle / (2 pi)
  turns -= rint(turns);
  float sn, co;
  sincospif((float)(2.0 * turns), &sn, &co);
  return make_float2(co, sn);
}

// Rotation frequencies theta_i = base^(-2 i / r), i < r / 2 <= 128, computed on the host in double
// precision and passed to the kernels by value.
struct RopeFreqs {
  double theta[128];
};

// (cos, sin) of pos * base^(-2 i / r).  The angle is formed in double precision (positions of
// tens of thousands would lose ~1e-3 rad in fp32), reduced to a fraction of a turn in double,
// and only then handed to the fp32 sincospi.  log2_base = log2(base).
__device__ __forceinline__ float2 rope_cos_sin(int pos, int i, int r, double log2_base) {
  const double theta = exp2(-2.0 * (double)i / (double)r * log2_base);
  double turns = (double)pos * theta * 0.15915494309189535;   // angle / (2 pi)
  turns -= rint(turns);
  float sn, co;
  sincospif((float)(2.0 * turns), &sn, &co);
  return make_float2(co, sn);
}

// ---------------------------------------------------------------------------------------
// k_dec_qhat: grid (B, r3 / 32), 256 threads.  CTA (b, y) finishes the new token's latent
// projections and forms its per-head queries for the 32 latent key coordinates
// [32 y, 32 y + 32):
//   row      = sum over the split-K partials of [qt | k | v]            (fp32)
//   k, v     -> latent RoPE on k at position L = cache_len[b]; bf16 copies for the attention
//               kernel; appended to the caches at slot L when `append`
//   w[a, c]  = sum_q qt[q] C[a, q, c]         (the core contracted with the query first:
//   qhat_h   = mult * sum_a U1[h, a] w[a, :]   C x_2 qt x_1 U1, Eq. 9, so that the n_H
//                                              per-head matrices G_h are never formed)
//   qhat_h  <- qhat_h R(L, r3), stored bf16 [B, nH, r3]
// The core is read with 16-byte loads that are all issued before anything waits on them:
// warp w, lane (rg = lane / 4, ch = lane % 4) owns chunk ch of the CTA's 64-byte column range
// in the core rows q = 8 w + rg + 64 i, for AB = 8 / NQ slices a at a time (NQ = ceil(r2/64)).
// part: [splits][Mpad][r2 + r3 + t3] fp32.
// ---------------------------------------------------------------------------------------
constexpr int DQ_CW = 32;       // latent key coordinates per CTA
constexpr int DQ_MAX_R1 = 32;   // head ranks r1, t1 supported by the shared-memory tables
constexpr int DQ_MAX_R2 = 256;

template <int NQ>
__global__ void __launch_bounds__(256, 2)
k_dec_qhat(const float* __restrict__ part, int splits, long split_stride, int nH, int r1, int r2, int r3, int t3,
           const bf16* __restrict__ C, const bf16* __restrict__ U1, float mult, bf16* __restrict__ qhat,
           bf16* __restrict__ knew, bf16* __restrict__ vnew, bf16* __restrict__ Kc, bf16* __restrict__ Vc, int Lmax,
           const int32_t* __restrict__ cache_len, int rope, const RopeFreqs freqs, int append, int shared_kv,
           unsigned int* err) {
  constexpr int AB = 8 / NQ;                        // core slices per batch (8 loads of 16 bytes in flight per thread)
  __shared__ float qt_s[DQ_MAX_R2];                 // latent query of the new token
  __shared__ float k_s[DQ_CW];                      // this CTA's coordinates of the new key (unrotated)
  __shared__ float2 cs_s[DQ_CW / 2];                // (cos, sin) at position L for this CTA's pairs
  __shared__ float u1_s[32 * DQ_MAX_R1];            // U1 as fp32
  __shared__ float w_s[DQ_MAX_R1][DQ_CW];
  __shared__ float red_s[8][AB][DQ_CW];
  const int b = blockIdx.x, c0 = blockIdx.y * DQ_CW;
  const int ncol = r2 + r3 + t3;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int rg = lane / 4, ch = lane % 4;
  const uint4* Cq = reinterpret_cast<const uint4*>(C);
  const int nch = r3 / 8;                           // 16-byte chunks per core row
  const int chunk = c0 / 8 + ch;

  auto load_batch = [&](int a0, uint4 (&v)[AB * NQ]) {
#pragma unroll
    for (int u = 0; u < AB * NQ; ++u) {
      const int a = a0 + u / NQ, q = warp * 8 + rg + 64 * (u % NQ);
      v[u] = (a < r1 && q < r2) ? Cq[((long)a * r2 + q) * nch + chunk] : make_uint4(0u, 0u, 0u, 0u);
    }
  };
  uint4 v[AB * NQ];
  load_batch(0, v);                                 // in flight while the projections are finished

  int L = cache_len[b];
  if (L < 0 || L >= Lmax) {
    if (threadIdx.x == 0 && blockIdx.y == 0) atomicOr(err, (unsigned)TA_DEVERR_BAD_CACHE_LEN);
    L = clamp_len(L, Lmax);
  }
  // Everything above and the two tables below depend on the call's inputs only (core, U1, cache_len)
  // and runs while the projection GEMM before this kernel finishes; its partial sums are read after
  // pdl_enter(), and nothing is written before it.
  for (int i = threadIdx.x; i < nH * r1; i += blockDim.x) u1_s[i] = __bfloat162float(U1[i]);
  if (threadIdx.x < DQ_CW / 2) {
    cs_s[threadIdx.x] = rope ? rope_cos_sin_theta(L, freqs.theta[c0 / 2 + threadIdx.x]) : make_float2(1.f, 0.f);
  }
  pdl_enter();
  // split-K sums: all of qt, this CTA's 32 key coordinates, and the value coordinates c with
  // (c / 32) % gridDim.y == blockIdx.y
  const float* prow = part + (long)b * ncol;
  [[maybe_unused]] const int nB = gridDim.x;         // sequences
  // the split-K partials are [splits][rows padded to 128][ncol]: this sequence's row must lie in every split
  const bool prow_ok = TA_IDX_OK(err, (long)b * ncol, ncol, split_stride) &&
                       TA_IDX_OK(err, (long)(splits - 1) * split_stride + (long)b * ncol, ncol, (long)splits * split_stride);
  for (int c = threadIdx.x; c < r2 + DQ_CW; c += blockDim.x) {
    const int col = c < r2 ? c : r2 + c0 + (c - r2);
    float acc = 0.f;
    if (prow_ok) for (int s = 0; s < splits; ++s) acc += prow[s * split_stride + col];
    if (c < r2) qt_s[c] = acc; else k_s[c - r2] = acc;
  }
  for (int c = threadIdx.x; c < t3; c += blockDim.x) {
    if ((c / DQ_CW) % gridDim.y != blockIdx.y) continue;
    float acc = 0.f;
    if (prow_ok) for (int s = 0; s < splits; ++s) acc += prow[s * split_stride + r2 + r3 + c];
    const bf16 vv = __float2bfloat16_rn(acc);
    if (TA_IDX_OK(err, (long)b * t3 + c, 1, (long)nB * t3)) vnew[(long)b * t3 + c] = vv;
    // shared_kv == 1 (one cache, no RoPE): the key row written below is the value row; == 2 (one cache with
    // latent RoPE): the cache holds un-rotated rows, i.e. this value row, and the rotated key is not stored
    if (append && shared_kv != 1 && TA_IDX_OK(err, ((long)b * Lmax + L) * t3 + c, 1, (long)nB * Lmax * t3))
      Vc[((long)b * Lmax + L) * t3 + c] = vv;   // shared cache: the key row written below is the value row
  }
  __syncthreads();
  if (threadIdx.x < DQ_CW / 2) {                    // new key, rotated
    const int i = threadIdx.x;
    const float xe = k_s[2 * i], xo = k_s[2 * i + 1];
    const float2 cs = cs_s[i];
    const __nv_bfloat162 kv = __floats2bfloat162_rn(xe * cs.x - xo * cs.y, xe * cs.y + xo * cs.x);
    if (TA_IDX_OK(err, (long)b * r3 + c0 + 2 * i, 2, (long)nB * r3))
      *reinterpret_cast<__nv_bfloat162*>(knew + (long)b * r3 + c0 + 2 * i) = kv;
    if (append && shared_kv != 2 && TA_IDX_OK(err, ((long)b * Lmax + L) * r3 + c0 + 2 * i, 2, (long)nB * Lmax * r3))
      *reinterpret_cast<__nv_bfloat162*>(Kc + ((long)b * Lmax + L) * r3 + c0 + 2 * i) = kv;
  }
  // ---- w[a, c0 + .] for batches of AB slices ----
  for (int a0 = 0; a0 < r1; a0 += AB) {
    float acc[AB][8];
#pragma unroll
    for (int j = 0; j < AB; ++j)
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[j][e] = 0.f;
#pragma unroll
    for (int u = 0; u < AB * NQ; ++u) {
      const int q = warp * 8 + rg + 64 * (u % NQ);
      const float xq = q < r2 ? qt_s[q] : 0.f;
      const uint32_t wv[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 cv = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&wv[e]));
        acc[u / NQ][2 * e] = fmaf(xq, cv.x, acc[u / NQ][2 * e]);
        acc[u / NQ][2 * e + 1] = fmaf(xq, cv.y, acc[u / NQ][2 * e + 1]);
      }
    }
    if (a0 + AB < r1) load_batch(a0 + AB, v);       // next batch in flight during the reduction
#pragma unroll
    for (int j = 0; j < AB; ++j)
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        float t = acc[j][e];
        t += __shfl_xor_sync(0xffffffffu, t, 4);
        t += __shfl_xor_sync(0xffffffffu, t, 8);
        t += __shfl_xor_sync(0xffffffffu, t, 16);
        if (rg == 0) red_s[warp][j][ch * 8 + e] = t;
      }
    __syncthreads();
    for (int i = threadIdx.x; i < AB * DQ_CW; i += blockDim.x) {
      const int j = i / DQ_CW, c = i % DQ_CW;
      if (a0 + j < r1) {
        float t = 0.f;
#pragma unroll
        for (int w8 = 0; w8 < 8; ++w8) t += red_s[w8][j][c];
        w_s[a0 + j][c] = t;
      }
    }
    __syncthreads();
  }
  // ---- qhat_h for this CTA's coordinates ----
  for (int item = threadIdx.x; item < nH * (DQ_CW / 2); item += blockDim.x) {
    const int h = item / (DQ_CW / 2), cp = item % (DQ_CW / 2);
    float xe = 0.f, xo = 0.f;
    for (int a = 0; a < r1; ++a) {
      const float u = u1_s[h * r1 + a];
      xe = fmaf(u, w_s[a][2 * cp], xe);
      xo = fmaf(u, w_s[a][2 * cp + 1], xo);
    }
    xe *= mult; xo *= mult;
    const float2 cs = cs_s[cp];
    if (TA_IDX_OK(err, ((long)b * nH + h) * r3 + c0 + 2 * cp, 2, (long)nB * nH * r3))
      *reinterpret_cast<__nv_bfloat162*>(qhat + ((long)b * nH + h) * r3 + c0 + 2 * cp) =
          __floats2bfloat162_rn(xe * cs.x - xo * cs.y, xe * cs.y + xo * cs.x);
  }
}

// ---------------------------------------------------------------------------------------
// k_dec_out: grid (B, DO_JS), 256 threads.  Every CTA of a sequence merges the partials of
// the attention CTAs whose tile range intersected the sequence (log-sum-exp weights), then
// applies the output-side core with the head mode contracted first (the n_H matrices Gt_h are
// never formed), for its share of the t2 output coordinates:
//   o_h      = merged, normalised attention output of head h             [nH][t3]
//   u[a, :]  = sum_h Ut1[h, a] o_h                                       [t1][t3]
//   z[j]     = sum_a sum_c Ct[a, j, c] u[a, c]                           (= sum_h Gt_h o_h)
// z is written as bf16 [B, t2].  Dynamic shared memory: see dec_out_smem().
// ---------------------------------------------------------------------------------------
constexpr int DO_JS = 4;        // CTAs per sequence (t2 is a multiple of 32, so each gets >= 8 rows)

__host__ __device__ inline size_t dec_out_smem(int nH, int t1, int t3) {
  return sizeof(float) * (32 * (size_t)t3 + (size_t)MAX_GRID * 32 + (size_t)t1 * t3 + (size_t)nH * t1);
}

__global__ void __launch_bounds__(256)
k_dec_out(const float* __restrict__ part_o, const float* __restrict__ part_ml, const int32_t* __restrict__ cache_len,
          int B, int Lmax, int nH, int t1, int t2, int t3, int grid_attn, const bf16* __restrict__ Ct,
          const bf16* __restrict__ Ut1, bf16* __restrict__ z, unsigned int* err) {
  extern __shared__ __align__(16) float do_smem[];
  float* o_s = do_smem;                    // [32][t3]
  float* w_s = o_s + 32 * t3;              // [MAX_GRID][32]
  float* u_s = w_s + MAX_GRID * 32;        // [t1][t3]
  float* ut1_s = u_s + t1 * t3;            // [nH][t1]
  __shared__ float inv_l[32];
  __shared__ int on_s[MAX_GRID];
  const int b = blockIdx.x;
  const int jn = t2 / DO_JS, jbeg = blockIdx.y * jn;      // this CTA's output rows [jbeg, jbeg + jn)
  const int nch = t3 / 8;                  // 16-byte chunks per core row: 8, 12 or 16
  // pull this CTA's rows of the output core towards L2 while the merge runs
  {
    const char* cbase = reinterpret_cast<const char*>(Ct);
    const long row_bytes = (long)t3 * 2, span = (long)jn * row_bytes;
    for (int a = 0; a < t1; ++a)
      for (long off = (long)threadIdx.x * 128; off < span; off += (long)blockDim.x * 128)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(cbase + ((long)a * t2 + jbeg) * row_bytes + off));
  }
  __shared__ long long wtot_s[8];
  __shared__ long long first_s;
  int lo, hi;
  long excl;
  const long total = block_tile_scan(cache_len, B, Lmax, lo, hi, excl, wtot_s);
  if (b >= lo && b < hi) {
    long f = excl;
    for (int i = lo; i < b; ++i) f += tiles_of(clamp_len(cache_len[i], Lmax));
    first_s = f;
  }
  __syncthreads();
  const long first = (long)first_s;
  const long nt = tiles_of(clamp_len(cache_len[b], Lmax));
  // CTAs i with [first_i, first_{i+1}) intersecting [first, first + nt)
  long i0 = first * grid_attn / total;
  while (i0 > 0 && cta_first_tile(i0, total, grid_attn) > first) --i0;
  while (cta_first_tile(i0 + 1, total, grid_attn) <= first) ++i0;
  long i1 = i0;
  while (i1 + 1 < grid_attn && cta_first_tile(i1 + 1, total, grid_attn) < first + nt) ++i1;
  int np = (int)(i1 - i0 + 1);
  // this sequence's partials occupy the slots i0 + b .. i1 + b of the grid_attn + B that exist
  if (!TA_IDX_OK(err, i0 + b, np, (long)grid_attn + B)) np = 0;
  for (int i = threadIdx.x; i < nH * t1; i += blockDim.x) ut1_s[i] = __bfloat162float(Ut1[i]);
  // which of the np candidate CTAs wrote a partial for this sequence (a CTA whose tile range is
  // empty wrote nothing: its slot holds stale bytes that must not be used as numbers)
  for (int k = threadIdx.x; k < np; k += blockDim.x) {
    const long i = i0 + k;
    on_s[k] = cta_first_tile(i, total, grid_attn) != cta_first_tile(i + 1, total, grid_attn);
  }
  __syncthreads();
  // Up to here only inputs of the call were read (cache_len, Ut1, the prefetch of the output core), while
  // the attention kernel before this one finishes; its partials are read after pdl_enter().
  pdl_enter();
  if (threadIdx.x < 32) {
    // log-sum-exp over the partials of head h; four (max, sum) pairs are loaded at a time
    const int h = threadIdx.x;
    const float2* ml = reinterpret_cast<const float2*>(part_ml) + (i0 + b) * 32 + h;
    float M = -INFINITY, Lsum = 0.f;
    for (int k0 = 0; k0 < np; k0 += 4) {
      float2 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) v[u] = (k0 + u < np) ? ml[(long)(k0 + u) * 32] : make_float2(-INFINITY, 0.f);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (k0 + u < np && on_s[k0 + u] && v[u].x > -INFINITY) {
          const float Mn = fmaxf(M, v[u].x);
          Lsum = Lsum * ex2(M - Mn) + v[u].y * ex2(v[u].x - Mn);
          M = Mn;
        }
      }
    }
    for (int k0 = 0; k0 < np; k0 += 4) {
      float2 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) v[u] = (k0 + u < np) ? ml[(long)(k0 + u) * 32] : make_float2(-INFINITY, 0.f);
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (k0 + u < np) w_s[(k0 + u) * 32 + h] = (on_s[k0 + u] && v[u].x > -INFINITY) ? ex2(v[u].x - M) : 0.f;
    }
    inv_l[h] = 1.f / Lsum;
  }
  __syncthreads();
  // merged (not yet normalised) outputs: a thread owns up to 4 float4 of the [nH][t3] block
  // (nH * t3 / 4 <= 1024 = 4 * blockDim.x for nH <= 32, t3 <= 128); for the usual case of at most four
  // partials all of its loads are issued before any is used
  {
    const int n4 = nH * t3 / 4;
    const float4* po = reinterpret_cast<const float4*>(part_o + (i0 + b) * 32 * t3);
    for (int k0 = 0; k0 < np || k0 == 0; k0 += 4) {
      float4 v[4][4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int e4 = threadIdx.x + e * 256;
#pragma unroll
        for (int u = 0; u < 4; ++u)
          v[e][u] = (e4 < n4 && k0 + u < np) ? po[(long)(k0 + u) * 8 * t3 + e4] : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int e4 = threadIdx.x + e * 256;
        if (e4 < n4) {
          const int h = (e4 * 4) / t3;
          float4 acc = k0 == 0 ? make_float4(0.f, 0.f, 0.f, 0.f) : reinterpret_cast<float4*>(o_s)[e4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const float wg = (k0 + u < np) ? w_s[(k0 + u) * 32 + h] : 0.f;
            if (wg != 0.f) {     // a zero weight marks a slot whose bytes are not numbers to be used
              acc.x += wg * v[e][u].x; acc.y += wg * v[e][u].y; acc.z += wg * v[e][u].z; acc.w += wg * v[e][u].w;
            }
          }
          reinterpret_cast<float4*>(o_s)[e4] = acc;
        }
      }
    }
  }
  __syncthreads();
  // u[a, c] = sum_h Ut1[h, a] o_h[c] / l_h; a thread owns column c and runs of four slices a
  {
    const int ngrp = blockDim.x / t3 > 0 ? blockDim.x / t3 : 1;     // thread groups over the slices
    const int c = threadIdx.x % t3, grp = threadIdx.x / t3;
    if (grp < ngrp) {
      for (int a0 = grp * 4; a0 < t1; a0 += ngrp * 4) {
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        for (int h = 0; h < nH; ++h) {
          const float ov = o_s[h * t3 + c] * inv_l[h];
#pragma unroll
          for (int u = 0; u < 4; ++u)
            if (a0 + u < t1) acc[u] = fmaf(ut1_s[h * t1 + a0 + u], ov, acc[u]);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (a0 + u < t1) u_s[(a0 + u) * t3 + c] = acc[u];
      }
    }
  }
  __syncthreads();
  // z[j]: lane group g = lane / nch of warp w owns output row j = jbeg + (w * rpl + g) + 8 * rpl * jj and
  // walks the slices a with 16-byte loads, PF of them in flight.
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int rpl = 32 / nch;                // rows per warp-wide load: 4, 2 or 2
  const int g = lane / nch, ch = lane % nch;
  const uint4* Cq = reinterpret_cast<const uint4*>(Ct);
  constexpr int PF = 8, JJ = 2;
  // (the rows of this CTA were prefetched into L2 at the top, so every batch costs one L2 round trip;
  // a lane group takes JJ output rows at a time, JJ * PF loads in flight)
  for (int jl = warp * rpl + (g < rpl ? g : 0); jl < jn; jl += 8 * rpl * JJ) {     // uniform trip count per warp
    float acc[JJ];
#pragma unroll
    for (int jj = 0; jj < JJ; ++jj) acc[jj] = 0.f;
    for (int a0 = 0; a0 < t1; a0 += PF) {
      uint4 v[JJ][PF];
#pragma unroll
      for (int jj = 0; jj < JJ; ++jj) {
        const int j = jbeg + jl + jj * 8 * rpl;
#pragma unroll
        for (int u = 0; u < PF; ++u)
          v[jj][u] = (g < rpl && a0 + u < t1 && jl + jj * 8 * rpl < jn) ? Cq[((long)(a0 + u) * t2 + j) * nch + ch]
                                                                        : make_uint4(0u, 0u, 0u, 0u);
      }
#pragma unroll
      for (int u = 0; u < PF; ++u) {
        if (a0 + u < t1) {
          const float4 u0 = reinterpret_cast<const float4*>(u_s + (a0 + u) * t3 + ch * 8)[0];
          const float4 u1 = reinterpret_cast<const float4*>(u_s + (a0 + u) * t3 + ch * 8)[1];
#pragma unroll
          for (int jj = 0; jj < JJ; ++jj) {
            const uint32_t wv[4] = {v[jj][u].x, v[jj][u].y, v[jj][u].z, v[jj][u].w};
            const float2 k0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&wv[0]));
            const float2 k1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&wv[1]));
            const float2 k2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&wv[2]));
            const float2 k3 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&wv[3]));
            float t = acc[jj];
            t = fmaf(u0.x, k0.x, t); t = fmaf(u0.y, k0.y, t); t = fmaf(u0.z, k1.x, t); t = fmaf(u0.w, k1.y, t);
            t = fmaf(u1.x, k2.x, t); t = fmaf(u1.y, k2.y, t); t = fmaf(u1.z, k3.x, t); t = fmaf(u1.w, k3.y, t);
            acc[jj] = t;
          }
        }
      }
    }
    // sum over the nch lanes of the group (groups are aligned to multiples of nch lanes)
#pragma unroll
    for (int jj = 0; jj < JJ; ++jj) {
      float t = (g >= rpl) ? 0.f : acc[jj];
      for (int off = 1; off < nch; off <<= 1) {
        const float o = __shfl_down_sync(0xffffffffu, t, off);
        if (ch + off < nch) t += o;
      }
      const int jrow = jl + jj * 8 * rpl;
      if (g < rpl && ch == 0 && jrow < jn && TA_IDX_OK(err, (long)b * t2 + jbeg + jrow, 1, (long)B * t2))
        z[(long)b * t2 + jbeg + jrow] = __float2bfloat16_rn(t);
    }
  }
}

}  // namespace dec
}  // namespace ta
