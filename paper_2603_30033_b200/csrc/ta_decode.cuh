// Decode step over the latent KV cache (Eq. 9, "KV Caching"): kernels of the bf16 path.
//
// k_dec_attn streams every sequence's latent K / V cache exactly once.  The cache is cut into
// tiles of 128 keys; the flat list of tiles of all sequences is divided evenly over the CTAs
// (one per SM), so that the load is balanced for any mix of cache lengths.  Each CTA walks its
// tile range, keeps an online-softmax state per sequence segment, and writes one partial
// (max, sum, unnormalised O for all heads) per segment; k_dec_merge combines the partials of
// a sequence with log-sum-exp weights and applies the output-side core (Z = sum_h o_h Gt_h^T).
//
// All n_H (<= 32) heads share each K / V byte, so the arithmetic is 2 * n_H flop per cached
// element -- beyond plain FMA throughput at HBM speed.  The products therefore run on the
// tensor cores with the heads as the M dimension (two m16 tiles) of mma.sync m16n8k16:
//   warp (mt, kq), mt = head half, kq = 32-key quarter of the tile
//   S[16 heads x 32 keys] = Qhat_mt K_q^T ; online softmax with quad shuffles ; O += P V_q
// K / V tiles arrive by TMA (3-D tensor map, 128-byte swizzle, conflict-free ldmatrix) through
// a 3-stage ring fed by a dedicated producer warp.
#pragma once

#include "ta_common.cuh"
#include "ta_sm100.cuh"

namespace ta {
namespace dec {

using namespace sm100;

constexpr int TK = 128;                 // keys per tile
constexpr int CONSUMER_WARPS = 8;
constexpr int THREADS = 32 * (CONSUMER_WARPS + 1);
constexpr int STAGES = 3;
constexpr int SUB_BYTES = 128 * 64 * 2;
constexpr int MAX_SUB = 2;              // r3, t3 <= 128
constexpr int STAGE_BYTES = 2 * MAX_SUB * SUB_BYTES;   // K tile + V tile
constexpr size_t SMEM_BYTES = 1024 + (size_t)STAGES * STAGE_BYTES;
constexpr int MAX_GRID = 160;           // partial weights table in the merge kernel

struct Params {
  int B, nH, Lmax, grid;
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

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// Byte offset of (row, 16-byte chunk) inside a tile made of [128 x 64] sub-tiles with 128-byte swizzle.
__device__ __forceinline__ uint32_t swz(int row, int chunk) {
  return (uint32_t)((chunk >> 3) * SUB_BYTES + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

template <int R3, int T3>
__global__ void __launch_bounds__(THREADS, 1)
k_dec_attn(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t full_bar[STAGES], empty_bar[STAGES];
  __shared__ int abort_flag;
  __shared__ float ml_s[CONSUMER_WARPS][16][2];
  __shared__ __align__(16) float obuf[32 * T3];

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* tiles = smem_raw + (base - smem_u32(smem_raw));
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  Abort ab{&abort_flag, p.err};
  constexpr int KSUB = (R3 + 63) / 64, VSUB = (T3 + 63) / 64;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], CONSUMER_WARPS);
    }
    fence_barrier_init();
  }
  __syncthreads();

  // ---- this CTA's range of the flat tile list ----
  long total = 0;
  for (int b = 0; b < p.B; ++b) total += tiles_of(clamp_len(p.cache_len[b], p.Lmax));
  const long t_begin = cta_first_tile(blockIdx.x, total, gridDim.x);
  const long t_end = cta_first_tile(blockIdx.x + 1, total, gridDim.x);
  int b0 = 0;
  long seq_first = 0;   // global index of the first tile of sequence b0
  if (t_begin < t_end) {
    while (true) {
      const long nt = tiles_of(clamp_len(p.cache_len[b0], p.Lmax));
      if (seq_first + nt > t_begin) break;
      seq_first += nt;
      ++b0;
    }
  }

  if (warp == CONSUMER_WARPS) {
    // ------------------------------- TMA producer -------------------------------
    if (elect_one() && t_begin < t_end) {
      tma_prefetch_desc(&tmK);
      tma_prefetch_desc(&tmV);
      int b = b0;
      long first = seq_first;
      long nt = tiles_of(clamp_len(p.cache_len[b], p.Lmax));
      int it = 0;
      for (long t = t_begin; t < t_end; ++t, ++it) {
        while (t >= first + nt) {
          first += nt;
          ++b;
          nt = tiles_of(clamp_len(p.cache_len[b], p.Lmax));
        }
        const int s = it % STAGES;
        const uint32_t ph = (it / STAGES) & 1;
        if (!mbar_wait(&empty_bar[s], ph ^ 1, ab)) break;
        mbar_expect_tx(&full_bar[s], (uint32_t)((KSUB + VSUB) * SUB_BYTES));
        uint8_t* kt = tiles + (size_t)s * STAGE_BYTES;
        uint8_t* vt = kt + MAX_SUB * SUB_BYTES;
        const int row = (int)(t - first) * TK;
        for (int kk = 0; kk < KSUB; ++kk) tma_load_3d(kt + kk * SUB_BYTES, &tmK, &full_bar[s], kk * 64, row, b);
        for (int kk = 0; kk < VSUB; ++kk) tma_load_3d(vt + kk * SUB_BYTES, &tmV, &full_bar[s], kk * 64, row, b);
      }
    }
  } else if (t_begin < t_end) {
    // ------------------------------- consumers ----------------------------------
    const int mt = warp / 4, kq = warp % 4;
    const int g = lane / 4, tq = lane % 4;
    int b = b0;
    long first = seq_first;
    int it = 0;
    bool ok = true;
    long t = t_begin;
    while (t < t_end && ok) {
      // ---- one segment: tiles [t, seg_end) of sequence b ----
      const int L = clamp_len(p.cache_len[b], p.Lmax);
      const long nt = tiles_of(L);
      const long seg_end = (first + nt < t_end) ? first + nt : t_end;
      // Qhat fragments (A operand): rows = heads 16*mt + {g, g+8}
      uint32_t qa[R3 / 16][4];
      {
        const int h_lo = 16 * mt + g, h_hi = h_lo + 8;
        const bf16* q_lo = p.qhat + ((long)b * p.nH + h_lo) * R3;
        const bf16* q_hi = p.qhat + ((long)b * p.nH + h_hi) * R3;
#pragma unroll
        for (int kb = 0; kb < R3 / 16; ++kb) {
          const int c = kb * 16 + 2 * tq;
          qa[kb][0] = h_lo < p.nH ? *reinterpret_cast<const uint32_t*>(q_lo + c) : 0u;
          qa[kb][1] = h_hi < p.nH ? *reinterpret_cast<const uint32_t*>(q_hi + c) : 0u;
          qa[kb][2] = h_lo < p.nH ? *reinterpret_cast<const uint32_t*>(q_lo + c + 8) : 0u;
          qa[kb][3] = h_hi < p.nH ? *reinterpret_cast<const uint32_t*>(q_hi + c + 8) : 0u;
        }
      }
      float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
      float o[T3 / 8][4];
#pragma unroll
      for (int n = 0; n < T3 / 8; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;

      for (; t < seg_end; ++t, ++it) {
        const int s = it % STAGES;
        const uint32_t ph = (it / STAGES) & 1;
        ok = mbar_wait(&full_bar[s], ph, ab);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        uint8_t* kt = tiles + (size_t)s * STAGE_BYTES;
        uint8_t* vt = kt + MAX_SUB * SUB_BYTES;
        const int k0 = (int)(t - first) * TK;
        const bool last_tile = (k0 + TK > L);        // contains the new token (index L) and possibly invalid rows
        if (last_tile) {
          // rows of this warp's quarter: patch the new token's row from the workspace, zero invalid V rows
          const int rnew = L - k0;
          for (int rr = 0; rr < 32; ++rr) {
            const int r = kq * 32 + rr;
            if (r == rnew) {
              if (lane * 4 < R3) {
                const uint2 kv = *reinterpret_cast<const uint2*>(p.knew + (long)b * R3 + lane * 4);
                *reinterpret_cast<uint2*>(kt + swz(r, lane >> 1) + (lane & 1) * 8) = kv;
              }
              if (lane * 4 < T3) {
                const uint2 vv = *reinterpret_cast<const uint2*>(p.vnew + (long)b * T3 + lane * 4);
                *reinterpret_cast<uint2*>(vt + swz(r, lane >> 1) + (lane & 1) * 8) = vv;
              }
            } else if (r > rnew) {
              if (lane * 4 < T3) *reinterpret_cast<uint2*>(vt + swz(r, lane >> 1) + (lane & 1) * 8) = make_uint2(0u, 0u);
            }
          }
          fence_proxy_async_smem();
          __syncwarp();
        }
        // ---- S = Qhat K^T for this warp's 32 keys ----
        float sc[4][4];
#pragma unroll
        for (int n = 0; n < 4; ++n) sc[n][0] = sc[n][1] = sc[n][2] = sc[n][3] = 0.f;
        const uint32_t kbase = smem_u32(kt), vbase = smem_u32(vt);
        {
          const int mi = lane >> 3, rl = lane & 7;
#pragma unroll
          for (int kb = 0; kb < R3 / 16; ++kb) {
#pragma unroll
            for (int np = 0; np < 2; ++np) {
              const int row = kq * 32 + (np * 2 + (mi >> 1)) * 8 + rl;
              const int chunk = kb * 2 + (mi & 1);
              uint32_t r0, r1, r2, r3;
              ldsm_x4(kbase + swz(row, chunk), r0, r1, r2, r3);
              mma_bf16(sc[np * 2], qa[kb], r0, r1);
              mma_bf16(sc[np * 2 + 1], qa[kb], r2, r3);
            }
          }
        }
        if (last_tile) {
#pragma unroll
          for (int n = 0; n < 4; ++n)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int key = k0 + kq * 32 + n * 8 + 2 * tq + (e & 1);
              if (key > L) sc[n][e] = -INFINITY;
            }
        }
        // ---- online softmax (rows g and g+8 of this head half) ----
        float corr[2];
        uint32_t pa[2][4];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          float mx = -INFINITY;
#pragma unroll
          for (int n = 0; n < 4; ++n) mx = fmaxf(mx, fmaxf(sc[n][2 * r], sc[n][2 * r + 1]));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
          const float m_new = fmaxf(m_run[r], mx);
          const float m_safe = (m_new == -INFINITY) ? 0.f : m_new;
          corr[r] = ex2(m_run[r] - m_safe);      // 0 when nothing was visible before
          m_run[r] = m_new;
          float rs = 0.f;
#pragma unroll
          for (int n = 0; n < 4; ++n) {
            sc[n][2 * r] = ex2(sc[n][2 * r] - m_safe);
            sc[n][2 * r + 1] = ex2(sc[n][2 * r + 1] - m_safe);
            rs += sc[n][2 * r] + sc[n][2 * r + 1];
          }
          l_run[r] = l_run[r] * corr[r] + rs;
        }
#pragma unroll
        for (int kb2 = 0; kb2 < 2; ++kb2) {
          pa[kb2][0] = pack_bf16(sc[2 * kb2][0], sc[2 * kb2][1]);
          pa[kb2][1] = pack_bf16(sc[2 * kb2][2], sc[2 * kb2][3]);
          pa[kb2][2] = pack_bf16(sc[2 * kb2 + 1][0], sc[2 * kb2 + 1][1]);
          pa[kb2][3] = pack_bf16(sc[2 * kb2 + 1][2], sc[2 * kb2 + 1][3]);
        }
#pragma unroll
        for (int n = 0; n < T3 / 8; ++n) {
          o[n][0] *= corr[0]; o[n][1] *= corr[0];
          o[n][2] *= corr[1]; o[n][3] *= corr[1];
        }
        // ---- O += P V for this warp's 32 keys ----
        {
          const int mi = lane >> 3, rl = lane & 7;
#pragma unroll
          for (int kb2 = 0; kb2 < 2; ++kb2) {
            const int row = kq * 32 + kb2 * 16 + (mi & 1) * 8 + rl;
#pragma unroll
            for (int n = 0; n < T3 / 8; n += 2) {
              uint32_t r0, r1, r2, r3;
              ldsm_x4_t(vbase + swz(row, n + (mi >> 1)), r0, r1, r2, r3);
              mma_bf16(o[n], pa[kb2], r0, r1);
              mma_bf16(o[n + 1], pa[kb2], r2, r3);
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[s]);
      }
      if (!ok) break;
      // ---- segment done: merge the four key-quarter warps of each head half, write the partial ----
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
        l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
      }
      if (tq == 0) {
        ml_s[warp][g][0] = m_run[0]; ml_s[warp][g][1] = l_run[0];
      }
      consumer_sync();
      // (rows g+8 are exchanged in a second pass to keep the table small)
      float Mx[2], Ls[2], own[2];
      {
        float M = -INFINITY;
        for (int k = 0; k < 4; ++k) M = fmaxf(M, ml_s[mt * 4 + k][g][0]);
        const float Ms = (M == -INFINITY) ? 0.f : M;
        float Lsum = 0.f;
        for (int k = 0; k < 4; ++k) Lsum += ml_s[mt * 4 + k][g][1] * ex2(ml_s[mt * 4 + k][g][0] - Ms);
        Mx[0] = M; Ls[0] = Lsum; own[0] = ex2(m_run[0] - Ms);
      }
      consumer_sync();
      if (tq == 0) {
        ml_s[warp][g][0] = m_run[1]; ml_s[warp][g][1] = l_run[1];
      }
      consumer_sync();
      {
        float M = -INFINITY;
        for (int k = 0; k < 4; ++k) M = fmaxf(M, ml_s[mt * 4 + k][g][0]);
        const float Ms = (M == -INFINITY) ? 0.f : M;
        float Lsum = 0.f;
        for (int k = 0; k < 4; ++k) Lsum += ml_s[mt * 4 + k][g][1] * ex2(ml_s[mt * 4 + k][g][0] - Ms);
        Mx[1] = M; Ls[1] = Lsum; own[1] = ex2(m_run[1] - Ms);
      }
      for (int k = 0; k < 4; ++k) {
        if (kq == k) {
#pragma unroll
          for (int n = 0; n < T3 / 8; ++n) {
            float* r_lo = obuf + (16 * mt + g) * T3 + n * 8 + 2 * tq;
            float* r_hi = r_lo + 8 * T3;
            if (k == 0) {
              r_lo[0] = o[n][0] * own[0]; r_lo[1] = o[n][1] * own[0];
              r_hi[0] = o[n][2] * own[1]; r_hi[1] = o[n][3] * own[1];
            } else {
              r_lo[0] += o[n][0] * own[0]; r_lo[1] += o[n][1] * own[0];
              r_hi[0] += o[n][2] * own[1]; r_hi[1] += o[n][3] * own[1];
            }
          }
        }
        consumer_sync();
      }
      {
        const long slot = (long)blockIdx.x + b;
        float4* dst = reinterpret_cast<float4*>(p.part_o + slot * 32 * T3);
        const float4* src = reinterpret_cast<const float4*>(obuf);
        for (int i = threadIdx.x; i < 32 * T3 / 4; i += 256) dst[i] = src[i];
        if (kq == 0 && tq == 0) {
          float* ml = p.part_ml + slot * 64;
          ml[(16 * mt + g) * 2 + 0] = Mx[0]; ml[(16 * mt + g) * 2 + 1] = Ls[0];
          ml[(16 * mt + g + 8) * 2 + 0] = Mx[1]; ml[(16 * mt + g + 8) * 2 + 1] = Ls[1];
        }
      }
      consumer_sync();
      // next sequence
      first += nt;
      ++b;
    }
  }
}

// ---------------------------------------------------------------------------------------
// Per sequence b (one CTA): finishes the new token's latent projections and forms its
// per-head queries.
//   row      = sum over the split-K partials of [qt | k | v]            (fp32)
//   k, v     -> latent RoPE on k at position L = cache_len[b]; bf16 copies for the attention
//               kernel; appended to the caches at slot L when `append`
//   w[a, :]  = qt C[a]                        (the core contracted with the query first:
//   qhat_h   = mult * sum_a U1[h, a] w[a, :]   C x_2 qt x_1 U1, Eq. 9, so that the n_H
//                                              per-head matrices G_h are never formed)
//   qhat_h  <- qhat_h R(L, r3), stored bf16 [B, nH, r3]
// part: [splits][Mpad][r2 + r3 + t3] fp32.  Dynamic shared memory: see dec_qhat_smem().
// ---------------------------------------------------------------------------------------
__host__ __device__ inline size_t dec_qhat_smem(int nH, int r1, int r2, int r3, int t3) {
  return sizeof(float) * ((size_t)(r2 + r3 + t3) + (size_t)r1 * r3 + (size_t)nH * r1) + sizeof(float2) * (size_t)(r3 / 2);
}

__global__ void __launch_bounds__(256)
k_dec_qhat(const float* __restrict__ part, int splits, long split_stride, int nH, int r1, int r2, int r3, int t3,
           const bf16* __restrict__ C, const bf16* __restrict__ U1, float mult, bf16* __restrict__ qhat,
           bf16* __restrict__ knew, bf16* __restrict__ vnew, bf16* __restrict__ Kc, bf16* __restrict__ Vc, int Lmax,
           const int32_t* __restrict__ cache_len, int rope, double base, int append, unsigned int* err) {
  extern __shared__ __align__(16) float dq_smem[];
  const int ncol = r2 + r3 + t3, half = r3 / 2;
  float2* cs_s = reinterpret_cast<float2*>(dq_smem);   // [r3/2] (cos, sin) at position L
  float* row = dq_smem + 2 * half;          // [ncol]
  float* w_s = row + ncol;                  // [r1][r3]
  float* u1_s = w_s + r1 * r3;              // [nH][r1]
  const int b = blockIdx.x;
  int L = cache_len[b];
  if (L < 0 || L >= Lmax) {
    if (threadIdx.x == 0) atomicOr(err, (unsigned)TA_DEVERR_BAD_CACHE_LEN);
    L = clamp_len(L, Lmax);
  }
  for (int c = threadIdx.x; c < ncol; c += blockDim.x) {
    float acc = 0.f;
    for (int s = 0; s < splits; ++s) acc += part[s * split_stride + (long)b * ncol + c];
    row[c] = acc;
  }
  for (int i = threadIdx.x; i < nH * r1; i += blockDim.x) u1_s[i] = __bfloat162float(U1[i]);
  for (int i = threadIdx.x; i < r1 * r3; i += blockDim.x) w_s[i] = 0.f;
  for (int i = threadIdx.x; i < half; i += blockDim.x) {
    float2 cs = make_float2(1.f, 0.f);
    if (rope) {
      const double theta = pow(base, -2.0 * (double)i / (double)r3);
      double sn, co;
      sincos((double)L * theta, &sn, &co);
      cs = make_float2((float)co, (float)sn);
    }
    cs_s[i] = cs;
  }
  __syncthreads();
  // new key (rotated) and value
  for (int i = threadIdx.x; i < half; i += blockDim.x) {
    const float xe = row[r2 + 2 * i], xo = row[r2 + 2 * i + 1];
    const float2 cs = cs_s[i];
    const __nv_bfloat162 v = __floats2bfloat162_rn(xe * cs.x - xo * cs.y, xe * cs.y + xo * cs.x);
    *reinterpret_cast<__nv_bfloat162*>(knew + (long)b * r3 + 2 * i) = v;
    if (append) *reinterpret_cast<__nv_bfloat162*>(Kc + ((long)b * Lmax + L) * r3 + 2 * i) = v;
  }
  for (int c = threadIdx.x; c < t3; c += blockDim.x) {
    const bf16 v = __float2bfloat16_rn(row[r2 + r3 + c]);
    vnew[(long)b * t3 + c] = v;
    if (append) Vc[((long)b * Lmax + L) * t3 + c] = v;
  }
  // w[a, c] = sum_q qt[q] C[a, q, c].  A thread owns one 16-byte chunk (8 values of c) of the core
  // rows q = rg, rg + nrg, ... ; the loads of slice a + 1 are issued before the FMAs of slice a so
  // that a full batch of independent 16-byte loads is always in flight; the row groups of a CTA are
  // combined with shared-memory atomic adds (w_s was zeroed above).
  {
    constexpr int PF = 8;                      // loads in flight per thread and slice
    const int nch = r3 / 8;                    // 16-byte chunks per core row (r3 is a multiple of 32)
    const int nrg = blockDim.x / nch;          // row groups
    const int ch = threadIdx.x % nch, rg = threadIdx.x / nch;
    if (rg < nrg) {
      const uint4* Cq = reinterpret_cast<const uint4*>(C);
      for (int q0 = rg; q0 < r2; q0 += nrg * PF) {
        uint4 v[PF];
#pragma unroll
        for (int u = 0; u < PF; ++u) {
          const int q = q0 + u * nrg;
          v[u] = q < r2 ? Cq[(long)q * nch + ch] : make_uint4(0u, 0u, 0u, 0u);
        }
        for (int a = 0; a < r1; ++a) {
          uint4 vn[PF];
          if (a + 1 < r1) {
#pragma unroll
            for (int u = 0; u < PF; ++u) {
              const int q = q0 + u * nrg;
              vn[u] = q < r2 ? Cq[((long)(a + 1) * r2 + q) * nch + ch] : make_uint4(0u, 0u, 0u, 0u);
            }
          }
          float acc[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[e] = 0.f;
#pragma unroll
          for (int u = 0; u < PF; ++u) {
            const int q = q0 + u * nrg;
            const float xq = q < r2 ? row[q] : 0.f;
            const uint32_t wv[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float2 cv = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&wv[e]));
              acc[2 * e] = fmaf(xq, cv.x, acc[2 * e]);
              acc[2 * e + 1] = fmaf(xq, cv.y, acc[2 * e + 1]);
            }
          }
#pragma unroll
          for (int e = 0; e < 8; ++e) atomicAdd(&w_s[a * r3 + ch * 8 + e], acc[e]);
          if (a + 1 < r1) {
#pragma unroll
            for (int u = 0; u < PF; ++u) v[u] = vn[u];
          }
        }
      }
    }
  }
  __syncthreads();
  for (int item = threadIdx.x; item < nH * half; item += blockDim.x) {
    const int h = item / half, cp = item % half;
    float xe = 0.f, xo = 0.f;
    for (int a = 0; a < r1; ++a) {
      const float u = u1_s[h * r1 + a];
      xe = fmaf(u, w_s[a * r3 + 2 * cp], xe);
      xo = fmaf(u, w_s[a * r3 + 2 * cp + 1], xo);
    }
    xe *= mult; xo *= mult;
    const float2 cs = cs_s[cp];
    *reinterpret_cast<__nv_bfloat162*>(qhat + ((long)b * nH + h) * r3 + 2 * cp) =
        __floats2bfloat162_rn(xe * cs.x - xo * cs.y, xe * cs.y + xo * cs.x);
  }
}

// ---------------------------------------------------------------------------------------
// Per sequence b (one CTA): log-sum-exp merge of the partials written by the attention CTAs
// whose tile range intersected the sequence, then the output-side core with the head mode
// contracted first (the n_H matrices Gt_h are never formed):
//   o_h      = merged, normalised attention output of head h             [nH][t3]
//   u[a, :]  = sum_h Ut1[h, a] o_h                                       [t1][t3]
//   z[j]     = sum_a sum_c Ct[a, j, c] u[a, c]                           [t2]   (= sum_h Gt_h o_h)
// z is written as bf16 [B, t2].  Dynamic shared memory: see dec_out_smem().
// ---------------------------------------------------------------------------------------
__host__ __device__ inline size_t dec_out_smem(int nH, int t1, int t3) {
  return sizeof(float) * (32 * (size_t)t3 + (size_t)MAX_GRID * 32 + (size_t)t1 * t3 + (size_t)nH * t1);
}

__global__ void __launch_bounds__(256)
k_dec_out(const float* __restrict__ part_o, const float* __restrict__ part_ml, const int32_t* __restrict__ cache_len,
          int B, int Lmax, int nH, int t1, int t2, int t3, int grid_attn, const bf16* __restrict__ Ct,
          const bf16* __restrict__ Ut1, bf16* __restrict__ z) {
  extern __shared__ __align__(16) float do_smem[];
  float* o_s = do_smem;                    // [32][t3]
  float* w_s = o_s + 32 * t3;              // [MAX_GRID][32]
  float* u_s = w_s + MAX_GRID * 32;        // [t1][t3]
  float* ut1_s = u_s + t1 * t3;            // [nH][t1]
  __shared__ float inv_l[32];
  const int b = blockIdx.x;
  long total = 0, first = 0;
  for (int i = 0; i < B; ++i) {
    if (i == b) first = total;
    total += tiles_of(clamp_len(cache_len[i], Lmax));
  }
  const long nt = tiles_of(clamp_len(cache_len[b], Lmax));
  // CTAs i with [first_i, first_{i+1}) intersecting [first, first + nt)
  long i0 = first * grid_attn / total;
  while (i0 > 0 && cta_first_tile(i0, total, grid_attn) > first) --i0;
  while (cta_first_tile(i0 + 1, total, grid_attn) <= first) ++i0;
  long i1 = i0;
  while (i1 + 1 < grid_attn && cta_first_tile(i1 + 1, total, grid_attn) < first + nt) ++i1;
  const int np = (int)(i1 - i0 + 1);
  for (int i = threadIdx.x; i < nH * t1; i += blockDim.x) ut1_s[i] = __bfloat162float(Ut1[i]);
  if (threadIdx.x < 32) {
    const int h = threadIdx.x;
    float M = -INFINITY;
    for (int k = 0; k < np; ++k) {
      const long i = i0 + k;
      if (cta_first_tile(i, total, grid_attn) == cta_first_tile(i + 1, total, grid_attn)) continue;   // empty CTA
      M = fmaxf(M, part_ml[((i + b) * 32 + h) * 2]);
    }
    float Lsum = 0.f;
    for (int k = 0; k < np; ++k) {
      const long i = i0 + k;
      float wgt = 0.f;
      if (cta_first_tile(i, total, grid_attn) != cta_first_tile(i + 1, total, grid_attn)) {
        const float m = part_ml[((i + b) * 32 + h) * 2], l = part_ml[((i + b) * 32 + h) * 2 + 1];
        wgt = (m == -INFINITY) ? 0.f : ex2(m - M);
        Lsum += wgt * l;
      }
      w_s[k * 32 + h] = wgt;
    }
    inv_l[h] = 1.f / Lsum;
  }
  __syncthreads();
  for (int e4 = threadIdx.x; e4 < nH * t3 / 4; e4 += blockDim.x) {
    const int h = (e4 * 4) / t3;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int k = 0; k < np; ++k) {
      const float wgt = w_s[k * 32 + h];
      if (wgt != 0.f) {
        const float4 v = reinterpret_cast<const float4*>(part_o + (i0 + k + b) * 32 * t3)[e4];
        acc.x += wgt * v.x; acc.y += wgt * v.y; acc.z += wgt * v.z; acc.w += wgt * v.w;
      }
    }
    const float il = inv_l[h];
    reinterpret_cast<float4*>(o_s)[e4] = make_float4(acc.x * il, acc.y * il, acc.z * il, acc.w * il);
  }
  __syncthreads();
  for (int e = threadIdx.x; e < t1 * t3; e += blockDim.x) {
    const int a = e / t3, c = e % t3;
    float acc = 0.f;
    for (int h = 0; h < nH; ++h) acc = fmaf(ut1_s[h * t1 + a], o_s[h * t3 + c], acc);
    u_s[e] = acc;
  }
  __syncthreads();
  // z[j] = sum_{a,c} Ct[a, j, c] u[a, c].  A warp takes JB output rows j at a time; its lanes are
  // split into groups of nch = t3 / 8 lanes, each group reading one core row (a, j, :) in 16-byte
  // chunks, so that JB * ceil(t1 / rows-per-load) independent loads are in flight per lane.
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int nwarp = blockDim.x / 32;
  constexpr int JB = 4;
  const int nch = t3 / 8;                 // 8, 12 or 16
  const int rpl = 32 / nch;               // core rows per warp-wide load
  const int la = lane / nch, ch = lane % nch;
  const bool lane_on = la < rpl;
  const uint4* Cq = reinterpret_cast<const uint4*>(Ct);
  for (int j0 = warp * JB; j0 < t2; j0 += nwarp * JB) {
    float acc[JB];
#pragma unroll
    for (int jj = 0; jj < JB; ++jj) acc[jj] = 0.f;
    if (lane_on) {
      for (int a0 = la; a0 < t1; a0 += rpl * 4) {
        uint4 v[4][JB];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int a = a0 + u * rpl;
#pragma unroll
          for (int jj = 0; jj < JB; ++jj) {
            const int j = j0 + jj;
            v[u][jj] = (a < t1 && j < t2) ? Cq[((long)a * t2 + j) * nch + ch] : make_uint4(0u, 0u, 0u, 0u);
          }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int a = a0 + u * rpl;
          if (a < t1) {
            const float4 u0 = reinterpret_cast<const float4*>(u_s + a * t3 + ch * 8)[0];
            const float4 u1 = reinterpret_cast<const float4*>(u_s + a * t3 + ch * 8)[1];
#pragma unroll
            for (int jj = 0; jj < JB; ++jj) {
              const uint32_t wv[4] = {v[u][jj].x, v[u][jj].y, v[u][jj].z, v[u][jj].w};
              const float2 c0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&wv[0]));
              const float2 c1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&wv[1]));
              const float2 c2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&wv[2]));
              const float2 c3 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&wv[3]));
              float t = acc[jj];
              t = fmaf(u0.x, c0.x, t); t = fmaf(u0.y, c0.y, t); t = fmaf(u0.z, c1.x, t); t = fmaf(u0.w, c1.y, t);
              t = fmaf(u1.x, c2.x, t); t = fmaf(u1.y, c2.y, t); t = fmaf(u1.z, c3.x, t); t = fmaf(u1.w, c3.y, t);
              acc[jj] = t;
            }
          }
        }
      }
    }
#pragma unroll
    for (int jj = 0; jj < JB; ++jj) {
      float t = acc[jj];
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) t += __shfl_xor_sync(0xffffffffu, t, off);
      if (lane == 0 && j0 + jj < t2) z[(long)b * t2 + j0 + jj] = __float2bfloat16_rn(t);
    }
  }
}

}  // namespace dec
}  // namespace ta
