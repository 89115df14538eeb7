// Decode attention over the latent KV cache (Eq. 9) on tcgen05 tensor cores.
//
// Streams every sequence's latent K / V cache exactly once.  All n_H (<= 32) heads share each K / V byte, so the
// arithmetic is 2 n_H flop per cached element: beyond plain FMA throughput at HBM speed, hence tensor cores.  The
// two products of a 128-key tile run as UMMA instructions with the KEYS on the M dimension, so that
// no tensor work is spent on padding the (at most 32) heads up to a 128-row tile:
//   S^T [128 keys x 32 heads] = K_tile [128 x r3] * Qhat^T          A = K tile as loaded (K-major), B = Qhat (K-major)
//   O^T [t3 x 32 heads]      += V_tile^T [t3 x 128] * P [128 x 32]  A = V tile as loaded (M-major), B = P (K-major, bf16)
// The scores of one tile sit in TMEM with one key per lane and one head per column.  NWG softmax
// warpgroups work on EVERY tile, each on HPW = 32 / NWG of the 32 head columns: a thread owns one key and
// HPW heads (the per-tile work of a thread is a latency chain, so more, thinner threads finish a tile sooner).
// The per-head maximum over the keys of a tile is a reduction ACROSS threads (a transposing butterfly of
// warp shuffles, then four values per head through shared memory); it only moves the reference maximum
// of a head when that grows by more than 8 (factor 256), so the accumulator in TMEM is rescaled rarely.
// P goes back through shared memory (B operands are read from there); the row sums stay in registers
// per thread and are reduced once per segment.  Score and P buffers are double-buffered, the output
// accumulator is single: tile t + 1 is scored and exponentiated while P V of tile t runs, and a segment
// ends with each warpgroup writing its heads of the partial (max, sum, unnormalised O) of (CTA, sequence).
//
//   warp 0       TMA producer: Qhat of the segment's sequence, K / V ring
//   warp 1       TMEM allocation, MMA issue
//   warps 4 + 4 g .. 7 + 4 g   softmax warpgroup g (heads HPW g .. HPW g + HPW - 1)
// TMEM columns: S_0 [0,32) S_1 [32,64) O [64,96).
// Every wait is bounded (Abort): on a timeout the CTA raises the device error word and leaves.
//
// ROT = true: one shared latent cache L^KV (Sec. 3.1) together with latent RoPE (Definition 2).  The cache then
// holds UN-rotated rows: the value side uses a tile as it was loaded, and a fourth warpgroup (thread = key
// row = TMEM lane) writes the rotated copy K_n R(n, r3) of every tile into TMEM (bf16 pairs, columns
// [128, 256), two buffers), from where it feeds the score product as the A operand.
// cos / sin of n theta_i = (k0 + row) theta_i come by angle addition from the thread's own constants for `row`
// (registers) and the tile's 64 base values for k0 (formed per tile with the angle reduced in double precision).
//   warps 12..15  rotation warpgroup (ROT only)
#pragma once

#include "ta_common.cuh"
#include "ta_decode.cuh"
#include "ta_sm100.cuh"

namespace ta {
namespace decu {

using namespace sm100;
using dec::clamp_len;
using dec::tiles_of;

constexpr int TK = 128;                  // keys per tile
constexpr int NWG = 2;                    // softmax warpgroups (4 was measured: slower, 138 us against 118 us with the shared cache)
constexpr int HPW = 32 / NWG;             // head columns per warpgroup
constexpr int THREADS = 128 + 128 * NWG;
constexpr int THREADS_ROT = THREADS + 128;           // plus the rotation warpgroup
constexpr uint32_t TMEM_KROT = 128;                   // first TMEM column of the two rotated key tiles (64 columns each)
constexpr int MAX_STAGES = 6;
constexpr int SUB_BYTES = 128 * 64 * 2;  // [128 keys x 64] bf16
constexpr int MAX_SUB = 2;               // r3, t3 <= 128
constexpr int STAGE_BYTES = 2 * MAX_SUB * SUB_BYTES;   // K tile + V tile
constexpr int QSUB_BYTES = 32 * 64 * 2;  // [32 heads x 64] bf16 (Qhat and P sub-tiles)
constexpr int QBUF_BYTES = MAX_SUB * QSUB_BYTES;
constexpr int PBUF_BYTES = 2 * QSUB_BYTES;             // [32 heads x 128 keys] bf16
constexpr int RING_BYTES = 3 * STAGE_BYTES;            // three K + V stages, or six K-only stages (shared cache)
// ring | Qhat (two segments in flight) | P_0 | P_1
constexpr size_t SMEM_BYTES = 1024 + (size_t)RING_BYTES + 2 * QBUF_BYTES + 2 * PBUF_BYTES;
constexpr float kRescaleThreshold = 8.f;

struct Params {
  int B, nH, Lmax, r3, t3;
  int shared_kv;       // 1: one latent cache L^KV (Sec. 3.1): the K tile is the V tile
  const int32_t* cache_len;
  const bf16* knew;    // [B, r3] rotated new key
  const bf16* vnew;    // [B, t3] new value
  float* part_o;       // [grid + B][32][t3]
  float* part_ml;      // [grid + B][32][2]  (max in log2 units, sum)
  unsigned int* err;
};

// Walks this CTA's range of the flat tile list, sequence by sequence.
struct Walk {
  const int32_t* cache_len;
  int Lmax;
  long t_begin, t_end;
  int b;
  long first, nt;
  int L;
  __device__ void init(const Params& p, long tb, long te, int b0, long first0) {
    cache_len = p.cache_len; Lmax = p.Lmax; t_begin = tb; t_end = te;
    b = b0; first = first0;
    L = clamp_len(cache_len[b], Lmax);
    nt = tiles_of(L);
  }
  __device__ void seek(long t) {
    while (t >= first + nt) {
      first += nt;
      ++b;
      L = clamp_len(cache_len[b], Lmax);
      nt = tiles_of(L);
    }
  }
  __device__ bool seg_start(long t) const { return t == t_begin || t == first; }
  __device__ bool seg_end(long t) const { return t == t_end - 1 || t == first + nt - 1; }
  __device__ int k0(long t) const { return (int)(t - first) * TK; }
  __device__ bool last_tile(long t) const { return k0(t) + TK > L; }
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// maximum of x over the 32 lanes of the warp, in every lane (one instruction)
__device__ __forceinline__ float warp_max(float x) {
  float r;
  asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ uint32_t swz(int row, int chunk) {
  return (uint32_t)((chunk >> 3) * SUB_BYTES + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

// sum of x over the 32 lanes of the warp, in every lane
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
  return x;
}

template <int N> struct TmemCols;
template <> struct TmemCols<16> {
  static __device__ __forceinline__ void ld(uint32_t a, uint32_t (&r)[16]) { tmem_ld16(a, r); }
  static __device__ __forceinline__ void st(uint32_t a, const uint32_t (&r)[16]) { tmem_st16(a, r); }
};
template <> struct TmemCols<8> {
  static __device__ __forceinline__ void ld(uint32_t a, uint32_t (&r)[8]) { tmem_ld8(a, r); }
  static __device__ __forceinline__ void st(uint32_t a, const uint32_t (&r)[8]) { tmem_st8(a, r); }
};

template <bool ROT, int R3C>
__global__ void __launch_bounds__(ROT ? THREADS_ROT : THREADS, 1)
k_dec_attn_umma(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                const __grid_constant__ CUtensorMap tmQ, const Params p, const dec::RopeFreqs freqs) {
  // cache_len was final before the preceding kernel (which forms the queries and appends the new row)
  // began: set-up and the tile split run while it finishes, and every role passes pdl_enter() before it
  // touches anything else.  (Requesting the first cache tiles ahead of that wait as well was measured:
  // no gain with two caches, 6 us slower with the shared cache.)
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t full_bar[MAX_STAGES], empty_bar[MAX_STAGES], q_full[2], q_empty[2];
  __shared__ uint64_t s_full[2], s_free[2], p_full[2], p_free[2], o_read, patched, wg_bar[NWG];
  __shared__ uint64_t kr_full[2], kr_free[2];        // ROT: rotated key tile written / consumed by the score product
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  // per tile: the four warps' maxima per head of each warpgroup, as bf16 (the reference maximum only has
  // to be the same for all threads and close to the true one), double-buffered by tile parity because a
  // warp may start the next tile while another still reads this one's; per segment: the warps' row sums
  __shared__ __align__(16) __nv_bfloat16 mxh[NWG][2][4][HPW];   // [wg][tile parity][warp][head]
  __shared__ float sum_s[NWG][4][HPW];                          // [wg][warp][head]
  __shared__ long long wtot_s[THREADS_ROT / 32];
  __shared__ int loc_b;
  __shared__ long long loc_first;

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* ring = smem_raw + (base - smem_u32(smem_raw));
  uint8_t* qbuf = ring + (size_t)RING_BYTES;
  uint8_t* pbuf = qbuf + 2 * QBUF_BYTES;
  // With one shared latent cache a stage holds a K tile only: twice the stages.
  const int STAGES = p.shared_kv ? 6 : 3;
  const int stage_bytes = p.shared_kv ? MAX_SUB * SUB_BYTES : STAGE_BYTES;

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  Abort ab{&abort_flag, p.err};
  const int ksub = (p.r3 + 63) / 64, vsub = (p.t3 + 63) / 64;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < MAX_STAGES; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&q_full[i], 1);
      mbar_init(&q_empty[i], 1);
      mbar_init(&s_full[i], 1);
      mbar_init(&s_free[i], 4 * NWG);   // the scores are in registers: one arrival per softmax warp
      mbar_init(&p_full[i], 4 * NWG);   // P is in shared memory: one arrival per softmax warp
      mbar_init(&p_free[i], 1);         // the P V product that read this P buffer is complete
    }
    for (int i = 0; i < NWG; ++i) mbar_init(&wg_bar[i], 4);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&kr_full[i], 4);        // one arrival per rotation warp
      mbar_init(&kr_free[i], 1);
    }
    mbar_init(&o_read, 4 * NWG);
    mbar_init(&patched, 4);
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(&tmem_slot, ROT ? 256 : 128);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_slot;
  const uint32_t tm_o = tmem + 64;

  // ---- this CTA's range of the flat tile list ----
  int lo, hi;
  long excl;
  const long total = dec::block_tile_scan(p.cache_len, p.B, p.Lmax, lo, hi, excl, wtot_s);
  const long t_begin = dec::cta_first_tile(blockIdx.x, total, gridDim.x);
  const long t_end = dec::cta_first_tile(blockIdx.x + 1, total, gridDim.x);
  {
    long f = excl;
    for (int b = lo; b < hi; ++b) {
      const long nt = tiles_of(clamp_len(p.cache_len[b], p.Lmax));
      if (t_begin >= f && t_begin < f + nt) { loc_b = b; loc_first = f; }
      f += nt;
    }
  }
  __syncthreads();
  const bool have_work = t_begin < t_end;
  const int b0 = have_work ? loc_b : 0;
  const long seq_first = have_work ? (long)loc_first : 0;

  if (warp < 4) {
   asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
   if (have_work && warp == 0) {
    // ------------------------------- TMA producer -------------------------------
    if (elect_one()) {
      tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmQ);
      Walk w;
      w.init(p, t_begin, t_end, b0, seq_first);
      auto load_tile = [&](long t, int s) {     // K / V tile t (w is positioned on it) into ring stage s
        mbar_expect_tx(&full_bar[s], (uint32_t)((ksub + (p.shared_kv ? 0 : vsub)) * SUB_BYTES));
        uint8_t* kt = ring + (size_t)s * stage_bytes;
        uint8_t* vt = kt + MAX_SUB * SUB_BYTES;
        const int row = w.k0(t);
        for (int kk = 0; kk < ksub; ++kk) tma_load_3d(kt + kk * SUB_BYTES, &tmK, &full_bar[s], kk * 64, row, w.b);
        if (!p.shared_kv)
          for (int kk = 0; kk < vsub; ++kk) tma_load_3d(vt + kk * SUB_BYTES, &tmV, &full_bar[s], kk * 64, row, w.b);
      };
      pdl_enter();
      int it = 0, seg = -1;
      for (long t = t_begin; t < t_end; ++t, ++it) {
        w.seek(t);
        if (w.seg_start(t)) {
          ++seg;
          const int qb = seg & 1;
          if (!mbar_wait(&q_empty[qb], ((seg >> 1) & 1) ^ 1, ab)) break;
          mbar_expect_tx(&q_full[qb], (uint32_t)(ksub * QSUB_BYTES));
          for (int kk = 0; kk < ksub; ++kk)
            tma_load_2d(qbuf + qb * QBUF_BYTES + kk * QSUB_BYTES, &tmQ, &q_full[qb], kk * 64, w.b * p.nH);
        }
        const int s = it % STAGES;
        if (!mbar_wait(&empty_bar[s], ((it / STAGES) & 1) ^ 1, ab)) break;
        load_tile(t, s);
      }
    } else {
      pdl_enter();
    }
   } else if (have_work && warp == 1) {
    // ------------------------------- MMA issuer ---------------------------------
    pdl_enter();
    if (elect_one()) {
      // This one thread issues 16 small MMAs per tile, so its own instruction stream matters: descriptors
      // are formed once per operand and stepped by constants, the K loops are unrolled, and the (at most
      // two) tiles between score issue and P V issue sit in registers.
      const uint32_t idesc_qk = umma_idesc_bf16(128, 32);
      const uint32_t idesc_pv = umma_idesc_bf16(128, 32) | (1u << 15);   // A = V tile is M-major
      const int ksteps = p.r3 / 16;
      const uint64_t dq0 = umma_desc_kmajor_sw128(smem_u32(qbuf));
      const uint64_t dp0 = umma_desc_kmajor_sw128(smem_u32(pbuf));
      const uint64_t dk0 = umma_desc_kmajor_sw128(smem_u32(ring));
      const uint64_t dv0 = umma_desc_mnmajor_sw128(smem_u32(ring) + (p.shared_kv ? 0u : (uint32_t)(MAX_SUB * SUB_BYTES)), SUB_BYTES);
      const uint64_t stage_step = (uint64_t)(stage_bytes >> 4);          // descriptor address fields count 16 bytes
      // pending P V products, oldest first; a tile's state in one word: it << 8 | stage << 4 | first tile of its segment
      uint32_t pq0 = 0, pq1 = 0;
      int pv_seg0 = 0, pv_seg1 = 0, n_pend = 0;
      bool ok = true;
      auto issue_pv = [&](uint32_t code, int sg) -> bool {
        const int it = (int)(code >> 8), st = (int)((code >> 4) & 15), buf = it & 1;
        const bool first = (code & 1u) != 0;
        if (!mbar_wait(&p_full[buf], (uint32_t)((it >> 1) & 1), ab)) return false;
        // the accumulator of the previous segment must have been read before it is overwritten
        if (first && sg > 0 && !mbar_wait(&o_read, (uint32_t)((sg - 1) & 1), ab)) return false;
        tc_fence_after();
        const uint64_t dv = dv0 + stage_step * (uint64_t)st;
        const uint64_t dp = dp0 + (uint64_t)(buf * (PBUF_BYTES >> 4));
        umma_ss(tm_o, dv, dp, idesc_pv, first ? 0u : 1u);
#pragma unroll
        for (int ks = 1; ks < TK / 16; ++ks)
          umma_ss(tm_o, dv + (uint64_t)(ks * 128), dp + (uint64_t)((ks >> 2) * (QSUB_BYTES >> 4) + (ks & 3) * 2), idesc_pv, 1u);
        umma_commit(&p_free[buf]);
        umma_commit(&empty_bar[st]);
        return true;
      };
      auto pop_pv = [&]() -> bool {
        const bool good = issue_pv(pq0, pv_seg0);
        pq0 = pq1; pv_seg0 = pv_seg1;
        --n_pend;
        return good;
      };
      Walk w;
      w.init(p, t_begin, t_end, b0, seq_first);
      const int n_tiles = (int)(t_end - t_begin);
      int seg = -1, st = 0, n_last = 0;
      uint32_t st_par = 0;
      for (int it = 0; it < n_tiles && ok; ++it) {
        while (n_pend > 1 && ok) ok = pop_pv();      // the scores run one tile ahead of the P V products
        if (!ok) break;
        const long t = t_begin + it;
        w.seek(t);
        const int buf = it & 1, j = it >> 1;
        const bool first = w.seg_start(t);
        if (first) {
          ++seg;
          if (!(ok = mbar_wait(&q_full[seg & 1], (uint32_t)((seg >> 1) & 1), ab))) break;
        }
        if (ROT) {
          // the rotation warpgroup has seen the tile arrive, written its rotated copy and (last tile of a
          // sequence) patched the new token's row into both
          if (!(ok = mbar_wait(&kr_full[buf], (uint32_t)(j & 1), ab))) break;
        } else if (!(ok = mbar_wait(&full_bar[st], st_par, ab))) break;
        if (!ROT && w.last_tile(t)) {
          // Warpgroup 0 patches this tile only after it has flushed the segments before it, and such a
          // flush waits for every P V issued so far: issue the pending ones first.
          while (n_pend > 0 && ok) ok = pop_pv();
          if (!ok) break;
          if (!(ok = mbar_wait(&patched, (uint32_t)(n_last & 1), ab))) break;
          ++n_last;
        }
        // both warpgroups have taken the scores of tile it - 2 out of this buffer
        if (j > 0 && !(ok = mbar_wait(&s_free[buf], (uint32_t)((j - 1) & 1), ab))) break;
        tc_fence_after();
        {
          const uint64_t dk = dk0 + stage_step * (uint64_t)st;
          const uint64_t dq = dq0 + (uint64_t)((seg & 1) * (QBUF_BYTES >> 4));
          const uint32_t d = tmem + (uint32_t)buf * 32u;
          const uint32_t akr = tmem + TMEM_KROT + (uint32_t)buf * 64u;    // ROT: the rotated key tile, 8 columns per K step
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            if (ks < ksteps) {
              const uint64_t dqk = dq + (uint64_t)((ks >> 2) * (QSUB_BYTES >> 4) + (ks & 3) * 2);
              if (ROT) umma_ts(d, akr + (uint32_t)ks * 8u, dqk, idesc_qk, ks != 0 ? 1u : 0u);
              else umma_ss(d, dk + (uint64_t)((ks >> 2) * (SUB_BYTES >> 4) + (ks & 3) * 2), dqk, idesc_qk, ks != 0 ? 1u : 0u);
            }
          umma_commit(&s_full[buf]);
          if (ROT) umma_commit(&kr_free[buf]);
          if (w.seg_end(t)) umma_commit(&q_empty[seg & 1]);   // the segment's Qhat buffer is free once these complete
        }
        {
          const uint32_t code = ((uint32_t)it << 8) | ((uint32_t)st << 4) | (first ? 1u : 0u);
          if (n_pend == 0) { pq0 = code; pv_seg0 = seg; } else { pq1 = code; pv_seg1 = seg; }
          ++n_pend;
        }
        if (++st == STAGES) { st = 0; st_par ^= 1u; }
      }
      while (ok && n_pend > 0) ok = pop_pv();
    }
   }
  } else {
   // setmaxnreg.inc blocks until the registers exist: the request must fit the pool the CTA was launched
   // with (registers at launch x threads) minus what the first warpgroup keeps.  2 warpgroups: 168 x 384
   // = 64512 = 128 x 56 + 256 x 224.  4 warpgroups: 96 x 640 = 61440 >= 128 x 56 + 512 x 104 = 60416.
   static_assert(NWG == 2 || NWG == 4, "register budgets below are written for 2 or 4 softmax warpgroups");
   // ROT (512 threads, 128 registers at launch): 128 x 56 + 256 x 128 (unchanged) + 128 x 200 = 65536.
   if (ROT && warp >= 12) asm volatile("setmaxnreg.inc.sync.aligned.u32 200;");
   else if (ROT) { }
   else if (NWG == 2) asm volatile("setmaxnreg.inc.sync.aligned.u32 224;");
   else asm volatile("setmaxnreg.inc.sync.aligned.u32 104;");
   if (ROT && warp >= 12) {
    if (have_work) {
     pdl_enter();
     // ------------------------------- rotation warpgroup --------------------------
     constexpr int HALF = R3C / 2;                // coordinate pairs per row
     const int q = warp - 12;
     const int tid = q * 32 + lane;              // key row of a tile
     float ac[HALF > 0 ? HALF : 1], as_[HALF > 0 ? HALF : 1];   // (cos, sin)(tid theta_i)
#pragma unroll
     for (int i = 0; i < HALF; ++i) {
       const float2 cs = dec::rope_cos_sin_theta(tid, freqs.theta[i]);
       ac[i] = cs.x; as_[i] = cs.y;
     }
     auto wait_all = [&](uint64_t* bar, uint32_t parity) -> bool {
       bool good = mbar_wait(bar, parity, ab);
       return __all_sync(0xffffffffu, good);
     };
     const float2 step_lo = dec::rope_cos_sin_theta(TK, freqs.theta[lane]);
     const float2 step_hi = dec::rope_cos_sin_theta(TK, freqs.theta[32 + (lane & 31)]);
     float2 base_lo = make_float2(1.f, 0.f), base_hi = make_float2(1.f, 0.f);
     Walk w;
     w.init(p, t_begin, t_end, b0, seq_first);
     int it = 0;
     bool ok = true;
     for (long t = t_begin; t < t_end && ok; ++t, ++it) {
       w.seek(t);
       const int s = it % STAGES, buf = it & 1, j = it >> 1;
       if (!(ok = wait_all(&full_bar[s], (uint32_t)((it / STAGES) & 1)))) break;
       if (j > 0 && !(ok = wait_all(&kr_free[buf], (uint32_t)((j - 1) & 1)))) break;   // score product of tile it - 2 is done
       tc_fence_after();
       const int k0 = w.k0(t);
       // (cos, sin)(k0 theta_i) of this tile: lane l holds the values of pairs l and l + 32; they reach the
       // other lanes by shuffles (all lanes of a warp work on the same pair index at the same time).  At the
       // first tile of a segment they are formed with the angle reduced in double precision; from tile to tile
       // they advance by the rotation through 128 theta_i (at most 256 steps of 1e-7 each: far below bf16).
       if (w.seg_start(t)) {
         base_lo = dec::rope_cos_sin_theta(k0, freqs.theta[lane]);
         base_hi = (HALF > 32) ? dec::rope_cos_sin_theta(k0, freqs.theta[32 + (lane & 31)]) : make_float2(1.f, 0.f);
       } else {
         base_lo = make_float2(base_lo.x * step_lo.x - base_lo.y * step_lo.y, base_lo.y * step_lo.x + base_lo.x * step_lo.y);
         base_hi = make_float2(base_hi.x * step_hi.x - base_hi.y * step_hi.y, base_hi.y * step_hi.x + base_hi.x * step_hi.y);
       }
       uint8_t* raw = ring + (size_t)s * stage_bytes;
       const bool last = w.last_tile(t);
       const int rnew = w.L - k0;               // row of the new token (last tile of a sequence only)
       const bool is_new = last && tid == rnew;
       const uint32_t kaddr = tmem + TMEM_KROT + (uint32_t)buf * 64u + ((uint32_t)(q * 32) << 16);
#pragma unroll
       for (int hf = 0; hf < 2; ++hf) {         // 32 TMEM columns = 64 coordinates at a time
         if (hf * 64 < R3C) {
           uint32_t o[32];
#pragma unroll
           for (int cc = 0; cc < 8; ++cc) {
             const int c = hf * 8 + cc;         // 16-byte chunk of the row
             if (c < R3C / 8) {
               const uint4 v = *reinterpret_cast<const uint4*>(raw + swz(tid, c));
               const uint32_t wv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
               for (int e = 0; e < 4; ++e) {
                 const int i = 4 * c + e;
                 const float2 x = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&wv[e]));
                 const float2 bs = make_float2(__shfl_sync(0xffffffffu, i < 32 ? base_lo.x : base_hi.x, i & 31),
                                               __shfl_sync(0xffffffffu, i < 32 ? base_lo.y : base_hi.y, i & 31));
                 const float cs_c = ac[i] * bs.x - as_[i] * bs.y, cs_s = as_[i] * bs.x + ac[i] * bs.y;   // angle addition
                 const uint32_t rot = pack_bf16(x.x * cs_c - x.y * cs_s, x.x * cs_s + x.y * cs_c);
                 o[4 * cc + e] = rot;
               }
             } else {
#pragma unroll
               for (int e = 0; e < 4; ++e) o[4 * cc + e] = 0u;
             }
           }
           if (is_new) {
             // the new token's rotated key comes from the workspace
             const uint4* kn = reinterpret_cast<const uint4*>(p.knew + (long)w.b * p.r3) + hf * 8;
#pragma unroll
             for (int cc = 0; cc < 8; ++cc)
               if (hf * 8 + cc < R3C / 8) {
                 const uint4 v = kn[cc];
                 o[4 * cc] = v.x; o[4 * cc + 1] = v.y; o[4 * cc + 2] = v.z; o[4 * cc + 3] = v.w;
               }
           }
           tmem_st32(kaddr + (uint32_t)hf * 32u, o);
         }
       }
       tmem_st_wait();
       if (last) {
         // as VALUES the new token's un-rotated latent row comes from the workspace and rows past it must be
         // zero (their probabilities are zero, but the slots may hold anything)
         if (tid == rnew) {
           const uint4* vs = reinterpret_cast<const uint4*>(p.vnew + (long)w.b * p.t3);
           for (int c = 0; c < R3C / 8; ++c) *reinterpret_cast<uint4*>(raw + swz(tid, c)) = vs[c];
         } else if (tid > rnew) {
           for (int c = 0; c < R3C / 8; ++c) *reinterpret_cast<uint4*>(raw + swz(tid, c)) = make_uint4(0u, 0u, 0u, 0u);
         }
       }
       tc_fence_before();
       fence_proxy_async_smem();
       __syncwarp();
       if (lane == 0) mbar_arrive(&kr_full[buf]);
     }
    }
   } else if (have_work) {
    pdl_enter();
    // ------------------------------- softmax warpgroups --------------------------
    const int wg = (warp - 4) / 4;              // heads [HPW wg, HPW wg + HPW)
    const int q = warp % 4;                     // TMEM lane quadrant
    const int tid = q * 32 + lane;              // key row of a score tile / value coordinate of O^T
    const int hl = lane % HPW;                  // the head (within the group) whose maxima this lane combines
    const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
    // this thread's P element of head HPW wg + j lives at p_row0 + j * 128 + ((p_chunk ^ (j & 7)) << 4) in a P buffer
    const uint32_t p_row0 = (uint32_t)(tid >> 6) * QSUB_BYTES + (uint32_t)(wg * HPW) * 128 + (uint32_t)(tid & 7) * 2;
    const int p_chunk = (tid & 63) >> 3;        // (HPW wg + j) & 7 == j & 7 (HPW is a multiple of 8)
    uint32_t p_sw[8];                           // offset of head row j (mod 8) incl. the 128-byte swizzle
#pragma unroll
    for (int e = 0; e < 8; ++e) p_sw[e] = (uint32_t)(e * 128 + ((p_chunk ^ e) << 4));
    uint32_t wg_phase = 0;
    bool ok = true;
    auto wg_sync = [&]() -> bool {
      __syncwarp();
      if (lane == 0) mbar_arrive(&wg_bar[wg]);
      bool good = mbar_wait(&wg_bar[wg], wg_phase & 1, ab);
      ++wg_phase;
      return __all_sync(0xffffffffu, good);
    };
    auto wait_all = [&](uint64_t* bar, uint32_t parity) -> bool {
      bool good = mbar_wait(bar, parity, ab);
      return __all_sync(0xffffffffu, good);
    };
    Walk w;
    w.init(p, t_begin, t_end, b0, seq_first);
    int it = 0, n_seen = 0;    // tiles of the current segment handled so far
    float m_used[HPW], l_acc[HPW];
    float m_lane = -INFINITY;  // m_used[hl]
    for (long t = t_begin; t < t_end && ok; ++t, ++it) {
      w.seek(t);
      if (w.seg_start(t)) {
        n_seen = 0;
        m_lane = -INFINITY;
#pragma unroll
        for (int h = 0; h < HPW; ++h) { m_used[h] = -INFINITY; l_acc[h] = 0.f; }
      }
      const int buf = it & 1, j = it >> 1;
      const int k0 = w.k0(t), L = w.L;
      const bool last_tile = w.last_tile(t);
      if (!ROT && last_tile && wg == 0) {
        const int s = it % STAGES;
        // the tile holding the new token: its row comes from the workspace, rows past it are invalid
        if (!(ok = wait_all(&full_bar[s], (uint32_t)((it / STAGES) & 1)))) break;
        uint8_t* kt = ring + (size_t)s * stage_bytes;
        uint8_t* vt = p.shared_kv ? kt : kt + MAX_SUB * SUB_BYTES;
        const int rnew = L - k0;
        if (tid == rnew) {
          const uint4* ks = reinterpret_cast<const uint4*>(p.knew + (long)w.b * p.r3);
          for (int c = 0; c < p.r3 / 8; ++c) *reinterpret_cast<uint4*>(kt + swz(tid, c)) = ks[c];
          const uint4* vs = reinterpret_cast<const uint4*>(p.vnew + (long)w.b * p.t3);
          for (int c = 0; c < p.t3 / 8; ++c) *reinterpret_cast<uint4*>(vt + swz(tid, c)) = vs[c];
        } else if (tid > rnew) {
          for (int c = 0; c < p.t3 / 8; ++c) *reinterpret_cast<uint4*>(vt + swz(tid, c)) = make_uint4(0u, 0u, 0u, 0u);
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&patched);
      }
      if (!(ok = wait_all(&s_full[buf], (uint32_t)(j & 1)))) break;
      tc_fence_after();
      uint32_t sr[HPW];
      TmemCols<HPW>::ld(tmem + (uint32_t)buf * 32u + (uint32_t)(wg * HPW) + lane_addr, sr);
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&s_free[buf]);       // the scores of tile it + 2 may overwrite the buffer
      float sc[HPW];
#pragma unroll
      for (int h = 0; h < HPW; ++h) sc[h] = __uint_as_float(sr[h]);
      if (last_tile && (k0 + tid) > L) {       // keys past the new token do not exist
#pragma unroll
        for (int h = 0; h < HPW; ++h) sc[h] = -INFINITY;
      }
      // ---- maximum per head over the 128 keys of the tile: one warp-wide max per head, lane 0 publishes ----
      {
        uint32_t pk[HPW / 2];
#pragma unroll
        for (int h = 0; h < HPW; h += 2) pk[h >> 1] = pack_bf16(warp_max(sc[h]), warp_max(sc[h + 1]));
        if (lane == 0) {
          uint4* dst = reinterpret_cast<uint4*>(&mxh[wg][buf][q][0]);
#pragma unroll
          for (int u = 0; u < HPW / 8; ++u) dst[u] = make_uint4(pk[4 * u], pk[4 * u + 1], pk[4 * u + 2], pk[4 * u + 3]);
        }
      }
      if (!(ok = wg_sync())) break;
      const float mt = fmaxf(fmaxf(__bfloat162float(mxh[wg][buf][0][hl]), __bfloat162float(mxh[wg][buf][1][hl])),
                             fmaxf(__bfloat162float(mxh[wg][buf][2][hl]), __bfloat162float(mxh[wg][buf][3][hl])));
      // every tile holds at least one visible key (the last one holds the new token), so mt is finite
      const bool need = mt > m_lane + kRescaleThreshold;
      if (__any_sync(0xffffffffu, need)) {
        const float m_new = need ? mt : m_lane;
        const float f_lane = need ? ex2(m_lane - m_new) : 1.f;     // exp2(-inf) = 0 on the first tile
        float fac[HPW];
#pragma unroll
        for (int h = 0; h < HPW; ++h) {
          fac[h] = __shfl_sync(0xffffffffu, f_lane, h);
          m_used[h] = __shfl_sync(0xffffffffu, m_new, h);
          l_acc[h] *= fac[h];
        }
        m_lane = m_new;
        if (n_seen > 0) {
          // P V of the previous tile must be complete before its accumulator columns are rescaled
          if (!(ok = wait_all(&p_free[(it - 1) & 1], (uint32_t)(((it - 1) >> 1) & 1)))) break;
          tc_fence_after();
          uint32_t o[HPW];
          TmemCols<HPW>::ld(tm_o + (uint32_t)(wg * HPW) + lane_addr, o);
          tmem_ld_wait();
#pragma unroll
          for (int h = 0; h < HPW; ++h) o[h] = __float_as_uint(__uint_as_float(o[h]) * fac[h]);
          TmemCols<HPW>::st(tm_o + (uint32_t)(wg * HPW) + lane_addr, o);
          tmem_st_wait();
        }
      }
      // the P V product of tile it - 2 must have finished reading this P buffer
      if (j > 0 && !(ok = wait_all(&p_free[buf], (uint32_t)((j - 1) & 1)))) break;
      // ---- p = exp2(s - m), bf16, into the P operand; row sums per thread ----
      {
        uint8_t* my_p = pbuf + buf * PBUF_BYTES + p_row0;
#pragma unroll
        for (int h = 0; h < HPW; ++h) {
          const float pv = ex2(sc[h] - m_used[h]);
          l_acc[h] += pv;
          *reinterpret_cast<__nv_bfloat16*>(my_p + (h >> 3) * 1024 + p_sw[h & 7]) = __float2bfloat16_rn(pv);
        }
      }
      fence_proxy_async_smem();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&p_full[buf]);
      ++n_seen;
      if (w.seg_end(t)) {
        // ---- segment done: this warpgroup's 16 heads of the partial of (CTA, sequence) ----
        if (!(ok = wait_all(&p_free[buf], (uint32_t)(j & 1)))) break;      // P V of this tile is complete
        tc_fence_after();
        uint32_t o[HPW];
        TmemCols<HPW>::ld(tm_o + (uint32_t)(wg * HPW) + lane_addr, o);
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&o_read);       // the next segment may overwrite the accumulator
#pragma unroll
        for (int h = 0; h < HPW; ++h) {
          const float ws = warp_sum(l_acc[h]);       // row sums over this warp's 32 keys
          if (lane == h) sum_s[wg][q][h] = ws;
        }
        if (!(ok = wg_sync())) break;
        const long slot = (long)blockIdx.x + w.b;
        // one partial slot per (CTA, sequence) pair that can occur: gridDim.x + B of them
        const bool slot_ok = TA_IDX_OK(p.err, slot, 1, (long)gridDim.x + p.B);
        if (slot_ok && q == 0 && lane < HPW) {
          float* ml = p.part_ml + slot * 64 + (wg * HPW + lane) * 2;
          ml[0] = m_lane;
          ml[1] = sum_s[wg][0][lane] + sum_s[wg][1][lane] + sum_s[wg][2][lane] + sum_s[wg][3][lane];
        }
        if (slot_ok && tid < p.t3) {
          float* dst = p.part_o + slot * 32 * p.t3 + (long)(wg * HPW) * p.t3 + tid;
#pragma unroll
          for (int h = 0; h < HPW; ++h) dst[h * p.t3] = __uint_as_float(o[h]);
        }
        if (!(ok = wg_sync())) break;      // sum_s is free again before the next segment's flush writes it
      }
    }
   }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, ROT ? 256 : 128);
}

}  // namespace decu
}  // namespace ta
