// Flash-style attention over the latent K / V pair on tcgen05 tensor cores (Sec. 3.3 of the
// paper: online softmax over key chunks, one K/V chunk pair shared by all heads), with the
// per-head latent queries of Definition 2 formed inside the kernel.
//
// A work item = (sequence b, 128 query rows, a run of head pairs).  The grid is persistent: one CTA per SM walks
// the items blockIdx.x, 2 G - 1 - blockIdx.x, 2 G + blockIdx.x, ... of the list ordered heaviest first (G = grid
// size; the back-and-forth order evens out the causal items' sizes), so that a CTA's start-up (TMEM allocation,
// barriers, first loads: about 3 us) is paid once per SM and the next item's tiles are already on their way
// while the current item finishes.  For every head pair (h, h+1) of an item's run:
//   prologue   Qhat_i = Qt G_{h+i} on the tensor core (Qt tile loaded once per CTA, G tiles
//              streamed through the V ring), latent RoPE applied while the result moves
//              TMEM -> registers -> shared memory (bf16, the swizzled K-major layout UMMA reads)
//   main loop  both heads use the same latent K / V tiles, so every tile is loaded once and serves two score
//              tiles.  The score tiles of the pair are produced in the order (key tile j, head i) -> t = 2 j + i
//              into ONE score buffer: as soon as the softmax warpgroup of tile t holds it in registers, tile
//              t + 1 (the other head's) is issued, so a warpgroup that finishes a tile finds its next scores
//              ready, and the two warpgroups' exponentials overlap instead of waiting for each other's MMAs
//   epilogue   O_i / l as bf16 into the head's idle Qhat tile, then out by a TMA tensor store that
//              completes in the background while the warpgroup starts on the next head pair
// In the unfused mode (query rank r2 > 128: the Qt tile would not fit) Qhat is read from
// global memory instead and a CTA handles a single head pair.
//
//   warp 0        TMA producer: Qt (once per item), G tiles, K ring, V ring
//   warp 1        score issuer: S = Qhat_i K^T (smem x smem)
//   warp 2        value issuer: Qhat_i = Qt G_i^T, O_i += P_i V (P from TMEM, V^T tile K-major from shared memory)
//   warps 4..7    softmax for head h   : thread t owns query row t (TMEM lane t)
//   warps 8..11   softmax for head h+1
// Two issuing threads, because an issuing thread is held until the tensor core has accepted its MMAs; the value
// issuer lets a score tile that is ready at the same time go first (the tensor core runs MMAs in issue order, and
// an idle warpgroup waits for the scores while nobody waits for the P V product).
//
// The value tile comes from the transposed latent values V^T [B, t3, N] (written by the projection kernel), so
// that both MMAs read K-major operands (an MN-major B operand costs about 40 cycles more per instruction).
//
// TMEM columns: S [0,128)  P_0 [128,192)  P_1 [192,256) (bf16, two per column)  O_0 [256,256+t3)  O_1 [384,384+t3);
// the prologue's Qhat_0 / Qhat_1 accumulators occupy S and P_0|P_1.  Scores arrive in log2 units (softmax scale *
// log2 e is folded into G_h), so exp2 is used.  The running maximum is only raised when it grows by more than 8
// (factor 256), which keeps the O rescaling off the common path; l and O stay consistent
// because both use the same stale maximum.
#pragma once

#include "ta_common.cuh"
#include "ta_sm100.cuh"

// Which of every eight consecutive score pairs of a row take their exponential on the FMA pipe instead of the
// MUFU unit (bit c & 7); a build-time option, none by default.  Measured on the long causal prefill (attention
// kernel, CUDA events).  With one score buffer per head, where one warp per scheduler exponentiated at a time:
// none 1.000 ms, 2 of 8 0.983 ms, 3 of 8 1.014 ms.  With the one shared score buffer, where both warpgroups
// exponentiate at once and the hand-over chain of the buffer sets the pace: none 0.819 - 0.824 ms, 1 of 8 0.825,
// 2 of 8 0.836 - 0.845, 3 of 8 0.913 - 0.915 (the polynomial's instructions lengthen each warp's tile; the MUFU
// unit, 49 % busy, is not what the warps wait for).
#ifndef TA_FMA_EXP_MASK
#define TA_FMA_EXP_MASK 0x00u
#endif

namespace ta {
namespace attn {

using namespace sm100;

constexpr int BQ = 128;        // query rows per tile
constexpr int BKV = 128;       // keys per tile
constexpr int THREADS = 384;
constexpr int SUB_BYTES = 128 * 64 * 2;   // one [128 x 64] bf16 sub-tile (128-byte rows)
constexpr int MAX_SUB = 2;                 // r2 (fused), r3, t3 <= 128
constexpr int KV_STAGES = 2;
constexpr float kRescaleThreshold = 8.f;
// Qt tile | Qhat_0 | Qhat_1 | K ring | V ring
constexpr size_t SMEM_BYTES = 1024 + (size_t)(3 * MAX_SUB + 2 * KV_STAGES * MAX_SUB) * SUB_BYTES;

struct Params {
  int B, N, nH, r2, r3, t3;
  int causal;
  int n_qt;          // query tiles per sequence
  int n_hp;          // head pairs
  int hp_per_item;   // consecutive head pairs handled by one CTA (1 in the unfused mode)
  int n_hg;          // head-pair groups = ceil(n_hp / hp_per_item)
  int n_items;       // work items = n_qt * B * n_hg
  int fused;         // 1: tmQ is the map of Qt [B, N, r2] and Qhat is formed in the prologue
  const float4* rope;   // (cos, sin) for the rows of this call in the rope_unit_index layout, or nullptr (fused mode only)
  bf16* O;           // [B, N, nH, t3] (written through the tensor map tmO)
  unsigned int* err;
};

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// exp2 of a pair on the FMA pipe.  x is split into n = round(x) and f = x - n in [-0.5, 0.5] by adding
// 1.5 * 2^23 + 127, whose float sum holds n + 127 in its low mantissa bits; 2^f comes from a cubic (relative
// error 7.5e-5, well inside the 2^-9 of the bf16 probabilities) and 2^n is that sum's bit pattern shifted into
// the exponent field.  Valid for x <= 128; x below -125 (masked scores are -inf) is clamped there.
__device__ __forceinline__ float2 exp2_fma_pair(float2 x) {
  x.x = fmaxf(x.x, -125.f);
  x.y = fmaxf(x.y, -125.f);
  const float kMagic = 12583039.f;   // 1.5 * 2^23 + 127
  const float2 t = __fadd2_rn(x, make_float2(kMagic, kMagic));
  const float2 n = __fadd2_rn(t, make_float2(-kMagic, -kMagic));
  const float2 f = __fadd2_rn(x, make_float2(-n.x, -n.y));
  float2 p = __ffma2_rn(make_float2(0.0551716685f, 0.0551716685f), f, make_float2(0.242611125f, 0.242611125f));
  p = __ffma2_rn(p, f, make_float2(0.693260968f, 0.693260968f));
  p = __ffma2_rn(p, f, make_float2(0.999928057f, 0.999928057f));
  const float2 sc = make_float2(__uint_as_float(__float_as_uint(t.x) << 23), __uint_as_float(__float_as_uint(t.y) << 23));
  return __fmul2_rn(p, sc);
}
constexpr uint32_t kFmaExpMask = TA_FMA_EXP_MASK;

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// Register budget per warpgroup: the producer / MMA warpgroup gives registers to the two softmax
// warpgroups, which hold a whole 128-column score row per thread.
__device__ __forceinline__ void regs_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 56;"); }
__device__ __forceinline__ void regs_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 224;"); }

// Waits until the shared-memory counter *c has reached `target` (bounded like the barrier waits).
__device__ __forceinline__ bool wait_count(const int* c, int target, const Abort& ab) {
  const volatile int* vc = c;
  if (*vc >= target) return true;
  const long long t0 = clock64();
  while (true) {
    if (*vc >= target) return true;
    if (ab.raised()) return false;
    if (clock64() - t0 > kWaitBudgetCycles) {
      ab.raise();
      return false;
    }
  }
}

// Eight-or-fewer K = 16 steps of one 128 x N product over K-major, 128-byte-swizzled shared-memory tiles whose
// 64-element K blocks are SUB_BYTES apart: the step offsets are immediates added to the descriptors' address field.
__device__ __forceinline__ void issue_kmajor_ss(uint32_t d_tmem, uint64_t ad, uint64_t bd, uint32_t idesc, int ksteps) {
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
    if (ks < ksteps) {
      const uint64_t o = (uint64_t)(((uint32_t)(ks >> 2) * SUB_BYTES + (uint32_t)(ks & 3) * 32) >> 4);
      umma_ss(d_tmem, ad + o, bd + o, idesc, ks != 0);
    }
  }
}
// O += P V over one 128-key tile: A = P from TMEM (bf16, 8 columns per step), B = the transposed value tile.
__device__ __forceinline__ void issue_kmajor_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_saddr, uint32_t idesc, bool acc) {
  const uint64_t bd = umma_desc_kmajor_sw128(b_saddr);
#pragma unroll
  for (int ks = 0; ks < BKV / 16; ++ks) {
    const uint64_t o = (uint64_t)(((uint32_t)(ks >> 2) * SUB_BYTES + (uint32_t)(ks & 3) * 32) >> 4);
    umma_ts(d_tmem, a_tmem + (uint32_t)ks * 8, bd + o, idesc, acc || ks != 0);
  }
}

// The k-th work item of this CTA (see the header comment); false when the CTA has run out of items.
struct Item {
  int b, qt, q0, hp_begin, hp_end, nt;
};
__device__ __forceinline__ bool get_item(const Params& p, int k, Item& im) {
  const int G = (int)gridDim.x;
  const long item64 = (long)k * G + ((k & 1) ? (G - 1 - (int)blockIdx.x) : (int)blockIdx.x);
  if (item64 >= p.n_items) return false;
  unsigned item = (unsigned)item64;          // (n_items < 2^30: 32-bit divisions, every role calls this per item)
  const int hg = (int)(item % (unsigned)p.n_hg); item /= (unsigned)p.n_hg;
  im.b = (int)(item % (unsigned)p.B); item /= (unsigned)p.B;
  im.qt = p.n_qt - 1 - (int)item;            // heaviest (largest query tile) first
  im.q0 = im.qt * BQ;
  im.hp_begin = hg * p.hp_per_item;
  im.hp_end = min(p.n_hp, im.hp_begin + p.hp_per_item);
  const int n_kt_all = (p.N + BKV - 1) / BKV;
  im.nt = p.causal ? min(n_kt_all, im.qt + 1) : n_kt_all;
  return true;
}

__global__ void __launch_bounds__(THREADS, 1)
k_attn_prefill(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmG,
               const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
               const __grid_constant__ CUtensorMap tmO, const Params p) {
  pdl_enter();
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t q_full, qt_free, k_full[KV_STAGES], k_empty[KV_STAGES], v_full[KV_STAGES], v_empty[KV_STAGES];
  __shared__ uint64_t s_full[2], s_free[2], p_full[2], o_full[2], qh_done[2], qh_ready[2];
  __shared__ uint64_t o_staged[2], stage_free[2];   // output rows are in shared memory / the output store has read them
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  __shared__ int qk_issued;    // score tiles issued so far by this CTA (written by the score issuer, read by the value issuer)

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* tiles = smem_raw + (base - smem_u32(smem_raw));
  uint8_t* qt_tile = tiles;
  uint8_t* q_tile[2] = {tiles + MAX_SUB * SUB_BYTES, tiles + 2 * MAX_SUB * SUB_BYTES};
  uint8_t* k_ring = tiles + 3 * MAX_SUB * SUB_BYTES;
  uint8_t* v_ring = k_ring + KV_STAGES * MAX_SUB * SUB_BYTES;

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int qsub = (p.r2 + 63) / 64, ksub = (p.r3 + 63) / 64, vsub = (p.t3 + 63) / 64;
  Abort ab{&abort_flag, p.err};

  if (threadIdx.x == 0) {
    abort_flag = 0;
    qk_issued = 0;
    mbar_init(&q_full, 1);
    mbar_init(&qt_free, 1);       // the item's per-head query MMAs have read the Qt tile
    for (int s = 0; s < KV_STAGES; ++s) {
      mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 1);
      mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&s_full[i], 1);
      mbar_init(&s_free[i], 4);     // one arrival per softmax warp: the score tile is in registers
      mbar_init(&p_full[i], 4);     // one arrival per softmax warp
      mbar_init(&o_full[i], 1);
      mbar_init(&qh_done[i], 1);
      mbar_init(&qh_ready[i], 4);   // one arrival per softmax warp
      mbar_init(&o_staged[i], 4);
      mbar_init(&stage_free[i], 1);
    }
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(&tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_slot;
  const uint32_t tm_s = tmem;                               // the one score buffer, used by the two heads in turn
  const uint32_t tm_p[2] = {tmem + 128, tmem + 192};        // probabilities (bf16, two per column)
  const uint32_t tm_o[2] = {tmem + 256, tmem + 384};
  const uint32_t tm_qh[2] = {tmem, tmem + 128};             // prologue accumulators: S and the two P blocks

  if (warp < 4) {
   regs_dec();
   if (warp == 0) {
    // ------------------------------- TMA producer -------------------------------
    if (elect_one()) {
      tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
      if (p.fused) tma_prefetch_desc(&tmG);
      int it_k = 0, it_v = 0;          // ring iterations issued so far
      bool ok = true;
      Item im;
      for (int k = 0; ok && get_item(p, k, im); ++k) {
      const int b = im.b, q0 = im.q0, nt = im.nt;
      for (int hp = im.hp_begin; hp < im.hp_end && ok; ++hp) {
        const int h0 = hp * 2;
        const int nh = (h0 + 1) < p.nH ? 2 : 1;
        if (p.fused) {
          if (hp == im.hp_begin) {
            // the previous item's per-head query MMAs must have read the Qt tile
            if (k > 0 && !(ok = mbar_wait(&qt_free, (uint32_t)((k - 1) & 1), ab))) break;
            mbar_expect_tx(&q_full, (uint32_t)(qsub * SUB_BYTES));
            for (int kk = 0; kk < qsub; ++kk) tma_load_3d(qt_tile + kk * SUB_BYTES, &tmQ, &q_full, kk * 64, q0, b);
          }
          // G_{h0+i} (stored [r3 rows, r2] K-major) travels through the V ring
          for (int i = 0; i < nh && ok; ++i, ++it_v) {
            const int s = it_v % KV_STAGES;
            if (!(ok = mbar_wait(&v_empty[s], ((it_v / KV_STAGES) & 1) ^ 1, ab))) break;
            mbar_expect_tx(&v_full[s], (uint32_t)(qsub * p.r3 * 128));
            for (int kk = 0; kk < qsub; ++kk)
              tma_load_2d(v_ring + (s * MAX_SUB + kk) * SUB_BYTES, &tmG, &v_full[s], kk * 64, (h0 + i) * p.r3);
          }
        } else {
          mbar_expect_tx(&q_full, (uint32_t)(nh * ksub * SUB_BYTES));
          for (int i = 0; i < nh; ++i)
            for (int kk = 0; kk < ksub; ++kk)
              tma_load_3d(q_tile[i] + kk * SUB_BYTES, &tmQ, &q_full, (h0 + i) * p.r3 + kk * 64, q0, b);
        }
        for (int j = 0; j < nt && ok; ++j, ++it_k, ++it_v) {
          const int sk = it_k % KV_STAGES, sv = it_v % KV_STAGES;
          if (!(ok = mbar_wait(&k_empty[sk], ((it_k / KV_STAGES) & 1) ^ 1, ab))) break;
          mbar_expect_tx(&k_full[sk], (uint32_t)(ksub * SUB_BYTES));
          for (int kk = 0; kk < ksub; ++kk)
            tma_load_3d(k_ring + (sk * MAX_SUB + kk) * SUB_BYTES, &tmK, &k_full[sk], kk * 64, j * BKV, b);
          if (!(ok = mbar_wait(&v_empty[sv], ((it_v / KV_STAGES) & 1) ^ 1, ab))) break;
          // value tile, transposed in global memory: [t3 rows][128 keys] as two 64-key blocks of 128-byte rows
          mbar_expect_tx(&v_full[sv], (uint32_t)(2 * p.t3 * 128));
          for (int kk = 0; kk < 2; ++kk)
            tma_load_3d(v_ring + (sv * MAX_SUB + kk) * SUB_BYTES, &tmV, &v_full[sv], j * BKV + kk * 64, 0, b);
        }
      }
      }
    }
   } else if (warp == 1) {
    // ------------------------------- score issuer: S = Qhat_i K^T ---------------------------------
    if (elect_one()) {
      const uint32_t idesc_qk = umma_idesc_bf16(BQ, BKV);
      const int ksteps = p.r3 / 16;
      int it_k = 0;                    // K ring iterations consumed so far
      int ns0 = 0, ns1 = 0;            // score tiles issued so far for head 0 / head 1 of the pairs (s_free phases)
      int gp0 = 0, gp1 = 0;            // head pairs handled so far per head (qh_ready phases)
      int n_issued = 0;
      bool ok = true;
      Item im;
      for (int k = 0; ok && get_item(p, k, im); ++k) {
      const int nt = im.nt;
      for (int hp = im.hp_begin; hp < im.hp_end && ok; ++hp) {
        const int nh = (hp * 2 + 1) < p.nH ? 2 : 1;
        if (!p.fused && !(ok = mbar_wait(&q_full, 0, ab))) break;     // (one item and one pair per CTA in this mode)
        // The pair's score tiles in issue order: t = j * nh + i for key tile j and head i.  Tile t is issued as soon
        // as the warpgroup of tile t - 1 holds that tile in registers, so the next scores are ready whenever a
        // warpgroup finishes a tile.  (Tile 0 waits for the reads of the previous pair's last tiles instead.)
        const int n_tiles = nt * nh;
        uint32_t sk = 0;
        for (int t = 0; t < n_tiles && ok; ++t) {
          const int i = (nh == 2) ? (t & 1) : 0;
          // Long rows: everything that does not depend on the score buffer first, since the hand-over of the buffer
          // is the critical path of the tile sequence.  Short rows (a few tiles per pair) measured faster the other
          // way round: there the K tile of a new pair is what arrives last.
          auto wait_operands = [&]() -> bool {
            if (i == 0) {
              sk = (uint32_t)(it_k % KV_STAGES);
              if (!mbar_wait(&k_full[sk], (it_k / KV_STAGES) & 1, ab)) return false;
            }
            return !(t < nh && p.fused) || mbar_wait(&qh_ready[i], (uint32_t)((i ? gp1 : gp0) & 1), ab);
          };
          const bool operands_first = nt >= 8;
          if (operands_first && !(ok = wait_operands())) break;
          if (t >= 1) {
            const int ip = (nh == 2) ? (i ^ 1) : 0;
            if (!(ok = mbar_wait_poll(&s_free[ip], (uint32_t)(((ip ? ns1 : ns0) - 1) & 1), ab))) break;
          } else {
            if (ns0 > 0 && !(ok = mbar_wait_poll(&s_free[0], (uint32_t)((ns0 - 1) & 1), ab))) break;
            if (ns1 > 0 && !(ok = mbar_wait_poll(&s_free[1], (uint32_t)((ns1 - 1) & 1), ab))) break;
          }
          if (!operands_first && !(ok = wait_operands())) break;
          const uint64_t ad = umma_desc_kmajor_sw128(smem_u32(tiles) + (uint32_t)(1 + i) * (MAX_SUB * SUB_BYTES));
          const uint64_t bd = umma_desc_kmajor_sw128(smem_u32(k_ring) + sk * (MAX_SUB * SUB_BYTES));
          tc_fence_after();
          issue_kmajor_ss(tm_s, ad, bd, idesc_qk, ksteps);
          umma_commit(&s_full[i]);
          *(volatile int*)&qk_issued = ++n_issued;
          if (i) ++ns1; else ++ns0;
          if (i == nh - 1) { umma_commit(&k_empty[sk]); ++it_k; }
        }
        ++gp0;
        if (nh == 2) ++gp1;
      }
      }
    }
   } else if (warp == 2) {
    // ------------------------------- value issuer: Qhat_i = Qt G_i^T, O_i += P_i V ------------------
    if (elect_one()) {
      const uint32_t idesc_pv = umma_idesc_bf16(BQ, (uint32_t)p.t3);
      const uint32_t idesc_qh = umma_idesc_bf16(BQ, (uint32_t)p.r3);
      int it_v = 0;                    // V ring iterations consumed so far
      int np0 = 0, np1 = 0;            // P V products issued so far per head (p_full phases)
      int ns0 = 0, ns1 = 0;            // score tiles of the finished pairs per head (s_free phases)
      int n_before = 0;                // score tiles of the finished pairs, both heads
      bool ok = true;
      Item im;
      for (int k = 0; ok && get_item(p, k, im); ++k) {
      const int nt = im.nt;
      for (int hp = im.hp_begin; hp < im.hp_end && ok; ++hp) {
        const int g = hp - im.hp_begin;
        const int nh = (hp * 2 + 1) < p.nH ? 2 : 1;
        if (p.fused) {
          if (g == 0 && !(ok = mbar_wait(&q_full, (uint32_t)(k & 1), ab))) break;
          // the prologue accumulates into the score and probability columns: the last score tiles of the previous
          // pair must have been read (its P V products precede these MMAs in this thread's issue order)
          if (ns0 > 0 && !(ok = mbar_wait_poll(&s_free[0], (uint32_t)((ns0 - 1) & 1), ab))) break;
          if (ns1 > 0 && !(ok = mbar_wait_poll(&s_free[1], (uint32_t)((ns1 - 1) & 1), ab))) break;
          for (int i = 0; i < nh && ok; ++i, ++it_v) {
            const uint32_t s = (uint32_t)(it_v % KV_STAGES);
            if (!(ok = mbar_wait(&v_full[s], (it_v / KV_STAGES) & 1, ab))) break;
            tc_fence_after();
            issue_kmajor_ss(tmem + (uint32_t)i * 128u, umma_desc_kmajor_sw128(smem_u32(qt_tile)),
                            umma_desc_kmajor_sw128(smem_u32(v_ring) + s * (MAX_SUB * SUB_BYTES)), idesc_qh, p.r2 / 16);
            umma_commit(&qh_done[i]);
            umma_commit(&v_empty[s]);
          }
          if (!ok) break;
          if (hp == im.hp_end - 1) umma_commit(&qt_free);   // the item's last use of the Qt tile
        }
        const int n_tiles = nt * nh;
        uint32_t sv = 0;
        for (int t = 0; t < n_tiles && ok; ++t) {
          const int i = (nh == 2) ? (t & 1) : 0;
          const int j = (nh == 2) ? (t >> 1) : t;
          if (i == 0) {
            sv = (uint32_t)(it_v % KV_STAGES);
            if (!(ok = mbar_wait(&v_full[sv], (it_v / KV_STAGES) & 1, ab))) break;
          }
          if (!(ok = mbar_wait_poll(&p_full[i], (uint32_t)((i ? np1 : np0) & 1), ab))) break;
          if (i) ++np1; else ++np0;
          // The tensor core runs MMAs in issue order, and an idle warpgroup is waiting for score tile t + 2 while
          // nobody waits for this product: when both are ready at about the same time the scores go first.  (Tile
          // t + 2 only needs tile t + 1 to have been read, which does not depend on this product.)
          if (t + 2 < n_tiles && !(ok = wait_count(&qk_issued, n_before + t + 3, ab))) break;
          tc_fence_after();
          issue_kmajor_ts(tmem + 256u + (uint32_t)i * 128u, tmem + 128u + (uint32_t)i * 64u,
                          smem_u32(v_ring) + sv * (MAX_SUB * SUB_BYTES), idesc_pv, j != 0);
          umma_commit(&o_full[i]);
          if (i == nh - 1) { umma_commit(&v_empty[sv]); ++it_v; }
        }
        ns0 += nt;
        if (nh == 2) ns1 += nt;
        n_before += n_tiles;
      }
      }
    }
   }
  } else {
    regs_inc();
    // ------------------------------- softmax / correction / epilogue -------------
    const int i = (warp - 4) / 4;              // which head of the pair
    const int q = warp % 4;                    // TMEM lane quadrant
    const int rloc = q * 32 + lane;            // row inside the tile
    const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
    int jt = 0;                                // tiles consumed so far (parity of s_full / p_full / o_full)
    int g = 0;                                 // head pairs this warpgroup has handled so far (parity of the per-pair barriers)
    int g_two = 0;                             // ... of which had two heads (parity of the other head's qh_ready)
    bool ok = true;
    Item im;
    for (int k = 0; ok && get_item(p, k, im); ++k) {
    const int b = im.b, q0 = im.q0, nt = im.nt;
    const int row = q0 + rloc;                 // query row inside the sequence
    for (int hp = im.hp_begin; hp < im.hp_end && ok; ++hp) {
      const int h0 = hp * 2;
      const bool two_heads = (h0 + 1) < p.nH;
      if (i == 1 && !two_heads) continue;         // odd head count: the last pair has one head
      // The previous pair's output store must have finished reading this head's Qhat tile before the tile is written
      // again: waited for as late as possible (the fused prologue reads and rotates its first chunk before).
      auto wait_stage_free = [&]() -> bool {
        if (g == 0) return true;
        if (q == 0 && lane == 0) {
          tma_store_wait_read();
          mbar_arrive(&stage_free[i]);
        }
        const bool w = mbar_wait(&stage_free[i], (uint32_t)((g - 1) & 1), ab);
        return __all_sync(0xffffffffu, w);
      };
      if (!p.fused && !(ok = wait_stage_free())) break;
      if (p.fused) {
        // ---- prologue: Qhat row from TMEM, latent RoPE, bf16, swizzled K-major store ----
        ok = mbar_wait(&qh_done[i], (uint32_t)(g & 1), ab);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        const float4* tab = (p.rope && row < p.N) ? p.rope + rope_unit_index(row, 0, p.r3 / 4) : nullptr;
        for (int ch = 0; ch < p.r3 / 32; ++ch) {
          uint32_t r[32];
          tmem_ld32(tm_qh[i] + lane_addr + ch * 32, r);
          tmem_ld_wait();
          uint32_t o[16];
          if (tab) {
            const float4* t4 = tab + ch * 8 * 32;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
              const float4 cs = t4[c * 32];      // (cos, sin) of two consecutive pairs
              const float xe0 = __uint_as_float(r[4 * c]), xo0 = __uint_as_float(r[4 * c + 1]);
              const float xe1 = __uint_as_float(r[4 * c + 2]), xo1 = __uint_as_float(r[4 * c + 3]);
              o[2 * c] = pack_bf16(xe0 * cs.x - xo0 * cs.y, xe0 * cs.y + xo0 * cs.x);
              o[2 * c + 1] = pack_bf16(xe1 * cs.z - xo1 * cs.w, xe1 * cs.w + xo1 * cs.z);
            }
          } else {
#pragma unroll
            for (int c = 0; c < 16; ++c) o[c] = pack_bf16(__uint_as_float(r[2 * c]), __uint_as_float(r[2 * c + 1]));
          }
          if (ch == 0 && !(ok = wait_stage_free())) break;
          uint8_t* dst = q_tile[i] + (ch >> 1) * SUB_BYTES + rloc * 128;
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            const int chunk = (ch & 1) * 4 + v;
            *reinterpret_cast<uint4*>(dst + ((chunk ^ (rloc & 7)) << 4)) =
                make_uint4(o[4 * v], o[4 * v + 1], o[4 * v + 2], o[4 * v + 3]);
          }
        }
        if (!ok) break;
        tc_fence_before();
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&qh_ready[i]);
      }
      float m_used = -INFINITY, l = 0.f;
      for (int j = 0; j < nt; ++j, ++jt) {
        ok = mbar_wait(&s_full[i], (uint32_t)(jt & 1), ab);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        uint32_t sr[128];
        {
          uint32_t (*c)[32] = reinterpret_cast<uint32_t (*)[32]>(sr);
          tmem_ld32(tm_s + lane_addr + 0, c[0]);
          tmem_ld32(tm_s + lane_addr + 32, c[1]);
          tmem_ld32(tm_s + lane_addr + 64, c[2]);
          tmem_ld32(tm_s + lane_addr + 96, c[3]);
          tmem_ld_wait();
        }
        // the tile is in registers: the tensor core may write the other head's (or the next) scores into the buffer
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&s_free[i]);
        const int k0 = j * BKV;
        const bool need_mask = (p.causal && (k0 + BKV - 1 > q0)) || (k0 + BKV > p.N);
        if (need_mask) {
          const int lim = p.causal ? min(row, p.N - 1) : (p.N - 1);   // last visible key index
#pragma unroll
          for (int c = 0; c < 128; ++c)
            if (k0 + c > lim) sr[c] = 0xff800000u;   // -inf
        }
        float mt;
        {
          float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;   // four independent chains
#pragma unroll
          for (int c = 0; c < 128; c += 8) {
            m0 = max3(m0, __uint_as_float(sr[c]), __uint_as_float(sr[c + 1]));
            m1 = max3(m1, __uint_as_float(sr[c + 2]), __uint_as_float(sr[c + 3]));
            m2 = max3(m2, __uint_as_float(sr[c + 4]), __uint_as_float(sr[c + 5]));
            m3 = max3(m3, __uint_as_float(sr[c + 6]), __uint_as_float(sr[c + 7]));
          }
          mt = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
        }
        const bool need = (mt > m_used + kRescaleThreshold) && (mt > -INFINITY);
        if (__any_sync(0xffffffffu, need)) {
          const float m_new = need ? mt : m_used;
          const float factor = need ? fast_exp2(m_used - m_new) : 1.f;   // exp2(-inf) = 0 on the first tile
          if (j > 0) {
            ok = mbar_wait(&o_full[i], (uint32_t)((jt - 1) & 1), ab);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            for (int ch = 0; ch < p.t3 / 32; ++ch) {
              uint32_t o[32];
              tmem_ld32(tm_o[i] + lane_addr + ch * 32, o);
              tmem_ld_wait();
#pragma unroll
              for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * factor);
              tmem_st32(tm_o[i] + lane_addr + ch * 32, o);
            }
          }
          l *= factor;
          m_used = m_new;
        }
        // p = exp2(s - m) two at a time (packed fp32 add), row sum in four packed accumulators;
        // the bf16 pairs overwrite the score registers in place (pair c lands in sr[c])
        {
          const float2 negm = make_float2(-m_used, -m_used);
          float2 rs[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
          for (int c = 0; c < 64; ++c) {
            const float2 x = __fadd2_rn(make_float2(__uint_as_float(sr[2 * c]), __uint_as_float(sr[2 * c + 1])), negm);
            const float2 pp = ((kFmaExpMask >> (c & 7)) & 1u) ? exp2_fma_pair(x) : make_float2(fast_exp2(x.x), fast_exp2(x.y));
            rs[c & 3] = __fadd2_rn(rs[c & 3], pp);
            sr[c] = pack_bf16(pp.x, pp.y);
          }
          const float2 r01 = __fadd2_rn(rs[0], rs[1]), r23 = __fadd2_rn(rs[2], rs[3]);
          l += (r01.x + r01.y) + (r23.x + r23.y);
        }
        // P_i is free once the previous P V product of this head has read it; on a pair's first tile head 0 also
        // waits until head 1's prologue has taken its Qhat accumulator out of the P columns
        if (j > 0) {
          ok = mbar_wait(&o_full[i], (uint32_t)((jt - 1) & 1), ab);
        } else if (p.fused && i == 0 && two_heads) {
          ok = mbar_wait(&qh_ready[1], (uint32_t)(g_two & 1), ab);
        }
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        {
          uint32_t (*c)[32] = reinterpret_cast<uint32_t (*)[32]>(sr);
          tmem_st32(tm_p[i] + lane_addr + 0, c[0]);
          tmem_st32(tm_p[i] + lane_addr + 32, c[1]);
          tmem_st_wait();
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_full[i]);
      }
      if (!ok) break;
      ok = mbar_wait(&o_full[i], (uint32_t)((jt - 1) & 1), ab);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      // ---- epilogue: normalised row -> this head's Qhat tile (free now: every MMA of the pair is
      // complete) in the 128-byte-swizzled layout, then one TMA store per 64-column block; rows
      // beyond N and columns beyond t3 are clipped by the tensor map ----
      const float inv = 1.f / l;
      for (int ch = 0; ch < p.t3 / 32; ++ch) {
        uint32_t o[32];
        tmem_ld32(tm_o[i] + lane_addr + ch * 32, o);
        tmem_ld_wait();
        uint8_t* dst = q_tile[i] + (ch >> 1) * SUB_BYTES + rloc * 128;
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          uint32_t w[4];
#pragma unroll
          for (int e = 0; e < 4; ++e)
            w[e] = pack_bf16(__uint_as_float(o[8 * v + 2 * e]) * inv, __uint_as_float(o[8 * v + 2 * e + 1]) * inv);
          const int chunk = (ch & 1) * 4 + v;
          *reinterpret_cast<uint4*>(dst + ((chunk ^ (rloc & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
        }
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(&o_staged[i]);
      if (q == 0 && lane == 0) {
        if (mbar_wait(&o_staged[i], (uint32_t)(g & 1), ab)) {      // all four warps' rows are in shared memory
          for (int kk = 0; kk < vsub; ++kk) tma_store_4d(&tmO, q_tile[i] + kk * SUB_BYTES, kk * 64, h0 + i, q0, b);
          tma_store_commit();
        }
      }
      tc_fence_before();   // the next head pair's MMAs overwrite O_i after these reads
      ++g;
      if (two_heads) ++g_two;
    }
    }
    if (q == 0 && lane == 0) tma_store_wait_all();   // the stores read shared memory: finish before the CTA may exit
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 512);
}

}  // namespace attn
}  // namespace ta
