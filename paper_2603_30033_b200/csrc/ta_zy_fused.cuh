// Output side of the layer in one kernel (Eqs. 5-6 with Definition 1):
//   Z = O [G~_1; ...; G~_nH]^T      [128 rows x t2]  (K = n_H t3)   -- stays on chip
//   Y = Z U~2^T                     [128 rows x d]   (K = t2)
// One CTA owns 128 consecutive tokens.  Phase 1 is a K-loop of tcgen05 MMAs into a TMEM
// accumulator; the epilogue warps turn that accumulator into a bf16 tile in shared memory laid out as
// a K-major, 128-byte-swizzled UMMA A operand; phase 2 walks the d / 128 column chunks of Y with two
// TMEM accumulators, so that the conversion + coalesced store of one chunk overlaps the MMAs of the
// next.  One TMA ring (uniform stage size) serves both phases, the producer runs ahead across the
// phase boundary.  The Z tile and the staging tile are idle until phase 1 has ended, so phase 1 uses
// them as two more ring stages: its O tiles come from HBM, and the bytes in flight per SM set its pace.
//   warp 0      TMA producer        warp 1   TMEM allocation + MMA issue        warps 2..9  epilogue
// (two epilogue warps per TMEM lane quadrant, one per half of a tile's columns: the conversion and store
// of a chunk is a latency chain per thread, and it, not the tensor core, paces phase 2)
#pragma once

#include "ta_common.cuh"
#include "ta_sm100.cuh"

namespace ta {
namespace zy {

using namespace sm100;

constexpr int THREADS = 320;
constexpr int BN2 = 128;                         // columns of Y per chunk
constexpr int SUB_BYTES = 128 * 64 * 2;          // one [128 x 64] bf16 sub-tile
constexpr int MAX_STAGES = 4;
constexpr int EXTRA_STAGES = 2;                  // phase 1 only: the Z tile and the staging tile
constexpr int STAGE_BYTES = 2 * SUB_BYTES;       // phase 1: O tile (16 KB) + G~ tile (<= 16 KB); phase 2: U~2 chunk (<= 32 KB)
constexpr int STAGING_PITCH = (BN2 + 8) * 2;     // bytes per staged output row
static_assert(128 * STAGING_PITCH >= STAGE_BYTES, "the staging tile doubles as a ring stage");
// ring | Z tile (two sub-tiles) | staging tile
__host__ __device__ constexpr size_t smem_bytes(int stages) {
  return 1024 + (size_t)stages * STAGE_BYTES + 2 * SUB_BYTES + (size_t)128 * STAGING_PITCH;
}

struct Params {
  int M;            // tokens
  int K1;           // n_H * t3
  int t2, d;        // t2 <= 128 (multiple of 32), d a multiple of 128
  int stages;
  bf16* Y;          // [M, d]
  unsigned int* err;
};

__global__ void __launch_bounds__(THREADS, 1)
k_zy_fused(const __grid_constant__ CUtensorMap tmO, const __grid_constant__ CUtensorMap tmG,
           const __grid_constant__ CUtensorMap tmU, const Params p) {
  pdl_enter();
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t full_bar[MAX_STAGES + EXTRA_STAGES], empty_bar[MAX_STAGES + EXTRA_STAGES];
  __shared__ uint64_t z_full, z_ready, acc_full[2], acc_empty[2];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* ring = smem_raw + (base - smem_u32(smem_raw));
  const int S = p.stages;
  uint8_t* z_tile = ring + (size_t)S * STAGE_BYTES;        // = ring stage S during phase 1
  uint8_t* staging = z_tile + 2 * SUB_BYTES;               // = ring stage S + 1 during phase 1
  const int S1 = S + EXTRA_STAGES;                         // ring depth of phase 1

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int m0 = blockIdx.x * 128;
  const int nkb1 = (p.K1 + 63) / 64;        // K blocks of phase 1
  const int nsub2 = (p.t2 + 63) / 64;       // 64-wide K sub-tiles of phase 2
  const int nchunk = p.d / BN2;
  Abort ab{&abort_flag, p.err};
  // use count of ring stage s < S at the end of phase 1 (phase 2 continues each stage's barrier phases)
  auto uses1 = [&](int s) { return nkb1 > s ? (nkb1 - s + S1 - 1) / S1 : 0; };

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < MAX_STAGES + EXTRA_STAGES; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    mbar_init(&z_full, 1);
    mbar_init(&z_ready, 8);          // one arrival per epilogue warp
    for (int u = 0; u < 2; ++u) {
      mbar_init(&acc_full[u], 1);
      mbar_init(&acc_empty[u], 8);
    }
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(&tmem_base_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_slot;
  const uint32_t tm_z = tmem;                                              // [0, t2)
  auto tm_y = [&](int buf) { return tmem + 128u + (uint32_t)buf * BN2; };  // [128, 384)

  if (warp == 0) {
    if (elect_one()) {
      tma_prefetch_desc(&tmO); tma_prefetch_desc(&tmG); tma_prefetch_desc(&tmU);
      bool ok = true;
      for (int kb = 0; kb < nkb1 && ok; ++kb) {
        const int s = kb % S1;
        if (!(ok = mbar_wait(&empty_bar[s], ((kb / S1) & 1) ^ 1, ab))) break;
        mbar_expect_tx(&full_bar[s], (uint32_t)(SUB_BYTES + p.t2 * 128));
        tma_load_2d(ring + s * STAGE_BYTES, &tmO, &full_bar[s], kb * 64, m0);
        tma_load_2d(ring + s * STAGE_BYTES + SUB_BYTES, &tmG, &full_bar[s], kb * 64, 0);
      }
      for (int n = 0; n < nchunk && ok; ++n) {
        const int s = n % S;
        if (!(ok = mbar_wait(&empty_bar[s], ((uses1(s) + n / S) & 1) ^ 1, ab))) break;
        mbar_expect_tx(&full_bar[s], (uint32_t)(nsub2 * SUB_BYTES));
        for (int kk = 0; kk < nsub2; ++kk)
          tma_load_2d(ring + s * STAGE_BYTES + kk * SUB_BYTES, &tmU, &full_bar[s], kk * 64, n * BN2);
      }
    }
  } else if (warp == 1) {
    if (elect_one()) {
      const uint32_t idesc1 = umma_idesc_bf16(128, (uint32_t)p.t2);
      const uint32_t idesc2 = umma_idesc_bf16(128, BN2);
      bool ok = true;
      // ---- phase 1: Z = O Gt^T ----
      for (int kb = 0; kb < nkb1 && ok; ++kb) {
        const int s = kb % S1;
        if (!(ok = mbar_wait(&full_bar[s], (kb / S1) & 1, ab))) break;
        tc_fence_after();
        const uint32_t a_addr = smem_u32(ring + s * STAGE_BYTES), b_addr = a_addr + SUB_BYTES;
        const int nks = min(4, (p.K1 - kb * 64) / 16);
        for (int k = 0; k < nks; ++k)
          umma_ss(tm_z, umma_desc_kmajor_sw128(a_addr + k * 32), umma_desc_kmajor_sw128(b_addr + k * 32), idesc1,
                  (kb | k) != 0 ? 1u : 0u);
        umma_commit(&empty_bar[s]);
      }
      if (ok) umma_commit(&z_full);
      // ---- phase 2: Y chunks = Z Ut2^T ----
      if (ok) ok = mbar_wait(&z_ready, 0, ab);     // the bf16 Z tile is in shared memory
      const uint32_t z_addr = smem_u32(z_tile);
      for (int n = 0; n < nchunk && ok; ++n) {
        const int s = n % S, buf = n & 1;
        if (!(ok = mbar_wait(&acc_empty[buf], ((n >> 1) & 1) ^ 1, ab))) break;
        if (!(ok = mbar_wait(&full_bar[s], (uses1(s) + n / S) & 1, ab))) break;
        tc_fence_after();
        const uint32_t b_addr = smem_u32(ring + s * STAGE_BYTES);
        for (int ks = 0; ks < p.t2 / 16; ++ks) {
          const uint32_t off = (uint32_t)(ks >> 2) * SUB_BYTES + (uint32_t)(ks & 3) * 32;
          umma_ss(tm_y(buf), umma_desc_kmajor_sw128(z_addr + off), umma_desc_kmajor_sw128(b_addr + off), idesc2, ks != 0);
        }
        umma_commit(&empty_bar[s]);
        umma_commit(&acc_full[buf]);
      }
    }
  } else {
    // epilogue warps: warp w owns TMEM lanes / tile rows [32 (w % 4), 32 (w % 4) + 32) and the column
    // half hf = (w - 2) / 4 of every tile
    const int q = warp % 4, hf = (warp - 2) >> 2;
    const int rloc = q * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
    bool ok = mbar_wait(&z_full, 0, ab);
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      tc_fence_after();
      // Z row -> bf16 -> K-major swizzled A tile
      for (int ch = hf; ch < p.t2 / 32; ch += 2) {
        uint32_t r[32];
        tmem_ld32(tm_z + lane_addr + ch * 32, r);
        tmem_ld_wait();
        uint8_t* dst = z_tile + (ch >> 1) * SUB_BYTES + rloc * 128;
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          uint32_t w[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) w[e] = pack_bf16(__uint_as_float(r[8 * v + 2 * e]), __uint_as_float(r[8 * v + 2 * e + 1]));
          const int chunk = (ch & 1) * 4 + v;
          *reinterpret_cast<uint4*>(dst + ((chunk ^ (rloc & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
        }
      }
      tc_fence_before();
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(&z_ready);
      // Y chunks
      for (int n = 0; n < nchunk; ++n) {
        const int buf = n & 1;
        ok = mbar_wait(&acc_full[buf], (uint32_t)((n >> 1) & 1), ab);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        for (int ch = 2 * hf; ch < 2 * hf + 2; ++ch) {
          uint32_t r[32];
          tmem_ld32(tm_y(buf) + lane_addr + ch * 32, r);
          tmem_ld_wait();
          uint4* sdst = reinterpret_cast<uint4*>(staging + (size_t)rloc * STAGING_PITCH + ch * 64);
#pragma unroll
          for (int i = 0; i < 4; ++i)
            sdst[i] = make_uint4(pack_bf16(__uint_as_float(r[8 * i]), __uint_as_float(r[8 * i + 1])),
                                 pack_bf16(__uint_as_float(r[8 * i + 2]), __uint_as_float(r[8 * i + 3])),
                                 pack_bf16(__uint_as_float(r[8 * i + 4]), __uint_as_float(r[8 * i + 5])),
                                 pack_bf16(__uint_as_float(r[8 * i + 6]), __uint_as_float(r[8 * i + 7])));
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&acc_empty[buf]);   // the MMA warp may overwrite this accumulator now
        // the warp writes its half (128 bytes) of its 32 rows: 8 lanes x 16 bytes per row, four rows per pass
        const int rsub = lane / 8, cc = hf * 8 + lane % 8;
        for (int r0 = 0; r0 < 32; r0 += 4) {
          const int rr = q * 32 + r0 + rsub;
          const int grow = m0 + rr;
          if (grow < p.M) {
            const uint4 v = *reinterpret_cast<const uint4*>(staging + (size_t)rr * STAGING_PITCH + cc * 16);
            if (TA_IDX_OK(p.err, (long)grow * p.d + n * BN2 + cc * 8, 8, (long)p.M * p.d))
              *reinterpret_cast<uint4*>(p.Y + (long)grow * p.d + n * BN2 + cc * 8) = v;
          }
        }
        __syncwarp();   // the warp's staging rows are free again before its next chunk is converted
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 512);
}

}  // namespace zy
}  // namespace ta
