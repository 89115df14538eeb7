// C[M, N] = A[M, K] * B[N, K]^T on the 5th-generation tensor cores (tcgen05.mma, bf16 inputs,
// fp32 accumulation in TMEM), operands streamed by TMA through a shared-memory ring.
// One CTA computes `ncb` adjacent 128 x BN output tiles of the same 128 rows (BN a multiple of 32, at
// most 256; ncb accumulators side by side in TMEM), so that the A tile is loaded once for all of them:
//   warp 0      TMA producer (one elected lane)
//   warp 1      TMEM allocation + MMA issue (one elected lane)
//   warps 2..9  epilogue: TMEM -> registers -> global, two warps per TMEM lane quadrant
// The N range is a concatenation of up to three segments (e.g. [Qt | K | V] of the latent
// projections), each with its own destination and epilogue (plain, latent RoPE on column
// pairs, fp32), so that one launch serves several logical outputs.
#pragma once

#include "ta_common.cuh"
#include "ta_sm100.cuh"

namespace ta {
namespace umma_gemm {

using namespace sm100;

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int MAX_STAGES = 4;
constexpr int THREADS = 320;   // producer warp, MMA warp, eight epilogue warps
constexpr int MAX_BN = 256;
// Dynamic shared memory of one CTA: the ring is sized for the stage count and tile width of
// the launch, so that short-K problems (one or two K blocks) leave room for several CTAs
// per SM and one CTA's epilogue overlaps another's loads and MMAs.
// The epilogue reuses the ring as a [128][BN + 8] bf16 staging tile, so the ring is never smaller than that.
__host__ __device__ constexpr size_t smem_bytes(int stages, int bn, int b_mn_major, int ncb = 1) {
  const size_t ring = (size_t)stages * (BM * BK * 2 + (size_t)ncb * (b_mn_major ? (bn + 63) / 64 * 64 : bn) * BK * 2);
  const size_t stage_tile = (size_t)BM * (bn + 8) * 2;
  return 1024 /*align slack*/ + (ring > stage_tile ? ring : stage_tile);
}
// TMEM columns to allocate for a tile width (power of two >= 32).
__host__ __device__ constexpr uint32_t tmem_cols(int bn) { return bn <= 32 ? 32u : (bn <= 64 ? 64u : (bn <= 128 ? 128u : 256u)); }

enum { EP_BF16 = 0, EP_BF16_ROPE = 1, EP_F32 = 2 };

struct Seg {
  int n_begin;   // first column of this segment in the concatenated N
  int width;     // columns in this segment (a multiple of the tile width BN)
  int mode;      // EP_*
  void* out;     // destination, row-major [M, width] with leading dimension ld (elements); nullptr = not stored
  long ld;
  void* out2;    // optional second bf16 copy: element (row = b*n_pos + n, c) -> out2[b*batch2 + n*ld2 + c]
  long ld2, batch2;
  void* outT;    // optional transposed bf16 copy: element (row = b*n_pos + n, c) -> outT[b*batchT + c*ldT + n]
  long ldT, batchT;
  int bmap;      // which B tensor map (0..2) holds this segment's columns
  int b_n_off;   // N coordinate of the segment's first column inside that map
};

struct Params {
  int M, K, BN, nseg;
  int ncb;                 // column blocks (accumulators) per CTA: 1, or nseg when every segment is one block wide
  int stages;              // ring depth, 1..MAX_STAGES
  int b_mn_major;          // 1: B is given as [K, N] with N contiguous (no transpose needed)
  Seg seg[3];
  const float4* rope_tab;  // (cos, sin) pairs of positions 0 .. n_pos - 1 in the rope_unit_index layout; EP_BF16_ROPE only
  int n_pos, rope_half;    // row -> position = row % n_pos; RoPE period in columns = 2*rope_half
  int early;               // 0: everything waits for the preceding kernel; 1: A and B were complete before the
                           // preceding kernel started, only the epilogue (tables, outputs) waits; 2: B only
  int kb_per_split;        // split-K: 64-wide K blocks per blockIdx.z (0 = no split); EP_F32 outputs only
  long split_stride;       // elements between the partial outputs of consecutive splits
  unsigned int* err;
};

__global__ void __launch_bounds__(THREADS, 2)
k_umma_gemm(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
            const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmB2, const Params p) {
  // Operands that were final before the preceding kernel of the stream began may be fetched while that
  // kernel still runs (Params::early); every thread still passes pdl_enter() before it touches anything
  // the preceding kernel writes, and before it lets the next kernel be scheduled.
  if (p.early == 0) pdl_enter();
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t full_bar[MAX_STAGES], empty_bar[MAX_STAGES], acc_bar;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* tiles = smem_raw + (base - smem_u32(smem_raw));
  // MN-major B arrives as [64 k-rows x 64 columns] boxes: a tile of BN columns takes ceil(BN / 64) of
  // them (columns past the tensor's edge are zero-filled by TMA and never multiplied).
  const int n_bbox = (p.BN + 63) / 64;
  const uint32_t a_bytes = BM * BK * 2;
  const uint32_t b_bytes = p.b_mn_major ? (uint32_t)n_bbox * (64 * BK * 2) : (uint32_t)p.BN * BK * 2;
  const int ncb = p.ncb;
  const uint32_t stage_sz = a_bytes + (uint32_t)ncb * b_bytes;
  auto a_tile = [&](int s) { return tiles + (size_t)s * stage_sz; };
  auto b_tile = [&](int s, int cb) { return tiles + (size_t)s * stage_sz + a_bytes + (size_t)cb * b_bytes; };
  const int STAGES = p.stages;

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * p.BN * ncb;
  const int num_kb_all = (p.K + BK - 1) / BK;
  const int kb_begin = p.kb_per_split > 0 ? (int)blockIdx.z * p.kb_per_split : 0;
  const int num_kb = p.kb_per_split > 0 ? min(p.kb_per_split, num_kb_all - kb_begin) : num_kb_all;
  Abort ab{&abort_flag, p.err};
  // segment of column block cb, and where its columns sit in their B tensor map
  auto seg_of = [&](int cb) {
    const int nb = n0 + cb * p.BN;
    int si = 0;
    while (si + 1 < p.nseg && nb >= p.seg[si + 1].n_begin) ++si;
    return si;
  };
  auto bmap_of = [&](int si) { return p.seg[si].bmap == 0 ? &tmB0 : (p.seg[si].bmap == 1 ? &tmB1 : &tmB2); };
  const uint32_t acc_cols = tmem_cols(p.BN);                 // columns of one accumulator
  uint32_t ncols_tmem = acc_cols;                            // allocation: power of two >= ncb accumulators
  while (ncols_tmem < (uint32_t)ncb * acc_cols) ncols_tmem *= 2;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    mbar_init(&acc_bar, 1);
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(&tmem_base_slot, ncols_tmem);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;

  if (warp == 0) {
    if (elect_one()) {
      tma_prefetch_desc(&tmA);
      tma_prefetch_desc(bmap_of(seg_of(0)));
      auto load_b = [&](int kb) {
        const int s = kb % STAGES;
        const int kx = (kb_begin + kb) * BK;
        for (int cb = 0; cb < ncb; ++cb) {
          const int si = seg_of(cb);
          const int bn0 = n0 + cb * p.BN - p.seg[si].n_begin + p.seg[si].b_n_off;
          const CUtensorMap* tmB = bmap_of(si);
          if (!p.b_mn_major) {
            tma_load_2d(b_tile(s, cb), tmB, &full_bar[s], kx, bn0);
          } else {
            for (int j = 0; j < n_bbox; ++j)   // one [64 k-rows x 64 n] box per 64 columns
              tma_load_2d(b_tile(s, cb) + j * (64 * BK * 2), tmB, &full_bar[s], bn0 + j * 64, kx);
          }
        }
      };
      int b_ahead = 0;               // K blocks whose B tiles were requested before the wait
      if (p.early == 2) {
        b_ahead = num_kb < STAGES ? num_kb : STAGES;
        for (int kb = 0; kb < b_ahead; ++kb) {
          mbar_expect_tx(&full_bar[kb], stage_sz);
          load_b(kb);
        }
        asm volatile("griddepcontrol.wait;" ::: "memory");
      }
      for (int kb = 0; kb < num_kb; ++kb) {
        const int s = kb % STAGES;
        const uint32_t ph = (kb / STAGES) & 1;
        if (kb >= b_ahead) {
          if (!mbar_wait(&empty_bar[s], ph ^ 1, ab)) break;
          mbar_expect_tx(&full_bar[s], stage_sz);
          load_b(kb);
        }
        tma_load_2d(a_tile(s), &tmA, &full_bar[s], (kb_begin + kb) * BK, m0);
      }
    }
    if (p.early) pdl_enter();
  } else if (warp == 1) {
    if (elect_one()) {
      const uint32_t idesc = umma_idesc_bf16(BM, p.BN) | (p.b_mn_major ? (1u << 16) : 0u);
      bool ok = true;
      for (int kb = 0; kb < num_kb && ok; ++kb) {
        const int s = kb % STAGES;
        const uint32_t ph = (kb / STAGES) & 1;
        ok = mbar_wait(&full_bar[s], ph, ab);
        if (!ok) break;
        tc_fence_after();
        const uint32_t a_addr = smem_u32(a_tile(s));
        for (int cb = 0; cb < ncb; ++cb) {
        const uint32_t b_addr = smem_u32(b_tile(s, cb));
#pragma unroll
        for (int k = 0; k < BK / 16; ++k) {
          const uint64_t ad = umma_desc_kmajor_sw128(a_addr + k * 32);
          uint64_t bd;
          if (!p.b_mn_major) {
            bd = umma_desc_kmajor_sw128(b_addr + k * 32);
          } else {
            // MN-major, 128-byte swizzle: 64-column blocks 8192 B apart (leading offset), groups of
            // 8 k-rows 1024 B apart (stride offset); a K = 16 step advances 16 rows = 2048 B.
            bd = 0;
            bd |= (uint64_t)(((b_addr + k * 2048) & 0x3FFFFu) >> 4);
            bd |= (uint64_t)((64u * BK * 2u) >> 4) << 16;
            bd |= (uint64_t)(1024u >> 4) << 32;
            bd |= (uint64_t)1 << 46;
            bd |= (uint64_t)2 << 61;
          }
          umma_ss(tmem_base + (uint32_t)cb * acc_cols, ad, bd, idesc, (kb | k) != 0 ? 1u : 0u);
        }
        }
        umma_commit(&empty_bar[s]);   // frees the stage once these MMAs have read it
      }
      umma_commit(&acc_bar);          // accumulator complete
    }
    if (p.early) pdl_enter();
  } else {
    // epilogue: warp w owns TMEM lanes [32*(w%4), 32*(w%4)+32) and every second 32-column chunk of the
    // tile (two warps per lane quadrant: the conversion / store chain per thread is what takes the time)
    if (p.early) pdl_enter();
    const int q = warp % 4, hf = (warp - 2) >> 2;
    const int row = m0 + q * 32 + lane;
    const bool ok = mbar_wait(&acc_bar, 0, ab);
    tc_fence_after();
    if (ok) for (int cb = 0; cb < ncb; ++cb) {
      const Seg sg = p.seg[seg_of(cb)];
      const int c0 = n0 + cb * p.BN - sg.n_begin;       // first column of this block inside its segment
      const uint32_t acc = tmem_base + (uint32_t)cb * acc_cols + ((uint32_t)(q * 32) << 16);
      const int rloc = q * 32 + lane;
      const int npos = p.n_pos > 0 ? row % p.n_pos : row;
      if (sg.mode == EP_F32) {
        for (int ch = hf; ch < p.BN / 32; ch += 2) {
          uint32_t r[32];
          tmem_ld32(acc + (uint32_t)(ch * 32), r);
          tmem_ld_wait();
          if (row >= p.M) continue;
          const long off = (long)blockIdx.z * p.split_stride + (long)row * sg.ld + c0 + ch * 32;
          // extent of the partial-sum tensor as seen from this segment's base: splits x [M rows of ld]
          if (!TA_IDX_OK(p.err, off, 32, (long)(gridDim.z - 1) * p.split_stride + (long)(p.M - 1) * sg.ld + sg.width)) continue;
          float4* dst = reinterpret_cast<float4*>(static_cast<float*>(sg.out) + off);
#pragma unroll
          for (int i = 0; i < 8; ++i)
            dst[i] = make_float4(__uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1]), __uint_as_float(r[4 * i + 2]),
                                 __uint_as_float(r[4 * i + 3]));
        }
      } else {
        // bf16 outputs: every thread converts its own accumulator row into a staging tile in shared
        // memory (the ring is idle once the accumulator is complete; rows padded by 16 bytes keep the
        // 16-byte stores of a quarter-warp on distinct banks), then each warp writes the 64-byte row
        // segments of its chunks out, eight rows per 16-byte store instruction.
        const int pitch = (p.BN + 8) * 2;
        uint8_t* stage = tiles;
        // transposed copy in 16-byte pieces (8 consecutive positions of one column) when 8-row groups never
        // straddle a sequence
        const bool outT_vec = sg.outT && (p.n_pos > 0 ? p.n_pos % 8 == 0 : p.M % 8 == 0);
        for (int ch = hf; ch < p.BN / 32; ch += 2) {
          uint32_t r[32];
          tmem_ld32(acc + (uint32_t)(ch * 32), r);
          tmem_ld_wait();
          const int col = c0 + ch * 32;
          uint32_t o[16];
          if (sg.mode == EP_BF16_ROPE) {
            const int period = 2 * p.rope_half;
            // eight units (two pairs each) of this row's position; the 32 rows of the warp read neighbouring entries
            const float4* tab = p.rope_tab + rope_unit_index(npos, (col % period) >> 2, p.rope_half / 2);
            if (row < p.M) {
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const float4 cs = tab[i * 32];
                const float xe0 = __uint_as_float(r[4 * i]), xo0 = __uint_as_float(r[4 * i + 1]);
                const float xe1 = __uint_as_float(r[4 * i + 2]), xo1 = __uint_as_float(r[4 * i + 3]);
                o[2 * i] = pack_bf16(xe0 * cs.x - xo0 * cs.y, xe0 * cs.y + xo0 * cs.x);
                o[2 * i + 1] = pack_bf16(xe1 * cs.z - xo1 * cs.w, xe1 * cs.w + xo1 * cs.z);
              }
            }
          } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) o[i] = pack_bf16(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
          }
          if (sg.outT && !outT_vec && row < p.M) {
            // transposed copy, general form: for a fixed column the 32 lanes of the warp write 32 consecutive positions
            const int gb = p.n_pos > 0 ? row / p.n_pos : 0, gn = p.n_pos > 0 ? row % p.n_pos : row;
            [[maybe_unused]] const long nbT = p.n_pos > 0 ? (p.M + p.n_pos - 1) / p.n_pos : 1;
            uint16_t* dstT = static_cast<uint16_t*>(sg.outT) + (long)gb * sg.batchT + gn;
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const long o0 = (long)(col + 2 * i) * sg.ldT;
              if (TA_IDX_OK(p.err, (long)gb * sg.batchT + o0 + gn, 1, nbT * sg.batchT)) dstT[o0] = (uint16_t)(o[i] & 0xffffu);
              if (TA_IDX_OK(p.err, (long)gb * sg.batchT + o0 + sg.ldT + gn, 1, nbT * sg.batchT)) dstT[o0 + sg.ldT] = (uint16_t)(o[i] >> 16);
            }
          }
          uint4* sdst = reinterpret_cast<uint4*>(stage + (size_t)rloc * pitch + ch * 64);
#pragma unroll
          for (int i = 0; i < 4; ++i) sdst[i] = make_uint4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
        }
        __syncwarp();
        if (outT_vec) {
          // lane -> column (lane / 4) of a group of 8 and 8-row group (lane % 4) of the warp's 32 rows: the four
          // lanes of a column write 64 contiguous bytes
          const int r8 = q * 32 + (lane % 4) * 8, grow0 = m0 + r8;
          if (grow0 < p.M) {
            const int gb = p.n_pos > 0 ? grow0 / p.n_pos : 0, gn = p.n_pos > 0 ? grow0 % p.n_pos : grow0;
            [[maybe_unused]] const long nbT = p.n_pos > 0 ? (p.M + p.n_pos - 1) / p.n_pos : 1;
            for (int ch = hf; ch < p.BN / 32; ch += 2) {
#pragma unroll
              for (int cg = 0; cg < 4; ++cg) {
                const int cl = ch * 32 + cg * 8 + lane / 4;
                const uint8_t* src = stage + (size_t)r8 * pitch + cl * 2;
                uint32_t w[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  const uint32_t lo = *reinterpret_cast<const uint16_t*>(src + (size_t)(2 * e) * pitch);
                  const uint32_t hi = *reinterpret_cast<const uint16_t*>(src + (size_t)(2 * e + 1) * pitch);
                  w[e] = lo | (hi << 16);
                }
                const long off = (long)gb * sg.batchT + (long)(c0 + cl) * sg.ldT + gn;
                if (TA_IDX_OK(p.err, off, 8, nbT * sg.batchT))
                  *reinterpret_cast<uint4*>(static_cast<bf16*>(sg.outT) + off) = make_uint4(w[0], w[1], w[2], w[3]);
              }
            }
          }
        }
        const int rsub = lane / 4, cc = lane % 4;
        for (int ch = hf; ch < p.BN / 32; ch += 2) {
          for (int r0 = 0; r0 < 32; r0 += 8) {
            const int rr = q * 32 + r0 + rsub;
            const int grow = m0 + rr;
            if (grow >= p.M) continue;
            const uint4 v = *reinterpret_cast<const uint4*>(stage + (size_t)rr * pitch + ch * 64 + cc * 16);
            const int col = c0 + ch * 32 + cc * 8;
            if (sg.out && TA_IDX_OK(p.err, (long)grow * sg.ld + col, 8, (long)(p.M - 1) * sg.ld + sg.width))
              *reinterpret_cast<uint4*>(static_cast<bf16*>(sg.out) + (long)grow * sg.ld + col) = v;
            if (sg.out2) {
              const int gb = p.n_pos > 0 ? grow / p.n_pos : 0, gn = p.n_pos > 0 ? grow % p.n_pos : grow;
              const long off2 = (long)gb * sg.batch2 + (long)gn * sg.ld2 + col;
              // the second copy is [sequences][batch2]: rows n < n_pos of each sequence, `width` columns
              [[maybe_unused]] const long nb2 = p.n_pos > 0 ? (p.M + p.n_pos - 1) / p.n_pos : 1;
              if (TA_IDX_OK(p.err, off2, 8, (nb2 - 1) * sg.batch2 + (long)((p.n_pos > 0 ? p.n_pos : p.M) - 1) * sg.ld2 + sg.width))
                *reinterpret_cast<uint4*>(static_cast<bf16*>(sg.out2) + off2) = v;
            }
          }
        }
        __syncwarp();   // the warp's staging rows are free again before the next block is converted
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, ncols_tmem);
}

}  // namespace umma_gemm
}  // namespace ta
