// Tensor-core path for bf16 storage: weight preparation, tcgen05 GEMMs for the latent
// projections / per-head queries / output side, and the attention kernel.
//
//   prep      G_h (scaled by softmax scale * log2 e) and Gt_h from the cores (C x_1 U1, Definition 2),
//             stored as K-major B operands; RoPE cos/sin table
//   proj      [Qt | K | V] = X [U2 | U3 | Ut3]   (Sec. 3.1), the three factors read in place as
//             MN-major B operands; latent RoPE applied to K in the epilogue
//   qhat      Qhat[T, (h, c)] = Qt [G_1 | ... | G_nH], latent RoPE per head in the epilogue (Eq. 12)
//   attention online softmax over key tiles, one shared latent K / V pair for all heads (Sec. 3.3)
//   z, y      Z = O [Gt_1; ...; Gt_nH]^T,  Y = Z Ut2^T   (Eqs. 5-6)
#include "ta_common.cuh"
#include "ta_umma_gemm.cuh"
#include "ta_attn_prefill.cuh"
#include "ta_decode.cuh"
#include "ta_decode_umma.cuh"
#include "ta_zy_fused.cuh"

#include <math.h>

#include <algorithm>

namespace ta {
namespace {

// ---- driver entry point for tensor-map creation (no link-time dependency on libcuda) --------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// bf16 tensor of up to 4 dims; dims[0] is innermost (contiguous); strides in elements for dims 1..rank-1.
bool make_tmap(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_elems,
               const uint32_t* box, CUtensorMapSwizzle swz) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  cuuint64_t gdim[4], gstr[3];
  cuuint32_t bx[4], es[4];
  for (int i = 0; i < rank; ++i) { gdim[i] = dims[i]; bx[i] = box[i]; es[i] = 1; }
  for (int i = 0; i + 1 < rank; ++i) gstr[i] = strides_elems[i] * 2;
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gdim, gstr, bx, es,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

bool tmap_2d(CUtensorMap* m, const void* base, uint64_t cols, uint64_t rows, uint64_t ld, uint32_t box_cols,
             uint32_t box_rows) {
  uint64_t dims[2] = {cols, rows}, str[1] = {ld};
  uint32_t box[2] = {box_cols, box_rows};
  return make_tmap(m, base, 2, dims, str, box, CU_TENSOR_MAP_SWIZZLE_128B);
}

// ---- weight preparation -------------------------------------------------------------------
// One launch for everything that depends on the weights and positions only:
//   blocks [0, g1)        G^T : GcatT[h, c, b] = bf16(mult * sum_a U1[h,a] C[a,b,c])     (C x_1 U1, Definition 2)
//   blocks [g1, g1+g2)    Gt  : GtP[j, h, c]   = bf16(sum_a Ut1[h,a] Ct[a,j,c])
//   blocks [g1+g2, ...)   (cos, sin) table for positions pos0 .. pos0 + n_pos - 1
struct PrepParams {
  const bf16 *C, *U1, *Ct, *Ut1;
  bf16 *GcatT, *GtP;
  float4* rope;     // rope_unit_index layout
  int nH, r1, r2, r3, t1, t2, t3;
  int n_pos, pos0;
  float mult;
  dec::RopeFreqs freqs;
  int g1, g2, g3;
  unsigned int* err;
};

constexpr int PREP_THREADS = 128;

__device__ __forceinline__ void unpack8(const uint4& v, float (&f)[8]) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float2 t = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[e]));
    f[2 * e] = t.x; f[2 * e + 1] = t.y;
  }
}
__device__ __forceinline__ uint4 pack8(const float (&f)[8]) {
  return make_uint4(sm100::pack_bf16(f[0], f[1]), sm100::pack_bf16(f[2], f[3]), sm100::pack_bf16(f[4], f[5]),
                    sm100::pack_bf16(f[6], f[7]));
}

// acc[0..8) = sum_a u[a] * C[a, row, c0 .. c0 + 8): 16-byte loads along the contiguous index of the core,
// four slices requested before the first is used.
__device__ __forceinline__ void head_core_8(const bf16* __restrict__ Cbase, long slice_stride, const bf16* __restrict__ u,
                                            int r1, float (&acc)[8]) {
#pragma unroll
  for (int e = 0; e < 8; ++e) acc[e] = 0.f;
  for (int a0 = 0; a0 < r1; a0 += 4) {
    uint4 v[4];
#pragma unroll
    for (int k = 0; k < 4; ++k)
      v[k] = (a0 + k < r1) ? *reinterpret_cast<const uint4*>(Cbase + (long)(a0 + k) * slice_stride) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (a0 + k < r1) {
        const float ua = __bfloat162float(u[a0 + k]);
        float f[8];
        unpack8(v[k], f);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = fmaf(ua, f[e], acc[e]);
      }
    }
  }
}

__global__ void __launch_bounds__(PREP_THREADS) k_prefill_prep(const PrepParams p) {
  pdl_enter();
  __shared__ __align__(16) bf16 tile[32][40];     // [c][b], rows padded to 80 bytes (16-byte aligned, conflict-poor)
  const int blk = blockIdx.x, t = threadIdx.x;
  if (blk < p.g1) {
    // G^T tile: head h, 32 query coordinates b x 32 key coordinates c.  Read along c (contiguous in the
    // core), transpose through shared memory, write along b (contiguous in GcatT[h, c, b]).
    const int tc = p.r3 / 32, tb = p.r2 / 32;
    const int h = blk / (tb * tc), b0 = ((blk / tc) % tb) * 32, c0 = (blk % tc) * 32;
    {
      const int bl = t / 4, cc = (t % 4) * 8;
      float acc[8];
      head_core_8(p.C + ((long)(b0 + bl) * p.r3 + c0 + cc), (long)p.r2 * p.r3, p.U1 + (long)h * p.r1, p.r1, acc);
#pragma unroll
      for (int e = 0; e < 8; ++e) tile[cc + e][bl] = __float2bfloat16_rn(acc[e] * p.mult);
    }
    __syncthreads();
    {
      const int cl = t / 4, bb = (t % 4) * 8;
      if (TA_IDX_OK(p.err, ((long)h * p.r3 + c0 + cl) * p.r2 + b0 + bb, 8, (long)p.nH * p.r3 * p.r2))
        *reinterpret_cast<uint4*>(p.GcatT + ((long)h * p.r3 + c0 + cl) * p.r2 + b0 + bb) =
            *reinterpret_cast<const uint4*>(&tile[cl][bb]);
    }
  } else if (blk < p.g1 + p.g2) {
    // GtP[j, h, c .. c + 8): the value coordinate c is contiguous in the core and in the output
    const long i = (long)(blk - p.g1) * PREP_THREADS + t;
    const int cch = p.t3 / 8;
    const long total = (long)p.t2 * p.nH * cch;
    if (i < total) {
      const int c8 = (int)(i % cch) * 8, h = (int)((i / cch) % p.nH), j = (int)(i / ((long)cch * p.nH));
      float acc[8];
      head_core_8(p.Ct + ((long)j * p.t3 + c8), (long)p.t2 * p.t3, p.Ut1 + (long)h * p.t1, p.t1, acc);
      if (TA_IDX_OK(p.err, ((long)j * p.nH + h) * p.t3 + c8, 8, (long)p.t2 * p.nH * p.t3))
        *reinterpret_cast<uint4*>(p.GtP + ((long)j * p.nH + h) * p.t3 + c8) = pack8(acc);
    }
  } else {
    // (cos, sin) table: one unit (two pairs of one position) per thread, in storage order (see rope_unit_index),
    // so that the stores of a warp are contiguous; the positions that pad the last block of 32 are filled too
    const int units = p.r3 / 4;
    const long o = (long)(blk - p.g1 - p.g2) * PREP_THREADS + t;
    const long total = (long)((p.n_pos + 31) / 32) * 32 * units;
    if (o < total) {
      const int n = (int)(o / (32L * units)) * 32 + (int)(o % 32), u = (int)((o / 32) % units);
      const float2 c0 = dec::rope_cos_sin_theta(p.pos0 + n, p.freqs.theta[2 * u]);
      const float2 c1 = dec::rope_cos_sin_theta(p.pos0 + n, p.freqs.theta[2 * u + 1]);
      if (TA_IDX_OK(p.err, o, 1, total)) p.rope[o] = make_float4(c0.x, c0.y, c1.x, c1.y);
    }
  }
}

// theta_i = base^(-2 i / r3) in double precision, i < r3 / 2 (r3 <= 256 on this path)
dec::RopeFreqs rope_freqs(const tucker_attn_desc& d) {
  dec::RopeFreqs f;
  const int half = d.r3 / 2;
  for (int i = 0; i < 128; ++i)
    f.theta[i] = (d.rope && i < half) ? pow((double)d.rope_base, -2.0 * (double)i / (double)d.r3) : 0.0;
  return f;
}

bool umma_attention_ok(const tucker_attn_desc& d) { return d.r3 <= 128 && d.t3 <= 128; }
// The per-head queries are formed inside the attention kernel when the Qt tile fits next to the
// other tiles in shared memory.
bool attention_fuses_qhat(const tucker_attn_desc& d) {
  return umma_attention_ok(d) && d.r2 <= 128 && !(d.flags & (TA_FLAG_FMA_ATTENTION | TA_FLAG_SEPARATE_QUERIES));
}

// ---- workspace ----------------------------------------------------------------------------
// Row pitch (elements) of the transposed value tensor: a TMA global stride is a multiple of 16 bytes.
long value_ld(int N) { return ((long)N + 7) / 8 * 8; }
struct FastWs {
  float4* rope;   // (cos, sin) of every position and pair, rope_unit_index layout
  bf16* GcatT;    // [n_H * r3, r2]      B operand of the per-head query GEMM
  bf16* GtP;      // [t2, n_H * t3]      B operand of the Z GEMM
  bf16* Qt;       // [T, r2]
  bf16* K;        // [T, r3]  rotated
  bf16* V;        // [T, t3]                 (the FMA attention reads the values token-major)
  bf16* Vt;       // [B, t3, value_ld(N)]    transposed values: the K-major B operand of P V in the tensor-core attention
  bf16* Qhat;     // [T, n_H * r3]
  bf16* O;        // [T, n_H * t3]
  bf16* Z;        // [T, t2]
};

size_t carve_fast(const tucker_attn_desc& d, char* base, FastWs* w) {
  Carver c(base);
  const size_t T = (size_t)d.B * d.N;
  FastWs t;
  t.rope = c.take<float4>(d.rope ? rope_table_units(d.N, d.r3) : 0);
  t.GcatT = c.take<bf16>((size_t)d.n_H * d.r3 * d.r2);
  t.GtP = c.take<bf16>((size_t)d.t2 * d.n_H * d.t3);
  t.Qt = c.take<bf16>(T * d.r2);
  t.K = c.take<bf16>(T * d.r3);
  t.V = c.take<bf16>(T * d.t3);
  t.Vt = c.take<bf16>((size_t)d.B * d.t3 * value_ld(d.N));
  t.Qhat = c.take<bf16>(attention_fuses_qhat(d) ? 0 : T * d.n_H * d.r3);
  t.O = c.take<bf16>(T * d.n_H * d.t3);
  t.Z = c.take<bf16>(T * d.t2);
  if (w) *w = t;
  return c.off;
}

int pick_bn(int width) {
  if (width % 128 == 0) return 128;
  if (width % 96 == 0) return 96;
  if (width % 64 == 0) return 64;
  return 32;
}

// One B operand of a GEMM: K-major [n, K] (row = output column) or, with Params::b_mn_major,
// MN-major [K, n] (row = K index); `ld` = elements between rows.
struct BOperand {
  const bf16* ptr;
  long ld;
  int n;
};

// C[M, Ntot] = A[M, K] * B^T, the N range being the concatenation of gp.seg[], each segment
// taking its columns from B operand seg.bmap starting at column seg.b_n_off.
int launch_gemm(Problem& p, const bf16* A, long lda, int M, int K, const BOperand* bops, int nb, int Ntot, int BN,
                umma_gemm::Params gp, int splits = 1) {
  CUtensorMap tmA, tmB[3];
  if (!tmap_2d(&tmA, A, (uint64_t)K, (uint64_t)M, (uint64_t)lda, 64, 128)) return TA_ERR_CUDA;
  for (int i = 0; i < 3; ++i) {
    const BOperand& b = bops[i < nb ? i : 0];
    if (!gp.b_mn_major) {
      if (!tmap_2d(&tmB[i], b.ptr, (uint64_t)K, (uint64_t)b.n, (uint64_t)b.ld, 64, (uint32_t)BN)) return TA_ERR_CUDA;
    } else {
      if (!tmap_2d(&tmB[i], b.ptr, (uint64_t)b.n, (uint64_t)K, (uint64_t)b.ld, 64, 64)) return TA_ERR_CUDA;
    }
  }
  const int num_kb = gp.kb_per_split > 0 ? gp.kb_per_split : (K + 63) / 64;
  gp.M = M; gp.K = K; gp.BN = BN; gp.err = p.dev_err;
  if (gp.ncb < 1) gp.ncb = 1;
  constexpr size_t kMaxSmem = 226 * 1024;
  gp.stages = num_kb < 3 ? (num_kb < 1 ? 1 : num_kb) : 3;
  while (gp.stages > 1 && umma_gemm::smem_bytes(gp.stages, BN, gp.b_mn_major, gp.ncb) > kMaxSmem) --gp.stages;
  if (umma_gemm::smem_bytes(gp.stages, BN, gp.b_mn_major, gp.ncb) > kMaxSmem || Ntot % (BN * gp.ncb) != 0)
    return TA_ERR_UNSUPPORTED_SHAPE;
  static PerDeviceFlag attr;
  TA_CUDA_TRY(ensure_dynamic_smem(attr, (const void*)umma_gemm::k_umma_gemm, (int)kMaxSmem));
  dim3 grid(Ntot / (BN * gp.ncb), (M + 127) / 128, splits);
  (void)launch_pdl(umma_gemm::k_umma_gemm, grid, dim3(umma_gemm::THREADS),
                   umma_gemm::smem_bytes(gp.stages, BN, gp.b_mn_major, gp.ncb), p.stream, tmA, tmB[0], tmB[1], tmB[2], gp);
  TA_LAUNCH_CHECK(p);
  return TA_OK;
}

// Widest tile width (128 / 96 / 64 / 32) dividing all three widths.
int common_bn(int a, int b, int c) {
  const int cand[4] = {128, 96, 64, 32};
  for (int bn : cand)
    if (a % bn == 0 && b % bn == 0 && c % bn == 0) return bn;
  return 0;
}

bool tmap_3d(CUtensorMap* m, const void* base, uint64_t cols, uint64_t rows, uint64_t batches, uint64_t ld,
             uint64_t batch_stride, uint32_t box_cols, uint32_t box_rows) {
  uint64_t dims[3] = {cols, rows, batches}, str[2] = {ld, batch_stride};
  uint32_t box[3] = {box_cols, box_rows, 1};
  return make_tmap(m, base, 3, dims, str, box, CU_TENSOR_MAP_SWIZZLE_128B);
}

int sm_count();
size_t l2_bytes();

// Consecutive head pairs per work item.  Causal items differ in size, so many small items balance best over
// the persistent grid: one pair per item (two were measured equal on the long causal prefill, 951 us both, three
// and more worse).  Without a mask all items are equal and an item that keeps several head pairs re-uses its
// Qt tile, as long as the number of waves does not grow.
int head_pairs_per_item(const tucker_attn_desc& d, int n_qt, int n_hp) {
  if (d.causal) return 1;
  const long sms = sm_count();
  int best = 1;
  long best_cost = -1;
  for (int hpi = 1; hpi <= n_hp; ++hpi) {
    const long items = (long)n_qt * d.B * ((n_hp + hpi - 1) / hpi);
    const long cost = ((items + sms - 1) / sms) * hpi;
    if (best_cost < 0 || cost <= best_cost) { best_cost = cost; best = hpi; }
  }
  return best;
}

// Q: Qt [T, r2] when the kernel forms Qhat itself (G = GcatT [n_H * r3, r2] then), else Qhat [T, n_H * r3].
// Vt: the values transposed, [B, t3, value_ld(N)].
int umma_attention(Problem& p, bool fused, const bf16* Q, const bf16* G, const float4* rope, const bf16* K,
                   const bf16* Vt, bf16* O) {
  const tucker_attn_desc& d = p.d;
  CUtensorMap tmQ, tmG, tmK, tmV, tmO;
  {
    // O [B, N, nH, t3] as a 4-D tensor (t3, head, row, sequence); one store box = 64 columns x 128 rows of one head
    const uint64_t dims[4] = {(uint64_t)d.t3, (uint64_t)d.n_H, (uint64_t)d.N, (uint64_t)d.B};
    const uint64_t str[3] = {(uint64_t)d.t3, (uint64_t)d.n_H * d.t3, (uint64_t)d.N * d.n_H * d.t3};
    const uint32_t box[4] = {64, 1, 128, 1};
    if (!make_tmap(&tmO, O, 4, dims, str, box, CU_TENSOR_MAP_SWIZZLE_128B)) return TA_ERR_CUDA;
  }
  if (fused) {
    if (!tmap_3d(&tmQ, Q, d.r2, d.N, d.B, d.r2, (uint64_t)d.N * d.r2, 64, 128)) return TA_ERR_CUDA;
    if (!tmap_2d(&tmG, G, (uint64_t)d.r2, (uint64_t)d.n_H * d.r3, (uint64_t)d.r2, 64, (uint32_t)d.r3)) return TA_ERR_CUDA;
  } else {
    const uint64_t qcols = (uint64_t)d.n_H * d.r3;
    if (!tmap_3d(&tmQ, Q, qcols, d.N, d.B, qcols, (uint64_t)d.N * qcols, 64, 128)) return TA_ERR_CUDA;
    tmG = tmQ;
  }
  if (!tmap_3d(&tmK, K, d.r3, d.N, d.B, d.r3, (uint64_t)d.N * d.r3, 64, 128)) return TA_ERR_CUDA;
  // (keys, value column, sequence): keys beyond N are zero-filled by TMA, the row pitch is padded to 16 bytes
  if (!tmap_3d(&tmV, Vt, d.N, d.t3, d.B, (uint64_t)value_ld(d.N), (uint64_t)d.t3 * value_ld(d.N), 64, (uint32_t)d.t3))
    return TA_ERR_CUDA;
  attn::Params ap;
  ap.B = d.B; ap.N = d.N; ap.nH = d.n_H; ap.r2 = d.r2; ap.r3 = d.r3; ap.t3 = d.t3; ap.causal = d.causal;
  ap.n_qt = (d.N + attn::BQ - 1) / attn::BQ;
  ap.n_hp = (d.n_H + 1) / 2;
  ap.hp_per_item = fused ? head_pairs_per_item(d, ap.n_qt, ap.n_hp) : 1;
  ap.n_hg = (ap.n_hp + ap.hp_per_item - 1) / ap.hp_per_item;
  ap.fused = fused ? 1 : 0;
  ap.rope = (fused && d.rope) ? rope : nullptr;
  ap.O = O; ap.err = p.dev_err;
  static PerDeviceFlag attr;
  TA_CUDA_TRY(ensure_dynamic_smem(attr, (const void*)attn::k_attn_prefill, (int)attn::SMEM_BYTES));
  const long items = (long)ap.n_qt * d.B * ap.n_hg;
  if (items >= (1L << 30)) return TA_ERR_UNSUPPORTED_SHAPE;
  ap.n_items = (int)items;
  // persistent grid: one CTA per SM walks the item list (the unfused mode keeps one item per CTA)
  const long grid = fused ? std::min<long>(items, sm_count()) : items;
  prof_begin(p);
  (void)launch_pdl(attn::k_attn_prefill, dim3((unsigned)grid), dim3(attn::THREADS), attn::SMEM_BYTES, p.stream, tmQ, tmG,
                   tmK, tmV, tmO, ap);
  prof_end(p);
  TA_LAUNCH_CHECK(p);
  return TA_OK;
}

umma_gemm::Seg seg(int n_begin, int width, int mode, void* out, long ld) {
  umma_gemm::Seg s;
  s.n_begin = n_begin; s.width = width; s.mode = mode; s.out = out; s.ld = ld;
  s.out2 = nullptr; s.ld2 = 0; s.batch2 = 0;
  s.outT = nullptr; s.ldT = 0; s.batchT = 0;
  s.bmap = 0; s.b_n_off = n_begin;
  return s;
}

}  // namespace

bool fast_fwd_supported(const tucker_attn_desc& d) {
  auto ok32 = [](int r) { return r >= 32 && r <= 256 && r % 32 == 0; };
  if (!ok32(d.r2) || !ok32(d.r3) || !ok32(d.t2) || !ok32(d.t3)) return false;
  if (d.d_model % 64) return false;
  if ((long)d.B * d.N >= (1L << 24)) return false;
  return true;
}

size_t fast_fwd_workspace(const tucker_attn_desc& d) { return carve_fast(d, nullptr, nullptr); }

int fast_fwd(Problem& p) {
  const tucker_attn_desc& d = p.d;
  FastWs w;
  carve_fast(d, p.ws, &w);
  const int T = d.B * d.N;
  const float LOG2E = 1.4426950408889634f;
  const bool tc_attn = umma_attention_ok(d) && !(d.flags & TA_FLAG_FMA_ATTENTION);

  // ---- weight preparation: head-mode core contractions and the RoPE table, one launch ----
  {
    PrepParams pp;
    pp.C = (const bf16*)p.C; pp.U1 = (const bf16*)p.U1; pp.Ct = (const bf16*)p.Ct; pp.Ut1 = (const bf16*)p.Ut1;
    pp.GcatT = w.GcatT; pp.GtP = w.GtP; pp.rope = w.rope;
    pp.nH = d.n_H; pp.r1 = d.r1; pp.r2 = d.r2; pp.r3 = d.r3; pp.t1 = d.t1; pp.t2 = d.t2; pp.t3 = d.t3;
    pp.n_pos = d.N; pp.pos0 = d.pos0; pp.err = p.dev_err;
    pp.mult = tc_attn ? p.scale * LOG2E : p.scale;
    pp.freqs = rope_freqs(d);
    // one block per 32 x 32 tile of every G_h^T, one thread per 8 outputs of Gt / 4 entries of the table
    pp.g1 = d.n_H * (d.r2 / 32) * (d.r3 / 32);
    pp.g2 = (int)(((long)d.n_H * d.t2 * (d.t3 / 8) + PREP_THREADS - 1) / PREP_THREADS);
    pp.g3 = d.rope ? (int)((rope_table_units(d.N, d.r3) + PREP_THREADS - 1) / PREP_THREADS) : 0;
    (void)launch_pdl(k_prefill_prep, dim3(pp.g1 + pp.g2 + pp.g3), dim3(PREP_THREADS), 0, p.stream, pp);
    TA_LAUNCH_CHECK(p);
  }

  int rc;
  // ---- latent projections: one launch, the three factors read in place ([d, r], MN-major B) ----
  {
    umma_gemm::Params gp = {};
    gp.rope_tab = w.rope; gp.n_pos = d.N; gp.rope_half = d.r3 / 2;
    gp.b_mn_major = 1;
    const int kmode = d.rope ? umma_gemm::EP_BF16_ROPE : umma_gemm::EP_BF16;
    const int bn = common_bn(d.r2, d.r3, d.t3);
    if (!bn) return TA_ERR_UNSUPPORTED_SHAPE;
    // shared key / value projection: K is V, two segments instead of three
    const int nseg = p.shared_kv ? 2 : 3;
    gp.nseg = nseg;
    gp.seg[0] = seg(0, d.r2, umma_gemm::EP_BF16, w.Qt, d.r2);
    gp.seg[1] = seg(d.r2, d.r3, kmode, w.K, d.r3);
    gp.seg[2] = seg(d.r2 + d.r3, d.t3, umma_gemm::EP_BF16, w.V, d.t3);
    for (int i = 0; i < 3; ++i) { gp.seg[i].bmap = i; gp.seg[i].b_n_off = 0; }
    if (p.Kc) {
      // one shared cache with latent RoPE holds the un-rotated latent rows: only the value segment is copied out
      if (!p.shared_rope) { gp.seg[1].out2 = p.Kc; gp.seg[1].ld2 = d.r3; gp.seg[1].batch2 = (long)p.Lmax * d.r3; }
      gp.seg[2].out2 = p.Vc; gp.seg[2].ld2 = d.t3; gp.seg[2].batch2 = (long)p.Lmax * d.t3;
    }
    if (tc_attn) {
      // the tensor-core attention takes the value tile with the key index contiguous (K-major operand of P V)
      umma_gemm::Seg& vs = gp.seg[nseg - 1];
      vs.outT = w.Vt; vs.ldT = value_ld(d.N); vs.batchT = (long)d.t3 * value_ld(d.N);
      if (!p.shared_kv) vs.out = nullptr;   // nobody reads the token-major copy
    }
    const BOperand bops[3] = {{(const bf16*)p.U2, d.r2, d.r2}, {(const bf16*)p.U3, d.r3, d.r3}, {(const bf16*)p.Ut3, d.t3, d.t3}};
    const int ntot = d.r2 + d.r3 + (p.shared_kv ? 0 : d.t3);
    // When X does not fit the L2 cache, each segment's pass over it would come from HBM again; one
    // CTA then takes all segments of its 128 rows (one accumulator per segment) and X is read once.
    // (Measured: with X resident in L2 the three narrower CTAs per row tile are the faster form.)
    const bool one_block_each = d.r2 == bn && d.r3 == bn && d.t3 == bn;
    if (one_block_each && (size_t)T * d.d_model * sizeof(bf16) > l2_bytes() && (T + 127) / 128 >= sm_count() * 4 / 5)
      gp.ncb = nseg;
    gp.early = 1;   // X and the factors are inputs of the call: only the epilogue needs the preparation kernel's table
    if ((rc = launch_gemm(p, (const bf16*)p.X, d.d_model, T, d.d_model, bops, 3, ntot, bn, gp))) return rc;
  }
  const bf16* Vlat = p.shared_kv ? w.K : w.V;   // latent values
  const bool fuse_q = tc_attn && attention_fuses_qhat(d);
  // ---- per-head queries with latent RoPE (only when the attention kernel does not form them) ----
  if (!fuse_q) {
    umma_gemm::Params gp = {};
    gp.rope_tab = w.rope; gp.n_pos = d.N; gp.rope_half = d.r3 / 2;
    gp.nseg = 1;
    gp.seg[0] = seg(0, d.n_H * d.r3, d.rope ? umma_gemm::EP_BF16_ROPE : umma_gemm::EP_BF16, w.Qhat, (long)d.n_H * d.r3);
    const BOperand bop = {w.GcatT, d.r2, d.n_H * d.r3};
    if ((rc = launch_gemm(p, w.Qt, d.r2, T, d.r2, &bop, 1, d.n_H * d.r3, pick_bn(d.r3), gp))) return rc;
  }
  // ---- attention ----
  if (tc_attn) {
    if ((rc = umma_attention(p, fuse_q, fuse_q ? w.Qt : w.Qhat, w.GcatT, w.rope, w.K, w.Vt, w.O))) return rc;
  } else {
    if ((rc = simt_attention_bf16(p, w.Qhat, w.K, Vlat, w.O))) return rc;
  }
  // ---- output side ----
  if (d.t2 <= 128 && d.d_model % zy::BN2 == 0 && !(d.flags & TA_FLAG_SEPARATE_OUTPUT_GEMMS)) {
    // one kernel: Z = O Gt^T stays on chip and feeds Y = Z Ut2^T
    const int K1 = d.n_H * d.t3;
    CUtensorMap tmO, tmG, tmU;
    if (!tmap_2d(&tmO, w.O, (uint64_t)K1, (uint64_t)T, (uint64_t)K1, 64, 128)) return TA_ERR_CUDA;
    if (!tmap_2d(&tmG, w.GtP, (uint64_t)K1, (uint64_t)d.t2, (uint64_t)K1, 64, (uint32_t)d.t2)) return TA_ERR_CUDA;
    if (!tmap_2d(&tmU, p.Ut2, (uint64_t)d.t2, (uint64_t)d.d_model, (uint64_t)d.t2, 64, 128)) return TA_ERR_CUDA;
    zy::Params zp;
    zp.M = T; zp.K1 = K1; zp.t2 = d.t2; zp.d = d.d_model; zp.stages = zy::MAX_STAGES;
    zp.Y = (bf16*)p.Y; zp.err = p.dev_err;
    static PerDeviceFlag attr;
    TA_CUDA_TRY(ensure_dynamic_smem(attr, (const void*)zy::k_zy_fused, (int)zy::smem_bytes(zy::MAX_STAGES)));
    (void)launch_pdl(zy::k_zy_fused, dim3((T + 127) / 128), dim3(zy::THREADS), zy::smem_bytes(zp.stages), p.stream, tmO, tmG,
                     tmU, zp);
    TA_LAUNCH_CHECK(p);
  } else {
    {
      umma_gemm::Params gp = {};
      gp.n_pos = d.N;
      gp.nseg = 1;
      gp.seg[0] = seg(0, d.t2, umma_gemm::EP_BF16, w.Z, d.t2);
      const BOperand bop = {w.GtP, (long)d.n_H * d.t3, d.t2};
      if ((rc = launch_gemm(p, w.O, (long)d.n_H * d.t3, T, d.n_H * d.t3, &bop, 1, d.t2, pick_bn(d.t2), gp))) return rc;
    }
    {
      umma_gemm::Params gp = {};
      gp.n_pos = d.N;
      gp.nseg = 1;
      gp.seg[0] = seg(0, d.d_model, umma_gemm::EP_BF16, p.Y, d.d_model);
      const BOperand bop = {(const bf16*)p.Ut2, d.t2, d.d_model};
      // short K (t2) and a wide N: 256-wide tiles halve the number of CTAs and of A-tile reads
      const int bn = (d.d_model % 256 == 0) ? 256 : pick_bn(d.d_model);
      if ((rc = launch_gemm(p, w.Z, d.t2, T, d.t2, &bop, 1, d.d_model, bn, gp))) return rc;
    }
  }
  return TA_OK;
}

int umma_gemm_f32_partials(Problem& p, const bf16* A, long lda, int M, const bf16* B, long ldb, int N, int K, int splits,
                           float* out, long split_stride) {
  if (K % 64 || N % 64 || splits < 1 || (K / 64) % splits) return TA_ERR_UNSUPPORTED_SHAPE;
  umma_gemm::Params gp = {};
  gp.nseg = 1;
  gp.seg[0] = seg(0, N, umma_gemm::EP_F32, out, N);
  gp.kb_per_split = (K / 64) / splits;
  gp.split_stride = split_stride;
  const BOperand bop = {B, ldb, N};
  return launch_gemm(p, A, lda, M, K, &bop, 1, N, pick_bn(N), gp, splits);
}

// ---------------------------------------------------------------------------------------------
// decode
// ---------------------------------------------------------------------------------------------
namespace {

constexpr int kProjSplits = 16;

// Device properties, looked up once per device ordinal (a process may drive several GPUs).
struct DeviceProps {
  std::mutex m;
  int sms[kMaxDevices] = {};
  size_t l2[kMaxDevices] = {};
};
DeviceProps g_props;

int current_device_slot() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
  return dev;
}

int sm_count() {
  const int dev = current_device_slot();
  std::lock_guard<std::mutex> lock(g_props.m);
  if (!g_props.sms[dev]) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    g_props.sms[dev] = n;
  }
  return g_props.sms[dev];
}

size_t l2_bytes() {
  const int dev = current_device_slot();
  std::lock_guard<std::mutex> lock(g_props.m);
  if (!g_props.l2[dev]) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrL2CacheSize, dev) != cudaSuccess || v <= 0) v = 126 << 20;
    g_props.l2[dev] = (size_t)v;
  }
  return g_props.l2[dev];
}

// number of K splits of the decode projection GEMM: the largest divisor of the K-block count <= kProjSplits
int proj_splits(int d_model) {
  const int nkb = d_model / 64;
  for (int s = kProjSplits; s > 1; --s)
    if (nkb % s == 0) return s;
  return 1;
}

int decode_grid() { return sm_count() < dec::MAX_GRID ? sm_count() : dec::MAX_GRID; }

struct FastDecWs {
  float* proj_part;   // [splits][Mpad][r2 + r3 + t3] split-K partial sums of the new tokens' projections
  bf16 *knew, *vnew;  // [B][r3] rotated new key, [B][t3] new value
  bf16* qhat;         // [B][n_H][r3] rotated, scaled per-head queries
  bf16* z;            // [B][t2]
  float *part_o, *part_ml;
};

size_t carve_fast_dec(const tucker_attn_desc& d, char* base, FastDecWs* w) {
  Carver c(base);
  FastDecWs t;
  const size_t Mpad = (size_t)((d.B + 127) / 128) * 128;
  const size_t ncol = (size_t)d.r2 + d.r3 + d.t3;
  t.proj_part = c.take<float>((size_t)kProjSplits * Mpad * ncol);
  t.knew = c.take<bf16>((size_t)d.B * d.r3);
  t.vnew = c.take<bf16>((size_t)d.B * d.t3);
  t.qhat = c.take<bf16>((size_t)d.B * d.n_H * d.r3);
  t.z = c.take<bf16>((size_t)d.B * d.t2);
  const size_t slots = (size_t)dec::MAX_GRID + d.B;
  t.part_o = c.take<float>(slots * 32 * d.t3);
  t.part_ml = c.take<float>(slots * 64);
  if (w) *w = t;
  return c.off;
}

// The cache-streaming kernel (tcgen05, keys on the M dimension, ranks at run time).  With one shared cache and
// latent RoPE (p.shared_rope) the instance with the rotation warpgroup runs: the cache holds un-rotated rows.
template <bool ROT, int R3C>
int launch_dec_attn_inst(Problem& p, const CUtensorMap& tmK, const CUtensorMap& tmV, const CUtensorMap& tmQ,
                         const decu::Params& up, int grid, const dec::RopeFreqs& freqs) {
  static PerDeviceFlag attr;
  TA_CUDA_TRY(ensure_dynamic_smem(attr, (const void*)decu::k_dec_attn_umma<ROT, R3C>, (int)decu::SMEM_BYTES));
  prof_begin(p);
  (void)launch_pdl(decu::k_dec_attn_umma<ROT, R3C>, dim3(grid), dim3(ROT ? decu::THREADS_ROT : decu::THREADS),
                   decu::SMEM_BYTES, p.stream, tmK, tmV, tmQ, up, freqs);
  prof_end(p);
  TA_LAUNCH_CHECK(p);
  return TA_OK;
}

int launch_dec_attn_umma(Problem& p, const CUtensorMap& tmK, const CUtensorMap& tmV, const dec::Params& dp, int grid) {
  const tucker_attn_desc& d = p.d;
  CUtensorMap tmQ;   // Qhat [B * n_H rows, r3]: one box = 32 rows (all heads of a sequence) x 64 columns
  if (!tmap_2d(&tmQ, dp.qhat, (uint64_t)d.r3, (uint64_t)d.B * d.n_H, (uint64_t)d.r3, 64, 32)) return TA_ERR_CUDA;
  decu::Params up;
  up.B = dp.B; up.nH = dp.nH; up.Lmax = dp.Lmax; up.r3 = d.r3; up.t3 = d.t3; up.shared_kv = dp.shared_kv;
  up.cache_len = dp.cache_len; up.knew = dp.knew; up.vnew = dp.vnew;
  up.part_o = dp.part_o; up.part_ml = dp.part_ml; up.err = dp.err;
  if (p.shared_rope) {
    const dec::RopeFreqs freqs = rope_freqs(d);
    switch (d.r3) {
      case 64: return launch_dec_attn_inst<true, 64>(p, tmK, tmV, tmQ, up, grid, freqs);
      case 96: return launch_dec_attn_inst<true, 96>(p, tmK, tmV, tmQ, up, grid, freqs);
      case 128: return launch_dec_attn_inst<true, 128>(p, tmK, tmV, tmQ, up, grid, freqs);
      default: return TA_ERR_UNSUPPORTED_SHAPE;
    }
  }
  dec::RopeFreqs none = {};
  return launch_dec_attn_inst<false, 0>(p, tmK, tmV, tmQ, up, grid, none);
}

bool dec_rank_ok(int r3, int t3) {
  return (r3 == 128 && t3 == 128) || (r3 == 64 && t3 == 64) || (r3 == 96 && t3 == 96) || (r3 == 128 && t3 == 64) ||
         (r3 == 64 && t3 == 128);
}

}  // namespace

bool fast_decode_supported(const tucker_attn_desc& d, int32_t Lmax) {
  auto ok32 = [](int r) { return r >= 32 && r <= 256 && r % 32 == 0; };
  if (!ok32(d.r2) || !ok32(d.t2) || !dec_rank_ok(d.r3, d.t3)) return false;
  if (d.d_model % 64 || d.n_H > 32 || d.B > 4096) return false;
  if (d.r1 > 32 || d.t1 > 32) return false;      // shared-memory tables of the per-sequence kernels
  (void)Lmax;
  return true;
}

size_t fast_decode_workspace(const tucker_attn_desc& d, int32_t) { return carve_fast_dec(d, nullptr, nullptr); }

// Launch sequence of one decode step (Eq. 9):
//   1  split-K GEMM   partial [qt | k | v] = x [U2 | U3 | Ut3]           (factors read in place)
//   2  k_dec_qhat     finish the projections, latent RoPE, cache append, per-head queries (core
//                     contracted with the query first; no per-head G_h)
//   3  k_dec_attn_umma  stream the latent caches once, all heads per tile (tcgen05)
//   4  k_dec_out      merge the partials, output-side core -> z
//   5  GEMM           y = z Ut2^T
int fast_decode(Problem& p) {
  const tucker_attn_desc& d = p.d;
  FastDecWs w;
  carve_fast_dec(d, p.ws, &w);
  const float LOG2E = 1.4426950408889634f;
  const int ncol = d.r2 + d.r3 + d.t3;
  const int Mpad = (d.B + 127) / 128 * 128;
  const int splits = proj_splits(d.d_model);
  int rc;
  // ---- 1: projections of the new tokens, split over K ----
  {
    umma_gemm::Params gp = {};
    gp.b_mn_major = 1;
    gp.nseg = 3;
    gp.seg[0] = seg(0, d.r2, umma_gemm::EP_F32, w.proj_part, ncol);
    gp.seg[1] = seg(d.r2, d.r3, umma_gemm::EP_F32, w.proj_part + d.r2, ncol);
    gp.seg[2] = seg(d.r2 + d.r3, d.t3, umma_gemm::EP_F32, w.proj_part + d.r2 + d.r3, ncol);
    for (int i = 0; i < 3; ++i) { gp.seg[i].bmap = i; gp.seg[i].b_n_off = 0; }
    gp.kb_per_split = (d.d_model / 64) / splits;
    gp.split_stride = (long)Mpad * ncol;
    const int bn = (d.r2 % 64 == 0 && d.r3 % 64 == 0 && d.t3 % 64 == 0) ? 64 : 32;
    const BOperand bops[3] = {{(const bf16*)p.U2, d.r2, d.r2}, {(const bf16*)p.U3, d.r3, d.r3}, {(const bf16*)p.Ut3, d.t3, d.t3}};
    if ((rc = launch_gemm(p, (const bf16*)p.X, d.d_model, d.B, d.d_model, bops, 3, ncol, bn, gp, splits))) return rc;
  }
  // ---- 2: finish, RoPE, append, per-head queries ----
  {
    const dim3 grid(d.B, d.r3 / dec::DQ_CW);
    const dec::RopeFreqs freqs = rope_freqs(d);
    auto launch = [&](auto kernel) {
      (void)launch_pdl(kernel, grid, dim3(256), 0, p.stream, w.proj_part, splits, (long)Mpad * ncol, d.n_H, d.r1, d.r2,
                       d.r3, d.t3, (const bf16*)p.C, (const bf16*)p.U1, p.scale * LOG2E, w.qhat, w.knew, w.vnew,
                       (bf16*)p.Kc, (bf16*)p.Vc, p.Lmax, p.cache_len, d.rope, freqs, p.append, p.shared_rope ? 2 : p.shared_kv, p.dev_err);
    };
    switch ((d.r2 + 63) / 64) {
      case 1: launch(dec::k_dec_qhat<1>); break;
      case 2: launch(dec::k_dec_qhat<2>); break;
      case 3: launch(dec::k_dec_qhat<3>); break;
      default: launch(dec::k_dec_qhat<4>); break;
    }
    TA_LAUNCH_CHECK(p);
  }
  // ---- 3: attention over the latent cache ----
  {
    CUtensorMap tmK, tmV;
    if (!tmap_3d(&tmK, p.Kc, d.r3, p.Lmax, d.B, d.r3, (uint64_t)p.Lmax * d.r3, 64, 128)) return TA_ERR_CUDA;
    if (!tmap_3d(&tmV, p.Vc, d.t3, p.Lmax, d.B, d.t3, (uint64_t)p.Lmax * d.t3, 64, 128)) return TA_ERR_CUDA;
    dec::Params dp;
    dp.B = d.B; dp.nH = d.n_H; dp.Lmax = p.Lmax; dp.grid = decode_grid();
    dp.shared_kv = p.shared_kv;
    dp.cache_len = p.cache_len; dp.qhat = w.qhat; dp.knew = w.knew; dp.vnew = w.vnew;
    dp.part_o = w.part_o; dp.part_ml = w.part_ml; dp.err = p.dev_err;
    rc = launch_dec_attn_umma(p, tmK, tmV, dp, dp.grid);
    if (rc) return rc;
    // ---- 4: merge the partials, output-side core ----
    static PerDeviceFlag out_attr;
    TA_CUDA_TRY(ensure_dynamic_smem(out_attr, (const void*)dec::k_dec_out, (int)dec::dec_out_smem(32, 32, 128)));
    (void)launch_pdl(dec::k_dec_out, dim3(d.B, dec::DO_JS), dim3(256), dec::dec_out_smem(d.n_H, d.t1, d.t3), p.stream,
                     w.part_o, w.part_ml, p.cache_len, d.B, p.Lmax, d.n_H, d.t1, d.t2, d.t3, dp.grid, (const bf16*)p.Ct,
                     (const bf16*)p.Ut1, w.z, p.dev_err);
    TA_LAUNCH_CHECK(p);
  }
  // ---- 5: y = z Ut2^T ----
  {
    umma_gemm::Params gp = {};
    gp.n_pos = d.B;
    gp.nseg = 1;
    gp.seg[0] = seg(0, d.d_model, umma_gemm::EP_BF16, p.Y, d.d_model);
    const BOperand bop = {(const bf16*)p.Ut2, d.t2, d.d_model};
    gp.early = 2;   // the factor Ut2 is an input of the call; z comes from the preceding kernel
    if ((rc = launch_gemm(p, w.z, d.t2, d.B, d.t2, &bop, 1, d.d_model, pick_bn(d.d_model), gp))) return rc;
  }
  return TA_OK;
}

}  // namespace ta

// ---- self-test of the bounded waits -------------------------------------------------------
namespace ta {
namespace {
// One CTA, two warps.  Lane 0 of warp 0 waits on an mbarrier that nothing ever arrives on; its wait gives up
// after `budget_cycles`, raises the CTA's abort flag and sets the device error word.  Lane 0 of warp 1 waits
// on a second such barrier with the full budget and must come back through the abort flag.  out[0] / out[1]
// receive what the two waits returned (0 = gave up), out[2] the cycles the second wait took.
__global__ void k_wait_selftest(unsigned int* err, long long budget_cycles, int* out) {
  __shared__ uint64_t bar[2];
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    sm100::mbar_init(&bar[0], 1);
    sm100::mbar_init(&bar[1], 1);
    sm100::fence_barrier_init();
  }
  __syncthreads();
  sm100::Abort ab{&abort_flag, err};
  if (threadIdx.x == 0) out[0] = sm100::mbar_wait(&bar[0], 0, ab, budget_cycles) ? 1 : 0;
  if (threadIdx.x == 32) {
    const long long t0 = clock64();
    out[1] = sm100::mbar_wait(&bar[1], 0, ab) ? 1 : 0;
    out[2] = (int)((clock64() - t0) >> 10);
  }
}
}  // namespace
int wait_selftest(unsigned int* dev_err, int budget_us, int* out_dev, cudaStream_t stream) {
  const long long cycles = (long long)budget_us * 2000LL;      // about 2 GHz
  k_wait_selftest<<<1, 64, 0, stream>>>(dev_err, cycles, out_dev);
  return cudaGetLastError() == cudaSuccess ? TA_OK : TA_ERR_CUDA;
}
}  // namespace ta
