/*
 * tucker_attn.h -- C ABI of the B200 (sm_100a) Tucker-attention forward library.
 *
 * One Tucker-factorised attention layer ("Tucker Attention", Definition 1 of the paper):
 * the pre-softmax tensor  W  = C  x_1 U1  x_2 U2  x_3 U3   (n_H x d x d, ranks r1,r2,r3) and
 * the post-softmax tensor Wt = Ct x_1 Ut1 x_2 Ut2 x_3 Ut3  (ranks t1,t2,t3; mode 2 = output,
 * mode 3 = value because the transposed per-head matrices are stacked, Eq. 3) are never
 * formed.  The library evaluates Eq. 6 ("full-rank MHA" on these tensors) in the order of
 * Sec. 3 of the paper:
 *
 *   Qt = X U2,  K = X U3,  V = X Ut3                 latent projections; K, V are the KV cache (Sec. 3.1)
 *   G_h  = sum_a U1[h,a]  C[a,:,:]                   head-mode core contraction C x_1 U1 (Def. 2, Sec. 3.3)
 *   Gt_h = sum_a Ut1[h,a] Ct[a,:,:]
 *   Qhat_h = Qt G_h                                  per-head latent queries (Def. 2)
 *   latent RoPE: Qhat_{h,m} R(m,r3),  K_n R(n,r3)    rotation in the latent key dimension (Eq. 12, App. C.2)
 *   S_h = Qhat_h K^T * scale, causal mask, row softmax (online, never materialised; Sec. 3.3)
 *   O_h = P_h V
 *   Z   = sum_h O_h Gt_h^T ;  Y = Z Ut2^T            value/output-side factors (Eqs. 5-6)
 *
 * and the cached decode step of Eq. 9 for one new token per sequence.
 *
 * General conventions
 *   - Every data pointer is CALLER-OWNED DEVICE memory unless stated otherwise; row-major,
 *     contiguous, 16-byte aligned.  The library never allocates, frees or keeps a pointer
 *     after the call returns.  Scratch space is passed in as `workspace`.
 *   - Calls are asynchronous on `cuda_stream` (a cudaStream_t cast to void*; NULL = default
 *     stream).  No host synchronisation happens inside a call, and tucker_attn_fwd /
 *     tucker_attn_decode read no device memory on the host, so (after one ordinary call per
 *     device, which sets kernel attributes) they can be captured into a CUDA graph and replayed
 *     on new contents of the same buffers.
 *   - Storage type (`dtype`): TA_DTYPE_F32 = float everywhere (plain FMA arithmetic, no
 *     tensor cores); TA_DTYPE_BF16 = __nv_bfloat16 for X, weights, caches and Y with fp32
 *     accumulation.
 *   - Return value: TA_OK (0) or a negative tucker_attn_status.  Nothing throws, aborts or
 *     traps.  Argument errors are detected on the host before anything is launched.
 *   - RoPE convention: interleaved coordinate pairs (2i, 2i+1) of the r3 latent key
 *     coordinates, angle pos * rope_base^(-2i/r3); x'[2i] = x[2i] cos - x[2i+1] sin,
 *     x'[2i+1] = x[2i] sin + x[2i+1] cos; the same rotation for Qhat rows and K rows.
 *     The K cache holds ROTATED keys.
 */
#ifndef TUCKER_ATTN_H_
#define TUCKER_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define TA_API __attribute__((visibility("default")))
#else
#define TA_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  TA_OK = 0,
  TA_ERR_INVALID_ARG = -1,         /* null pointer, non-positive size, rank/shape inconsistency, odd r3 with rope */
  TA_ERR_UNSUPPORTED_SHAPE = -2,   /* a rank or size outside what the kernels were built for */
  TA_ERR_WORKSPACE_TOO_SMALL = -3, /* workspace_bytes < tucker_attn_*_workspace_bytes(...) */
  TA_ERR_CUDA = -4,                /* a CUDA runtime / driver call failed (launch, tensor map) */
  TA_ERR_DEVICE_TIMEOUT = -5       /* a bounded device-side wait gave up; returned by tucker_attn_sync_status only
                                      (the launching call itself is asynchronous and has returned TA_OK by then) */
} tucker_attn_status;

enum { TA_DTYPE_F32 = 0, TA_DTYPE_BF16 = 1 };

/* Problem descriptor (host memory, read during the call only). */
typedef struct {
  int32_t B;          /* independent sequences (no cross-sequence terms) */
  int32_t N;          /* tokens per sequence (prefill); ignored by decode */
  int32_t d_model;    /* embedding width d */
  int32_t n_H;        /* heads; d_model % n_H == 0; d_H = d_model / n_H */
  int32_t r1, r2, r3; /* pre-softmax tensor: head, query, key ranks   (Definition 1) */
  int32_t t1, t2, t3; /* post-softmax tensor: head, output, value ranks (Definition 1) */
  int32_t causal;     /* 1: key n visible to query m iff n <= m */
  int32_t rope;       /* 1: latent RoPE in r3 (Definition 2); needs r3 even */
  float   rope_base;  /* e.g. 10000, 500000 */
  int32_t pos0;       /* absolute position of token 0 of every sequence (prefill) */
  float   scale;      /* softmax scale; <= 0 selects 1/sqrt(d_model/n_H) (Eq. 4) */
  int32_t dtype;      /* TA_DTYPE_F32 or TA_DTYPE_BF16 */
  int32_t flags;      /* TA_FLAG_* bits, 0 = let the library choose */
} tucker_attn_desc;

enum {
  TA_FLAG_FORCE_GENERIC = 1,          /* run the shape-generic FMA kernels even where a tensor-core path exists */
  /* Alternative routes through the bf16 tensor-core prefill path; same results within rounding, kept so that
   * the routes can be checked against each other: */
  TA_FLAG_FMA_ATTENTION = 0x200,      /* tensor-core GEMMs, but the attention itself on the FMA kernel */
  TA_FLAG_SEPARATE_QUERIES = 0x400,   /* per-head queries from a separate GEMM instead of the attention prologue */
  TA_FLAG_SEPARATE_OUTPUT_GEMMS = 0x800  /* Z and Y from two GEMM launches instead of the fused output kernel */
};

/* Bytes of scratch the corresponding call needs for this descriptor (0 on invalid descriptor). */
TA_API size_t tucker_attn_fwd_workspace_bytes(const tucker_attn_desc* desc);
TA_API size_t tucker_attn_decode_workspace_bytes(const tucker_attn_desc* desc, int32_t Lmax);

/*
 * Prefill forward of one layer (Definition 1 evaluated through Eq. 6; Sec. 3.1-3.3).
 *   X    [B, N, d_model]                       in
 *   C    [r1, r2, r3]   U1  [n_H, r1]   U2  [d_model, r2]   U3  [d_model, r3]      in
 *   Ct   [t1, t2, t3]   Ut1 [n_H, t1]   Ut2 [d_model, t2]   Ut3 [d_model, t3]      in
 *   Y    [B, N, d_model]                       out
 *   Kcache_out [B, Lmax, r3], Vcache_out [B, Lmax, t3]   optional out (both NULL or both set,
 *        Lmax >= N): rows 0..N-1 of every sequence receive the rotated latent keys and the
 *        latent values (the KV cache of Sec. 3.1); other rows are left untouched.
 *   workspace: >= tucker_attn_fwd_workspace_bytes(desc) bytes, 256-byte aligned.
 * All steps, including the weight-only core contraction, run inside the call.
 *
 * Shared key / value projection (Sec. 3.1, "L^KV = X U3"): pass the SAME pointer for U3 and Ut3
 * (then r3 == t3).  Kcache_out may then equal Vcache_out: ONE cache of N r3 entries instead of 2 N r3.
 * Without RoPE the latent keys are the latent values and are projected once.  With latent RoPE
 * (Definition 2) the keys are the rotated latent rows and the values the un-rotated ones; the one cache
 * receives the UN-rotated rows (the paper does not say what the single cache holds in this case: the
 * un-rotated row serves as the value as it is, and its key is re-formed by rotating it when it is read).
 * Kcache_out == Vcache_out with distinct U3 / Ut3 pointers or r3 != t3 is TA_ERR_INVALID_ARG.
 */
TA_API int tucker_attn_fwd(const tucker_attn_desc* desc, const void* X,
                    const void* C, const void* U1, const void* U2, const void* U3,
                    const void* Ct, const void* Ut1, const void* Ut2, const void* Ut3,
                    void* Y, void* Kcache_out, void* Vcache_out, int32_t Lmax,
                    void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * One cached decode step (Eq. 9, "KV Caching"): for every sequence b the new token x[b] at
 * position L = cache_len[b] attends to cache slots 0..L-1 and to itself.
 *   x         [B, d_model]                     in
 *   Kcache    [B, Lmax, r3] rotated latent keys, Vcache [B, Lmax, t3]   in (and out if append)
 *   cache_len [B] int32, DEVICE memory; 0 <= cache_len[b] < Lmax (checked on the device: an
 *             out-of-range entry is clamped and flagged in the device error word)
 *   append    1: the new rotated key / value are also written to slot cache_len[b]
 *             (the caller increments its lengths); 0: the caches are not modified
 *   y         [B, d_model]                     out
 *   desc->N, desc->pos0, desc->causal are ignored.
 *
 * Shared latent cache (Sec. 3.1): Kcache == Vcache is accepted when U3 == Ut3 (same pointer) and
 * r3 == t3; the step then reads every cached row once (half the bytes) and appends one row.  With
 * rope == 1 that cache holds UN-rotated latent rows (see tucker_attn_fwd): every key tile is rotated
 * by R(n, r3) on chip after it has been loaded, the values are the rows as stored, and the appended
 * row is the un-rotated one.  Any other call with Kcache == Vcache is TA_ERR_INVALID_ARG.
 */
TA_API int tucker_attn_decode(const tucker_attn_desc* desc, const void* x,
                       const void* C, const void* U1, const void* U2, const void* U3,
                       const void* Ct, const void* Ut1, const void* Ut2, const void* Ut3,
                       void* Kcache, void* Vcache, int32_t Lmax,
                       const int32_t* cache_len, int32_t append,
                       void* y, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Decode step without a caller-supplied workspace (the paper has no counterpart: this is a
 * packaging variant of tucker_attn_decode, same arithmetic, same kernels).
 *
 * For callers that cannot allocate device memory on this path -- a serving loop whose memory
 * was carved up once at start-up by an allocator it does not own, a plug-in whose host
 * framework forbids cudaMalloc outside its own pool, a latency-critical loop that cannot
 * take the device-wide synchronisation cudaMalloc / cudaFree imply.  The scratch space lives
 * in a static device array of TA_STATIC_SCRATCH_BYTES inside the library; every GPU that
 * loads the library holds that much memory until the process exits.  The call itself makes
 * no cudaMalloc / cudaFree and uses no allocating library routine.
 *
 * Arguments are those of tucker_attn_decode without `workspace` / `workspace_bytes`; inputs
 * and outputs remain caller-owned device memory.
 *
 * Limits and behaviour
 *   - Returns TA_ERR_WORKSPACE_TOO_SMALL, before anything is launched, when
 *     tucker_attn_decode_workspace_bytes(desc, Lmax) exceeds TA_STATIC_SCRATCH_BYTES
 *     (the benchmark decode shape, B = 64, n_H = 32, d = 4096, ranks 128, fits); use
 *     tucker_attn_decode with your own buffer for larger problems.  Other errors as for
 *     tucker_attn_decode.
 *   - The first call on each device looks up the array's device address (with that device
 *     current) and caches it; make that first call outside any stream capture.
 *   - All calls on a device share the one array.  Calls that may overlap on the GPU
 *     (different streams, or different host threads) race on it: serialise them, e.g. keep
 *     them on one stream.  Nothing in the scratch needs to start at zero -- each call
 *     rewrites what it reads -- so back-to-back calls need no clearing in between.
 */
#define TA_STATIC_SCRATCH_BYTES (16u << 20)
TA_API int tucker_attn_decode_static(const tucker_attn_desc* desc, const void* x,
                              const void* C, const void* U1, const void* U2, const void* U3,
                              const void* Ct, const void* Ut1, const void* Ut2, const void* Ut3,
                              void* Kcache, void* Vcache, int32_t Lmax,
                              const int32_t* cache_len, int32_t append,
                              void* y, void* cuda_stream);

/*
 * Weight packers: the paper's special cases as Tucker attention (Sec. 2.2; Lemma 1 and
 * Theorems 1-3 and their proofs).  They write the two cores and six factors that
 * tucker_attn_fwd / tucker_attn_decode take, so that MHA, GQA / MQA and MLA weights run
 * through the same kernels.  All pointers are caller-owned device memory, row-major, of the
 * storage type `dtype` (inputs and outputs alike); asynchronous on `cuda_stream`; no
 * workspace.  d_H = d_model / n_H (d_model must be a multiple of n_H).  Returns TA_OK,
 * TA_ERR_INVALID_ARG (null pointer, bad sizes or dtype) or TA_ERR_CUDA.
 *
 * tucker_pack_gqa: n_H query heads, n_G <= n_H key / value heads, head i using group
 * floor(i n_G / n_H) (n_G = 1 is MQA).  Inputs WQ [d, d], WKg [d, n_G d_H], WVg [d, n_G d_H]
 * (heads are column blocks of width d_H), WO [d, d] (head i = rows i d_H ..).  Outputs,
 * ranks (n_H, d, n_G d_H) for both tensors:
 *   C, Ct [n_H, d, n_G d_H] selector cores, U1, Ut1 [n_H, n_H] = I, U2 [d, d] = WQ,
 *   U3 [d, n_G d_H] = WKg, Ut2 [d, d] = WO^T, Ut3 [d, n_G d_H] = WVg.
 * tucker_pack_mha: the same with n_G = n_H (WK, WV [d, d]).
 * The result equals sum_i softmax(X WQ_i (X WK_g(i))^T / sqrt(d_H)) X WV_g(i) WO_i exactly
 * (Eq. 1); with rope = 1 the latent RoPE acts on the n_G d_H key coordinates as one
 * rotation over the whole width, which is NOT the per-head RoPE of a trained MHA / GQA model
 * unless n_G = 1 (the MQA case of App. C.2).
 *
 * tucker_pack_mla: MLA without RoPE.  Inputs WDQ [d, dcq], WUQ [dcq, d], WDKV [d, dck],
 * WUK [dck, d], WDV [d, dck] (pass WDKV again for a shared latent), WUV [dck, d], WO [d, d];
 * the up-projections are column-split into heads.  Outputs, ranks (n_H, dcq, dck) and
 * (n_H, d, dck): C [n_H, dcq, dck] with C[i] = WUQ_i WUK_i^T, Ct [n_H, d, dck] with
 * Ct[i, o, c] = (WUV_i WO_i)[c, o], U1, Ut1 [n_H, n_H] = I, U2 [d, dcq] = WDQ,
 * U3 [d, dck] = WDKV, Ut2 [d, d] = I, Ut3 [d, dck] = WDV.
 */
TA_API int tucker_pack_gqa(int32_t d_model, int32_t n_H, int32_t n_G, int32_t dtype,
                    const void* WQ, const void* WKg, const void* WVg, const void* WO,
                    void* C, void* U1, void* U2, void* U3, void* Ct, void* Ut1, void* Ut2, void* Ut3,
                    void* cuda_stream);
TA_API int tucker_pack_mha(int32_t d_model, int32_t n_H, int32_t dtype,
                    const void* WQ, const void* WK, const void* WV, const void* WO,
                    void* C, void* U1, void* U2, void* U3, void* Ct, void* Ut1, void* Ut2, void* Ut3,
                    void* cuda_stream);
TA_API int tucker_pack_mla(int32_t d_model, int32_t n_H, int32_t dcq, int32_t dck, int32_t dtype,
                    const void* WDQ, const void* WUQ, const void* WDKV, const void* WUK,
                    const void* WDV, const void* WUV, const void* WO,
                    void* C, void* U1, void* U2, void* U3, void* Ct, void* Ut1, void* Ut2, void* Ut3,
                    void* cuda_stream);

/*
 * HOSVD initialiser: pretrained MHA weights -> Tucker-attention weights (App. C.1, paragraph "MHA to Tucker
 * Attention": a higher-order SVD of the n_H x d x d weight tensors), with the singular spectra of the three mode
 * unfoldings that Sec. 2.1 ("Informed Compression Across All Modes") uses to choose the ranks.  fp32 throughout;
 * all pointers caller-owned device memory; asynchronous on `cuda_stream`; no host synchronisation.
 *
 * tucker_mha_weight_tensors: W[i] = WQ_i WK_i^T and Wt[i] = (WV_i WO_i)^T (Eqs. 2-3: the per-head matrices,
 * the second stack transposed so that mode 2 is the output and mode 3 the value mode), both [n_H, d, d], from
 * WQ, WK, WV [d, d] (heads = column blocks of width d / n_H) and WO [d, d] (head i = rows i d_H ..).
 *
 * tucker_hosvd_init: for one tensor W [n_H, d, d] and ranks (r1, r2, r3), 1 <= r1 <= n_H <= 64, r2, r3 <= d <= 8192:
 *   U_j [n_j, r_j]   the r_j leading left singular vectors of the mode-j unfolding (orthonormal columns, each with
 *                    its largest component positive), from the eigenvectors of the Gram matrix Mat_j Mat_j^T
 *   C [r1, r2, r3]   the core W x_1 U1^T x_2 U2^T x_3 U3^T
 *   spectra          optional [n_H + 2 d]: all singular values of the mode-1, mode-2 and mode-3 unfoldings, each
 *                    block descending (divide by the first entry of a block for the normalised spectrum)
 * so that W ~ C x_1 U1 x_2 U2 x_3 U3 with squared error <= the sum of the squared truncated singular values.
 * Call it once for the pre-softmax tensor (-> C, U1, U2, U3) and once for the post-softmax tensor (-> Ct, Ut1,
 * Ut2, Ut3).  The two d-sized Gram matrices run on the tensor cores when d is a multiple of 64 (bf16 high / low
 * split, fp32 accumulation, about 2^-16 relative), else on fp32 FMA kernels; eigenvectors by one-sided Jacobi
 * sweeps in fp32.  Singular values below about 1e-3 of the largest are at the noise level of that arithmetic.
 * workspace: >= tucker_hosvd_workspace_bytes(d_model, n_H, r2, r3) bytes, 256-byte aligned.
 * Returns TA_OK, TA_ERR_INVALID_ARG, TA_ERR_WORKSPACE_TOO_SMALL, TA_ERR_UNSUPPORTED_SHAPE or TA_ERR_CUDA.
 */
TA_API size_t tucker_hosvd_workspace_bytes(int32_t d_model, int32_t n_H, int32_t r2, int32_t r3);
TA_API int tucker_hosvd_init(int32_t d_model, int32_t n_H, int32_t r1, int32_t r2, int32_t r3, const float* W,
                      float* C, float* U1, float* U2, float* U3, float* spectra,
                      void* workspace, size_t workspace_bytes, void* cuda_stream);
TA_API int tucker_mha_weight_tensors(int32_t d_model, int32_t n_H, const float* WQ, const float* WK,
                              const float* WV, const float* WO, float* W, float* Wt, void* cuda_stream);

/* Human-readable name of a status code (static storage). */
TA_API const char* tucker_attn_status_string(int status);

/*
 * Device error word.  Kernels never trap: a bounded wait that ran out, an out-of-range cache length or (in
 * the checking build) an index that failed its bounds check sets a bit in a per-device word and the kernel
 * carries on without the offending access, or returns.  This call
 * synchronises `cuda_stream`, reads and clears the word of the current device and returns
 * it (0 = clean; otherwise a bit set of TA_DEVERR_*), or a negative status on CUDA errors.
 */
enum {
  TA_DEVERR_WAIT_TIMEOUT = 1,   /* an mbarrier / flag wait hit its iteration limit */
  TA_DEVERR_BAD_CACHE_LEN = 2,  /* cache_len[b] outside [0, Lmax) */
  TA_DEVERR_BAD_INDEX = 4       /* a bounds check failed (only in the -DTA_BOUNDS_CHECK build, see tucker_attn_bounds_checked) */
};
TA_API int tucker_attn_last_device_error(void* cuda_stream);

/*
 * The same read, folded into a status code for callers that only want to know whether the work queued so
 * far went through (no counterpart in the paper).  Synchronises `cuda_stream`, reads and clears the device
 * error word and returns TA_OK when it was clean, else TA_ERR_DEVICE_TIMEOUT (a bounded wait gave up: results
 * of the calls since the last read are invalid), TA_ERR_INVALID_ARG (a cache_len entry was out of range and
 * was clamped) or TA_ERR_CUDA (the read itself failed, or a bounds check of the checking build fired), in
 * that order of precedence.
 */
TA_API int tucker_attn_sync_status(void* cuda_stream);

/*
 * 1 when this library was compiled with -DTA_BOUNDS_CHECK, 0 otherwise.  In that build the kernels of the
 * tensor-core paths and of the decode step compare every global index they form for a store (outputs, caches,
 * workspace regions) and for a load from the workspace with the extent of the tensor addressed, set
 * TA_DEVERR_BAD_INDEX and skip the access on a failure; nothing traps.  TMA transfers are bounded by their
 * tensor maps in either build.  The normal build carries no such checks and never sets that bit.
 */
TA_API int tucker_attn_bounds_checked(void);

/*
 * Self-test of the bounded waits (no counterpart in the paper).  Launches a one-block kernel
 * in which one thread waits on a barrier that nothing ever signals, with a wait budget of
 * about `budget_us` microseconds (1 .. 100000), and a second thread waits on another such
 * barrier with the library's normal budget.  The first wait must give up and set
 * TA_DEVERR_WAIT_TIMEOUT in the device error word; the second must return at once through
 * the block's abort flag.  `out` is caller-owned device memory for three int32: what the
 * two waits returned (0 = gave up) and the second wait's duration in units of 1024 cycles.
 * Asynchronous on `cuda_stream`; the context stays usable.  Returns TA_OK,
 * TA_ERR_INVALID_ARG or TA_ERR_CUDA.
 */
TA_API int tucker_attn_selftest_wait_timeout(int32_t budget_us, int32_t* out, void* cuda_stream);

/* Which path the last tucker_attn_fwd / tucker_attn_decode call on this thread took:
 * 0 = none yet, 1 = generic FMA kernels, 2 = tensor-core kernels.  Number of kernels that
 * call launched. */
TA_API int tucker_attn_last_path(void);
TA_API int tucker_attn_last_launch_count(void);

/*
 * Profiling hook (no counterpart in the paper; measurement plumbing).  Registers two
 * caller-owned cudaEvent_t handles (created with timing enabled) for the calling thread.
 * While registered, every tucker_attn_fwd / tucker_attn_decode call records `ev_start`
 * immediately before and `ev_stop` immediately after its dominant kernel (the attention
 * kernel: scores + online softmax + PV) on the call's stream, so that the caller can read
 * that kernel's duration with cudaEventElapsedTime after synchronising.  Pass NULL, NULL to
 * unregister.  Returns TA_OK, or TA_ERR_INVALID_ARG if exactly one handle is NULL.
 */
TA_API int tucker_attn_set_profile_events(void* ev_start, void* ev_stop);

/*
 * Measurement probe (no counterpart in the paper's experiments; it prices the kernel that Sec. 3.3 leaves to
 * future work, scores formed from the factorised core as S_h = sum_a U1[h, a] (Qt C_a K^T)).  Runs ONLY the
 * step that form would add to the softmax warps -- mixing r1 plane tiles into the score tiles of a head pair,
 * r1 multiply-adds per score and head -- for `tiles` [128 x 128] tiles per block on `n_blocks` blocks of 256
 * threads (one per SM is the attention kernel's occupancy).  u1 [2, r1] fp32 mixing weights; cycles
 * [n_blocks] receives each block's clock64 count for the loop; sink [n_blocks * 256] receives checksums.
 * All device memory, caller-owned.  Returns TA_OK, TA_ERR_INVALID_ARG (r1 > 16, null pointers) or TA_ERR_CUDA.
 */
TA_API int tucker_probe_plane_mix(int32_t tiles, int32_t r1, int32_t n_blocks, const float* u1, long long* cycles,
                           float* sink, void* cuda_stream);

/*
 * Measurement probe (no counterpart in the paper): cycles per tcgen05.mma of shape 128 x N x 16 (bf16 in, fp32
 * accumulate) when one thread issues `iters` x 8 of them back to back, by operand source: mode 0 = A and B in
 * shared memory, K-major; 1 = A in TMEM; 2 = B MN-major in shared memory (a tile used where it lies, as the value
 * tiles and the in-place factor matrices are).  N in {64, 128, 256}.  cycles [n_blocks] (device) receives each
 * block's clock64 count for the whole sequence including the final commit.  Decides, with numbers, which operand
 * layouts the kernels should prefer.  Returns TA_OK, TA_ERR_INVALID_ARG or TA_ERR_CUDA.
 */
TA_API int tucker_probe_mma_rate(int32_t mode, int32_t N, int32_t iters, int32_t n_blocks, long long* cycles,
                          void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* TUCKER_ATTN_H_ */
