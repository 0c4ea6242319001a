// C ABI of the Mixture-of-Attentions drafter hot path (see include/moa.h for the contract).
// Host-side validation and launch sequencing only; every step of the path runs in the kernels.
#include "../../include/moa.h"

#include <stdio.h>
#include <string.h>
#include <mutex>
#include <new>

#include <nvtx3/nvToolsExt.h>

#include "moa_attn.cuh"
#include "moa_attn_tc.cuh"
#include "moa_basic.cuh"
#include "moa_codec.cuh"
#include "moa_phases.cuh"
#include "moa_tree.cuh"
#include "moa_verify.cuh"
#include "moa_wstream.cuh"

using namespace moa;

// One NVTX range per compute call of the C ABI (a profiler's timeline then shows the calls by name; without a
// tool attached a range costs a function-pointer test).
struct NvtxRange {
  explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
};
#define MOA_RANGE() NvtxRange nvtx_range__(__func__)

static thread_local char g_cuda_err[256] = "";
static thread_local long long g_launches = 0;

enum { PROF_MAX = 512, WMAP_MAX = 64, PREFILL_ROWS = 256, TC_MIN_KEYS = 2048, RN_ROWS_PER_CTA_FROM = 64 };

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct WeightMap {
  const void* ptr;
  int n, k;
  CUtensorMap tm;
};

struct moa_ctx {
  moa_config c;
  moa_weights w;
  int sm_count;
  size_t elt;          // bytes per T
  TreeLayout tl;
  // tensor-core path (bf16 only)
  EncodeTiledFn encode;
  WeightMap wmap[WMAP_MAX];
  int n_wmap;
  int n_wmap_base;     // maps of the drafter's own matrices; those of the Target-Layer-Inference layers follow
  // Target Layer Inference (Section 3.2): the last N decoder layers of the LLM, off when tli.n_layers == 0
  moa_tli_config tli;
  moa_tli_layer tli_w[MOA_MAX_TLI];
  moa_tli_caches tli_c;
  bool fast;           // weight-streaming tcgen05 GEMMs usable
  bool coop;           // cooperative launches available: the dense LSA pass can run as one persistent kernel
  int smem_optin;      // largest dynamic shared memory a CTA may ask for
  int last_n_ops;      // phase kinds of the last fused launch (for moa_profile_phases)
  int last_kinds[PM_MAX_OPS];
  // measurement hooks: event pairs around the LM-head launches
  bool prof_on;
  int prof_n;
  cudaEvent_t prof_ev[2 * PROF_MAX];
  bool prof_made;
};

// ---------------------------------------------------------------------------------------------
// workspace carving (same arithmetic in moa_state_bytes and in the calls)
// ---------------------------------------------------------------------------------------------
struct Workspace {
  size_t xres, xn, part, narrow, obuf, logits, pmax, psum, cval, cid, mrg_ms, mrg_val, mrg_id, kvf, kvn, att_o, att_ml, q32, trace, total;
  int rows_cap, draft_rows, chunk_tok, part_rows, wide;
  long long att_units;   // (row, head, part) triples the split-attention partial buffers hold
};

static inline int imax(int a, int b) { return a > b ? a : b; }
static inline int imin(int a, int b) { return a < b ? a : b; }

static Workspace plan_workspace(const moa_config& c, const moa_tli_config& t, size_t elt, int chunk_tok) {
  Workspace p;
  p.chunk_tok = chunk_tok;
  p.draft_rows = c.max_batch * c.tree_topk;
  p.rows_cap = imax(p.draft_rows, chunk_tok * c.n_stack);
  p.part_rows = imax(640, p.rows_cap);      // room for several K-split planes when there are few rows
  const int dmax = imax(c.d_model, c.d_stack);
  const int qkv_lsa = (c.lsa_hq + 2 * c.lsa_hkv) * c.head_dim;
  const int qkv_sa = (c.sa_hq + 2 * c.sa_hkv) * c.head_dim;
  const int q_ca = imax(c.ca_hq * c.head_dim, 2 * c.ca_hkv * c.head_dim);
  const bool tli = t.n_layers > 0;
  const int qkv_tli = tli ? (t.hq + 2 * t.hkv) * c.head_dim : 0;
  const int fmax = imax(imax(c.lsa_mlp, tli ? t.mlp : 0), imax(c.sa_mlp, c.ca_mlp));
  p.wide = imax(imax(imax(qkv_lsa, imax(qkv_sa, qkv_tli)), imax(q_ca, 2 * fmax)), dmax);
  const int narrow = imax(imax(qkv_lsa, imax(qkv_sa, qkv_tli)), imax(q_ca, fmax));
  const int omax = imax(imax(c.lsa_hq, tli ? t.hq : 0), imax(c.sa_hq, c.ca_hq)) * c.head_dim;
  const size_t n_sub = (size_t)4 * ((c.vocab + WS_BM - 1) / WS_BM);
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o += (bytes + 255) / 256 * 256; return at; };
  p.xres = take((size_t)p.rows_cap * dmax * sizeof(float));      // residual stream, fp32
  const size_t xpad = 256;                                       // an X buffer's low-order rows start up to 256 rows in
  p.xn = take(((size_t)p.rows_cap + xpad) * dmax * elt);         // normalised GEMM operand, T
  p.part = take((size_t)p.part_rows * p.wide * sizeof(float));   // GEMM outputs: K-split partial planes, fp32
  p.narrow = take(((size_t)p.rows_cap + xpad) * narrow * elt);   // q|k|v or silu(gate)*up, T
  p.obuf = take(((size_t)p.rows_cap + xpad) * omax * elt);       // attention output, T
  p.logits = take(elt == 4 ? (size_t)p.draft_rows * c.vocab * sizeof(float) : 256);   // fp32 path only
  p.pmax = take(n_sub * p.draft_rows * sizeof(float));           // LM-head partials per 32-row vocabulary slice
  p.psum = take(n_sub * p.draft_rows * sizeof(float));
  p.cval = take(n_sub * p.draft_rows * c.tree_topk * sizeof(float));
  p.cid = take(n_sub * p.draft_rows * c.tree_topk * sizeof(int));
  p.mrg_ms = take((size_t)p.draft_rows * MERGE_MAXCHUNKS * 2 * sizeof(float));     // LM-head merge, level-1 results
  p.mrg_val = take((size_t)p.draft_rows * MERGE_MAXCHUNKS * MERGE_MAXB * sizeof(float));
  p.mrg_id = take((size_t)p.draft_rows * MERGE_MAXCHUNKS * MERGE_MAXB * sizeof(int));
  p.kvf = take((size_t)chunk_tok * c.d_stack * sizeof(float));   // LSA output rows, fp32
  p.kvn = take(((size_t)chunk_tok + xpad) * c.d_stack * elt);    // their normalised copy, T
  const int gmax = imax(imax(c.sa_hq / c.sa_hkv, c.ca_hq / c.ca_hkv), tli ? t.hq / t.hkv : 0);
  const int hqmax = imax(imax(c.sa_hq, c.ca_hq), tli ? t.hq : 0);
  p.att_units = (long long)c.tree_topk * gmax * 2 * 160 + 2ll * p.draft_rows * hqmax;
  if (p.att_units < 10ll * p.draft_rows * hqmax) p.att_units = 10ll * p.draft_rows * hqmax;   // up to ten parts per (row, head)
  p.att_o = take(elt == 2 ? (size_t)p.att_units * c.head_dim * sizeof(float) : 256);   // split-KV partial outputs
  p.att_ml = take(elt == 2 ? (size_t)p.att_units * 2 * sizeof(float) : 256);           // their (max, sum)
  // draft-step queries in fp32; the whole-sequence drafter pass works in chunks of up to PREFILL_ROWS rows
  p.q32 = take(elt == 2 ? (size_t)imax(p.draft_rows, imin(p.rows_cap, PREFILL_ROWS)) * hqmax * c.head_dim * sizeof(float) : 256);
  p.trace = take((2 * PM_MAX_OPS + 2) * sizeof(unsigned long long));   // phase timestamps of the last fused launch
  p.total = o;
  return p;
}

// Largest token chunk whose plan fits in ws_bytes (plan size is monotone in the chunk); 0 if none.
static int chunk_from_bytes(const moa_config& c, const moa_tli_config& t, size_t elt, size_t ws_bytes) {
  if (plan_workspace(c, t, elt, 1).total > ws_bytes) return 0;
  int lo = 1;
  while (lo < (1 << 20) && plan_workspace(c, t, elt, lo * 2).total <= ws_bytes) lo *= 2;
  int hi = lo * 2;
  while (lo + 1 < hi) {
    const int mid = lo + (hi - lo) / 2;
    if (plan_workspace(c, t, elt, mid).total <= ws_bytes) lo = mid; else hi = mid;
  }
  return lo;
}

// ---------------------------------------------------------------------------------------------
// helpers
// ---------------------------------------------------------------------------------------------
#define MOA_CHECK_LAUNCH()                                                                               \
  do {                                                                                                   \
    ++g_launches;                                                                                        \
    cudaError_t e__ = cudaGetLastError();                                                                \
    if (e__ != cudaSuccess) {                                                                            \
      snprintf(g_cuda_err, sizeof(g_cuda_err), "%s:%d %s", __FILE__, __LINE__, cudaGetErrorString(e__)); \
      return MOA_ERR_CUDA;                                                                               \
    }                                                                                                    \
  } while (0)
#define MOA_TRY(x)                      \
  do {                                  \
    moa_status s__ = (x);               \
    if (s__ != MOA_OK) return s__;      \
  } while (0)

static inline bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }
static inline unsigned blocks_for(size_t total, int threads) { return (unsigned)((total + threads - 1) / threads); }

// Launch with programmatic dependent launch allowed: the kernel may start while its predecessor in the stream is
// still running and does its independent set-up (and, for the weight-streaming GEMM, its first weight loads)
// until its griddepcontrol.wait; see pdl_trigger / pdl_wait in moa_common.cuh.
template <typename... KArgs, typename... Args>
static void launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);     // errors surface through cudaGetLastError()
}

// 2-D bf16 tensor map: global [rows, k] row-major, box 64 x box_rows, 128-byte swizzle, zero fill outside.
static bool encode_map(const moa_ctx* ctx, CUtensorMap* tm, const void* ptr, int rows, int k, int box_rows) {
  cuuint64_t dims[2] = {(cuuint64_t)k, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)k * 2};
  cuuint32_t box[2] = {(cuuint32_t)WS_BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = ctx->encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) snprintf(g_cuda_err, sizeof(g_cuda_err), "cuTensorMapEncodeTiled failed (%d)", (int)r);
  return r == CUDA_SUCCESS;
}

static const WeightMap* find_wmap(const moa_ctx* ctx, const void* w) {
  for (int i = 0; i < ctx->n_wmap; ++i)
    if (ctx->wmap[i].ptr == w) return &ctx->wmap[i];
  return nullptr;
}

// K-split count: best use of the SMs' waves, fewest splits among near-equal choices.
static int pick_splits(int tiles, int kb_total, int R, int part_rows, int sms) {
  const int smax = imax(1, imin(imin(8, kb_total), part_rows / imax(R, 1)));
  int best = 1;
  double best_eff = 0.0;
  for (int s = 1; s <= smax; ++s) {
    const int units = tiles * s;
    const int waves = (units + sms - 1) / sms;
    const double eff = (double)units / ((double)waves * sms);
    if (eff > best_eff + 0.02) { best_eff = eff; best = s; }
  }
  return best;
}

struct LinOut {          // where a linear layer left its result: `splits` fp32 planes of [R, ld]
  const float* part;
  int splits;
  size_t plane;
  int ld;
};

template <int NPAD, bool XS2 = false>
static moa_status launch_ws(cudaStream_t s, const WsParams& P, int grid) {
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(wstream_gemm_kernel<NPAD, XS2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         ws_smem_bytes(NPAD, XS2));
    if (e != cudaSuccess) {
      snprintf(g_cuda_err, sizeof(g_cuda_err), "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
      return MOA_ERR_CUDA;
    }
    attr_set = true;
  }
  launch_pdl(wstream_gemm_kernel<NPAD, XS2>, dim3(grid), dim3(WS_THREADS), ws_smem_bytes(NPAD, XS2), s, P);
  MOA_CHECK_LAUNCH();
  return MOA_OK;
}

static moa_status launch_ws_any(cudaStream_t s, const WsParams& P, int npad, int grid, bool xs2 = false) {
  if (xs2) {                       // two-term activations of more than 128 rows
    switch (npad) {
      case 160: return launch_ws<160, true>(s, P, grid);
      case 192: return launch_ws<192, true>(s, P, grid);
      case 224: return launch_ws<224, true>(s, P, grid);
      default: return launch_ws<256, true>(s, P, grid);
    }
  }
  switch (npad) {
    case 16: return launch_ws<16>(s, P, grid);
    case 32: return launch_ws<32>(s, P, grid);
    case 64: return launch_ws<64>(s, P, grid);
    case 128: return launch_ws<128>(s, P, grid);
    case 160: return launch_ws<160>(s, P, grid);
    case 192: return launch_ws<192>(s, P, grid);
    case 224: return launch_ws<224>(s, P, grid);
    default: return launch_ws<256>(s, P, grid);
  }
}

// MMA N (and activation-tile rows) for R rows: a power of two up to 128, then the next multiple of 32 -- a
// smaller activation tile leaves room for more stages of the weight ring (R = 160: six stages instead of four).
static inline int npad_for(int R) { return R <= 16 ? 16 : R <= 32 ? 32 : R <= 64 ? 64 : R <= 128 ? 128 : imin(256, (R + 31) / 32 * 32); }

// Up to 128 rows, bf16 activations travel between kernels as two terms (hi + lo): the low-order rows start at this
// row offset of every X buffer (0: single term). Producers and the GEMM that consumes them derive it from the same R.
// (129 to 256 rows: the low-order rows start at row 256 and the GEMM multiplies the two terms one after the other
// into the same accumulator; more rows: a single term.)
constexpr int LO_ROW_WIDE = 256;
static inline int lo_rows_of(size_t elt, int R) {
  if (elt != 2 || R <= 0 || R > 256) return 0;
  return R <= 128 ? npad_for(R) : LO_ROW_WIDE;
}

// Launch shape of rope_store_kernel for R rows of n_heads heads: eight threads per head; with few rows blocks of 64
// threads (8 heads each) spread a row over several CTAs, with many rows blocks of 256 threads (32 heads each).
static inline void rope_shape(const moa_ctx* ctx, int R, int n_heads, dim3* grid, dim3* block) {
  (void)ctx;
  const int per_block = R <= 32 ? 8 : 32;
  *grid = dim3(R, (n_heads + per_block - 1) / per_block);
  *block = dim3(per_block * 8);
}

static bool fast_shape(const moa_ctx* ctx, int K, int nseg, const void* const* W) {
  if (!ctx->fast || K % WS_BK != 0) return false;
  for (int i = 0; i < nseg; ++i)
    if (!find_wmap(ctx, W[i])) return false;
  return true;
}

// Linear layer(s) sharing one input: Y[:, col_i : col_i + N_i] = X W_i^T for up to three weight matrices.
// Result: fp32 partial planes in the workspace's `part` buffer (see LinOut).
template <typename T>
static moa_status linear(moa_ctx* ctx, cudaStream_t s, const T* X, int R, int K, int nseg, const void* const* W,
                         const int* N, char* ws, const Workspace& p, LinOut* out, void* status_word) {
  float* part = (float*)(ws + p.part);
  int ntot = 0;
  for (int i = 0; i < nseg; ++i) ntot += N[i];
  out->part = part;
  out->ld = ntot;
  out->plane = (size_t)R * ntot;
  out->splits = 1;
  if (R <= 0) return MOA_OK;
  if (sizeof(T) == 2 && fast_shape(ctx, K, nseg, W)) {
    WsParams P;
    memset(&P, 0, sizeof(P));
    P.n_seg = nseg;
    int tiles = 0, col = 0;
    for (int i = 0; i < nseg; ++i) {
      P.tmW[i] = find_wmap(ctx, W[i])->tm;
      P.seg_n[i] = N[i];
      P.seg_tile0[i] = tiles;
      P.seg_col[i] = col;
      tiles += (N[i] + WS_BM - 1) / WS_BM;
      col += N[i];
    }
    P.tiles_total = tiles;
    P.kb_total = K / WS_BK;
    P.mode = 0;
    P.ldo = ntot;
    P.plane = out->plane;
    P.status = (int*)status_word;
    const int nblk = (R + 255) / 256;
    const int lo = lo_rows_of(sizeof(T), R);
    const bool wide = lo == LO_ROW_WIDE && R > 128;      // two activation tiles per stage instead of one tile of both terms
    P.xsplit = (lo > 0 && !wide) ? 1 : 0;
    P.lo_row = lo;
    P.splits = pick_splits(tiles * nblk, P.kb_total, R, p.part_rows, ctx->sm_count);
    out->splits = P.splits;
    for (int r0 = 0; r0 < R; r0 += 256) {
      const int rows = imin(256, R - r0);
      const int npad = (lo > 0 && !wide) ? 2 * lo : npad_for(rows);
      if (!encode_map(ctx, &P.tmX, (const bf16*)X + (size_t)r0 * K, lo > 0 ? lo + rows : rows, K, npad)) return MOA_ERR_CUDA;
      P.R = rows;
      P.out = part + (size_t)r0 * ntot;
      const int units = tiles * P.splits;
      MOA_TRY(launch_ws_any(s, P, npad, imin(units, ctx->sm_count), wide));
    }
    return MOA_OK;
  }
  int col = 0;
  for (int i = 0; i < nseg; ++i) {
    dim3 grid((N[i] + 63) / 64, (R + 63) / 64);
    launch_pdl(gemm_fma_kernel<T>, dim3(grid), dim3(256), 0, s, X, (const T*)W[i], R, N[i], K, nullptr, 0, part + col, ntot);
    MOA_CHECK_LAUNCH();
    col += N[i];
  }
  return MOA_OK;
}

template <int DH, bool QSPLIT, bool PSPLIT>
static moa_status launch_attn_split(cudaStream_t s, const AttnParams& P, int nseq, int nwarps) {
  static bool attr_set = false;
  const int smem = (QSPLIT ? 2 : 1) * nwarps * 16 * DH * 2 + 4 * AT_KB * DH * 2;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(attn_split_kernel<DH, QSPLIT, PSPLIT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (QSPLIT ? 2 : 1) * 8 * 16 * DH * 2 + 4 * AT_KB * DH * 2);
    if (e != cudaSuccess) {
      snprintf(g_cuda_err, sizeof(g_cuda_err), "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
      return MOA_ERR_CUDA;
    }
    attr_set = true;
  }
  dim3 grid(P.n_parts, P.hkv * P.q_tiles, nseq);
  launch_pdl(attn_split_kernel<DH, QSPLIT, PSPLIT>, dim3(grid), dim3(nwarps * 32), smem, s, P);
  MOA_CHECK_LAUNCH();
  if (P.n_parts > 1) {
    const int n_rh = nseq * P.rows_per_seq * P.hq;
    const int share = P.n_parts >= CB_SHARE_FROM ? 1 : 0;
    launch_pdl(attn_combine_kernel<DH>, dim3(share ? n_rh : (n_rh + CB_WARPS - 1) / CB_WARPS), dim3(CB_WARPS * 32), 0, s, P.part_o,
               P.part_ml, P.n_parts, n_rh, share, P.out, P.out_lo, P.hq);
    MOA_CHECK_LAUNCH();
  }
  return MOA_OK;
}

// softmax(q K^T / sqrt(dh)) V for R = nseq * rows_per_seq query rows. Segment A: a cache (or the LSA rows
// themselves) with max_len positions at most on the host's count; segment B: tree slots masked per row.
template <typename T>
static moa_status attention(moa_ctx* ctx, cudaStream_t s, char* ws, const Workspace& p, int dh, const T* q,
                            const float* q32, int q_splits, size_t q_plane, int q_ld, int R, int hq, int hkv, const T* kA, const T* vA, int capA, int posA_ld, const int* lenA,
                            int nA_fixed, int max_len, const T* kB, const T* vB, int capB, const int* slotsB,
                            int slots_ld, int nB, int n_slots, int rows_per_seq, T* out,
                            RowLimit lim = RowLimit{nullptr, 0, 0}, void* status_word = nullptr, bool cache_settled = false) {
  // cache_settled: segment A and its lengths were complete before the launch chain of this call began (a draft step: the
  // caches are written by the append calls, which end with an ordinary launch), so a kernel may read them before it
  // waits on its predecessor in the chain
  if (R <= 0) return MOA_OK;
  if (sizeof(T) == 2) {
    AttnParams P;
    memset(&P, 0, sizeof(P));
    P.lim = lim;
    P.status = (int*)status_word;
    const int nseq = R / rows_per_seq;
    P.q = (const bf16*)q; P.q32 = q32; P.q_splits = q_splits; P.q_plane = q_plane; P.q_ld = q_ld;
    P.hq = hq; P.hkv = hkv; P.group = hq / hkv;
    P.rows_per_seq = rows_per_seq;
    P.kA = (const bf16*)kA; P.vA = (const bf16*)vA; P.capA = capA; P.posA_ld = posA_ld;
    P.lenA = lenA; P.nA_fixed = nA_fixed;
    P.kB = (const bf16*)kB; P.vB = (const bf16*)vB; P.capB = capB;
    P.slotsB = slotsB; P.slots_ld = slots_ld; P.nB = nB; P.n_slots = n_slots;
    const int Qn = rows_per_seq * P.group;
    const int nwarps = imin(8, (Qn + 15) / 16);
    P.q_tiles = (Qn + nwarps * 16 - 1) / (nwarps * 16);
    const int has_tree = (kB != nullptr && nB > 0) ? 1 : 0;
    P.part_o = (float*)(ws + p.att_o);
    P.part_ml = (float*)(ws + p.att_ml);
    P.out = (bf16*)out;
    P.out_lo = lo_rows_of(sizeof(T), R);
    P.scale_log2 = 1.4426950408889634f / sqrtf((float)dh);
    // Long dense caches (fp32 queries, head size 128, no per-row limits): the tcgen05 kernel, one CTA per (kv head,
    // sequence, key range) and one more per sequence for the tree segment, if any; the parts are merged by the same
    // kernel as the split-KV parts.
    if (q32 && dh == 128 && !lim.active() && ctx->fast && Qn <= 128 && posA_ld == hkv * dh && kA != nullptr &&
        max_len >= TC_MIN_KEYS && n_slots <= 256) {
      const int blocks = (max_len + TC_KB - 1) / TC_KB;
      int n_split = imax(1, imin(blocks, ctx->sm_count / imax(1, nseq * hkv)));
      const long long per_part = (long long)R * hq;
      while (n_split > 1 && per_part * (n_split + has_tree) > p.att_units) --n_split;
      if (per_part * (n_split + has_tree) > p.att_units) return MOA_ERR_WORKSPACE;
      AttnTcParams TP;
      memset(&TP, 0, sizeof(TP));
      P.n_split = n_split;
      P.n_parts = n_split + has_tree;
      TP.a = P;
      TP.early_cache = cache_settled ? 1 : 0;
      const int cache_rows = ctx->c.max_batch * capA;
      if (!encode_map(ctx, &TP.tmK, kA, cache_rows, hkv * dh, TC_KB) || !encode_map(ctx, &TP.tmV, vA, cache_rows, hkv * dh, TC_KB))
        return MOA_ERR_CUDA;
      if (has_tree && (!encode_map(ctx, &TP.tmKB, kB, ctx->c.max_batch * capB, hkv * dh, TC_KB) ||
                       !encode_map(ctx, &TP.tmVB, vB, ctx->c.max_batch * capB, hkv * dh, TC_KB)))
        return MOA_ERR_CUDA;
      static bool tc_attr = false;
      if (!tc_attr) {
        cudaError_t e = cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_BYTES);
        if (e != cudaSuccess) {
          snprintf(g_cuda_err, sizeof(g_cuda_err), "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
          return MOA_ERR_CUDA;
        }
        tc_attr = true;
      }
      const dim3 tgrid(hkv, nseq, n_split + has_tree);
      launch_pdl(attn_tc_kernel, tgrid, dim3(TC_THREADS), TC_SMEM_BYTES, s, TP);
      MOA_CHECK_LAUNCH();
      if (P.n_parts > 1) {
        const int n_rh = nseq * rows_per_seq * hq;
        const int share = P.n_parts >= CB_SHARE_FROM ? 1 : 0;
        launch_pdl(attn_combine_kernel<128>, dim3(share ? n_rh : (n_rh + CB_WARPS - 1) / CB_WARPS), dim3(CB_WARPS * 32), 0, s, P.part_o,
                   P.part_ml, P.n_parts, n_rh, share, P.out, P.out_lo, P.hq);
        MOA_CHECK_LAUNCH();
      }
      return MOA_OK;
    }
    const int blocks = imax(1, (max_len + AT_KB - 1) / AT_KB);
    // cache parts plus the tree part fill one wave of two CTAs per SM: a few CTAs more would run alone afterwards
    int n_split = imax(1, imin(blocks, (2 * ctx->sm_count) / imax(1, nseq * hkv * P.q_tiles) - has_tree));
    const long long per_part = (long long)R * hq;
    while (n_split > 1 && per_part * (n_split + has_tree) > p.att_units) --n_split;
    if (per_part * (n_split + has_tree) > p.att_units && n_split + has_tree > 1) return MOA_ERR_WORKSPACE;
    P.n_split = n_split;
    P.n_parts = n_split + has_tree;
    // fp32 queries and the probabilities are split into two bf16 terms each
    if (q32)
      return dh == 128 ? launch_attn_split<128, true, true>(s, P, nseq, nwarps) : launch_attn_split<64, true, true>(s, P, nseq, nwarps);
    return dh == 128 ? launch_attn_split<128, false, false>(s, P, nseq, nwarps) : launch_attn_split<64, false, false>(s, P, nseq, nwarps);
  }
  dim3 grid(R, hq);
  if (dh == 128)
    launch_pdl(attn_rows_kernel<T, 128>, dim3(grid), dim3(128), 0, s, q, q_ld, hq, hkv, kA, vA, capA, posA_ld, lenA, nA_fixed, kB, vB, capB,
                                                  slotsB, slots_ld, nB, rows_per_seq, lim, out);
  else
    launch_pdl(attn_rows_kernel<T, 64>, dim3(grid), dim3(128), 0, s, q, q_ld, hq, hkv, kA, vA, capA, posA_ld, lenA, nA_fixed, kB, vB, capB,
                                                 slotsB, slots_ld, nB, rows_per_seq, lim, out);
  MOA_CHECK_LAUNCH();
  return MOA_OK;
}

// xres += previous linear's result; xn = RMSNorm(xres; gain) (skipped when gain == nullptr)
template <typename T>
static moa_status residual_norm(cudaStream_t s, const moa_ctx* ctx, char* ws, const Workspace& p, int R, int K,
                                const LinOut* lo, const void* gain, void* hidden_out) {
  if (R <= 0) return MOA_OK;
  // few rows: a cluster of 8 CTAs per row (a row alone cannot fill the machine); many rows: one CTA per row
  if (R < RN_ROWS_PER_CTA_FROM && K % (RN_CLUSTER * 8) == 0 && K / RN_CLUSTER <= 256 * 8 * (RN_MAX_PER_THREAD / 4)) {
    launch_pdl(residual_norm_cluster_kernel<T>, dim3(dim3(RN_CLUSTER, R)), dim3(256), 0, s, 
        (float*)(ws + p.xres), lo ? lo->part : nullptr, lo ? lo->splits : 0, lo ? lo->plane : 0, K, (const T*)gain,
        ctx->c.rms_eps, (T*)(ws + p.xn), (T*)hidden_out, lo_rows_of(sizeof(T), R));
    MOA_CHECK_LAUNCH();
    return MOA_OK;
  }
  launch_pdl(residual_norm_kernel<T>, dim3(R), dim3(256), 0, s, (float*)(ws + p.xres), lo ? lo->part : nullptr, lo ? lo->splits : 0,
                                            lo ? lo->plane : 0, K, (const T*)gain, ctx->c.rms_eps, (T*)(ws + p.xn),
                                            (T*)hidden_out, lo_rows_of(sizeof(T), R));
  MOA_CHECK_LAUNCH();
  return MOA_OK;
}

// MLP, given xn = RMSNorm(xres) already in place: leaves the down-projection in `lo`
// (the caller folds it into the residual stream together with the next normalisation).
template <typename T>
static moa_status mlp_block(cudaStream_t s, moa_ctx* ctx, const Workspace& p, char* ws, int R, int K, int F,
                            const void* wgate, const void* wup, const void* wdown, LinOut* lo, void* status_word) {
  const T* xn = (const T*)(ws + p.xn);
  T* h = (T*)(ws + p.narrow);
  const void* W2[2] = {wgate, wup};
  const int N2[2] = {F, F};
  MOA_TRY(linear<T>(ctx, s, xn, R, K, 2, W2, N2, ws, p, lo, status_word));
  const size_t total = (size_t)R * F;
  if (total) {
    launch_pdl(silu_mul_split_kernel<T>, dim3(blocks_for(total / 8, 256)), dim3(256), 0, s, lo->part, lo->splits, lo->plane, F, h, total,
               lo_rows_of(sizeof(T), R));
    MOA_CHECK_LAUNCH();
  }
  const void* W1[1] = {wdown};
  const int N1[1] = {K};
  return linear<T>(ctx, s, h, R, F, 1, W1, N1, ws, p, lo, status_word);
}

// ---------------------------------------------------------------------------------------------
// typed implementations
// ---------------------------------------------------------------------------------------------
template <typename T>
static moa_status lsa_forward_t(moa_ctx* ctx, moa_state* st, const void* h_stack, const SeqSplit& split, void* kv_out,
                                char* ws, const Workspace& p, cudaStream_t s) {
  const moa_config& c = ctx->c;
  const moa_weights& w = ctx->w;
  const int S = c.n_stack, D = c.d_stack, dh = c.head_dim;
  const int nq = c.lsa_hq * dh, nkv = c.lsa_hkv * dh, ld = nq + 2 * nkv;
  void* status_word = (char*)st->tree + ctx->tl.status;
  float* xres = (float*)(ws + p.xres);
  T* xn = (T*)(ws + p.xn);
  T* narrow = (T*)(ws + p.narrow);
  T* obuf = (T*)(ws + p.obuf);
  float* kvf = (float*)(ws + p.kvf);
  T* kvn = (T*)(ws + p.kvn);
  const int total = split.off[split.n_seq];
  LinOut lo;
  for (int t0 = 0; t0 < total; t0 += p.chunk_tok) {
    const int nt = (total - t0) < p.chunk_tok ? (total - t0) : p.chunk_tok;
    const int R = nt * S;
    const T* x = (const T*)h_stack + (size_t)t0 * S * D;
    // pre-norm and q, k, v projections of every (token, layer) row: rows of [q | k | v]
    launch_pdl(rmsnorm_rows_kernel<T, T>, dim3(R), dim3(256), 0, s, x, nullptr, 0, (const T*)w.lsa_norm1, D, c.rms_eps, xres, xn,
               lo_rows_of(sizeof(T), R), (int*)status_word);
    MOA_CHECK_LAUNCH();
    const void* W3[3] = {w.lsa_wq, w.lsa_wk, w.lsa_wv};
    const int N3[3] = {nq, nkv, nkv};
    MOA_TRY(linear<T>(ctx, s, xn, R, D, 3, W3, N3, ws, p, &lo, status_word));
    {
      const size_t tot = (size_t)R * ld;
      launch_pdl(sum_cast_kernel<T>, dim3(blocks_for(tot / 8, 256)), dim3(256), 0, s, lo.part, lo.splits, lo.plane, tot, narrow);
      MOA_CHECK_LAUNCH();
    }
    // attention over the S layer rows of the same token (full mask): "sequence" = token, cap = S
    MOA_TRY(attention<T>(ctx, s, ws, p, dh, narrow, nullptr, 1, 0, ld, R, c.lsa_hq, c.lsa_hkv, narrow + nq, narrow + nq + nkv, S, ld,
                         nullptr, S, S, (const T*)nullptr, (const T*)nullptr, 0, nullptr, 0, 0, 0, S, obuf));
    // out-projection + residual, MLP + residual
    const void* W1[1] = {w.lsa_wo};
    const int N1[1] = {D};
    MOA_TRY(linear<T>(ctx, s, obuf, R, nq, 1, W1, N1, ws, p, &lo, status_word));
    MOA_TRY(residual_norm<T>(s, ctx, ws, p, R, D, &lo, w.lsa_norm2, nullptr));
    MOA_TRY(mlp_block<T>(s, ctx, p, ws, R, D, c.lsa_mlp, w.lsa_wgate, w.lsa_wup, w.lsa_wdown, &lo, status_word));
    MOA_TRY(residual_norm<T>(s, ctx, ws, p, R, D, &lo, nullptr, nullptr));
    // mean over layers
    T* kvo = kv_out ? (T*)kv_out + (size_t)t0 * D : nullptr;
    launch_pdl(mean_layers_kernel<T>, dim3(dim3(nt, (D + 255) / 256)), dim3(256), 0, s, xres, S, D, kvf, kvo);
    MOA_CHECK_LAUNCH();
    // cross-attention keys / values of the new positions, appended to the cache
    launch_pdl(rmsnorm_rows_kernel<float, T>, dim3(nt), dim3(256), 0, s, kvf, nullptr, 0, (const T*)w.ca_normkv, D, c.rms_eps, nullptr, kvn,
               lo_rows_of(sizeof(T), nt), (int*)status_word);
    MOA_CHECK_LAUNCH();
    const int ckv = c.ca_hkv * dh;
    const void* W2[2] = {w.ca_wk, w.ca_wv};
    const int N2[2] = {ckv, ckv};
    MOA_TRY(linear<T>(ctx, s, kvn, nt, D, 2, W2, N2, ws, p, &lo, status_word));
    launch_pdl(cache_append_kernel<T>, dim3(nt), dim3(256), 0, s, lo.part, lo.splits, lo.plane, 2 * ckv, 0, ckv, ckv, st->ca_len, c.max_ctx,
                                              split, t0, (T*)st->ca_k, (T*)st->ca_v, (int*)status_word);
    MOA_CHECK_LAUNCH();
  }
  add_len_kernel<<<1, 64, 0, s>>>(st->ca_len, split, c.max_ctx);
  MOA_CHECK_LAUNCH();
  return MOA_OK;
}

template <typename T>
static moa_status sa_append_t(moa_ctx* ctx, moa_state* st, const int* tok, const SeqSplit& split, char* ws,
                              const Workspace& p, cudaStream_t s) {
  const moa_config& c = ctx->c;
  const moa_weights& w = ctx->w;
  const int E = c.d_model, dh = c.head_dim, nkv = c.sa_hkv * dh;
  void* status_word = (char*)st->tree + ctx->tl.status;
  T* xn = (T*)(ws + p.xn);
  const int total = split.off[split.n_seq];
  LinOut lo;
  for (int t0 = 0; t0 < total; t0 += p.rows_cap) {
    const int R = (total - t0) < p.rows_cap ? (total - t0) : p.rows_cap;
    launch_pdl(rmsnorm_rows_kernel<T, T>, dim3(R), dim3(256), 0, s, (const T*)w.embed, tok + t0, c.vocab, (const T*)w.sa_norm1, E,
                                                c.rms_eps, nullptr, xn, lo_rows_of(sizeof(T), R), (int*)status_word);
    MOA_CHECK_LAUNCH();
    const void* W2[2] = {w.sa_wk, w.sa_wv};
    const int N2[2] = {nkv, nkv};
    MOA_TRY(linear<T>(ctx, s, xn, R, E, 2, W2, N2, ws, p, &lo, status_word));
    RopeRows rr;
    memset(&rr, 0, sizeof(rr));
    rr.mode = 1;
    rr.max_ctx = c.max_ctx;
    rr.split = split;
    rr.row0 = t0;
    dim3 rgrid, rblock;
    rope_shape(ctx, R, 2 * c.sa_hkv, &rgrid, &rblock);
    launch_pdl(rope_store_kernel<T>, rgrid, rblock, 0, s, lo.part, lo.splits, lo.plane, 2 * nkv, 0, 0, nkv, 0, c.sa_hkv, dh,
                                           c.sa_rope_theta, st->sa_len, rr, (T*)nullptr, (float*)nullptr, (T*)st->sa_k, (T*)st->sa_v, (int*)status_word);
    MOA_CHECK_LAUNCH();
  }
  add_len_kernel<<<1, 64, 0, s>>>(st->sa_len, split, c.max_ctx);
  MOA_CHECK_LAUNCH();
  return MOA_OK;
}

// LM head + log-softmax + top-B on xn = RMSNorm(o_hat; final_norm)
template <typename T>
static moa_status lm_head_t(moa_ctx* ctx, cudaStream_t s, char* ws, const Workspace& p, int R, int* topk_id,
                            float* topk_logp, void* status_word) {
  const moa_config& c = ctx->c;
  const int E = c.d_model, V = c.vocab, B = c.tree_topk;
  const T* xn = (const T*)(ws + p.xn);
  const void* W1[1] = {ctx->w.lm_head};
  const bool timed = ctx->prof_on && ctx->prof_n < PROF_MAX;
  if (sizeof(T) == 2) {
    if (R > 256 || !fast_shape(ctx, E, 1, W1)) return MOA_ERR_SHAPE;   // validated at moa_create
    if (4 * ((V + WS_BM - 1) / WS_BM) > MERGE_CHUNK * MERGE_MAXCHUNKS) return MOA_ERR_SHAPE;
    WsParams P;
    memset(&P, 0, sizeof(P));
    P.n_seg = 1;
    P.tmW[0] = find_wmap(ctx, ctx->w.lm_head)->tm;
    P.seg_n[0] = V;
    P.tiles_total = (V + WS_BM - 1) / WS_BM;
    P.kb_total = E / WS_BK;
    P.splits = 1;
    P.mode = 1;
    P.R = R;
    P.B = B;
    P.p_max = (float*)(ws + p.pmax);
    P.p_sum = (float*)(ws + p.psum);
    P.c_val = (float*)(ws + p.cval);
    P.c_id = (int*)(ws + p.cid);
    P.status = (int*)status_word;
    const int lo = lo_rows_of(sizeof(T), R);
    const bool wide = lo == LO_ROW_WIDE && R > 128;
    P.xsplit = (lo > 0 && !wide) ? 1 : 0;
    P.lo_row = lo;
    const int npad = (lo > 0 && !wide) ? 2 * lo : npad_for(R);
    if (!encode_map(ctx, &P.tmX, xn, lo > 0 ? lo + R : R, E, npad)) return MOA_ERR_CUDA;
    if (timed) cudaEventRecord(ctx->prof_ev[2 * ctx->prof_n], s);
    MOA_TRY(launch_ws_any(s, P, npad, imin(P.tiles_total, ctx->sm_count), wide));
    if (timed) cudaEventRecord(ctx->prof_ev[2 * ctx->prof_n++ + 1], s);
    MergeScratch sc;
    sc.ms = (float*)(ws + p.mrg_ms);
    sc.val = (float*)(ws + p.mrg_val);
    sc.id = (int*)(ws + p.mrg_id);
    sc.count = (int*)status_word + TREE_STATUS_WORDS;      // per-row arrival counters behind the status words
    const int n_sub = 4 * P.tiles_total;
    launch_pdl(lm_merge_kernel, dim3((n_sub + MERGE_CHUNK - 1) / MERGE_CHUNK, R), dim3(MERGE_THREADS), 0, s, P.p_max, P.p_sum,
               P.c_val, P.c_id, n_sub, R, B, sc, topk_id, topk_logp);
    MOA_CHECK_LAUNCH();
    return MOA_OK;
  }
  float* logits = (float*)(ws + p.logits);
  if (timed) cudaEventRecord(ctx->prof_ev[2 * ctx->prof_n], s);
  {
    dim3 grid((V + 63) / 64, (R + 63) / 64);
    launch_pdl(gemm_fma_kernel<T>, dim3(grid), dim3(256), 0, s, xn, (const T*)ctx->w.lm_head, R, V, E, nullptr, 0, logits, V);
    MOA_CHECK_LAUNCH();
  }
  if (timed) cudaEventRecord(ctx->prof_ev[2 * ctx->prof_n++ + 1], s);
  launch_pdl(lse_topk_rows_kernel, dim3(R), dim3(256), 0, s, logits, V, B, topk_id, topk_logp);
  MOA_CHECK_LAUNCH();
  return MOA_OK;
}

// The drafter over whole token sequences in one pass (Section 3.1.2: causal SA mask, CA with an optional
// K-step-bounded mask): sequence by sequence, in chunks of up to PREFILL_ROWS rows. A chunk's keys / values go
// into the self-attention prefix cache first, so its attention reads them, and those of the earlier chunks, there.
template <typename T>
static moa_status drafter_prefill_t(moa_ctx* ctx, moa_state* st, const int* tok, const SeqSplit& split, const int* ca_limit,
                                    void* hidden_out, char* ws, const Workspace& p, cudaStream_t s) {
  const moa_config& c = ctx->c;
  const moa_weights& w = ctx->w;
  void* status_word = (char*)st->tree + ctx->tl.status;
  const int E = c.d_model, dh = c.head_dim, V = c.vocab;
  const int nq = c.sa_hq * dh, nkv = c.sa_hkv * dh, cq = c.ca_hq * dh, ckv = c.ca_hkv * dh;
  float* xres = (float*)(ws + p.xres);
  T* xn = (T*)(ws + p.xn);
  T* narrow = (T*)(ws + p.narrow);
  T* obuf = (T*)(ws + p.obuf);
  float* q32 = sizeof(T) == 2 ? (float*)(ws + p.q32) : nullptr;
  const int chunk_rows = imin(p.rows_cap, PREFILL_ROWS);
  LinOut lo;
  for (int b = 0; b < split.n_seq; ++b) {
    const int n = split.off[b + 1] - split.off[b];
    const int base = st->sa_len_host[b], ca_n = st->ca_len_host[b];
    SeqSplit one;                         // rows of this call map to sequence b at offsets 0 .. n-1
    one.n_seq = b + 1;
    for (int i = 0; i <= 64; ++i) one.off[i] = i <= b ? 0 : n;
    const T* sa_k = (const T*)st->sa_k + (size_t)b * c.max_ctx * nkv;
    const T* sa_v = (const T*)st->sa_v + (size_t)b * c.max_ctx * nkv;
    const T* ca_k = (const T*)st->ca_k + (size_t)b * c.max_ctx * ckv;
    const T* ca_v = (const T*)st->ca_v + (size_t)b * c.max_ctx * ckv;
    for (int r0 = 0; r0 < n; r0 += chunk_rows) {
      const int R = imin(chunk_rows, n - r0);
      const int g0 = split.off[b] + r0;                 // first row of the chunk in the caller's arrays
      // ---- self-attention block ----
      launch_pdl(rmsnorm_rows_kernel<T, T>, dim3(R), dim3(256), 0, s, (const T*)w.embed, tok + g0, V, (const T*)w.sa_norm1, E, c.rms_eps,
                 xres, xn, lo_rows_of(sizeof(T), R), (int*)status_word);
      MOA_CHECK_LAUNCH();
      {
        const void* W3[3] = {w.sa_wq, w.sa_wk, w.sa_wv};
        const int N3[3] = {nq, nkv, nkv};
        MOA_TRY(linear<T>(ctx, s, xn, R, E, 3, W3, N3, ws, p, &lo, status_word));
      }
      RopeRows rr;
      memset(&rr, 0, sizeof(rr));
      rr.mode = 1;
      rr.max_ctx = c.max_ctx;
      rr.split = one;
      rr.row0 = r0;
      dim3 rgrid, rblock;
      rope_shape(ctx, R, c.sa_hq + 2 * c.sa_hkv, &rgrid, &rblock);
      launch_pdl(rope_store_kernel<T>, rgrid, rblock, 0, s, lo.part, lo.splits, lo.plane, nq + 2 * nkv, 0, nq,
                 nq + nkv, c.sa_hq, c.sa_hkv, dh, c.sa_rope_theta, st->sa_len, rr, narrow, q32, (T*)st->sa_k, (T*)st->sa_v, (int*)status_word);
      MOA_CHECK_LAUNCH();
      // row i of the chunk sits at position base + r0 + i and sees positions 0 .. base + r0 + i
      MOA_TRY(attention<T>(ctx, s, ws, p, dh, narrow, q32, 1, 0, nq, R, c.sa_hq, c.sa_hkv, sa_k, sa_v, c.max_ctx, nkv, nullptr,
                           base + r0 + R, base + r0 + R, (const T*)nullptr, (const T*)nullptr, 0, nullptr, 0, 0, 0, R, obuf,
                           RowLimit{nullptr, base + r0 + 1, 1}));
      {
        const void* W1[1] = {w.sa_wo};
        const int N1[1] = {E};
        MOA_TRY(linear<T>(ctx, s, obuf, R, nq, 1, W1, N1, ws, p, &lo, status_word));
      }
      MOA_TRY(residual_norm<T>(s, ctx, ws, p, R, E, &lo, w.sa_norm2, nullptr));
      MOA_TRY(mlp_block<T>(s, ctx, p, ws, R, E, c.sa_mlp, w.sa_wgate, w.sa_wup, w.sa_wdown, &lo, status_word));
      // ---- cross-attention block ----
      MOA_TRY(residual_norm<T>(s, ctx, ws, p, R, E, &lo, w.ca_normq, nullptr));
      {
        const void* W1[1] = {w.ca_wq};
        const int N1[1] = {cq};
        MOA_TRY(linear<T>(ctx, s, xn, R, E, 1, W1, N1, ws, p, &lo, status_word));
        if (!q32) {
          const size_t tot = (size_t)R * cq;
          launch_pdl(sum_cast_kernel<T>, dim3(blocks_for(tot / 8, 256)), dim3(256), 0, s, lo.part, lo.splits, lo.plane, tot, narrow);
          MOA_CHECK_LAUNCH();
        }
      }
      MOA_TRY(attention<T>(ctx, s, ws, p, dh, narrow, q32 ? lo.part : nullptr, lo.splits, lo.plane, cq, R, c.ca_hq, c.ca_hkv, ca_k, ca_v,
                           c.max_ctx, ckv, nullptr, ca_n, ca_n, (const T*)nullptr, (const T*)nullptr, 0, nullptr, 0, 0, 0, R, obuf,
                           RowLimit{ca_limit ? ca_limit + g0 : nullptr, 0, 0}));
      {
        const void* W1[1] = {w.ca_wo};
        const int N1[1] = {E};
        MOA_TRY(linear<T>(ctx, s, obuf, R, cq, 1, W1, N1, ws, p, &lo, status_word));
      }
      MOA_TRY(residual_norm<T>(s, ctx, ws, p, R, E, &lo, w.ca_norm2, nullptr));
      MOA_TRY(mlp_block<T>(s, ctx, p, ws, R, E, c.ca_mlp, w.ca_wgate, w.ca_wup, w.ca_wdown, &lo, status_word));
      MOA_TRY(residual_norm<T>(s, ctx, ws, p, R, E, &lo, nullptr, (T*)hidden_out + (size_t)g0 * E));
    }
  }
  add_len_kernel<<<1, 64, 0, s>>>(st->sa_len, split, c.max_ctx);
  MOA_CHECK_LAUNCH();
  return MOA_OK;
}

// One causal self-attention block over (a prefix cache, the row's drafted ancestors, itself) plus its MLP:
// the drafter's SA block and every Target-Layer-Inference decoder layer have this shape (Section 3.1.2,
// Section 3.2). On entry xn holds the block's normalised input and xres the residual stream; on exit the
// MLP's down-projection is pending in `lo` (folded in by the next residual_norm).
struct TreeAttnLayer {
  const void *wq, *wk, *wv, *wo, *norm2, *wgate, *wup, *wdown;
  int hq, hkv, mlp;
  float theta;
  const void *ck, *cv;     // prefix cache T [max_batch, max_ctx, hkv, dh]
  void *tk, *tv;           // tree slots T [max_batch, NS, hkv, dh]
};

template <typename T>
static moa_status tree_attn_layer(moa_ctx* ctx, moa_state* st, cudaStream_t s, char* ws, const Workspace& p, int R,
                                  int rows_per_seq, int max_len, const int* row_anc, const TreeAttnLayer& a, LinOut* lo,
                                  void* status_word) {
  const moa_config& c = ctx->c;
  const TreeLayout& L = ctx->tl;
  const int step = st->step, B = c.tree_topk, D = c.tree_depth, E = c.d_model, dh = c.head_dim;
  T* xn = (T*)(ws + p.xn);
  T* narrow = (T*)(ws + p.narrow);
  T* obuf = (T*)(ws + p.obuf);
  // bf16 path: the queries stay in fp32 and are split into two bf16 terms by the attention kernel
  float* q32 = sizeof(T) == 2 ? (float*)(ws + p.q32) : nullptr;
  const int nq = a.hq * dh, nkv = a.hkv * dh;
  {
    const void* W3[3] = {a.wq, a.wk, a.wv};
    const int N3[3] = {nq, nkv, nkv};
    MOA_TRY(linear<T>(ctx, s, xn, R, E, 3, W3, N3, ws, p, lo, status_word));
  }
  RopeRows rr;
  memset(&rr, 0, sizeof(rr));
  rr.mode = 0;
  rr.step = step;
  rr.B = B;
  rr.slots = L.NS;
  dim3 rgrid, rblock;
  rope_shape(ctx, R, a.hq + 2 * a.hkv, &rgrid, &rblock);
  launch_pdl(rope_store_kernel<T>, rgrid, rblock, 0, s, lo->part, lo->splits, lo->plane, nq + 2 * nkv, 0, nq,
             nq + nkv, a.hq, a.hkv, dh, a.theta, st->sa_len, rr, narrow, q32, (T*)a.tk, (T*)a.tv, (int*)status_word);
  MOA_CHECK_LAUNCH();
  MOA_TRY(attention<T>(ctx, s, ws, p, dh, narrow, q32, 1, 0, nq, R, a.hq, a.hkv, (const T*)a.ck, (const T*)a.cv, c.max_ctx, nkv,
                       st->sa_len, 0, max_len, (const T*)a.tk, (const T*)a.tv, L.NS, row_anc, D, step + 1,
                       step == 0 ? 1 : 1 + step * B, rows_per_seq, obuf, RowLimit{nullptr, 0, 0}, status_word, true));
  {
    const void* W1[1] = {a.wo};
    const int N1[1] = {E};
    MOA_TRY(linear<T>(ctx, s, obuf, R, nq, 1, W1, N1, ws, p, lo, status_word));
  }
  MOA_TRY(residual_norm<T>(s, ctx, ws, p, R, E, lo, a.norm2, nullptr));
  return mlp_block<T>(s, ctx, p, ws, R, E, a.mlp, a.wgate, a.wup, a.wdown, lo, status_word);
}

template <typename T>
static moa_status draft_step_t(moa_ctx* ctx, moa_state* st, int batch, int* topk_id, float* topk_logp,
                               void* hidden_out, char* ws, const Workspace& p, cudaStream_t s) {
  const moa_config& c = ctx->c;
  const moa_weights& w = ctx->w;
  const TreeLayout& L = ctx->tl;
  const TreePtrs tp = tree_ptrs(st->tree, L);
  void* status_word = (char*)st->tree + L.status;
  const int step = st->step, B = c.tree_topk, D = c.tree_depth;
  const int R = step == 0 ? batch : batch * B;
  const int rows_per_seq = step == 0 ? 1 : B;
  const int nbB = c.max_batch * B;
  const int E = c.d_model, dh = c.head_dim, V = c.vocab;
  const int cur = step & 1;
  const int* row_tok = tp.row_tok + (size_t)cur * nbB;
  const int* row_anc = tp.row_anc + (size_t)cur * nbB * D;
  float* xres = (float*)(ws + p.xres);
  T* xn = (T*)(ws + p.xn);
  T* narrow = (T*)(ws + p.narrow);
  T* obuf = (T*)(ws + p.obuf);
  float* q32 = sizeof(T) == 2 ? (float*)(ws + p.q32) : nullptr;
  LinOut lo;
  int max_sa = 0, max_ca = 0;
  for (int b = 0; b < batch; ++b) {
    max_sa = imax(max_sa, st->sa_len_host[b]);
    max_ca = imax(max_ca, st->ca_len_host[b]);
  }

  // ---- self-attention block ----
  launch_pdl(rmsnorm_rows_kernel<T, T>, dim3(R), dim3(256), 0, s, (const T*)w.embed, row_tok, V, (const T*)w.sa_norm1, E, c.rms_eps, xres, xn,
             lo_rows_of(sizeof(T), R), (int*)status_word);
  MOA_CHECK_LAUNCH();
  {
    TreeAttnLayer a = {w.sa_wq, w.sa_wk, w.sa_wv, w.sa_wo, w.sa_norm2, w.sa_wgate, w.sa_wup, w.sa_wdown,
                       c.sa_hq, c.sa_hkv, c.sa_mlp, c.sa_rope_theta, st->sa_k, st->sa_v,
                       (char*)st->tree + L.tk, (char*)st->tree + L.tv};
    MOA_TRY(tree_attn_layer<T>(ctx, st, s, ws, p, R, rows_per_seq, max_sa, row_anc, a, &lo, status_word));
  }

  // ---- cross-attention block ----
  MOA_TRY(residual_norm<T>(s, ctx, ws, p, R, E, &lo, w.ca_normq, nullptr));
  const int cq = c.ca_hq * dh, ckv = c.ca_hkv * dh;
  {
    const void* W1[1] = {w.ca_wq};
    const int N1[1] = {cq};
    MOA_TRY(linear<T>(ctx, s, xn, R, E, 1, W1, N1, ws, p, &lo, status_word));
    if (!q32) {                              // fp32 path: queries in the storage type
      const size_t tot = (size_t)R * cq;
      launch_pdl(sum_cast_kernel<T>, dim3(blocks_for(tot / 8, 256)), dim3(256), 0, s, lo.part, lo.splits, lo.plane, tot, narrow);
      MOA_CHECK_LAUNCH();
    }
  }
  // bf16 path: the attention kernel reads the projection's split planes itself (fp32 queries, two bf16 terms)
  MOA_TRY(attention<T>(ctx, s, ws, p, dh, narrow, q32 ? lo.part : nullptr, lo.splits, lo.plane, cq, R, c.ca_hq, c.ca_hkv,
                       (const T*)st->ca_k, (const T*)st->ca_v, c.max_ctx, ckv, st->ca_len, 0, max_ca, (const T*)nullptr,
                       (const T*)nullptr, 0, nullptr, 0, 0, 0, rows_per_seq, obuf, RowLimit{nullptr, 0, 0}, status_word, true));
  {
    const void* W1[1] = {w.ca_wo};
    const int N1[1] = {E};
    MOA_TRY(linear<T>(ctx, s, obuf, R, cq, 1, W1, N1, ws, p, &lo, status_word));
  }
  MOA_TRY(residual_norm<T>(s, ctx, ws, p, R, E, &lo, w.ca_norm2, nullptr));
  MOA_TRY(mlp_block<T>(s, ctx, p, ws, R, E, c.ca_mlp, w.ca_wgate, w.ca_wup, w.ca_wdown, &lo, status_word));

  // ---- Target Layer Inference: the last N decoder layers of the LLM on the drafted rows (Section 3.2) ----
  for (int l = 0; l < ctx->tli.n_layers; ++l) {
    const moa_tli_layer& t = ctx->tli_w[l];
    MOA_TRY(residual_norm<T>(s, ctx, ws, p, R, E, &lo, t.norm1, nullptr));
    TreeAttnLayer a = {t.wq, t.wk, t.wv, t.wo, t.norm2, t.wgate, t.wup, t.wdown,
                       ctx->tli.hq, ctx->tli.hkv, ctx->tli.mlp, ctx->tli.rope_theta, ctx->tli_c.k[l], ctx->tli_c.v[l],
                       (char*)st->tree + L.tli_tk[l], (char*)st->tree + L.tli_tv[l]};
    MOA_TRY(tree_attn_layer<T>(ctx, st, s, ws, p, R, rows_per_seq, max_sa, row_anc, a, &lo, status_word));
  }

  // ---- LM head, log-softmax, top-B ----
  MOA_TRY(residual_norm<T>(s, ctx, ws, p, R, E, &lo, w.final_norm, hidden_out));
  return lm_head_t<T>(ctx, s, ws, p, R, topk_id, topk_logp, status_word);
}

// ---------------------------------------------------------------------------------------------
// phase-machine paths (bf16): one cooperative kernel per drafter forward / per LSA pass
// ---------------------------------------------------------------------------------------------
struct PmBuild {
  PmParams P;
  moa_ctx* ctx;
  int NB, grid;
  int unit_run;          // units scheduled so far (rotates the CTA that gets unit 0 of the next GEMM)
  size_t attn_bytes;     // shared memory the layer self-attention phase needs (laid over the ring)
  moa_status err;
};

static void pm_init(PmBuild& b, moa_ctx* ctx, void* tree, const TreeLayout& L, char* ws, const Workspace& p) {
  memset(&b.P, 0, sizeof(b.P));
  b.ctx = ctx;
  b.grid = ctx->sm_count;
  b.unit_run = 0;
  b.attn_bytes = 4096;
  b.err = MOA_OK;
  b.NB = 256;
  b.P.sync = (int*)((char*)tree + L.status) + 4;
  b.P.flags = (int*)((char*)tree + L.flags);
  b.P.status = (int*)((char*)tree + L.status);
  b.P.trace = ctx->prof_on ? (unsigned long long*)(ws + p.trace) : nullptr;
}

static PmOp* pm_op(PmBuild& b, int kind, int gemm, int rows, int cols) {
  if (b.P.n_ops >= PM_MAX_OPS) { b.err = MOA_ERR_SHAPE; return &b.P.op[PM_MAX_OPS - 1]; }
  PmOp* op = &b.P.op[b.P.n_ops++];
  memset(op, 0, sizeof(*op));
  op->kind = kind; op->gemm = gemm; op->rows = rows; op->cols = cols;
  return op;
}

// Adds a GEMM phase: X buffer [R (+ low half), K] times up to three weight matrices. mode as in PmGemm.
static int pm_gemm(PmBuild& b, const void* X, int R, int K, int nseg, const void* const* W, const int* N, int mode,
                   float* part, int part_rows) {
  if (b.P.n_gemms >= PM_MAX_GEMMS) { b.err = MOA_ERR_SHAPE; return 0; }
  const int gi = b.P.n_gemms++;
  PmGemm& G = b.P.g[gi];
  memset(&G, 0, sizeof(G));
  G.n_seg = nseg; G.mode = mode; G.R = R;
  int tiles = 0, col = 0;
  for (int i = 0; i < nseg; ++i) {
    const WeightMap* wm = find_wmap(b.ctx, W[i]);
    if (!wm) { b.err = MOA_ERR_SHAPE; return gi; }
    b.P.tm[gi][i] = wm->tm;
    G.seg_n[i] = N[i]; G.seg_tile0[i] = tiles; G.seg_col[i] = col;
    tiles += (N[i] + WS_BM - 1) / WS_BM;
    col += N[i];
  }
  if (mode == 4) tiles = (N[0] + WS_BM - 1) / WS_BM;      // gate and up tiles travel in pairs
  G.tiles_total = tiles;
  G.kb_total = K / WS_BK;
  G.rows_per_block = mode == 4 ? 128 : b.NB;
  G.row_blocks = mode >= 2 ? (R + G.rows_per_block - 1) / G.rows_per_block : 1;
  G.splits = mode == 0 ? pick_splits(tiles, G.kb_total, R, part_rows, b.grid) : 1;
  G.units = tiles * G.splits * G.row_blocks;
  G.rot = b.unit_run % b.grid;
  b.unit_run += G.units;
  G.ldo = col;
  G.plane = (size_t)R * col;
  G.out = part;
  const int rows_total = R;
  cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows_total};
  cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  cuuint32_t box[2] = {(cuuint32_t)WS_BK, (cuuint32_t)G.rows_per_block};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = b.ctx->encode(&b.P.tm[gi][3], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(X), dims, strides,
                             box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    snprintf(g_cuda_err, sizeof(g_cuda_err), "cuTensorMapEncodeTiled (activations) failed (%d)", (int)r);
    b.err = MOA_ERR_CUDA;
  }
  pm_op(b, PH_GEMM, gi, R, col);
  return gi;
}

template <int NB>
static moa_status pm_launch_nb(cudaStream_t s, const PmParams& P, int grid, size_t smem) {
  static size_t attr = 0;
  if (smem > attr) {
    cudaError_t e = cudaFuncSetAttribute(phase_machine_kernel<NB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) {
      snprintf(g_cuda_err, sizeof(g_cuda_err), "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
      return MOA_ERR_CUDA;
    }
    attr = smem;
  }
  void* args[1] = {(void*)&P};
  cudaError_t e = cudaLaunchCooperativeKernel((const void*)phase_machine_kernel<NB>, dim3(grid), dim3(PM_THREADS), args,
                                              smem, s);
  ++g_launches;
  if (e != cudaSuccess) {
    snprintf(g_cuda_err, sizeof(g_cuda_err), "cooperative launch: %s", cudaGetErrorString(e));
    return MOA_ERR_CUDA;
  }
  return MOA_OK;
}

static moa_status pm_launch(PmBuild& b, cudaStream_t s) {
  if (b.err != MOA_OK) return b.err;
  b.ctx->last_n_ops = b.P.n_ops;
  for (int i = 0; i < b.P.n_ops; ++i) b.ctx->last_kinds[i] = b.P.op[i].kind;
  const int stage = WS_W_BYTES + b.NB * WS_BK * 2;
  const size_t fixed = PM_FIXED_SMEM;                     // alignment slack, barriers, descriptor copies
  int stages = (int)(((size_t)b.ctx->smem_optin - fixed) / stage);
  if (stages > PM_MAX_STAGES) stages = PM_MAX_STAGES;
  if (stages < 2 || (size_t)stages * stage < b.attn_bytes) return MOA_ERR_SHAPE;
  b.P.stages = stages;
  b.P.alias_attn = 1;                                     // the attention scratch lies over the ring
  b.P.attn_off = 0u;
  return pm_launch_nb<256>(s, b.P, b.grid, fixed + (size_t)stages * stage);
}

// Layer Self-Attention phase: one warp per (token, query head), rows staged by bulk asynchronous copies.
static int pm_lsa_warps(const moa_ctx* ctx, int S, int dh) {      // warps of a CTA that fit their stacks (0: none)
  const int s_pad = (S + 15) & ~15;
  const size_t per_warp = (size_t)3 * s_pad * (dh * 2 + 16) + 16;
  const int stage = WS_W_BYTES + 256 * WS_BK * 2;
  const size_t avail = (size_t)((ctx->smem_optin - PM_FIXED_SMEM) / stage) * stage;
  return S > 128 ? 0 : imin(PM_WWARPS, (int)(avail / per_warp));
}
static void pm_lsa_attention_op(PmBuild& b, int R, int n_tok, int S, int hq, int hkv, int dh, const bf16* qkv, int ld, bf16* out) {
  const int s_pad = (S + 15) & ~15;
  const size_t per_warp = (size_t)3 * s_pad * (dh * 2 + 16) + 16;
  const int n_warps = pm_lsa_warps(b.ctx, S, dh);
  if (n_warps < 1) { b.err = MOA_ERR_SHAPE; return; }         // ruled out by pm_usable()
  if (n_warps * per_warp > b.attn_bytes) b.attn_bytes = n_warps * per_warp;
  PmOp* op = pm_op(b, PH_LSA_ATTN, -1, R, n_tok);
  op->p[0] = qkv; op->p[1] = out;
  op->i[0] = ld; op->i[1] = hq; op->i[2] = hkv; op->i[3] = S; op->i[4] = n_warps; op->i[5] = 0; op->i[6] = dh;
  op->f[0] = 1.4426950408889634f / sqrtf((float)dh);
}

static void pm_resnorm(PmBuild& b, int gemm, int R, int K, float* xres, const void* gain, bf16* xn, void* hidden,
                       float eps) {
  PmOp* op = pm_op(b, PH_RESNORM, gemm, R, K);
  op->p[2] = gain; op->p[3] = xres; op->p[4] = xn; op->p[5] = hidden;
  op->i[1] = 0; op->f[0] = eps;
}

// One LSA pass over nt tokens (rows t0*S .. of h_stack) in the dense regime (more than 256 rows).
static moa_status lsa_pass_pm(moa_ctx* ctx, moa_state* st, const bf16* x, int nt, int t0, const SeqSplit& split,
                              bf16* kv_out, char* ws, const Workspace& p, cudaStream_t s) {
  const moa_config& c = ctx->c;
  const moa_weights& w = ctx->w;
  const TreeLayout& L = ctx->tl;
  const int S = c.n_stack, D = c.d_stack, dh = c.head_dim, F = c.lsa_mlp;
  const int nq = c.lsa_hq * dh, nkv = c.lsa_hkv * dh, ld = nq + 2 * nkv, ckv = c.ca_hkv * dh;
  const int R = nt * S;
  float* xres = (float*)(ws + p.xres);
  bf16* xn = (bf16*)(ws + p.xn);
  bf16* narrow = (bf16*)(ws + p.narrow);
  bf16* obuf = (bf16*)(ws + p.obuf);
  float* part = (float*)(ws + p.part);
  float* kvf = (float*)(ws + p.kvf);
  bf16* kvn = (bf16*)(ws + p.kvn);
  PmBuild b;
  pm_init(b, ctx, st->tree, L, ws, p);
  b.P.split = split;
  {
    PmOp* op = pm_op(b, PH_ROWS_NORM, -1, R, D);
    op->p[0] = x; op->p[2] = w.lsa_norm1; op->p[3] = xres; op->p[4] = xn;
    op->i[1] = 0; op->f[0] = c.rms_eps;
  }
  const void* W3[3] = {w.lsa_wq, w.lsa_wk, w.lsa_wv};
  const int N3[3] = {nq, nkv, nkv};
  const void* Wo[1] = {w.lsa_wo};
  const int No[1] = {D};
  const int g0 = pm_gemm(b, xn, R, D, 3, W3, N3, 2, nullptr, 0);
  b.P.g[g0].out16 = narrow; b.P.g[g0].ld16 = ld;
  pm_lsa_attention_op(b, R, nt, S, c.lsa_hq, c.lsa_hkv, dh, narrow, ld, obuf);
  const int g1 = pm_gemm(b, obuf, R, nq, 1, Wo, No, 3, xres, 0);
  b.P.g[g1].ldo = D;
  pm_resnorm(b, -1, R, D, xres, w.lsa_norm2, xn, nullptr, c.rms_eps);
  const void* W2[2] = {w.lsa_wgate, w.lsa_wup};
  const int N2[2] = {F, F};
  const int g2 = pm_gemm(b, xn, R, D, 2, W2, N2, 4, nullptr, 0);
  b.P.g[g2].out16 = narrow; b.P.g[g2].ld16 = F;
  const void* Wd[1] = {w.lsa_wdown};
  const int g3 = pm_gemm(b, narrow, R, F, 1, Wd, No, 3, xres, 0);
  b.P.g[g3].ldo = D;
  {
    PmOp* op = pm_op(b, PH_MEAN_NORM, -1, nt, D);
    op->p[0] = xres; op->p[1] = kvf; op->p[2] = kv_out; op->p[3] = w.ca_normkv; op->p[4] = kvn;
    op->i[0] = S; op->i[1] = 0; op->f[0] = c.rms_eps;
  }
  {
    const void* Wkv[2] = {w.ca_wk, w.ca_wv};
    const int Nkv[2] = {ckv, ckv};
    const int g = pm_gemm(b, kvn, nt, D, 2, Wkv, Nkv, 0, part, p.part_rows);
    PmOp* op = pm_op(b, PH_CACHE_APPEND, g, nt, 2 * ckv);
    op->p[0] = st->ca_len; op->p[1] = st->ca_k; op->p[2] = st->ca_v;
    op->i[0] = ckv; op->i[1] = c.max_ctx; op->i[2] = t0;
  }
  return pm_launch(b, s);
}

static bool pm_usable(const moa_ctx* ctx) {
  if (!ctx->fast || !ctx->coop || ctx->c.dtype != MOA_BF16 || ctx->sm_count > 256) return false;
  const moa_weights& w = ctx->w;
  const void* all[] = {w.lsa_wq, w.lsa_wk, w.lsa_wv, w.lsa_wo, w.lsa_wgate, w.lsa_wup, w.lsa_wdown, w.ca_wk, w.ca_wv};
  for (const void* m : all)
    if (!find_wmap(ctx, m)) return false;
  const moa_config& c = ctx->c;
  if (c.d_stack % 64 != 0 || c.lsa_mlp % 64 != 0) return false;
  return pm_lsa_warps(ctx, c.n_stack, c.head_dim) >= 1;       // a token's stack of q, k, v rows fits in shared memory
}

// ---------------------------------------------------------------------------------------------
// exported functions
// ---------------------------------------------------------------------------------------------
extern "C" {

const char* moa_status_str(moa_status s) {
  switch (s) {
    case MOA_OK: return "ok";
    case MOA_ERR_NULL: return "null pointer";
    case MOA_ERR_SHAPE: return "bad shape";
    case MOA_ERR_DTYPE: return "bad dtype";
    case MOA_ERR_ALIGN: return "pointer not 16-byte aligned";
    case MOA_ERR_WORKSPACE: return "workspace too small";
    case MOA_ERR_CAPACITY: return "capacity exceeded";
    case MOA_ERR_STATE: return "call out of order";
    case MOA_ERR_ARCH: return "device is not compute capability 10.x";
    case MOA_ERR_CUDA: return "CUDA error";
    case MOA_ERR_TIMEOUT: return "device-side wait timed out";
    case MOA_ERR_NONFINITE: return "a log-probability was not a number";
  }
  return "unknown";
}

const char* moa_last_cuda_error(void) { return g_cuda_err; }

static moa_status validate_config(const moa_config* c) {
  if (c->dtype != MOA_F32 && c->dtype != MOA_BF16) return MOA_ERR_DTYPE;
  if (c->head_dim != 64 && c->head_dim != 128) return MOA_ERR_SHAPE;
  const int dims[] = {c->d_model, c->d_stack, c->lsa_mlp, c->sa_mlp, c->ca_mlp};
  for (int d : dims)
    if (d <= 0 || d % 16 != 0) return MOA_ERR_SHAPE;
  if (c->dtype == MOA_BF16 && c->d_model % 64 != 0) return MOA_ERR_SHAPE;   // the fused LM head streams 64-wide k blocks
  if (c->n_stack <= 0 || c->vocab <= 0) return MOA_ERR_SHAPE;
  const int hq[] = {c->lsa_hq, c->sa_hq, c->ca_hq}, hkv[] = {c->lsa_hkv, c->sa_hkv, c->ca_hkv};
  for (int i = 0; i < 3; ++i)
    if (hq[i] <= 0 || hkv[i] <= 0 || hq[i] % hkv[i] != 0) return MOA_ERR_SHAPE;
  if (c->max_batch <= 0 || c->max_batch > MOA_MAX_BATCH) return MOA_ERR_SHAPE;
  if (c->max_ctx <= 0) return MOA_ERR_SHAPE;
  if (c->tree_topk <= 0 || c->tree_topk > MOA_MAX_TOPK || c->tree_topk > c->vocab) return MOA_ERR_SHAPE;
  if (c->tree_depth <= 0 || c->tree_depth > MOA_MAX_DEPTH) return MOA_ERR_SHAPE;
  if (c->tree_keep <= 0) return MOA_ERR_SHAPE;
  if ((long long)c->max_batch * c->tree_topk > 256) return MOA_ERR_SHAPE;   // rows of one draft step
  if (!(c->rms_eps >= 0.f) || !(c->sa_rope_theta >= 0.f)) return MOA_ERR_SHAPE;
  return MOA_OK;
}

moa_status moa_create(const moa_config* cfg, const moa_weights* w, moa_ctx** out) {
  if (!cfg || !w || !out) return MOA_ERR_NULL;
  *out = nullptr;
  MOA_TRY(validate_config(cfg));
  const void* const* wp = (const void* const*)w;
  for (size_t i = 0; i < sizeof(moa_weights) / sizeof(void*); ++i) {
    if (!wp[i]) return MOA_ERR_NULL;
    if (!aligned16(wp[i])) return MOA_ERR_ALIGN;
  }
  int dev = 0;
  cudaDeviceProp prop;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaGetDeviceProperties(&prop, dev);
  if (e != cudaSuccess) {
    snprintf(g_cuda_err, sizeof(g_cuda_err), "moa_create: %s", cudaGetErrorString(e));
    return MOA_ERR_CUDA;
  }
  if (prop.major != 10) return MOA_ERR_ARCH;
  moa_ctx* ctx = new (std::nothrow) moa_ctx;
  if (!ctx) return MOA_ERR_NULL;
  ctx->c = *cfg;
  ctx->w = *w;
  ctx->sm_count = prop.multiProcessorCount;
  ctx->elt = cfg->dtype == MOA_F32 ? 4 : 2;
  ctx->tl = make_tree_layout(cfg->max_batch, cfg->tree_topk, cfg->tree_depth, cfg->sa_hkv, cfg->head_dim, ctx->elt);
  ctx->prof_on = false;
  ctx->prof_n = 0;
  ctx->prof_made = false;
  ctx->encode = nullptr;
  ctx->n_wmap = 0;
  ctx->fast = false;
  ctx->coop = prop.cooperativeLaunch != 0;
  ctx->smem_optin = (int)prop.sharedMemPerBlockOptin;
  ctx->last_n_ops = 0;
  ctx->n_wmap_base = 0;
  memset(&ctx->tli, 0, sizeof(ctx->tli));
  memset(ctx->tli_w, 0, sizeof(ctx->tli_w));
  memset(&ctx->tli_c, 0, sizeof(ctx->tli_c));
  if (cfg->dtype == MOA_BF16) {
    // tensor maps of every weight matrix whose inner dimension the streaming GEMM can take
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) {
      snprintf(g_cuda_err, sizeof(g_cuda_err), "moa_create: cuTensorMapEncodeTiled unavailable");
      delete ctx;
      return MOA_ERR_CUDA;
    }
    ctx->encode = (EncodeTiledFn)fn;
    const int dh = cfg->head_dim, E = cfg->d_model, Din = cfg->d_stack;
    struct { const void* p; int n, k; } mats[] = {
        {w->lm_head, cfg->vocab, E},
        {w->lsa_wq, cfg->lsa_hq * dh, Din}, {w->lsa_wk, cfg->lsa_hkv * dh, Din}, {w->lsa_wv, cfg->lsa_hkv * dh, Din},
        {w->lsa_wo, Din, cfg->lsa_hq * dh}, {w->lsa_wgate, cfg->lsa_mlp, Din}, {w->lsa_wup, cfg->lsa_mlp, Din},
        {w->lsa_wdown, Din, cfg->lsa_mlp},
        {w->sa_wq, cfg->sa_hq * dh, E}, {w->sa_wk, cfg->sa_hkv * dh, E}, {w->sa_wv, cfg->sa_hkv * dh, E},
        {w->sa_wo, E, cfg->sa_hq * dh}, {w->sa_wgate, cfg->sa_mlp, E}, {w->sa_wup, cfg->sa_mlp, E},
        {w->sa_wdown, E, cfg->sa_mlp},
        {w->ca_wq, cfg->ca_hq * dh, E}, {w->ca_wk, cfg->ca_hkv * dh, Din}, {w->ca_wv, cfg->ca_hkv * dh, Din},
        {w->ca_wo, E, cfg->ca_hq * dh}, {w->ca_wgate, cfg->ca_mlp, E}, {w->ca_wup, cfg->ca_mlp, E},
        {w->ca_wdown, E, cfg->ca_mlp}};
    for (auto& m : mats) {
      if (m.k % WS_BK != 0) continue;    // such a matrix takes the generic GEMM
      WeightMap& wm = ctx->wmap[ctx->n_wmap];
      wm.ptr = m.p;
      wm.n = m.n;
      wm.k = m.k;
      if (!encode_map(ctx, &wm.tm, m.p, m.n, m.k, WS_BM)) {
        delete ctx;
        return MOA_ERR_CUDA;
      }
      ++ctx->n_wmap;
    }
    ctx->fast = true;
    ctx->n_wmap_base = ctx->n_wmap;
  }
  *out = ctx;
  return MOA_OK;
}

moa_status moa_tli_configure(moa_ctx* ctx, const moa_tli_config* cfg, const moa_tli_layer* layers_host,
                             const moa_tli_caches* caches) {
  if (!ctx || !cfg) return MOA_ERR_NULL;
  const moa_config& c = ctx->c;
  const int n = cfg->n_layers;
  if (n < 0 || n > MOA_MAX_TLI) return MOA_ERR_SHAPE;
  if (n > 0) {
    if (!layers_host || !caches) return MOA_ERR_NULL;
    if (cfg->hq <= 0 || cfg->hkv <= 0 || cfg->hq % cfg->hkv != 0) return MOA_ERR_SHAPE;
    if (cfg->mlp <= 0 || cfg->mlp % 16 != 0 || !(cfg->rope_theta >= 0.f)) return MOA_ERR_SHAPE;
    for (int l = 0; l < n; ++l) {
      const void* const* wp = (const void* const*)&layers_host[l];
      for (size_t i = 0; i < sizeof(moa_tli_layer) / sizeof(void*); ++i) {
        if (!wp[i]) return MOA_ERR_NULL;
        if (!aligned16(wp[i])) return MOA_ERR_ALIGN;
      }
      if (!caches->k[l] || !caches->v[l]) return MOA_ERR_NULL;
      if (!aligned16(caches->k[l]) || !aligned16(caches->v[l])) return MOA_ERR_ALIGN;
    }
  }
  // tensor maps of the layers' matrices follow the drafter's own (bf16 path)
  ctx->n_wmap = ctx->n_wmap_base;
  if (n > 0 && ctx->fast) {
    const int dh = c.head_dim, E = c.d_model;
    for (int l = 0; l < n; ++l) {
      const moa_tli_layer& t = layers_host[l];
      struct { const void* p; int n, k; } mats[] = {
          {t.wq, cfg->hq * dh, E}, {t.wk, cfg->hkv * dh, E}, {t.wv, cfg->hkv * dh, E}, {t.wo, E, cfg->hq * dh},
          {t.wgate, cfg->mlp, E}, {t.wup, cfg->mlp, E}, {t.wdown, E, cfg->mlp}};
      for (auto& m : mats) {
        if (m.k % WS_BK != 0 || find_wmap(ctx, m.p)) continue;
        if (ctx->n_wmap >= WMAP_MAX) return MOA_ERR_SHAPE;
        WeightMap& wm = ctx->wmap[ctx->n_wmap];
        wm.ptr = m.p;
        wm.n = m.n;
        wm.k = m.k;
        if (!encode_map(ctx, &wm.tm, m.p, m.n, m.k, WS_BM)) {
          ctx->n_wmap = ctx->n_wmap_base;
          return MOA_ERR_CUDA;
        }
        ++ctx->n_wmap;
      }
    }
  }
  memset(&ctx->tli, 0, sizeof(ctx->tli));
  memset(ctx->tli_w, 0, sizeof(ctx->tli_w));
  memset(&ctx->tli_c, 0, sizeof(ctx->tli_c));
  if (n > 0) {
    ctx->tli = *cfg;
    for (int l = 0; l < n; ++l) ctx->tli_w[l] = layers_host[l];
    ctx->tli_c = *caches;
  }
  ctx->tl = make_tree_layout(c.max_batch, c.tree_topk, c.tree_depth, c.sa_hkv, c.head_dim, ctx->elt, n, n > 0 ? cfg->hkv : 0);
  return MOA_OK;
}

void moa_destroy(moa_ctx* ctx) {
  if (!ctx) return;
  if (ctx->prof_made)
    for (int i = 0; i < 2 * PROF_MAX; ++i) cudaEventDestroy(ctx->prof_ev[i]);
  delete ctx;
}

moa_status moa_profile_begin(moa_ctx* ctx) {
  if (!ctx) return MOA_ERR_NULL;
  if (!ctx->prof_made) {
    for (int i = 0; i < 2 * PROF_MAX; ++i) {
      cudaError_t e = cudaEventCreate(&ctx->prof_ev[i]);
      if (e != cudaSuccess) {
        snprintf(g_cuda_err, sizeof(g_cuda_err), "moa_profile_begin: %s", cudaGetErrorString(e));
        for (int j = 0; j < i; ++j) cudaEventDestroy(ctx->prof_ev[j]);
        return MOA_ERR_CUDA;
      }
    }
    ctx->prof_made = true;
  }
  ctx->prof_n = 0;
  ctx->prof_on = true;
  return MOA_OK;
}

moa_status moa_profile_end(moa_ctx* ctx, double* ms_total, int32_t* launches) {
  if (!ctx || !ms_total || !launches) return MOA_ERR_NULL;
  if (!ctx->prof_on) return MOA_ERR_STATE;
  ctx->prof_on = false;
  double total = 0.0;
  for (int i = 0; i < ctx->prof_n; ++i) {
    cudaError_t e = cudaEventSynchronize(ctx->prof_ev[2 * i + 1]);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, ctx->prof_ev[2 * i], ctx->prof_ev[2 * i + 1]);
    if (e != cudaSuccess) {
      snprintf(g_cuda_err, sizeof(g_cuda_err), "moa_profile_end: %s", cudaGetErrorString(e));
      return MOA_ERR_CUDA;
    }
    total += ms;
  }
  *ms_total = total;
  *launches = ctx->prof_n;
  return MOA_OK;
}

int64_t moa_launch_count(void) { return g_launches; }

moa_status moa_trace_begin(void* dev_buf, int32_t cap) {
#ifdef MOA_TRACE
  if (!dev_buf) return MOA_ERR_NULL;
  if (cap <= 0) return MOA_ERR_SHAPE;
  const int zero = 0;
  unsigned long long* b = (unsigned long long*)dev_buf;
  cudaError_t e = cudaMemcpyToSymbol(g_moa_trace_n, &zero, sizeof(int));
  if (e == cudaSuccess) e = cudaMemcpyToSymbol(g_moa_trace_cap, &cap, sizeof(int));
  if (e == cudaSuccess) e = cudaMemcpyToSymbol(g_moa_trace_buf, &b, sizeof(b));
  if (e != cudaSuccess) {
    snprintf(g_cuda_err, sizeof(g_cuda_err), "moa_trace_begin: %s", cudaGetErrorString(e));
    return MOA_ERR_CUDA;
  }
  return MOA_OK;
#else
  (void)dev_buf; (void)cap;
  return MOA_ERR_STATE;
#endif
}

moa_status moa_trace_end(int32_t* n_out) {
#ifdef MOA_TRACE
  if (!n_out) return MOA_ERR_NULL;
  unsigned long long* none = nullptr;
  int n = 0;
  cudaError_t e = cudaDeviceSynchronize();
  if (e == cudaSuccess) e = cudaMemcpyFromSymbol(&n, g_moa_trace_n, sizeof(int));
  if (e == cudaSuccess) e = cudaMemcpyToSymbol(g_moa_trace_buf, &none, sizeof(none));
  if (e != cudaSuccess) {
    snprintf(g_cuda_err, sizeof(g_cuda_err), "moa_trace_end: %s", cudaGetErrorString(e));
    return MOA_ERR_CUDA;
  }
  *n_out = n;
  return MOA_OK;
#else
  (void)n_out;
  return MOA_ERR_STATE;
#endif
}

moa_status moa_profile_phases(moa_ctx* ctx, const void* ws, size_t ws_bytes, int32_t cap, double* us_out,
                              double* wait_us_out, int32_t* kind_out, int32_t* n_out, void* stream) {
  if (!ctx || !ws || !us_out || !kind_out || !n_out) return MOA_ERR_NULL;
  const int chunk = chunk_from_bytes(ctx->c, ctx->tli, ctx->elt, ws_bytes);
  if (chunk < 1) return MOA_ERR_WORKSPACE;
  const Workspace p = plan_workspace(ctx->c, ctx->tli, ctx->elt, chunk);
  unsigned long long t[2 * PM_MAX_OPS + 1];
  cudaError_t e = cudaMemcpyAsync(t, (const char*)ws + p.trace, sizeof(t), cudaMemcpyDeviceToHost, (cudaStream_t)stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
  if (e != cudaSuccess) {
    snprintf(g_cuda_err, sizeof(g_cuda_err), "moa_profile_phases: %s", cudaGetErrorString(e));
    return MOA_ERR_CUDA;
  }
  const int n = ctx->last_n_ops < cap ? ctx->last_n_ops : cap;
  for (int i = 0; i < n; ++i) {
    us_out[i] = (double)(t[2 * i + 2] - t[2 * i]) * 1e-3;
    if (wait_us_out) wait_us_out[i] = (double)(t[2 * i + 2] - t[2 * i + 1]) * 1e-3;
    kind_out[i] = ctx->last_kinds[i];
  }
  *n_out = n;
  return MOA_OK;
}

moa_status moa_state_bytes(const moa_ctx* ctx, int32_t lsa_chunk_tokens, size_t* tree_bytes, size_t* workspace_bytes) {
  if (!ctx) return MOA_ERR_NULL;
  if (lsa_chunk_tokens < 1) return MOA_ERR_SHAPE;
  if (tree_bytes) *tree_bytes = ctx->tl.total;
  if (workspace_bytes) *workspace_bytes = plan_workspace(ctx->c, ctx->tli, ctx->elt, lsa_chunk_tokens).total;
  return MOA_OK;
}

static moa_status check_state(const moa_ctx* ctx, const moa_state* st, int batch) {
  if (!ctx || !st) return MOA_ERR_NULL;
  if (batch <= 0 || batch > ctx->c.max_batch) return MOA_ERR_SHAPE;
  const void* ptrs[] = {st->ca_k, st->ca_v, st->sa_k, st->sa_v, st->ca_len, st->sa_len, st->tree};
  for (const void* p : ptrs) {
    if (!p) return MOA_ERR_NULL;
    if (!aligned16(p)) return MOA_ERR_ALIGN;
  }
  if (!st->ca_len_host || !st->sa_len_host) return MOA_ERR_NULL;
  return MOA_OK;
}

static moa_status make_split(const int32_t* n_host, int batch, SeqSplit* sp) {
  sp->n_seq = batch;
  long long run = 0;
  for (int b = 0; b < batch; ++b) {
    if (n_host[b] < 0) return MOA_ERR_SHAPE;
    sp->off[b] = (int)run;
    run += n_host[b];
    if (run > 0x3fffffff) return MOA_ERR_SHAPE;
  }
  for (int b = batch; b <= 64; ++b) sp->off[b] = (int)run;
  return MOA_OK;
}

moa_status moa_state_set_len(moa_ctx* ctx, moa_state* st, int32_t which, const int32_t* len_host, int32_t batch,
                             void* stream) {
  MOA_TRY(check_state(ctx, st, batch));
  if (!len_host) return MOA_ERR_NULL;
  if (which != 0 && which != 1) return MOA_ERR_SHAPE;
  LenVals lv;
  lv.n = batch;
  for (int b = 0; b < batch; ++b) {
    if (len_host[b] < 0 || len_host[b] > ctx->c.max_ctx) return MOA_ERR_CAPACITY;
    lv.v[b] = len_host[b];
  }
  int32_t* host = which == 0 ? st->ca_len_host : st->sa_len_host;
  for (int b = 0; b < batch; ++b) host[b] = len_host[b];
  set_len_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(which == 0 ? st->ca_len : st->sa_len, lv);
  MOA_CHECK_LAUNCH();
  return MOA_OK;
}

moa_status moa_lsa_forward(moa_ctx* ctx, moa_state* st, const void* h_stack, const int32_t* n_tok_host, int32_t batch,
                           void* kv_out, void* ws, size_t ws_bytes, void* stream) {
  MOA_RANGE();
  MOA_TRY(check_state(ctx, st, batch));
  if (!n_tok_host || !ws) return MOA_ERR_NULL;
  SeqSplit split;
  MOA_TRY(make_split(n_tok_host, batch, &split));
  const int total = split.off[batch];
  if (total > 0 && !h_stack) return MOA_ERR_NULL;
  if (!aligned16(h_stack) || !aligned16(kv_out) || !aligned16(ws)) return MOA_ERR_ALIGN;
  for (int b = 0; b < batch; ++b)
    if ((long long)st->ca_len_host[b] + n_tok_host[b] > ctx->c.max_ctx) return MOA_ERR_CAPACITY;
  const int chunk = chunk_from_bytes(ctx->c, ctx->tli, ctx->elt, ws_bytes);
  if (chunk < 1) return MOA_ERR_WORKSPACE;
  const Workspace p = plan_workspace(ctx->c, ctx->tli, ctx->elt, chunk);
  moa_status r;
  // Passes with more than 256 (token, layer) rows run as one persistent kernel with tensor-core GEMMs whose
  // epilogues are fused (dense regime); smaller ones take the weight-streaming kernels launch by launch.
  if (pm_usable(ctx) && (long long)imin(p.chunk_tok, total) * ctx->c.n_stack > 256) {
    r = MOA_OK;
    const int S = ctx->c.n_stack, D = ctx->c.d_stack;
    // passes of at most 256 tokens (the key/value projection of a pass is one activation block)
    const int per_pass = imin(p.chunk_tok, 256);
    for (int t0 = 0; t0 < total && r == MOA_OK; t0 += per_pass) {
      const int nt = imin(per_pass, total - t0);
      r = lsa_pass_pm(ctx, st, (const bf16*)h_stack + (size_t)t0 * S * D, nt, t0, split,
                      kv_out ? (bf16*)kv_out + (size_t)t0 * D : nullptr, (char*)ws, p, (cudaStream_t)stream);
    }
    if (r == MOA_OK) {
      add_len_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(st->ca_len, split, ctx->c.max_ctx);
      MOA_CHECK_LAUNCH();
    }
  } else {
    r = ctx->c.dtype == MOA_F32
            ? lsa_forward_t<float>(ctx, st, h_stack, split, kv_out, (char*)ws, p, (cudaStream_t)stream)
            : lsa_forward_t<bf16>(ctx, st, h_stack, split, kv_out, (char*)ws, p, (cudaStream_t)stream);
  }
  if (r == MOA_OK)
    for (int b = 0; b < batch; ++b) st->ca_len_host[b] += n_tok_host[b];
  return r;
}

moa_status moa_sa_append(moa_ctx* ctx, moa_state* st, const int32_t* tok, const int32_t* n_host, int32_t batch, void* ws,
                         size_t ws_bytes, void* stream) {
  MOA_RANGE();
  MOA_TRY(check_state(ctx, st, batch));
  if (!n_host || !ws) return MOA_ERR_NULL;
  SeqSplit split;
  MOA_TRY(make_split(n_host, batch, &split));
  if (split.off[batch] > 0 && !tok) return MOA_ERR_NULL;
  if (!aligned16(ws)) return MOA_ERR_ALIGN;
  for (int b = 0; b < batch; ++b)
    if ((long long)st->sa_len_host[b] + n_host[b] > ctx->c.max_ctx) return MOA_ERR_CAPACITY;
  const int chunk = chunk_from_bytes(ctx->c, ctx->tli, ctx->elt, ws_bytes);
  if (chunk < 1) return MOA_ERR_WORKSPACE;
  const Workspace p = plan_workspace(ctx->c, ctx->tli, ctx->elt, chunk);
  moa_status r = ctx->c.dtype == MOA_F32 ? sa_append_t<float>(ctx, st, tok, split, (char*)ws, p, (cudaStream_t)stream)
                                         : sa_append_t<bf16>(ctx, st, tok, split, (char*)ws, p, (cudaStream_t)stream);
  if (r == MOA_OK)
    for (int b = 0; b < batch; ++b) st->sa_len_host[b] += n_host[b];
  return r;
}

moa_status moa_drafter_prefill(moa_ctx* ctx, moa_state* st, const int32_t* tok, const int32_t* n_host, int32_t batch,
                               const int32_t* ca_limit, void* hidden_out, void* ws, size_t ws_bytes, void* stream) {
  MOA_RANGE();
  MOA_TRY(check_state(ctx, st, batch));
  if (!n_host || !ws || !hidden_out) return MOA_ERR_NULL;
  SeqSplit split;
  MOA_TRY(make_split(n_host, batch, &split));
  if (split.off[batch] > 0 && !tok) return MOA_ERR_NULL;
  if (!aligned16(ws) || !aligned16(hidden_out)) return MOA_ERR_ALIGN;
  for (int b = 0; b < batch; ++b)
    if ((long long)st->sa_len_host[b] + n_host[b] > ctx->c.max_ctx) return MOA_ERR_CAPACITY;
  const int chunk = chunk_from_bytes(ctx->c, ctx->tli, ctx->elt, ws_bytes);
  if (chunk < 1) return MOA_ERR_WORKSPACE;
  const Workspace p = plan_workspace(ctx->c, ctx->tli, ctx->elt, chunk);
  moa_status r = ctx->c.dtype == MOA_F32
                     ? drafter_prefill_t<float>(ctx, st, tok, split, ca_limit, hidden_out, (char*)ws, p, (cudaStream_t)stream)
                     : drafter_prefill_t<bf16>(ctx, st, tok, split, ca_limit, hidden_out, (char*)ws, p, (cudaStream_t)stream);
  if (r == MOA_OK)
    for (int b = 0; b < batch; ++b) st->sa_len_host[b] += n_host[b];
  return r;
}

moa_status moa_tree_begin(moa_ctx* ctx, moa_state* st, const int32_t* root_tok, int32_t batch, void* stream) {
  MOA_RANGE();
  MOA_TRY(check_state(ctx, st, batch));
  if (!root_tok) return MOA_ERR_NULL;
  for (int b = 0; b < batch; ++b)
    if (st->sa_len_host[b] < 0 || st->sa_len_host[b] > ctx->c.max_ctx) return MOA_ERR_CAPACITY;
  const TreePtrs tp = tree_ptrs(st->tree, ctx->tl);
  tree_begin_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(tp, root_tok, batch, ctx->c.max_batch * ctx->c.tree_topk,
                                                         ctx->c.tree_depth);
  MOA_CHECK_LAUNCH();
  st->step = 0;
  return MOA_OK;
}

moa_status moa_draft_step(moa_ctx* ctx, moa_state* st, int32_t batch, int32_t* topk_id, float* topk_logp,
                          void* hidden_out, void* ws, size_t ws_bytes, void* stream) {
  MOA_RANGE();
  MOA_TRY(check_state(ctx, st, batch));
  if (!topk_id || !topk_logp || !ws) return MOA_ERR_NULL;
  if (!aligned16(topk_id) || !aligned16(topk_logp) || !aligned16(hidden_out) || !aligned16(ws)) return MOA_ERR_ALIGN;
  if (st->step < 0 || st->step >= ctx->c.tree_depth) return MOA_ERR_STATE;
  const int chunk = chunk_from_bytes(ctx->c, ctx->tli, ctx->elt, ws_bytes);
  if (chunk < 1) return MOA_ERR_WORKSPACE;
  const Workspace p = plan_workspace(ctx->c, ctx->tli, ctx->elt, chunk);
  return ctx->c.dtype == MOA_F32
             ? draft_step_t<float>(ctx, st, batch, topk_id, topk_logp, hidden_out, (char*)ws, p, (cudaStream_t)stream)
             : draft_step_t<bf16>(ctx, st, batch, topk_id, topk_logp, hidden_out, (char*)ws, p, (cudaStream_t)stream);
}

moa_status moa_tree_expand(moa_ctx* ctx, moa_state* st, int32_t batch, const int32_t* topk_id, const float* topk_logp,
                           int32_t* out_tok, int32_t* out_parent, int32_t* out_depth, float* out_score, int32_t* out_n,
                           void* stream) {
  MOA_RANGE();
  MOA_TRY(check_state(ctx, st, batch));
  if (!topk_id || !topk_logp) return MOA_ERR_NULL;
  if (st->step < 0 || st->step >= ctx->c.tree_depth) return MOA_ERR_STATE;
  const int any = (out_tok != 0) + (out_parent != 0) + (out_depth != 0) + (out_score != 0);
  if (any != 0 && any != 4) return MOA_ERR_NULL;   // the four node arrays come together or not at all
  const moa_config& c = ctx->c;
  const TreeLayout& L = ctx->tl;
  const TreePtrs tp = tree_ptrs(st->tree, L);
  const int last = (st->step + 1 == c.tree_depth) ? 1 : 0;
  const size_t smem = ((size_t)(L.P > 256 ? L.P : 256) + L.P) * 4;
  launch_pdl(tree_expand_kernel, dim3(batch), dim3(512), smem, (cudaStream_t)stream, tp, c.tree_topk, c.tree_depth, L.P, c.tree_keep, st->step,
                                                                 batch, c.max_batch * c.tree_topk, topk_id, topk_logp,
                                                                 last, out_tok, out_parent, out_depth, out_score, out_n);
  MOA_CHECK_LAUNCH();
  st->step += 1;
  return MOA_OK;
}

moa_status moa_tree_attn_mask(const int32_t* parent, int32_t batch, int32_t n, void* mask_out, int32_t packed,
                              void* stream) {
  MOA_RANGE();
  if (!parent || !mask_out) return MOA_ERR_NULL;
  if (batch < 0 || n < 0 || (long long)batch * n > 0x3fffffff) return MOA_ERR_SHAPE;
  if (packed != 0 && packed != 1) return MOA_ERR_SHAPE;
  if (!aligned16(parent) || !aligned16(mask_out)) return MOA_ERR_ALIGN;
  const int total = batch * n;
  if (total == 0) return MOA_OK;
  tree_mask_kernel<<<(total + 127) / 128, 128, 0, (cudaStream_t)stream>>>(
      parent, batch, n, packed ? nullptr : (unsigned char*)mask_out, packed ? (unsigned long long*)mask_out : nullptr);
  MOA_CHECK_LAUNCH();
  return MOA_OK;
}

// ---------------------------------------------------------------------------------------------
// moa_sa_append_static: moa_sa_append with its scratch in a fixed device array of this library.
// ---------------------------------------------------------------------------------------------
enum : size_t { SA_STATIC_XN_BYTES = 512u * 1024u, SA_STATIC_PART_BYTES = 4u * 1024u * 1024u };
static __device__ __align__(256) unsigned char g_sa_static_scratch[SA_STATIC_XN_BYTES + SA_STATIC_PART_BYTES];
enum { SA_STATIC_MAX_DEVICES = 64 };
static void* g_sa_static_ptr[SA_STATIC_MAX_DEVICES];    // device address of the array on each device, 0 = not looked up
static std::mutex g_sa_static_mutex;

// Device address of the scratch array on the current device. The array's name is only a host-side handle
// of the symbol, so the address is asked for once per device, with that device current.
static moa_status sa_static_scratch(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess && (dev < 0 || dev >= SA_STATIC_MAX_DEVICES)) e = cudaErrorInvalidDevice;
  if (e == cudaSuccess) {
    std::lock_guard<std::mutex> lock(g_sa_static_mutex);
    if (!g_sa_static_ptr[dev]) {
      void* ptr = nullptr;
      e = cudaGetSymbolAddress((void**)&ptr, g_sa_static_scratch);
      if (e == cudaSuccess && ptr) g_sa_static_ptr[dev] = ptr;
    }
    *out = g_sa_static_ptr[dev];
  }
  if (e != cudaSuccess || !*out) {
    snprintf(g_cuda_err, sizeof(g_cuda_err), "moa_sa_append_static: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
    return MOA_ERR_CUDA;
  }
  return MOA_OK;
}

moa_status moa_sa_append_static(moa_ctx* ctx, moa_state* st, const int32_t* tok, const int32_t* n_host, int32_t batch,
                                void* stream) {
  MOA_RANGE();
  MOA_TRY(check_state(ctx, st, batch));
  if (!n_host) return MOA_ERR_NULL;
  SeqSplit split;
  MOA_TRY(make_split(n_host, batch, &split));
  const int total = split.off[batch];
  if (total > 0 && !tok) return MOA_ERR_NULL;
  for (int b = 0; b < batch; ++b)
    if ((long long)st->sa_len_host[b] + n_host[b] > ctx->c.max_ctx) return MOA_ERR_CAPACITY;
  const moa_config& c = ctx->c;
  const size_t kv_row_bytes = (size_t)2 * c.sa_hkv * c.head_dim * sizeof(float);
  const size_t xn_rows = (size_t)total + lo_rows_of(ctx->elt, total);     // bf16: a second, low-order term per row
  if (total > MOA_SA_STATIC_MAX_TOKENS || xn_rows * c.d_model * ctx->elt > SA_STATIC_XN_BYTES ||
      (size_t)total * kv_row_bytes > SA_STATIC_PART_BYTES) {
    snprintf(g_cuda_err, sizeof(g_cuda_err),
             "moa_sa_append_static: %d tokens of width %d exceed the fixed scratch (at most %d tokens, %zu bytes of "
             "normalised rows, %zu bytes of projected rows)",
             total, c.d_model, (int)MOA_SA_STATIC_MAX_TOKENS, (size_t)SA_STATIC_XN_BYTES, (size_t)SA_STATIC_PART_BYTES);
    return MOA_ERR_WORKSPACE;
  }
  void* scratch = nullptr;
  MOA_TRY(sa_static_scratch(&scratch));
  // the two regions moa_sa_append carves out of a caller workspace, laid over the fixed array instead
  Workspace p;
  memset(&p, 0, sizeof(p));
  p.xn = 0;
  p.part = SA_STATIC_XN_BYTES;
  p.rows_cap = MOA_SA_STATIC_MAX_TOKENS;                         // one pass
  p.part_rows = (int)(SA_STATIC_PART_BYTES / kv_row_bytes);      // bounds the K-split planes
  p.total = SA_STATIC_XN_BYTES + SA_STATIC_PART_BYTES;
  moa_status r = c.dtype == MOA_F32 ? sa_append_t<float>(ctx, st, tok, split, (char*)scratch, p, (cudaStream_t)stream)
                                    : sa_append_t<bf16>(ctx, st, tok, split, (char*)scratch, p, (cudaStream_t)stream);
  if (r == MOA_OK)
    for (int b = 0; b < batch; ++b) st->sa_len_host[b] += n_host[b];
  return r;
}

moa_status moa_verify_greedy(const int32_t* tok, const int32_t* parent, int32_t batch, int32_t n, const void* target_logits,
                             int32_t logits_dtype, int32_t vocab, int32_t cap, int32_t* choice, int32_t* acc_slot,
                             int32_t* acc_tok, int32_t* acc_len, int32_t* next_tok, void* stream) {
  MOA_RANGE();
  if (!tok || !parent || !target_logits || !choice || !acc_slot || !acc_tok || !acc_len || !next_tok) return MOA_ERR_NULL;
  if (batch <= 0 || batch > MOA_MAX_BATCH || n <= 0 || vocab <= 0 || cap <= 0) return MOA_ERR_SHAPE;
  if (logits_dtype != MOA_F32 && logits_dtype != MOA_BF16) return MOA_ERR_DTYPE;
  if ((long long)batch * n > 65535) return MOA_ERR_SHAPE;          // one cluster per row along gridDim.y
  cudaStream_t s = (cudaStream_t)stream;
  // few rows: a cluster of CTAs per row, so that the rows fill the GPU; many rows: one CTA per row
  static int sms_of[64];                 // SM count per device, asked for once (the entry point has no context)
  int sms = 148, dev = 0;
  if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64) {
    if (sms_of[dev] == 0) cudaDeviceGetAttribute(&sms_of[dev], cudaDevAttrMultiProcessorCount, dev);
    if (sms_of[dev] > 0) sms = sms_of[dev];
  }
  const int rows = batch * n;
  const bool spread = rows < 4 * sms;
  if (logits_dtype == MOA_F32) {
    if (spread) launch_pdl(argmax_rows_kernel<float, AM_CLUSTER>, dim3(AM_CLUSTER, rows), dim3(256), 0, s, (const float*)target_logits, vocab, choice);
    else launch_pdl(argmax_rows_kernel<float, 1>, dim3(1, rows), dim3(256), 0, s, (const float*)target_logits, vocab, choice);
  } else {
    if (spread) launch_pdl(argmax_rows_kernel<bf16, AM_CLUSTER>, dim3(AM_CLUSTER, rows), dim3(256), 0, s, (const bf16*)target_logits, vocab, choice);
    else launch_pdl(argmax_rows_kernel<bf16, 1>, dim3(1, rows), dim3(256), 0, s, (const bf16*)target_logits, vocab, choice);
  }
  MOA_CHECK_LAUNCH();
  launch_pdl(verify_walk_kernel, dim3((batch + 3) / 4), dim3(128), 0, s, tok, parent, (const int*)choice, batch, n, cap, acc_slot,
             acc_tok, acc_len, next_tok);
  MOA_CHECK_LAUNCH();
  return MOA_OK;
}

moa_status moa_pack_tree(const int32_t* tok, const int32_t* parent, int64_t count, void* msg, void* stream) {
  MOA_RANGE();
  if (!tok || !parent || !msg) return MOA_ERR_NULL;
  if (count < 0 || count > (1ll << 31)) return MOA_ERR_SHAPE;
  if ((uintptr_t)msg & 3u) return MOA_ERR_ALIGN;
  if (count == 0) return MOA_OK;
  launch_pdl(pack_tree_kernel, dim3(blocks_for((size_t)count, 256)), dim3(256), 0, (cudaStream_t)stream, tok, parent, (size_t)count,
             (uint32_t*)msg);
  MOA_CHECK_LAUNCH();
  return MOA_OK;
}

moa_status moa_unpack_tree(const void* msg, int64_t count, int32_t* tok, int32_t* parent, void* stream) {
  MOA_RANGE();
  if (!tok || !parent || !msg) return MOA_ERR_NULL;
  if (count < 0 || count > (1ll << 31)) return MOA_ERR_SHAPE;
  if ((uintptr_t)msg & 3u) return MOA_ERR_ALIGN;
  if (count == 0) return MOA_OK;
  launch_pdl(unpack_tree_kernel, dim3(blocks_for((size_t)count, 256)), dim3(256), 0, (cudaStream_t)stream, (const uint32_t*)msg,
             (size_t)count, tok, parent);
  MOA_CHECK_LAUNCH();
  return MOA_OK;
}

moa_status moa_quantize_rows(const void* x, int32_t dtype, int64_t rows, int32_t width, int8_t* codes, float* scales,
                             void* stream) {
  MOA_RANGE();
  if (!x || !codes || !scales) return MOA_ERR_NULL;
  if (dtype != MOA_F32 && dtype != MOA_BF16) return MOA_ERR_DTYPE;
  if (rows < 0 || width <= 0 || rows > (1ll << 31)) return MOA_ERR_SHAPE;
  if (rows == 0) return MOA_OK;
  const int per = dtype == MOA_F32 ? 4 : 8;
  const int vec = (width % per == 0 && aligned16(x) && ((uintptr_t)codes & 7u) == 0) ? 1 : 0;
  const unsigned grid = blocks_for((size_t)rows, 8);
  if (dtype == MOA_F32)
    launch_pdl(quantize_rows_kernel<float>, dim3(grid), dim3(256), 0, (cudaStream_t)stream, (const float*)x, (long long)rows, width, vec,
               codes, scales);
  else
    launch_pdl(quantize_rows_kernel<bf16>, dim3(grid), dim3(256), 0, (cudaStream_t)stream, (const bf16*)x, (long long)rows, width, vec,
               codes, scales);
  MOA_CHECK_LAUNCH();
  return MOA_OK;
}

moa_status moa_dequantize_rows(const int8_t* codes, const float* scales, int64_t rows, int32_t width, void* out, int32_t dtype,
                               void* stream) {
  MOA_RANGE();
  if (!out || !codes || !scales) return MOA_ERR_NULL;
  if (dtype != MOA_F32 && dtype != MOA_BF16) return MOA_ERR_DTYPE;
  if (rows < 0 || width <= 0 || rows > (1ll << 31)) return MOA_ERR_SHAPE;
  if (rows == 0) return MOA_OK;
  const int vec = (width % 16 == 0 && aligned16(codes) && aligned16(out)) ? 1 : 0;
  const size_t total = (size_t)rows * width;
  if ((vec ? total / 16 : total) > 256ull * 0x7fffffffull) return MOA_ERR_SHAPE;       // grid size
  const unsigned grid = blocks_for(vec ? total / 16 : total, 256);
  if (dtype == MOA_F32)
    launch_pdl(dequantize_rows_kernel<float>, dim3(grid), dim3(256), 0, (cudaStream_t)stream, codes, scales, (long long)rows, width, vec,
               (float*)out);
  else
    launch_pdl(dequantize_rows_kernel<bf16>, dim3(grid), dim3(256), 0, (cudaStream_t)stream, codes, scales, (long long)rows, width, vec,
               (bf16*)out);
  MOA_CHECK_LAUNCH();
  return MOA_OK;
}

moa_status moa_state_status(moa_ctx* ctx, moa_state* st, void* stream) {
  if (!ctx || !st || !st->tree) return MOA_ERR_NULL;
  int word = 0;
  cudaError_t e = cudaMemcpyAsync(&word, (char*)st->tree + ctx->tl.status, sizeof(int), cudaMemcpyDeviceToHost,
                                  (cudaStream_t)stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
  if (e != cudaSuccess) {
    snprintf(g_cuda_err, sizeof(g_cuda_err), "moa_state_status: %s", cudaGetErrorString(e));
    return MOA_ERR_CUDA;
  }
  return (moa_status)word;
}

}  // extern "C"
