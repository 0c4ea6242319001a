// C ABI of the Mixture-of-Attentions drafter hot path (see include/moa.h for the contract).
// Host-side validation and launch sequencing only; every step of the path runs in the kernels.
#include "../../include/moa.h"

#include <stdio.h>
#include <string.h>
#include <new>

#include "moa_basic.cuh"
#include "moa_tree.cuh"

using namespace moa;

static thread_local char g_cuda_err[256] = "";
static thread_local long long g_launches = 0;

enum { PROF_MAX = 512 };

struct moa_ctx {
  moa_config c;
  moa_weights w;
  int sm_count;
  size_t elt;          // bytes per T
  TreeLayout tl;
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
  size_t xres, xn, wide, narrow, obuf, logits, kvf, kvn, total;
  int rows_cap, draft_rows, chunk_tok;
};

static inline int imax(int a, int b) { return a > b ? a : b; }

static Workspace plan_workspace(const moa_config& c, size_t elt, int chunk_tok) {
  Workspace p;
  p.chunk_tok = chunk_tok;
  p.draft_rows = c.max_batch * c.tree_topk;
  p.rows_cap = imax(p.draft_rows, chunk_tok * c.n_stack);
  const int dmax = imax(c.d_model, c.d_stack);
  const int qkv_lsa = (c.lsa_hq + 2 * c.lsa_hkv) * c.head_dim;
  const int qkv_sa = (c.sa_hq + 2 * c.sa_hkv) * c.head_dim;
  const int q_ca = imax(c.ca_hq * c.head_dim, 2 * c.ca_hkv * c.head_dim);
  const int fmax = imax(c.lsa_mlp, imax(c.sa_mlp, c.ca_mlp));
  const int wide = imax(imax(qkv_lsa, qkv_sa), imax(q_ca, 2 * fmax));
  const int narrow = imax(imax(qkv_lsa, qkv_sa), imax(q_ca, fmax));
  const int omax = imax(c.lsa_hq, imax(c.sa_hq, c.ca_hq)) * c.head_dim;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o += (bytes + 255) / 256 * 256; return at; };
  p.xres = take((size_t)p.rows_cap * dmax * sizeof(float));     // residual stream, fp32
  p.xn = take((size_t)p.rows_cap * dmax * elt);                 // normalised GEMM operand, T
  p.wide = take((size_t)p.rows_cap * wide * sizeof(float));     // q, k, v or gate, up: fp32
  p.narrow = take((size_t)p.rows_cap * narrow * elt);           // q, k, v or silu(gate)*up: T
  p.obuf = take((size_t)p.rows_cap * omax * elt);               // attention output, T
  p.logits = take((size_t)p.draft_rows * c.vocab * sizeof(float));
  p.kvf = take((size_t)chunk_tok * c.d_stack * sizeof(float));  // LSA output rows, fp32
  p.kvn = take((size_t)chunk_tok * c.d_stack * elt);            // their normalised copy, T
  p.total = o;
  return p;
}

// Largest token chunk whose plan fits in ws_bytes (plan size is monotone in the chunk); 0 if none.
static int chunk_from_bytes(const moa_config& c, size_t elt, size_t ws_bytes) {
  if (plan_workspace(c, elt, 1).total > ws_bytes) return 0;
  int lo = 1;
  while (lo < (1 << 20) && plan_workspace(c, elt, lo * 2).total <= ws_bytes) lo *= 2;
  int hi = lo * 2;
  while (lo + 1 < hi) {
    const int mid = lo + (hi - lo) / 2;
    if (plan_workspace(c, elt, mid).total <= ws_bytes) lo = mid; else hi = mid;
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

template <typename T>
static moa_status gemm(cudaStream_t s, const T* A, const void* W, int R, int N, int K, const float* res, int ldr,
                       float* C, int ldc) {
  if (R <= 0 || N <= 0) return MOA_OK;
  dim3 grid((N + 63) / 64, (R + 63) / 64);
  gemm_fma_kernel<T><<<grid, 256, 0, s>>>(A, (const T*)W, R, N, K, res, ldr, C, ldc);
  MOA_CHECK_LAUNCH();
  return MOA_OK;
}

template <typename T>
static moa_status attention(cudaStream_t s, int dh, const T* q, int R, int hq, int hkv, const T* kA, const T* vA,
                            int capA, const int* lenA, int nA_fixed, const T* kB, const T* vB, int capB,
                            const int* slotsB, int slots_ld, int nB, int rows_per_seq, T* out) {
  if (R <= 0) return MOA_OK;
  dim3 grid(R, hq);
  if (dh == 128)
    attn_rows_kernel<T, 128><<<grid, 128, 0, s>>>(q, hq, hkv, kA, vA, capA, lenA, nA_fixed, kB, vB, capB, slotsB,
                                                  slots_ld, nB, rows_per_seq, out);
  else
    attn_rows_kernel<T, 64><<<grid, 128, 0, s>>>(q, hq, hkv, kA, vA, capA, lenA, nA_fixed, kB, vB, capB, slotsB,
                                                 slots_ld, nB, rows_per_seq, out);
  MOA_CHECK_LAUNCH();
  return MOA_OK;
}

template <typename T>
static moa_status cast_flat(cudaStream_t s, const float* x, T* y, size_t total) {
  if (total == 0) return MOA_OK;
  cast_flat_kernel<T><<<(unsigned)((total + 255) / 256), 256, 0, s>>>(x, y, total);
  MOA_CHECK_LAUNCH();
  return MOA_OK;
}

// MLP with residual: xres += W_down (silu(W_gate n) * (W_up n)), n = RMSNorm(xres; gain)
template <typename T>
static moa_status mlp_block(cudaStream_t s, const moa_ctx* ctx, const Workspace& p, char* ws, int R, int K, int F,
                            const void* gain, const void* wgate, const void* wup, const void* wdown) {
  float* xres = (float*)(ws + p.xres);
  T* xn = (T*)(ws + p.xn);
  float* gate = (float*)(ws + p.wide);
  float* up = gate + (size_t)R * F;
  T* h = (T*)(ws + p.narrow);
  rmsnorm_rows_kernel<float, T><<<R, 256, 0, s>>>(xres, nullptr, 0, (const T*)gain, K, ctx->c.rms_eps, nullptr, xn);
  MOA_CHECK_LAUNCH();
  MOA_TRY(gemm<T>(s, xn, wgate, R, F, K, nullptr, 0, gate, F));
  MOA_TRY(gemm<T>(s, xn, wup, R, F, K, nullptr, 0, up, F));
  const size_t total = (size_t)R * F;
  silu_mul_kernel<T><<<(unsigned)((total + 255) / 256), 256, 0, s>>>(gate, up, F, F, h, total);
  MOA_CHECK_LAUNCH();
  return gemm<T>(s, h, wdown, R, K, F, xres, K, xres, K);
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
  const int nq = c.lsa_hq * dh, nkv = c.lsa_hkv * dh;
  float* xres = (float*)(ws + p.xres);
  T* xn = (T*)(ws + p.xn);
  float* wide = (float*)(ws + p.wide);
  T* narrow = (T*)(ws + p.narrow);
  T* obuf = (T*)(ws + p.obuf);
  float* kvf = (float*)(ws + p.kvf);
  T* kvn = (T*)(ws + p.kvn);
  const int total = split.off[split.n_seq];
  for (int t0 = 0; t0 < total; t0 += p.chunk_tok) {
    const int nt = (total - t0) < p.chunk_tok ? (total - t0) : p.chunk_tok;
    const int R = nt * S;
    const T* x = (const T*)h_stack + (size_t)t0 * S * D;
    // pre-norm and q, k, v projections of every (token, layer) row; three dense fp32 blocks
    rmsnorm_rows_kernel<T, T><<<R, 256, 0, s>>>(x, nullptr, 0, (const T*)w.lsa_norm1, D, c.rms_eps, xres, xn);
    MOA_CHECK_LAUNCH();
    float* qf = wide;
    float* kf = qf + (size_t)R * nq;
    float* vf = kf + (size_t)R * nkv;
    MOA_TRY(gemm<T>(s, xn, w.lsa_wq, R, nq, D, nullptr, 0, qf, nq));
    MOA_TRY(gemm<T>(s, xn, w.lsa_wk, R, nkv, D, nullptr, 0, kf, nkv));
    MOA_TRY(gemm<T>(s, xn, w.lsa_wv, R, nkv, D, nullptr, 0, vf, nkv));
    MOA_TRY(cast_flat<T>(s, wide, narrow, (size_t)R * (nq + 2 * nkv)));
    const T* qd = narrow;
    const T* kd = qd + (size_t)R * nq;
    const T* vd = kd + (size_t)R * nkv;
    // attention over the S layer rows of the same token (full mask): "sequence" = token, cap = S
    MOA_TRY(attention<T>(s, dh, qd, R, c.lsa_hq, c.lsa_hkv, kd, vd, S, nullptr, S, nullptr, nullptr, 0, nullptr, 0, 0,
                         S, obuf));
    // out-projection + residual, MLP + residual
    MOA_TRY(gemm<T>(s, obuf, w.lsa_wo, R, D, nq, xres, D, xres, D));
    MOA_TRY(mlp_block<T>(s, ctx, p, ws, R, D, c.lsa_mlp, w.lsa_norm2, w.lsa_wgate, w.lsa_wup, w.lsa_wdown));
    // mean over layers
    T* kvo = kv_out ? (T*)kv_out + (size_t)t0 * D : nullptr;
    mean_layers_kernel<T><<<nt, 256, 0, s>>>(xres, S, D, kvf, kvo);
    MOA_CHECK_LAUNCH();
    // cross-attention keys / values of the new positions, appended to the cache
    rmsnorm_rows_kernel<float, T><<<nt, 256, 0, s>>>(kvf, nullptr, 0, (const T*)w.ca_normkv, D, c.rms_eps, nullptr, kvn);
    MOA_CHECK_LAUNCH();
    const int ckv = c.ca_hkv * dh;
    float* ckf = wide;
    float* cvf = ckf + (size_t)nt * ckv;
    MOA_TRY(gemm<T>(s, kvn, w.ca_wk, nt, ckv, D, nullptr, 0, ckf, ckv));
    MOA_TRY(gemm<T>(s, kvn, w.ca_wv, nt, ckv, D, nullptr, 0, cvf, ckv));
    cache_append_kernel<T><<<nt, 256, 0, s>>>(ckf, ckv, 0, nt * ckv, ckv, st->ca_len, c.max_ctx, split, t0,
                                              (T*)st->ca_k, (T*)st->ca_v);
    MOA_CHECK_LAUNCH();
  }
  add_len_kernel<<<1, 64, 0, s>>>(st->ca_len, split);
  MOA_CHECK_LAUNCH();
  return MOA_OK;
}

template <typename T>
static moa_status sa_append_t(moa_ctx* ctx, moa_state* st, const int* tok, const SeqSplit& split, char* ws,
                              const Workspace& p, cudaStream_t s) {
  const moa_config& c = ctx->c;
  const moa_weights& w = ctx->w;
  const int E = c.d_model, dh = c.head_dim, nkv = c.sa_hkv * dh;
  T* xn = (T*)(ws + p.xn);
  float* wide = (float*)(ws + p.wide);
  const int total = split.off[split.n_seq];
  for (int t0 = 0; t0 < total; t0 += p.rows_cap) {
    const int R = (total - t0) < p.rows_cap ? (total - t0) : p.rows_cap;
    rmsnorm_rows_kernel<T, T><<<R, 256, 0, s>>>((const T*)w.embed, tok + t0, c.vocab, (const T*)w.sa_norm1, E,
                                                c.rms_eps, nullptr, xn);
    MOA_CHECK_LAUNCH();
    float* kf = wide;
    float* vf = kf + (size_t)R * nkv;
    MOA_TRY(gemm<T>(s, xn, w.sa_wk, R, nkv, E, nullptr, 0, kf, nkv));
    MOA_TRY(gemm<T>(s, xn, w.sa_wv, R, nkv, E, nullptr, 0, vf, nkv));
    RopeRows rr;
    memset(&rr, 0, sizeof(rr));
    rr.mode = 1;
    rr.max_ctx = c.max_ctx;
    rr.split = split;
    rr.row0 = t0;
    // k and v rows are dense [R, nkv] blocks: leading dimension nkv, v block R*nkv elements after k
    rope_store_kernel<T><<<R, 128, 0, s>>>(kf, nkv, 0, 0, R * nkv, 0, c.sa_hkv, dh, c.sa_rope_theta, st->sa_len, rr,
                                           (T*)nullptr, (T*)st->sa_k, (T*)st->sa_v);
    MOA_CHECK_LAUNCH();
  }
  add_len_kernel<<<1, 64, 0, s>>>(st->sa_len, split);
  MOA_CHECK_LAUNCH();
  return MOA_OK;
}

template <typename T>
static moa_status draft_step_t(moa_ctx* ctx, moa_state* st, int batch, int* topk_id, float* topk_logp,
                               void* hidden_out, char* ws, const Workspace& p, cudaStream_t s) {
  const moa_config& c = ctx->c;
  const moa_weights& w = ctx->w;
  const TreeLayout& L = ctx->tl;
  const TreePtrs tp = tree_ptrs(st->tree, L);
  const int step = st->step, B = c.tree_topk, D = c.tree_depth;
  const int R = step == 0 ? batch : batch * B;
  const int rows_per_seq = step == 0 ? 1 : B;
  const int nbB = c.max_batch * B;
  const int E = c.d_model, dh = c.head_dim, V = c.vocab;
  const int cur = step & 1;
  const int* row_tok = tp.row_tok + (size_t)cur * nbB;
  const int* row_anc = tp.row_anc + (size_t)cur * nbB * D;
  T* tk = (T*)((char*)st->tree + L.tk);
  T* tv = (T*)((char*)st->tree + L.tv);
  float* xres = (float*)(ws + p.xres);
  T* xn = (T*)(ws + p.xn);
  float* wide = (float*)(ws + p.wide);
  T* narrow = (T*)(ws + p.narrow);
  T* obuf = (T*)(ws + p.obuf);
  float* logits = (float*)(ws + p.logits);

  // ---- self-attention block ----
  rmsnorm_rows_kernel<T, T><<<R, 256, 0, s>>>((const T*)w.embed, row_tok, V, (const T*)w.sa_norm1, E, c.rms_eps, xres, xn);
  MOA_CHECK_LAUNCH();
  const int nq = c.sa_hq * dh, nkv = c.sa_hkv * dh;
  float* qf = wide;
  float* kf = qf + (size_t)R * nq;
  float* vf = kf + (size_t)R * nkv;
  MOA_TRY(gemm<T>(s, xn, w.sa_wq, R, nq, E, nullptr, 0, qf, nq));
  MOA_TRY(gemm<T>(s, xn, w.sa_wk, R, nkv, E, nullptr, 0, kf, nkv));
  MOA_TRY(gemm<T>(s, xn, w.sa_wv, R, nkv, E, nullptr, 0, vf, nkv));
  RopeRows rr;
  memset(&rr, 0, sizeof(rr));
  rr.mode = 0;
  rr.step = step;
  rr.B = B;
  rr.slots = L.NS;
  // q, k, v blocks have different leading dimensions; the kernel indexes a row as base + r*ld + off, so
  // it is launched once for q (+ a k/v pass that writes nothing is avoided by giving hkv = 0) and once for k, v.
  rope_store_kernel<T><<<R, 128, 0, s>>>(qf, nq, 0, 0, 0, c.sa_hq, 0, dh, c.sa_rope_theta, st->sa_len, rr, narrow,
                                         (T*)nullptr, (T*)nullptr);
  MOA_CHECK_LAUNCH();
  rope_store_kernel<T><<<R, 128, 0, s>>>(kf, nkv, 0, 0, R * nkv, 0, c.sa_hkv, dh, c.sa_rope_theta, st->sa_len, rr,
                                         (T*)nullptr, tk, tv);
  MOA_CHECK_LAUNCH();
  MOA_TRY(attention<T>(s, dh, narrow, R, c.sa_hq, c.sa_hkv, (const T*)st->sa_k, (const T*)st->sa_v, c.max_ctx,
                       st->sa_len, 0, tk, tv, L.NS, row_anc, D, step + 1, rows_per_seq, obuf));
  MOA_TRY(gemm<T>(s, obuf, w.sa_wo, R, E, nq, xres, E, xres, E));
  MOA_TRY(mlp_block<T>(s, ctx, p, ws, R, E, c.sa_mlp, w.sa_norm2, w.sa_wgate, w.sa_wup, w.sa_wdown));

  // ---- cross-attention block ----
  const int cq = c.ca_hq * dh;
  rmsnorm_rows_kernel<float, T><<<R, 256, 0, s>>>(xres, nullptr, 0, (const T*)w.ca_normq, E, c.rms_eps, nullptr, xn);
  MOA_CHECK_LAUNCH();
  MOA_TRY(gemm<T>(s, xn, w.ca_wq, R, cq, E, nullptr, 0, wide, cq));
  MOA_TRY(cast_flat<T>(s, wide, narrow, (size_t)R * cq));
  MOA_TRY(attention<T>(s, dh, narrow, R, c.ca_hq, c.ca_hkv, (const T*)st->ca_k, (const T*)st->ca_v, c.max_ctx,
                       st->ca_len, 0, nullptr, nullptr, 0, nullptr, 0, 0, rows_per_seq, obuf));
  MOA_TRY(gemm<T>(s, obuf, w.ca_wo, R, E, cq, xres, E, xres, E));
  MOA_TRY(mlp_block<T>(s, ctx, p, ws, R, E, c.ca_mlp, w.ca_norm2, w.ca_wgate, w.ca_wup, w.ca_wdown));

  // ---- LM head, log-softmax, top-B ----
  if (hidden_out) MOA_TRY(cast_flat<T>(s, xres, (T*)hidden_out, (size_t)R * E));
  rmsnorm_rows_kernel<float, T><<<R, 256, 0, s>>>(xres, nullptr, 0, (const T*)w.final_norm, E, c.rms_eps, nullptr, xn);
  MOA_CHECK_LAUNCH();
  const bool timed = ctx->prof_on && ctx->prof_n < PROF_MAX;
  if (timed) cudaEventRecord(ctx->prof_ev[2 * ctx->prof_n], s);
  MOA_TRY(gemm<T>(s, xn, w.lm_head, R, V, E, nullptr, 0, logits, V));
  if (timed) cudaEventRecord(ctx->prof_ev[2 * ctx->prof_n++ + 1], s);
  lse_topk_rows_kernel<<<R, 256, 0, s>>>(logits, V, B, topk_id, topk_logp);
  MOA_CHECK_LAUNCH();
  return MOA_OK;
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
  if (c->n_stack <= 0 || c->vocab <= 0) return MOA_ERR_SHAPE;
  const int hq[] = {c->lsa_hq, c->sa_hq, c->ca_hq}, hkv[] = {c->lsa_hkv, c->sa_hkv, c->ca_hkv};
  for (int i = 0; i < 3; ++i)
    if (hq[i] <= 0 || hkv[i] <= 0 || hq[i] % hkv[i] != 0) return MOA_ERR_SHAPE;
  if (c->max_batch <= 0 || c->max_batch > MOA_MAX_BATCH) return MOA_ERR_SHAPE;
  if (c->max_ctx <= 0) return MOA_ERR_SHAPE;
  if (c->tree_topk <= 0 || c->tree_topk > MOA_MAX_TOPK || c->tree_topk > c->vocab) return MOA_ERR_SHAPE;
  if (c->tree_depth <= 0 || c->tree_depth > MOA_MAX_DEPTH) return MOA_ERR_SHAPE;
  if (c->tree_keep <= 0) return MOA_ERR_SHAPE;
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
  *out = ctx;
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

moa_status moa_state_bytes(const moa_ctx* ctx, int32_t lsa_chunk_tokens, size_t* tree_bytes, size_t* workspace_bytes) {
  if (!ctx) return MOA_ERR_NULL;
  if (lsa_chunk_tokens < 1) return MOA_ERR_SHAPE;
  if (tree_bytes) *tree_bytes = ctx->tl.total;
  if (workspace_bytes) *workspace_bytes = plan_workspace(ctx->c, ctx->elt, lsa_chunk_tokens).total;
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
  MOA_TRY(check_state(ctx, st, batch));
  if (!n_tok_host || !ws) return MOA_ERR_NULL;
  SeqSplit split;
  MOA_TRY(make_split(n_tok_host, batch, &split));
  const int total = split.off[batch];
  if (total > 0 && !h_stack) return MOA_ERR_NULL;
  if (!aligned16(h_stack) || !aligned16(kv_out) || !aligned16(ws)) return MOA_ERR_ALIGN;
  for (int b = 0; b < batch; ++b)
    if ((long long)st->ca_len_host[b] + n_tok_host[b] > ctx->c.max_ctx) return MOA_ERR_CAPACITY;
  const int chunk = chunk_from_bytes(ctx->c, ctx->elt, ws_bytes);
  if (chunk < 1) return MOA_ERR_WORKSPACE;
  const Workspace p = plan_workspace(ctx->c, ctx->elt, chunk);
  moa_status r = ctx->c.dtype == MOA_F32
                     ? lsa_forward_t<float>(ctx, st, h_stack, split, kv_out, (char*)ws, p, (cudaStream_t)stream)
                     : lsa_forward_t<bf16>(ctx, st, h_stack, split, kv_out, (char*)ws, p, (cudaStream_t)stream);
  if (r == MOA_OK)
    for (int b = 0; b < batch; ++b) st->ca_len_host[b] += n_tok_host[b];
  return r;
}

moa_status moa_sa_append(moa_ctx* ctx, moa_state* st, const int32_t* tok, const int32_t* n_host, int32_t batch, void* ws,
                         size_t ws_bytes, void* stream) {
  MOA_TRY(check_state(ctx, st, batch));
  if (!n_host || !ws) return MOA_ERR_NULL;
  SeqSplit split;
  MOA_TRY(make_split(n_host, batch, &split));
  if (split.off[batch] > 0 && !tok) return MOA_ERR_NULL;
  if (!aligned16(ws)) return MOA_ERR_ALIGN;
  for (int b = 0; b < batch; ++b)
    if ((long long)st->sa_len_host[b] + n_host[b] > ctx->c.max_ctx) return MOA_ERR_CAPACITY;
  const int chunk = chunk_from_bytes(ctx->c, ctx->elt, ws_bytes);
  if (chunk < 1) return MOA_ERR_WORKSPACE;
  const Workspace p = plan_workspace(ctx->c, ctx->elt, chunk);
  moa_status r = ctx->c.dtype == MOA_F32 ? sa_append_t<float>(ctx, st, tok, split, (char*)ws, p, (cudaStream_t)stream)
                                         : sa_append_t<bf16>(ctx, st, tok, split, (char*)ws, p, (cudaStream_t)stream);
  if (r == MOA_OK)
    for (int b = 0; b < batch; ++b) st->sa_len_host[b] += n_host[b];
  return r;
}

moa_status moa_tree_begin(moa_ctx* ctx, moa_state* st, const int32_t* root_tok, int32_t batch, void* stream) {
  MOA_TRY(check_state(ctx, st, batch));
  if (!root_tok) return MOA_ERR_NULL;
  for (int b = 0; b < batch; ++b)   // the deepest forwarded row sits at sa_len + D - 1; positions are not stored
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
  MOA_TRY(check_state(ctx, st, batch));
  if (!topk_id || !topk_logp || !ws) return MOA_ERR_NULL;
  if (!aligned16(topk_id) || !aligned16(topk_logp) || !aligned16(hidden_out) || !aligned16(ws)) return MOA_ERR_ALIGN;
  if (st->step < 0 || st->step >= ctx->c.tree_depth) return MOA_ERR_STATE;
  const int chunk = chunk_from_bytes(ctx->c, ctx->elt, ws_bytes);
  if (chunk < 1) return MOA_ERR_WORKSPACE;
  const Workspace p = plan_workspace(ctx->c, ctx->elt, chunk);
  return ctx->c.dtype == MOA_F32
             ? draft_step_t<float>(ctx, st, batch, topk_id, topk_logp, hidden_out, (char*)ws, p, (cudaStream_t)stream)
             : draft_step_t<bf16>(ctx, st, batch, topk_id, topk_logp, hidden_out, (char*)ws, p, (cudaStream_t)stream);
}

moa_status moa_tree_expand(moa_ctx* ctx, moa_state* st, int32_t batch, const int32_t* topk_id, const float* topk_logp,
                           int32_t* out_tok, int32_t* out_parent, int32_t* out_depth, float* out_score, int32_t* out_n,
                           void* stream) {
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
  tree_expand_kernel<<<batch, 512, smem, (cudaStream_t)stream>>>(tp, c.tree_topk, c.tree_depth, L.P, c.tree_keep, st->step,
                                                                 batch, c.max_batch * c.tree_topk, topk_id, topk_logp,
                                                                 last, out_tok, out_parent, out_depth, out_score, out_n);
  MOA_CHECK_LAUNCH();
  st->step += 1;
  return MOA_OK;
}

moa_status moa_tree_attn_mask(const int32_t* parent, int32_t batch, int32_t n, void* mask_out, int32_t packed,
                              void* stream) {
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
