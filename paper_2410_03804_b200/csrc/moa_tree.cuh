// Dynamic draft tree (EAGLE-2 style, Section 2.2 of the paper): node pool, frontier selection,
// final top-m cut and the ancestor mask. Integer work plus fp32 score adds and compares; every
// choice orders by (score descending, pool index ascending) so results are unique.
#pragma once
#include "moa_common.cuh"

namespace moa {

constexpr int TREE_STATUS_WORDS = 8;      // status word, barrier words of the fused kernels
constexpr int TREE_ROW_COUNTERS = 256;    // per draft-row arrival counters of the LM-head merge (zero between launches)

// Byte offsets inside the caller-owned tree blob.
struct TreeLayout {
  int nb, B, D, P, NS;     // sequences, breadth, depth, pool size per sequence, tree K/V slots per sequence
  size_t status;           // int[8 + 256]: [0] status word, [4..6] grid-barrier counter, abort word, exit counter,
                           // [8..] the LM-head merge's per-row arrival counters
  size_t flags;            // int[256 * 32]: per-CTA grid-barrier flags of the fused kernels, one 128-byte line each
  size_t root_tok;         // int[nb]
  size_t frontier;         // int[nb*B]        pool index of each frontier node (-1: the root)
  size_t row_tok;          // int[2][nb*B]     token of each row, double-buffered by step parity
  size_t row_anc;          // int[2][nb*B*D]   tree K/V slots of a row's ancestors and, last, itself
  size_t pool_tok, pool_parent, pool_depth;   // int[nb*P]
  size_t pool_score;       // float[nb*P]
  size_t tk, tv;           // T[nb][NS][hkv][dh]
  int n_tli;               // decoder layers of the LLM run on the drafted rows (Section 3.2), 0..4
  size_t tli_tk[4], tli_tv[4];   // per such layer T[nb][NS][tli_hkv][dh]: the drafted rows' keys / values in it
  size_t total;
};

__host__ inline TreeLayout make_tree_layout(int nb, int B, int D, int hkv, int dh, size_t elt, int n_tli = 0,
                                            int tli_hkv = 0) {
  TreeLayout L;
  L.nb = nb; L.B = B; L.D = D;
  L.P = B + (D - 1) * B * B;
  L.NS = 1 + B * (D - 1);
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o += (bytes + 255) / 256 * 256; return at; };
  L.status = take((TREE_STATUS_WORDS + TREE_ROW_COUNTERS) * sizeof(int));
  L.flags = take((size_t)256 * 32 * sizeof(int));
  L.root_tok = take((size_t)nb * sizeof(int));
  L.frontier = take((size_t)nb * B * sizeof(int));
  L.row_tok = take((size_t)2 * nb * B * sizeof(int));
  L.row_anc = take((size_t)2 * nb * B * D * sizeof(int));
  L.pool_tok = take((size_t)nb * L.P * sizeof(int));
  L.pool_parent = take((size_t)nb * L.P * sizeof(int));
  L.pool_depth = take((size_t)nb * L.P * sizeof(int));
  L.pool_score = take((size_t)nb * L.P * sizeof(float));
  L.tk = take((size_t)nb * L.NS * hkv * dh * elt);
  L.tv = take((size_t)nb * L.NS * hkv * dh * elt);
  L.n_tli = n_tli;
  for (int l = 0; l < 4; ++l) {
    L.tli_tk[l] = L.tli_tv[l] = 0;
    if (l < n_tli) {
      L.tli_tk[l] = take((size_t)nb * L.NS * tli_hkv * dh * elt);
      L.tli_tv[l] = take((size_t)nb * L.NS * tli_hkv * dh * elt);
    }
  }
  L.total = o;
  return L;
}

struct TreePtrs {
  int *status, *root_tok, *frontier, *row_tok, *row_anc, *pool_tok, *pool_parent, *pool_depth;
  float* pool_score;
};
__host__ inline TreePtrs tree_ptrs(void* blob, const TreeLayout& L) {
  char* p = (char*)blob;
  TreePtrs t;
  t.status = (int*)(p + L.status);
  t.root_tok = (int*)(p + L.root_tok);
  t.frontier = (int*)(p + L.frontier);
  t.row_tok = (int*)(p + L.row_tok);
  t.row_anc = (int*)(p + L.row_anc);
  t.pool_tok = (int*)(p + L.pool_tok);
  t.pool_parent = (int*)(p + L.pool_parent);
  t.pool_depth = (int*)(p + L.pool_depth);
  t.pool_score = (float*)(p + L.pool_score);
  return t;
}

// Root of each sequence: row b of step 0 carries the root token and sees tree slot 0 (itself).
__global__ void tree_begin_kernel(TreePtrs t, const int* __restrict__ root_tok, int batch, int nbB, int D) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b == 0) t.status[0] = DEV_OK;
  if (b >= batch) return;
  t.root_tok[b] = root_tok[b];
  t.row_tok[b] = root_tok[b];          // buffer 0, row b
  t.row_anc[(size_t)b * D + 0] = 0;    // buffer 0
}

__device__ __forceinline__ bool score_before(float sa, int ia, float sb, int ib) {
  return sa > sb || (sa == sb && ia < ib);
}

// One block per sequence. step = number of expansions done before this one.
// Rows of this step: R_seq = 1 (step 0) or B. Children: C = R_seq * B, appended at pool index
// base + r*B + j with base = 0 (step 0) or B + (step-1)*B*B.
// When last != 0 the final cut (top m of the pool, listed by pool index behind the root) is written.
__global__ void __launch_bounds__(512) tree_expand_kernel(TreePtrs t, int B, int D, int P, int m, int step, int batch,
                                                          int nbB, const int* __restrict__ topk_id,
                                                          const float* __restrict__ topk_logp, int last,
                                                          int* __restrict__ out_tok, int* __restrict__ out_parent,
                                                          int* __restrict__ out_depth, float* __restrict__ out_score,
                                                          int* __restrict__ out_n) {
  pdl_trigger();
  pdl_wait(KID_EXPAND);
  extern __shared__ unsigned char smem_raw[];
  float* c_score = (float*)smem_raw;                 // [max(C, P)]
  int* c_aux = (int*)(c_score + (P > 256 ? P : 256)); // [P] kept flags / slots
  const int b = blockIdx.x;
  const int tid = threadIdx.x;
  const int Rs = step == 0 ? 1 : B;
  const int C = Rs * B;
  const int base = step == 0 ? 0 : B + (step - 1) * B * B;
  const int cur = step & 1, nxt = cur ^ 1;
  int* pool_tok = t.pool_tok + (size_t)b * P;
  int* pool_parent = t.pool_parent + (size_t)b * P;
  int* pool_depth = t.pool_depth + (size_t)b * P;
  float* pool_score = t.pool_score + (size_t)b * P;
  int* frontier = t.frontier + (size_t)b * B;
  const int row0 = step == 0 ? b : b * B;            // first row of this sequence in the [R, B] inputs
  if (base + C > P) {                                 // cannot happen when the host counted steps right
    if (tid == 0) atomicMax(t.status, DEV_ERR_BOUNDS);
    return;
  }
  // 1. children: score and pool append
  for (int c = tid; c < C; c += blockDim.x) {
    const int r = c / B, j = c - r * B;
    int par = step == 0 ? -1 : frontier[r];
    if (step > 0 && (unsigned)par >= (unsigned)P) {     // a frontier entry is a pool index by construction
      atomicMax(t.status, DEV_ERR_BOUNDS);
      par = 0;
    }
    const float ps = step == 0 ? 0.f : pool_score[par];
    float s = ps + topk_logp[(size_t)(row0 + r) * B + j];
    // The ranks below are a permutation only under a total order, and a NaN compares false with everything: a
    // log-probability that is not a number (a fault upstream) ranks last and is reported, instead of leaving
    // frontier entries unwritten.
    if (s != s) {
      atomicMax(t.status, DEV_ERR_NONFINITE);
      s = -INFINITY;
    }
    c_score[c] = s;
    pool_tok[base + c] = topk_id[(size_t)(row0 + r) * B + j];
    pool_parent[base + c] = par;
    pool_depth[base + c] = step + 1;
    pool_score[base + c] = s;
  }
  __syncthreads();
  // 2. next frontier: rank of each child among the children
  const int* anc_cur = t.row_anc + ((size_t)cur * nbB + row0) * D;
  int* anc_nxt = t.row_anc + ((size_t)nxt * nbB + (size_t)b * B) * D;
  int* tok_nxt = t.row_tok + (size_t)nxt * nbB + (size_t)b * B;
  for (int c = tid; c < C; c += blockDim.x) {
    const float s = c_score[c];
    int rank = 0;
    for (int o = 0; o < C; ++o) rank += score_before(c_score[o], o, s, c) ? 1 : 0;
    if (rank < B) {
      const int r = c / B;
      // the new row `rank` is child c of old row r: ancestors = r's ancestors (incl. r) + own slot
      for (int d = 0; d <= step; ++d) anc_nxt[(size_t)rank * D + d] = anc_cur[(size_t)r * D + d];
      if (step + 1 < D) anc_nxt[(size_t)rank * D + step + 1] = 1 + step * B + rank;
      tok_nxt[rank] = pool_tok[base + c];
      c_aux[rank] = base + c;
    }
  }
  __syncthreads();
  // the frontier array is read above (parents), so it is replaced only after every thread is done
  for (int i = tid; i < B; i += blockDim.x) frontier[i] = c_aux[i];
  if (!last) return;
  __syncthreads();
  // 3. final cut: rank of every pool node; kept = rank < m; slot = 1 + number of kept nodes before it
  const int n_pool = base + C;
  for (int i = tid; i < n_pool; i += blockDim.x) c_score[i] = pool_score[i];
  __syncthreads();
  for (int i = tid; i < n_pool; i += blockDim.x) {
    const float s = c_score[i];
    int rank = 0;
    for (int o = 0; o < n_pool; ++o) rank += score_before(c_score[o], o, s, i) ? 1 : 0;
    c_aux[i] = rank < m ? 1 : 0;
  }
  __syncthreads();
  if (tid == 0) {                                    // exclusive scan of the kept flags (<= a few hundred)
    int run = 0;
    for (int i = 0; i < n_pool; ++i) {
      const int k = c_aux[i];
      c_aux[i] = k ? (1 + run) : 0;                  // slot number, 0 = dropped
      run += k;
    }
    if (out_n) out_n[b] = 1 + run;
  }
  __syncthreads();
  if (!out_tok) return;
  const int W = m + 1;
  for (int s = tid; s < W; s += blockDim.x) {        // defaults, then the root
    out_tok[(size_t)b * W + s] = s == 0 ? t.root_tok[b] : -1;
    out_parent[(size_t)b * W + s] = -1;
    out_depth[(size_t)b * W + s] = s == 0 ? 0 : -1;
    out_score[(size_t)b * W + s] = 0.f;
  }
  __syncthreads();
  for (int i = tid; i < n_pool; i += blockDim.x) {
    const int s = c_aux[i];
    if (s == 0) continue;
    const int par = pool_parent[i];
    out_tok[(size_t)b * W + s] = pool_tok[i];
    out_parent[(size_t)b * W + s] = par < 0 ? 0 : c_aux[par];
    out_depth[(size_t)b * W + s] = pool_depth[i];
    out_score[(size_t)b * W + s] = c_score[i];
  }
}

// mask[b][i][j] = 1 iff j == i or j is an ancestor of i. One thread per (b, i) walks up the parents.
__global__ void tree_mask_kernel(const int* __restrict__ parent, int batch, int n, unsigned char* __restrict__ mask8,
                                 unsigned long long* __restrict__ mask64) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= batch * n) return;
  const int b = idx / n, i = idx - b * n;
  const int* par = parent + (size_t)b * n;
  const int words = (n + 63) / 64;
  if (mask8) {
    unsigned char* row = mask8 + ((size_t)b * n + i) * n;
    for (int j = 0; j < n; ++j) row[j] = 0;
  } else {
    unsigned long long* row = mask64 + ((size_t)b * n + i) * words;
    for (int w = 0; w < words; ++w) row[w] = 0ull;
  }
  if (i > 0 && par[i] < 0) return;                    // unused slot
  int j = i;
  for (int hops = 0; j >= 0 && hops <= n; ++hops) {   // bounded: a malformed parent array cannot loop forever
    if (mask8) mask8[((size_t)b * n + i) * n + j] = 1;
    else mask64[((size_t)b * n + i) * words + (j >> 6)] |= 1ull << (j & 63);
    const int p = par[j];
    j = (p < j) ? p : -1;
  }
}

}  // namespace moa
