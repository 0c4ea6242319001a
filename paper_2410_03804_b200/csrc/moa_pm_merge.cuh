// Phase machine, part 4: LM-head merge (Eq. 1 + the B most probable tokens): one CTA per activation row.
//
// The LM-head GEMM's epilogue leaves, per activation row, n_sub partial results -- each the (max, sum of
// exponentials) and the sorted B best (logit, id) of a disjoint piece of the vocabulary. This phase forms
// logsumexp over the pieces, then the global top-B by (value descending, id ascending): the B-th best list
// head is a threshold no final entry can rank after, only the (at most B) lists whose head passes it can
// contribute, and their survivors (at most B*B) are ranked by counting.
#pragma once
#include "moa_pm_common.cuh"

namespace moa {

//  p[0] ids out, p[1] logp out; i[1] B; rows = R. Partials come from the GEMM op.gemm.
__device__ __noinline__ void pm_merge(PmSmem& S, const PmOp& op, uint8_t* scratch, int wt) {
  const PmGemm& G = S.g[op.gemm];
  const float* p_max = G.p_max;
  const float* p_sum = G.p_sum;
  const float* c_val = G.c_val;
  const int* c_id = G.c_id;
  const int n_sub = G.n_sub;
  int* ids = (int*)op.p[0];
  float* logp = (float*)op.p[1];
  const int B = op.i[1], R = op.rows;
  const int NONE = 0x7fffffff;
  float* red = reinterpret_cast<float*>(scratch);               // [8]
  float* w_val = red + 8;                                       // [6][16]
  int* w_id = reinterpret_cast<int*>(w_val + PM_WWARPS * 16);   // [6][16]
  float* s_val = reinterpret_cast<float*>(w_id + PM_WWARPS * 16);   // [256]
  int* s_id = reinterpret_cast<int*>(s_val + 256);              // [256]
  float* t_val = reinterpret_cast<float*>(s_id + 256);
  int* t_id = reinterpret_cast<int*>(t_val + 1);
  int* n_surv = t_id + 1;
  const int lane = wt & 31, wid = wt >> 5;
  for (int r = blockIdx.x; r < R; r += gridDim.x) {
    wbar();
    if (wt == 0) *n_surv = 0;
    if (wt < B) { ids[(size_t)r * B + wt] = -1; logp[(size_t)r * B + wt] = -INFINITY; }
    // heads of the lists this thread owns, kept in registers
    float hv[PM_MERGE_OWN], pm[PM_MERGE_OWN], ps[PM_MERGE_OWN];
    int hi[PM_MERGE_OWN];
    float m = -INFINITY;
#pragma unroll
    for (int j = 0; j < PM_MERGE_OWN; ++j) {
      const int s = wt + j * PM_WORKERS;
      hv[j] = -INFINITY; hi[j] = NONE; pm[j] = -INFINITY; ps[j] = 0.f;
      if (s < n_sub) {
        hv[j] = __ldcg(c_val + ((size_t)r * n_sub + s) * B);
        hi[j] = __ldcg(c_id + ((size_t)r * n_sub + s) * B);
        pm[j] = __ldcg(p_max + (size_t)r * n_sub + s);
        ps[j] = __ldcg(p_sum + (size_t)r * n_sub + s);
      }
    }
#pragma unroll
    for (int j = 0; j < PM_MERGE_OWN; ++j) m = fmaxf(m, pm[j]);
    // logsumexp
    m = warp_max(m);
    if (lane == 0) red[wid] = m;
    wbar();
    m = red[0];
#pragma unroll
    for (int i = 1; i < PM_WWARPS; ++i) m = fmaxf(m, red[i]);
    wbar();
    float se = 0.f;
#pragma unroll
    for (int j = 0; j < PM_MERGE_OWN; ++j)
      if (pm[j] > -INFINITY) se += ps[j] * __expf(pm[j] - m);
    se = worker_sum(se, red, wt);
    const float lse = m + logf(se);
    // per warp: its B best heads, by rounds of "best ranking strictly after the previous pick"
    float pv = INFINITY;
    int pi = -1;
    for (int round = 0; round < B; ++round) {
      float bv = -INFINITY;
      int bi = NONE;
#pragma unroll
      for (int j = 0; j < PM_MERGE_OWN; ++j)
        if (ranks_before(pv, pi, hv[j], hi[j]) && ranks_before(hv[j], hi[j], bv, bi)) { bv = hv[j]; bi = hi[j]; }
      warp_best(bv, bi);
      pv = bv; pi = bi;
      if (lane == 0) { w_val[wid * 16 + round] = bv; w_id[wid * 16 + round] = bi; }
    }
    wbar();
    if (wid == 0) {                          // the B-th best over the six sorted warp lists
      float qv = INFINITY;
      int qi = -1;
      for (int round = 0; round < B; ++round) {
        float bv = -INFINITY;
        int bi = NONE;
        if (lane < PM_WWARPS) {
          for (int k = 0; k < B; ++k) {
            const float v = w_val[lane * 16 + k];
            const int id = w_id[lane * 16 + k];
            if (ranks_before(qv, qi, v, id)) { bv = v; bi = id; break; }
          }
        }
        warp_best(bv, bi);
        qv = bv; qi = bi;
      }
      if (lane == 0) { *t_val = qv; *t_id = qi; }
    }
    wbar();
    const float tv = *t_val;
    const int ti = *t_id;
    // survivors: entries of the owned lists ranking at or before the threshold
#pragma unroll
    for (int j = 0; j < PM_MERGE_OWN; ++j) {
      const int s = wt + j * PM_WORKERS;
      if (s >= n_sub || hi[j] == NONE || ranks_before(tv, ti, hv[j], hi[j])) continue;
      for (int c = 0; c < B; ++c) {
        const float v = c == 0 ? hv[j] : __ldcg(c_val + ((size_t)r * n_sub + s) * B + c);
        const int id = c == 0 ? hi[j] : __ldcg(c_id + ((size_t)r * n_sub + s) * B + c);
        if (ranks_before(tv, ti, v, id)) break;
        const int at = atomicAdd(n_surv, 1);
        if (at < 256) { s_val[at] = v; s_id[at] = id; }
      }
    }
    wbar();
    const int ns = *n_surv < 256 ? *n_surv : 256;
    for (int i = wt; i < ns; i += PM_WORKERS) {
      const float v = s_val[i];
      const int id = s_id[i];
      int rank = 0;
      for (int j = 0; j < ns; ++j) rank += ranks_before(s_val[j], s_id[j], v, id) ? 1 : 0;
      if (rank < B && id != NONE) {
        ids[(size_t)r * B + rank] = id;
        logp[(size_t)r * B + rank] = v - lse;
      }
    }
  }
}

}  // namespace moa
