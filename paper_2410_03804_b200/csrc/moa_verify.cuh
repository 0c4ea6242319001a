// Greedy verification of the kept draft tree (Section 2.2, step 2 with Tree Attention; Algorithm 1, the step
// that identifies the K' verified tokens): the LLM's choice at every kept slot is the arg-max of its logits
// there (ties: smallest id); from the root, the child that carries the chosen token is accepted, and the walk
// stops at the first slot without such a child. Byte and index work; the arg-max streams the logits once.
#pragma once
#include "moa_common.cuh"

namespace moa {

__device__ __forceinline__ void best_of(float v, int i, float& bv, int& bi) {
  if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
}

// One CTA per logits row [V] of type T (float or bf16): choice[row] = arg-max, smallest id among equals.
// 16-byte loads when the row starts on a 16-byte boundary, scalar loads otherwise; NaNs never win.
template <typename T>
__global__ void __launch_bounds__(512) argmax_rows_kernel(const T* __restrict__ logits, int V, int* __restrict__ choice) {
  pdl_trigger();
  pdl_wait();
  constexpr int PER = 16 / sizeof(T);
  const T* row = logits + (size_t)blockIdx.x * V;
  float bv = -INFINITY;
  int bi = 0x7fffffff;
  const bool vec = ((reinterpret_cast<uintptr_t>(row) & 15u) == 0);
  const int nvec = vec ? V / PER : 0;
  for (int c = threadIdx.x; c < nvec; c += blockDim.x) {
    const uint4 raw = __ldcs(reinterpret_cast<const uint4*>(row) + c);
    float x[PER];
    if constexpr (sizeof(T) == 4) {
      x[0] = __uint_as_float(raw.x); x[1] = __uint_as_float(raw.y);
      x[2] = __uint_as_float(raw.z); x[3] = __uint_as_float(raw.w);
    } else {
      const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        x[2 * e] = __uint_as_float(w[e] << 16);               // a bf16 is the upper half of a float
        x[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
      }
    }
#pragma unroll
    for (int e = 0; e < PER; ++e) best_of(x[e], c * PER + e, bv, bi);
  }
  for (int i = nvec * PER + threadIdx.x; i < V; i += blockDim.x) best_of(to_f(row[i]), i, bv, bi);
  // block reduction
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    best_of(ov, oi, bv, bi);
  }
  __shared__ float sv[32];
  __shared__ int si[32];
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  if (lane == 0) { sv[wid] = bv; si[wid] = bi; }
  __syncthreads();
  if (wid == 0) {
    bv = lane < nw ? sv[lane] : -INFINITY;
    bi = lane < nw ? si[lane] : 0x7fffffff;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      best_of(ov, oi, bv, bi);
    }
    if (lane == 0) choice[blockIdx.x] = bi == 0x7fffffff ? 0 : bi;     // a row of NaNs / -inf: token 0
  }
}

// One thread per sequence walks the accepted path. tok, parent, choice: [batch, n]; acc_*: [batch, cap].
__global__ void verify_walk_kernel(const int* __restrict__ tok, const int* __restrict__ parent, const int* __restrict__ choice,
                                   int batch, int n, int cap, int* __restrict__ acc_slot, int* __restrict__ acc_tok,
                                   int* __restrict__ acc_len, int* __restrict__ next_tok) {
  pdl_trigger();
  pdl_wait();
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= batch) return;
  const int* t = tok + (size_t)b * n;
  const int* p = parent + (size_t)b * n;
  const int* ch = choice + (size_t)b * n;
  int cur = 0, len = 1;
  acc_slot[(size_t)b * cap] = 0;
  acc_tok[(size_t)b * cap] = t[0];
  while (len < cap) {
    const int want = ch[cur];
    int nxt = -1;
    for (int c = cur + 1; c < n; ++c)          // a child sits behind its parent; the first match wins
      if (p[c] == cur && t[c] == want) { nxt = c; break; }
    if (nxt < 0) break;
    cur = nxt;
    acc_slot[(size_t)b * cap + len] = cur;
    acc_tok[(size_t)b * cap + len] = t[cur];
    ++len;
  }
  for (int i = len; i < cap; ++i) { acc_slot[(size_t)b * cap + i] = -1; acc_tok[(size_t)b * cap + i] = -1; }
  acc_len[b] = len;
  next_tok[b] = ch[cur];
}

}  // namespace moa
