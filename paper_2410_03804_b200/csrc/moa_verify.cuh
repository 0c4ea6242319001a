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

// A thread-block cluster of CL CTAs per logits row [V] of type T (float or bf16; CL = AM_CLUSTER when there are
// few rows and the row must be spread to fill the GPU, 1 when the rows alone do): every CTA scans one
// slice of the row, the slices' (value, id) pairs meet in the shared memory of the cluster's first CTA, which
// writes choice[row] = arg-max, smallest id among equals. Slices start on multiples of 8 elements, so a row
// that starts on a 16-byte boundary is read with 16-byte loads (scalar loads otherwise); NaNs never win.
constexpr int AM_CLUSTER = 8;

template <typename T, int CL>
__global__ void __cluster_dims__(CL, 1, 1) __launch_bounds__(256)
    argmax_rows_kernel(const T* __restrict__ logits, int V, int* __restrict__ choice) {
  pdl_trigger();
  pdl_wait();
  constexpr int PER = 16 / sizeof(T);
  const int rank = blockIdx.x;                     // the cluster spans blockIdx.x
  const T* row = logits + (size_t)blockIdx.y * V;
  const int per_cta = ((V + CL - 1) / CL + 7) & ~7;
  const int e0 = min(V, rank * per_cta), e1 = min(V, e0 + per_cta);
  float bv = -INFINITY;
  int bi = 0x7fffffff;
  const bool vec = ((reinterpret_cast<uintptr_t>(row) & 15u) == 0);
  const int nvec = vec ? (e1 - e0) / PER : 0;
  constexpr int UN = 4;                            // independent 16-byte loads in flight per thread
  for (int c0 = threadIdx.x; c0 < nvec; c0 += UN * blockDim.x) {
    uint4 raw[UN];
#pragma unroll
    for (int u = 0; u < UN; ++u) {
      const int c = c0 + u * blockDim.x;
      raw[u] = c < nvec ? __ldcs(reinterpret_cast<const uint4*>(row + e0) + c) : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int u = 0; u < UN; ++u) {
      const int c = c0 + u * blockDim.x;
      if (c >= nvec) continue;
      float x[PER];
      if constexpr (sizeof(T) == 4) {
        x[0] = __uint_as_float(raw[u].x); x[1] = __uint_as_float(raw[u].y);
        x[2] = __uint_as_float(raw[u].z); x[3] = __uint_as_float(raw[u].w);
      } else {
        const uint32_t w[4] = {raw[u].x, raw[u].y, raw[u].z, raw[u].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          x[2 * e] = __uint_as_float(w[e] << 16);               // a bf16 is the upper half of a float
          x[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
        }
      }
      // a thread meets its elements in increasing index order, so "strictly greater" keeps the smallest id
      float vm = x[0];
#pragma unroll
      for (int e = 1; e < PER; ++e) vm = fmaxf(vm, x[e]);
      if (vm > bv) {
        bv = vm;
#pragma unroll
        for (int e = PER - 1; e >= 0; --e)
          if (x[e] == vm) bi = e0 + c * PER + e;
      }
    }
  }
  for (int i = e0 + nvec * PER + threadIdx.x; i < e1; i += blockDim.x) best_of(to_f(row[i]), i, bv, bi);
  // CTA reduction
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    best_of(ov, oi, bv, bi);
  }
  __shared__ float sv[32];
  __shared__ int si[32];
  __shared__ float cv[CL];                         // used in the cluster's first CTA: one slot per rank
  __shared__ int ci[CL];
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
    if (lane == 0) {                               // hand the slice's result to rank 0's shared memory
      uint32_t rv, ri;
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rv) : "r"(smem_u32(&cv[rank])), "r"(0));
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ri) : "r"(smem_u32(&ci[rank])), "r"(0));
      asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(rv), "f"(bv) : "memory");
      asm volatile("st.shared::cluster.s32 [%0], %1;" ::"r"(ri), "r"(bi) : "memory");
    }
  }
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
  if (rank == 0 && threadIdx.x == 0) {
    float fv = -INFINITY;
    int fi = 0x7fffffff;
#pragma unroll
    for (int j = 0; j < CL; ++j) best_of(cv[j], ci[j], fv, fi);
    choice[blockIdx.y] = fi == 0x7fffffff ? 0 : fi;           // a row of NaNs / -inf: token 0
  }
}

// One warp per sequence walks the accepted path: the lanes look at 32 candidate children at a time.
// tok, parent, choice: [batch, n]; acc_*: [batch, cap].
__global__ void __launch_bounds__(128) verify_walk_kernel(const int* __restrict__ tok, const int* __restrict__ parent,
                                                          const int* __restrict__ choice, int batch, int n, int cap,
                                                          int* __restrict__ acc_slot, int* __restrict__ acc_tok,
                                                          int* __restrict__ acc_len, int* __restrict__ next_tok) {
  pdl_trigger();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (b >= batch) return;
  const int* t = tok + (size_t)b * n;
  const int* p = parent + (size_t)b * n;
  const int* ch = choice + (size_t)b * n;
  int cur = 0, len = 1;
  if (lane == 0) { acc_slot[(size_t)b * cap] = 0; acc_tok[(size_t)b * cap] = t[0]; }
  while (len < cap) {
    const int want = ch[cur];
    int nxt = -1;
    for (int c0 = cur + 1; c0 < n && nxt < 0; c0 += 32) {      // a child sits behind its parent; the first match wins
      const int c = c0 + lane;
      const bool hit = c < n && p[c] == cur && t[c] == want;
      const unsigned m = __ballot_sync(0xffffffffu, hit);
      if (m) nxt = c0 + __ffs(m) - 1;
    }
    if (nxt < 0) break;
    cur = nxt;
    if (lane == 0) { acc_slot[(size_t)b * cap + len] = cur; acc_tok[(size_t)b * cap + len] = t[cur]; }
    ++len;
  }
  for (int i = len + lane; i < cap; i += 32) { acc_slot[(size_t)b * cap + i] = -1; acc_tok[(size_t)b * cap + i] = -1; }
  if (lane == 0) { acc_len[b] = len; next_tok[b] = ch[cur]; }
}

}  // namespace moa
