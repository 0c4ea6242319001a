// Split-KV attention for the drafter's three attentions on the bf16 path (sm_100a).
//
// One CTA = one (sequence, kv head, query tile, key split). All query vectors that share a kv head --
// (rows of the sequence) x (query heads of the group) -- are stacked into the M dimension of
// mma.sync.m16n8k16 (16 queries per warp), so every cached key / value byte is read from HBM once per
// sequence and kv head whatever the number of tree rows or grouped heads. Keys and values stream
// through shared memory in blocks of 64 positions (cp.async, two stages, XOR-swizzled 16-byte chunks,
// ldmatrix); scores, softmax statistics and the output accumulate in fp32 (flash-style online softmax,
// probabilities rounded to bf16 for the P.V product).
//
// Key set of a row = segment A: positions 0..len-1 of a cache  [seq, capA, (posA_ld)]  (unmasked)
//                  + segment B: the sequence's tree slots, masked per row by its ancestor list.
// Splits 0..n_split-1 cover segment A; one more part (index n_split) covers segment B when present.
// With a single part the normalised output is written directly; otherwise each part leaves
// (max, sum, unnormalised output) and attn_combine_kernel merges them.
#pragma once
#include "moa_common.cuh"

namespace moa {

constexpr int AT_KB = 64;        // keys per block

struct AttnParams {
  const bf16* q; int q_ld;               // query row r, head h at q + r*q_ld + h*DH
  const float* q32;                      // QSPLIT kernels: the same layout in fp32 (q is unused then), possibly as
  int q_splits; size_t q_plane;          // q_splits split-K planes of a GEMM, q_plane elements apart, summed on load
  int hq, hkv, group;                    // group = hq / hkv
  int rows_per_seq;                      // query rows of one sequence (tree rows, or LSA layers)
  const bf16* kA; const bf16* vA; int capA; int posA_ld;   // segment A: (seq*capA + j)*posA_ld + g*DH
  const int* lenA; int nA_fixed;         // valid positions: lenA[seq] or the fixed count
  RowLimit lim;                          // optional per-row bound on segment A (whole-sequence pass)
  const bf16* kB; const bf16* vB; int capB;                // segment B: ((seq*capB + slot)*hkv + g)*DH
  const int* slotsB; int slots_ld; int nB; int n_slots;    // row's ancestor slots [nB]; slots in use
  int n_split;                           // splits of segment A
  int n_parts;                           // n_split + (segment B ? 1 : 0)
  int q_tiles;                           // query tiles per (seq, kv head)
  float* part_o; float* part_ml;         // [R*hq][n_parts][DH], [R*hq][n_parts][2]
  bf16* out;                             // [R, hq*DH]
  int out_lo;                            // > 0: the low-order term of every output goes to row out_lo + r
  float scale_log2;                      // log2(e) / sqrt(DH)
  int* status;                           // device status word (debug-build index checks)
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int sz = valid ? 16 : 0;         // zero-fills the 16 bytes when the source row does not exist
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// 2^x by the special-function unit (x <= 0 here; 2^-inf = 0).
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Byte offset of (row, 16-byte chunk) in a tile of DH-wide bf16 rows, chunks XOR-swizzled by the row.
template <int DH>
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
  return (uint32_t)(row * (DH * 2) + ((chunk ^ (row & 7)) << 4));
}

// QSPLIT: the queries arrive in fp32 and are split into two bf16 terms (q = hi + lo, lo = the part of q
// that hi's 8-bit mantissa dropped); scores are Q_hi.K^T + Q_lo.K^T, so they carry the queries at about 16 bits
// of mantissa while the cached keys stay in their 16-bit storage type. This keeps a peaked softmax (keys
// with outlier channels) from amplifying the rounding of q.
template <int DH, bool QSPLIT, bool PSPLIT>
__global__ void __launch_bounds__(256) attn_split_kernel(const AttnParams P) {
  pdl_trigger();
  pdl_wait(KID_ATTN);
  constexpr int CH = DH / 8;                 // 16-byte chunks per row
  constexpr int KS = DH / 16;                // k-steps of the Q.K^T product
  constexpr int TILE_BYTES = AT_KB * DH * 2;
  extern __shared__ __align__(128) uint8_t at_smem[];
  __shared__ unsigned long long allow[16][4];     // per sequence row: bit per tree slot (<= 256 slots)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  const int part = blockIdx.x;
  const int g = blockIdx.y / P.q_tiles, qt = blockIdx.y - g * P.q_tiles;
  const int seq = blockIdx.z;
  const int QT = nwarps * 16;                // queries per tile
  const int Qn = P.rows_per_seq * P.group;   // queries per (seq, kv head)
  const uint32_t sQ = smem_u32(at_smem);
  const uint32_t sQlo = sQ + QT * DH * 2;    // QSPLIT only
  const uint32_t sKV = sQ + (QSPLIT ? 2 : 1) * QT * DH * 2;     // [2 stages][K tile | V tile]

  const bool tree_part = part >= P.n_split;
  // key range of this part
  int k_begin, k_end;
  if (!tree_part) {
    const int len = P.lenA ? P.lenA[seq] : P.nA_fixed;
    if (threadIdx.x == 0) MOA_DEV_CHECK(len >= 0 && len <= P.capA, P.status);
    const int blocks = (len + AT_KB - 1) / AT_KB;
    const int b0 = (int)(((long long)part * blocks) / P.n_split), b1 = (int)(((long long)(part + 1) * blocks) / P.n_split);
    k_begin = b0 * AT_KB;
    k_end = min(b1 * AT_KB, len);
    if (P.lim.active()) {                  // limits do not decrease with the row: the tile's last row has the largest
      const int q_last = min(Qn, (qt + 1) * QT) - 1;
      k_end = min(k_end, P.lim.of(seq * P.rows_per_seq + q_last / P.group));
    }
  } else {
    k_begin = 0;
    k_end = P.n_slots;
    if (threadIdx.x < 64) allow[threadIdx.x >> 2][threadIdx.x & 3] = 0ull;
    __syncthreads();
    if (threadIdx.x < P.rows_per_seq && threadIdx.x < 16) {
      const int r = seq * P.rows_per_seq + threadIdx.x;
      for (int i = 0; i < P.nB; ++i) {
        const int slot = P.slotsB[(size_t)r * P.slots_ld + i];
        MOA_DEV_CHECK(slot >= 0 && slot < P.n_slots && slot < P.capB, P.status);
        if (slot >= 0 && slot < 256) allow[threadIdx.x][slot >> 6] |= 1ull << (slot & 63);
      }
    }
  }

  // A thread always copies the same 16-byte column of the rows r0, r0 + rstep, ...: one pointer increment per row.
  const int ld_c = threadIdx.x & (CH - 1), ld_r0 = threadIdx.x / CH, ld_rstep = blockDim.x / CH;
  const size_t row_stride = tree_part ? (size_t)P.hkv * DH : (size_t)P.posA_ld;       // elements between two positions
  const size_t seg_base = tree_part ? ((size_t)seq * P.capB * P.hkv + g) * DH : (size_t)seq * P.capA * P.posA_ld + g * DH;
  const bf16* const k_src = (tree_part ? P.kB : P.kA) + seg_base + ld_c * 8;
  const bf16* const v_src = (tree_part ? P.vB : P.vA) + seg_base + ld_c * 8;
  auto load_block = [&](int stage, int k0) {
    const uint32_t sK = sKV + stage * 2 * TILE_BYTES, sV = sK + TILE_BYTES;
    size_t off = (size_t)(k0 + ld_r0) * row_stride;
    for (int kr = ld_r0; kr < AT_KB; kr += ld_rstep, off += (size_t)ld_rstep * row_stride) {
      const bool valid = k0 + kr < k_end;
      const size_t o = valid ? off : 0;                    // an address inside the segment; nothing is read when !valid
      const uint32_t d = tile_off<DH>(kr, ld_c);
      cp_async16(sK + d, k_src + o, valid);
      cp_async16(sV + d, v_src + o, valid);
    }
  };

  const int n_blocks = (k_end - k_begin + AT_KB - 1) / AT_KB;
  if (n_blocks > 0) load_block(0, k_begin);      // on its way while the queries are staged
  cp_async_commit();

  // ---- Q tile -> shared (zero rows for queries beyond Qn) ----
  if (QSPLIT) {
    // fp32 queries: four 8-element pieces per thread at a time, all their loads in flight before the first is used
    // (one memory round trip per four pieces instead of one per piece)
    for (int i0 = threadIdx.x; i0 < QT * CH; i0 += 4 * blockDim.x) {
      float x[4][8];
      bool valid[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + u * blockDim.x;
        const int ql = i / CH, c = i - ql * CH;
        const int qi = qt * QT + ql;
        valid[u] = i < QT * CH && qi < Qn;
        if (valid[u]) {
          const int row = seq * P.rows_per_seq + qi / P.group;
          const int head = g * P.group + qi % P.group;
          load8_planes(P.q32 + (size_t)row * P.q_ld + head * DH + c * 8, P.q_splits, P.q_plane, x[u]);
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + u * blockDim.x;
        if (i >= QT * CH) continue;
        const int ql = i / CH, c = i - ql * CH;
        uint32_t hi[4] = {0u, 0u, 0u, 0u}, lo[4] = {0u, 0u, 0u, 0u};
        if (valid[u]) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const bf16 h0 = __float2bfloat16_rn(x[u][2 * e]), h1 = __float2bfloat16_rn(x[u][2 * e + 1]);
            hi[e] = pack_bf16(__bfloat162float(h0), __bfloat162float(h1));
            lo[e] = pack_bf16(x[u][2 * e] - __bfloat162float(h0), x[u][2 * e + 1] - __bfloat162float(h1));
          }
        }
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sQ + tile_off<DH>(ql, c)), "r"(hi[0]), "r"(hi[1]),
                     "r"(hi[2]), "r"(hi[3]) : "memory");
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sQlo + tile_off<DH>(ql, c)), "r"(lo[0]), "r"(lo[1]),
                     "r"(lo[2]), "r"(lo[3]) : "memory");
      }
    }
  } else {
    for (int i = threadIdx.x; i < QT * CH; i += blockDim.x) {
      const int ql = i / CH, c = i - ql * CH;
      const int qi = qt * QT + ql;
      const bool valid = qi < Qn;
      const int row = seq * P.rows_per_seq + (valid ? qi / P.group : 0);
      const int head = g * P.group + (valid ? qi % P.group : 0);
      cp_async16(sQ + tile_off<DH>(ql, c), P.q + (size_t)row * P.q_ld + head * DH + c * 8, valid);
    }
  }
  cp_async_commit();

  cp_async_wait<0>();            // Q and the first key / value block have landed
  __syncthreads();

  // ---- Q fragments of this warp's 16 queries ----
  uint32_t qf[KS][4];
  {
    const int row = warp * 16 + (lane & 15);
#pragma unroll
    for (int ks = 0; ks < KS; ++ks)
      ldsm_x4(sQ + tile_off<DH>(row, ks * 2 + (lane >> 4)), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
  }
  const int gq = lane >> 2, tq = lane & 3;
  // the two query rows of this thread: warp*16 + gq and + 8
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  float o[DH / 8][4];
#pragma unroll
  for (int i = 0; i < DH / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  int seqrow[2];                 // sequence-local row of each query (for the tree mask)
  int limrow[2];                 // its bound on segment A
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int qi = qt * QT + warp * 16 + gq + 8 * h;
    seqrow[h] = qi < Qn ? qi / P.group : 0;
    limrow[h] = P.lim.active() ? P.lim.of(seq * P.rows_per_seq + seqrow[h]) : 0x7fffffff;
  }

  for (int blk = 0; blk < n_blocks; ++blk) {
    const int stage = blk & 1;
    if (blk + 1 < n_blocks) load_block(stage ^ 1, k_begin + (blk + 1) * AT_KB);
    cp_async_commit();
    cp_async_wait<1>();          // block `blk` has landed
    __syncthreads();
    const uint32_t sK = sKV + stage * 2 * TILE_BYTES, sV = sK + TILE_BYTES;
    const int k0 = k_begin + blk * AT_KB;

    // S = Q K^T over the block's 64 keys: 8 n-tiles of 8 keys
    float s[AT_KB / 8][4];
#pragma unroll
    for (int nt = 0; nt < AT_KB / 8; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
    // Tensor-core instructions that add into the same accumulator wait for one another, so they are issued
    // accumulator by accumulator in rounds: the eight key tiles' fragments are loaded first, then every round
    // touches each of the eight accumulators once.
#pragma unroll
    for (int ks2 = 0; ks2 < KS / 2; ++ks2) {
      uint32_t ql0[4], ql1[4];         // QSPLIT: the low query terms of these two k-steps
      if (QSPLIT) {
        const int row = warp * 16 + (lane & 15);
        ldsm_x4(sQlo + tile_off<DH>(row, (2 * ks2) * 2 + (lane >> 4)), ql0[0], ql0[1], ql0[2], ql0[3]);
        ldsm_x4(sQlo + tile_off<DH>(row, (2 * ks2 + 1) * 2 + (lane >> 4)), ql1[0], ql1[1], ql1[2], ql1[3]);
      }
      uint32_t kb[AT_KB / 8][4];       // two k-steps: chunks 4*ks2 .. 4*ks2+3 of key row nt*8 + lane%8
#pragma unroll
      for (int nt = 0; nt < AT_KB / 8; ++nt)
        ldsm_x4(sK + tile_off<DH>(nt * 8 + (lane & 7), ks2 * 4 + (lane >> 3)), kb[nt][0], kb[nt][1], kb[nt][2], kb[nt][3]);
#pragma unroll
      for (int nt = 0; nt < AT_KB / 8; ++nt) mma_bf16_16816(s[nt], qf[2 * ks2], kb[nt][0], kb[nt][1]);
#pragma unroll
      for (int nt = 0; nt < AT_KB / 8; ++nt) mma_bf16_16816(s[nt], qf[2 * ks2 + 1], kb[nt][2], kb[nt][3]);
      if (QSPLIT) {
#pragma unroll
        for (int nt = 0; nt < AT_KB / 8; ++nt) mma_bf16_16816(s[nt], ql0, kb[nt][0], kb[nt][1]);
#pragma unroll
        for (int nt = 0; nt < AT_KB / 8; ++nt) mma_bf16_16816(s[nt], ql1, kb[nt][2], kb[nt][3]);
      }
    }
    // mask, block row max (of the raw scores: the scale is positive and goes into the exponent's multiply-add).
    // Most blocks of a cache segment need no mask at all (warp-uniform test).
    float mx[2] = {-INFINITY, -INFINITY};
    if (!tree_part && !P.lim.active() && k0 + AT_KB <= k_end) {
#pragma unroll
      for (int nt = 0; nt < AT_KB / 8; ++nt) {
#pragma unroll
        for (int e = 0; e < 4; ++e) mx[e >> 1] = fmaxf(mx[e >> 1], s[nt][e]);
      }
    } else {
#pragma unroll
      for (int nt = 0; nt < AT_KB / 8; ++nt) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int key = k0 + nt * 8 + tq * 2 + (e & 1);
          const int h = e >> 1;
          bool ok = key < k_end;
          if (tree_part && ok) ok = (allow[seqrow[h]][key >> 6] >> (key & 63)) & 1ull;
          if (!tree_part && ok) ok = key < limrow[h];
          const float v = ok ? s[nt][e] : -INFINITY;
          s[nt][e] = v;
          mx[h] = fmaxf(mx[h], v);
        }
      }
    }
    float corr[2], msub[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
      mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
      const float mn = fmaxf(m_run[h], mx[h] * P.scale_log2);       // log2 domain
      corr[h] = (m_run[h] == -INFINITY) ? 0.f : ex2_approx(m_run[h] - mn);
      msub[h] = (mn == -INFINITY) ? 0.f : mn;      // a fully masked row keeps p = exp2(-inf) = 0
      m_run[h] = mn;
    }
    float rs[2] = {0.f, 0.f};
    uint32_t pf[AT_KB / 16][4], pl[AT_KB / 16][4];      // probabilities as hi (+ lo with PSPLIT) bf16 terms
#pragma unroll
    for (int nt = 0; nt < AT_KB / 8; ++nt) {
      const float p0 = ex2_approx(fmaf(s[nt][0], P.scale_log2, -msub[0])), p1 = ex2_approx(fmaf(s[nt][1], P.scale_log2, -msub[0]));
      const float p2 = ex2_approx(fmaf(s[nt][2], P.scale_log2, -msub[1])), p3 = ex2_approx(fmaf(s[nt][3], P.scale_log2, -msub[1]));
      rs[0] += p0 + p1;
      rs[1] += p2 + p3;
      const uint32_t h01 = pack_bf16(p0, p1), h23 = pack_bf16(p2, p3);     // a bf16 is the upper half of a float
      pf[nt >> 1][(nt & 1) * 2 + 0] = h01;
      pf[nt >> 1][(nt & 1) * 2 + 1] = h23;
      if (PSPLIT) {
        pl[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(p0 - __uint_as_float(h01 << 16), p1 - __uint_as_float(h01 & 0xffff0000u));
        pl[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p2 - __uint_as_float(h23 << 16), p3 - __uint_as_float(h23 & 0xffff0000u));
      }
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) l_run[h] = l_run[h] * corr[h] + rs[h];
    if (__any_sync(0xffffffffu, corr[0] != 1.f || corr[1] != 1.f)) {      // the running maxima settle after a few blocks
#pragma unroll
      for (int i = 0; i < DH / 8; ++i) {
        o[i][0] *= corr[0]; o[i][1] *= corr[0];
        o[i][2] *= corr[1]; o[i][3] *= corr[1];
      }
    }
    // O += P V: k-steps of 16 keys, n-tiles of 8 output columns (two per ldmatrix); same issue order in rounds
    // over independent accumulators, four ldmatrix results (eight output tiles) at a time
#pragma unroll
    for (int kk = 0; kk < AT_KB / 16; ++kk) {
      const int key = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
      for (int n4 = 0; n4 < DH / 64; ++n4) {
        uint32_t vb[4][4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
          ldsm_x4_t(sV + tile_off<DH>(key, (n4 * 4 + j) * 2 + (lane >> 4)), vb[j][0], vb[j][1], vb[j][2], vb[j][3]);
#pragma unroll
        for (int j = 0; j < 4; ++j) mma_bf16_16816(o[2 * (n4 * 4 + j)], pf[kk], vb[j][0], vb[j][1]);
#pragma unroll
        for (int j = 0; j < 4; ++j) mma_bf16_16816(o[2 * (n4 * 4 + j) + 1], pf[kk], vb[j][2], vb[j][3]);
        if (PSPLIT) {
#pragma unroll
          for (int j = 0; j < 4; ++j) mma_bf16_16816(o[2 * (n4 * 4 + j)], pl[kk], vb[j][0], vb[j][1]);
#pragma unroll
          for (int j = 0; j < 4; ++j) mma_bf16_16816(o[2 * (n4 * 4 + j) + 1], pl[kk], vb[j][2], vb[j][3]);
        }
      }
    }
    __syncthreads();             // the stage may be overwritten by the next prefetch
  }
  cp_async_wait<0>();

  // ---- finish: row sums across the quad, then write ----
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 1);
    l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 2);
  }
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int qi = qt * QT + warp * 16 + gq + 8 * h;
    if (qi >= Qn) continue;
    const int row = seq * P.rows_per_seq + qi / P.group;
    const int head = g * P.group + qi % P.group;
    if (P.n_parts == 1) {
      const float inv = l_run[h] > 0.f ? 1.f / l_run[h] : 0.f;
      bf16* dst = P.out + ((size_t)row * P.hq + head) * DH;
      bf16* dlo = P.out + ((size_t)(P.out_lo + row) * P.hq + head) * DH;
#pragma unroll
      for (int i = 0; i < DH / 8; ++i) {
        const float a = o[i][2 * h] * inv, b = o[i][2 * h + 1] * inv;
        const bf16 ha = __float2bfloat16_rn(a), hb = __float2bfloat16_rn(b);
        *reinterpret_cast<uint32_t*>(dst + i * 8 + tq * 2) = pack_bf16(__bfloat162float(ha), __bfloat162float(hb));
        if (P.out_lo > 0)
          *reinterpret_cast<uint32_t*>(dlo + i * 8 + tq * 2) = pack_bf16(a - __bfloat162float(ha), b - __bfloat162float(hb));
      }
    } else {
      const size_t pidx = ((size_t)row * P.hq + head) * P.n_parts + part;
      float* dst = P.part_o + pidx * DH;
#pragma unroll
      for (int i = 0; i < DH / 8; ++i)
        *reinterpret_cast<float2*>(dst + i * 8 + tq * 2) = make_float2(o[i][2 * h], o[i][2 * h + 1]);
      if (tq == 0) {
        P.part_ml[pidx * 2 + 0] = m_run[h];      // log2 domain
        P.part_ml[pidx * 2 + 1] = l_run[h];
      }
    }
  }
}

// out[row, head, :] = sum_p 2^(m_p - M) O_p / sum_p 2^(m_p - M) l_p. The merge is a chain of dependent memory
// round trips, so it is spread as wide as the parts allow. share = 1 (many parts): one CTA of CB_WARPS warps per
// (row, head); every warp loads the parts' (max, sum) pairs (one per lane) for the common maximum and the weights,
// then adds up its share of the partial outputs (parts w, w + CB_WARPS, ..., two in flight) and the warps' sums
// meet in shared memory. share = 0 (few parts): one warp per (row, head), CB_WARPS of them per CTA.
constexpr int CB_WARPS = 4;
constexpr int CB_SHARE_FROM = 9;       // parts from which a (row, head) gets a whole CTA

template <int DH>
__global__ void __launch_bounds__(CB_WARPS * 32) attn_combine_kernel(const float* __restrict__ part_o,
                                                                    const float* __restrict__ part_ml, int n_parts, int n_rh,
                                                                    int share, bf16* __restrict__ out, int out_lo, int hq) {
  pdl_trigger();
  pdl_wait(KID_ATTN_MERGE);
  __shared__ float acc_sh[CB_WARPS][DH];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int rh = share ? blockIdx.x : blockIdx.x * CB_WARPS + w;
  const int first = share ? w : 0, step = share ? CB_WARPS : 1;      // this warp's parts: first, first + step, ...
  const bool live = rh < n_rh;
  float M = -INFINITY;
  float L = 0.f, acc[DH / 32];
#pragma unroll
  for (int e = 0; e < DH / 32; ++e) acc[e] = 0.f;
  if (live) {
    for (int p0 = 0; p0 < n_parts; p0 += 32) {
      const float m = p0 + lane < n_parts ? part_ml[((size_t)rh * n_parts + p0 + lane) * 2] : -INFINITY;
      M = fmaxf(M, warp_max(m));
    }
    for (int p0 = 0; p0 < n_parts; p0 += 32) {
      float wl = 0.f, ww = 0.f;
      if (p0 + lane < n_parts) {
        const float2 ml = *reinterpret_cast<const float2*>(part_ml + ((size_t)rh * n_parts + p0 + lane) * 2);
        ww = ml.x == -INFINITY ? 0.f : exp2f(ml.x - M);
        wl = ww * ml.y;
      }
      L += warp_sum(wl);
      const int np = min(32, n_parts - p0);
      for (int pp = first; pp < np; pp += 2 * step) {          // two parts in flight
        float x[2][DH / 32];
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
          for (int e = 0; e < DH / 32; ++e)
            x[u][e] = pp + u * step < np ? part_o[((size_t)rh * n_parts + p0 + pp + u * step) * DH + lane + 32 * e] : 0.f;
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const float wu = __shfl_sync(0xffffffffu, ww, (pp + u * step) & 31);
          if (pp + u * step < np)
#pragma unroll
            for (int e = 0; e < DH / 32; ++e) acc[e] += wu * x[u][e];
        }
      }
    }
  }
  if (share) {
#pragma unroll
    for (int e = 0; e < DH / 32; ++e) acc_sh[w][lane + 32 * e] = acc[e];
    __syncthreads();
    if (w != 0) return;
#pragma unroll
    for (int e = 0; e < DH / 32; ++e) {
      float a = 0.f;
#pragma unroll
      for (int k = 0; k < CB_WARPS; ++k) a += acc_sh[k][lane + 32 * e];      // fixed order
      acc[e] = a;
    }
  }
  if (!live) return;
  const float inv = L > 0.f ? 1.f / L : 0.f;
#pragma unroll
  for (int e = 0; e < DH / 32; ++e) {
    const float a = acc[e] * inv;
    const bf16 h = __float2bfloat16_rn(a);
    out[(size_t)rh * DH + lane + 32 * e] = h;
    if (out_lo > 0) out[((size_t)out_lo * hq + rh) * DH + lane + 32 * e] = __float2bfloat16_rn(a - __bfloat162float(h));
  }
}

}  // namespace moa
