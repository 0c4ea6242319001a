// Attention over a long cache segment on the 5th-generation tensor cores (sm_100a, head size 128).
//
// The split-KV kernel of moa_attn.cuh issues its products with mma.sync from a handful of warps, and at long
// context (tens of thousands of cached positions per kv head) it is bound by that instruction stream, not by HBM.
// Here one CTA per (sequence, kv head, key range) keeps all queries that share the kv head -- (rows of the
// sequence) x (query heads of the group), at most 128 -- as the M = 128 operand and streams the cache through a TMA
// ring of 128-position blocks:
//   warp 0      TMA producer: K block [128, 128] and V block [128, 128] per stage (128-byte swizzle), three stages
//   warp 1      one thread issues tcgen05.mma:  S = Q_hi K^T + Q_lo K^T   (A = Q in TENSOR MEMORY, B = K, K-major,
//                                                                          N = 128: one chain of 16 products)
//                                               O += P_hi V + P_lo V      (A = P in tensor memory, B = V as it lies in
//                                                                          the cache: MN-major)
//               The tensor pipe sets the pace: a product costs about 50 cycles at N = 64 and 64 at N = 128 whatever
//               its operands' source, so blocks of 128 positions halve the cost of the scores per position.
//   warps 2..9  softmax: two threads per query row (tensor-memory lane), one per half of the block's 128 scores. A
//               thread reads its 64 scores, the two exchange their maxima through shared memory, keep the running
//               reference maximum and their part of the sum in the log2 domain, and write the probabilities as two
//               bf16 terms over the scores (P_hi takes the first 64 columns of the score buffer, P_lo the other 64).
// Tensor memory (512 columns): Q_hi | Q_lo at 0 (64 columns each: two bf16 per column), two score / probability buffers
// at 128 and 256 (the scores of block b + 1 are formed while the softmax of block b runs), the output accumulator at
// 384. The output accumulator is rescaled only when a row's maximum has grown by more than 2^8 since its last rescale
// (probabilities then stay below 256), so the rescale -- a TMEM load, multiply, store of the row -- happens a few
// times per range, not per block.
// Each CTA leaves (max, sum, unnormalised output) per query for attn_combine_kernel, in the layout of the split-KV
// kernel (or the normalised rows when the range is the attention's only part). A self-attention's tree segment (the
// sequence's drafted slots, masked per row by its ancestor list) is one more CTA of the same grid: same pipeline over
// the tree's keys / values, with the row's slot bitmap applied to the scores. Queries arrive in fp32 and enter as two
// bf16 terms, as in the split-KV kernel.
// Every mbarrier wait is bounded; on expiry the CTA raises the abort flag, drains, frees TMEM and reports
// DEV_ERR_TIMEOUT through the status word.
#pragma once
#include "moa_attn.cuh"
#include "moa_wstream.cuh"

namespace moa {

constexpr int TC_KB = 128;                // cache positions per block
constexpr int TC_DH = 128;
constexpr int TC_STAGES = 3;
constexpr int TC_THREADS = 320;            // TMA warp, MMA warp, eight softmax warps (two per tensor-memory lane quadrant)
constexpr int TC_KV_BYTES = TC_KB * TC_DH * 2;        // K (or V) block: two 64-column chunks of [128 rows x 128 B]
constexpr int TC_STAGE_BYTES = 2 * TC_KV_BYTES;       // 64 KB
constexpr int TC_Q_BYTES = 128 * TC_DH * 2;           // staging of one query term; the two terms lie over the last stage
constexpr int TC_X_BYTES = 2 * 2 * 128 * 4;           // row maxima exchanged between the two threads of a row
constexpr int TC_SMEM_BYTES = TC_STAGES * TC_STAGE_BYTES + TC_X_BYTES + 1024 + 256;
constexpr uint32_t TC_TM_Q = 0, TC_TM_S = 128, TC_TM_O = 384;   // tensor-memory columns (see above)
constexpr float TC_RESCALE_LOG2 = 8.f;

struct AttnTcParams {
  CUtensorMap tmK, tmV;      // cache [positions of all sequences, hkv * 128], box 64 columns x 64 positions, swizzle 128B
  CUtensorMap tmKB, tmVB;    // tree slots [slots of all sequences, hkv * 128], same box (used when a.n_parts > a.n_split)
  AttnParams a;              // queries (fp32), lengths, part buffers; part a.n_split, if any, is the tree segment
  int early_cache;           // the cache segment (and its lengths) were complete before the chain this launch belongs to
                             // began: its first blocks may be fetched before the wait on the preceding kernel
};

// Shared-memory descriptor of an MN-major bf16 operand with the 128-byte swizzle: 64 elements along MN are contiguous
// (one 128-byte row per K index), 8 K-rows make a 1024-byte group (stride byte offset), the next 64 MN elements
// start `lbo` bytes further (leading byte offset).
__device__ __forceinline__ uint64_t umma_desc_mn_sw128(uint32_t saddr, uint32_t lbo) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) |
         (2ull << 61);
}
// Instruction descriptor as umma_idesc_bf16, with B taken MN-major.
__host__ __device__ constexpr uint32_t umma_idesc_bf16_bmn(int m, int n) { return umma_idesc_bf16(m, n) | (1u << 16); }

// tcgen05.mma with the A operand in tensor memory: row r of A in lane r, elements 2 j and 2 j + 1 of a row as the low and
// high half of column j (a K = 16 step takes 8 columns).
__device__ __forceinline__ void tc_mma_bf16_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// 64 consecutive columns of this thread's lane in one instruction
__device__ __forceinline__ void tc_ld64(uint32_t taddr, float* v) {
  uint32_t r[64];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x64.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, "
      "%32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, "
      "%48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]),
        "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]),
        "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]),
        "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 64; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tc_st8(uint32_t taddr, const uint32_t* r) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"r"(taddr), "r"(r[0]), "r"(r[1]),
               "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}
__device__ __forceinline__ void tc_st16(uint32_t taddr, const float* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
        "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
        "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
        "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15]))
      : "memory");
}

// Barrier 1 over the 256 softmax threads that also ORs a flag: every thread gets the same answer, so a failed wait
// anywhere takes all of them out of their loop at the same barrier (nobody is left waiting at the next one).
__device__ __forceinline__ bool tc_bar_any(bool mine) {
  uint32_t any;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.or.pred p, 1, 256, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(any)
      : "r"((uint32_t)(mine ? 1u : 0u))
      : "memory");
  return any != 0u;
}

__global__ void __launch_bounds__(TC_THREADS, 1) attn_tc_kernel(const __grid_constant__ AttnTcParams P) {
  extern __shared__ uint8_t tc_smem_raw[];
  const uint32_t base = (smem_u32(tc_smem_raw) + 1023u) & ~1023u;
  uint8_t* bp = tc_smem_raw + (base - smem_u32(tc_smem_raw));
  // Key and value blocks have rings of their own (a key block is free again once its scores are formed, a block time
  // before its value block): K0 K1 V0 V1 K2 V2. The last pair doubles as the query staging area at start-up.
  auto k_off = [&](int st) { return (uint32_t)(st < TC_STAGES - 1 ? st * TC_KV_BYTES : 2 * (TC_STAGES - 1) * TC_KV_BYTES); };
  auto v_off = [&](int st) { return (uint32_t)(st < TC_STAGES - 1 ? (TC_STAGES - 1 + st) * TC_KV_BYTES : (2 * (TC_STAGES - 1) + 1) * TC_KV_BYTES); };
  constexpr uint32_t oQhi = 2 * (TC_STAGES - 1) * TC_KV_BYTES, oQlo = oQhi + TC_Q_BYTES;
  constexpr uint32_t oX = TC_STAGES * TC_STAGE_BYTES, oBar = oX + TC_X_BYTES;
  const uint32_t bar0 = base + oBar;
  auto kfull_bar = [&](int s) { return bar0 + 8u * s; };
  auto kempty_bar = [&](int s) { return bar0 + 8u * (TC_STAGES + s); };
  auto vfull_bar = [&](int s) { return bar0 + 8u * (2 * TC_STAGES + s); };
  auto vempty_bar = [&](int s) { return bar0 + 8u * (3 * TC_STAGES + s); };
  auto sfull_bar = [&](int i) { return bar0 + 8u * (4 * TC_STAGES + i); };
  auto pfull_bar = [&](int i) { return bar0 + 8u * (4 * TC_STAGES + 2 + i); };
  const uint32_t pempty_bar = bar0 + 8u * (4 * TC_STAGES + 4), qfull_bar = pempty_bar + 8u, ofull_bar = qfull_bar + 8u;
  uint32_t* tmem_slot = (uint32_t*)(bp + oBar + 8 * (4 * TC_STAGES + 7));
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);
  float* xm = reinterpret_cast<float*>(bp + oX);       // [buffer][half][row]

  const AttnParams& A = P.a;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = blockIdx.x, seq = blockIdx.y, part = blockIdx.z;      // parts along z: the tree part's CTAs are launched last
  const int Qn = A.rows_per_seq * A.group;           // <= 128, checked by the host
  pdl_trigger();

  if (threadIdx.x == 0) {
    for (int s = 0; s < TC_STAGES; ++s) {
      mbar_init(kfull_bar(s), 1); mbar_init(kempty_bar(s), 1);
      mbar_init(vfull_bar(s), 1); mbar_init(vempty_bar(s), 1);
    }
    for (int i = 0; i < 2; ++i) { mbar_init(sfull_bar(i), 1); mbar_init(pfull_bar(i), 256); }
    mbar_init(pempty_bar, 1);
    mbar_init(qfull_bar, 256);
    mbar_init(ofull_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // The queries and the tree slots come from the kernels just before this one. A cache segment that was complete
  // before the chain began needs no wait: its producer warp sends its first blocks at once and waits after.
  const bool tree_part = part >= A.n_split;          // the grid's last CTA along z when the attention has a tree segment
  const bool early = P.early_cache != 0 && !tree_part;
  if (!(early && warp == 0)) pdl_wait(KID_ATTN);
  int k_begin, k_end, n_blocks;
  if (!tree_part) {
    const int len = A.lenA ? A.lenA[seq] : A.nA_fixed;
    const int blocks = (len + TC_KB - 1) / TC_KB;
    const int b0 = (int)(((long long)part * blocks) / A.n_split), b1 = (int)(((long long)(part + 1) * blocks) / A.n_split);
    k_begin = b0 * TC_KB;
    k_end = min(b1 * TC_KB, len);
    n_blocks = b1 - b0;
  } else {
    k_begin = 0;
    k_end = min(A.n_slots, 256);                     // slot bitmaps hold 256 slots (the host checks)
    n_blocks = (k_end + TC_KB - 1) / TC_KB;
  }

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      const int x0 = g * TC_DH;
      bool waited = !early;
      bool ok = true;
      for (int b = 0; b < n_blocks && ok; ++b) {
        const int st = b % TC_STAGES;
        if (st == TC_STAGES - 1 && b < TC_STAGES) {
          // the last stage holds the query staging until the queries are in tensor memory
          if (!waited) { pdl_wait(KID_ATTN); waited = true; }
          if (!mbar_wait(qfull_bar, 0u, abort_flag)) break;
        }
        const uint32_t k = (uint32_t)(b / TC_STAGES);
        const int y = seq * (tree_part ? A.capB : A.capA) + k_begin + b * TC_KB;
        const CUtensorMap* tk = tree_part ? &P.tmKB : &P.tmK;
        const CUtensorMap* tv = tree_part ? &P.tmVB : &P.tmV;
        if (!mbar_wait(kempty_bar(st), (k & 1u) ^ 1u, abort_flag)) break;
        mbar_expect_tx(kfull_bar(st), TC_KV_BYTES);
        tma_load_2d(base + k_off(st), tk, x0, y, kfull_bar(st));
        tma_load_2d(base + k_off(st) + TC_KV_BYTES / 2, tk, x0 + 64, y, kfull_bar(st));
        if (!mbar_wait(vempty_bar(st), (k & 1u) ^ 1u, abort_flag)) break;
        mbar_expect_tx(vfull_bar(st), TC_KV_BYTES);
        tma_load_2d(base + v_off(st), tv, x0, y, vfull_bar(st));
        tma_load_2d(base + v_off(st) + TC_KV_BYTES / 2, tv, x0 + 64, y, vfull_bar(st));
      }
      if (!waited) pdl_wait(KID_ATTN);
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0 && n_blocks > 0) {
      constexpr uint32_t IDESC_S = umma_idesc_bf16(128, TC_KB);
      constexpr uint32_t IDESC_O = umma_idesc_bf16_bmn(128, TC_DH);
      bool ok = mbar_wait(qfull_bar, 0u, abort_flag);
      tc_fence_after();
      // S of block b into score buffer b & 1: both query terms, A from tensor memory, one chain of 16 products. The
      // buffer held the probabilities of block b - 2, whose P V product has been issued before (program order): the
      // tensor pipe runs in issue order.
      auto issue_s = [&](int b) -> bool {
        const int st = b % TC_STAGES, i = b & 1;
        if (!mbar_wait(kfull_bar(st), (uint32_t)(b / TC_STAGES) & 1u, abort_flag)) return false;
        tc_fence_after();
        const uint64_t kd = umma_desc_sw128(base + k_off(st));
        const uint32_t d = tmem_base + TC_TM_S + (uint32_t)(i * TC_KB);
#pragma unroll
        for (int ks = 0; ks < TC_DH / 16; ++ks) {          // k-steps 0..3 in the first 64-column chunk of K, 4..7 in the second
          const uint64_t ko = (uint64_t)((ks >> 2) * (TC_KV_BYTES / 2 / 16) + 2 * (ks & 3));
          tc_mma_bf16_ta(d, tmem_base + TC_TM_Q + (uint32_t)(ks * 8), kd + ko, IDESC_S, ks > 0 ? 1u : 0u);
          tc_mma_bf16_ta(d, tmem_base + TC_TM_Q + 64u + (uint32_t)(ks * 8), kd + ko, IDESC_S, 1u);
        }
        tc_commit(sfull_bar(i));
        tc_commit(kempty_bar(st));                // the keys are done with once the scores are formed
        return true;
      };
      if (ok) ok = issue_s(0);
      for (int b = 0; b < n_blocks && ok; ++b) {
        if (b + 1 < n_blocks && !issue_s(b + 1)) { ok = false; break; }
        const int i = b & 1;
        if (!mbar_wait(pfull_bar(i), (uint32_t)(b >> 1) & 1u, abort_flag)) { ok = false; break; }
        if (!mbar_wait(vfull_bar(b % TC_STAGES), (uint32_t)(b / TC_STAGES) & 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t vaddr = base + v_off(b % TC_STAGES);
        const uint32_t pt = tmem_base + TC_TM_S + (uint32_t)(i * TC_KB);       // P_hi in its first 64 columns, P_lo in the next 64
        const uint32_t d = tmem_base + TC_TM_O;
#pragma unroll
        for (int ks = 0; ks < TC_KB / 16; ++ks)
          tc_mma_bf16_ta(d, pt + (uint32_t)(ks * 8), umma_desc_mn_sw128(vaddr + ks * 2048, TC_KV_BYTES / 2), IDESC_O, (b > 0 || ks > 0) ? 1u : 0u);
#pragma unroll
        for (int ks = 0; ks < TC_KB / 16; ++ks)
          tc_mma_bf16_ta(d, pt + 64u + (uint32_t)(ks * 8), umma_desc_mn_sw128(vaddr + ks * 2048, TC_KV_BYTES / 2), IDESC_O, 1u);
        tc_commit(pempty_bar);                    // O is at rest once this completes
        tc_commit(vempty_bar(b % TC_STAGES));     // the values are done with
      }
      if (ok) tc_commit(ofull_bar);
    }
  } else {
    // ------------------------------ softmax: two threads per query row, one per half of a block's 128 scores ------------------------------
    const int wi = warp - 2;                           // 0..7
    const int half = wi >> 2;                          // which 64 scores of a block (and which 64 output columns at the end)
    const int quad = warp & 3;                         // TMEM lane quadrant of this warp
    const int ql = quad * 32 + lane;                   // query row = TMEM lane
    const int st_i = threadIdx.x - 64;                 // 0..255 among the softmax threads
    const bool valid = ql < Qn;
    const bool warp_live = quad * 32 < Qn;             // at least one real query in this warp
    const int row = seq * A.rows_per_seq + (valid ? ql / A.group : 0);
    const int head = g * A.group + (valid ? ql % A.group : 0);
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    // ---- queries -> two bf16 terms, staged in shared memory (rows beyond Qn are zero) ----
    // Every thread takes eight 8-element pieces (piece i = row i / 16, column piece i % 16), four at a time. The loads
    // of a batch are unconditional (rows beyond Qn read the last real row and are discarded) and go out together, two
    // split-K planes at a time, so a batch costs one memory round trip per two planes instead of one per piece.
    for (int i0 = st_i; i0 < 128 * 16; i0 += 4 * 256) {
      float x[4][8];
      const float* src[4];
      bool in[4];
      const bool batch_live = (i0 - st_i) / 16 < Qn;             // the batch's lowest row: uniform over the threads
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + u * 256;
        const int r = i >> 4, c = i & 15;
        in[u] = r < Qn;
        const int rc = in[u] ? r : Qn - 1;
        src[u] = A.q32 + (size_t)(seq * A.rows_per_seq + rc / A.group) * A.q_ld + (g * A.group + rc % A.group) * TC_DH + c * 8;
#pragma unroll
        for (int e = 0; e < 8; ++e) x[u][e] = 0.f;
      }
      if (batch_live) {
        for (int sp = 0; sp < A.q_splits; sp += 2) {
          const bool two = sp + 1 < A.q_splits;
          float4 a0[4], b0[4], a1[4], b1[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const float* p0 = src[u] + (size_t)sp * A.q_plane;
            const float* p1 = src[u] + (size_t)(two ? sp + 1 : sp) * A.q_plane;
            a0[u] = ldcg4(p0); b0[u] = ldcg4(p0 + 4);
            a1[u] = ldcg4(p1); b1[u] = ldcg4(p1 + 4);
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {                            // planes added in index order
            x[u][0] += a0[u].x; x[u][1] += a0[u].y; x[u][2] += a0[u].z; x[u][3] += a0[u].w;
            x[u][4] += b0[u].x; x[u][5] += b0[u].y; x[u][6] += b0[u].z; x[u][7] += b0[u].w;
            if (two) {
              x[u][0] += a1[u].x; x[u][1] += a1[u].y; x[u][2] += a1[u].z; x[u][3] += a1[u].w;
              x[u][4] += b1[u].x; x[u][5] += b1[u].y; x[u][6] += b1[u].z; x[u][7] += b1[u].w;
            }
          }
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + u * 256;
        const int r = i >> 4, c = i & 15;
        uint32_t hi[4] = {0u, 0u, 0u, 0u}, lo[4] = {0u, 0u, 0u, 0u};
        if (in[u]) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const bf16 h0 = __float2bfloat16_rn(x[u][2 * e]), h1 = __float2bfloat16_rn(x[u][2 * e + 1]);
            hi[e] = pack_bf16(__bfloat162float(h0), __bfloat162float(h1));
            lo[e] = pack_bf16(x[u][2 * e] - __bfloat162float(h0), x[u][2 * e + 1] - __bfloat162float(h1));
          }
        }
        // staging: rows of 256 bytes, 16-byte piece c of row r at piece c ^ (r & 15) (a thread reads back its own row)
        const uint32_t off = (uint32_t)(r * 256 + ((c ^ (r & 15)) << 4));
        *reinterpret_cast<uint4*>(bp + oQhi + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
        *reinterpret_cast<uint4*>(bp + oQlo + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
      }
    }
    asm volatile("bar.sync 1, 256;" ::: "memory");
    // each term into tensor memory as the A operand of the score products: row = lane, elements 2 j and 2 j + 1 of the
    // row in column j. The threads of half 0 write the high-order term, those of half 1 the low-order one.
    {
      const uint8_t* src = bp + (half == 0 ? oQhi : oQlo) + ql * 256;
      const uint32_t tq = tmem_base + TC_TM_Q + lane_addr + (uint32_t)(half * 64);
#pragma unroll
      for (int c = 0; c < 16; c += 2) {
        const uint4 a0 = *reinterpret_cast<const uint4*>(src + (((c) ^ (ql & 15)) << 4));
        const uint4 a1 = *reinterpret_cast<const uint4*>(src + (((c + 1) ^ (ql & 15)) << 4));
        const uint32_t w8[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
        tc_st8(tq + (uint32_t)(c * 4), w8);
      }
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // the staging bytes become a ring stage
    tc_fence_before();
    mbar_arrive(qfull_bar);

    // tree segment: bit per slot this row may see (its ancestors and itself), 64 slots per word
    unsigned long long allow[4] = {0ull, 0ull, 0ull, 0ull};
    if (tree_part && valid) {
      for (int i = 0; i < A.nB; ++i) {
        const int slot = A.slotsB[(size_t)row * A.slots_ld + i];
        MOA_DEV_CHECK(slot >= 0 && slot < A.n_slots && slot < A.capB, A.status);
        if (slot >= 0 && slot < 256) allow[slot >> 6] |= 1ull << (slot & 63);
      }
    }
    float m_ref = -INFINITY, l_run = 0.f;
    const uint32_t tOh = tmem_base + TC_TM_O + lane_addr + (uint32_t)(half * 64);     // this thread's half of the output columns
    bool ok = true;          // false once any softmax thread has seen a wait fail; changes only at a barrier, for all at once
    bool fail = false;       // this thread's own failed waits since the last barrier
    for (int b = 0; b < n_blocks; ++b) {
      const int i = b & 1;
      if (!mbar_wait(sfull_bar(i), (uint32_t)(b >> 1) & 1u, abort_flag)) fail = true;
      tc_fence_after();
      const uint32_t tS = tmem_base + TC_TM_S + lane_addr + (uint32_t)(i * TC_KB);
      float s[64];
      if (warp_live) tc_ld64(tS + (uint32_t)(half * 64), s);        // this thread's 64 scores: one load, one wait
      const int n_blk = min(TC_KB, k_end - (k_begin + b * TC_KB));      // positions of this block inside the range
      const int n_in = max(0, min(64, n_blk - half * 64));              // of them in this thread's half
      if (n_blk < TC_KB) {
        // A ragged last block: positions beyond the range carry whatever the cache holds there. Their probabilities are
        // exactly zero, but zero times a non-finite stale value is not, so those V rows are cleared in shared memory,
        // once the block's values have landed (its scores being complete says nothing about them).
        if (!mbar_wait(vfull_bar(b % TC_STAGES), (uint32_t)(b / TC_STAGES) & 1u, abort_flag)) fail = true;
        uint8_t* v = bp + v_off(b % TC_STAGES);
        for (int j = st_i; j < (TC_KB - n_blk) * 16; j += 256) {
          const int r = n_blk + (j >> 4), c16 = j & 15;                  // row, 16-byte piece of its 256 bytes
          *reinterpret_cast<uint4*>(v + (c16 >> 3) * (TC_KV_BYTES / 2) + r * 128 + (c16 & 7) * 16) = make_uint4(0u, 0u, 0u, 0u);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      }
      // maximum of this thread's raw scores (the scale is positive and goes into the exponent's multiply-add)
      float mx = -INFINITY;
      if (warp_live) {
        if (tree_part) {                                   // the row sees its ancestors' slots and its own only
          const unsigned long long word = allow[(2 * b + half) & 3];
#pragma unroll
          for (int c = 0; c < 64; ++c) {
            s[c] = (c < n_in && ((word >> c) & 1ull)) ? s[c] : -INFINITY;
            mx = fmaxf(mx, s[c]);
          }
        } else if (n_in == 64) {
          float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};      // four chains instead of one
#pragma unroll
          for (int c = 0; c < 64; ++c) m4[c & 3] = fmaxf(m4[c & 3], s[c]);
          mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
        } else {
#pragma unroll
          for (int c = 0; c < 64; ++c) {
            s[c] = c < n_in ? s[c] : -INFINITY;
            mx = fmaxf(mx, s[c]);
          }
        }
      }
      // the row's two threads exchange their maxima (buffers alternate, so one barrier per block is enough); behind the
      // barrier both have their scores in registers, and the probabilities may overwrite either half of the buffer
      xm[(i * 2 + half) * 128 + ql] = mx;
      if (tc_bar_any(fail || *abort_flag != 0)) { ok = false; break; }
      mx = fmaxf(mx, xm[(i * 2 + (half ^ 1)) * 128 + ql]);
      const float m_blk = mx * A.scale_log2;
      float f = 1.f;
      if (warp_live) {
        if (m_ref == -INFINITY) {
          m_ref = m_blk;                                   // nothing accumulated yet for this row
        } else if (m_blk > m_ref + TC_RESCALE_LOG2) {
          f = ex2_approx(m_ref - m_blk);
          m_ref = m_blk;
          l_run *= f;
        }
      }
      if (b > 0 && warp_live && __any_sync(0xffffffffu, f != 1.f)) {
        // rare: a row's accumulator moves to a new reference; the previous product must have left the tensor cores
        if (!mbar_wait(pempty_bar, ((uint32_t)b & 1u) ^ 1u, abort_flag)) fail = true;   // seen by all at the next barrier
        tc_fence_after();
#pragma unroll 1
        for (int c = 0; c < 64 && !fail; c += 16) {
          float o[16];
          tc_ld16(tOh + (uint32_t)c, o);
#pragma unroll
          for (int e = 0; e < 16; ++e) o[e] *= f;
          tc_st16(tOh + (uint32_t)c, o);
        }
      }
      if (warp_live) {
        // probabilities as two bf16 terms over the scores: P_hi in columns 0..63 of the buffer (two positions per column),
        // P_lo in 64..127; this thread's 64 positions take 32 columns of each
        const float msub = m_ref == -INFINITY ? 0.f : m_ref;
        float rs[2] = {0.f, 0.f};
#pragma unroll
        for (int c = 0; c < 64; c += 16) {
          uint32_t hi[8], lo[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const float p0 = ex2_approx(fmaf(s[c + 2 * e], A.scale_log2, -msub)), p1 = ex2_approx(fmaf(s[c + 2 * e + 1], A.scale_log2, -msub));
            rs[0] += p0;
            rs[1] += p1;
            const uint32_t h = pack_bf16(p0, p1);
            hi[e] = h;
            lo[e] = pack_bf16(p0 - __uint_as_float(h << 16), p1 - __uint_as_float(h & 0xffff0000u));
          }
          tc_st8(tS + (uint32_t)(half * 32 + c / 2), hi);
          tc_st8(tS + 64u + (uint32_t)(half * 32 + c / 2), lo);
        }
        l_run += rs[0] + rs[1];
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      }
      tc_fence_before();
      mbar_arrive(pfull_bar(i));
    }
    // ---- the range's result: (max, sum, unnormalised output) per query, or the normalised rows when this range is the
    //      attention's only part; each of the row's two threads takes 64 output columns ----
    if (ok && n_blocks > 0 && !mbar_wait(ofull_bar, 0u, abort_flag)) fail = true;
    tc_fence_after();
    if (!ok || fail) *abort_flag = 1;
    (void)tc_bar_any(false);                               // every exchange read of the loop is behind us
    xm[half * 128 + ql] = l_run;
    const bool dead = tc_bar_any(!ok || fail || *abort_flag != 0);       // the same for all: the TMEM loads below are warp-wide
    const float L = l_run + xm[(half ^ 1) * 128 + ql];
    const bool seen = n_blocks > 0 && m_ref != -INFINITY;
    const size_t pidx = ((size_t)row * A.hq + head) * A.n_parts + part;
    const float inv = (seen && L > 0.f) ? 1.f / L : 0.f;
#pragma unroll 1
    for (int c = 0; c < 64; c += 16) {
      float o[16];
      if (n_blocks > 0 && warp_live && !dead) {
        tc_ld16(tOh + (uint32_t)c, o);
      } else {
#pragma unroll
        for (int e = 0; e < 16; ++e) o[e] = 0.f;
      }
      if (!valid) continue;
      if (!seen) {
#pragma unroll
        for (int e = 0; e < 16; ++e) o[e] = 0.f;
      }
      const int col = half * 64 + c;
      if (A.n_parts == 1) {
        bf16* dst = A.out + ((size_t)row * A.hq + head) * TC_DH + col;
        bf16* dlo = A.out + ((size_t)(A.out_lo + row) * A.hq + head) * TC_DH + col;
        uint32_t hi[8], lo[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float a0 = o[2 * e] * inv, a1 = o[2 * e + 1] * inv;
          const bf16 h0 = __float2bfloat16_rn(a0), h1 = __float2bfloat16_rn(a1);
          hi[e] = pack_bf16(__bfloat162float(h0), __bfloat162float(h1));
          lo[e] = pack_bf16(a0 - __bfloat162float(h0), a1 - __bfloat162float(h1));
        }
        *reinterpret_cast<uint4*>(dst) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
        *reinterpret_cast<uint4*>(dst + 8) = make_uint4(hi[4], hi[5], hi[6], hi[7]);
        if (A.out_lo > 0) {
          *reinterpret_cast<uint4*>(dlo) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
          *reinterpret_cast<uint4*>(dlo + 8) = make_uint4(lo[4], lo[5], lo[6], lo[7]);
        }
      } else {
        float* dst = A.part_o + pidx * TC_DH + col;
#pragma unroll
        for (int e = 0; e < 16; e += 4) *reinterpret_cast<float4*>(dst + e) = make_float4(o[e], o[e + 1], o[e + 2], o[e + 3]);
      }
    }
    if (half == 0 && valid && A.n_parts > 1) {
      A.part_ml[pidx * 2 + 0] = seen ? m_ref : -INFINITY;      // log2 domain, as attn_combine_kernel expects
      A.part_ml[pidx * 2 + 1] = seen ? L : 0.f;
    }
  }

  // ------------------------------ teardown ------------------------------
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
  if (threadIdx.x == 0 && *abort_flag && A.status) atomicMax(A.status, DEV_ERR_TIMEOUT);
}

}  // namespace moa
