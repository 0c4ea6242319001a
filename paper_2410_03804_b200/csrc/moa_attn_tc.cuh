// Attention over a long cache segment on the 5th-generation tensor cores (sm_100a, head size 128).
//
// The split-KV kernel of moa_attn.cuh issues its products with mma.sync from a handful of warps, and at long
// context (tens of thousands of cached positions per kv head) it is bound by that instruction stream, not by HBM.
// Here one CTA per (sequence, kv head, key range) keeps all queries that share the kv head -- (rows of the
// sequence) x (query heads of the group), at most 128 -- as the M = 128 operand in shared memory and streams the
// cache through a TMA ring of 64-position blocks:
//   warp 0      TMA producer: K block [64, 128] and V block [64, 128] per stage (128-byte swizzle)
//   warp 1      one thread issues tcgen05.mma:  S = Q_hi K^T + Q_lo K^T   (A = Q, B = K, both K-major; fp32 in TMEM)
//                                               O += P_hi V + P_lo V      (A = P from shared memory, K-major;
//                                                                          B = V as it lies in the cache: MN-major)
//   warps 2..5  softmax: thread t owns query row t (TMEM lane t): reads its 64 scores, keeps the running maximum
//               and sum in the log2 domain, writes the probabilities as two bf16 terms into the swizzled P tiles.
// The output accumulator stays in TMEM for the whole key range; it is rescaled only when a row's maximum has grown
// by more than 2^8 since the last rescale (probabilities then stay below 256, well inside fp32 / bf16 range), so
// the rescale -- a TMEM load, multiply, store of the row -- happens a few times per range, not per block.
// Each CTA leaves (max, sum, unnormalised output) per query for attn_combine_kernel, in the layout of the split-KV
// kernel, so the tree part of a self-attention (masked per row, a few dozen slots) still runs there and the parts
// are merged together. Queries arrive in fp32 and enter as two bf16 terms, as in the split-KV kernel.
// Every mbarrier wait is bounded; on expiry the CTA raises the abort flag, drains, frees TMEM and reports
// DEV_ERR_TIMEOUT through the status word.
#pragma once
#include "moa_attn.cuh"
#include "moa_wstream.cuh"

namespace moa {

constexpr int TC_KB = 64;                 // cache positions per block
constexpr int TC_DH = 128;
constexpr int TC_STAGES = 3;
constexpr int TC_THREADS = 192;
constexpr int TC_Q_BYTES = 128 * TC_DH * 2;           // one query term: two 64-column chunks of [128 rows x 128 B]
constexpr int TC_P_BYTES = 128 * TC_KB * 2;           // one probability term: [128 rows x 128 B]
constexpr int TC_KV_BYTES = TC_KB * TC_DH * 2;        // K (or V) block: two 64-column chunks of [64 rows x 128 B]
constexpr int TC_STAGE_BYTES = 2 * TC_KV_BYTES;
constexpr int TC_SMEM_BYTES = 2 * TC_Q_BYTES + 2 * TC_P_BYTES + TC_STAGES * TC_STAGE_BYTES + 1024 + 256;
constexpr float TC_RESCALE_LOG2 = 8.f;

struct AttnTcParams {
  CUtensorMap tmK, tmV;      // cache [positions of all sequences, hkv * 128], box 64 columns x 64 positions, swizzle 128B
  AttnParams a;              // queries (fp32), lengths, part buffers; n_parts counts the tree part too
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

// Byte offset of element (row, col) in a tile of 128-byte rows whose 16-byte chunks are XORed with row & 7.
__device__ __forceinline__ uint32_t sw128_off(int row, int col) {
  return (uint32_t)(row * 128 + ((((col >> 3) ^ (row & 7))) << 4) + (col & 7) * 2);
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

__global__ void __launch_bounds__(TC_THREADS, 1) attn_tc_kernel(const __grid_constant__ AttnTcParams P) {
  extern __shared__ uint8_t tc_smem_raw[];
  const uint32_t base = (smem_u32(tc_smem_raw) + 1023u) & ~1023u;
  uint8_t* bp = tc_smem_raw + (base - smem_u32(tc_smem_raw));
  constexpr uint32_t oQhi = 0, oQlo = TC_Q_BYTES, oPhi = 2 * TC_Q_BYTES, oPlo = oPhi + TC_P_BYTES, oKV = oPlo + TC_P_BYTES,
                     oBar = oKV + TC_STAGES * TC_STAGE_BYTES;
  const uint32_t bar0 = base + oBar;
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (TC_STAGES + s); };
  auto sfull_bar = [&](int i) { return bar0 + 8u * (2 * TC_STAGES + i); };
  auto sempty_bar = [&](int i) { return bar0 + 8u * (2 * TC_STAGES + 2 + i); };
  const uint32_t pfull_bar = bar0 + 8u * (2 * TC_STAGES + 4), pempty_bar = pfull_bar + 8u, qfull_bar = pfull_bar + 16u,
                 ofull_bar = pfull_bar + 24u;
  uint32_t* tmem_slot = (uint32_t*)(bp + oBar + 8 * (2 * TC_STAGES + 8));
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

  const AttnParams& A = P.a;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int part = blockIdx.x, g = blockIdx.y, seq = blockIdx.z;
  const int Qn = A.rows_per_seq * A.group;           // <= 128, checked by the host
  pdl_trigger();

  if (threadIdx.x == 0) {
    for (int s = 0; s < TC_STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(sfull_bar(i), 1); mbar_init(sempty_bar(i), 128); }
    mbar_init(pfull_bar, 128);
    mbar_init(pempty_bar, 1);
    mbar_init(qfull_bar, 128);
    mbar_init(ofull_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(256u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tS = tmem_base, tO = tmem_base + 128u;          // S buffers at columns 0 and 64, O at 128..255

  // the cache was written by earlier kernels of the stream, and so were the queries
  pdl_wait(KID_ATTN);
  const int len = A.lenA ? A.lenA[seq] : A.nA_fixed;
  const int blocks = (len + TC_KB - 1) / TC_KB;
  const int b0 = (int)(((long long)part * blocks) / A.n_split), b1 = (int)(((long long)(part + 1) * blocks) / A.n_split);
  const int k_begin = b0 * TC_KB, k_end = min(b1 * TC_KB, len);
  const int n_blocks = b1 - b0;

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      const int x0 = g * TC_DH;
      for (int b = 0; b < n_blocks; ++b) {
        const int st = b % TC_STAGES;
        const uint32_t k = (uint32_t)(b / TC_STAGES);
        if (!mbar_wait(empty_bar(st), (k & 1u) ^ 1u, abort_flag)) break;
        mbar_expect_tx(full_bar(st), TC_STAGE_BYTES);
        const uint32_t dst = base + oKV + st * TC_STAGE_BYTES;
        const int y = seq * A.capA + k_begin + b * TC_KB;
        tma_load_2d(dst, &P.tmK, x0, y, full_bar(st));
        tma_load_2d(dst + TC_KV_BYTES / 2, &P.tmK, x0 + 64, y, full_bar(st));
        tma_load_2d(dst + TC_KV_BYTES, &P.tmV, x0, y, full_bar(st));
        tma_load_2d(dst + TC_KV_BYTES + TC_KV_BYTES / 2, &P.tmV, x0 + 64, y, full_bar(st));
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0 && n_blocks > 0) {
      constexpr uint32_t IDESC_S = umma_idesc_bf16(128, TC_KB);
      constexpr uint32_t IDESC_O = umma_idesc_bf16_bmn(128, TC_DH);
      bool ok = mbar_wait(qfull_bar, 0u, abort_flag);
      tc_fence_after();
      auto issue_s = [&](int b) -> bool {
        const int st = b % TC_STAGES, i = b & 1;
        if (!mbar_wait(full_bar(st), (uint32_t)(b / TC_STAGES) & 1u, abort_flag)) return false;
        if (!mbar_wait(sempty_bar(i), ((uint32_t)(b >> 1) & 1u) ^ 1u, abort_flag)) return false;
        tc_fence_after();
        const uint32_t kaddr = base + oKV + st * TC_STAGE_BYTES;
#pragma unroll
        for (int ks = 0; ks < TC_DH / 16; ++ks) {
          const uint64_t bd = umma_desc_sw128(kaddr + (ks >> 2) * (TC_KV_BYTES / 2)) + 2u * (ks & 3);
          tc_mma_bf16(tS + (uint32_t)(i * TC_KB), umma_desc_sw128(base + oQhi + (ks >> 2) * (TC_Q_BYTES / 2)) + 2u * (ks & 3), bd, IDESC_S,
                      ks > 0 ? 1u : 0u);
        }
#pragma unroll
        for (int ks = 0; ks < TC_DH / 16; ++ks) {
          const uint64_t bd = umma_desc_sw128(kaddr + (ks >> 2) * (TC_KV_BYTES / 2)) + 2u * (ks & 3);
          tc_mma_bf16(tS + (uint32_t)(i * TC_KB), umma_desc_sw128(base + oQlo + (ks >> 2) * (TC_Q_BYTES / 2)) + 2u * (ks & 3), bd, IDESC_S, 1u);
        }
        tc_commit(sfull_bar(i));
        return true;
      };
      if (ok) ok = issue_s(0);
      for (int b = 0; b < n_blocks && ok; ++b) {
        if (b + 1 < n_blocks && !issue_s(b + 1)) { ok = false; break; }
        if (!mbar_wait(pfull_bar, (uint32_t)b & 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t vaddr = base + oKV + (b % TC_STAGES) * TC_STAGE_BYTES + TC_KV_BYTES;
#pragma unroll
        for (int ks = 0; ks < TC_KB / 16; ++ks)
          tc_mma_bf16(tO, umma_desc_sw128(base + oPhi) + 2u * ks, umma_desc_mn_sw128(vaddr + ks * 2048, TC_KV_BYTES / 2), IDESC_O,
                      (b > 0 || ks > 0) ? 1u : 0u);
#pragma unroll
        for (int ks = 0; ks < TC_KB / 16; ++ks)
          tc_mma_bf16(tO, umma_desc_sw128(base + oPlo) + 2u * ks, umma_desc_mn_sw128(vaddr + ks * 2048, TC_KV_BYTES / 2), IDESC_O, 1u);
        tc_commit(pempty_bar);                    // P may be overwritten, O may be rescaled
        tc_commit(empty_bar(b % TC_STAGES));      // the stage's K and V are done with
      }
      if (ok) tc_commit(ofull_bar);
    }
  } else {
    // ------------------------------ softmax: one thread per query row ------------------------------
    const int quad = warp & 3;                         // TMEM lane quadrant of this warp
    const int ql = quad * 32 + lane;                   // query row = TMEM lane
    const int st_i = threadIdx.x - 64;                 // 0..127 among these threads
    const bool valid = ql < Qn;
    const bool warp_live = quad * 32 < Qn;             // at least one real query in this warp
    const int row = seq * A.rows_per_seq + (valid ? ql / A.group : 0);
    const int head = g * A.group + (valid ? ql % A.group : 0);
    // ---- queries -> two bf16 terms in shared memory (rows beyond Qn are zero) ----
    for (int i0 = st_i; i0 < 128 * 16; i0 += 4 * 128) {
      float x[4][8];
      bool in[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + u * 128;
        const int r = i >> 4, c = i & 15;
        in[u] = r < Qn;
        if (in[u])
          load8_planes(A.q32 + (size_t)(seq * A.rows_per_seq + r / A.group) * A.q_ld + (g * A.group + r % A.group) * TC_DH + c * 8,
                       A.q_splits, A.q_plane, x[u]);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + u * 128;
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
        const uint32_t off = (uint32_t)((c >> 3) * (TC_Q_BYTES / 2)) + sw128_off(r, (c & 7) * 8);
        *reinterpret_cast<uint4*>(bp + oQhi + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
        *reinterpret_cast<uint4*>(bp + oQlo + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
      }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    mbar_arrive(qfull_bar);

    float m_ref = -INFINITY, l_run = 0.f;
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    bool ok = true;
    for (int b = 0; b < n_blocks && ok; ++b) {
      const int i = b & 1;
      if (!mbar_wait(sfull_bar(i), (uint32_t)(b >> 1) & 1u, abort_flag)) { ok = false; break; }
      tc_fence_after();
      float s[TC_KB];
      if (warp_live) {
#pragma unroll
        for (int c = 0; c < TC_KB; c += 16) tc_ld16(tS + lane_addr + (uint32_t)(i * TC_KB + c), s + c);
      }
      tc_fence_before();
      mbar_arrive(sempty_bar(i));
      {
        // A ragged last block: positions beyond the range carry whatever the cache holds there. Their probabilities are
        // exactly zero, but zero times a non-finite stale value is not, so those V rows are cleared in shared memory
        // (the block has landed: its scores are complete).
        const int n_keep = min(TC_KB, k_end - (k_begin + b * TC_KB));
        if (n_keep < TC_KB) {
          uint8_t* v = bp + oKV + (b % TC_STAGES) * TC_STAGE_BYTES + TC_KV_BYTES;
          for (int j = st_i; j < (TC_KB - n_keep) * 16; j += 128) {
            const int r = n_keep + (j >> 4), c16 = j & 15;                   // row, 16-byte piece of its 256 bytes
            *reinterpret_cast<uint4*>(v + (c16 >> 3) * (TC_KV_BYTES / 2) + r * 128 + (c16 & 7) * 16) = make_uint4(0u, 0u, 0u, 0u);
          }
        }
      }
      // block maximum of the raw scores (the scale is positive and goes into the exponent's multiply-add)
      const int n_in = min(TC_KB, k_end - (k_begin + b * TC_KB));       // positions of this block inside the range
      float mx = -INFINITY;
      if (warp_live) {
        if (n_in == TC_KB) {
#pragma unroll
          for (int c = 0; c < TC_KB; ++c) mx = fmaxf(mx, s[c]);
        } else {
#pragma unroll
          for (int c = 0; c < TC_KB; ++c) {
            s[c] = c < n_in ? s[c] : -INFINITY;
            mx = fmaxf(mx, s[c]);
          }
        }
      }
      const float m_blk = mx * A.scale_log2;
      // PV of the block before this one must be done: P is free and O is at rest
      if (!mbar_wait(pempty_bar, (uint32_t)(b - 1) & 1u, abort_flag)) { ok = false; break; }
      tc_fence_after();
      if (warp_live) {
        float f = 1.f;
        if (m_ref == -INFINITY) {
          m_ref = m_blk;                                   // nothing accumulated yet for this row
        } else if (m_blk > m_ref + TC_RESCALE_LOG2) {
          f = ex2_approx(m_ref - m_blk);
          m_ref = m_blk;
          l_run *= f;
        }
        if (b > 0 && __any_sync(0xffffffffu, f != 1.f)) {  // rare: the row's output accumulator moves to the new reference
#pragma unroll 1
          for (int c = 0; c < TC_DH; c += 16) {
            float o[16];
            tc_ld16(tO + lane_addr + (uint32_t)c, o);
#pragma unroll
            for (int e = 0; e < 16; ++e) o[e] *= f;
            tc_st16(tO + lane_addr + (uint32_t)c, o);
          }
          asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        }
        const float msub = m_ref == -INFINITY ? 0.f : m_ref;
        float rs = 0.f;
#pragma unroll
        for (int c = 0; c < TC_KB; c += 8) {
          uint32_t hi[4], lo[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float p0 = ex2_approx(fmaf(s[c + 2 * e], A.scale_log2, -msub)), p1 = ex2_approx(fmaf(s[c + 2 * e + 1], A.scale_log2, -msub));
            rs += p0 + p1;
            const uint32_t h = pack_bf16(p0, p1);
            hi[e] = h;
            lo[e] = pack_bf16(p0 - __uint_as_float(h << 16), p1 - __uint_as_float(h & 0xffff0000u));
          }
          const uint32_t off = sw128_off(ql, c);
          *reinterpret_cast<uint4*>(bp + oPhi + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
          *reinterpret_cast<uint4*>(bp + oPlo + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        }
        l_run += rs;
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      tc_fence_before();
      mbar_arrive(pfull_bar);
    }
    // ---- the range's result: (max, sum, unnormalised output) per query, or the normalised rows when this is the only part ----
    if (ok && n_blocks > 0) ok = mbar_wait(ofull_bar, 0u, abort_flag);
    tc_fence_after();
    if (ok && warp_live) {
      const size_t pidx = ((size_t)row * A.hq + head) * A.n_parts + part;
      const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
#pragma unroll 1
      for (int c = 0; c < TC_DH; c += 16) {
        float o[16];
        if (n_blocks > 0) {
          tc_ld16(tO + lane_addr + (uint32_t)c, o);
        } else {
#pragma unroll
          for (int e = 0; e < 16; ++e) o[e] = 0.f;
        }
        if (!valid) continue;
        if (A.n_parts == 1) {
          bf16* dst = A.out + ((size_t)row * A.hq + head) * TC_DH + c;
          bf16* dlo = A.out + ((size_t)(A.out_lo + row) * A.hq + head) * TC_DH + c;
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
          float* dst = A.part_o + pidx * TC_DH + c;
#pragma unroll
          for (int e = 0; e < 16; e += 4) *reinterpret_cast<float4*>(dst + e) = make_float4(o[e], o[e + 1], o[e + 2], o[e + 3]);
        }
      }
      if (valid && A.n_parts > 1) {
        A.part_ml[pidx * 2 + 0] = m_ref;           // log2 domain, as attn_combine_kernel expects
        A.part_ml[pidx * 2 + 1] = l_run;
      }
    }
  }

  // ------------------------------ teardown ------------------------------
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256u) : "memory");
  }
  if (threadIdx.x == 0 && *abort_flag && A.status) atomicMax(A.status, DEV_ERR_TIMEOUT);
}

}  // namespace moa
