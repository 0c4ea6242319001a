// Phase machine, part 3: the attention phase and the merge of its parts.
//
// Same scheme as attn_split_kernel (moa_attn.cuh): one unit = (sequence, kv head, query tile, part); all
// queries sharing a kv head are stacked in the M dimension of mma.sync.m16n8k16; keys / values stream
// through shared memory in blocks of 32 positions, up to four blocks in flight. Queries that arrive in fp32
// are split into two bf16 terms (and so are the probabilities), so scores and outputs carry them at ~16 bits.
#pragma once
#include "moa_pm_common.cuh"

namespace moa {

//  p[0] q bf16 (or null), p[1] q32 fp32 (or null; may be split planes), p[2] kA, p[3] vA, p[4] lenA (or null),
//  p[5] kB, p[6] vB, p[7] slotsB, p[8] part_o, p[9] part_ml, p[10] out (X buffer)
//  i[0] q_ld, i[1] hq, i[2] hkv, i[3] rows_per_seq, i[4] capA, i[5] posA_ld, i[6] nA_fixed, i[7] capB,
//  i[8] slots_ld, i[9] nB, i[10] n_slots, i[11] n_split, i[12] q_splits, i[13] out lo_rows, i[14] head size;
//  rows = R, cols = n_seq;  f[0] scale_log2;  q plane stride = the planes of GEMM op.gemm when op.gemm >= 0
template <int DH>
__device__ __noinline__ void pm_attention(PmSmem& S, const PmOp& op, uint8_t* smem_gen, uint32_t smem_sh, int wt) {
  constexpr int CH = DH / 8, KS = DH / 16, TILE_BYTES = PM_KB * DH * 2, QT = PM_WWARPS * 16;
  const bf16* q16 = (const bf16*)op.p[0];
  const float* q32 = (const float*)op.p[1];
  const bf16* kA = (const bf16*)op.p[2];
  const bf16* vA = (const bf16*)op.p[3];
  const int* lenA = (const int*)op.p[4];
  const bf16* kB = (const bf16*)op.p[5];
  const bf16* vB = (const bf16*)op.p[6];
  const int* slotsB = (const int*)op.p[7];
  float* part_o = (float*)op.p[8];
  float* part_ml = (float*)op.p[9];
  bf16* out = (bf16*)op.p[10];
  const int q_ld = op.i[0], hq = op.i[1], hkv = op.i[2], rows_per_seq = op.i[3], capA = op.i[4], posA_ld = op.i[5];
  const int nA_fixed = op.i[6], capB = op.i[7], slots_ld = op.i[8], nB = op.i[9], n_slots = op.i[10];
  const int n_split = op.i[11], q_splits = op.i[12], out_lo = op.i[13];
  const int n_seq = op.cols;
  const float scale_log2 = op.f[0];
  const size_t q_plane = op.gemm >= 0 ? S.g[op.gemm].plane : 0;
  const bool qsplit = q32 != nullptr;
  const int group = hq / hkv;
  const int Qn = rows_per_seq * group;
  const int q_tiles = (Qn + QT - 1) / QT;
  const bool has_tree = kB != nullptr && nB > 0;
  const int n_parts = n_split + (has_tree ? 1 : 0);
  const int q_rows = (Qn < QT ? ((Qn + 15) & ~15) : QT);     // rows of the Q tile actually staged
  const uint32_t sQ = smem_sh, sQlo = sQ + q_rows * DH * 2;
  const uint32_t sKV = sQlo + q_rows * DH * 2;
  unsigned long long* allow =
      reinterpret_cast<unsigned long long*>(smem_gen + 2 * q_rows * DH * 2 + 2 * PM_KVST * TILE_BYTES);
  const int warp = wt >> 5, lane = wt & 31;
  const int gq = lane >> 2, tq = lane & 3;
  const long long n_units = (long long)n_seq * hkv * q_tiles * n_parts;

  for (long long unit = blockIdx.x; unit < n_units; unit += gridDim.x) {
    const int part = (int)(unit % n_parts);
    long long t = unit / n_parts;
    const int qt = (int)(t % q_tiles); t /= q_tiles;
    const int g = (int)(t % hkv);
    const int seq = (int)(t / hkv);
    const bool tree_part = part >= n_split;
    int k_begin, k_end;
    wbar();                                   // the previous unit is done with shared memory
    if (!tree_part) {
      const int len = lenA ? __ldcg(lenA + seq) : nA_fixed;
      const int blocks = (len + PM_KB - 1) / PM_KB;
      const int b0 = (int)(((long long)part * blocks) / n_split), b1 = (int)(((long long)(part + 1) * blocks) / n_split);
      k_begin = b0 * PM_KB;
      k_end = min(b1 * PM_KB, len);
    } else {
      k_begin = 0;
      k_end = n_slots;
      if (wt < 64) allow[wt] = 0ull;
      wbar();
      for (int idx = wt; idx < min(rows_per_seq, 16) * nB; idx += PM_WORKERS) {     // one ancestor slot per thread
        const int rl = idx / nB, i = idx - rl * nB;
        const int slot = __ldcg(slotsB + (size_t)(seq * rows_per_seq + rl) * slots_ld + i);
        if (slot >= 0 && slot < 256) atomicOr(&allow[rl * 4 + (slot >> 6)], 1ull << (slot & 63));
      }
    }
    auto load_block = [&](int stage, int k0) {
      const uint32_t sK = sKV + stage * 2 * TILE_BYTES, sV = sK + TILE_BYTES;
      for (int i = wt; i < PM_KB * CH; i += PM_WORKERS) {
        const int kr = i / CH, c = i - kr * CH;
        const int j = k0 + kr;
        const bool valid = j < k_end;
        size_t off;
        if (!tree_part) off = ((size_t)seq * capA + (valid ? j : 0)) * posA_ld + g * DH + c * 8;
        else off = (((size_t)seq * capB + (valid ? j : 0)) * hkv + g) * DH + c * 8;
        cp_async16(sK + tile_off<DH>(kr, c), (tree_part ? kB : kA) + off, valid);
        cp_async16(sV + tile_off<DH>(kr, c), (tree_part ? vB : vA) + off, valid);
      }
    };
    const int n_blocks = (k_end - k_begin + PM_KB - 1) / PM_KB;
#pragma unroll
    for (int pb = 0; pb < PM_KVST; ++pb) {    // the first blocks all go out at once: one memory round trip
      if (pb < n_blocks) load_block(pb, k_begin + pb * PM_KB);
      cp_async_commit();
    }
    // ---- Q tile -> shared ----
    for (int i = wt; i < q_rows * CH; i += PM_WORKERS) {
      const int ql = i / CH, c = i - ql * CH;
      const int qi = qt * QT + ql;
      const bool valid = qi < Qn;
      const int row = seq * rows_per_seq + (valid ? qi / group : 0);
      const int head = g * group + (valid ? qi % group : 0);
      uint32_t hi[4] = {0u, 0u, 0u, 0u}, lo[4] = {0u, 0u, 0u, 0u};
      if (valid) {
        if (qsplit) {
          float x[8];
          load8_planes(q32 + (size_t)row * q_ld + head * DH + c * 8, q_splits, q_plane, x);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const bf16 h0 = __float2bfloat16_rn(x[2 * e]), h1 = __float2bfloat16_rn(x[2 * e + 1]);
            hi[e] = pack_bf16(__bfloat162float(h0), __bfloat162float(h1));
            lo[e] = pack_bf16(x[2 * e] - __bfloat162float(h0), x[2 * e + 1] - __bfloat162float(h1));
          }
        } else {
          const uint4 u = __ldcg(reinterpret_cast<const uint4*>(q16 + (size_t)row * q_ld + head * DH + c * 8));
          hi[0] = u.x; hi[1] = u.y; hi[2] = u.z; hi[3] = u.w;
        }
      }
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sQ + tile_off<DH>(ql, c)), "r"(hi[0]), "r"(hi[1]),
                   "r"(hi[2]), "r"(hi[3]) : "memory");
      if (qsplit)
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sQlo + tile_off<DH>(ql, c)), "r"(lo[0]),
                     "r"(lo[1]), "r"(lo[2]), "r"(lo[3]) : "memory");
    }
    wbar();                                   // Q tile (and the tree bitmaps) are in place
    const bool active = warp * 16 < q_rows;   // warps beyond the staged queries only keep the barriers company

    uint32_t qf[KS][4];
    if (active) {
      const int row = warp * 16 + (lane & 15);
#pragma unroll
      for (int ks = 0; ks < KS; ++ks)
        ldsm_x4(sQ + tile_off<DH>(row, ks * 2 + (lane >> 4)), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
    }
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    float o[DH / 8][4];
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    int seqrow[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int qi = qt * QT + warp * 16 + gq + 8 * h;
      seqrow[h] = qi < Qn ? qi / group : 0;
    }
    for (int blk = 0; blk < n_blocks; ++blk) {
      const int stage = blk % PM_KVST;
      cp_async_wait<PM_KVST - 1>();           // PM_KVST + blk groups committed so far: block blk has landed
      wbar();
      if (active) {
        const uint32_t sK = sKV + stage * 2 * TILE_BYTES, sV = sK + TILE_BYTES;
        const int k0 = k_begin + blk * PM_KB;
        float s[PM_KB / 8][4];
#pragma unroll
        for (int nt = 0; nt < PM_KB / 8; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
        for (int ks2 = 0; ks2 < KS / 2; ++ks2) {
          uint32_t ql0[4] = {0u, 0u, 0u, 0u}, ql1[4] = {0u, 0u, 0u, 0u};
          if (qsplit) {
            const int row = warp * 16 + (lane & 15);
            ldsm_x4(sQlo + tile_off<DH>(row, (2 * ks2) * 2 + (lane >> 4)), ql0[0], ql0[1], ql0[2], ql0[3]);
            ldsm_x4(sQlo + tile_off<DH>(row, (2 * ks2 + 1) * 2 + (lane >> 4)), ql1[0], ql1[1], ql1[2], ql1[3]);
          }
#pragma unroll
          for (int nt = 0; nt < PM_KB / 8; ++nt) {
            uint32_t b0, b1, b2, b3;
            ldsm_x4(sK + tile_off<DH>(nt * 8 + (lane & 7), ks2 * 4 + (lane >> 3)), b0, b1, b2, b3);
            mma_bf16_16816(s[nt], qf[2 * ks2], b0, b1);
            mma_bf16_16816(s[nt], qf[2 * ks2 + 1], b2, b3);
            if (qsplit) {
              mma_bf16_16816(s[nt], ql0, b0, b1);
              mma_bf16_16816(s[nt], ql1, b2, b3);
            }
          }
        }
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nt = 0; nt < PM_KB / 8; ++nt) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int key = k0 + nt * 8 + tq * 2 + (e & 1);
            const int h = e >> 1;
            bool ok = key < k_end;
            if (tree_part && ok) ok = (allow[seqrow[h] * 4 + (key >> 6)] >> (key & 63)) & 1ull;
            const float v = ok ? s[nt][e] * scale_log2 : -INFINITY;
            s[nt][e] = v;
            mx[h] = fmaxf(mx[h], v);
          }
        }
        float corr[2], msub[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
          mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
          const float mn = fmaxf(m_run[h], mx[h]);
          corr[h] = (m_run[h] == -INFINITY) ? 0.f : exp2f(m_run[h] - mn);
          msub[h] = (mn == -INFINITY) ? 0.f : mn;
          m_run[h] = mn;
        }
        float rs[2] = {0.f, 0.f};
        uint32_t pf[PM_KB / 16][4], pl[PM_KB / 16][4];   // probabilities as hi (+ lo) bf16 terms
#pragma unroll
        for (int nt = 0; nt < PM_KB / 8; ++nt) {
          const float p0 = exp2f(s[nt][0] - msub[0]), p1 = exp2f(s[nt][1] - msub[0]);
          const float p2 = exp2f(s[nt][2] - msub[1]), p3 = exp2f(s[nt][3] - msub[1]);
          rs[0] += p0 + p1;
          rs[1] += p2 + p3;
          const bf16 h0 = __float2bfloat16_rn(p0), h1 = __float2bfloat16_rn(p1), h2 = __float2bfloat16_rn(p2),
                     h3 = __float2bfloat16_rn(p3);
          pf[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(__bfloat162float(h0), __bfloat162float(h1));
          pf[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(__bfloat162float(h2), __bfloat162float(h3));
          pl[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(p0 - __bfloat162float(h0), p1 - __bfloat162float(h1));
          pl[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p2 - __bfloat162float(h2), p3 - __bfloat162float(h3));
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) l_run[h] = l_run[h] * corr[h] + rs[h];
#pragma unroll
        for (int i = 0; i < DH / 8; ++i) {
          o[i][0] *= corr[0]; o[i][1] *= corr[0];
          o[i][2] *= corr[1]; o[i][3] *= corr[1];
        }
#pragma unroll
        for (int kk = 0; kk < PM_KB / 16; ++kk) {
#pragma unroll
          for (int n2 = 0; n2 < DH / 16; ++n2) {
            uint32_t b0, b1, b2, b3;
            const int key = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
            ldsm_x4_t(sV + tile_off<DH>(key, n2 * 2 + (lane >> 4)), b0, b1, b2, b3);
            mma_bf16_16816(o[2 * n2], pf[kk], b0, b1);
            mma_bf16_16816(o[2 * n2 + 1], pf[kk], b2, b3);
            if (qsplit) {
              mma_bf16_16816(o[2 * n2], pl[kk], b0, b1);
              mma_bf16_16816(o[2 * n2 + 1], pl[kk], b2, b3);
            }
          }
        }
      }
      wbar();                                 // the stage is free again
      if (blk + PM_KVST < n_blocks) load_block(stage, k_begin + (blk + PM_KVST) * PM_KB);
      cp_async_commit();
    }
    cp_async_wait<0>();
    if (!active) continue;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 1);
      l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 2);
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int qi = qt * QT + warp * 16 + gq + 8 * h;
      if (qi >= Qn) continue;
      const int row = seq * rows_per_seq + qi / group;
      const int head = g * group + qi % group;
      if (n_parts == 1) {
        const float inv = l_run[h] > 0.f ? 1.f / l_run[h] : 0.f;
        const size_t ldx = (size_t)hq * DH;
#pragma unroll
        for (int i = 0; i < DH / 8; ++i) {
          const float a = o[i][2 * h] * inv, b = o[i][2 * h + 1] * inv;
          const bf16 ha = __float2bfloat16_rn(a), hb = __float2bfloat16_rn(b);
          const size_t col = (size_t)head * DH + i * 8 + tq * 2;
          *reinterpret_cast<uint32_t*>(out + (size_t)row * ldx + col) = pack_bf16(__bfloat162float(ha), __bfloat162float(hb));
          if (out_lo > 0)
            *reinterpret_cast<uint32_t*>(out + (size_t)(out_lo + row) * ldx + col) =
                pack_bf16(a - __bfloat162float(ha), b - __bfloat162float(hb));
        }
      } else {
        const size_t pidx = ((size_t)row * hq + head) * n_parts + part;
        float* dst = part_o + pidx * DH;
#pragma unroll
        for (int i = 0; i < DH / 8; ++i)
          *reinterpret_cast<float2*>(dst + i * 8 + tq * 2) = make_float2(o[i][2 * h], o[i][2 * h + 1]);
        if (tq == 0) {
          part_ml[pidx * 2 + 0] = m_run[h];
          part_ml[pidx * 2 + 1] = l_run[h];
        }
      }
    }
  }
}

// Merge of the attention parts: one warp per (row, head).  p[0] part_o, p[1] part_ml, p[2] out X buffer;
// i[0] n_parts, i[1] dh, i[2] lo_rows; rows = R, cols = hq.
__device__ __noinline__ void pm_combine(const PmOp& op, int wt) {
  const float* part_o = (const float*)op.p[0];
  const float* part_ml = (const float*)op.p[1];
  bf16* out = (bf16*)op.p[2];
  const int n_parts = op.i[0], dh = op.i[1], lo_rows = op.i[2], hq = op.cols, R = op.rows;
  const int lane = wt & 31;
  const int gw = (int)blockIdx.x * PM_WWARPS + (wt >> 5), nw = (int)gridDim.x * PM_WWARPS;
  const size_t ldx = (size_t)hq * dh;
  for (int rh = gw; rh < R * hq; rh += nw) {
    // (max, sum) of every part: one part per lane, then the weights of the parts by shuffles
    float M = -INFINITY;
    for (int p0 = 0; p0 < n_parts; p0 += 32) {
      const float m = p0 + lane < n_parts ? __ldcg(part_ml + ((size_t)rh * n_parts + p0 + lane) * 2) : -INFINITY;
      M = fmaxf(M, warp_max(m));
    }
    float L = 0.f, acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int p0 = 0; p0 < n_parts; p0 += 32) {
      float wl = 0.f, ww = 0.f;
      if (p0 + lane < n_parts) {
        const float2 ml = __ldcg(reinterpret_cast<const float2*>(part_ml + ((size_t)rh * n_parts + p0 + lane) * 2));
        ww = ml.x == -INFINITY ? 0.f : exp2f(ml.x - M);
        wl = ww * ml.y;
      }
      L += warp_sum(wl);
      const int np = min(32, n_parts - p0);
      for (int pp = 0; pp < np; pp += 4) {
        float x[4][4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
          for (int e = 0; e < 4; ++e)
            x[u][e] = (pp + u < np && e < dh / 32)
                          ? __ldcg(part_o + ((size_t)rh * n_parts + p0 + pp + u) * dh + lane + 32 * e) : 0.f;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const float wu = __shfl_sync(0xffffffffu, ww, (pp + u) & 31);
          if (pp + u < np)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[e] += wu * x[u][e];
        }
      }
    }
    const int row = rh / hq, head = rh - row * hq;
    const float inv = L > 0.f ? 1.f / L : 0.f;
    for (int e = 0; e < dh / 32; ++e) {
      const float a = acc[e] * inv;
      const bf16 h = __float2bfloat16_rn(a);
      const size_t col = (size_t)head * dh + lane + 32 * e;
      out[(size_t)row * ldx + col] = h;
      if (lo_rows > 0) out[(size_t)(lo_rows + row) * ldx + col] = __float2bfloat16_rn(a - __bfloat162float(h));
    }
  }
}

}  // namespace moa
