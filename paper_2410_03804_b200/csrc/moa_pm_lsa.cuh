// Phase machine, part 6: Layer Self-Attention proper (Section 3.1.1): for every token, bidirectional
// attention over its S stacked layer rows, tokens independent.
//
// The sequence is tiny (S = 32..80 rows) and there are very many of them (tokens x heads), so the unit of
// work is one (token, query head) per WARP, with no CTA-level synchronisation at all:
//   - the warp's lanes issue one bulk asynchronous copy (TMA engine, cp.async.bulk) per row of q, k and v
//     into the warp's own shared-memory tiles (rows padded by 16 bytes so that ldmatrix is conflict-free),
//     all landing on the warp's mbarrier;
//   - scores by mma.sync (16 query rows at a time against all keys), softmax in fp32 with the row maximum
//     and sum exchanged by quad shuffles, probabilities as bf16 (hi, and lo when the output is split), P.V by
//     mma.sync, normalised rows written straight into the out-projection's X buffer.
#pragma once
#include "moa_pm_common.cuh"

namespace moa {

__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}

//  p[0] qkv rows (bf16 [R, ld]: q | k | v), p[1] out X buffer [R (+lo), hq*dh]
//  i[0] ld, i[1] hq, i[2] hkv, i[3] S, i[4] warps per CTA that take units, i[5] out lo_rows, i[6] head size;
//  rows = R, cols = tokens; f[0] scale_log2
template <int DH, int NT>       // NT = key tiles of 8 the registers are sized for (S <= 8 * NT)
__device__ __noinline__ void pm_lsa_attention(const PmOp& op, uint8_t* smem_gen, uint32_t smem_sh, int wt,
                                              volatile int* abort_flag) {
  constexpr int KS = DH / 16;
  constexpr int ROWB = DH * 2 + 16;            // padded row: 8 consecutive rows start in 8 different 16-byte banks
  const bf16* qkv = (const bf16*)op.p[0];
  bf16* out = (bf16*)op.p[1];
  const int ld = op.i[0], hq = op.i[1], hkv = op.i[2], S = op.i[3], n_warps = op.i[4], out_lo = op.i[5];
  const int n_tok = op.cols;
  const float scale_log2 = op.f[0];
  const int group = hq / hkv, nq = hq * DH, nkv = hkv * DH;
  const int s_pad = (S + 15) & ~15;
  const int nt_n = s_pad >> 3, mt_n = s_pad >> 4;
  const int warp = wt >> 5, lane = wt & 31;
  if (warp >= n_warps) return;
  const uint32_t tile_bytes = (uint32_t)s_pad * ROWB;
  const uint32_t per_warp = 3 * tile_bytes + 16;
  const uint32_t sQ = smem_sh + warp * per_warp, sK = sQ + tile_bytes, sV = sK + tile_bytes;
  const uint32_t bar = sV + tile_bytes;
  uint8_t* mine = smem_gen + warp * per_warp;
  // the tiles start as zeros (rows S .. s_pad-1 stay zero: a zero value row times a zero probability is zero)
  for (uint32_t i = lane * 16; i < 3 * tile_bytes; i += 32 * 16) *reinterpret_cast<uint4*>(mine + i) = make_uint4(0, 0, 0, 0);
  if (lane == 0) mbar_init(bar, 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncwarp();
  const int gq = lane >> 2, tq = lane & 3;
  const long long n_units = (long long)n_tok * hq;
  uint32_t parity = 0;
  const long long gw = (long long)blockIdx.x * n_warps + warp, nw = (long long)gridDim.x * n_warps;
  for (long long u = gw; u < n_units; u += nw) {
    const int t = (int)(u / hq), h = (int)(u - (long long)t * hq), g = h / group;
    // ---- stage the token's q, k, v rows of this head ----
    if (lane == 0) mbar_expect_tx(bar, (uint32_t)(3 * S * DH * 2));
    __syncwarp();
    for (int r = lane; r < S; r += 32) {
      const bf16* row = qkv + (size_t)(t * S + r) * ld;
      bulk_copy_g2s(sQ + r * ROWB, row + h * DH, DH * 2, bar);
      bulk_copy_g2s(sK + r * ROWB, row + nq + g * DH, DH * 2, bar);
      bulk_copy_g2s(sV + r * ROWB, row + nq + nkv + g * DH, DH * 2, bar);
    }
    if (!mbar_wait(bar, parity, abort_flag)) return;
    parity ^= 1u;
    // ---- 16 query rows at a time ----
    for (int mt = 0; mt < mt_n; ++mt) {
      uint32_t qf[KS][4];
      {
        const int row = mt * 16 + (lane & 15);
#pragma unroll
        for (int ks = 0; ks < KS; ++ks)
          ldsm_x4(sQ + row * ROWB + (ks * 2 + (lane >> 4)) * 16, qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
      }
      float s[NT][4];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        if (nt < nt_n) {
#pragma unroll
          for (int ks2 = 0; ks2 < KS / 2; ++ks2) {
            uint32_t b0, b1, b2, b3;
            ldsm_x4(sK + (nt * 8 + (lane & 7)) * ROWB + (ks2 * 4 + (lane >> 3)) * 16, b0, b1, b2, b3);
            mma_bf16_16816(s[nt], qf[2 * ks2], b0, b1);
            mma_bf16_16816(s[nt], qf[2 * ks2 + 1], b2, b3);
          }
        }
      }
      // softmax over the S keys: this thread holds rows gq and gq + 8 of the tile, two keys per key tile
      float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int key = nt * 8 + tq * 2 + (e & 1);
          const float v = (nt < nt_n && key < S) ? s[nt][e] * scale_log2 : -INFINITY;
          s[nt][e] = v;
          mx[e >> 1] = fmaxf(mx[e >> 1], v);
        }
      }
      float sum[2] = {0.f, 0.f};
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        mx[hh] = fmaxf(mx[hh], __shfl_xor_sync(0xffffffffu, mx[hh], 1));
        mx[hh] = fmaxf(mx[hh], __shfl_xor_sync(0xffffffffu, mx[hh], 2));
      }
      uint32_t pf[NT / 2][4], pl[NT / 2][4];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const float p0 = exp2f(s[nt][0] - mx[0]), p1 = exp2f(s[nt][1] - mx[0]);
        const float p2 = exp2f(s[nt][2] - mx[1]), p3 = exp2f(s[nt][3] - mx[1]);
        sum[0] += p0 + p1;
        sum[1] += p2 + p3;
        const bf16 h0 = __float2bfloat16_rn(p0), h1 = __float2bfloat16_rn(p1), h2 = __float2bfloat16_rn(p2),
                   h3 = __float2bfloat16_rn(p3);
        pf[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(__bfloat162float(h0), __bfloat162float(h1));
        pf[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(__bfloat162float(h2), __bfloat162float(h3));
        pl[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(p0 - __bfloat162float(h0), p1 - __bfloat162float(h1));
        pl[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p2 - __bfloat162float(h2), p3 - __bfloat162float(h3));
      }
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        sum[hh] += __shfl_xor_sync(0xffffffffu, sum[hh], 1);
        sum[hh] += __shfl_xor_sync(0xffffffffu, sum[hh], 2);
      }
      // O = P V
      float o[DH / 8][4];
#pragma unroll
      for (int i = 0; i < DH / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
#pragma unroll
      for (int kk = 0; kk < NT / 2; ++kk) {
        if (kk < mt_n) {
#pragma unroll
          for (int n2 = 0; n2 < DH / 16; ++n2) {
            uint32_t b0, b1, b2, b3;
            const int key = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
            ldsm_x4_t(sV + key * ROWB + (n2 * 2 + (lane >> 4)) * 16, b0, b1, b2, b3);
            mma_bf16_16816(o[2 * n2], pf[kk], b0, b1);
            mma_bf16_16816(o[2 * n2 + 1], pf[kk], b2, b3);
            if (out_lo > 0) {
              mma_bf16_16816(o[2 * n2], pl[kk], b0, b1);
              mma_bf16_16816(o[2 * n2 + 1], pl[kk], b2, b3);
            }
          }
        }
      }
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const int qrow = mt * 16 + gq + 8 * hh;
        if (qrow >= S) continue;
        const float inv = 1.f / sum[hh];
        const size_t ldx = (size_t)hq * DH;
        const size_t row = (size_t)t * S + qrow;
#pragma unroll
        for (int i = 0; i < DH / 8; ++i) {
          const float a = o[i][2 * hh] * inv, b = o[i][2 * hh + 1] * inv;
          const bf16 ha = __float2bfloat16_rn(a), hb = __float2bfloat16_rn(b);
          const size_t col = (size_t)h * DH + i * 8 + tq * 2;
          *reinterpret_cast<uint32_t*>(out + row * ldx + col) = pack_bf16(__bfloat162float(ha), __bfloat162float(hb));
          if (out_lo > 0)
            *reinterpret_cast<uint32_t*>(out + (size_t)(out_lo + row) * ldx + col) =
                pack_bf16(a - __bfloat162float(ha), b - __bfloat162float(hb));
        }
      }
    }
    __syncwarp();          // every lane is done with the tiles before the next unit's copies land in them
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
}

}  // namespace moa
