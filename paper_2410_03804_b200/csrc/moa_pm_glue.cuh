// Phase machine, part 2: the glue phases between the GEMMs (norms, layer mean, cache append). Each is executed by the 192 worker threads of every CTA; its units are spread over the grid.
// Everything another CTA wrote earlier in the same launch is read with ld.global.cg (past L1).
#pragma once
#include "moa_pm_common.cuh"

namespace moa {

// Row normalisation family. One CTA per row (or one warp per row when there are many rows).
//  source of row r:  x[r] (PH_ROWS_NORM) | xres[r] + split planes (PH_RESNORM)
//  p[0] src rows (bf16), p[2] gain (bf16) or null, p[3] xres (fp32) or null, p[4] xbuf or null,
//  p[5] hidden_out (bf16) or null; i[1] lo_rows; f[0] eps.
__device__ __noinline__ void pm_norm_rows(PmSmem& S, const PmOp& op, int wt) {
  const int R = op.rows, K = op.cols, kind = op.kind;
  const bf16* src = (const bf16*)op.p[0];
  const bf16* gain = (const bf16*)op.p[2];
  float* xres = (float*)op.p[3];
  bf16* xbuf = (bf16*)op.p[4];
  bf16* hidden = (bf16*)op.p[5];
  const int lo_rows = op.i[1];
  const float eps = op.f[0];
  const float* part = nullptr;
  int splits = 0;
  size_t plane = 0;
  if (kind == PH_RESNORM && op.gemm >= 0) {
    part = S.g[op.gemm].out; splits = S.g[op.gemm].splits; plane = S.g[op.gemm].plane;
  }
  const int nch = K >> 3;
  auto load_chunk = [&](int r, size_t srow, int c, float* v) {
    if (kind == PH_RESNORM) {
      const float4 a = ldcg4(xres + (size_t)r * K + c * 8), b = ldcg4(xres + (size_t)r * K + c * 8 + 4);
      v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
      if (part) {
        float t[8];
        load8_planes(part + (size_t)r * K + c * 8, splits, plane, t);
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] += t[i];
      }
    } else {
      bf16x8_to_float(*reinterpret_cast<const uint4*>(src + srow * K + c * 8), v);
    }
  };
  auto src_row = [&](int r) -> size_t { return (size_t)r; };
  auto finish_chunk = [&](int r, int c, const float* v, float rinv) {
    if (xres && (kind != PH_RESNORM || part)) {
      *reinterpret_cast<float4*>(xres + (size_t)r * K + c * 8) = make_float4(v[0], v[1], v[2], v[3]);
      *reinterpret_cast<float4*>(xres + (size_t)r * K + c * 8 + 4) = make_float4(v[4], v[5], v[6], v[7]);
    }
    if (hidden) {
      uint32_t w[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) w[e] = pack_bf16(v[2 * e], v[2 * e + 1]);
      *reinterpret_cast<uint4*>(hidden + (size_t)r * K + c * 8) = make_uint4(w[0], w[1], w[2], w[3]);
    }
    if (gain && xbuf) {
      float g8[8], y[8];
      bf16x8_to_float(*reinterpret_cast<const uint4*>(gain + c * 8), g8);
#pragma unroll
      for (int i = 0; i < 8; ++i) y[i] = v[i] * rinv * g8[i];
      xbuf_store8(xbuf, (size_t)K, r, c * 8, lo_rows, y);
    }
  };
  const bool need_norm = gain != nullptr && xbuf != nullptr;
  if (R >= 4 * (int)gridDim.x) {
    // many rows: one warp per row, two passes over the row
    const int lane = wt & 31;
    const int gw = (int)blockIdx.x * PM_WWARPS + (wt >> 5), nw = (int)gridDim.x * PM_WWARPS;
    for (int r = gw; r < R; r += nw) {
      const size_t srow = src_row(r);
      float ss = 0.f;
      if (need_norm) {
        for (int c = lane; c < nch; c += 32) {
          float v[8];
          load_chunk(r, srow, c, v);
#pragma unroll
          for (int i = 0; i < 8; ++i) ss += v[i] * v[i];
        }
        ss = warp_sum(ss);
      }
      const float rinv = rsqrtf(ss / (float)K + eps);
      for (int c = lane; c < nch; c += 32) {
        float v[8];
        load_chunk(r, srow, c, v);
        finish_chunk(r, c, v, rinv);
      }
    }
    return;
  }
  for (int r = blockIdx.x; r < R; r += gridDim.x) {
    const size_t srow = src_row(r);
    float v[PM_MAXCH][8];
    float ss = 0.f;
#pragma unroll
    for (int j = 0; j < PM_MAXCH; ++j) {
      const int c = wt + j * PM_WORKERS;
      if (c < nch) {
        load_chunk(r, srow, c, v[j]);
#pragma unroll
        for (int i = 0; i < 8; ++i) ss += v[j][i] * v[j][i];
      }
    }
    for (int c = wt + PM_MAXCH * PM_WORKERS; c < nch; c += PM_WORKERS) {     // rows wider than the register copy
      float t[8];
      load_chunk(r, srow, c, t);
#pragma unroll
      for (int i = 0; i < 8; ++i) ss += t[i] * t[i];
    }
    float rinv = 0.f;
    if (need_norm) {
      ss = worker_sum(ss, S.red, wt);
      rinv = rsqrtf(ss / (float)K + eps);
    }
#pragma unroll
    for (int j = 0; j < PM_MAXCH; ++j) {
      const int c = wt + j * PM_WORKERS;
      if (c < nch) finish_chunk(r, c, v[j], rinv);
    }
    for (int c = wt + PM_MAXCH * PM_WORKERS; c < nch; c += PM_WORKERS) {
      float t[8];
      load_chunk(r, srow, c, t);
      finish_chunk(r, c, t, rinv);
    }
  }
}


// LSA tail: xres (+ planes of the down projection) -> mean over the S layer rows of a token -> kvf (fp32),
// kv_out (bf16, optional), kvn = RMSNorm(mean; gain) into an X buffer. One CTA per token.
//  p[0] xres, p[1] kvf, p[2] kv_out, p[3] gain, p[4] kvn xbuf; i[0] S, i[1] lo_rows; rows = tokens, cols = D; f[0] eps
__device__ __noinline__ void pm_mean_norm(PmSmem& S_, const PmOp& op, int wt) {
  const float* xres = (const float*)op.p[0];
  float* kvf = (float*)op.p[1];
  bf16* kv_out = (bf16*)op.p[2];
  const bf16* gain = (const bf16*)op.p[3];
  bf16* kvn = (bf16*)op.p[4];
  const int S = op.i[0], lo_rows = op.i[1], D = op.cols, nch = D >> 3, n_tok = op.rows;
  const float eps = op.f[0];
  const float* part = nullptr;
  int splits = 0;
  size_t plane = 0;
  if (op.gemm >= 0) { part = S_.g[op.gemm].out; splits = S_.g[op.gemm].splits; plane = S_.g[op.gemm].plane; }
  for (int t = blockIdx.x; t < n_tok; t += gridDim.x) {
    float ss = 0.f;
    for (int c = wt; c < nch; c += PM_WORKERS) {
      float m[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      for (int l0 = 0; l0 < S; l0 += 4) {                  // four layer rows in flight at a time
        float4 a[4], b[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (l0 + u < S) {
            const size_t at = ((size_t)t * S + l0 + u) * D + c * 8;
            a[u] = ldcg4(xres + at); b[u] = ldcg4(xres + at + 4);
          }
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (l0 + u < S) {
            m[0] += a[u].x; m[1] += a[u].y; m[2] += a[u].z; m[3] += a[u].w;
            m[4] += b[u].x; m[5] += b[u].y; m[6] += b[u].z; m[7] += b[u].w;
          }
        if (part) {
          for (int u = 0; u < 4 && l0 + u < S; ++u) {
            float v[8];
            load8_planes(part + ((size_t)t * S + l0 + u) * D + c * 8, splits, plane, v);
#pragma unroll
            for (int i = 0; i < 8; ++i) m[i] += v[i];
          }
        }
      }
      const float invS = 1.f / (float)S;
#pragma unroll
      for (int i = 0; i < 8; ++i) { m[i] *= invS; ss += m[i] * m[i]; }
      *reinterpret_cast<float4*>(kvf + (size_t)t * D + c * 8) = make_float4(m[0], m[1], m[2], m[3]);
      *reinterpret_cast<float4*>(kvf + (size_t)t * D + c * 8 + 4) = make_float4(m[4], m[5], m[6], m[7]);
      if (kv_out) xbuf_store8(kv_out, (size_t)D, t, c * 8, 0, m);
    }
    ss = worker_sum(ss, S_.red, wt);
    const float rinv = rsqrtf(ss / (float)D + eps);
    for (int c = wt; c < nch; c += PM_WORKERS) {
      const float4 a = *reinterpret_cast<const float4*>(kvf + (size_t)t * D + c * 8);      // this thread wrote it
      const float4 b = *reinterpret_cast<const float4*>(kvf + (size_t)t * D + c * 8 + 4);
      float g8[8];
      bf16x8_to_float(*reinterpret_cast<const uint4*>(gain + c * 8), g8);
      const float y[8] = {a.x * rinv * g8[0], a.y * rinv * g8[1], a.z * rinv * g8[2], a.w * rinv * g8[3],
                          b.x * rinv * g8[4], b.y * rinv * g8[5], b.z * rinv * g8[6], b.w * rinv * g8[7]};
      xbuf_store8(kvn, (size_t)D, t, c * 8, lo_rows, y);
    }
  }
}

// Cross-attention cache append: planes [tokens, k | v] -> bf16 cache rows at (seq, len[seq] + i).
//  p[0] len, p[1] kdst, p[2] vdst; i[0] width, i[1] max_ctx, i[2] first token of this pass; rows = tokens
__device__ __noinline__ void pm_cache_append(PmSmem& S, const PmOp& op, int wt, int* status) {
  const PmGemm& G = S.g[op.gemm];
  const float* out = G.out;
  const int splits = G.splits;
  const size_t plane = G.plane;
  const int* len = (const int*)op.p[0];
  bf16* kdst = (bf16*)op.p[1];
  bf16* vdst = (bf16*)op.p[2];
  const int width = op.i[0], max_ctx = op.i[1], row0 = op.i[2], nch = width >> 3, n_tok = op.rows;
  for (int r = blockIdx.x; r < n_tok; r += gridDim.x) {
    const int t = row0 + r;
    const int seq = S.split.seq_of(t);
    const int i = t - S.split.off[seq];
    const int at = __ldcg(len + seq) + i;
    if (at < i || at >= max_ctx) {                       // the device count decides: a row outside the cache is dropped and reported
      if (wt == 0 && status) atomicMax(status, DEV_ERR_BOUNDS);
      continue;
    }
    const size_t dst = (size_t)seq * max_ctx + at;
    for (int c = wt; c < 2 * nch; c += PM_WORKERS) {
      const bool isv = c >= nch;
      const int cc = isv ? c - nch : c;
      float v[8];
      load8_planes(out + (size_t)r * 2 * width + (isv ? width : 0) + cc * 8, splits, plane, v);
      xbuf_store8((isv ? vdst : kdst) + dst * width, (size_t)width, 0, cc * 8, 0, v);
    }
  }
}

}  // namespace moa
