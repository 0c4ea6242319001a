// Generic kernels of the drafter forward: normalisation, an FMA GEMM for the fp32 path and for
// shapes the tensor-core kernels do not take, rotary embedding + cache writes, a plain attention
// row kernel, SwiGLU glue, layer mean, and a row-wise logsumexp + top-B over stored logits.
#pragma once
#include "moa_common.cuh"

namespace moa {

// ---------------------------------------------------------------------------------------------
// RMSNorm (pre-norm of every attention / MLP): y = x * g / sqrt(mean(x^2) + eps).
// One block per row. Input either gathered from the embedding table (tok != nullptr) or read from
// x[row]. Optionally also writes the un-normalised row in fp32 (the residual stream).
// ---------------------------------------------------------------------------------------------
// 8 consecutive elements <-> fp32 registers
template <typename T> __device__ __forceinline__ void load8(const T* p, float* v);
template <> __device__ __forceinline__ void load8<float>(const float* p, float* v) {
  const float4 a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
template <> __device__ __forceinline__ void load8<bf16>(const bf16* p, float* v) {
  bf16x8_to_float(*reinterpret_cast<const uint4*>(p), v);
}
template <typename T> __device__ __forceinline__ void store8(T* p, const float* v);
template <> __device__ __forceinline__ void store8<float>(float* p, const float* v) {
  *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
  *reinterpret_cast<float4*>(p + 4) = make_float4(v[4], v[5], v[6], v[7]);
}
template <> __device__ __forceinline__ void store8<bf16>(bf16* p, const float* v) {
  *reinterpret_cast<uint4*>(p) = make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]),
                                            pack_bf16(v[6], v[7]));
}

// Row r, columns k..k+7 of an X buffer [rows, K]: bf16 buffers with lo_rows > 0 also get the low-order term.
template <typename T> __device__ __forceinline__ void store8_x(T* xb, size_t K, int r, int k, int lo_rows, const float* v);
template <> __device__ __forceinline__ void store8_x<float>(float* xb, size_t K, int r, int k, int, const float* v) {
  store8<float>(xb + (size_t)r * K + k, v);
}
template <> __device__ __forceinline__ void store8_x<bf16>(bf16* xb, size_t K, int r, int k, int lo_rows, const float* v) {
  xbuf_store8(xb, K, r, k, lo_rows, v);
}

constexpr int RN_CHUNKS = 8;     // 8-element chunks of a row one thread of a 256-thread block keeps in registers

template <typename TIN, typename T>
__global__ void __launch_bounds__(256) rmsnorm_rows_kernel(const TIN* __restrict__ x, const int* __restrict__ tok,
                                                           int vocab, const T* __restrict__ gain, int K, float eps,
                                                           float* __restrict__ res_out, T* __restrict__ y, int lo_rows,
                                                           int* __restrict__ status) {
  pdl_trigger();
  pdl_wait(KID_NORM);
  __shared__ float red[33];
  const int r = blockIdx.x;
  const TIN* xr;
  if (tok != nullptr) {
    int t = tok[r];
    if (threadIdx.x == 0) MOA_DEV_CHECK(t >= 0 && t < vocab, status);
    t = t < 0 ? 0 : (t >= vocab ? vocab - 1 : t);
    xr = x + (size_t)t * K;
  } else {
    xr = x + (size_t)r * K;
  }
  // one pass: the row's chunks stay in registers between the sum of squares and the scaling (rows wider than
  // 256 * 8 * RN_CHUNKS elements re-read the rest)
  const int nch = K >> 3;
  float v[RN_CHUNKS][8];
  float ss = 0.f;
#pragma unroll
  for (int j = 0; j < RN_CHUNKS; ++j) {
    const int c = threadIdx.x + j * 256;
    if (c < nch) {
      load8<TIN>(xr + c * 8, v[j]);
#pragma unroll
      for (int i = 0; i < 8; ++i) ss += v[j][i] * v[j][i];
    }
  }
  for (int c = threadIdx.x + RN_CHUNKS * 256; c < nch; c += 256) {
    float t8[8];
    load8<TIN>(xr + c * 8, t8);
#pragma unroll
    for (int i = 0; i < 8; ++i) ss += t8[i] * t8[i];
  }
  ss = block_sum(ss, red);
  const float rinv = rsqrtf(ss / (float)K + eps);
  auto finish = [&](int c, const float* a) {
    if (res_out) store8<float>(res_out + (size_t)r * K + c * 8, a);
    float g8[8], o[8];
    load8<T>(gain + c * 8, g8);
#pragma unroll
    for (int i = 0; i < 8; ++i) o[i] = a[i] * rinv * g8[i];
    store8_x<T>(y, (size_t)K, r, c * 8, lo_rows, o);
  };
#pragma unroll
  for (int j = 0; j < RN_CHUNKS; ++j) {
    const int c = threadIdx.x + j * 256;
    if (c < nch) finish(c, v[j]);
  }
  for (int c = threadIdx.x + RN_CHUNKS * 256; c < nch; c += 256) {
    float t8[8];
    load8<TIN>(xr + c * 8, t8);
    finish(c, t8);
  }
}

// ---------------------------------------------------------------------------------------------
// C[R, N] (fp32, leading dimension ldc) = A[R, K] * W[N, K]^T (+ res[R, N] with leading dim ldr).
// Classic 64x64x16 shared-memory tiling, 256 threads, 4x4 outputs per thread, fp32 FMA.
// K must be a multiple of 16.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) gemm_fma_kernel(const T* __restrict__ A, const T* __restrict__ W,
                                                       int R, int N, int K, const float* res, int ldr,
                                                       float* C, int ldc) {
  pdl_trigger();
  pdl_wait(KID_GEMM);
  __shared__ float As[16][64 + 4];
  __shared__ float Ws[16][64 + 4];
  const int tid = threadIdx.x;
  const int n0 = blockIdx.x * 64, r0 = blockIdx.y * 64;
  const int lrow = tid >> 2, lk = (tid & 3) * 4;   // loader: 64 rows x 4 groups of 4 k
  const int ty = tid >> 4, tx = tid & 15;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (int k0 = 0; k0 < K; k0 += 16) {
    {
      const int ar = r0 + lrow;
      const int wn = n0 + lrow;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        As[lk + j][lrow] = ar < R ? to_f<T>(A[(size_t)ar * K + k0 + lk + j]) : 0.f;
        Ws[lk + j][lrow] = wn < N ? to_f<T>(W[(size_t)wn * K + k0 + lk + j]) : 0.f;
      }
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      float a[4], w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) w[j] = Ws[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = r0 + ty * 4 + i;
    if (r >= R) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= N) continue;
      float v = acc[i][j];
      if (res) v += res[(size_t)r * ldr + n];
      C[(size_t)r * ldc + n] = v;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Glue between GEMMs. A GEMM leaves `splits` fp32 partial planes (`plane` elements apart, one per
// K split); every consumer adds them in a fixed order, so results are deterministic.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float sum_splits(const float* p, size_t plane, int splits) {
  float s = 0.f;
  for (int i = 0; i < splits; ++i) s += p[(size_t)i * plane];
  return s;
}

// xres[r, :] += sum of partial planes [R, K]; then, if gain != nullptr, xn = RMSNorm(xres; gain) as T;
// optionally also copies the updated xres to hidden_out as T. One block per row.
template <typename T>
__global__ void __launch_bounds__(256) residual_norm_kernel(float* __restrict__ xres, const float* __restrict__ part,
                                                            int splits, size_t plane, int K, const T* __restrict__ gain,
                                                            float eps, T* __restrict__ xn, T* __restrict__ hidden_out,
                                                            int lo_rows) {
  pdl_trigger();
  pdl_wait(KID_RESNORM);
  __shared__ float red[33];
  const int r = blockIdx.x;
  const int nch = K >> 3;
  float ss = 0.f;
  for (int c = threadIdx.x; c < nch; c += 256) {
    float v[8];
    load8<float>(xres + (size_t)r * K + c * 8, v);
    if (part) {
      float t8[8];
      load8_planes(part + (size_t)r * K + c * 8, splits, plane, t8);
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] += t8[i];
      store8<float>(xres + (size_t)r * K + c * 8, v);
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) ss += v[i] * v[i];
  }
  if (gain == nullptr && hidden_out == nullptr) return;
  ss = block_sum(ss, red);
  const float rinv = rsqrtf(ss / (float)K + eps);
  for (int c = threadIdx.x; c < nch; c += 256) {
    float v[8];
    load8<float>(xres + (size_t)r * K + c * 8, v);        // this thread wrote it
    if (hidden_out) store8<T>(hidden_out + (size_t)r * K + c * 8, v);
    if (gain) {
      float g8[8], o[8];
      load8<T>(gain + c * 8, g8);
#pragma unroll
      for (int i = 0; i < 8; ++i) o[i] = v[i] * rinv * g8[i];
      store8_x<T>(xn, (size_t)K, r, c * 8, lo_rows, o);
    }
  }
}

// Same operation spread over a thread-block cluster of 8 CTAs per row: each CTA owns K/8 columns, keeps
// them in registers, and the row's sum of squares is exchanged through distributed shared memory (added
// in rank order, so the result does not depend on scheduling). Needs K % 64 == 0 and K <= 32768.
constexpr int RN_CLUSTER = 8;
constexpr int RN_MAX_PER_THREAD = 8;

template <typename T>
__global__ void __cluster_dims__(RN_CLUSTER, 1, 1) __launch_bounds__(256)
    residual_norm_cluster_kernel(float* __restrict__ xres, const float* __restrict__ part, int splits, size_t plane,
                                 int K, const T* __restrict__ gain, float eps, T* __restrict__ xn,
                                 T* __restrict__ hidden_out, int lo_rows) {
  pdl_trigger();
  pdl_wait(KID_RESNORM);
  __shared__ float red[33];
  __shared__ float cta_ss;
  const int r = blockIdx.y;
  const int rank = blockIdx.x;                       // cluster spans blockIdx.x = 0..7
  const int cpc = K / RN_CLUSTER;                    // columns per CTA (a multiple of 8: K % 64 == 0)
  const int c0 = rank * cpc;
  const int nch = cpc >> 3;
  float v[RN_MAX_PER_THREAD / 4][8];                 // up to two 8-element chunks per thread
  float ss = 0.f;
#pragma unroll
  for (int j = 0; j < RN_MAX_PER_THREAD / 4; ++j) {
    const int c = threadIdx.x + j * 256;
    if (c < nch) {
      const size_t idx = (size_t)r * K + c0 + c * 8;
      load8<float>(xres + idx, v[j]);
      if (part) {
        float t8[8];
        load8_planes(part + idx, splits, plane, t8);
#pragma unroll
        for (int i = 0; i < 8; ++i) v[j][i] += t8[i];
        store8<float>(xres + idx, v[j]);
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) ss += v[j][i] * v[j][i];
    }
  }
  if (gain == nullptr && hidden_out == nullptr) return;     // uniform over the whole grid
  ss = block_sum(ss, red);
  if (threadIdx.x == 0) cta_ss = ss;
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
  float total = 0.f;
  {
    const uint32_t local = (uint32_t)__cvta_generic_to_shared(&cta_ss);
#pragma unroll
    for (int j = 0; j < RN_CLUSTER; ++j) {
      uint32_t remote;
      float x;
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(j));
      asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(x) : "r"(remote) : "memory");
      total += x;
    }
  }
  // no CTA may exit (and release its shared memory) before every peer has read its slot
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
  const float rinv = rsqrtf(total / (float)K + eps);
#pragma unroll
  for (int j = 0; j < RN_MAX_PER_THREAD / 4; ++j) {
    const int c = threadIdx.x + j * 256;
    if (c < nch) {
      const size_t idx = (size_t)r * K + c0 + c * 8;
      if (hidden_out) store8<T>(hidden_out + idx, v[j]);
      if (gain) {
        float g8[8], o[8];
        load8<T>(gain + c0 + c * 8, g8);
#pragma unroll
        for (int i = 0; i < 8; ++i) o[i] = v[j][i] * rinv * g8[i];
        store8_x<T>(xn, (size_t)K, r, c0 + c * 8, lo_rows, o);
      }
    }
  }
}

// h = silu(sum gate) * (sum up): a partial plane row holds [gate | up] (2F columns). One thread per 8 columns.
template <typename T>
__global__ void silu_mul_split_kernel(const float* __restrict__ part, int splits, size_t plane, int F,
                                      T* __restrict__ h, size_t total, int lo_rows) {
  pdl_trigger();
  pdl_wait(KID_SILU);
  const size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 8;
  if (i >= total) return;
  const size_t r = i / F;
  const int c = (int)(i - r * F);
  float g8[8], u8[8], o[8];
  load8_planes(part + r * 2 * F + c, splits, plane, g8);
  load8_planes(part + r * 2 * F + F + c, splits, plane, u8);
#pragma unroll
  for (int k = 0; k < 8; ++k) o[k] = g8[k] / (1.f + __expf(-g8[k])) * u8[k];
  store8_x<T>(h, (size_t)F, (int)r, c, lo_rows, o);
}

// y = T(sum of planes), flat. One thread per 8 elements.
template <typename T>
__global__ void sum_cast_kernel(const float* __restrict__ part, int splits, size_t plane, size_t total,
                                T* __restrict__ y) {
  pdl_trigger();
  pdl_wait(KID_SUMCAST);
  const size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 8;
  if (i >= total) return;
  float v[8];
  load8_planes(part + i, splits, plane, v);
  store8<T>(y + i, v);
}

// ---------------------------------------------------------------------------------------------
// Rotary embedding + stores. One block per row. The input may be `splits` partial planes (plane
// elements apart) that are summed on the fly.
//   q (optional): fp32 [R, hq*dh] at qkv + q_off (leading dim ld) -> rotated, T [R, hq*dh] (or fp32 into qdst32)
//   k, v: fp32 [R, hkv*dh] -> k rotated; written as T to  kdst/vdst + dst_index(row) * hkv*dh
// Row r sits at position pos_base[seq(r)] + pos_add(r). Angles are formed in double:
// angle = pos * theta^(-2i/dh), element i paired with i + dh/2. theta == 0: no rotation.
// mode 0 (draft rows): seq = step0 ? r : r / B; pos_add = step; dst = seq * slots + self_slot
// mode 1 (prefix append): seq from split; i = r - off[seq]; pos_add = i; dst = seq * max_ctx + len + i
// ---------------------------------------------------------------------------------------------
struct RopeRows {
  int mode;
  int step, B, slots;      // mode 0
  int max_ctx;             // mode 1
  SeqSplit split;          // mode 1 (rows are relative to row0)
  int row0;
};

template <typename T>
__global__ void __launch_bounds__(256) rope_store_kernel(const float* __restrict__ qkv, int splits, size_t plane, int ld, int q_off, int k_off,
                                  int v_off,
                                  int hq, int hkv, int dh, float theta, const int* __restrict__ pos_base,
                                  RopeRows rr, T* __restrict__ qdst, float* __restrict__ qdst32, T* __restrict__ kdst,
                                  T* __restrict__ vdst, int* __restrict__ status) {
  pdl_trigger();
  pdl_wait(KID_ROPE);
  __shared__ float cs[64], sn[64];
  const int r = blockIdx.x;
  int seq, pos_add;
  size_t dst;
  bool store_kv = true;
  if (rr.mode == 0) {
    seq = rr.step == 0 ? r : r / rr.B;
    pos_add = rr.step;
    const int slot = rr.step == 0 ? 0 : 1 + (rr.step - 1) * rr.B + (r % rr.B);
    if (threadIdx.x == 0 && blockIdx.y == 0) MOA_DEV_CHECK(slot < rr.slots, status);
    dst = (size_t)seq * rr.slots + slot;
  } else {
    const int t = rr.row0 + r;
    seq = rr.split.seq_of(t);
    pos_add = t - rr.split.off[seq];
    dst = (size_t)seq * rr.max_ctx + pos_base[seq] + pos_add;
    // The host checked the capacity against its own count when the call was enqueued; a replayed graph can have
    // moved the device count since. A row that would land outside the cache is dropped and reported.
    if (pos_base[seq] + pos_add >= rr.max_ctx || pos_base[seq] < 0) {
      store_kv = false;
      if (threadIdx.x == 0 && blockIdx.y == 0 && status) atomicMax(status, DEV_ERR_BOUNDS);
    }
  }
  const int pos = pos_base[seq] + pos_add;
  const int half = dh >> 1;
  if (threadIdx.x < half) {
    if (theta == 0.f) {
      cs[threadIdx.x] = 1.f;
      sn[threadIdx.x] = 0.f;
    } else {
      const double inv = exp2(-2.0 * (double)threadIdx.x / (double)dh * log2((double)theta));
      double s, c;
      sincos((double)pos * inv, &s, &c);
      cs[threadIdx.x] = (float)c;
      sn[threadIdx.x] = (float)s;
    }
  }
  __syncthreads();
  const float* row0 = qkv + (size_t)r * ld;
  // Heads: query heads (when qdst is given), then key heads, then value heads. Eight threads share a head, each with
  // 8 consecutive elements of both halves (16-byte loads of every split plane, planes added in a fixed order); the
  // block's blockDim.x / 8 groups take heads blockIdx.y * groups + g, then every gridDim.y * groups-th one.
  const int nqh = qdst ? hq : 0;
  const int n_heads = nqh + 2 * hkv;
  const int groups = blockDim.x >> 3, slot = threadIdx.x >> 3, j0 = threadIdx.x & 7;
  for (int hh = blockIdx.y * groups + slot; hh < n_heads; hh += gridDim.y * groups) {
    int h = hh;
    const bool is_q = h < nqh;
    if (!is_q) h -= nqh;
    if (!is_q && !store_kv) continue;
    if (is_q || h < hkv) {                               // rotated: element i pairs with i + dh/2
      const int off = (is_q ? q_off : k_off) + h * dh;
      for (int i = j0; i < (half >> 3); i += 8) {
        float a[8], b2[8], o1[8], o2[8];
        load8_planes(row0 + off + i * 8, splits, plane, a);
        load8_planes(row0 + off + half + i * 8, splits, plane, b2);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float c = cs[i * 8 + e], sv = sn[i * 8 + e];
          o1[e] = a[e] * c - b2[e] * sv;
          o2[e] = b2[e] * c + a[e] * sv;
        }
        if (is_q) {
          const size_t at = (size_t)r * hq * dh + h * dh + i * 8;
          if (qdst32) {                  // rotated queries kept in fp32 (the attention kernel splits them)
            store8<float>(qdst32 + at, o1);
            store8<float>(qdst32 + at + half, o2);
          } else {
            store8<T>(qdst + at, o1);
            store8<T>(qdst + at + half, o2);
          }
        } else {
          const size_t at = dst * hkv * dh + h * dh + i * 8;
          store8<T>(kdst + at, o1);
          store8<T>(kdst + at + half, o2);
        }
      }
      continue;
    }
    h -= hkv;
    for (int i = j0; i < (dh >> 3); i += 8) {
      float v8[8];
      load8_planes(row0 + v_off + h * dh + i * 8, splits, plane, v8);
      store8<T>(vdst + dst * hkv * dh + h * dh + i * 8, v8);
    }
  }
}

// Cross-attention cache append: fp32 [n, hkv*dh] k and v rows -> T cache rows at (seq, ca_len[seq] + i).
template <typename T>
__global__ void cache_append_kernel(const float* __restrict__ kv, int splits, size_t plane, int ld, int k_off, int v_off,
                                    int width,
                                    const int* __restrict__ len, int max_ctx, SeqSplit split, int row0,
                                    T* __restrict__ kdst, T* __restrict__ vdst, int* __restrict__ status) {
  pdl_trigger();
  pdl_wait(KID_APPEND);
  const int r = blockIdx.x;
  const int t = row0 + r;
  const int seq = split.seq_of(t);
  const int i = t - split.off[seq];
  if (len[seq] < 0 || len[seq] + i >= max_ctx) {       // see rope_store_kernel: the device count decides
    if (threadIdx.x == 0 && status) atomicMax(status, DEV_ERR_BOUNDS);
    return;
  }
  const size_t dst = ((size_t)seq * max_ctx + len[seq] + i) * width;
  const int nch = width >> 3;
  for (int c = threadIdx.x; c < 2 * nch; c += blockDim.x) {      // one thread per 8 columns of k, then of v
    const bool isv = c >= nch;
    const int cc = (isv ? c - nch : c) * 8;
    float v8[8];
    load8_planes(kv + (size_t)r * ld + (isv ? v_off : k_off) + cc, splits, plane, v8);
    store8<T>((isv ? vdst : kdst) + dst + cc, v8);
  }
}

__global__ void add_len_kernel(int* len, SeqSplit split, int max_ctx) {
  const int b = threadIdx.x;
  if (b < split.n_seq) len[b] = min(max_ctx, len[b] + split.off[b + 1] - split.off[b]);
}
struct LenVals { int n; int v[64]; };
__global__ void set_len_kernel(int* len, LenVals lv) {
  const int b = threadIdx.x;
  if (b < lv.n) len[b] = lv.v[b];
}

// ---------------------------------------------------------------------------------------------
// Attention, one block (4 warps) per (query row, query head): softmax(q K^T / sqrt(dh)) V in fp32.
// Key set = segment A: keys 0..nA-1 of sequence `seq` in a cache [n_seq, capA, hkv, dh]
//         + segment B: nB listed slots of a second cache [n_seq, capB, hkv, dh] (tree nodes).
// Row -> sequence: seq = r / rows_per_seq. nA = lenA ? lenA[seq] : nA_fixed.
// q_ld: elements between query rows; posA_ld: elements between consecutive positions of segment A
// (hkv*dh for a dense cache; larger when k and v sit inside wider rows).
// Each warp walks keys warp, warp+4, ...; a lane owns dh/32 consecutive elements.
// ---------------------------------------------------------------------------------------------
template <typename T, int DH>
__global__ void __launch_bounds__(128) attn_rows_kernel(const T* __restrict__ q, int q_ld, int hq, int hkv,
                                                        const T* __restrict__ kA, const T* __restrict__ vA, int capA,
                                                        int posA_ld,
                                                        const int* __restrict__ lenA, int nA_fixed,
                                                        const T* __restrict__ kB, const T* __restrict__ vB, int capB,
                                                        const int* __restrict__ slotsB, int slots_ld, int nB,
                                                        int rows_per_seq, RowLimit lim, T* __restrict__ out) {
  pdl_trigger();
  pdl_wait(KID_ATTN);
  constexpr int VEC = DH / 32;
  __shared__ float s_m[4], s_l[4], s_acc[4][DH];
  const int r = blockIdx.x, h = blockIdx.y;
  const int g = h / (hq / hkv);
  const int seq = r / rows_per_seq;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nA = min(lenA ? lenA[seq] : nA_fixed, lim.of(r));
  const float scale = rsqrtf((float)DH);
  float qv[VEC];
#pragma unroll
  for (int e = 0; e < VEC; ++e) qv[e] = to_f<T>(q[(size_t)r * q_ld + h * DH + lane * VEC + e]) * scale;
  float m = -INFINITY, l = 0.f, acc[VEC];
#pragma unroll
  for (int e = 0; e < VEC; ++e) acc[e] = 0.f;
  const int n = nA + nB;
  for (int j = warp; j < n; j += 4) {
    const T *kp, *vp;
    if (j < nA) {
      const size_t o = ((size_t)seq * capA + j) * posA_ld + g * DH + lane * VEC;
      kp = kA + o;
      vp = vA + o;
    } else {
      const int slot = slotsB[(size_t)r * slots_ld + (j - nA)];
      const size_t o = (((size_t)seq * capB + slot) * hkv + g) * DH + lane * VEC;
      kp = kB + o;
      vp = vB + o;
    }
    float s = 0.f;
#pragma unroll
    for (int e = 0; e < VEC; ++e) s = fmaf(qv[e], to_f<T>(kp[e]), s);
    s = warp_sum(s);
    const float mn = fmaxf(m, s);
    const float corr = __expf(m - mn);     // m = -inf at the first key: exp(-inf) = 0
    const float p = __expf(s - mn);
    l = l * corr + p;
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[e] = acc[e] * corr + p * to_f<T>(vp[e]);
    m = mn;
  }
  if (lane == 0) { s_m[warp] = m; s_l[warp] = l; }
#pragma unroll
  for (int e = 0; e < VEC; ++e) s_acc[warp][lane * VEC + e] = acc[e];
  __syncthreads();
  if (warp == 0) {
    float M = fmaxf(fmaxf(s_m[0], s_m[1]), fmaxf(s_m[2], s_m[3]));
    float L = 0.f, o[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) o[e] = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const float c = s_m[w] == -INFINITY ? 0.f : __expf(s_m[w] - M);
      L += s_l[w] * c;
#pragma unroll
      for (int e = 0; e < VEC; ++e) o[e] += s_acc[w][lane * VEC + e] * c;
    }
    const float inv = L > 0.f ? 1.f / L : 0.f;
#pragma unroll
    for (int e = 0; e < VEC; ++e) out[((size_t)r * hq + h) * DH + lane * VEC + e] = from_f<T>(o[e] * inv);
  }
}

// kv[t, :] = mean over the S layer rows of Z[t, s, :] (fp32 in; fp32 and optional T out).
template <typename T>
__global__ void mean_layers_kernel(const float* __restrict__ Z, int S, int D, float* __restrict__ kvf,
                                   T* __restrict__ kv_out) {
  pdl_trigger();
  pdl_wait(KID_MEAN);
  const int t = blockIdx.x;                                   // grid (tokens, ceil(D / blockDim.x))
  const int c = blockIdx.y * blockDim.x + threadIdx.x;
  if (c >= D) return;
  float s = 0.f;
  for (int l = 0; l < S; ++l) s += Z[((size_t)t * S + l) * D + c];
  s *= 1.f / (float)S;
  kvf[(size_t)t * D + c] = s;
  if (kv_out) kv_out[(size_t)t * D + c] = from_f<T>(s);
}

// ---------------------------------------------------------------------------------------------
// Row-wise log-softmax top-B over stored logits z[R, V] (fp32): lse = max + log(sum exp(z - max)),
// then B rounds of block arg-max in the order (value descending, id ascending).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ bool better(float va, int ia, float vb, int ib) {   // (va, ia) ranks before (vb, ib)
  return va > vb || (va == vb && ia < ib);
}

__global__ void __launch_bounds__(256) lse_topk_rows_kernel(const float* __restrict__ z, int V, int B,
                                                            int* __restrict__ ids, float* __restrict__ logp) {
  pdl_trigger();
  pdl_wait(KID_LM_MERGE);
  __shared__ float red[33];
  __shared__ float s_v[8];
  __shared__ int s_i[8];
  __shared__ float pick_v;
  __shared__ int pick_i;
  const int r = blockIdx.x;
  const float* zr = z + (size_t)r * V;
  float mx = -INFINITY;
  for (int i = threadIdx.x; i < V; i += blockDim.x) mx = fmaxf(mx, zr[i]);
  mx = block_max(mx, red);
  float se = 0.f;
  for (int i = threadIdx.x; i < V; i += blockDim.x) se += expf(zr[i] - mx);
  se = block_sum(se, red);
  const float lse = mx + logf(se);
  float pv = INFINITY;
  int pi = -1;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  for (int b = 0; b < B; ++b) {
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    for (int i = threadIdx.x; i < V; i += blockDim.x) {
      const float v = zr[i];
      if (better(pv, pi, v, i) && better(v, i, bv, bi)) { bv = v; bi = i; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
    }
    if (lane == 0) { s_v[wid] = bv; s_i[wid] = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
      float fv = s_v[0];
      int fi = s_i[0];
      for (int w = 1; w < 8; ++w)
        if (better(s_v[w], s_i[w], fv, fi)) { fv = s_v[w]; fi = s_i[w]; }
      pick_v = fv;
      pick_i = fi;
      ids[(size_t)r * B + b] = fi == 0x7fffffff ? -1 : fi;
      logp[(size_t)r * B + b] = fv - lse;
    }
    __syncthreads();
    pv = pick_v;
    pi = pick_i;
  }
}

}  // namespace moa
