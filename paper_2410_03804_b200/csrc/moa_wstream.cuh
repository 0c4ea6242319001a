// Weight-streaming GEMM for sm_100a:  Y^T[n, r] = sum_k W[n, k] * X[r, k]   (bf16 in, fp32 accumulate)
//
// The weight matrix is the big operand: it is streamed from HBM exactly once per call, 128 rows x 64
// columns (16 KB) per pipeline stage, by TMA into 128B-swizzled shared memory, and fed to the 5th-gen
// tensor cores as the A operand (M = 128) of tcgen05.mma. The R activation rows (R <= 256 per call) are
// the B operand (N = R padded to 16/32/64/128/256), re-fetched from L2 next to each weight tile.
// Accumulators live in TMEM, double-buffered so that the epilogue of one tile overlaps the MMAs of the
// next. One CTA per SM, persistent over work units (weight tile x K split), 10 warps:
//   warp 0     : TMA producer (one lane)
//   warp 1     : TMEM allocation + MMA issue (one lane)
//   warps 2..9 : epilogue, two per TMEM lane quadrant (alternate groups of 16 activation rows)
// Epilogues:
//   mode 0: fp32 partial sums, out[split][r][col0 + n]  (the consumer adds the splits in a fixed order,
//           so results are deterministic and need no atomics or zero-filled buffers)
//   mode 1: LM head -- per 32 vocabulary rows and per activation row: max, sum of exponentials and
//           the B largest logits with their ids, sorted; the logits never go to HBM (Eq. 1 + top-B).
// Every mbarrier wait is bounded: on expiry the CTA raises an abort flag, drains, frees TMEM, writes
// DEV_ERR_TIMEOUT to the status word and returns.
#pragma once
#include <cuda.h>

#include "moa_common.cuh"

namespace moa {

constexpr int WS_BM = 128;         // weight rows per tile (MMA M)
constexpr int WS_BK = 64;          // k elements per stage: 128 bytes of bf16 = one swizzle row
constexpr int WS_THREADS = 320;     // TMA warp, MMA warp, eight epilogue warps (two per TMEM lane quadrant)
constexpr int WS_W_BYTES = WS_BM * WS_BK * 2;
constexpr int EPI_U = 4;          // activation rows the LM-head epilogue sorts side by side
constexpr int WS_SMEM_BUDGET = 224 * 1024;    // ring of stages; 1.25 KB more for alignment and barriers stays under 227 KB
constexpr long long WS_WAIT_CYCLES = 4000000000ll;   // ~2 s at boost clock

struct WsParams {
  CUtensorMap tmW[3];      // weight matrices [n_i, K], box 64 x 128, swizzle 128B
  CUtensorMap tmX;         // activations [R, K], box 64 x NPAD, swizzle 128B, rows >= R read as zero
  int n_seg;
  int seg_n[3];            // rows of each weight matrix
  int seg_tile0[3];        // first tile index of each segment
  int seg_col[3];          // first output column of each segment
  int tiles_total;
  int R;                   // valid activation rows
  int kb_total;            // K / 64
  int splits;              // K splits per tile
  int mode;                // 0: fp32 partials, 1: LM-head partial top-B
  int xsplit;              // activations carried as two bf16 terms: rows [0, R) hi, rows [NPAD/2, NPAD/2 + R) lo
  int lo_row;              // XS2 kernels: first row of the low-order terms in the activation buffer
  int ldo;                 // mode 0: columns of one partial plane
  float* out;              // mode 0: plane `split` starts at out + split * plane; row r, column c at [r * ldo + c]
  size_t plane;            // mode 0: elements between two partial planes
  int B;                   // mode 1
  float* p_max;            // mode 1: [R][4*tiles]
  float* p_sum;            //         [R][4*tiles]
  float* c_val;            //         [R][4*tiles][B]
  int* c_id;               //         [R][4*tiles][B]
  int* status;             // device status word (may be nullptr)
};

// xs2: the stage holds two activation tiles (high-order and low-order terms), multiplied one after the other into
// the same accumulator -- the two-term form for more than 128 rows, where the terms no longer fit side by side
// in the N of one instruction.
__host__ __device__ constexpr int ws_stage_bytes(int npad, bool xs2 = false) { return WS_W_BYTES + (xs2 ? 2 : 1) * npad * WS_BK * 2; }
__host__ __device__ constexpr int ws_stages(int npad, bool xs2 = false) {
  return (WS_SMEM_BUDGET / ws_stage_bytes(npad, xs2)) > 12 ? 12 : (WS_SMEM_BUDGET / ws_stage_bytes(npad, xs2));
}
__host__ __device__ constexpr int ws_smem_bytes(int npad, bool xs2 = false) {
  return ws_stages(npad, xs2) * ws_stage_bytes(npad, xs2) + 1024 + 256;
}

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Non-blocking look at a barrier phase (try_wait may park the thread for a while; a polling loop must not).
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait. Returns false when the abort flag is up or the time limit passed (and raises the flag).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try(bar, parity)) return true;
  const long long t0 = clock64();
  for (uint32_t spin = 1;; ++spin) {
    if (mbar_try(bar, parity)) return true;
    if ((spin & 255u) == 0u) {
      if (*abort_flag) return false;
      if (clock64() - t0 > WS_WAIT_CYCLES) {
        *abort_flag = 1;
        return false;
      }
    }
  }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
// The same copy with an L2 eviction-priority hint. Weight tiles are read once per call: marking them evict-first
// keeps a gigabyte of LM-head weights from flushing what the chain re-reads (activations, partial planes, the
// attention caches, the kernels' own code) out of L2.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(bar), "l"(pol)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor of a K-major bf16 tile stored as 128-byte rows with the 128B swizzle:
// 8-row groups lie 1024 bytes apart (stride byte offset), the leading byte offset is unused.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) |
         (2ull << 61);
}
// Instruction descriptor: D = fp32, A = B = bf16, both K-major, M = 128, N = npad.
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int m, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

__device__ __forceinline__ bool ranks_before(float va, int ia, float vb, int ib) {
  return va > vb || (va == vb && ia < ib);
}

// ---------------------------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------------------------
template <int NPAD, bool XS2>
__global__ void __launch_bounds__(WS_THREADS, 1) wstream_gemm_kernel(const __grid_constant__ WsParams P) {
  constexpr int STAGES = ws_stages(NPAD, XS2);
  constexpr int STAGE_BYTES = ws_stage_bytes(NPAD, XS2);
  constexpr int X_BYTES = NPAD * WS_BK * 2;       // one activation tile
  // two accumulators of NPAD columns; the allocation is a power of two of at least 32 columns
  constexpr uint32_t TMEM_COLS = (2 * NPAD) <= 32 ? 32 : (2 * NPAD) <= 64 ? 64 : (2 * NPAD) <= 128 ? 128 : (2 * NPAD) <= 256 ? 256 : 512;
  constexpr uint32_t IDESC = umma_idesc_bf16(WS_BM, NPAD);

  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;       // swizzled tiles need 1024-byte alignment
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  uint64_t* bars = (uint64_t*)(base_ptr + STAGES * STAGE_BYTES);      // full[STAGES], empty[STAGES], tfull[2], tempty[2]
  const uint32_t bar0 = base + STAGES * STAGE_BYTES;
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
  auto tfull_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + b); };
  auto tempty_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + 2 + b); };
  uint32_t* tmem_slot = (uint32_t*)(bars + 2 * STAGES + 4);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int units = P.tiles_total * P.splits;
  pdl_trigger();       // the next kernel of the chain may start its own set-up

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(tfull_bar(b), 1);
      mbar_init(tempty_bar(b), 256);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // unit -> (tile, split) -> (segment, first weight row, k-block range)
  auto decode = [&](int u, int& seg, int& n0, int& kb0, int& kb1, int& split, int& tile) {
    tile = u / P.splits;
    split = u - tile * P.splits;
    seg = 0;
    if (P.n_seg > 1 && tile >= P.seg_tile0[1]) seg = 1;
    if (P.n_seg > 2 && tile >= P.seg_tile0[2]) seg = 2;
    n0 = (tile - P.seg_tile0[seg]) * WS_BM;
    kb0 = (int)(((long long)split * P.kb_total) / P.splits);
    kb1 = (int)(((long long)(split + 1) * P.kb_total) / P.splits);
  };

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      // Weights depend on nothing: the tiles of the first ring pass go out at once. The activations were
      // written by the kernel before this one, so their tiles wait for it (programmatic dependent launch).
      const uint64_t w_policy = l2_policy_evict_first();
      uint32_t pre = 0;
      for (int u = blockIdx.x; u < units && pre < (uint32_t)STAGES; u += gridDim.x) {
        int seg, n0, kb0, kb1, split, tile;
        decode(u, seg, n0, kb0, kb1, split, tile);
        for (int kb = kb0; kb < kb1 && pre < (uint32_t)STAGES; ++kb, ++pre) {
          mbar_expect_tx(full_bar(pre), STAGE_BYTES);
          tma_load_2d_hint(base + pre * STAGE_BYTES, &P.tmW[seg], kb * WS_BK, n0, full_bar(pre), w_policy);
        }
      }
      pdl_wait(KID_GEMM);
      {
        uint32_t i2 = 0;
        for (int u = blockIdx.x; u < units && i2 < pre; u += gridDim.x) {
          int seg, n0, kb0, kb1, split, tile;
          decode(u, seg, n0, kb0, kb1, split, tile);
          for (int kb = kb0; kb < kb1 && i2 < pre; ++kb, ++i2) {
            tma_load_2d(base + i2 * STAGE_BYTES + WS_W_BYTES, &P.tmX, kb * WS_BK, 0, full_bar(i2));
            if (XS2) tma_load_2d(base + i2 * STAGE_BYTES + WS_W_BYTES + X_BYTES, &P.tmX, kb * WS_BK, P.lo_row, full_bar(i2));
          }
        }
      }
      uint32_t it = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < units && ok; u += gridDim.x) {
        int seg, n0, kb0, kb1, split, tile;
        decode(u, seg, n0, kb0, kb1, split, tile);
        const CUtensorMap* tw = &P.tmW[seg];
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          if (it < pre) continue;               // went out above
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) { ok = false; break; }
          mbar_expect_tx(full_bar(s), STAGE_BYTES);
          const uint32_t dst = base + s * STAGE_BYTES;
          tma_load_2d_hint(dst, tw, kb * WS_BK, n0, full_bar(s), w_policy);
          tma_load_2d(dst + WS_W_BYTES, &P.tmX, kb * WS_BK, 0, full_bar(s));
          if (XS2) tma_load_2d(dst + WS_W_BYTES + X_BYTES, &P.tmX, kb * WS_BK, P.lo_row, full_bar(s));
        }
      }
      if (!ok) {
        // give the copies already issued a bounded time to land before the CTA tears down
        const uint32_t pending = it < (uint32_t)STAGES ? it : (uint32_t)STAGES;
        for (uint32_t j = 0; j < pending; ++j) {
          const uint32_t i2 = it - 1 - j;
          const long long t0 = clock64();
          while (!mbar_try(full_bar(i2 % STAGES), (i2 / STAGES) & 1u) && clock64() - t0 < 20000000ll) {
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0) {
      uint32_t it = 0;
      int j = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < units && ok; u += gridDim.x, ++j) {
        int seg, n0, kb0, kb1, split, tile;
        decode(u, seg, n0, kb0, kb1, split, tile);
        const int buf = j & 1;
        const uint32_t bph = (uint32_t)(j >> 1) & 1u;
        if (!mbar_wait(tempty_bar(buf), bph ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * NPAD);
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          if (!mbar_wait(full_bar(s), ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t wa = base + s * STAGE_BYTES;
          const uint64_t adesc = umma_desc_sw128(wa);
          const uint64_t bdesc = umma_desc_sw128(wa + WS_W_BYTES);
#pragma unroll
          for (int kk = 0; kk < WS_BK / 16; ++kk) {
            // advancing 16 k-elements = 32 bytes inside the swizzled row: +2 in the descriptor's 16-byte units
            tc_mma_bf16(d_tmem, adesc + 2u * kk, bdesc + 2u * kk, IDESC, (kb > kb0 || kk > 0) ? 1u : 0u);
          }
          if (XS2) {                       // W x = W hi + W lo, the second product into the same accumulator
            const uint64_t ldesc = umma_desc_sw128(wa + WS_W_BYTES + X_BYTES);
#pragma unroll
            for (int kk = 0; kk < WS_BK / 16; ++kk) tc_mma_bf16(d_tmem, adesc + 2u * kk, ldesc + 2u * kk, IDESC, 1u);
          }
          tc_commit(empty_bar(s));       // frees the stage once these MMAs have read it
        }
        if (ok) tc_commit(tfull_bar(buf));
      }
    }
  } else {
    // ------------------------------ epilogue ------------------------------
    const int q = warp & 3;                 // TMEM lane quadrant this warp may read
    const int ehalf = (warp - 2) >> 2;      // the quadrant's two warps take alternate groups of 16 activation rows
    int j = 0;
    bool ok = true;
    for (int u = blockIdx.x; u < units && ok; u += gridDim.x, ++j) {
      int seg, n0, kb0, kb1, split, tile;
      decode(u, seg, n0, kb0, kb1, split, tile);
      const int buf = j & 1;
      const uint32_t bph = (uint32_t)(j >> 1) & 1u;
      if (!mbar_wait(tfull_bar(buf), bph, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const int nrow = n0 + q * 32 + lane;                  // weight row inside the segment
      const bool valid = nrow < P.seg_n[seg];
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * NPAD);
      if (P.mode == 0) {
        float* plane = P.out + (size_t)split * P.plane + P.seg_col[seg] + nrow;
#pragma unroll 1
        for (int c0 = ehalf * 16; c0 < NPAD; c0 += 32) {
          if (c0 >= P.R) break;
          float v[16];
          tc_ld16(taddr + c0, v);
          if (P.xsplit) {                       // W x = W hi + W lo
            float w2[16];
            tc_ld16(taddr + NPAD / 2 + c0, w2);
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] += w2[i];
          }
          if (valid) {
#pragma unroll
            for (int i = 0; i < 16; ++i)
              if (c0 + i < P.R) plane[(size_t)(c0 + i) * P.ldo] = v[i];
          }
        }
      } else {
        const int sub = tile * 4 + q;                         // 32-row vocabulary slice
        const int n_sub = 4 * P.tiles_total;
        const int B = P.B;
#pragma unroll 1
        for (int c0 = ehalf * 16; c0 < NPAD; c0 += 32) {
          if (c0 >= P.R) break;
          float v[16];
          tc_ld16(taddr + c0, v);
          if (P.xsplit) {
            float w2[16];
            tc_ld16(taddr + NPAD / 2 + c0, w2);
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] += w2[i];
          }
          // EPI_U activation rows at a time: their shuffle chains are independent and interleave
#pragma unroll
          for (int i = 0; i < 16; i += EPI_U) {
            if (c0 + i < P.R) {
              float val[EPI_U], wmax[EPI_U], wsum[EPI_U];
              int id[EPI_U];
#pragma unroll
              for (int u = 0; u < EPI_U; ++u) {
                val[u] = valid ? v[i + u] : -INFINITY;
                id[u] = nrow;
                wmax[u] = val[u];
              }
#pragma unroll
              for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
                for (int u = 0; u < EPI_U; ++u) wmax[u] = fmaxf(wmax[u], __shfl_xor_sync(0xffffffffu, wmax[u], o));
              }
#pragma unroll
              for (int u = 0; u < EPI_U; ++u) wsum[u] = (valid && wmax[u] > -INFINITY) ? __expf(val[u] - wmax[u]) : 0.f;
#pragma unroll
              for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
                for (int u = 0; u < EPI_U; ++u) wsum[u] += __shfl_xor_sync(0xffffffffu, wsum[u], o);
              }
              // bitonic sort of the 32 (value, id) pairs: best (largest value, then smallest id) ends in lane 0
#pragma unroll
              for (int k = 2; k <= 32; k <<= 1) {
#pragma unroll
                for (int jj = k >> 1; jj > 0; jj >>= 1) {
                  const bool want_better = ((lane & jj) == 0) == ((lane & k) == 0);
#pragma unroll
                  for (int u = 0; u < EPI_U; ++u) {
                    const float ov = __shfl_xor_sync(0xffffffffu, val[u], jj);
                    const int oi = __shfl_xor_sync(0xffffffffu, id[u], jj);
                    if (want_better == ranks_before(ov, oi, val[u], id[u])) { val[u] = ov; id[u] = oi; }
                  }
                }
              }
#pragma unroll
              for (int u = 0; u < EPI_U; ++u) {
                const int r = c0 + i + u;
                if (r < P.R) {
                  const size_t at = (size_t)r * n_sub + sub;       // row-major over slices: the merge reads them coalesced
                  if (lane < B) {
                    P.c_val[at * B + lane] = val[u];
                    P.c_id[at * B + lane] = id[u];
                  }
                  if (lane == 0) {
                    P.p_max[at] = wmax[u];
                    P.p_sum[at] = wsum[u];
                  }
                }
              }
            }
          }
        }
      }
      tc_fence_before();
      mbar_arrive(tempty_bar(buf));
    }
  }

  // ------------------------------ teardown ------------------------------
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
  if (threadIdx.x == 0 && *abort_flag && P.status) atomicMax(P.status, DEV_ERR_TIMEOUT);
}

// ---------------------------------------------------------------------------------------------
// LM-head merge: combines the per-slice partials of one activation row into logsumexp and the global top-B,
// ordered by (log-probability descending, id ascending). The kernel is latency-bound (a few MB, many
// dependent steps), so a row is spread over several CTAs and the steps are kept few:
//   level 1, CTA (chunk, row): MERGE_CHUNK slices of the row.
//     1. every thread loads (max, sum exp, best value, best id) of the <= MERGE_OWN slices it owns;
//     2. the chunk's (max, sum exp);
//     3. threshold = the B-th best slice head of the chunk (each slice list is sorted, so its head is its
//        best): B rounds of "best ranking strictly after the previous pick", per warp over registers, then
//        over the warp lists;
//     4. only slices whose head ranks at or before the threshold can contribute (at most B of them): their
//        owners load the whole B-entry list and keep what passes the threshold (at most B*B survivors),
//        which are ranked by counting: the chunk's sorted top-B goes to global scratch;
//   level 2, the LAST CTA of the row to finish (one atomic arrival per CTA on the row's counter, which the
//     last one sets back to zero): logsumexp over the chunks, rank by counting over the chunks' B entries each.
// The global top-B is a subset of the union of the chunks' top-B lists, so the result is exact.
// ---------------------------------------------------------------------------------------------
constexpr int MERGE_THREADS = 256;
constexpr int MERGE_MAXB = 16;
constexpr int MERGE_OWN = 2;                                // slices per thread
constexpr int MERGE_CHUNK = MERGE_THREADS * MERGE_OWN;      // slices per CTA
constexpr int MERGE_MAXCHUNKS = 16;                         // up to 8192 slices = 262144 vocabulary rows
constexpr int MERGE_WARPS = MERGE_THREADS / 32;

__device__ __forceinline__ void warp_best(float& bv, int& bi) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (ranks_before(ov, oi, bv, bi)) { bv = ov; bi = oi; }
  }
}

struct MergeScratch {      // level-1 results, [R][n_chunks] each
  float* ms;               // (max, sum exp) pairs
  float* val;              // [B] sorted values
  int* id;                 // [B] their ids
  int* count;              // [R] arrival counters: zero before the first launch, left at zero by every launch
};

__global__ void __launch_bounds__(MERGE_THREADS) lm_merge_kernel(const float* __restrict__ p_max,
                                                                 const float* __restrict__ p_sum,
                                                                 const float* __restrict__ c_val,
                                                                 const int* __restrict__ c_id, int n_sub, int R, int B,
                                                                 MergeScratch sc, int* __restrict__ ids,
                                                                 float* __restrict__ logp) {
  pdl_trigger();
  pdl_wait(KID_LM_MERGE);
  __shared__ float red[33];
  __shared__ float w_val[MERGE_WARPS][MERGE_MAXB];
  __shared__ int w_id[MERGE_WARPS][MERGE_MAXB];
  __shared__ float t_val;
  __shared__ int t_id;
  __shared__ float s_val[MERGE_MAXB * MERGE_MAXB];
  __shared__ int s_id[MERGE_MAXB * MERGE_MAXB];
  __shared__ int n_surv;
  __shared__ int is_last;
  __shared__ float lse_sh;
  const int chunk = blockIdx.x, n_chunks = gridDim.x, r = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int NONE = 0x7fffffff;
  const size_t row = (size_t)r * n_sub;
  const size_t slot = (size_t)r * n_chunks + chunk;
  if (tid == 0) n_surv = 0;
  if (tid < B) { sc.val[slot * B + tid] = -INFINITY; sc.id[slot * B + tid] = NONE; }
  // 1. this thread's slices
  float hv[MERGE_OWN], pm[MERGE_OWN], ps[MERGE_OWN];
  int hi[MERGE_OWN];
#pragma unroll
  for (int j = 0; j < MERGE_OWN; ++j) {
    const int s = chunk * MERGE_CHUNK + tid + j * MERGE_THREADS;
    const bool in = s < n_sub;
    pm[j] = in ? p_max[row + s] : -INFINITY;
    ps[j] = in ? p_sum[row + s] : 0.f;
    hv[j] = in ? c_val[(row + s) * B] : -INFINITY;
    hi[j] = in ? c_id[(row + s) * B] : NONE;
  }
  // 2. the chunk's (max, sum exp)
  float m = -INFINITY;
#pragma unroll
  for (int j = 0; j < MERGE_OWN; ++j) m = fmaxf(m, pm[j]);
  m = block_max(m, red);
  float se = 0.f;
#pragma unroll
  for (int j = 0; j < MERGE_OWN; ++j)
    if (pm[j] > -INFINITY) se += ps[j] * __expf(pm[j] - m);
  se = block_sum(se, red);
  if (tid == 0) { sc.ms[slot * 2] = m; sc.ms[slot * 2 + 1] = se; }
  // 3a. per warp: the B best heads among this warp's slices
  float pv = INFINITY;
  int pi = -1;
  for (int round = 0; round < B; ++round) {
    float bv = -INFINITY;
    int bi = NONE;
#pragma unroll
    for (int j = 0; j < MERGE_OWN; ++j)
      if (ranks_before(pv, pi, hv[j], hi[j]) && ranks_before(hv[j], hi[j], bv, bi)) { bv = hv[j]; bi = hi[j]; }
    warp_best(bv, bi);
    pv = bv;
    pi = bi;
    if (lane == 0) { w_val[wid][round] = bv; w_id[wid][round] = bi; }
  }
  __syncthreads();
  // 3b. warp 0: the B-th best over the sorted warp lists
  if (wid == 0) {
    float qv = INFINITY;
    int qi = -1;
    int cur = 0;                                  // this lane's list is sorted: a cursor is enough
    for (int round = 0; round < B; ++round) {
      float bv = (lane < MERGE_WARPS && cur < B) ? w_val[lane][cur] : -INFINITY;
      int bi = (lane < MERGE_WARPS && cur < B) ? w_id[lane][cur] : NONE;
      const float mv = bv;
      const int mi = bi;
      warp_best(bv, bi);
      if (mv == bv && mi == bi && bi != NONE) ++cur;   // this lane's head was taken
      qv = bv;
      qi = bi;
    }
    if (lane == 0) { t_val = qv; t_id = qi; }
  }
  __syncthreads();
  const float tv = t_val;
  const int ti = t_id;
  // 4. survivors: whole lists of the slices whose head passes, loaded at once
#pragma unroll
  for (int j = 0; j < MERGE_OWN; ++j) {
    const int s = chunk * MERGE_CHUNK + tid + j * MERGE_THREADS;
    if (s >= n_sub || hi[j] == NONE || ranks_before(tv, ti, hv[j], hi[j])) continue;
    float lv[MERGE_MAXB];
    int li[MERGE_MAXB];
#pragma unroll
    for (int c = 0; c < MERGE_MAXB; ++c) {
      lv[c] = c < B ? c_val[(row + s) * B + c] : -INFINITY;
      li[c] = c < B ? c_id[(row + s) * B + c] : NONE;
    }
#pragma unroll
    for (int c = 0; c < MERGE_MAXB; ++c) {
      if (c >= B || li[c] == NONE || ranks_before(tv, ti, lv[c], li[c])) continue;
      const int at = atomicAdd(&n_surv, 1);
      if (at < MERGE_MAXB * MERGE_MAXB) { s_val[at] = lv[c]; s_id[at] = li[c]; }
    }
  }
  __syncthreads();
  {
    const int ns = n_surv < MERGE_MAXB * MERGE_MAXB ? n_surv : MERGE_MAXB * MERGE_MAXB;
    if (tid < ns) {
      const float v = s_val[tid];
      const int id = s_id[tid];
      int rank = 0;
      for (int j = 0; j < ns; ++j) rank += ranks_before(s_val[j], s_id[j], v, id) ? 1 : 0;
      if (rank < B) { sc.val[slot * B + rank] = v; sc.id[slot * B + rank] = id; }
    }
  }
  // ---- arrival: the row's last CTA does level 2 ----
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int seen = atomicAdd(sc.count + r, 1);
    is_last = seen == n_chunks - 1 ? 1 : 0;
    if (is_last) sc.count[r] = 0;            // every CTA of the row has arrived: nobody touches it again
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  if (tid < B) { ids[(size_t)r * B + tid] = -1; logp[(size_t)r * B + tid] = -INFINITY; }
  if (wid == 0) {
    const bool in = lane < n_chunks;         // n_chunks <= MERGE_MAXCHUNKS <= 32
    const float cm = in ? __ldcg(sc.ms + ((size_t)r * n_chunks + lane) * 2) : -INFINITY;
    const float cs = in ? __ldcg(sc.ms + ((size_t)r * n_chunks + lane) * 2 + 1) : 0.f;
    const float M = warp_max(cm);
    const float S = warp_sum(cm > -INFINITY ? cs * __expf(cm - M) : 0.f);
    if (lane == 0) lse_sh = M + logf(S);
  }
  const int nc = n_chunks * B;               // <= 256 candidates, sorted within each chunk
  if (tid < nc) {
    s_val[tid] = __ldcg(sc.val + (size_t)r * n_chunks * B + tid);
    s_id[tid] = __ldcg(sc.id + (size_t)r * n_chunks * B + tid);
  }
  __syncthreads();
  if (tid < nc && s_id[tid] != NONE) {
    const float v = s_val[tid];
    const int id = s_id[tid];
    int rank = 0;
    for (int j = 0; j < nc; ++j) rank += ranks_before(s_val[j], s_id[j], v, id) ? 1 : 0;
    if (rank < B) {
      ids[(size_t)r * B + rank] = id;
      logp[(size_t)r * B + rank] = v - lse_sh;
    }
  }
}

}  // namespace moa
