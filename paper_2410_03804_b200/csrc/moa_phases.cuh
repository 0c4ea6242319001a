// Phase machine: one persistent cooperative kernel that runs a whole LSA pass of more than 256 (token, layer)
// rows -- the dense regime, where the projections are tensor-core-bound GEMMs -- as a list of phases separated by
// grid-wide barriers.
//
// Why one kernel: the pass is six GEMMs with fused epilogues and four short glue phases over the same rows;
// separate launches would write and re-read every intermediate through HBM and drain the tensor pipe at every
// link. Here one CTA per SM stays resident for the whole pass and
//   warp 0      streams weight tiles with TMA along the STATIC schedule of all GEMM phases, running ahead
//               of the phase that is executing (weights depend on nothing), as far as the shared-memory
//               ring allows; only the small activation tile of a stage waits for its phase to open;
//   warp 1      issues tcgen05.mma (weights = A operand, M = 128; activation rows = B operand);
//   warps 2..5  drain the TMEM accumulators (epilogues), and together with
//   warps 6..7  execute the glue phases (norms, layer self-attention, layer mean, cache append) between the GEMMs.
// Phases are separated by a grid barrier (one atomic arrival per CTA; the last arrival raises a flag per
// CTA, each on its own cache line; bounded polling; the launch is cooperative so all CTAs are resident).
// Every wait is bounded: on expiry a CTA raises the abort word, every CTA drains, frees TMEM and returns,
// and the status word reads MOA_ERR_TIMEOUT.
#pragma once
#include "moa_pm_common.cuh"
#include "moa_pm_glue.cuh"
#include "moa_pm_lsa.cuh"

namespace moa {

// A chain of tcgen05.mma instructions that accumulate into the same TMEM tile is serialised by the tensor
// pipe's latency, and with few activation rows (small N) that latency, not the math, sets the pace: four
// dependent K=16 steps per 16 KB weight stage cost about as much time as HBM needs to deliver the stage. So the
// k-steps of a stage rotate over PM_ACC independent accumulators, and the epilogue adds them up.
template <int NB>
__host__ __device__ constexpr int pm_acc() { return NB <= 64 ? 4 : (NB <= 128 ? 2 : 1); }

// 16 accumulator columns starting at column c of the unit's buffer: sum over the independent accumulators.
template <int NB>
__device__ __forceinline__ void pm_ld16(uint32_t taddr, int c, float* v) {
  tc_ld16(taddr + c, v);
#pragma unroll
  for (int a = 1; a < pm_acc<NB>(); ++a) {
    float w[16];
    tc_ld16(taddr + a * NB + c, w);
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] += w[i];
  }
}

// ---- epilogue of one GEMM unit: TMEM accumulator -> global, by the four epilogue warps ----
template <int NB>
__device__ __forceinline__ void pm_epilogue(const PmGemm& Gm, const PmUnit& d, uint32_t taddr, int q, int lane) {
  const int nrow = d.n0 + q * 32 + lane;
  const bool valid = nrow < Gm.seg_n[d.seg];
  const int r0 = d.rb * Gm.rows_per_block;
  const int rows = min(Gm.R - r0, Gm.rows_per_block);
  if (Gm.mode == 0) {
    float* plane = Gm.out + (size_t)d.split * Gm.plane + Gm.seg_col[d.seg] + nrow;
#pragma unroll 1
    for (int c0 = 0; c0 < rows; c0 += 16) {
      float v[16];
      pm_ld16<NB>(taddr, c0, v);
      if (valid) {
#pragma unroll
        for (int i = 0; i < 16; ++i)
          if (c0 + i < rows) plane[(size_t)(r0 + c0 + i) * Gm.ldo] = v[i];
      }
    }
  } else if (Gm.mode == 2 || Gm.mode == 3) {
    const int col = Gm.seg_col[d.seg] + nrow;
#pragma unroll 1
    for (int c0 = 0; c0 < rows; c0 += 16) {
      float v[16];
      pm_ld16<NB>(taddr, c0, v);
      if (valid) {
        if (Gm.mode == 2) {
#pragma unroll
          for (int i = 0; i < 16; ++i)
            if (c0 + i < rows) Gm.out16[(size_t)(r0 + c0 + i) * Gm.ld16 + col] = __float2bfloat16_rn(v[i]);
        } else {
          float old[16];
#pragma unroll
          for (int i = 0; i < 16; ++i)
            old[i] = c0 + i < rows ? __ldcg(Gm.out + (size_t)(r0 + c0 + i) * Gm.ldo + col) : 0.f;
#pragma unroll
          for (int i = 0; i < 16; ++i)
            if (c0 + i < rows) Gm.out[(size_t)(r0 + c0 + i) * Gm.ldo + col] = old[i] + v[i];
        }
      }
    }
  } else if (Gm.mode == 4) {
#pragma unroll 1
    for (int c0 = 0; c0 < rows; c0 += 16) {
      float gt[16], up[16];
      tc_ld16(taddr + c0, gt);
      tc_ld16(taddr + 128 + c0, up);
      if (valid) {
#pragma unroll
        for (int i = 0; i < 16; ++i)
          if (c0 + i < rows)
            Gm.out16[(size_t)(r0 + c0 + i) * Gm.ld16 + nrow] = __float2bfloat16_rn(gt[i] / (1.f + __expf(-gt[i])) * up[i]);
      }
    }
  }
}

// ---- MMA issuer role (one thread): walks the static schedule, one tcgen05.mma group per ring stage ----
template <int NB>
__device__ __noinline__ void pm_mma_role(const PmSmem& S, uint32_t base, uint32_t bar0, uint32_t tmem_base, int STAGES,
                                         volatile int* abort_flag) {
  constexpr int STAGE_BYTES = pm_stage_bytes<NB>();
  constexpr int ACC = pm_acc<NB>();
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (PM_MAX_STAGES + s); };
  auto tfull_bar = [&](int b) { return bar0 + 8u * (2 * PM_MAX_STAGES + b); };
  auto tempty_bar = [&](int b) { return bar0 + 8u * (2 * PM_MAX_STAGES + 2 + b); };
  const int G = (int)gridDim.x;
  int slot = 0;                     // ring slot and its phase parity, advanced stage by stage
  uint32_t slot_ph = 0;
  const uint64_t desc0 = umma_desc_sw128(base);   // descriptor of slot 0; slots lie STAGE_BYTES apart (< 256 KB in all)
  int j = 0;
  bool ok = true;
  for (int opi = 0; opi < S.n_ops && ok; ++opi) {
    if (S.op[opi].kind != PH_GEMM) continue;
    const PmGemm& Gm = S.g[S.op[opi].gemm];
    const bool gated = Gm.mode == 4;
    const uint32_t idesc = umma_idesc_bf16(WS_BM, gated ? 128 : NB);
    for (int u = pm_first_unit(Gm); u < Gm.units && ok; u += G, ++j) {
      PmUnit d;
      pm_decode(Gm, u, d);
      const int buf = j & 1;
      const uint32_t bph = (uint32_t)(j >> 1) & 1u;
      if (!mbar_wait(tempty_bar(buf), bph ^ 1u, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + (uint32_t)(buf * ACC * NB);
      for (int kb = d.kb0; kb < d.kb1; ++kb) {
        if (!mbar_wait(full_bar(slot), slot_ph, abort_flag)) { ok = false; break; }
        const uint64_t adesc = desc0 + (uint64_t)(slot * (STAGE_BYTES >> 4));
        const uint64_t bdesc = adesc + (uint64_t)((gated ? 2 * WS_W_BYTES : WS_W_BYTES) >> 4);
        const uint32_t acc0 = kb > d.kb0 ? 1u : 0u;
#pragma unroll
        for (int kk = 0; kk < WS_BK / 16; ++kk)   // k-step kk accumulates into accumulator kk % ACC
          tc_mma_bf16(d_tmem + (uint32_t)((kk % ACC) * NB), adesc + 2u * kk, bdesc + 2u * kk, idesc,
                      (acc0 | (kk >= ACC)) ? 1u : 0u);
        if (gated) {
          const uint64_t adesc2 = adesc + (uint64_t)(WS_W_BYTES >> 4);
#pragma unroll
          for (int kk = 0; kk < WS_BK / 16; ++kk)
            tc_mma_bf16(d_tmem + 128u, adesc2 + 2u * kk, bdesc + 2u * kk, idesc, (acc0 | (kk > 0)) ? 1u : 0u);
        }
        tc_commit(empty_bar(slot));
        if (++slot == STAGES) { slot = 0; slot_ph ^= 1u; }
      }
      if (ok) tc_commit(tfull_bar(buf));
    }
  }

}

// ---------------------------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------------------------
template <int NB>
__global__ void __launch_bounds__(PM_THREADS, 1) phase_machine_kernel(const __grid_constant__ PmParams P) {
  constexpr int STAGE_BYTES = pm_stage_bytes<NB>();
  constexpr int ACC = pm_acc<NB>();
  constexpr uint32_t TMEM_COLS = 2 * ACC * NB;        // two buffers of ACC accumulators (64 .. 512 columns)

  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const int STAGES = P.stages;
  uint64_t* bars = (uint64_t*)(base_ptr + STAGES * STAGE_BYTES);   // full[12], empty[12], tfull[2], tempty[2]
  const uint32_t bar0 = base + STAGES * STAGE_BYTES;
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (PM_MAX_STAGES + s); };
  auto tfull_bar = [&](int b) { return bar0 + 8u * (2 * PM_MAX_STAGES + b); };
  auto tempty_bar = [&](int b) { return bar0 + 8u * (2 * PM_MAX_STAGES + 2 + b); };
  uint32_t* tmem_slot = (uint32_t*)(bars + 2 * PM_MAX_STAGES + 4);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);
  volatile int* phase_open = (volatile int*)(tmem_slot + 2);
  PmSmem& S = *reinterpret_cast<PmSmem*>(base_ptr + STAGES * STAGE_BYTES + 512);
  uint8_t* attn_gen = base_ptr + P.attn_off;
  const uint32_t attn_sh = base + P.attn_off;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = (int)gridDim.x;

  {   // phase and GEMM descriptors -> shared memory
    const int n_op_words = (int)(sizeof(PmOp) * PM_MAX_OPS / 4), n_g_words = (int)(sizeof(PmGemm) * PM_MAX_GEMMS / 4);
    const int n_s_words = (int)(sizeof(SeqSplit) / 4);
    const int* src_op = reinterpret_cast<const int*>(&P.op[0]);
    const int* src_g = reinterpret_cast<const int*>(&P.g[0]);
    const int* src_s = reinterpret_cast<const int*>(&P.split);
    int* dst_op = reinterpret_cast<int*>(&S.op[0]);
    int* dst_g = reinterpret_cast<int*>(&S.g[0]);
    int* dst_s = reinterpret_cast<int*>(&S.split);
    for (int i = threadIdx.x; i < n_op_words; i += PM_THREADS) dst_op[i] = src_op[i];
    for (int i = threadIdx.x; i < n_g_words; i += PM_THREADS) dst_g[i] = src_g[i];
    for (int i = threadIdx.x; i < n_s_words; i += PM_THREADS) dst_s[i] = src_s[i];
    if (threadIdx.x == 0) S.n_ops = P.n_ops;
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < PM_MAX_STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(tfull_bar(b), 1);
      mbar_init(tempty_bar(b), 128);
    }
    *abort_flag = 0;
    *phase_open = 0;
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

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    // Weight tiles go out as soon as their ring slot is free, whatever phase is executing; the activation
    // tile of a stage goes out with them when its phase is already open (the common case, a tight loop), and
    // otherwise later, from a second cursor that trails the first by at most the ring depth.
    if (lane == 0) {
      PmCursor wc, xc;
      wc.init(S, P);
      xc = wc;
      uint32_t w_it = 0, x_it = 0;
      long long t_last = clock64();
      uint32_t idle = 0;
      int open_seen = 0;                // last value read from phase_open
      int fenced_open = -1;             // phases up to this one have been fenced for on this thread
      auto fence_for = [&](int opi) {
        if (fenced_open < opi) {        // first activation tile of a newly opened phase: order it after the
          __threadfence();              // other CTAs' generic-proxy writes that the barrier made visible
          asm volatile("fence.proxy.async;" ::: "memory");
          fenced_open = open_seen;
        }
      };
      while (!(wc.done(S) && x_it == w_it)) {
        // ---- trailing activation tiles ----
        if (x_it < w_it) {
          if (open_seen < xc.opi) open_seen = *phase_open;
          if (open_seen >= xc.opi) {
            fence_for(xc.opi);
            const int s = x_it % STAGES;
            tma_load_2d(base + s * STAGE_BYTES + xc.xoff, xc.tx, xc.kb * WS_BK, xc.xrow, full_bar(s));
            xc.next(S, P);
            ++x_it;
            idle = 0;
            continue;
          }
        }
        // ---- next weight tile ----
        bool issued = false;
        if (!wc.done(S) && w_it - x_it < (uint32_t)STAGES) {
          const int s = w_it % STAGES;
          const uint32_t ph = (w_it / STAGES) & 1u;
          if (open_seen < wc.opi) open_seen = *phase_open;
          const bool open = open_seen >= wc.opi;
          if ((open || !P.alias_attn) && (w_it < (uint32_t)STAGES || mbar_test(empty_bar(s), ph ^ 1u))) {
            mbar_expect_tx(full_bar(s), wc.bytes);
            const uint32_t dst = base + s * STAGE_BYTES;
            tma_load_2d(dst, wc.tw, wc.kb * WS_BK, wc.n0, full_bar(s));
            if (wc.tw2) tma_load_2d(dst + WS_W_BYTES, wc.tw2, wc.kb * WS_BK, wc.n0, full_bar(s));
            if (x_it == w_it) {
              if (open) {               // both cursors sit on this stage: send the activation tile along
                fence_for(wc.opi);
                tma_load_2d(dst + wc.xoff, wc.tx, wc.kb * WS_BK, wc.xrow, full_bar(s));
                ++x_it;
              } else {
                xc = wc;                // the trailing cursor starts here
              }
            }
            wc.next(S, P);
            ++w_it;
            if (x_it == w_it) xc = wc;
            issued = true;
          }
        }
        if (issued) { idle = 0; continue; }
        // nothing to send: step out of the scheduler's way (worker warps share this SM partition)
        __nanosleep(idle < 8u ? 40u : 200u);
        if ((++idle & 255u) == 0u) {
          if (*abort_flag) break;
          const long long now = clock64();
          if (idle == 256u) t_last = now;
          if (now - t_last > WS_WAIT_CYCLES) { *abort_flag = 1; break; }
        }
      }
      if (*abort_flag) {
        // weight copies whose activation half never went out cannot complete their barrier; give the ones in
        // flight a bounded time to land before the CTA tears down
        const long long t1 = clock64();
        while (clock64() - t1 < 20000000ll) {
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0) pm_mma_role<NB>(S, base, bar0, tmem_base, STAGES, abort_flag);
  } else {
#include "moa_phases_workers.inc"
  }

  // ------------------------------ teardown ------------------------------
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
  if (threadIdx.x == 0) {
    if (*abort_flag) {
      atomicExch(P.sync + 1, 1);
      if (P.status) atomicMax(P.status, DEV_ERR_TIMEOUT);
    }
    P.flags[(size_t)blockIdx.x * 32] = 0;     // nobody raises it again: every barrier of this launch is behind us
    __threadfence();
    const int done = atomicAdd(P.sync + 2, 1);
    if (done == G - 1) {           // last CTA out: every CTA is past every barrier, so the counters can be rearmed
      P.sync[0] = 0;
      P.sync[1] = 0;
      P.sync[2] = 0;
      __threadfence();
    }
  }
}

}  // namespace moa
