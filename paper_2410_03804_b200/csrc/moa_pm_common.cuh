// Phase machine, part 1: descriptors, small device helpers and the static GEMM schedule.
//
// The phase machine is one persistent cooperative kernel that runs a whole LSA pass of more than 256 (token,
// layer) rows as a list of phases separated by grid-wide barriers; see moa_phases.cuh for the kernel and the
// reasons. This file holds what its parts share.
#pragma once
#include "moa_attn.cuh"
#include "moa_basic.cuh"
#include "moa_wstream.cuh"

namespace moa {

constexpr int PM_THREADS = 256;
constexpr int PM_WORKERS = 192;          // warps 2..7
constexpr int PM_WWARPS = 6;
constexpr int PM_MAX_OPS = 16;
constexpr int PM_MAX_GEMMS = 10;
constexpr int PM_MAX_STAGES = 12;
constexpr int PM_MAXCH = 6;              // 8-element chunks a thread keeps of one row (rows up to 9216 wide)

enum PmKind : int {
  PH_GEMM = 0, PH_ROWS_NORM, PH_RESNORM, PH_MEAN_NORM, PH_CACHE_APPEND, PH_LSA_ATTN
};

struct PmGemm {            // (its tensor maps are PmParams.tm[gemm][0..2] weights, [3] activations)
  int n_seg, seg_n[3], seg_tile0[3], seg_col[3];
  int tiles_total;         // weight tiles (gated: gate/up tile pairs)
  int kb_total, splits, row_blocks;
  int units, rot;          // tiles_total * splits * row_blocks; unit u runs on CTA (u + rot) % grid
  int mode;                // 0 fp32 split planes, 2 bf16 store, 3 residual add, 4 gated SwiGLU
  int R;                   // valid activation rows
  int rows_per_block;      // X rows per unit: NB, or 128 when gated
  int ldo;                 // modes 0, 3: leading dimension of out
  int ld16;                // modes 2, 4
  size_t plane;            // mode 0: elements between split planes
  float* out;              // mode 0: planes; mode 3: fp32 residual stream
  bf16* out16;             // modes 2, 4
};

struct PmOp {
  int kind;
  int gemm;                // PH_GEMM: which; glue: the GEMM whose split planes are consumed (-1: none)
  int rows, cols;          // rows and width the op works on
  const void* p[12];
  int i[16];
  float f[2];
};

struct PmParams {
  CUtensorMap tm[PM_MAX_GEMMS][4];   // per GEMM: weight matrices [n_i, K] (box 64 x 128, swizzle 128B) and, last,
                                     // its X buffer [rows, K] (box 64 x NB; gated: 64 x 128)
  PmGemm g[PM_MAX_GEMMS];
  PmOp op[PM_MAX_OPS];
  SeqSplit split;          // PH_CACHE_APPEND
  int n_ops, n_gemms;
  int stages;              // ring depth
  int alias_attn;          // attention scratch lies over the ring: no weight run-ahead across phases
  uint32_t attn_off;       // byte offset of the attention scratch from the aligned shared-memory base
  int* sync;               // device int[4]: [0] barrier counter, [1] abort word, [2] exit counter
  int* flags;              // device int[grid * 32]: per-CTA barrier flag, one 128-byte line each (zero between launches)
  int* status;             // device status word
  unsigned long long* trace;   // [2 * PM_MAX_OPS + 1] ns timestamps of CTA 0: start, then per phase: work done, barrier passed
};

// What every role reads all the time, copied from the kernel parameters into shared memory at start-up
// (the tensor maps stay in parameter space, where TMA wants them).
struct PmSmem {
  PmOp op[PM_MAX_OPS];
  PmGemm g[PM_MAX_GEMMS];
  SeqSplit split;
  int n_ops;
  float red[8];            // worker-wide reductions
};
constexpr int PM_FIXED_SMEM = 1024 + 512 + (int)((sizeof(PmSmem) + 127) / 128) * 128;   // alignment slack, barriers, PmSmem

template <int NB>
__host__ __device__ constexpr int pm_stage_bytes() { return WS_W_BYTES + NB * WS_BK * 2; }

// ---------------------------------------------------------------------------------------------
// small helpers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void wbar() { asm volatile("bar.sync 1, %0;" ::"n"(PM_WORKERS) : "memory"); }

__device__ __forceinline__ float worker_sum(float v, float* red, int wt) {
  v = warp_sum(v);
  if ((wt & 31) == 0) red[wt >> 5] = v;
  wbar();
  float t = 0.f;
#pragma unroll
  for (int i = 0; i < PM_WWARPS; ++i) t += red[i];
  wbar();
  return t;
}

// ---------------------------------------------------------------------------------------------
// static schedule of the GEMM phases as seen by one CTA (same arithmetic in the three roles)
// ---------------------------------------------------------------------------------------------
struct PmUnit {
  int seg, n0, kb0, kb1, split, tile, rb;
};

__device__ __forceinline__ void pm_decode(const PmGemm& G, int u, PmUnit& d) {
  // unit -> (row-block group, tile, row block in group) with 4 row blocks per group, or (tile, split)
  int tile, rb = 0, split = 0;
  if (G.row_blocks > 1) {
    const int per_group = G.tiles_total * 4;
    const int grp = u / per_group;
    const int rem = u - grp * per_group;
    const int left = G.row_blocks - grp * 4;
    const int ge = left < 4 ? left : 4;
    tile = rem / ge;
    rb = grp * 4 + (rem - tile * ge);
  } else {
    tile = u / G.splits;
    split = u - tile * G.splits;
  }
  d.tile = tile; d.rb = rb; d.split = split;
  int seg = 0;
  if (G.n_seg > 1 && tile >= G.seg_tile0[1]) seg = 1;
  if (G.n_seg > 2 && tile >= G.seg_tile0[2]) seg = 2;
  if (G.mode == 4) seg = 0;
  d.seg = seg;
  d.n0 = (tile - G.seg_tile0[seg]) * WS_BM;
  d.kb0 = (int)(((long long)split * G.kb_total) / G.splits);
  d.kb1 = (int)(((long long)(split + 1) * G.kb_total) / G.splits);
}

__device__ __forceinline__ int pm_first_unit(const PmGemm& G) {
  const int g = (int)gridDim.x;
  int u = ((int)blockIdx.x - G.rot) % g;
  if (u < 0) u += g;
  return u;
}

// Cursor over (GEMM phase, unit, k block) of this CTA, in schedule order, with the per-unit values the
// producer needs for every stage worked out once per unit.
struct PmCursor {
  int opi;      // index into the phase list of the current GEMM phase (n_ops: done)
  int u, kb, kb1;
  const CUtensorMap* tw;   // weight map of the unit's segment
  const CUtensorMap* tw2;  // gated: the up-projection map, else null
  const CUtensorMap* tx;
  int n0, xrow;            // weight-tile row, activation-tile row
  uint32_t bytes, xoff;    // bytes one stage receives; offset of the activation tile inside the stage
  __device__ __forceinline__ void seek(const PmSmem& S, const PmParams& P) {     // first stage at or after (opi, u)
    while (opi < S.n_ops) {
      if (S.op[opi].kind == PH_GEMM) {
        const int gi = S.op[opi].gemm;
        const PmGemm& G = S.g[gi];
        if (u < 0) u = pm_first_unit(G);
        if (u < G.units) {
          PmUnit d;
          pm_decode(G, u, d);
          kb = d.kb0; kb1 = d.kb1;
          const bool gated = G.mode == 4;
          tw = &P.tm[gi][d.seg]; tw2 = gated ? &P.tm[gi][1] : nullptr; tx = &P.tm[gi][3];
          n0 = d.n0; xrow = d.rb * G.rows_per_block;
          xoff = gated ? 2 * WS_W_BYTES : WS_W_BYTES;
          bytes = xoff + (uint32_t)G.rows_per_block * WS_BK * 2;
          return;
        }
      }
      ++opi;
      u = -1;
    }
  }
  __device__ __forceinline__ void init(const PmSmem& S, const PmParams& P) { opi = 0; u = -1; kb = 0; kb1 = 0; seek(S, P); }
  __device__ __forceinline__ bool done(const PmSmem& S) const { return opi >= S.n_ops; }
  __device__ __forceinline__ void next(const PmSmem& S, const PmParams& P) {
    if (++kb < kb1) return;
    u += (int)gridDim.x;
    seek(S, P);
  }
};

}  // namespace moa
