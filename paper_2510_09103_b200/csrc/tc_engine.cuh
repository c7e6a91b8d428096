// A persistent, warp-specialised tcgen05 engine that runs a table of "items".  An item is a short
// list of K-loops ("segments") that accumulate into 128-row accumulators in tensor memory,
// followed by an epilogue that turns the accumulators into the result of one step of Algorithm 2:
//
//   refit of L (row panels of 128 rows of a block, Algorithm 2's L update):
//       D = g R^T + [L hi | L lo] X + [L0 hi | L0 lo] Y     X = [Bop1; Bop1], Bop1 = -(R R^T)/(1-b1)
//       L' = L + eta (1-b1) D                               Y = [Bop2; Bop2], Bop2 = b1 (R0 R^T)/(1-b1)
//   refit of R (column panels of 128 columns, the R update, computed transposed):
//       D = g^T L + [R^T hi | R^T lo] X' + [R0^T hi | R0^T lo] Y'   with -(L^T L)/(1-b1), b1 (L0^T L)/(1-b1)
//       R'^T = R^T + eta (1-b1) D
//   Gram item: one of the r x r matrices above, scaled and stored as a split-bf16 operand, twice, one
//       copy below the other, so that the hi and the lo columns of a factor meet the same rows.
//
// fp32 factors are carried into the bf16 tensor cores as hi + lo pairs (two bf16 numbers whose sum
// has ~16 significant bits); gradients are bf16 already and enter unchanged.  Operands with hi and
// lo parts are stored side by side ([rows, 2 half]: hi columns from 0, lo columns from `half`;
// half = rp = r rounded up to 16 while 2 rp <= 256, else rp rounded up to 64), so that used as the
// N side of an MMA the two parts land in two column ranges of the accumulator, which the epilogue
// adds.  While 2 rp <= 256 one MMA of N = 2 rp covers both parts; above that the hi and the lo part
// take one MMA of N = rp each, the second reading B from the chunk at which the lo part starts.
//
// A stage of the shared-memory ring holds `stage_k` (64 or 128) of K:
//   A  up to three operands of 128 rows x stage_k (K along x: boxes of 64 x 128) or stage_k x 128
//      columns (K along y: two boxes of 64 x stage_k).  All are multiplied with the same B and fill
//      one accumulator each: the more operands share a B, the fewer bytes a flop brings in
//   B  one 3-D box: stage_k rows x (64 x chunks) columns of a [rows, 2 half] array, i.e. the N side
//      read MN-major with its 64-column chunks one box apart
// Warp roles (512 threads, 128 registers each): warp 0 issues the TMA loads of a stage, warp 1 issues
// its MMAs, warps 4-7 add up g^2 per row from the gradient tiles of the first segment when the
// launch asks for it (the second-moment statistic of the block-mean form then needs no pass of its
// own over g), warps 8-15 drain the accumulators (two groups of four warps that take the 16-column
// pieces of an item alternately); warps 2 and 3 have no work.  The two issuing threads run dependent
// scalar code, so their per-stage instruction count is what bounds the rate; both loops are kept
// short.  With two accumulator buffers the epilogue of one item overlaps the K-loops of the next.
// Every wait is bounded; when one runs out the CTA records a status bit, stops taking work and
// leaves through the common exit (which frees its tensor memory).  A launch that finds the status
// word set on entry does nothing.
#pragma once

#include <cuda.h>

#include "tc_common.cuh"

namespace adapm {
namespace tc {

constexpr int kMaxSegs = 4;
constexpr int kMaxA = 3;
constexpr int kEngineThreads = 512;
constexpr uint32_t kTeamSpinDefault = 1u << 22;   // polls of 256 ns each: about a second
constexpr uint32_t kWaitSpinDefault = 1u << 23;   // mbarrier polls: at least as long as a team wait

enum : int32_t { EPI_FACTOR = 0, EPI_GRAM = 1, EPI_NONE = 2 };   // EPI_NONE: a filler that only keeps a CTA in step

struct Seg {
  int32_t map_a;             // 2-D tensor map: boxes of 64 x 128 (a_mode 0) or 64 x stage_k (a_mode 1)
  int32_t map_b;             // 3-D tensor map (64, rows, chunks), box 64 x stage_k x chunks
  int32_t ax[kMaxA], ay[kMaxA];   // element coordinates of the first box of each A operand
  int32_t k;                 // K extent, multiple of 16
  uint32_t tx_bytes;         // bytes one stage of this segment brings in
  int16_t a_mode;            // 0: K runs along x (K-major A), 1: K runs along y (MN-major A)
  int16_t n;                 // N of one MMA (multiple of 16, <= 256)
  int16_t n_a;               // A operands (1..kMaxA)
  int16_t n_mma;             // 1, or 2: a second MMA per K step reads B from chunk b2_chunk and adds at +d_part
  int16_t d_col[kMaxA];      // accumulator column of each A operand
  int16_t first;             // 1: its first MMA overwrites the accumulators
  int16_t b2_chunk, d_part;
  int16_t same_acc;          // 1: the A operands share one accumulator (all but the first always accumulate)
};

struct Item {
  Seg seg[kMaxSegs];
  int32_t n_seg;
  int32_t epi;
  // EPI_FACTOR: panel p (p < n_pan) has its accumulator at column acc_stride * p; the thread that owns
  // accumulator row q of panel p updates factor entries (owner = own0 + 128 p + q, k):
  //   f32[own_stride * owner + k_stride * k] += coef * (D[q][k] + D[q][rp + k])        k < r
  //   dst[owner][k] = hi, dst[owner][half + k] = lo                                    k < rp
  // EPI_GRAM: G[own0 + q][k] = coef * sum over n_sum parts (rp columns apart) of D[q][k]; stored like dst above,
  //   and once more stack_rows rows below                                              own0 + q, k < rp
  int32_t own0, own_count;   // first owner of the item and number of owners of the whole matrix
  int32_t n_pan, acc_stride;
  int32_t r, rp, half;
  int32_t n_sum, stack_rows;
  int32_t dst_ld;            // row pitch of the destination in elements
  int64_t f32_off;           // float offset of the factor in the state buffer
  int64_t own_stride, k_stride;
  int64_t dst_off;           // bf16 element offset of the destination array in the workspace
  int64_t sumsq_off;         // float offset in the workspace of the row sums of g^2 (row own0 first), or -1
  // Pacing of a team of CTAs that work through the same blocks (so that their reads of g meet in L2): before its
  // first load the item waits until team_counters[team] >= wait_count, after its last load it adds `signal`.
  // Pacing only: no data depends on it.
  int16_t team, signal;
  int32_t wait_count;
  float coef;
  int32_t cost;              // stages, for scheduling
};

// the fields of an Item its epilogue needs
struct ItemEpi {
  int32_t epi, own0, own_count, n_pan, acc_stride, r, rp, half, n_sum, stack_rows, dst_ld;
  int64_t f32_off, own_stride, k_stride, dst_off;
  float coef;
};

struct EngineArgs {
  const Item* items;
  int32_t n_items;
  const CUtensorMap* maps;
  float* f32_base;           // state buffer
  uint16_t* work_bf16;       // workspace viewed as bf16
  float* work_f32;           // workspace viewed as fp32 (row sums of g^2)
  int32_t* status;
  int32_t stage_k;           // 64 or 128
  int32_t stage_bytes;       // a_bytes + stage_k * 128 * (largest number of 64-column chunks of B)
  int32_t a_bytes;           // room for the A operands of a stage: (most operands of any segment) * 256 * stage_k
  int32_t n_stages;
  int32_t acc_cols;          // tensor-memory columns per accumulator buffer
  int32_t n_acc;             // 1 or 2 accumulator buffers
  const int32_t* cta_begin;  // CTA c runs items [cta_begin[c], cta_begin[c + 1]) in order
  int32_t sum_col;           // EPI_FACTOR: first of the tensor-memory columns the epilogue parks D0 + D1 in, or -1
  int32_t sumsq_on;          // 1: warps 4-7 follow the stages and sum g^2 for items that have sumsq_off >= 0
  int32_t* team_counters;    // one counter per team, zero at launch (nullptr when no item waits)
  uint32_t team_spin_limit, wait_spin_limit;
  const float* gscale;       // device scalar: every gradient counts as gscale[0] * g (nullptr: 1)
};

struct __align__(8) EngineShared {
  uint64_t full[8], empty[8], tfull[2], tempty[2];
  uint32_t tmem_base;
  int abort;
};

// The loads of one stage: NA operands of NBOX boxes each, then the B box.  Compile-time counts keep the issuing
// thread's instruction stream short (it runs dependent scalar code; its rate bounds the pipeline).
template <int NA, int NBOX>
__device__ __forceinline__ void load_stage(uint8_t* sa, int a_tile, int box_bytes, int a_bytes, const CUtensorMap* ma,
                                           const CUtensorMap* mb, const int* x, const int* y, int yb, uint64_t* bar) {
#pragma unroll
  for (int p = 0; p < NA; ++p)
#pragma unroll
    for (int j = 0; j < NBOX; ++j) tma_load_box(sa + p * a_tile + j * box_bytes, ma, x[p] + 64 * j, y[p], bar);
  tma_load_box3(sa + a_bytes, mb, 0, yb, 0, bar);
}

// The MMAs of one stage: nk K steps, NA operands, NM MMAs per operand and step.
template <int NA, int NM, bool MN_MAJOR_A>
__device__ __forceinline__ void mma_stage(uint32_t d_base, const Seg& S, uint32_t sa, int a_tile, uint32_t a_lbo,
                                          uint32_t blo, uint32_t b2, uint32_t dhi, uint32_t idesc, int nk,
                                          uint32_t& accumulate) {
  uint32_t alo[NA], dcol[NA];
#pragma unroll
  for (int p = 0; p < NA; ++p) {
    alo[p] = desc_lo(sa + (uint32_t)(p * a_tile), a_lbo);
    dcol[p] = d_base + (uint32_t)S.d_col[p];
  }
  const uint32_t d_part = (uint32_t)S.d_part;
  const bool same = S.same_acc != 0;
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    if (q < nk) {
      const uint32_t astep = MN_MAJOR_A ? (uint32_t)(q * 128) : (uint32_t)((q >> 2) * (kBoxBytes >> 4) + (q & 3) * 2);
      const uint64_t bd = desc_join(blo + (uint32_t)(q * 128), dhi);
#pragma unroll
      for (int p = 0; p < NA; ++p) {
        const uint64_t ad = desc_join(alo[p] + astep, dhi);
        const uint32_t acc_p = (p > 0 && same) ? 1u : accumulate;
        mma_bf16(dcol[p], ad, bd, idesc, acc_p);
        if (NM == 2) mma_bf16(dcol[p] + d_part, ad, desc_join(blo + b2 + (uint32_t)(q * 128), dhi), idesc, acc_p);
      }
      accumulate = 1u;
    }
  }
}

__global__ void __launch_bounds__(kEngineThreads, 1) tc_items_kernel(EngineArgs a) {
  extern __shared__ uint8_t dyn_smem[];
  __shared__ EngineShared sh;
  __shared__ int skip_launch;
  if (threadIdx.x == 0) skip_launch = *reinterpret_cast<volatile int32_t*>(a.status) != 0;
  __syncthreads();
  if (skip_launch) return;   // an earlier launch gave up: write nothing (the whole CTA decides together)
  uint8_t* stages = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(dyn_smem) + 1023) & ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort = &sh.abort;
  const uint32_t wlim = a.wait_spin_limit;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 8; ++i) { mbar_init(&sh.full[i], 1); mbar_init(&sh.empty[i], a.sumsq_on ? 5 : 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&sh.tfull[i], 1); mbar_init(&sh.tempty[i], 256); }
    sh.abort = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(&sh.tmem_base, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = sh.tmem_base;
  const int it_begin = a.cta_begin[blockIdx.x], it_end = a.cta_begin[blockIdx.x + 1];
  const int stage_k = a.stage_k;
  const int a_tile = 256 * stage_k;                 // bytes of one A operand of a stage
  const int ksteps = stage_k >> 4;                  // MMA K steps per full stage

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      uint32_t issued = 0;
      bool ok = true;
      for (int it = it_begin; it < it_end && ok; ++it) {
        const Item& I = a.items[it];
        if (I.wait_count > 0) {
          // Bounded like every wait here: a team member that never arrives ends this CTA with a status, not a
          // hang.  The bound is generous (about a second), because a member may start late when other work
          // holds SMs; the consumers' own bounds are longer still, so this is the wait that reports.
          volatile int32_t* cnt = a.team_counters + I.team;
          uint32_t spin = 0;
          while (*cnt < I.wait_count) {
            if (++spin >= a.team_spin_limit || ((spin & 255u) == 0 && *abort)) { ok = false; break; }
            __nanosleep(256);
          }
          if (!ok) {
            *abort = 1;
            atomicOr(a.status, ST_WAIT_TEAM);
            break;
          }
        }
        for (int s = 0; s < I.n_seg && ok; ++s) {
          const Seg S = I.seg[s];
          const CUtensorMap* ma = a.maps + S.map_a;
          const CUtensorMap* mb = a.maps + S.map_b;
          const int nst = (S.k + stage_k - 1) / stage_k;
          int x[kMaxA], y[kMaxA];
#pragma unroll
          for (int p = 0; p < kMaxA; ++p) { x[p] = S.ax[p]; y[p] = S.ay[p]; }
          int yb = 0;
          const int dx = S.a_mode ? 0 : stage_k, dy = S.a_mode ? stage_k : 0;
          // K along x: stage_k / 64 boxes of 64 x 128, 16 KB apart; K along y: two boxes of 64 x stage_k
          const int n_box = S.a_mode ? 2 : (stage_k >> 6);
          const int box_bytes = S.a_mode ? stage_k * 128 : kBoxBytes;
          for (int c = 0; c < nst; ++c) {
            if (!mbar_wait(&sh.empty[stage], phase ^ 1u, abort, a.status, ST_WAIT_EMPTY, wlim)) { ok = false; break; }
            uint8_t* sa = stages + stage * a.stage_bytes;
            uint64_t* bar = &sh.full[stage];
            mbar_arrive_expect_tx(bar, S.tx_bytes);
            if (n_box == 2) {
              if (S.n_a == 2) load_stage<2, 2>(sa, a_tile, box_bytes, a.a_bytes, ma, mb, x, y, yb, bar);
              else if (S.n_a == 3) load_stage<3, 2>(sa, a_tile, box_bytes, a.a_bytes, ma, mb, x, y, yb, bar);
              else load_stage<1, 2>(sa, a_tile, box_bytes, a.a_bytes, ma, mb, x, y, yb, bar);
            } else {
              if (S.n_a == 2) load_stage<2, 1>(sa, a_tile, box_bytes, a.a_bytes, ma, mb, x, y, yb, bar);
              else if (S.n_a == 3) load_stage<3, 1>(sa, a_tile, box_bytes, a.a_bytes, ma, mb, x, y, yb, bar);
              else load_stage<1, 1>(sa, a_tile, box_bytes, a.a_bytes, ma, mb, x, y, yb, bar);
            }
#pragma unroll
            for (int p = 0; p < kMaxA; ++p) { x[p] += dx; y[p] += dy; }
            yb += stage_k;
            ++issued;
            if (++stage == a.n_stages) { stage = 0; phase ^= 1u; }
          }
        }
        if (ok && I.signal) atomicAdd(a.team_counters + I.team, (int)I.signal);
      }
      if (!ok) {
        // leave no copy in flight: every stage that was filled must have landed before the CTA exits
        const int back = issued < (uint32_t)a.n_stages ? (int)issued : a.n_stages;
        for (int q = 0; q < back; ++q) {
          int st = stage - 1 - q;
          uint32_t ph = phase;
          if (st < 0) { st += a.n_stages; ph ^= 1u; }
          for (uint32_t spin = 0; spin < kSpinLimit && !mbar_try_wait(&sh.full[st], ph); ++spin) __nanosleep(64);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int j = 0;
      const uint32_t stages_u32 = smem_u32(stages);
      const uint32_t dhi = desc_hi();
      const uint32_t b_lbo = (uint32_t)stage_k * 128u;      // bytes between the 64-column chunks of B
      for (int it = it_begin; it < it_end && ok; ++it, ++j) {
        const Item& I = a.items[it];
        const int acc = j % a.n_acc;
        const uint32_t acc_phase = (uint32_t)(j / a.n_acc) & 1u;
        if (!mbar_wait(&sh.tempty[acc], acc_phase ^ 1u, abort, a.status, ST_WAIT_TMEM_EMPTY, wlim)) break;
        tc_fence_after();
        const uint32_t d_base = tmem_base + (uint32_t)(acc * a.acc_cols);
        for (int s = 0; s < I.n_seg && ok; ++s) {
          const Seg S = I.seg[s];
          const uint32_t idesc = make_idesc(S.n, S.a_mode != 0, true, false);
          const int nst = (S.k + stage_k - 1) / stage_k;
          // per K step of 16, in 16-byte units: K along x walks 32 B inside a box and 16 KB to the
          // next box; K along y walks 16 rows of 128 B
          const uint32_t a_lbo = S.a_mode ? b_lbo : 16u;
          const uint32_t b2 = ((uint32_t)S.b2_chunk * b_lbo) >> 4;
          uint32_t accumulate = S.first ? 0u : 1u;
          int k_left = S.k;
          for (int c = 0; c < nst; ++c, k_left -= stage_k) {
            if (!mbar_wait(&sh.full[stage], phase, abort, a.status, ST_WAIT_FULL, wlim)) { ok = false; break; }
            tc_fence_after();
            const uint32_t sa = stages_u32 + (uint32_t)(stage * a.stage_bytes);
            const uint32_t blo = desc_lo(sa + (uint32_t)a.a_bytes, b_lbo);
            const int nk = k_left >= stage_k ? ksteps : (k_left + 15) >> 4;
            if (S.n_mma == 2) {
              if (S.a_mode) {
                if (S.n_a == 2) mma_stage<2, 2, true>(d_base, S, sa, a_tile, a_lbo, blo, b2, dhi, idesc, nk, accumulate);
                else mma_stage<1, 2, true>(d_base, S, sa, a_tile, a_lbo, blo, b2, dhi, idesc, nk, accumulate);
              } else {
                if (S.n_a == 2) mma_stage<2, 2, false>(d_base, S, sa, a_tile, a_lbo, blo, b2, dhi, idesc, nk, accumulate);
                else mma_stage<1, 2, false>(d_base, S, sa, a_tile, a_lbo, blo, b2, dhi, idesc, nk, accumulate);
              }
            } else if (S.a_mode) {
              if (S.n_a == 2) mma_stage<2, 1, true>(d_base, S, sa, a_tile, a_lbo, blo, b2, dhi, idesc, nk, accumulate);
              else if (S.n_a == 3) mma_stage<3, 1, true>(d_base, S, sa, a_tile, a_lbo, blo, b2, dhi, idesc, nk, accumulate);
              else mma_stage<1, 1, true>(d_base, S, sa, a_tile, a_lbo, blo, b2, dhi, idesc, nk, accumulate);
            } else {
              if (S.n_a == 2) mma_stage<2, 1, false>(d_base, S, sa, a_tile, a_lbo, blo, b2, dhi, idesc, nk, accumulate);
              else if (S.n_a == 3) mma_stage<3, 1, false>(d_base, S, sa, a_tile, a_lbo, blo, b2, dhi, idesc, nk, accumulate);
              else mma_stage<1, 1, false>(d_base, S, sa, a_tile, a_lbo, blo, b2, dhi, idesc, nk, accumulate);
            }
            mma_commit(&sh.empty[stage]);
            if (++stage == a.n_stages) { stage = 0; phase ^= 1u; }
          }
        }
        if (ok) mma_commit(&sh.tfull[acc]);
      }
    }
  } else if (warp < 4) {
    // no work
  } else if (warp < 8) {
    // ------------------------------------------------------------------ row sums of g^2
    // The four warps follow every stage of the launch (their arrivals are part of each stage's release); for an
    // item with sumsq_off >= 0 they read the gradient tiles of the first segment (K along x), each warp 32 rows
    // of every panel.  Eight lanes share a row of a box (its eight 16-byte pieces,
    // whatever order the swizzle put them in), so a warp reads four rows per access without bank conflicts; a
    // lane keeps one partial sum per row it visits, and the eight partial sums of a row are added in a fixed
    // order at the end of the item.
    if (a.sumsq_on) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      const int rsub = 32 * (warp - 4) + (lane >> 3), piece = lane & 7;
      for (int it = it_begin; it < it_end && ok; ++it) {
        const Item& I = a.items[it];
        const bool mine = I.sumsq_off >= 0;
        float acc[kMaxA][8];
#pragma unroll
        for (int p = 0; p < kMaxA; ++p)
#pragma unroll
          for (int i = 0; i < 8; ++i) acc[p][i] = 0.f;
        int n_a0 = 0;
        for (int s = 0; s < I.n_seg && ok; ++s) {
          const int k = I.seg[s].k, n_a = I.seg[s].n_a;
          if (s == 0) n_a0 = n_a;
          const int nst = (k + stage_k - 1) / stage_k;
          const int n_box = stage_k >> 6;
          for (int c = 0; c < nst; ++c) {
            bool got = true;
            if (lane == 0) got = mbar_wait(&sh.full[stage], phase, abort, a.status, ST_WAIT_FULL, wlim);
            got = __shfl_sync(0xffffffffu, got, 0);
            if (!got) { ok = false; break; }
            if (mine && s == 0) {
              const uint8_t* sa = stages + stage * a.stage_bytes;
#pragma unroll
              for (int p = 0; p < kMaxA; ++p) {
                if (p < n_a) {
                  for (int jb = 0; jb < n_box; ++jb) {
                    const uint8_t* box = sa + p * a_tile + jb * kBoxBytes + piece * 16;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                      const uint4 v = *reinterpret_cast<const uint4*>(box + (4 * i + rsub) * 128);
                      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
                      float s2 = acc[p][i];
#pragma unroll
                      for (int e = 0; e < 4; ++e) {
                        const float lo = __uint_as_float(w[e] << 16), hi = __uint_as_float(w[e] & 0xffff0000u);
                        s2 = fmaf(lo, lo, s2);
                        s2 = fmaf(hi, hi, s2);
                      }
                      acc[p][i] = s2;
                    }
                  }
                }
              }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.empty[stage]);
            if (++stage == a.n_stages) { stage = 0; phase ^= 1u; }
          }
        }
        if (mine && ok) {
          float* out = a.work_f32 + I.sumsq_off;
#pragma unroll
          for (int p = 0; p < kMaxA; ++p) {
            if (p < n_a0) {
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                float s2 = acc[p][i];
                s2 += __shfl_xor_sync(0xffffffffu, s2, 1);
                s2 += __shfl_xor_sync(0xffffffffu, s2, 2);
                s2 += __shfl_xor_sync(0xffffffffu, s2, 4);
                const int row = 128 * p + 4 * i + rsub;
                if (piece == 0 && I.own0 + row < I.own_count) out[row] = s2;
              }
            }
          }
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int q = 32 * (warp & 3) + lane;               // accumulator row (= TMEM lane) of this thread
    const uint32_t lane_addr = (uint32_t)(32 * (warp & 3)) << 16;
    const int grp = (warp - 8) >> 2;                    // the two groups take the pieces of an item alternately
    const float gs = a.gscale ? *a.gscale : 1.f;
    int j = 0;
    for (int it = it_begin; it < it_end; ++it, ++j) {
      // scalar fields are copied once: the stores below could alias the item table as far as the
      // compiler can tell, and every re-read would be a round trip to global memory
      ItemEpi I;
      {
        const Item& G = a.items[it];
        I.epi = G.epi; I.own0 = G.own0; I.own_count = G.own_count; I.n_pan = G.n_pan; I.acc_stride = G.acc_stride;
        I.r = G.r; I.rp = G.rp; I.half = G.half; I.n_sum = G.n_sum; I.stack_rows = G.stack_rows;
        I.f32_off = G.f32_off; I.own_stride = G.own_stride; I.k_stride = G.k_stride;
        I.dst_off = G.dst_off; I.dst_ld = G.dst_ld; I.coef = G.coef;
      }
      const int acc = j % a.n_acc;
      const uint32_t acc_phase = (uint32_t)(j / a.n_acc) & 1u;
      const int rp = I.rp, r = I.r, half = I.half;
      const int np = rp >> 4;                             // 16-column pieces per panel
      const int total = I.epi == EPI_FACTOR ? I.n_pan * np : 0;
      // Gradients scaled by gs (global norm clipping): the factor update is linear in g, so the Gram operands
      // are divided by gs where they are made and the whole accumulator is multiplied by it here.
      const float coef = I.epi == EPI_FACTOR ? I.coef * gs : I.coef / gs;
      const bool has_work = I.epi == EPI_FACTOR ? grp < total : (I.epi == EPI_GRAM && grp == 0);
      const bool factor = I.epi == EPI_FACTOR && has_work;
      const int qc = lane & 3;
      float* fbase = a.f32_base + I.f32_off;
      // EPI_FACTOR has three forms.  The general one works in a "turned" layout: a thread reads its accumulator
      // row from tensor memory, then every quad of lanes transposes its 4 x 16 piece with shuffles, after which
      // lane c of the quad holds columns 4c .. 4c+3 of the quad's four rows; factor rows are then read and
      // written as 64-byte runs instead of one row per lane.
      // float4 path of that form: the four values of a lane are adjacent in memory and 16-byte aligned
      const bool vec4 = I.k_stride == 1 && (I.own_stride & 3) == 0 && (r & 3) == 0 && (I.f32_off & 3) == 0;
      // A factor whose consecutive owners are adjacent in memory (R, stored [r, n]) needs no turn: for
      // a fixed column the 32 rows of a warp are one 128-byte run already.
      const bool by_column = factor && I.own_stride == 1 && !vec4;
      // A factor stored row by row (L, [m, r]) whose rows start on 32-byte boundaries and hold a multiple of
      // eight values needs no turn either: a lane moves 32 bytes per access, which is a whole sector.
      const bool by_row = factor && I.k_stride == 1 && ((I.own_stride | r | I.f32_off) & 7) == 0;
      // piece u of the item: panel u / np, columns [16 (u % np), +16)
      auto fetch_old = [&](int u, float (*o)[4]) {
        const int pan = u / np, p = 16 * (u - pan * np);
        const int own_quad = I.own0 + 128 * pan + 32 * (warp & 3) + (lane & ~3);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int owner = own_quad + i;      // quad row i, this lane's four columns of it
          const int k = p + 4 * qc;
          const bool row_ok = owner < I.own_count;
          const float* fp = fbase + I.own_stride * owner + I.k_stride * k;
          if (vec4) {
            const float4 v = (row_ok && k < r) ? __ldcg(reinterpret_cast<const float4*>(fp)) : make_float4(0.f, 0.f, 0.f, 0.f);
            o[i][0] = v.x; o[i][1] = v.y; o[i][2] = v.z; o[i][3] = v.w;
          } else {
#pragma unroll
            for (int x = 0; x < 4; ++x) o[i][x] = (row_ok && k + x < r) ? __ldcg(fp + I.k_stride * x) : 0.f;
          }
        }
      };
      // old values of this thread's own row, columns [p, p+16), kept in the same registers as o[e / 4][e % 4]
      auto fetch_old_col = [&](int u, float (*o)[4]) {
        const int pan = u / np, p = 16 * (u - pan * np);
        const int own_row = I.own0 + 128 * pan + q;
        const float* fp = fbase + own_row + I.k_stride * p;
        const bool row_ok = own_row < I.own_count;
#pragma unroll
        for (int e = 0; e < 16; ++e) o[e >> 2][e & 3] = (row_ok && p + e < r) ? __ldcg(fp + I.k_stride * e) : 0.f;
      };
      auto fetch_old_row = [&](int u, float (*o)[4]) {
        const int pan = u / np, p = 16 * (u - pan * np);
        const int own_row = I.own0 + 128 * pan + q;
        const float* fp = fbase + I.own_stride * own_row + p;
        const bool row_ok = own_row < I.own_count;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (row_ok && p + 8 * h < r) {
            ldcg_f32x8(fp + 8 * h, &o[2 * h][0]);
          } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) o[2 * h + (e >> 2)][e & 3] = 0.f;
          }
        }
      };
      // old values travel one piece ahead in two register sets that swap roles (no copies, which
      // would wait for the loads); the first set is requested before the accumulator is waited for
      float oldA[4][4], oldB[4][4];
      if (by_row) fetch_old_row(grp, oldA);
      else if (by_column) fetch_old_col(grp, oldA);
      else if (factor) fetch_old(grp, oldA);
      // one lane per warp polls (fewer pollers on the barrier), then the warp agrees: the
      // tensor-memory loads below need all 32 lanes
      bool got = true;
      if (lane == 0) got = mbar_wait(&sh.tfull[acc], acc_phase, abort, a.status, ST_WAIT_TMEM_FULL, wlim);
      got = __shfl_sync(0xffffffffu, got, 0);
      if (!got) break;
      tc_fence_after();
      const uint32_t t0 = tmem_base + lane_addr + (uint32_t)(acc * a.acc_cols);
      // With one accumulator buffer the next item's MMAs wait for this epilogue.  Its memory traffic is the slow
      // part, so the sums D0 + D1 are first parked in spare tensor-memory columns (this warp's own lanes, the
      // same columns for every item) and the accumulator is handed back at once; the pieces below then read the
      // parked sums while the next main loop runs.  Each group parks the pieces it will work on.
      const bool parked = factor && a.sum_col >= 0;
      const uint32_t ts = tmem_base + lane_addr + (uint32_t)(a.sum_col < 0 ? 0 : a.sum_col);
      if (parked) {
        for (int u = grp; u < total; u += 2) {
          const int pan = u / np, p = 16 * (u - pan * np);
          float d0[16], d1[16];
          tmem_ld16(t0 + (uint32_t)(pan * I.acc_stride + p), d0);
          tmem_ld16(t0 + (uint32_t)(pan * I.acc_stride + rp + p), d1);
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 16; ++e) d0[e] += d1[e];
          tmem_st16(ts + (uint32_t)(pan * rp + p), d0);
        }
        tmem_st_wait();
      }
      const bool early = parked || !has_work;   // (a warp without work never reads the accumulator)
      if (early) {
        tc_fence_before();
        mbar_arrive(&sh.tempty[acc]);
      }
      // columns [p, p+16) of D0 + D1 of this thread's row of panel `pan`
      auto sum16 = [&](int pan, int p, float* sd) {
        if (parked) {
          tmem_ld16(ts + (uint32_t)(pan * rp + p), sd);
          tmem_ld_wait();
        } else {
          float d1[16];
          tmem_ld16(t0 + (uint32_t)(pan * I.acc_stride + p), sd);
          tmem_ld16(t0 + (uint32_t)(pan * I.acc_stride + rp + p), d1);
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 16; ++e) sd[e] += d1[e];
        }
      };
      if (!has_work) {
        // nothing to drain for this warp
      } else if (I.epi == EPI_FACTOR) {
        uint16_t* dst = a.work_bf16 + I.dst_off;
        // one piece in the turned form, old values in `o`
        auto piece = [&](int u, float (*o)[4]) {
          const int pan = u / np, p = 16 * (u - pan * np);
          const int own_quad = I.own0 + 128 * pan + 32 * (warp & 3) + (lane & ~3);
          float acc16[16];
          sum16(pan, p, acc16);
          float v[4][4];                 // v[j] = columns 4j .. 4j+3 of this thread's row
#pragma unroll
          for (int jj = 0; jj < 4; ++jj)
#pragma unroll
            for (int e = 0; e < 4; ++e) v[jj][e] = acc16[4 * jj + e];
          // quad transpose, first exchange (partner lane ^ 2): keep the half of the columns this lane's
          // final column group lies in, hand over the other half
          const bool up = (qc & 2) != 0, odd = (qc & 1) != 0;
          float k0[4], k1[4], g0[4], g1[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            k0[e] = up ? v[2][e] : v[0][e];
            k1[e] = up ? v[3][e] : v[1][e];
            const float s0 = up ? v[0][e] : v[2][e], s1 = up ? v[1][e] : v[3][e];
            g0[e] = __shfl_xor_sync(0xffffffffu, s0, 2);
            g1[e] = __shfl_xor_sync(0xffffffffu, s1, 2);
          }
          // second exchange (partner lane ^ 1): keep this lane's column group of the two rows held so far,
          // hand over the neighbour's; t[0..3] then belong to quad rows qc, qc^2, qc^1, qc^3
          float t[4][4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            t[0][e] = odd ? k1[e] : k0[e];
            t[1][e] = odd ? g1[e] : g0[e];
            const float s0 = odd ? k0[e] : k1[e], s1 = odd ? g0[e] : g1[e];
            t[2][e] = __shfl_xor_sync(0xffffffffu, s0, 1);
            t[3][e] = __shfl_xor_sync(0xffffffffu, s1, 1);
          }
          // order by row, so that in every access below the four lanes of a quad address one row
          float sd[4][4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int w = i ^ qc;          // 0 -> t[0], 2 -> t[1], 1 -> t[2], 3 -> t[3]
#pragma unroll
            for (int e = 0; e < 4; ++e) sd[i][e] = w == 0 ? t[0][e] : (w == 2 ? t[1][e] : (w == 1 ? t[2][e] : t[3][e]));
          }
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int owner = own_quad + i;
            if (owner >= I.own_count) continue;
            const int k = p + 4 * qc;
            float x[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) x[e] = k + e < r ? o[i][e] + coef * sd[i][e] : 0.f;
            float* fp = fbase + I.own_stride * owner + I.k_stride * k;
            if (vec4) {
              if (k < r) *reinterpret_cast<float4*>(fp) = make_float4(x[0], x[1], x[2], x[3]);
            } else {
#pragma unroll
              for (int e = 0; e < 4; ++e)
                if (k + e < r) fp[I.k_stride * e] = x[e];
            }
            uint32_t h01, l01, h23, l23;
            split_bf16x2(x[0], x[1], h01, l01);
            split_bf16x2(x[2], x[3], h23, l23);
            uint16_t* drow = dst + (int64_t)I.dst_ld * owner + k;
            *reinterpret_cast<uint2*>(drow) = make_uint2(h01, h23);
            *reinterpret_cast<uint2*>(drow + half) = make_uint2(l01, l23);
          }
        };
        // the same piece without the turn: this thread's row, columns [p, p+16)
        auto piece_col = [&](int u, float (*o)[4]) {
          const int pan = u / np, p = 16 * (u - pan * np);
          const int own_row = I.own0 + 128 * pan + q;
          float sd[16];
          sum16(pan, p, sd);
          if (own_row >= I.own_count) return;
          float* fp = fbase + own_row + I.k_stride * p;
          uint32_t hi[8], lo[8];
#pragma unroll
          for (int e = 0; e < 16; e += 2) {
            const float x0 = p + e < r ? o[e >> 2][e & 3] + coef * sd[e] : 0.f;
            const float x1 = p + e + 1 < r ? o[(e + 1) >> 2][(e + 1) & 3] + coef * sd[e + 1] : 0.f;
            if (p + e < r) __stcg(fp + I.k_stride * e, x0);
            if (p + e + 1 < r) __stcg(fp + I.k_stride * (e + 1), x1);
            split_bf16x2(x0, x1, hi[e >> 1], lo[e >> 1]);
          }
          uint16_t* drow = dst + (int64_t)I.dst_ld * own_row + p;
          st_b32x8(drow, hi);
          st_b32x8(drow + half, lo);
        };
        // and for a row-stored factor with aligned rows
        auto piece_row = [&](int u, float (*o)[4]) {
          const int pan = u / np, p = 16 * (u - pan * np);
          const int own_row = I.own0 + 128 * pan + q;
          float sd[16];
          sum16(pan, p, sd);
          if (own_row >= I.own_count) return;
          float x[16];
          uint32_t hi[8], lo[8];
#pragma unroll
          for (int e = 0; e < 16; e += 2) {
            x[e] = p + e < r ? o[e >> 2][e & 3] + coef * sd[e] : 0.f;
            x[e + 1] = p + e + 1 < r ? o[(e + 1) >> 2][(e + 1) & 3] + coef * sd[e + 1] : 0.f;
            split_bf16x2(x[e], x[e + 1], hi[e >> 1], lo[e >> 1]);
          }
          float* fp = fbase + I.own_stride * own_row + p;
          if (p < r) st_f32x8(fp, x);
          if (p + 8 < r) st_f32x8(fp + 8, x + 8);
          uint16_t* drow = dst + (int64_t)I.dst_ld * own_row + p;
          st_b32x8(drow, hi);
          st_b32x8(drow + half, lo);
        };
        // this group's pieces grp, grp + 2, ...: two per trip, the old values of the next one on their way
        if (by_row) {
#pragma unroll 1
          for (int u = grp; u < total; u += 4) {
            if (u + 2 < total) fetch_old_row(u + 2, oldB);
            piece_row(u, oldA);
            if (u + 2 < total) {
              if (u + 4 < total) fetch_old_row(u + 4, oldA);
              piece_row(u + 2, oldB);
            }
          }
        } else if (by_column) {
#pragma unroll 1
          for (int u = grp; u < total; u += 4) {
            if (u + 2 < total) fetch_old_col(u + 2, oldB);
            piece_col(u, oldA);
            if (u + 2 < total) {
              if (u + 4 < total) fetch_old_col(u + 4, oldA);
              piece_col(u + 2, oldB);
            }
          }
        } else {
#pragma unroll 1
          for (int u = grp; u < total; u += 4) {
            if (u + 2 < total) fetch_old(u + 2, oldB);
            piece(u, oldA);
            if (u + 2 < total) {
              if (u + 4 < total) fetch_old(u + 4, oldA);
              piece(u + 2, oldB);
            }
          }
        }
      } else if (I.epi == EPI_GRAM) {
        uint16_t* dst = a.work_bf16 + I.dst_off;
        const int row = I.own0 + q;
        for (int p = 0; p < rp; p += 16) {
          float d0[16], d1[16];
          tmem_ld16(t0 + (uint32_t)p, d0);
          tmem_ld16(t0 + (uint32_t)(rp + p), d1);
          if (I.n_sum == 4) {
            float d2[16], d3[16];
            tmem_ld16(t0 + (uint32_t)(2 * rp + p), d2);
            tmem_ld16(t0 + (uint32_t)(3 * rp + p), d3);
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 16; ++e) d0[e] = (d0[e] + d1[e]) + (d2[e] + d3[e]);
          } else {
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 16; ++e) d0[e] = d0[e] + d1[e];
          }
          if (row < rp) {
            uint32_t hi[8], lo[8];
#pragma unroll
            for (int e = 0; e < 16; e += 2) split_bf16x2(coef * d0[e], coef * d0[e + 1], hi[e >> 1], lo[e >> 1]);
            for (int copy = 0; copy < (I.stack_rows > 0 ? 2 : 1); ++copy) {
              uint16_t* drow = dst + (int64_t)I.dst_ld * (row + copy * I.stack_rows) + p;
              uint4* dh = reinterpret_cast<uint4*>(drow);
              uint4* dl = reinterpret_cast<uint4*>(drow + half);
              dh[0] = make_uint4(hi[0], hi[1], hi[2], hi[3]);
              dh[1] = make_uint4(hi[4], hi[5], hi[6], hi[7]);
              dl[0] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
              dl[1] = make_uint4(lo[4], lo[5], lo[6], lo[7]);
            }
          }
        }
      }
      if (!early) {
        tc_fence_before();
        mbar_arrive(&sh.tempty[acc]);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace tc
}  // namespace adapm
