// A persistent, warp-specialised tcgen05 engine that runs a table of "items".  An item is a short
// list of K-loops ("segments") that accumulate into one 128-row accumulator in tensor memory,
// followed by an epilogue that turns the accumulator into the result of one step of Algorithm 2:
//
//   refit of L (row panel of 128 rows of a block, Algorithm 2's L update):
//       D = g R^T + L Bop1^T + L0 Bop2^T          Bop1 = -(R R^T)/(1-b1),  Bop2 = b1 (R R0^T)/(1-b1)
//       L' = L + eta (1-b1) D
//   refit of R (column panel of 128 columns, the R update, computed transposed):
//       D = g^T L + R^T Bop3^T + R0^T Bop4^T       Bop3 = -(L^T L)/(1-b1),  Bop4 = b1 (L^T L0)/(1-b1)
//       R'^T = R^T + eta (1-b1) D
//   Gram item: one of the r x r matrices above, scaled and stored (transposed) as a split-bf16 operand.
//
// fp32 factors are carried into the bf16 tensor cores as hi + lo pairs (two bf16 numbers whose sum
// has ~16 significant bits); gradients are bf16 already and enter unchanged.  Operands with hi and
// lo parts are stored side by side ([rows, 2 rp]: hi columns then lo columns, rp = r rounded up to
// 16), so that used as the N side of an MMA the two parts land in two column ranges of the
// accumulator, which the epilogue adds.
//
// A stage of the shared-memory ring holds K = 128 of the operands:
//   A  two boxes of 64 x 128 (32 KB): 128 rows x K (K along x) or K x 128 columns (K along y)
//   A' optionally a second such operand (the next 128 rows / columns, or another column window):
//      both are multiplied with the same B and fill two accumulators, which halves the bytes of B
//      brought in per flop (the loads, not the tensor pipe, bound this kernel)
//   B  one 3-D box: K rows x (64 x nb_b) columns of an [rows, 2rp] array, i.e. the N side read
//      MN-major with its 64-column chunks one box apart
// Warp roles (320 threads): warp 0 issues the TMA loads of a stage, warp 1 issues its (up to)
// sixteen MMAs, warps 2-5 drain the first accumulator and warps 6-9 the second.  The two issuing
// threads run dependent scalar code, so
// their per-stage instruction count is what bounds the rate; both loops are kept short.  With two
// accumulator buffers the epilogue of one item overlaps the K-loops of the next.  Every wait is
// bounded; when one runs out the CTA records a status bit, stops taking work and leaves through the
// common exit (which frees its tensor memory).
#pragma once

#include <cuda.h>

#include "tc_common.cuh"

namespace adapm {
namespace tc {

constexpr int kMaxSegs = 6;
constexpr int kStageK = 128;
constexpr uint32_t kTeamSpinLimit = 1u << 24;    // polls of 256 ns each: about four seconds
constexpr int kStageABytes = 2 * kBoxBytes;      // the A side of a stage: 32 KB
constexpr int kEngineThreads = 320;

enum : int32_t { EPI_FACTOR = 0, EPI_GRAM = 1, EPI_NONE = 2 };   // EPI_NONE: a filler that only keeps a CTA in step

struct Seg {
  int32_t map_a;             // 2-D tensor map, box 64 x 128
  int32_t map_b;             // 3-D tensor map (64, rows, chunks), box 64 x b_rows x nb_b
  int32_t ax, ay;            // element coordinates of the first A box
  int32_t by;                // first K row of B
  int32_t k;                 // K extent, multiple of 16
  uint32_t b_lbo;            // bytes between the 64-column chunks of B in shared memory (= 128 * b_rows)
  uint32_t tx_bytes;         // bytes one stage of this segment brings in
  int16_t a_mode;            // 0: K runs along x (K-major A), 1: K runs along y (MN-major A)
  int16_t n;                 // MMA N (multiple of 16, <= 256)
  int16_t d_col;             // accumulator column this segment starts at
  int16_t first;             // 1: its first MMA overwrites the accumulator
  int16_t n_a;               // 1, or 2: a second A operand at (ax2, ay2) accumulates at column d_col2
  int16_t d_col2;
  int32_t ax2, ay2;
};

struct Item {
  Seg seg[kMaxSegs];
  int32_t n_seg;
  int32_t epi;
  // EPI_FACTOR: the thread that owns accumulator row q updates factor entries (owner = own0 + q, k):
  //   f32[own_stride * owner + k_stride * k] += coef * (D[q][k] + D[q][rp + k])        k < r
  //   dst[owner][k] = hi, dst[owner][rp + k] = lo                                      k < rp
  // EPI_GRAM: G[q][k] = coef * (D[q][k] + D[q][rp+k] + D[q][2rp+k] + D[q][3rp+k]);
  //   dst[q][k] = hi, dst[q][rp + k] = lo                                              q, k < rp
  int32_t own0, own_count;   // first owner and number of owners of the whole matrix
  int32_t own1;              // EPI_FACTOR: first owner of the second accumulator (columns from col2), or -1
  int32_t col2;
  int32_t r, rp;
  int64_t f32_off;           // float offset of the factor in the state buffer
  int64_t own_stride, k_stride;
  int64_t dst_off;           // bf16 element offset of the destination array in the workspace
  int32_t dst_ld;            // its row pitch in elements
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
  int32_t epi, own0, own_count, own1, col2, r, rp, dst_ld;
  int64_t f32_off, own_stride, k_stride, dst_off;
  float coef;
};

struct EngineArgs {
  const Item* items;
  int32_t n_items;
  const CUtensorMap* maps;
  float* f32_base;           // state buffer
  uint16_t* work_bf16;       // workspace viewed as bf16
  int32_t* status;
  int32_t stage_bytes;       // a_bytes + 16 KB * (largest number of 64-column chunks of B)
  int32_t a_bytes;           // kStageABytes, or twice that when segments with two A operands occur
  int32_t n_stages;
  int32_t acc_cols;          // tensor-memory columns per accumulator buffer
  int32_t n_acc;             // 1 or 2 accumulator buffers
  const int32_t* cta_begin;  // CTA c runs items [cta_begin[c], cta_begin[c + 1]) in order
  int32_t sum_col;           // EPI_FACTOR: first of the tensor-memory columns the epilogue parks D0 + D1 in, or -1
  int32_t* team_counters;    // one counter per team, zero at launch (nullptr when no item waits)
};

struct __align__(8) EngineShared {
  uint64_t full[8], empty[8], tfull[2], tempty[2];
  uint32_t tmem_base;
  int abort;
};

__device__ __forceinline__ int seg_stages(const Seg& s) { return (s.k + kStageK - 1) / kStageK; }

__global__ void __launch_bounds__(kEngineThreads, 1) tc_items_kernel(EngineArgs a) {
  extern __shared__ uint8_t dyn_smem[];
  __shared__ EngineShared sh;
  uint8_t* stages = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(dyn_smem) + 1023) & ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort = &sh.abort;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 8; ++i) { mbar_init(&sh.full[i], 1); mbar_init(&sh.empty[i], 1); }
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
          // hang.  The bound is generous (seconds), because a member may start late when other work holds SMs.
          volatile int32_t* cnt = a.team_counters + I.team;
          uint32_t spin = 0;
          while (*cnt < I.wait_count) {
            if (++spin >= kTeamSpinLimit || ((spin & 255u) == 0 && *abort)) { ok = false; break; }
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
          const int nst = seg_stages(S);
          // coordinates of the two A boxes and of the B box of the first stage, and their steps
          int x0 = S.ax, y0 = S.ay, x2 = S.ax2, y2 = S.ay2, yb = S.by;
          const int dx = S.a_mode ? 0 : kStageK, dy = S.a_mode ? kStageK : 0;
          for (int c = 0; c < nst; ++c) {
            if (!mbar_wait(&sh.empty[stage], phase ^ 1u, abort, a.status, ST_WAIT_EMPTY)) { ok = false; break; }
            uint8_t* sa = stages + stage * a.stage_bytes;
            uint64_t* bar = &sh.full[stage];
            mbar_arrive_expect_tx(bar, S.tx_bytes);
            tma_load_box(sa, ma, x0, y0, bar);
            tma_load_box(sa + kBoxBytes, ma, x0 + 64, y0, bar);
            if (S.n_a == 2) {
              tma_load_box(sa + kStageABytes, ma, x2, y2, bar);
              tma_load_box(sa + kStageABytes + kBoxBytes, ma, x2 + 64, y2, bar);
            }
            tma_load_box3(sa + a.a_bytes, mb, 0, yb, 0, bar);
            x0 += dx; y0 += dy; x2 += dx; y2 += dy; yb += kStageK;
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
      for (int it = it_begin; it < it_end && ok; ++it, ++j) {
        const Item& I = a.items[it];
        const int acc = j % a.n_acc;
        const uint32_t acc_phase = (uint32_t)(j / a.n_acc) & 1u;
        if (!mbar_wait(&sh.tempty[acc], acc_phase ^ 1u, abort, a.status, ST_WAIT_TMEM_EMPTY)) break;
        tc_fence_after();
        const uint32_t d_base = tmem_base + (uint32_t)(acc * a.acc_cols);
        for (int s = 0; s < I.n_seg && ok; ++s) {
          const Seg S = I.seg[s];
          const uint32_t idesc = make_idesc(S.n, S.a_mode != 0, true, false);
          const uint32_t d = d_base + (uint32_t)S.d_col, d2 = d_base + (uint32_t)S.d_col2;
          const int nst = seg_stages(S);
          // per K step of 16, in 16-byte units: K along x walks 32 B inside a box and 16 KB to the
          // next box; K along y walks 16 rows of 128 B
          const uint32_t a_lbo = S.a_mode ? (uint32_t)kBoxBytes : 16u;
          uint32_t accumulate = S.first ? 0u : 1u;
          int k_left = S.k;
          for (int c = 0; c < nst; ++c, k_left -= kStageK) {
            if (!mbar_wait(&sh.full[stage], phase, abort, a.status, ST_WAIT_FULL)) { ok = false; break; }
            tc_fence_after();
            const uint32_t sa = stages_u32 + (uint32_t)(stage * a.stage_bytes);
            const uint32_t alo = desc_lo(sa, a_lbo);
            const uint32_t alo2 = desc_lo(sa + kStageABytes, a_lbo);
            const uint32_t blo = desc_lo(sa + (uint32_t)a.a_bytes, S.b_lbo);
            const int nk = k_left >= kStageK ? 8 : (k_left + 15) >> 4;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              if (q < nk) {
                const uint32_t astep = S.a_mode ? (uint32_t)(q * 128) : (uint32_t)((q >> 2) * (kBoxBytes >> 4) + (q & 3) * 2);
                const uint64_t bd = desc_join(blo + (uint32_t)(q * 128), dhi);
                mma_bf16(d, desc_join(alo + astep, dhi), bd, idesc, accumulate);
                if (S.n_a == 2) mma_bf16(d2, desc_join(alo2 + astep, dhi), bd, idesc, accumulate);
                accumulate = 1u;
              }
            }
            mma_commit(&sh.empty[stage]);
            if (++stage == a.n_stages) { stage = 0; phase ^= 1u; }
          }
        }
        if (ok) mma_commit(&sh.tfull[acc]);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int q = 32 * (warp & 3) + lane;               // accumulator row (= TMEM lane) of this thread
    const uint32_t lane_addr = (uint32_t)(32 * (warp & 3)) << 16;
    const bool second = warp >= 6;                      // this warp drains the second accumulator
    int j = 0;
    for (int it = it_begin; it < it_end; ++it, ++j) {
      // scalar fields are copied once: the stores below could alias the item table as far as the
      // compiler can tell, and every re-read would be a round trip to global memory
      ItemEpi I;
      {
        const Item& G = a.items[it];
        I.epi = G.epi; I.own0 = G.own0; I.own_count = G.own_count; I.own1 = G.own1; I.col2 = G.col2;
        I.r = G.r; I.rp = G.rp; I.f32_off = G.f32_off; I.own_stride = G.own_stride; I.k_stride = G.k_stride;
        I.dst_off = G.dst_off; I.dst_ld = G.dst_ld; I.coef = G.coef;
      }
      const int acc = j % a.n_acc;
      const uint32_t acc_phase = (uint32_t)(j / a.n_acc) & 1u;
      const int rp = I.rp, r = I.r;
      // EPI_FACTOR works in a "turned" layout: a thread reads its accumulator row from tensor memory,
      // then every quad of lanes transposes its 4 x 16 piece with shuffles, after which lane c of the
      // quad holds columns 4c .. 4c+3 of the quad's four rows.  Factor rows are then read and written
      // as 64-byte runs instead of one row per lane.
      const bool has_work = !second || (I.epi == EPI_FACTOR && I.own1 >= 0);
      const bool factor = I.epi == EPI_FACTOR && has_work;
      const int qc = lane & 3;
      const int own_quad = (second ? I.own1 : I.own0) + 32 * (warp & 3) + (lane & ~3);
      float* fbase = a.f32_base + I.f32_off;
      // float4 path: the four values of a lane are adjacent in memory and 16-byte aligned
      const bool vec4 = I.k_stride == 1 && (I.own_stride & 3) == 0 && (r & 3) == 0 && (I.f32_off & 3) == 0;
      auto fetch_old = [&](int p, float (*o)[4]) {
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
      // old values travel one piece ahead in two register sets that swap roles (no copies, which
      // would wait for the loads); the first set is requested before the accumulator is waited for
      float oldA[4][4], oldB[4][4];
      // A factor whose consecutive owners are adjacent in memory (R, stored [r, n]) needs no turn: for
      // a fixed column the 32 rows of a warp are one 128-byte run already.  Old values of this
      // thread's own row, columns [p, p+16), kept in the same registers as o[e / 4][e % 4].
      const bool by_column = factor && I.own_stride == 1 && !vec4;
      const int own_row = (second ? I.own1 : I.own0) + q;
      auto fetch_old_col = [&](int p, float (*o)[4]) {
        const float* fp = fbase + own_row + I.k_stride * p;
        const bool row_ok = own_row < I.own_count;
#pragma unroll
        for (int e = 0; e < 16; ++e) o[e >> 2][e & 3] = (row_ok && p + e < r) ? __ldcg(fp + I.k_stride * e) : 0.f;
      };
      // A factor stored row by row (L, [m, r]) whose rows start on 32-byte boundaries and hold a multiple of
      // eight values needs no turn either: a lane moves 32 bytes per access, which is a whole sector.
      const bool by_row = factor && I.k_stride == 1 && ((I.own_stride | r | I.f32_off) & 7) == 0;
      auto fetch_old_row = [&](int p, float (*o)[4]) {
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
      if (by_row) fetch_old_row(0, oldA);
      else if (by_column) fetch_old_col(0, oldA);
      else if (factor) fetch_old(0, oldA);
      // one lane per warp polls (fewer pollers on the barrier), then the warp agrees: the
      // tensor-memory loads below need all 32 lanes
      bool got = true;
      if (lane == 0) got = mbar_wait(&sh.tfull[acc], acc_phase, abort, a.status, ST_WAIT_TMEM_FULL);
      got = __shfl_sync(0xffffffffu, got, 0);
      if (!got) break;
      tc_fence_after();
      const uint32_t t0 = tmem_base + lane_addr + (uint32_t)(acc * a.acc_cols + (second ? I.col2 : 0));
      // With one accumulator buffer the next item's MMAs wait for this epilogue.  Its memory traffic is the slow
      // part, so the sums D0 + D1 are first parked in spare tensor-memory columns (this warp's own lanes, the
      // same columns for every item) and the accumulator is handed back at once; the pieces below then read the
      // parked sums while the next main loop runs.
      const bool parked = factor && a.sum_col >= 0;
      const uint32_t ts = tmem_base + lane_addr + (uint32_t)(a.sum_col + (second ? rp : 0));
      if (parked) {
        for (int p = 0; p < rp; p += 16) {
          float d0[16], d1[16];
          tmem_ld16(t0 + (uint32_t)p, d0);
          tmem_ld16(t0 + (uint32_t)(rp + p), d1);
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 16; ++e) d0[e] += d1[e];
          tmem_st16(ts + (uint32_t)p, d0);
        }
        tmem_st_wait();
      }
      const bool early = parked || !has_work;   // (a warp without work never reads the accumulator)
      if (early) {
        tc_fence_before();
        mbar_arrive(&sh.tempty[acc]);
      }
      // columns [p, p+16) of D0 + D1 of this thread's row
      auto sum16 = [&](int p, float* sd) {
        if (parked) {
          tmem_ld16(ts + (uint32_t)p, sd);
          tmem_ld_wait();
        } else {
          float d1[16];
          tmem_ld16(t0 + (uint32_t)p, sd);
          tmem_ld16(t0 + (uint32_t)(rp + p), d1);
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 16; ++e) sd[e] += d1[e];
        }
      };
      if (!has_work) {
        // nothing to drain for this warp
      } else if (I.epi == EPI_FACTOR) {
        uint16_t* dst = a.work_bf16 + I.dst_off;
        // one piece: accumulator columns [p, p+16) of this thread's row, old values in `o`
        auto piece = [&](int p, float (*o)[4]) {
          float acc16[16];
          sum16(p, acc16);
          float v[4][4];                 // v[j] = columns 4j .. 4j+3 of this thread's row
#pragma unroll
          for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) v[j][e] = acc16[4 * j + e];
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
            for (int e = 0; e < 4; ++e) x[e] = k + e < r ? o[i][e] + I.coef * sd[i][e] : 0.f;
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
            *reinterpret_cast<uint2*>(drow + rp) = make_uint2(l01, l23);
          }
        };
        // the same piece without the turn: this thread's row, columns [p, p+16)
        auto piece_col = [&](int p, float (*o)[4]) {
          float sd[16];
          sum16(p, sd);
          if (own_row >= I.own_count) return;
          float* fp = fbase + own_row + I.k_stride * p;
          uint32_t hi[8], lo[8];
#pragma unroll
          for (int e = 0; e < 16; e += 2) {
            const float x0 = p + e < r ? o[e >> 2][e & 3] + I.coef * sd[e] : 0.f;
            const float x1 = p + e + 1 < r ? o[(e + 1) >> 2][(e + 1) & 3] + I.coef * sd[e + 1] : 0.f;
            if (p + e < r) __stcg(fp + I.k_stride * e, x0);
            if (p + e + 1 < r) __stcg(fp + I.k_stride * (e + 1), x1);
            split_bf16x2(x0, x1, hi[e >> 1], lo[e >> 1]);
          }
          uint16_t* drow = dst + (int64_t)I.dst_ld * own_row + p;
          st_b32x8(drow, hi);
          st_b32x8(drow + rp, lo);
        };
        // and for a row-stored factor with aligned rows
        auto piece_row = [&](int p, float (*o)[4]) {
          float sd[16];
          sum16(p, sd);
          if (own_row >= I.own_count) return;
          float x[16];
          uint32_t hi[8], lo[8];
#pragma unroll
          for (int e = 0; e < 16; e += 2) {
            x[e] = p + e < r ? o[e >> 2][e & 3] + I.coef * sd[e] : 0.f;
            x[e + 1] = p + e + 1 < r ? o[(e + 1) >> 2][(e + 1) & 3] + I.coef * sd[e + 1] : 0.f;
            split_bf16x2(x[e], x[e + 1], hi[e >> 1], lo[e >> 1]);
          }
          float* fp = fbase + I.own_stride * own_row + p;
          if (p < r) st_f32x8(fp, x);
          if (p + 8 < r) st_f32x8(fp + 8, x + 8);
          uint16_t* drow = dst + (int64_t)I.dst_ld * own_row + p;
          st_b32x8(drow, hi);
          st_b32x8(drow + rp, lo);
        };
        if (by_row) {
#pragma unroll 1
          for (int p = 0; p < rp; p += 32) {
            if (p + 16 < rp) fetch_old_row(p + 16, oldB);
            piece_row(p, oldA);
            if (p + 16 < rp) {
              if (p + 32 < rp) fetch_old_row(p + 32, oldA);
              piece_row(p + 16, oldB);
            }
          }
        } else if (by_column) {
#pragma unroll 1
          for (int p = 0; p < rp; p += 32) {
            if (p + 16 < rp) fetch_old_col(p + 16, oldB);
            piece_col(p, oldA);
            if (p + 16 < rp) {
              if (p + 32 < rp) fetch_old_col(p + 32, oldA);
              piece_col(p + 16, oldB);
            }
          }
        } else {
#pragma unroll 1
          for (int p = 0; p < rp; p += 32) {
            if (p + 16 < rp) fetch_old(p + 16, oldB);
            piece(p, oldA);
            if (p + 16 < rp) {
              if (p + 32 < rp) fetch_old(p + 32, oldA);
              piece(p + 16, oldB);
            }
          }
        }
      } else if (I.epi == EPI_GRAM) {
        uint16_t* dst = a.work_bf16 + I.dst_off;
        for (int p = 0; p < rp; p += 16) {
          float d0[16], d1[16], d2[16], d3[16];
          tmem_ld16(t0 + (uint32_t)p, d0);
          tmem_ld16(t0 + (uint32_t)(rp + p), d1);
          tmem_ld16(t0 + (uint32_t)(2 * rp + p), d2);
          tmem_ld16(t0 + (uint32_t)(3 * rp + p), d3);
          tmem_ld_wait();
          if (q < rp) {
            uint32_t hi[8], lo[8];
#pragma unroll
            for (int e = 0; e < 16; e += 2) {
              const float x0 = I.coef * ((d0[e] + d1[e]) + (d2[e] + d3[e]));
              const float x1 = I.coef * ((d0[e + 1] + d1[e + 1]) + (d2[e + 1] + d3[e + 1]));
              split_bf16x2(x0, x1, hi[e >> 1], lo[e >> 1]);
            }
            uint4* dh = reinterpret_cast<uint4*>(dst + (int64_t)I.dst_ld * q + p);
            uint4* dl = reinterpret_cast<uint4*>(dst + (int64_t)I.dst_ld * q + rp + p);
            dh[0] = make_uint4(hi[0], hi[1], hi[2], hi[3]);
            dh[1] = make_uint4(hi[4], hi[5], hi[6], hi[7]);
            dl[0] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
            dl[1] = make_uint4(lo[4], lo[5], lo[6], lo[7]);
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
