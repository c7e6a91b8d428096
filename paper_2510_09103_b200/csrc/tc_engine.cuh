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
//   Gram item: one of the r x r matrices above, scaled and stored as a split-bf16 B operand.
//
// fp32 factors are carried into the bf16 tensor cores as hi + lo pairs (two bf16 numbers whose sum
// has ~16 significant bits); gradients are bf16 already and enter unchanged.  Operands with hi and
// lo parts are stored side by side ([rows, 2 rp]: hi columns then lo columns, rp = r rounded up to
// 16), so that used as the N side of an MMA the two parts land in two column ranges of the
// accumulator, which the epilogue adds.
//
// Warp roles (192 threads): warp 0 issues TMA loads into a ring of stages, warp 1 issues the MMAs,
// warps 2-5 drain the accumulator.  With two accumulator buffers the epilogue of one item overlaps
// the K-loops of the next.  Every wait is bounded; when one runs out the CTA records a status bit,
// stops taking work and leaves through the common exit (which frees its tensor memory).
#pragma once

#include <cuda.h>

#include "tc_common.cuh"

namespace adapm {
namespace tc {

constexpr int kMaxSegs = 6;
constexpr int kStageABytes = 2 * kBoxBytes;      // the A side of a stage: 128 x 64 bf16
constexpr int kEngineThreads = 192;

enum : int32_t { EPI_FACTOR = 0, EPI_GRAM = 1, EPI_DUMP = 2 };

struct Seg {
  int32_t map_a, map_b;      // tensor-map indices
  int32_t ax, ay, bx, by;    // element coordinates of the first box of each operand
  int16_t a_mode, b_mode;    // 0: K runs along x (K-major), 1: K runs along y (MN-major)
  int16_t nb_b;              // 64-wide boxes of B per chunk = ceil(n / 64)
  int16_t n;                 // MMA N (multiple of 16, <= 256)
  int32_t k;                 // K extent, multiple of 16
  int16_t d_col;             // accumulator column this segment starts at
  int16_t first;             // 1: its first MMA overwrites the accumulator
};

struct Item {
  Seg seg[kMaxSegs];
  int32_t n_seg;
  int32_t epi;
  // EPI_FACTOR: the thread that owns accumulator row q updates factor entries (owner = own0 + q, k):
  //   f32[own_stride * owner + k_stride * k] += coef * (D[q][k] + D[q][rp + k])        k < r
  //   dst[owner][k] = hi, dst[owner][rp + k] = lo                                      k < rp
  // EPI_GRAM: G[q][k] = coef * (D[q][k] + D[q][rp+k] + D[q][2rp+k] + D[q][3rp+k]);
  //   dst[q][k] = hi, dst[rp + q][k] = lo                                              q, k < rp
  // EPI_DUMP: f32[q * n_dump + j] = D[q][j]                                            j < n_dump
  int32_t own0, own_count;   // first owner and number of owners of the whole matrix
  int32_t r, rp;
  int64_t f32_off;           // float offset in the state buffer (EPI_DUMP: in the dump buffer)
  int64_t own_stride, k_stride;
  int64_t dst_off;           // bf16 element offset of the destination array in the workspace
  int32_t dst_ld;            // its row pitch in elements
  int32_t n_dump;
  float coef;
  int32_t cost;              // chunks, for scheduling
};

struct EngineArgs {
  const Item* items;
  int32_t n_items;
  const CUtensorMap* maps;
  float* f32_base;           // state buffer (or dump buffer)
  uint16_t* work_bf16;       // workspace viewed as bf16
  int32_t* status;
  int32_t stage_bytes;       // kStageABytes + 8 KB * (largest nb_b)
  int32_t n_stages;
  int32_t acc_cols;          // tensor-memory columns per accumulator buffer
  int32_t n_acc;             // 1 or 2 accumulator buffers
};

struct __align__(8) EngineShared {
  uint64_t full[8], empty[8], tfull[2], tempty[2];
  uint32_t tmem_base;
  int abort;
};

__device__ __forceinline__ int seg_chunks(const Seg& s) { return (s.k + kBoxCols - 1) / kBoxCols; }

__global__ void __launch_bounds__(kEngineThreads, 1) tc_items_kernel(EngineArgs a) {
  extern __shared__ uint8_t dyn_smem[];
  __shared__ EngineShared sh;
  uint8_t* stages = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(dyn_smem) + 1023) & ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort = &sh.abort;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 8; ++i) { mbar_init(&sh.full[i], 1); mbar_init(&sh.empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&sh.tfull[i], 1); mbar_init(&sh.tempty[i], 128); }
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

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    // Lane 0 waits for the stage and arms its barrier; lanes 0..5 then issue one box each.
    {
      int stage = 0;
      uint32_t phase = 0;
      uint32_t issued = 0;
      bool ok = true;
      for (int it = blockIdx.x; it < a.n_items && ok; it += gridDim.x) {
        const Item& I = a.items[it];
        for (int s = 0; s < I.n_seg && ok; ++s) {
          const Seg S = I.seg[s];
          const int nch = seg_chunks(S);
          // this lane's box: lanes 0,1 the A side, lanes 2.. the B side
          const bool is_a = lane < 2;
          const int h = is_a ? lane : lane - 2;
          const bool active = lane < 2 + S.nb_b;
          const CUtensorMap* map = a.maps + (is_a ? S.map_a : S.map_b);
          const int mode = is_a ? S.a_mode : S.b_mode;
          const int x0 = (is_a ? S.ax : S.bx) + (mode ? 64 * h : 0);
          const int y0 = (is_a ? S.ay : S.by) + (mode ? 0 : 64 * h);
          const int dx = mode ? 0 : 64, dy = mode ? 64 : 0;
          const int soff = is_a ? h * kBoxBytes : kStageABytes + h * kBoxBytes;
          for (int c = 0; c < nch; ++c) {
            bool got = true;
            if (lane == 0) {
              got = mbar_wait(&sh.empty[stage], phase ^ 1u, abort, a.status, ST_WAIT_EMPTY);
              if (got) mbar_arrive_expect_tx(&sh.full[stage], (uint32_t)(2 + S.nb_b) * kBoxBytes);
            }
            got = __shfl_sync(0xffffffffu, got, 0);
            if (!got) { ok = false; break; }
            if (active)
              tma_load_box(stages + (size_t)stage * a.stage_bytes + soff, map, x0 + dx * c, y0 + dy * c, &sh.full[stage]);
            ++issued;
            if (++stage == a.n_stages) { stage = 0; phase ^= 1u; }
          }
        }
      }
      if (!ok && lane == 0) {
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
      for (int it = blockIdx.x; it < a.n_items && ok; it += gridDim.x, ++j) {
        const Item& I = a.items[it];
        const int acc = j % a.n_acc;
        const uint32_t acc_phase = (uint32_t)(j / a.n_acc) & 1u;
        if (!mbar_wait(&sh.tempty[acc], acc_phase ^ 1u, abort, a.status, ST_WAIT_TMEM_EMPTY)) break;
        tc_fence_after();
        const uint32_t d_base = tmem_base + (uint32_t)(acc * a.acc_cols);
        for (int s = 0; s < I.n_seg && ok; ++s) {
          const Seg S = I.seg[s];
          const uint32_t idesc = make_idesc(S.n, S.a_mode != 0, S.b_mode != 0, false);
          const int nch = seg_chunks(S);
          for (int c = 0; c < nch; ++c) {
            if (!mbar_wait(&sh.full[stage], phase, abort, a.status, ST_WAIT_FULL)) { ok = false; break; }
            tc_fence_after();
            const uint32_t sa = smem_u32(stages + (size_t)stage * a.stage_bytes);
            const uint32_t sb = sa + kStageABytes;
            int nk = (S.k - 64 * c + 15) / 16;
            nk = nk > 4 ? 4 : nk;
            for (int q = 0; q < nk; ++q) {
              const uint64_t da = S.a_mode ? desc_mn_major(sa, q) : desc_k_major(sa, q);
              const uint64_t db = S.b_mode ? desc_mn_major(sb, q) : desc_k_major(sb, q);
              const uint32_t accumulate = (S.first && c == 0 && q == 0) ? 0u : 1u;
              mma_bf16(d_base + (uint32_t)S.d_col, da, db, idesc, accumulate);
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
    int j = 0;
    for (int it = blockIdx.x; it < a.n_items; it += gridDim.x, ++j) {
      const Item& I = a.items[it];
      const int acc = j % a.n_acc;
      const uint32_t acc_phase = (uint32_t)(j / a.n_acc) & 1u;
      const int rp = I.rp, r = I.r;
      // EPI_FACTOR: the old factor values of the first 16 columns are requested before the wait
      const int owner = I.own0 + q;
      const bool own_ok = I.epi == EPI_FACTOR && owner < I.own_count;
      float* f = a.f32_base + I.f32_off + I.own_stride * owner;
      float old[16] = {};
      if (own_ok) {
#pragma unroll
        for (int e = 0; e < 16; ++e) old[e] = e < r ? f[I.k_stride * e] : 0.f;
      }
      // one lane per warp polls (fewer pollers on the barrier), then the warp agrees: the
      // tensor-memory loads below need all 32 lanes
      bool got = true;
      if (lane == 0) got = mbar_wait(&sh.tfull[acc], acc_phase, abort, a.status, ST_WAIT_TMEM_FULL);
      got = __shfl_sync(0xffffffffu, got, 0);
      if (!got) break;
      tc_fence_after();
      const uint32_t t0 = tmem_base + lane_addr + (uint32_t)(acc * a.acc_cols);
      if (I.epi == EPI_FACTOR) {
        uint16_t* dst = a.work_bf16 + I.dst_off + (int64_t)I.dst_ld * owner;
        for (int p = 0; p < rp; p += 16) {
          float d0[16], d1[16], nxt[16];
          tmem_ld16(t0 + (uint32_t)p, d0);
          tmem_ld16(t0 + (uint32_t)(rp + p), d1);
          if (own_ok && p + 16 < rp) {     // the next 16 old values travel while this piece is processed
#pragma unroll
            for (int e = 0; e < 16; ++e) nxt[e] = p + 16 + e < r ? f[I.k_stride * (p + 16 + e)] : 0.f;
          }
          tmem_ld_wait();
          if (own_ok) {
            uint32_t hi[8], lo[8];
            float x[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) x[e] = p + e < r ? old[e] + I.coef * (d0[e] + d1[e]) : 0.f;
#pragma unroll
            for (int e = 0; e < 16; ++e)
              if (p + e < r) f[I.k_stride * (p + e)] = x[e];
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              uint16_t h, l;
              split_bf16(x[e], h, l);
              if (e & 1) { hi[e >> 1] |= (uint32_t)h << 16; lo[e >> 1] |= (uint32_t)l << 16; }
              else { hi[e >> 1] = h; lo[e >> 1] = l; }
            }
            uint4* dh = reinterpret_cast<uint4*>(dst + p);
            uint4* dl = reinterpret_cast<uint4*>(dst + rp + p);
            dh[0] = make_uint4(hi[0], hi[1], hi[2], hi[3]);
            dh[1] = make_uint4(hi[4], hi[5], hi[6], hi[7]);
            dl[0] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
            dl[1] = make_uint4(lo[4], lo[5], lo[6], lo[7]);
#pragma unroll
            for (int e = 0; e < 16; ++e) old[e] = nxt[e];
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
            for (int e = 0; e < 16; ++e) {
              const float x = I.coef * ((d0[e] + d1[e]) + (d2[e] + d3[e]));
              uint16_t h, l;
              split_bf16(x, h, l);
              if (e & 1) { hi[e >> 1] |= (uint32_t)h << 16; lo[e >> 1] |= (uint32_t)l << 16; }
              else { hi[e >> 1] = h; lo[e >> 1] = l; }
            }
            uint4* dh = reinterpret_cast<uint4*>(dst + (int64_t)I.dst_ld * q + p);
            uint4* dl = reinterpret_cast<uint4*>(dst + (int64_t)I.dst_ld * (rp + q) + p);
            dh[0] = make_uint4(hi[0], hi[1], hi[2], hi[3]);
            dh[1] = make_uint4(hi[4], hi[5], hi[6], hi[7]);
            dl[0] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
            dl[1] = make_uint4(lo[4], lo[5], lo[6], lo[7]);
          }
        }
      } else {   // EPI_DUMP
        float* out = a.f32_base + I.f32_off + (int64_t)q * I.n_dump;
        for (int p = 0; p < I.n_dump; p += 16) {
          float d0[16];
          tmem_ld16(t0 + (uint32_t)p, d0);
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 16; ++e)
            if (p + e < I.n_dump) out[p + e] = d0[e];
        }
      }
      tc_fence_before();
      mbar_arrive(&sh.tempty[acc]);
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
