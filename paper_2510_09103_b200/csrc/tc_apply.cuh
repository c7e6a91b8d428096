// Tensor-core "apply" kernel of the low-rank path: rebuilds the corrected momentum tile by tile and
// writes the parameters (Algorithm 1 lines 4, 6, 8 and 9 combined):
//
//   m^c = cg g + c0 L0 R0 - c1 L R          (= g + c (P_{t-1} - P_t) with the correction on)
//   W  <- W - lr s_b ( clamp( m^c / (sqrt(v) + eps) ) + lambda_b W )
//
// An item is a 128-row panel of one block times a run of column tiles.  The split-bf16 rows
// [L0 hi | L0 lo | L hi | L lo] of the panel stay in shared memory for the whole run; per column tile
// the matching rows of [R0^T hi | R0^T lo | R^T hi | R^T lo] arrive one 64-column box at a time
// through a ring of 16 KB stages, and every 16 columns of a box are multiplied at once with the
// resident L columns they pair with (hi*hi and lo*hi for columns of a hi part, hi*lo for columns of
// a lo part; the new set with a negated A operand), so the accumulator ends up holding
// D = L0 R0 - L R.
//
// g and W never pass through registers on their way in or out: a mover thread brings them in
// quarter tiles (128 rows x 32 columns: 16 KB of W, 8 KB of g) by TMA into a small ring of
// shared-memory buffers, several quarters ahead of their use, and writes the updated W back from
// the same buffer by TMA.  Each of the 256 epilogue threads owns one row of the panel: it reads its
// accumulator row from tensor memory, its 16 columns of g and W from the (swizzled) buffer, and
// puts the new W back in place.  A per-element v, where a block has one, travels like W.
// The m x n matrices m_t, r_t and m^c are never stored.
//
// Ranks above 128 do not leave room for a resident L panel (4 rp columns of 128 rows).  The kernel's
// second form (kStream) streams L as well: a stage of its ring holds four boxes - 64 columns of
// L hi, L lo, R^T hi and R^T lo of one factor set - and feeds hi*hi, lo*hi and hi*lo for those
// columns; the previous set is always taken first, the refitted set second.  Everything after the
// accumulator (the g / W ring, the epilogue) is the same code.
#pragma once

#include <cuda.h>

#include "adapm_internal.h"
#include "device_math.cuh"
#include "tc_common.cuh"

namespace adapm {
namespace tc {

constexpr int kApplyThreads = 352;         // producer warp, MMA warp, eight epilogue warps, mover warp
constexpr int kApplyNT = 128;              // columns per tile
constexpr int kApplyQC = 32;               // columns per quarter tile
constexpr int kApplyMaxStages = 8;         // R ring depth limit
constexpr int kApplyMaxBufs = 6;           // g / W ring depth limit
constexpr int kWBoxBytes = 128 * kApplyQC * 4;   // a quarter tile of W: 128 rows of 128 bytes
constexpr int kGBoxBytes = 128 * kApplyQC * 2;   // and of g: 128 rows of 64 bytes
constexpr int kApplyBufBytes = kWBoxBytes + kGBoxBytes;    // + kWBoxBytes where a block has a per-element v

struct ApplyItem {
  int64_t off;               // element offset of the block in params / grads
  int64_t v_off;             // float offset of v in state
  int32_t rows, cols, r, rp;
  int32_t half;              // column at which the lo part of a factor set starts (a set is 2 half columns wide)
  int32_t map_l, map_r;      // split factors, previous and final set side by side: [rows, 4rp] and [cols, 4rp]
                             // = [hi0 | lo0 | hi1 | lo1], boxes of 64 x 128
  int32_t map_w, map_g;      // params and grads of the block, boxes of 32 x 128
  int32_t map_v;             // per-element v of the block (same boxes as params); unused with a group v
  int32_t map_sh;            // bf16 copy of the params (same boxes as grads); used when the launch has a shadow
  int32_t row0;              // first row of the panel
  int32_t tile0, n_tiles;    // column tiles [tile0, tile0 + n_tiles) of 128 columns
  int32_t nbc1, nbc2;        // 64-wide boxes across the 2rp columns of the previous set / the 4rp of both
  int32_t v_mode, v_group_rows;
  float lr_scale, wd;
};

struct ApplyArgs {
  const ApplyItem* items;
  int32_t n_items;
  const CUtensorMap* maps;
  float* state;
  int32_t* status;
  StepScalars sc;
  int32_t use_new;           // 0: c1 == 0, the refitted factors are not needed
  int32_t parity;            // 0: the left half of the operands holds the previous factors, 1: the right half
  const float* gscale;       // device scalar: every gradient counts as gscale[0] * g (nullptr: 1)
  int32_t shadow;            // 1: the bf16 copy of the parameters is written with W (ApplyItem::map_sh)
  int32_t r_region_off;      // byte offset of the R ring inside the dynamic shared memory
  int32_t n_rstages;         // R ring depth (1..kApplyMaxStages); a stage is one 64 x 128 box of R^T
  int32_t w_region_off;      // byte offset of the g / W ring
  int32_t n_bufs;            // g / W ring depth (1..kApplyMaxBufs)
  int32_t buf_bytes;         // one buffer: W, g and, if any block of the launch has a per-element v, v
};

struct __align__(8) ApplyShared {
  uint64_t lfull, lempty, rfull[kApplyMaxStages], rempty[kApplyMaxStages], tfull[2], tempty[2];
  uint64_t wfull[kApplyMaxBufs];   // a quarter's g and W have landed
  uint64_t wdone[kApplyMaxBufs];   // all eight epilogue warps have put their new W back
  uint32_t tmem_base;
  int abort;
};

template <bool kStream>
__global__ void __launch_bounds__(kApplyThreads, 1) tc_apply_kernel(ApplyArgs a) {
  extern __shared__ uint8_t dyn_smem[];
  __shared__ ApplyShared sh;
  __shared__ int skip_launch;
  if (threadIdx.x == 0) skip_launch = *reinterpret_cast<volatile int32_t*>(a.status) != 0;
  __syncthreads();
  if (skip_launch) return;   // an earlier launch of the step gave up: leave W and v untouched
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(dyn_smem) + 1023) & ~(uintptr_t)1023);
  uint8_t* smem_l = smem;
  uint8_t* smem_r = smem + a.r_region_off;
  uint8_t* smem_w = smem + a.w_region_off;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort = &sh.abort;
  const int n_sets = a.use_new ? 2 : 1;

  if (threadIdx.x == 0) {
    mbar_init(&sh.lfull, 1); mbar_init(&sh.lempty, 1);
    for (int i = 0; i < kApplyMaxStages; ++i) { mbar_init(&sh.rfull[i], 1); mbar_init(&sh.rempty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&sh.tfull[i], 1); mbar_init(&sh.tempty[i], 8); }
    for (int i = 0; i < kApplyMaxBufs; ++i) { mbar_init(&sh.wfull[i], 1); mbar_init(&sh.wdone[i], 8); }
    sh.abort = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(&sh.tmem_base, 256);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = sh.tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      uint32_t item_phase = 0, rphase = 0;
      int rs = 0;
      bool ok = true;
      int l_loads = 0, r_loads = 0;
      for (int it = blockIdx.x; it < a.n_items && ok; it += gridDim.x) {
        const ApplyItem I = a.items[it];
        if (kStream) {
          // a stage = 64 columns of [L hi, L lo, R^T hi, R^T lo] of one set; previous set first
          const int nbh = (I.rp + 63) >> 6;
          for (int t = 0; t < I.n_tiles && ok; ++t) {
            const int col0 = (I.tile0 + t) * kApplyNT;
            for (int si = 0; si < n_sets && ok; ++si) {
              const int xs = (si == 0 ? a.parity : 1 - a.parity) * 2 * I.half;
              for (int jb = 0; jb < nbh; ++jb) {
                if (!mbar_wait(&sh.rempty[rs], rphase ^ 1u, abort, a.status, ST_WAIT_EMPTY)) { ok = false; break; }
                uint8_t* st = smem_r + (size_t)rs * (4 * kBoxBytes);
                mbar_arrive_expect_tx(&sh.rfull[rs], 4u * kBoxBytes);
                tma_load_box(st, a.maps + I.map_l, xs + 64 * jb, I.row0, &sh.rfull[rs]);
                tma_load_box(st + kBoxBytes, a.maps + I.map_l, xs + I.half + 64 * jb, I.row0, &sh.rfull[rs]);
                tma_load_box(st + 2 * kBoxBytes, a.maps + I.map_r, xs + 64 * jb, col0, &sh.rfull[rs]);
                tma_load_box(st + 3 * kBoxBytes, a.maps + I.map_r, xs + I.half + 64 * jb, col0, &sh.rfull[rs]);
                ++r_loads;
                if (++rs == a.n_rstages) { rs = 0; rphase ^= 1u; }
              }
            }
          }
          continue;
        }
        if (!mbar_wait(&sh.lempty, item_phase ^ 1u, abort, a.status, ST_WAIT_EMPTY)) { ok = false; break; }
        const int nb = n_sets == 2 ? I.nbc2 : I.nbc1;
        // with only the previous set in use, and that set in the right half, the boxes start there
        const int x0 = (n_sets == 1 && a.parity) ? 2 * I.rp : 0;
        mbar_arrive_expect_tx(&sh.lfull, (uint32_t)nb * kBoxBytes);
        for (int bc = 0; bc < nb; ++bc)
          tma_load_box(smem_l + (size_t)bc * kBoxBytes, a.maps + I.map_l, x0 + 64 * bc, I.row0, &sh.lfull);
        ++l_loads;
        for (int t = 0; t < I.n_tiles && ok; ++t) {
          const int col0 = (I.tile0 + t) * kApplyNT;
          for (int bc = 0; bc < nb; ++bc) {
            if (!mbar_wait(&sh.rempty[rs], rphase ^ 1u, abort, a.status, ST_WAIT_EMPTY)) { ok = false; break; }
            mbar_arrive_expect_tx(&sh.rfull[rs], (uint32_t)kBoxBytes);
            tma_load_box(smem_r + (size_t)rs * kBoxBytes, a.maps + I.map_r, x0 + 64 * bc, col0, &sh.rfull[rs]);
            ++r_loads;
            if (++rs == a.n_rstages) { rs = 0; rphase ^= 1u; }
          }
        }
        item_phase ^= 1u;
      }
      if (!ok) {   // let the copies already issued land before the CTA exits
        if (l_loads)
          for (uint32_t spin = 0; spin < kSpinLimit && !mbar_try_wait(&sh.lfull, (uint32_t)(l_loads - 1) & 1u); ++spin)
            __nanosleep(64);
        const int back = r_loads < a.n_rstages ? r_loads : a.n_rstages;
        for (int q = 0; q < back; ++q) {
          int st = rs - 1 - q;
          uint32_t ph = rphase;
          if (st < 0) { st += a.n_rstages; ph ^= 1u; }
          for (uint32_t spin = 0; spin < kSpinLimit && !mbar_try_wait(&sh.rfull[st], ph); ++spin) __nanosleep(64);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t item_phase = 0, rphase = 0;
      int rs = 0;
      int j = 0;   // running tile count of this CTA
      bool ok = true;
      const uint32_t l_base = smem_u32(smem_l), r_base = smem_u32(smem_r);
      const uint32_t dhi = desc_hi();
      for (int it = blockIdx.x; it < a.n_items && ok; it += gridDim.x) {
        const ApplyItem I = a.items[it];
        const int ks = I.rp >> 4;     // 16-wide K steps per part (hi or lo of one set)
        const int ktot = n_sets * 2 * ks;
        const int nb = n_sets == 2 ? I.nbc2 : I.nbc1;
        const uint32_t idesc_pos = make_idesc(kApplyNT, false, false, false);
        const uint32_t idesc_neg = make_idesc(kApplyNT, false, false, true);
        const uint32_t la = desc_lo(l_base, 16);
        if (kStream) {
          const int nbh = (I.rp + 63) >> 6;
          for (int t = 0; t < I.n_tiles && ok; ++t, ++j) {
            const int acc = j & 1;
            const uint32_t acc_phase = (uint32_t)(j >> 1) & 1u;
            if (!mbar_wait(&sh.tempty[acc], acc_phase ^ 1u, abort, a.status, ST_WAIT_TMEM_EMPTY)) { ok = false; break; }
            const uint32_t d = tmem_base + (uint32_t)(acc * kApplyNT);
            uint32_t accumulate = 0;
            for (int si = 0; si < n_sets && ok; ++si) {
              const uint32_t idesc = si ? idesc_neg : idesc_pos;      // the refitted set enters negated
              for (int jb = 0; jb < nbh; ++jb) {
                if (!mbar_wait(&sh.rfull[rs], rphase, abort, a.status, ST_WAIT_FULL)) { ok = false; break; }
                tc_fence_after();
                const uint32_t st = r_base + (uint32_t)rs * (4u * kBoxBytes);
                const uint32_t ahi = desc_lo(st, 16), alo = desc_lo(st + kBoxBytes, 16);
                const uint32_t bhi = desc_lo(st + 2 * kBoxBytes, 16), blo = desc_lo(st + 3 * kBoxBytes, 16);
                for (int kk = 0; kk < 4; ++kk) {
                  if (4 * jb + kk >= ks) break;
                  const uint32_t o = (uint32_t)(kk * 2);
                  mma_bf16(d, desc_join(ahi + o, dhi), desc_join(bhi + o, dhi), idesc, accumulate);
                  mma_bf16(d, desc_join(alo + o, dhi), desc_join(bhi + o, dhi), idesc, 1u);
                  mma_bf16(d, desc_join(ahi + o, dhi), desc_join(blo + o, dhi), idesc, 1u);
                  accumulate = 1;
                }
                mma_commit(&sh.rempty[rs]);
                if (++rs == a.n_rstages) { rs = 0; rphase ^= 1u; }
              }
            }
            if (ok) mma_commit(&sh.tfull[acc]);
          }
          continue;
        }
        if (!mbar_wait(&sh.lfull, item_phase, abort, a.status, ST_WAIT_FULL)) break;
        for (int t = 0; t < I.n_tiles && ok; ++t, ++j) {
          const int acc = j & 1;
          const uint32_t acc_phase = (uint32_t)(j >> 1) & 1u;
          if (!mbar_wait(&sh.tempty[acc], acc_phase ^ 1u, abort, a.status, ST_WAIT_TMEM_EMPTY)) { ok = false; break; }
          const uint32_t d = tmem_base + (uint32_t)(acc * kApplyNT);
          uint32_t accumulate = 0;
          // K step k of the [.., 4rp] operands: box k / 4 (16 KB apart), 32 bytes per step inside it
          auto kstep = [](int k) { return (uint32_t)((k >> 2) * (kBoxBytes >> 4) + (k & 3) * 2); };
          for (int bc = 0; bc < nb; ++bc) {
            if (!mbar_wait(&sh.rfull[rs], rphase, abort, a.status, ST_WAIT_FULL)) { ok = false; break; }
            tc_fence_after();
            const uint32_t rb = desc_lo(r_base + (uint32_t)rs * kBoxBytes, 16);
            for (int kk = 0; kk < 4; ++kk) {
              const int kb = 4 * bc + kk;              // K step of [R0 hi | R0 lo | R hi | R lo] held by this box
              if (kb >= ktot) break;
              const int set = kb >= 2 * ks ? 1 : 0;
              const int w = kb - set * 2 * ks;         // K step inside the set: hi part, then lo part
              // the set that holds the refitted factors enters with a negated A operand
              const uint32_t idesc = (n_sets == 2 && (set ^ a.parity)) ? idesc_neg : idesc_pos;
              const uint64_t b = desc_join(rb + (uint32_t)(kk * 2), dhi);
              if (w < ks) {                            // hi * hi, lo * hi
                mma_bf16(d, desc_join(la + kstep(kb), dhi), b, idesc, accumulate);
                mma_bf16(d, desc_join(la + kstep(kb + ks), dhi), b, idesc, 1u);
              } else {                                 // hi * lo
                mma_bf16(d, desc_join(la + kstep(kb - ks), dhi), b, idesc, accumulate);
              }
              accumulate = 1;
            }
            mma_commit(&sh.rempty[rs]);
            if (++rs == a.n_rstages) { rs = 0; rphase ^= 1u; }
          }
          if (ok) mma_commit(&sh.tfull[acc]);
        }
        if (ok) mma_commit(&sh.lempty);
        item_phase ^= 1u;
      }
    }
  } else if (warp == 10) {
    // ------------------------------------------------------------------ g / W mover
    if (lane == 0) {
      // load cursor: runs n_bufs quarters ahead of the quarter being stored
      int ld_it = blockIdx.x, ld_q = 0, ld_nq = 0, n_loaded = 0;
      ApplyItem LI;
      if (ld_it < a.n_items) { LI = a.items[ld_it]; ld_nq = 4 * LI.n_tiles; }
      auto load_next = [&]() {
        const int b = n_loaded % a.n_bufs;
        uint8_t* buf = smem_w + (size_t)b * a.buf_bytes;
        const int col = (LI.tile0 + (ld_q >> 2)) * kApplyNT + (ld_q & 3) * kApplyQC;
        const bool with_v = LI.v_mode == ADAPM_V_ELEMENT;
        mbar_arrive_expect_tx(&sh.wfull[b], (uint32_t)(kApplyBufBytes + (with_v ? kWBoxBytes : 0)));
        tma_load_box(buf, a.maps + LI.map_w, col, LI.row0, &sh.wfull[b]);
        tma_load_box(buf + kWBoxBytes, a.maps + LI.map_g, col, LI.row0, &sh.wfull[b]);
        if (with_v) tma_load_box(buf + kApplyBufBytes, a.maps + LI.map_v, col, LI.row0, &sh.wfull[b]);
        ++n_loaded;
        if (++ld_q == ld_nq) {
          ld_it += gridDim.x; ld_q = 0; ld_nq = 0;
          if (ld_it < a.n_items) { LI = a.items[ld_it]; ld_nq = 4 * LI.n_tiles; }
        }
      };
      for (int i = 0; i < a.n_bufs && ld_it < a.n_items; ++i) load_next();
      int k = 0;   // running quarter count of this CTA
      bool ok = true;
      for (int it = blockIdx.x; it < a.n_items && ok; it += gridDim.x) {
        const ApplyItem I = a.items[it];
        for (int q = 0; q < 4 * I.n_tiles; ++q, ++k) {
          const int b = k % a.n_bufs;
          if (!mbar_wait(&sh.wdone[b], (uint32_t)(k / a.n_bufs) & 1u, abort, a.status, ST_WAIT_DRAIN)) { ok = false; break; }
          const int col = (I.tile0 + (q >> 2)) * kApplyNT + (q & 3) * kApplyQC;
          // (a quarter that lies past the last column is not stored)
          if (col < I.cols) {
            const uint8_t* buf = smem_w + (size_t)b * a.buf_bytes;
            tma_store_box(a.maps + I.map_w, col, I.row0, buf);
            if (a.shadow) tma_store_box(a.maps + I.map_sh, col, I.row0, buf + kWBoxBytes);
            if (I.v_mode == ADAPM_V_ELEMENT) tma_store_box(a.maps + I.map_v, col, I.row0, buf + kApplyBufBytes);
          }
          bulk_commit_group();
          if ((a.n_bufs < 2 || (k & 1)) && ld_it < a.n_items) {
            // two quarters at a time: their rows are neighbours in memory, and requests that reach DRAM
            // together share its open pages.  They go into this buffer and the one stored before it,
            // once both stores have read them.
            bulk_wait_group_read<0>();
            load_next();
            if (a.n_bufs >= 2 && ld_it < a.n_items) load_next();
          }
        }
      }
      bulk_wait_group<0>();
      if (!ok) {   // let the loads already issued land before the CTA exits
        for (int kk = k; kk < n_loaded; ++kk) {
          const uint32_t ph = (uint32_t)(kk / a.n_bufs) & 1u;
          for (uint32_t spin = 0; spin < kSpinLimit && !mbar_try_wait(&sh.wfull[kk % a.n_bufs], ph); ++spin)
            __nanosleep(64);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int e = warp - 2;
    const int wq4 = warp & 3;                             // which 32 accumulator rows this warp may read
    const int half = e >> 2;                              // which 16 columns of a quarter
    const uint32_t lane_addr = (uint32_t)(32 * wq4) << 16;
    const int rloc = 32 * wq4 + lane;                     // this thread's row of the panel
    StepScalars sc = a.sc;
    const float gs = a.gscale ? *a.gscale : 1.f;
    sc.cg *= gs;               // m^c = cg (gs g) + c0 D
    // byte offsets of this thread's 16-byte chunks inside a buffer: the 128-byte swizzle turns chunk c of
    // row r into chunk c ^ (r % 8), the 64-byte swizzle chunk c of a 64-byte row into c ^ ((r / 2) % 4)
    uint32_t w_at[4], g_at[2];
#pragma unroll
    for (int i = 0; i < 4; ++i) w_at[i] = (uint32_t)(rloc * 128 + (((4 * half + i) ^ (rloc & 7)) << 4));
#pragma unroll
    for (int i = 0; i < 2; ++i)
      g_at[i] = (uint32_t)(kWBoxBytes + rloc * 64 + (((2 * half + i) ^ ((rloc >> 1) & 3)) << 4));
    int j = 0, k = 0;   // running tile and quarter counts of this CTA
    bool ok = true;
    for (int it = blockIdx.x; it < a.n_items && ok; it += gridDim.x) {
      const ApplyItem I = a.items[it];
      const bool grouped = I.v_mode == ADAPM_V_BLOCKMEAN;
      const float lr_s = sc.lr * I.lr_scale;
      const int row = I.row0 + rloc;
      const bool rok = row < I.rows;
      // one denominator per row when v is a group scalar: m^c / (sqrt(v) + eps) becomes a product
      const float v_row = (rok && grouped) ? a.state[I.v_off + row / I.v_group_rows] : 0.f;
      const float kr = sc.inv_bc1 / (sqrtf(v_row * sc.inv_bc2) + sc.eps);
      const int n_q = 4 * I.n_tiles;
      for (int q = 0; q < n_q; ++q, ++k) {
        const int jt = j + (q >> 2), sub = q & 3;
        const int acc = jt & 1;
        const int b = k % a.n_bufs;
        if (sub == 0) {
          // one lane per warp polls, then the warp agrees: the tensor-memory loads need all 32 lanes
          bool got = true;
          if (lane == 0) got = mbar_wait(&sh.tfull[acc], (uint32_t)(jt >> 1) & 1u, abort, a.status, ST_WAIT_TMEM_FULL);
          got = __shfl_sync(0xffffffffu, got, 0);
          if (!got) { ok = false; break; }
          tc_fence_after();
        }
        float d[16];
        tmem_ld16(tmem_base + lane_addr + (uint32_t)(acc * kApplyNT + sub * kApplyQC + 16 * half), d);
        if (!mbar_wait(&sh.wfull[b], (uint32_t)(k / a.n_bufs) & 1u, abort, a.status, ST_WAIT_FULL)) ok = false;
        ok = __all_sync(0xffffffffu, ok);
        tmem_ld_wait();
        if (!ok) break;
        uint8_t* buf = smem_w + (size_t)b * a.buf_bytes;
        float gf[16];
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          const uint4 gg = *reinterpret_cast<const uint4*>(buf + g_at[i]);
          const uint32_t gw[4] = {gg.x, gg.y, gg.z, gg.w};
#pragma unroll
          for (int x = 0; x < 4; ++x) {
            gf[8 * i + 2 * x] = __uint_as_float(gw[x] << 16);
            gf[8 * i + 2 * x + 1] = __uint_as_float(gw[x] & 0xffff0000u);
          }
        }
        uint32_t shw[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          float4* wp = reinterpret_cast<float4*>(buf + w_at[i]);
          const float4 wo = *wp;
          float w[4] = {wo.x, wo.y, wo.z, wo.w};
          if (grouped) {
#pragma unroll
            for (int x = 0; x < 4; ++x) {
              float ratio = (sc.cg * gf[4 * i + x] + sc.c0 * d[4 * i + x]) * kr;
              ratio = ratio > sc.clip ? sc.clip : (ratio < -sc.clip ? -sc.clip : ratio);
              w[x] = w[x] - lr_s * (ratio + I.wd * w[x]);
            }
          } else {
            float4* vp = reinterpret_cast<float4*>(buf + kApplyBufBytes + w_at[i]);   // v lies like W
            const float4 vo = *vp;
            float vv[4] = {vo.x, vo.y, vo.z, vo.w};
#pragma unroll
            for (int x = 0; x < 4; ++x) {
              const float g1 = gf[4 * i + x];
              vv[x] = sc.beta2 * vv[x] + (1.f - sc.beta2) * ((gs * g1) * (gs * g1));
              w[x] = adapm_param_update(w[x], sc.cg * g1 + sc.c0 * d[4 * i + x], vv[x], sc, lr_s, I.wd);
            }
            *vp = make_float4(vv[0], vv[1], vv[2], vv[3]);
          }
          *wp = make_float4(w[0], w[1], w[2], w[3]);
          shw[2 * i] = pack_bf16x2(w[0], w[1]);
          shw[2 * i + 1] = pack_bf16x2(w[2], w[3]);
        }
        if (a.shadow) {
          // The bf16 copy of the new W takes the place of the gradient in the buffer (this thread's two 16-byte
          // pieces, already read): it has g's box shape and swizzle, and the mover stores it with the same kind of
          // tensor map.
          *reinterpret_cast<uint4*>(buf + g_at[0]) = make_uint4(shw[0], shw[1], shw[2], shw[3]);
          *reinterpret_cast<uint4*>(buf + g_at[1]) = make_uint4(shw[4], shw[5], shw[6], shw[7]);
        }
        // one arrival per warp: every lane orders its own writes (and tensor-memory reads), the warp meets
        fence_async_smem();
        if (sub == 3) tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(&sh.wdone[b]);
          if (sub == 3) mbar_arrive(&sh.tempty[acc]);
        }
      }
      j += I.n_tiles;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 256);
  }
}

}  // namespace tc
}  // namespace adapm
