// Tensor-core "apply" kernel of the low-rank path: rebuilds the corrected momentum tile by tile and
// writes the parameters (Algorithm 1 lines 4, 6, 8 and 9 combined):
//
//   m^c = cg g + c0 L0 R0 - c1 L R          (= g + c (P_{t-1} - P_t) with the correction on)
//   W  <- W - lr s_b ( clamp( m^c / (sqrt(v) + eps) ) + lambda_b W )
//
// An item is a 128-row panel of one block times a run of column tiles.  The split-bf16 rows of L0
// and L of the panel stay in shared memory for the whole run; per column tile the matching rows of
// R0^T and R^T arrive one 64-column box at a time through a ring of 16 KB stages, and every box is
// multiplied at once with the resident L columns it pairs with (hi*hi and lo*hi for a column of the
// hi half, hi*lo for a column of the lo half; the new pair with a negated A operand), so the
// accumulator ends up holding D = L0 R0 - L R.  Eight epilogue warps then stream g and W through
// registers: a thread reads one accumulator row from tensor memory, the warp turns its 32 x 16 piece around through a small
// shared-memory buffer so that four lanes share a row, and g / W are accessed as 64-byte row
// segments (the next piece's g and W are requested while the current one is processed).
// The ring is kept shallow on purpose: the part of the SM's 256 KB that the CTA does not claim as
// shared memory stays L1, and that L1 bounds how many g / W requests can be in flight.
// The m x n matrices m_t, r_t and m^c are never stored.
#pragma once

#include <cuda.h>

#include "adapm_internal.h"
#include "device_math.cuh"
#include "tc_common.cuh"

namespace adapm {
namespace tc {

constexpr int kApplyThreads = 320;
constexpr int kApplyNT = 128;              // columns per tile
constexpr int kStagePitch = 20;            // floats per row of a warp's 32 x 16 turn-around buffer
constexpr int kStageFloats = 32 * kStagePitch;
constexpr int kApplyMaxStages = 8;         // ring depth limit

struct ApplyItem {
  int64_t off;               // element offset of the block in params / grads
  int64_t v_off;             // float offset of v in state
  int32_t rows, cols, r, rp;
  int32_t map_l0, map_l1, map_r0, map_r1;   // split factors: [rows, 2rp] and [cols, 2rp], boxes of 64 x 128
  int32_t row0;              // first row of the panel
  int32_t tile0, n_tiles;    // column tiles [tile0, tile0 + n_tiles) of 128 columns
  int32_t nbc;               // 64-wide boxes across the 2rp split columns
  int32_t v_mode, v_group_rows;
  float lr_scale, wd;
};

struct ApplyArgs {
  const ApplyItem* items;
  int32_t n_items;
  const CUtensorMap* maps;
  float* params;
  const uint16_t* grads;
  float* state;
  int32_t* status;
  StepScalars sc;
  int32_t use_new;           // 0: c1 == 0, the refitted factors are not needed
  int32_t r_region_off;      // byte offset of the R ring inside the dynamic shared memory
  int32_t n_rstages;         // ring depth (1..kApplyMaxStages); a stage is one 64 x 128 box of R^T
  int32_t turn_off;          // byte offset of the turn-around buffers
};

struct __align__(8) ApplyShared {
  uint64_t lfull, lempty, rfull[kApplyMaxStages], rempty[kApplyMaxStages], tfull[2], tempty[2];
  uint32_t tmem_base;
  int abort;
};

__global__ void __launch_bounds__(kApplyThreads, 1) tc_apply_kernel(ApplyArgs a) {
  extern __shared__ uint8_t dyn_smem[];
  __shared__ ApplyShared sh;
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(dyn_smem) + 1023) & ~(uintptr_t)1023);
  uint8_t* smem_l = smem;
  uint8_t* smem_r = smem + a.r_region_off;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort = &sh.abort;
  const int n_sets = a.use_new ? 2 : 1;

  if (threadIdx.x == 0) {
    mbar_init(&sh.lfull, 1); mbar_init(&sh.lempty, 1);
    for (int i = 0; i < kApplyMaxStages; ++i) { mbar_init(&sh.rfull[i], 1); mbar_init(&sh.rempty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&sh.tfull[i], 1); mbar_init(&sh.tempty[i], 256); }
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
        if (!mbar_wait(&sh.lempty, item_phase ^ 1u, abort, a.status, ST_WAIT_EMPTY)) { ok = false; break; }
        mbar_arrive_expect_tx(&sh.lfull, (uint32_t)(n_sets * I.nbc) * kBoxBytes);
        for (int set = 0; set < n_sets; ++set) {
          const CUtensorMap* m = a.maps + (set ? I.map_l1 : I.map_l0);
          for (int bc = 0; bc < I.nbc; ++bc)
            tma_load_box(smem_l + (size_t)(set * I.nbc + bc) * kBoxBytes, m, 64 * bc, I.row0, &sh.lfull);
        }
        ++l_loads;
        for (int t = 0; t < I.n_tiles && ok; ++t) {
          const int col0 = (I.tile0 + t) * kApplyNT;
          for (int set = 0; set < n_sets && ok; ++set) {
            const CUtensorMap* m = a.maps + (set ? I.map_r1 : I.map_r0);
            for (int bc = 0; bc < I.nbc; ++bc) {
              if (!mbar_wait(&sh.rempty[rs], rphase ^ 1u, abort, a.status, ST_WAIT_EMPTY)) { ok = false; break; }
              mbar_arrive_expect_tx(&sh.rfull[rs], (uint32_t)kBoxBytes);
              tma_load_box(smem_r + (size_t)rs * kBoxBytes, m, 64 * bc, col0, &sh.rfull[rs]);
              ++r_loads;
              if (++rs == a.n_rstages) { rs = 0; rphase ^= 1u; }
            }
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
        const int ks = I.rp >> 4;     // 16-wide K steps per part
        if (!mbar_wait(&sh.lfull, item_phase, abort, a.status, ST_WAIT_FULL)) break;
        for (int t = 0; t < I.n_tiles && ok; ++t, ++j) {
          const int acc = j & 1;
          const uint32_t acc_phase = (uint32_t)(j >> 1) & 1u;
          if (!mbar_wait(&sh.tempty[acc], acc_phase ^ 1u, abort, a.status, ST_WAIT_TMEM_EMPTY)) { ok = false; break; }
          const uint32_t d = tmem_base + (uint32_t)(acc * kApplyNT);
          uint32_t accumulate = 0;
          // K step k of a [.., 2rp] operand: box k / 4 (16 KB apart), 32 bytes per step inside it
          auto kstep = [](int k) { return (uint32_t)((k >> 2) * (kBoxBytes >> 4) + (k & 3) * 2); };
          for (int set = 0; set < n_sets && ok; ++set) {
            const uint32_t idesc = make_idesc(kApplyNT, false, false, set == 1);
            const uint32_t la = desc_lo(l_base + (uint32_t)(set * I.nbc) * kBoxBytes, 16);
            for (int bc = 0; bc < I.nbc; ++bc) {
              if (!mbar_wait(&sh.rfull[rs], rphase, abort, a.status, ST_WAIT_FULL)) { ok = false; break; }
              tc_fence_after();
              const uint32_t rb = desc_lo(r_base + (uint32_t)rs * kBoxBytes, 16);
              for (int kk = 0; kk < 4; ++kk) {
                const int kb = 4 * bc + kk;            // K step of [R hi | R lo] held by this box
                if (kb >= 2 * ks) break;
                const uint64_t b = desc_join(rb + (uint32_t)(kk * 2), dhi);
                if (kb < ks) {                         // hi * hi, lo * hi
                  mma_bf16(d, desc_join(la + kstep(kb), dhi), b, idesc, accumulate);
                  mma_bf16(d, desc_join(la + kstep(ks + kb), dhi), b, idesc, 1u);
                } else {                               // hi * lo
                  mma_bf16(d, desc_join(la + kstep(kb - ks), dhi), b, idesc, accumulate);
                }
                accumulate = 1;
              }
              mma_commit(&sh.rempty[rs]);
              if (++rs == a.n_rstages) { rs = 0; rphase ^= 1u; }
            }
          }
          if (ok) mma_commit(&sh.tfull[acc]);
        }
        if (ok) mma_commit(&sh.lempty);
        item_phase ^= 1u;
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int e = warp - 2;
    const int wq4 = warp & 3;                             // which 32 accumulator rows this warp may read
    const int half = e >> 2;                              // which 64 columns of the tile
    const uint32_t lane_addr = (uint32_t)(32 * wq4) << 16;
    float* turn = reinterpret_cast<float*>(smem + a.turn_off) + e * kStageFloats;
    const StepScalars sc = a.sc;
    const int rsub = lane >> 2;                           // after the turn: row rsub + 8 i, i = 0..3
    const int csub = 4 * (lane & 3);                      // and four columns starting here
    int j = 0;
    bool ok = true;
    for (int it = blockIdx.x; it < a.n_items && ok; it += gridDim.x) {
      const ApplyItem I = a.items[it];
      const bool grouped = I.v_mode == ADAPM_V_BLOCKMEAN;
      const float lr_s = sc.lr * I.lr_scale;
      int64_t rbase[4];
      bool rok[4];
      float kr[4];   // one denominator per row when v is a group scalar: m^c / (sqrt(v) + eps) becomes a product
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int row = I.row0 + 32 * wq4 + rsub + 8 * i;
        rok[i] = row < I.rows;
        rbase[i] = I.off + (int64_t)row * I.cols;
        const float v_row = (rok[i] && grouped) ? a.state[I.v_off + row / I.v_group_rows] : 0.f;
        kr[i] = sc.inv_bc1 / (sqrtf(v_row * sc.inv_bc2) + sc.eps);
      }
      const int n_pieces = I.n_tiles * 4;                 // pieces of 16 columns this warp handles
      float4 wq[4], wn[4], vq[4], vn[4];     // vq / vn: per-element v, requested with W when v is not a group scalar
      uint2 gq[4], gn[4];
      auto piece_col = [&](int gi) { return (I.tile0 + (gi >> 2)) * kApplyNT + half * 64 + (gi & 3) * 16 + csub; };
      auto request = [&](int gi, float4* w, uint2* g, float4* v) {
        const int col = piece_col(gi);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const bool in = rok[i] && col + 4 <= I.cols;
          w[i] = in ? __ldcg(reinterpret_cast<const float4*>(a.params + rbase[i] + col)) : make_float4(0.f, 0.f, 0.f, 0.f);
          g[i] = in ? __ldcg(reinterpret_cast<const uint2*>(a.grads + rbase[i] + col)) : make_uint2(0u, 0u);
          if (!grouped)
            v[i] = in ? *reinterpret_cast<const float4*>(a.state + I.v_off + (rbase[i] - I.off) + col)
                      : make_float4(0.f, 0.f, 0.f, 0.f);
        }
      };
      request(0, wq, gq, vq);
      for (int gi = 0; gi < n_pieces; ++gi) {
        const int jt = j + (gi >> 2), sub = gi & 3;
        const int acc = jt & 1;
        if (gi + 1 < n_pieces) request(gi + 1, wn, gn, vn);
        if (sub == 0) {
          bool got = true;
          if (lane == 0) got = mbar_wait(&sh.tfull[acc], (uint32_t)(jt >> 1) & 1u, abort, a.status, ST_WAIT_TMEM_FULL);
          got = __shfl_sync(0xffffffffu, got, 0);
          if (!got) { ok = false; break; }
          tc_fence_after();
        }
        float d[16];
        tmem_ld16(tmem_base + lane_addr + (uint32_t)(acc * kApplyNT + half * 64 + sub * 16), d);
        tmem_ld_wait();
        float4* mine = reinterpret_cast<float4*>(turn + lane * kStagePitch);
        mine[0] = make_float4(d[0], d[1], d[2], d[3]);
        mine[1] = make_float4(d[4], d[5], d[6], d[7]);
        mine[2] = make_float4(d[8], d[9], d[10], d[11]);
        mine[3] = make_float4(d[12], d[13], d[14], d[15]);
        __syncwarp();
        const int col = piece_col(gi);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float4 dv = *reinterpret_cast<const float4*>(turn + (rsub + 8 * i) * kStagePitch + csub);
          if (!(rok[i] && col + 4 <= I.cols)) continue;
          const float dd[4] = {dv.x, dv.y, dv.z, dv.w};
          const float gf[4] = {__uint_as_float(gq[i].x << 16), __uint_as_float(gq[i].x & 0xffff0000u),
                               __uint_as_float(gq[i].y << 16), __uint_as_float(gq[i].y & 0xffff0000u)};
          float w[4] = {wq[i].x, wq[i].y, wq[i].z, wq[i].w};
          if (grouped) {
#pragma unroll
            for (int x = 0; x < 4; ++x) {
              float ratio = (sc.cg * gf[x] + sc.c0 * dd[x]) * kr[i];
              ratio = ratio > sc.clip ? sc.clip : (ratio < -sc.clip ? -sc.clip : ratio);
              w[x] = w[x] - lr_s * (ratio + I.wd * w[x]);
            }
          } else {
            float4* vp = reinterpret_cast<float4*>(a.state + I.v_off + (rbase[i] - I.off) + col);
            const float4 vo = vq[i];
            float vv[4] = {vo.x, vo.y, vo.z, vo.w};
#pragma unroll
            for (int x = 0; x < 4; ++x) {
              vv[x] = sc.beta2 * vv[x] + (1.f - sc.beta2) * (gf[x] * gf[x]);
              w[x] = adapm_param_update(w[x], sc.cg * gf[x] + sc.c0 * dd[x], vv[x], sc, lr_s, I.wd);
            }
            *vp = make_float4(vv[0], vv[1], vv[2], vv[3]);
          }
          *reinterpret_cast<float4*>(a.params + rbase[i] + col) = make_float4(w[0], w[1], w[2], w[3]);
        }
        __syncwarp();
        if (sub == 3) {
          tc_fence_before();
          mbar_arrive(&sh.tempty[acc]);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) { wq[i] = wn[i]; gq[i] = gn[i]; vq[i] = vn[i]; }
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
