// Tensor-core "apply" kernel of the low-rank path: rebuilds the corrected momentum tile by tile and
// writes the parameters (Algorithm 1 lines 4, 6, 8 and 9 combined):
//
//   m^c = cg g + c0 L0 R0 - c1 L R          (= g + c (P_{t-1} - P_t) with the correction on)
//   W  <- W - lr s_b ( clamp( m^c / (sqrt(v) + eps) ) + lambda_b W )
//
// An item is a 128-row panel of one block times a run of column tiles.  The split-bf16 rows of L0
// and L of the panel stay in shared memory for the whole run; per column tile the matching rows of
// R0^T and R^T are loaded and the products hi*hi + hi*lo + lo*hi of both factor pairs are
// accumulated into one accumulator (the new pair with a negated A operand), so the accumulator
// holds D = L0 R0 - L R.  Eight epilogue warps then stream g and W through registers.
// The m x n matrices m_t, r_t and m^c are never stored.
#pragma once

#include <cuda.h>

#include "adapm_internal.h"
#include "device_math.cuh"
#include "tc_common.cuh"

namespace adapm {
namespace tc {

constexpr int kApplyThreads = 320;

struct ApplyItem {
  int64_t off;               // element offset of the block in params / grads
  int64_t v_off;             // float offset of v in state
  int32_t rows, cols, r, rp;
  int32_t map_l0, map_l1, map_r0, map_r1;   // split factors: [rows, 2rp] and [cols, 2rp]
  int32_t row0;              // first row of the panel
  int32_t tile0, n_tiles;    // column tiles [tile0, tile0 + n_tiles) of width nt
  int32_t nt;                // 64 or 128
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
  int32_t r_region_off;      // byte offset of the R tile region inside the dynamic shared memory
};

struct __align__(8) ApplyShared {
  uint64_t lfull, lempty, rfull, rempty, tfull[2], tempty[2];
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
    mbar_init(&sh.lfull, 1); mbar_init(&sh.lempty, 1); mbar_init(&sh.rfull, 1); mbar_init(&sh.rempty, 1);
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
      uint32_t item_phase = 0, tile_phase = 0;
      bool ok = true;
      bool l_pending = false, r_pending = false;
      for (int it = blockIdx.x; it < a.n_items && ok; it += gridDim.x) {
        const ApplyItem I = a.items[it];
        const int rb_n = I.nt / 64;
        if (!mbar_wait(&sh.lempty, item_phase ^ 1u, abort, a.status, ST_WAIT_EMPTY)) { ok = false; break; }
        mbar_arrive_expect_tx(&sh.lfull, (uint32_t)(n_sets * I.nbc * 2) * kBoxBytes);
        for (int set = 0; set < n_sets; ++set) {
          const CUtensorMap* m = a.maps + (set ? I.map_l1 : I.map_l0);
          for (int bc = 0; bc < I.nbc; ++bc)
            for (int rb = 0; rb < 2; ++rb)
              tma_load_box(smem_l + (size_t)((set * I.nbc + bc) * 2 + rb) * kBoxBytes, m, 64 * bc, I.row0 + 64 * rb,
                           &sh.lfull);
        }
        l_pending = true;
        for (int t = 0; t < I.n_tiles; ++t) {
          if (!mbar_wait(&sh.rempty, tile_phase ^ 1u, abort, a.status, ST_WAIT_EMPTY)) { ok = false; break; }
          const int col0 = (I.tile0 + t) * I.nt;
          mbar_arrive_expect_tx(&sh.rfull, (uint32_t)(n_sets * I.nbc * rb_n) * kBoxBytes);
          for (int set = 0; set < n_sets; ++set) {
            const CUtensorMap* m = a.maps + (set ? I.map_r1 : I.map_r0);
            for (int bc = 0; bc < I.nbc; ++bc)
              for (int rb = 0; rb < rb_n; ++rb)
                tma_load_box(smem_r + (size_t)((set * I.nbc + bc) * rb_n + rb) * kBoxBytes, m, 64 * bc,
                             col0 + 64 * rb, &sh.rfull);
          }
          r_pending = true;
          tile_phase ^= 1u;
        }
        item_phase ^= 1u;
      }
      if (!ok) {   // let the copies already issued land before the CTA exits
        if (l_pending)
          for (uint32_t spin = 0; spin < kSpinLimit && !mbar_try_wait(&sh.lfull, item_phase ^ 1u) &&
                                  !mbar_try_wait(&sh.lfull, item_phase); ++spin) __nanosleep(64);
        if (r_pending)
          for (uint32_t spin = 0; spin < kSpinLimit && !mbar_try_wait(&sh.rfull, tile_phase ^ 1u) &&
                                  !mbar_try_wait(&sh.rfull, tile_phase); ++spin) __nanosleep(64);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t item_phase = 0, tile_phase = 0;
      int j = 0;   // running tile count of this CTA
      bool ok = true;
      const uint32_t l_base = smem_u32(smem_l), r_base = smem_u32(smem_r);
      for (int it = blockIdx.x; it < a.n_items && ok; it += gridDim.x) {
        const ApplyItem I = a.items[it];
        const int rb_n = I.nt / 64;
        const int ks = I.rp / 16;     // 16-wide K steps per part
        if (!mbar_wait(&sh.lfull, item_phase, abort, a.status, ST_WAIT_FULL)) break;
        for (int t = 0; t < I.n_tiles; ++t, ++j) {
          const int acc = j & 1;
          const uint32_t acc_phase = (uint32_t)(j >> 1) & 1u;
          if (!mbar_wait(&sh.rfull, tile_phase, abort, a.status, ST_WAIT_FULL)) { ok = false; break; }
          if (!mbar_wait(&sh.tempty[acc], acc_phase ^ 1u, abort, a.status, ST_WAIT_TMEM_EMPTY)) { ok = false; break; }
          tc_fence_after();
          const uint32_t d = tmem_base + (uint32_t)(acc * I.nt);
          uint32_t accumulate = 0;
          for (int set = 0; set < n_sets; ++set) {
            const uint32_t idesc = make_idesc(I.nt, false, false, set == 1);
            for (int pair = 0; pair < 3; ++pair) {
              const int pa = pair == 2 ? 1 : 0, pb = pair == 1 ? 1 : 0;   // hi*hi, hi*lo, lo*hi
              for (int s = 0; s < ks; ++s) {
                const int ka = pa * ks + s, kb = pb * ks + s;
                const uint64_t da = desc_k_major(l_base + (uint32_t)((set * I.nbc + (ka >> 2)) * 2) * kBoxBytes, ka & 3);
                const uint64_t db =
                    desc_k_major(r_base + (uint32_t)((set * I.nbc + (kb >> 2)) * rb_n) * kBoxBytes, kb & 3);
                mma_bf16(d, da, db, idesc, accumulate);
                accumulate = 1;
              }
            }
          }
          mma_commit(&sh.rempty);
          mma_commit(&sh.tfull[acc]);
          tile_phase ^= 1u;
        }
        if (ok) mma_commit(&sh.lempty);
        item_phase ^= 1u;
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int e = warp - 2;
    const int q = 32 * (warp & 3) + lane;                 // accumulator row of this thread
    const int half = e >> 2;                              // which half of the tile's columns
    const uint32_t lane_addr = (uint32_t)(32 * (warp & 3)) << 16;
    const StepScalars sc = a.sc;
    int j = 0;
    bool ok = true;
    for (int it = blockIdx.x; it < a.n_items && ok; it += gridDim.x) {
      const ApplyItem I = a.items[it];
      const int row = I.row0 + q;
      const bool row_ok = row < I.rows;
      const int hw = I.nt / 2;                            // columns per thread per tile: 32 or 64
      const float lr_s = sc.lr * I.lr_scale;
      float v_row = 0.f;
      const bool grouped = I.v_mode == ADAPM_V_BLOCKMEAN;
      if (row_ok && grouped) v_row = a.state[I.v_off + row / I.v_group_rows];
      // one denominator per row when v is a group scalar: m^c / (sqrt(v) + eps) becomes a multiplication
      const float k_ratio = sc.inv_bc1 / (sqrtf(v_row * sc.inv_bc2) + sc.eps);
      const int64_t row_base = I.off + (int64_t)row * I.cols;
      for (int t = 0; t < I.n_tiles; ++t, ++j) {
        const int acc = j & 1;
        const uint32_t acc_phase = (uint32_t)(j >> 1) & 1u;
        const int cb = (I.tile0 + t) * I.nt + half * hw;
        const uint32_t t0 = tmem_base + lane_addr + (uint32_t)(acc * I.nt + half * hw);
        bool waited = false;
        for (int c0 = 0; c0 < hw; c0 += 32) {
          // gradient and parameters of 32 columns, requested before the accumulator is needed
          uint4 gq[4];
          float4 wq[8];
          const int col = cb + c0;
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const bool in = row_ok && col + 8 * u + 8 <= I.cols;
            gq[u] = in ? __ldg(reinterpret_cast<const uint4*>(a.grads + row_base + col + 8 * u)) : make_uint4(0, 0, 0, 0);
            wq[2 * u] = in ? *reinterpret_cast<const float4*>(a.params + row_base + col + 8 * u) : make_float4(0, 0, 0, 0);
            wq[2 * u + 1] =
                in ? *reinterpret_cast<const float4*>(a.params + row_base + col + 8 * u + 4) : make_float4(0, 0, 0, 0);
          }
          if (!waited) {
            const bool got = mbar_wait(&sh.tfull[acc], acc_phase, abort, a.status, ST_WAIT_TMEM_FULL);
            if (!__all_sync(0xffffffffu, got)) { ok = false; break; }
            tc_fence_after();
            waited = true;
          }
          float d[32];
          tmem_ld16(t0 + (uint32_t)c0, d);
          tmem_ld16(t0 + (uint32_t)(c0 + 16), d + 16);
          tmem_ld_wait();
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            if (!(row_ok && col + 8 * u + 8 <= I.cols)) continue;
            float gf[8];
            GradBF16::unpack(gq[u], gf);
            float w[8] = {wq[2 * u].x, wq[2 * u].y, wq[2 * u].z, wq[2 * u].w,
                          wq[2 * u + 1].x, wq[2 * u + 1].y, wq[2 * u + 1].z, wq[2 * u + 1].w};
            float vv[8];
            float* vp = nullptr;
            if (I.v_mode == ADAPM_V_ELEMENT) {
              vp = a.state + I.v_off + (int64_t)row * I.cols + col + 8 * u;
              load8f(vp, vv);
            }
#pragma unroll
            for (int x = 0; x < 8; ++x) {
              const float g = gf[x];
              const float mc = sc.cg * g + sc.c0 * d[8 * u + x];
              if (grouped) {
                float ratio = mc * k_ratio;
                ratio = ratio > sc.clip ? sc.clip : (ratio < -sc.clip ? -sc.clip : ratio);
                w[x] = w[x] - lr_s * (ratio + I.wd * w[x]);
              } else {
                const float v = sc.beta2 * vv[x] + (1.f - sc.beta2) * (g * g);
                vv[x] = v;
                w[x] = adapm_param_update(w[x], mc, v, sc, lr_s, I.wd);
              }
            }
            if (vp) store8f(vp, vv);
            store8f(a.params + row_base + col + 8 * u, w);
          }
        }
        if (!ok) break;
        tc_fence_before();
        mbar_arrive(&sh.tempty[acc]);
      }
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
