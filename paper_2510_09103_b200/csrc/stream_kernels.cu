// Fused streaming update for blocks without momentum and with full momentum, and the block-mean
// reduction of g^2 for second-moment groups that do not fit one team of threads.
//
// Per element the kernel performs, in one pass over HBM (Algorithm 1 lines 7 and 9, Eq. 4):
//   v  <- beta2 v + (1-beta2) g^2            (per element, or once per group with the group mean of g^2)
//   m  <- beta1 m + (1-beta1) g              (full-momentum blocks only; m^c = m, else m^c = g)
//   W  <- W - lr s_b ( clamp( m^c / (sqrt(v)+eps) ) + lambda_b W )
// A work unit (one v group, or a 2048-element chunk) is owned by a team of 32 or 256 threads that
// keeps the unit's gradient in registers, so g is read from memory exactly once even when the
// group mean has to be known before any element can be updated.
#include "adapm_internal.h"
#include "device_math.cuh"

namespace adapm {

namespace {

template <int TEAM>
__device__ __forceinline__ float team_sum(float x, float* smem8) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  if (TEAM == 32) return x;
  const int w = threadIdx.x >> 5;
  __syncthreads();                       // smem8 may still be read from a previous use
  if ((threadIdx.x & 31) == 0) smem8[w] = x;
  __syncthreads();
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) s += smem8[i];   // same order in every thread
  return s;
}

// One work unit.  HAS_M: the block keeps full momentum; HAS_V: v is per element.
template <typename GT, int TEAM, bool HAS_M, bool HAS_V>
__device__ __forceinline__ void run_unit(const StreamBlk& B, int64_t unit, float* __restrict__ params,
                                         const typename GT::elem* __restrict__ grads, float* __restrict__ state,
                                         const StepScalars& sc, float* smem8, float gs, uint16_t* __restrict__ shadow) {
  const int lane = (TEAM == 32) ? (threadIdx.x & 31) : threadIdx.x;

  int64_t ustart, group;
  int ulen;
  if (B.v_mode == SV_GROUP_READY) {
    group = unit / B.units_per_group;
    const int64_t u = unit - group * B.units_per_group;
    const int64_t in_group = u * B.unit_elems;
    ustart = group * B.group_elems + in_group;
    const int64_t rem = B.group_elems - in_group;
    ulen = rem < B.unit_elems ? (int)rem : B.unit_elems;
  } else {
    group = unit;
    ustart = unit * (int64_t)B.unit_elems;
    const int64_t rem = B.numel - ustart;
    ulen = rem < B.unit_elems ? (int)rem : B.unit_elems;
  }
  const typename GT::elem* g = grads + B.off + ustart;
  float* W = params + B.off + ustart;
  float* M = HAS_M ? state + B.m_off + ustart : nullptr;
  float* V = HAS_V ? state + B.v_off + ustart : nullptr;
  const int nchunks = (ulen + kChunkElems - 1) / kChunkElems;
  const bool vec = B.vec_ok != 0;

  // ---- phase 1: gradient into registers, sum of squares --------------------------------------
  typename GT::raw8 graw[kTeamChunks];
  float ss = 0.f;
#pragma unroll
  for (int c = 0; c < kTeamChunks; ++c) {
    const int idx = lane + c * TEAM;
    if (idx < nchunks) {
      const int e0 = idx * kChunkElems;
      if (vec && e0 + kChunkElems <= ulen) {
        graw[c] = GT::load8(g + e0);
      } else {
        graw[c] = GT::load8_guarded(g + e0, ulen - e0);
      }
    }
  }
  if (B.v_mode == SV_GROUP_INLINE) {
#pragma unroll
    for (int c = 0; c < kTeamChunks; ++c) {
      if (lane + c * TEAM < nchunks) {
        float f[8];
        GT::unpack(graw[c], f);
#pragma unroll
        for (int i = 0; i < 8; ++i) ss = fmaf(f[i], f[i], ss);
      }
    }
  }

  // ---- phase 2: momentum, second moment, parameter write ------------------------------------
  // Chunks are taken four at a time: all loads of a batch are issued before its first store, so the
  // memory system sees them together instead of one round trip per chunk.  The first batch is asked
  // for before the group mean is reduced: its W (and m, v) do not depend on the mean, and the round
  // trip of the reduction's shuffles and of the old group scalar then overlaps theirs.
  constexpr int kBatch = ((HAS_M && HAS_V) || sizeof(typename GT::raw8) > 16) ? 2 : 4;
  auto load_batch = [&](int c0, float (*w)[8], float (*m)[8], float (*v)[8]) {
#pragma unroll
    for (int b = 0; b < kBatch; ++b) {
      const int idx = lane + (c0 + b) * TEAM;
      if (idx < nchunks) {
        const int e0 = idx * kChunkElems;
        if (vec && e0 + kChunkElems <= ulen) {
          load8f(W + e0, w[b]);
          if (HAS_M) load8f(M + e0, m[b]);
          if (HAS_V) load8f(V + e0, v[b]);
        } else {
          const int nval = ulen - e0;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const bool ok = i < nval;
            w[b][i] = ok ? W[e0 + i] : 0.f;
            if (HAS_M) m[b][i] = ok ? M[e0 + i] : 0.f;
            if (HAS_V) v[b][i] = ok ? V[e0 + i] : 0.f;
          }
        }
      }
    }
  };
  float w[kBatch][8], m[kBatch][8], v[kBatch][8];
  load_batch(0, w, m, v);

  float v_group = 0.f;
  if (B.v_mode == SV_GROUP_INLINE) {
    // one thread reads the old scalar and writes the new one; everyone else gets it by broadcast
    float v_old = 0.f;
    if (lane == 0) v_old = state[B.v_off + group];
    const float tot = team_sum<TEAM>(ss, smem8);
    if (TEAM == 32) {
      v_old = __shfl_sync(0xffffffffu, v_old, 0);
    } else {
      if (threadIdx.x == 0) smem8[8] = v_old;
      __syncthreads();
      v_old = smem8[8];
    }
    v_group = sc.beta2 * v_old + (1.f - sc.beta2) * ((gs * gs) * (tot / (float)ulen));
    if (lane == 0) state[B.v_off + group] = v_group;
  } else if (B.v_mode == SV_GROUP_READY) {
    v_group = state[B.v_off + group];
  }

  const float lr_s = sc.lr * B.lr_scale;
  const float a1 = 1.f - sc.beta1, a2 = 1.f - sc.beta2;
  // with a group scalar the division m^c / (sqrt(v) + eps) is one multiplication per element
  const float k_ratio = sc.inv_bc1 / (sqrtf(v_group * sc.inv_bc2) + sc.eps);
  // Blocks without momentum and with a group scalar hold only W per chunk: their second batch is requested
  // before the first is worked on (two register sets that swap roles).
  constexpr bool kTwoSets = !HAS_M && !HAS_V && kBatch * 2 == kTeamChunks;
  float w2[kTwoSets ? kBatch : 1][8];
  if (kTwoSets) load_batch(kBatch, w2, m, v);
#pragma unroll
  for (int c0 = 0; c0 < kTeamChunks; c0 += kBatch) {
    if (c0 > 0 && !kTwoSets) load_batch(c0, w, m, v);
    if (c0 > 0 && kTwoSets) {
#pragma unroll
      for (int b = 0; b < kBatch; ++b)
#pragma unroll
        for (int i = 0; i < 8; ++i) w[b][i] = w2[b][i];
    }
#pragma unroll
    for (int b = 0; b < kBatch; ++b) {
      const int idx = lane + (c0 + b) * TEAM;
      if (idx < nchunks) {
        const int e0 = idx * kChunkElems;
        const bool full = vec && e0 + kChunkElems <= ulen;
        float gf[8];
        GT::unpack(graw[c0 + b], gf);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          gf[i] *= gs;                       // the clipped gradient (gs = 1 without global clipping)
          float mc = gf[i];
          if (HAS_M) {
            m[b][i] = sc.beta1 * m[b][i] + a1 * gf[i];
            mc = m[b][i];
          }
          if (HAS_V) {
            v[b][i] = sc.beta2 * v[b][i] + a2 * (gf[i] * gf[i]);
            w[b][i] = adapm_param_update(w[b][i], mc, v[b][i], sc, lr_s, B.wd);
          } else {
            float ratio = mc * k_ratio;
            ratio = ratio > sc.clip ? sc.clip : (ratio < -sc.clip ? -sc.clip : ratio);
            w[b][i] = w[b][i] - lr_s * (ratio + B.wd * w[b][i]);
          }
        }
        if (shadow) {                        // bf16 copy of the new parameters
          uint16_t* sp = shadow + B.off + ustart + e0;
          if (full) {
            *reinterpret_cast<uint4*>(sp) = make_uint4(pack_bf16x2(w[b][0], w[b][1]), pack_bf16x2(w[b][2], w[b][3]),
                                                       pack_bf16x2(w[b][4], w[b][5]), pack_bf16x2(w[b][6], w[b][7]));
          } else {
            const int nval = ulen - e0 < 8 ? ulen - e0 : 8;
            for (int i = 0; i < nval; ++i) sp[i] = (uint16_t)(pack_bf16x2(w[b][i], 0.f) & 0xffffu);
          }
        }
        if (full) {
          store8f(W + e0, w[b]);
          if (HAS_M) store8f(M + e0, m[b]);
          if (HAS_V) store8f(V + e0, v[b]);
        } else {
          const int nval = ulen - e0 < 8 ? ulen - e0 : 8;
          for (int i = 0; i < nval; ++i) {
            W[e0 + i] = w[b][i];
            if (HAS_M) M[e0 + i] = m[b][i];
            if (HAS_V) V[e0 + i] = v[b][i];
          }
        }
      }
    }
  }
}

template <typename GT, int TEAM>
__device__ __forceinline__ void run_unit_any(const StreamBlk& B, int64_t unit, float* __restrict__ params,
                                             const typename GT::elem* __restrict__ grads, float* __restrict__ state,
                                             const StepScalars& sc, float* smem8, float gs,
                                             uint16_t* __restrict__ shadow) {
  const bool has_m = B.m_off >= 0, has_v = B.v_mode == SV_ELEMENT;
  if (has_m) {
    if (has_v) run_unit<GT, TEAM, true, true>(B, unit, params, grads, state, sc, smem8, gs, shadow);
    else run_unit<GT, TEAM, true, false>(B, unit, params, grads, state, sc, smem8, gs, shadow);
  } else {
    if (has_v) run_unit<GT, TEAM, false, true>(B, unit, params, grads, state, sc, smem8, gs, shadow);
    else run_unit<GT, TEAM, false, false>(B, unit, params, grads, state, sc, smem8, gs, shadow);
  }
}

template <typename GT>
__global__ void __launch_bounds__(256, 2) stream_update_kernel(const StreamBlk* __restrict__ tab,
                                                               const int32_t* __restrict__ cta_blk,
                                                               float* __restrict__ params,
                                                               const typename GT::elem* __restrict__ grads,
                                                               float* __restrict__ state, StepScalars sc,
                                                               const int32_t* __restrict__ status,
                                                               const float* __restrict__ gscale,
                                                               uint16_t* __restrict__ shadow) {
  __shared__ StreamBlk sB;
  __shared__ float smem8[12];
  if (threadIdx.x == 0) {
    sB = tab[cta_blk[blockIdx.x]];                       // which block this CTA works on
    if (*status != 0) sB.team = 0;                       // an earlier launch gave up: write nothing
  }
  __syncthreads();
  const int64_t cta_local = (int64_t)blockIdx.x - sB.first_cta;
  const float gs = gscale ? __ldg(gscale) : 1.f;
  if (sB.team == 32) {
    const int64_t unit = cta_local * 8 + (threadIdx.x >> 5);
    if (unit < sB.n_units) run_unit_any<GT, 32>(sB, unit, params, grads, state, sc, smem8, gs, shadow);
  } else if (sB.team == 256) {
    run_unit_any<GT, 256>(sB, cta_local, params, grads, state, sc, smem8, gs, shadow);
  }
}

// ---- group sums of squares ---------------------------------------------------------------------

template <typename GT>
__device__ __forceinline__ float warp_chunk_sumsq(const typename GT::elem* __restrict__ g, int len, bool vec) {
  const int lane = threadIdx.x & 31;
  const int nchunks = (len + kChunkElems - 1) / kChunkElems;
  float ss = 0.f;
#pragma unroll
  for (int c = 0; c < kTeamChunks; ++c) {
    const int idx = lane + c * 32;
    if (idx < nchunks) {
      const int e0 = idx * kChunkElems;
      typename GT::raw8 r = (vec && e0 + kChunkElems <= len) ? GT::load8(g + e0) : GT::load8_guarded(g + e0, len - e0);
      float f[8];
      GT::unpack(r, f);
#pragma unroll
      for (int i = 0; i < 8; ++i) ss = fmaf(f[i], f[i], ss);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  return ss;
}

template <typename GT>
__global__ void __launch_bounds__(256) reduce_partial_kernel(const ReduceJob* __restrict__ tab,
                                                             const int32_t* __restrict__ cta_job, int n_jobs,
                                                             int64_t n_units,
                                                             const typename GT::elem* __restrict__ grads,
                                                             float* __restrict__ work,
                                                             const int32_t* __restrict__ status) {
  const int64_t unit = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (unit >= n_units || *status != 0) return;
  int lo = cta_job[blockIdx.x];                       // job of the CTA's first unit; this warp's is at most 7 units on
  while (lo + 1 < n_jobs && tab[lo + 1].first_unit <= unit) ++lo;
  const ReduceJob J = tab[lo];
  const int64_t u = unit - J.first_unit;
  const int64_t group = u / J.chunks_per_group;
  const int64_t chunk = u - group * J.chunks_per_group;
  const int64_t in_group = chunk * kWarpUnitMax;
  const int64_t rem = J.group_elems - in_group;
  const int len = rem < kWarpUnitMax ? (int)rem : kWarpUnitMax;
  const bool vec = (J.group_elems % kChunkElems) == 0 || J.n_groups == 1;
  const float ss = warp_chunk_sumsq<GT>(grads + J.g_off + group * J.group_elems + in_group, len, vec);
  if ((threadIdx.x & 31) == 0) work[J.part_off + u] = ss;
}

__device__ __forceinline__ float warp_sum_partials(const float* __restrict__ p, int n) {
  const int lane = threadIdx.x & 31;
  float s = 0.f;
  for (int i = lane; i < n; i += 32) s += p[i];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  return s;
}

// One warp per group, or (kLane) one lane per group for jobs whose groups have few partial sums: a lane then
// adds its group's partial sums one after the other.  Either way the order of the additions is fixed.
constexpr int kLaneGroupMax = 64;     // partial sums per group up to which a lane takes a whole group

__global__ void __launch_bounds__(256) reduce_final_kernel(const ReduceJob* __restrict__ tab, int n_jobs,
                                                           int64_t n_groups, float* __restrict__ state,
                                                           const float* __restrict__ work, float beta2,
                                                           const int32_t* __restrict__ status,
                                                           const float* __restrict__ gscale) {
  // groups are taken 32 at a time by a warp; inside the 32, jobs with small groups go lane by lane
  const int64_t g0 = ((int64_t)blockIdx.x * 8 + (threadIdx.x >> 5)) * 32;
  if (g0 >= n_groups || *status != 0) return;
  const int lane = threadIdx.x & 31;
  const float gs2 = gscale ? gscale[1] : 1.f;      // the sums are of the unclipped gradient
  int lo = 0, hi = n_jobs - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (tab[mid].first_group <= g0) lo = mid; else hi = mid - 1;
  }
  const int64_t g_end = g0 + 32 < n_groups ? g0 + 32 : n_groups;
  int64_t g = g0;
  while (g < g_end) {                                // warp-uniform walk over the jobs these 32 groups fall in
    while (lo + 1 < n_jobs && tab[lo + 1].first_group <= g) ++lo;
    const ReduceJob J = tab[lo];
    const int64_t job_end = J.first_group + J.n_groups;
    const int64_t upto = job_end < g_end ? job_end : g_end;
    if (J.chunks_per_group <= kLaneGroupMax) {
      const int64_t mine = g + lane;
      if (mine < upto) {
        const int64_t group = mine - J.first_group;
        const float* p = work + J.part_off + group * J.chunks_per_group;
        float tot = 0.f;
        for (int i = 0; i < J.chunks_per_group; ++i) tot += p[i];
        float* v = state + J.v_off + group;
        *v = beta2 * (*v) + (1.f - beta2) * (gs2 * (tot / (float)J.group_elems));
      }
    } else {
      for (int64_t q = g; q < upto; ++q) {
        const int64_t group = q - J.first_group;
        const float tot = warp_sum_partials(work + J.part_off + group * J.chunks_per_group, J.chunks_per_group);
        if (lane == 0) {
          float* v = state + J.v_off + group;
          *v = beta2 * (*v) + (1.f - beta2) * (gs2 * (tot / (float)J.group_elems));
        }
      }
    }
    g = upto;
  }
}

// stand-alone block mean of g^2 (same two stages, caller's scratch)
template <typename GT>
__global__ void __launch_bounds__(256) meansq_partial_kernel(const typename GT::elem* __restrict__ g,
                                                             int64_t n_groups, int64_t group_elems,
                                                             int chunks_per_group, float* __restrict__ partial) {
  const int64_t unit = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (unit >= n_groups * chunks_per_group) return;
  const int64_t group = unit / chunks_per_group;
  const int64_t chunk = unit - group * chunks_per_group;
  const int64_t in_group = chunk * kWarpUnitMax;
  const int64_t rem = group_elems - in_group;
  const int len = rem < kWarpUnitMax ? (int)rem : kWarpUnitMax;
  const bool vec = (group_elems % kChunkElems) == 0 || n_groups == 1;
  const float ss = warp_chunk_sumsq<GT>(g + group * group_elems + in_group, len, vec);
  if ((threadIdx.x & 31) == 0) partial[unit] = ss;
}

__global__ void __launch_bounds__(256) meansq_final_kernel(const float* __restrict__ partial, int64_t n_groups,
                                                           int64_t group_elems, int chunks_per_group,
                                                           float* __restrict__ out) {
  const int64_t group = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (group >= n_groups) return;
  const float tot = warp_sum_partials(partial + group * chunks_per_group, chunks_per_group);
  if ((threadIdx.x & 31) == 0) out[group] = tot / (float)group_elems;
}

// ---- global gradient norm ---------------------------------------------------------------------------
// Stage 1: one CTA per chunk of up to 16384 elements of one block; every thread adds its elements in a fixed
// order, the warps and the CTA reduce in a fixed order.  Stage 2: one CTA adds the per-chunk sums in double,
// again in a fixed order, and writes s = min(1, c / norm) and s^2.
template <typename GT>
__global__ void __launch_bounds__(256) gradnorm_partial_kernel(const NormRange* __restrict__ tab,
                                                               const int32_t* __restrict__ cta_range,
                                                               const typename GT::elem* __restrict__ grads,
                                                               float* __restrict__ partials,
                                                               const int32_t* __restrict__ status) {
  __shared__ float warp_sums[8];
  if (*status != 0) return;
  const NormRange R = tab[cta_range[blockIdx.x]];
  const int64_t start = ((int64_t)blockIdx.x - R.first_cta) * kNormChunk;
  const int64_t rem = R.numel - start;
  const int len = rem < kNormChunk ? (int)rem : kNormChunk;
  const typename GT::elem* g = grads + R.off + start;
  const int nchunks = (len + kChunkElems - 1) / kChunkElems;
  float ss = 0.f;
  for (int idx = threadIdx.x; idx < nchunks; idx += 256) {
    const int e0 = idx * kChunkElems;
    typename GT::raw8 r = (e0 + kChunkElems <= len) ? GT::load8(g + e0) : GT::load8_guarded(g + e0, len - e0);
    float f[8];
    GT::unpack(r, f);
#pragma unroll
    for (int i = 0; i < 8; ++i) ss = fmaf(f[i], f[i], ss);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if ((threadIdx.x & 31) == 0) warp_sums[threadIdx.x >> 5] = ss;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) t += warp_sums[i];
    partials[blockIdx.x] = t;
  }
}

__global__ void __launch_bounds__(1024) gradnorm_final_kernel(const float* __restrict__ partials, int64_t n, float max_norm,
                                                              int check_finite, float* __restrict__ gscale,
                                                              int32_t* __restrict__ status) {
  __shared__ double sums[1024];
  if (*status != 0) return;
  double t = 0.0;
  for (int64_t i = threadIdx.x; i < n; i += 1024) t += (double)partials[i];
  sums[threadIdx.x] = t;
  __syncthreads();
  for (int o = 512; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) sums[threadIdx.x] += sums[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const double total = sums[0];
    float s = 1.f;
    if (!(total >= 0.0) || total > 3.0e38) {           // NaN or Inf somewhere in the gradient
      if (check_finite) atomicOr(status, 64);          // the rest of the step is skipped and the caller is told
      else s = (float)(total - total);                 // NaN: propagates like any other NaN gradient
    } else if (max_norm > 0.f && total > 0.0) {
      const double norm = sqrt(total);
      if (norm > (double)max_norm) s = (float)((double)max_norm / norm);
    }
    gscale[0] = s;
    gscale[1] = s * s;
  }
}

// dst[off + i] = src[off + i] for the listed ranges only (one CTA per chunk of up to kNormChunk floats): the padding
// between two sub-buffers of the state is never written
__global__ void __launch_bounds__(256) copy_ranges_kernel(const NormRange* __restrict__ tab,
                                                          const int32_t* __restrict__ cta_range, float* __restrict__ dst,
                                                          const float* __restrict__ src,
                                                          const int32_t* __restrict__ status) {
  if (*status != 0) return;
  const NormRange R = tab[cta_range[blockIdx.x]];
  const int64_t start = ((int64_t)blockIdx.x - R.first_cta) * kNormChunk;
  const int64_t rem = R.numel - start;
  const int len = rem < kNormChunk ? (int)rem : kNormChunk;
  const float* s = src + R.off + start;
  float* d = dst + R.off + start;
  const int n4 = len / 4;                       // range offsets are multiples of 64 floats, chunks of 16384
  for (int i = threadIdx.x; i < n4; i += 256)
    reinterpret_cast<float4*>(d)[i] = reinterpret_cast<const float4*>(s)[i];
  for (int i = 4 * n4 + threadIdx.x; i < len; i += 256) d[i] = s[i];
}

}  // namespace

#define ADAPM_LAUNCH_CHECK()                         \
  do {                                               \
    cudaError_t e__ = cudaGetLastError();            \
    if (e__ != cudaSuccess) {                        \
      set_cuda_error(e__, __func__);                 \
      return ADAPM_ECUDA;                            \
    }                                                \
  } while (0)

int launch_stream(const StreamBlk* d_tab, const int32_t* d_cta_blk, int64_t grid, const Bases& b,
                  const StepScalars& sc, int grad_dtype, cudaStream_t s) {
  if (grid <= 0) return ADAPM_OK;
  if (grad_dtype == ADAPM_GRAD_BF16)
    stream_update_kernel<GradBF16><<<(unsigned)grid, 256, 0, s>>>(d_tab, d_cta_blk, (float*)b.p[BASE_PARAMS],
                                                                 (const uint16_t*)b.p[BASE_GRADS],
                                                                 (float*)b.p[BASE_STATE], sc, b.status, b.gscale,
                                                                 b.shadow);
  else
    stream_update_kernel<GradF32><<<(unsigned)grid, 256, 0, s>>>(d_tab, d_cta_blk, (float*)b.p[BASE_PARAMS],
                                                                (const float*)b.p[BASE_GRADS],
                                                                (float*)b.p[BASE_STATE], sc, b.status, b.gscale,
                                                                b.shadow);
  ADAPM_LAUNCH_CHECK();
  return ADAPM_OK;
}

int launch_reduce_partial(const ReduceJob* d_tab, const int32_t* d_cta_job, int64_t n_jobs, int64_t n_units,
                          const void* grads, float* work, int grad_dtype, const int32_t* status, cudaStream_t s) {
  if (n_units <= 0) return ADAPM_OK;
  const unsigned grid = (unsigned)((n_units + 7) / 8);
  if (grad_dtype == ADAPM_GRAD_BF16)
    reduce_partial_kernel<GradBF16><<<grid, 256, 0, s>>>(d_tab, d_cta_job, (int)n_jobs, n_units, (const uint16_t*)grads,
                                                         work, status);
  else
    reduce_partial_kernel<GradF32><<<grid, 256, 0, s>>>(d_tab, d_cta_job, (int)n_jobs, n_units, (const float*)grads, work,
                                                        status);
  ADAPM_LAUNCH_CHECK();
  return ADAPM_OK;
}

int launch_reduce_final(const ReduceJob* d_tab, int64_t n_jobs, int64_t n_groups, float* state, const float* work,
                        float beta2, const int32_t* status, const float* gscale, cudaStream_t s) {
  if (n_groups <= 0) return ADAPM_OK;
  reduce_final_kernel<<<(unsigned)((n_groups + 255) / 256), 256, 0, s>>>(d_tab, (int)n_jobs, n_groups, state, work, beta2,
                                                                        status, gscale);
  ADAPM_LAUNCH_CHECK();
  return ADAPM_OK;
}

int launch_meansq_partial(const void* g, int grad_dtype, int64_t n_groups, int64_t group_elems, int chunks_per_group,
                          float* partial, cudaStream_t s) {
  const int64_t units = n_groups * chunks_per_group;
  if (units <= 0) return ADAPM_OK;
  const unsigned grid = (unsigned)((units + 7) / 8);
  if (grad_dtype == ADAPM_GRAD_BF16)
    meansq_partial_kernel<GradBF16><<<grid, 256, 0, s>>>((const uint16_t*)g, n_groups, group_elems, chunks_per_group,
                                                         partial);
  else
    meansq_partial_kernel<GradF32><<<grid, 256, 0, s>>>((const float*)g, n_groups, group_elems, chunks_per_group,
                                                        partial);
  ADAPM_LAUNCH_CHECK();
  return ADAPM_OK;
}

int launch_meansq_final(const float* partial, int64_t n_groups, int64_t group_elems, int chunks_per_group, float* out,
                        cudaStream_t s) {
  if (n_groups <= 0) return ADAPM_OK;
  meansq_final_kernel<<<(unsigned)((n_groups + 7) / 8), 256, 0, s>>>(partial, n_groups, group_elems, chunks_per_group,
                                                                    out);
  ADAPM_LAUNCH_CHECK();
  return ADAPM_OK;
}

int launch_gradnorm(const NormRange* d_tab, const int32_t* d_cta_range, int64_t n_ctas, const void* grads, int grad_dtype,
                    float* partials, float max_norm, int check_finite, float* gscale, int32_t* status, cudaStream_t s) {
  if (n_ctas <= 0) return ADAPM_OK;
  if (grad_dtype == ADAPM_GRAD_BF16)
    gradnorm_partial_kernel<GradBF16><<<(unsigned)n_ctas, 256, 0, s>>>(d_tab, d_cta_range, (const uint16_t*)grads, partials,
                                                                      status);
  else
    gradnorm_partial_kernel<GradF32><<<(unsigned)n_ctas, 256, 0, s>>>(d_tab, d_cta_range, (const float*)grads, partials,
                                                                     status);
  ADAPM_LAUNCH_CHECK();
  gradnorm_final_kernel<<<1, 1024, 0, s>>>(partials, n_ctas, max_norm, check_finite, gscale, status);
  ADAPM_LAUNCH_CHECK();
  return ADAPM_OK;
}

int launch_copy_ranges(const NormRange* d_tab, const int32_t* d_cta_range, int64_t n_ctas, float* dst, const float* src,
                       const int32_t* status, cudaStream_t s) {
  if (n_ctas <= 0) return ADAPM_OK;
  copy_ranges_kernel<<<(unsigned)n_ctas, 256, 0, s>>>(d_tab, d_cta_range, dst, src, status);
  ADAPM_LAUNCH_CHECK();
  return ADAPM_OK;
}

}  // namespace adapm
