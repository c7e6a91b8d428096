// CUDA-core (FFMA) kernels of the low-rank path: a batched strided GEMM that carries every product
// of Algorithm 2, the fused "apply" kernel that rebuilds m^c = cg g + c0 L0 R0 - c1 L R tile by tile
// and writes the parameters, and the L_0 initialiser.  This path is exact fp32 and handles every
// shape and gradient dtype; the tensor-core path replaces it where its layout rules are met.
#include "adapm_internal.h"
#include "device_math.cuh"

namespace adapm {

namespace {

constexpr int TM = 64, TN = 64, TK = 16;

template <bool BF16G>
__device__ __forceinline__ float load_operand(const void* base, bool is_grad, int64_t idx) {
  if (is_grad) {
    if (BF16G) return bf16_bits_to_float(static_cast<const uint16_t*>(base)[idx]);
    return static_cast<const float*>(base)[idx];
  }
  return static_cast<const float*>(base)[idx];
}

// acc[4][4] += X(i0.., k) Y(k, j0..) over k in [0, K); thread (ty, tx) owns rows ty*4.., cols tx*4..
template <bool BF16G>
__device__ __forceinline__ void tile_mainloop(float (&acc)[4][4], const void* X, bool x_grad, int64_t sxi,
                                              int64_t sxk, const void* Y, bool y_grad, int64_t syk, int64_t syj,
                                              int M, int N, int K, int i0, int j0, float (*Xs)[TM + 4],
                                              float (*Ys)[TN + 4]) {
  const int t = threadIdx.x;
  const int ty = t >> 4, tx = t & 15;
  // where this thread's four elements of each operand tile sit (fixed for the whole K loop)
  int xi[4], xk[4], yj[4], yk[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    if (sxk == 1) { xk[q] = t & 15; xi[q] = (t >> 4) + 16 * q; } else { xi[q] = t & 63; xk[q] = (t >> 6) + 4 * q; }
    if (syj == 1) { yj[q] = t & 63; yk[q] = (t >> 6) + 4 * q; } else { yk[q] = t & 15; yj[q] = (t >> 4) + 16 * q; }
  }
  // The next tile's elements are asked for before the present tile is multiplied: their round trip to memory
  // runs under the 256 FMAs per thread of a tile instead of between two tiles.
  float xr[4], yr[4];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int i = i0 + xi[q], k = k0 + xk[q];
      xr[q] = (i < M && k < K) ? load_operand<BF16G>(X, x_grad, (int64_t)i * sxi + (int64_t)k * sxk) : 0.f;
      const int j = j0 + yj[q], k2 = k0 + yk[q];
      yr[q] = (j < N && k2 < K) ? load_operand<BF16G>(Y, y_grad, (int64_t)k2 * syk + (int64_t)j * syj) : 0.f;
    }
  };
  if (K > 0) fetch(0);
  for (int k0 = 0; k0 < K; k0 += TK) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      Xs[xk[q]][xi[q]] = xr[q];
      Ys[yk[q]][yj[q]] = yr[q];
    }
    __syncthreads();
    if (k0 + TK < K) fetch(k0 + TK);
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      const float4 a = *reinterpret_cast<const float4*>(&Xs[kk][ty * 4]);
      const float4 b = *reinterpret_cast<const float4*>(&Ys[kk][tx * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w};
      const float bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[r][c] = fmaf(av[r], bv[c], acc[r][c]);
    }
    __syncthreads();
  }
}

template <typename T>
__device__ __forceinline__ const T& find_by_first_tile(const T* tab, int n, int64_t me) {
  int lo = 0, hi = n - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (tab[mid].first_tile <= me) lo = mid; else hi = mid - 1;
  }
  return tab[lo];
}

template <bool BF16G>
__global__ void __launch_bounds__(256, 3) gemm_kernel(const GemmProb* __restrict__ tab, int n_prob, Bases b) {
  __shared__ __align__(16) float Xs[TK][TM + 4];
  __shared__ __align__(16) float Ys[TK][TN + 4];
  __shared__ GemmProb sP;
  __shared__ int skip;
  if (threadIdx.x == 0) {
    sP = find_by_first_tile(tab, n_prob, (int64_t)blockIdx.x);
    skip = *b.status != 0;
  }
  __syncthreads();
  if (skip) return;
  const GemmProb& P = sP;
  const int64_t tile = (int64_t)blockIdx.x - P.first_tile;
  const int i0 = (int)(tile / P.tiles_n) * TM, j0 = (int)(tile % P.tiles_n) * TN;

  const size_t xsz = (P.x_base == BASE_GRADS && BF16G) ? 2 : 4, ysz = (P.y_base == BASE_GRADS && BF16G) ? 2 : 4;
  const void* X = static_cast<const char*>(b.p[P.x_base]) + (size_t)P.x_off * xsz;
  const void* Y = static_cast<const char*>(b.p[P.y_base]) + (size_t)P.y_off * ysz;
  float acc[4][4] = {};
  tile_mainloop<BF16G>(acc, X, P.x_base == BASE_GRADS, P.sxi, P.sxk, Y, P.y_base == BASE_GRADS, P.syk, P.syj, P.M,
                       P.N, P.K, i0, j0, Xs, Ys);

  float* C = static_cast<float*>(b.p[P.c_base]) + P.c_off;
  const float* Z1 = P.z1_base >= 0 ? static_cast<const float*>(b.p[P.z1_base]) + P.z1_off : nullptr;
  const float* Z2 = P.z2_base >= 0 ? static_cast<const float*>(b.p[P.z2_base]) + P.z2_off : nullptr;
  const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
  // a product with the gradient as an operand is a product with the clipped gradient
  const float gprod = (b.gscale && (P.x_base == BASE_GRADS || P.y_base == BASE_GRADS)) ? __ldg(b.gscale) : 1.f;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int i = i0 + ty * 4 + r;
    if (i >= P.M) continue;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const int j = j0 + tx * 4 + c;
      if (j >= P.N) continue;
      const int64_t o = (int64_t)i * P.ldc + j;
      float x = (P.alpha * gprod) * acc[r][c];
      if (P.beta != 0.f) x += P.beta * C[o];
      if (Z1) x += P.c1 * Z1[o];
      if (Z2) x += P.c2 * Z2[o];
      C[o] = x;
    }
  }
}

template <bool BF16G>
__global__ void __launch_bounds__(256) apply_simt_kernel(const ApplyBlk* __restrict__ tab, int n_blk, Bases b,
                                                         StepScalars sc) {
  __shared__ __align__(16) float Xs[TK][TM + 4];
  __shared__ __align__(16) float Ys[TK][TN + 4];
  __shared__ ApplyBlk sA;
  __shared__ int skip;
  if (threadIdx.x == 0) {
    sA = find_by_first_tile(tab, n_blk, (int64_t)blockIdx.x);
    skip = *b.status != 0;
  }
  __syncthreads();
  if (skip) return;
  const ApplyBlk& A = sA;
  const float gs = b.gscale ? __ldg(b.gscale) : 1.f;
  uint16_t* shadow = b.shadow ? b.shadow + A.off : nullptr;
  const int64_t tile = (int64_t)blockIdx.x - A.first_tile;
  const int i0 = (int)(tile / A.tiles_n) * TM, j0 = (int)(tile % A.tiles_n) * TN;
  const int m = A.rows, n = A.cols, r = A.rank;

  float* state = static_cast<float*>(b.p[BASE_STATE]);
  const float* L0 = state + A.l0_off;
  const float* R0 = state + A.r0_off;
  const float* L1 = static_cast<const float*>(b.p[A.l1_base]) + A.l1_off;
  const float* R1 = static_cast<const float*>(b.p[A.l1_base]) + A.r1_off;

  float p0[4][4] = {}, p1[4][4] = {};
  tile_mainloop<BF16G>(p0, L0, false, r, 1, R0, false, n, 1, m, n, r, i0, j0, Xs, Ys);   // P_{t-1} tile
  tile_mainloop<BF16G>(p1, L1, false, r, 1, R1, false, n, 1, m, n, r, i0, j0, Xs, Ys);   // P_t tile

  float* W = static_cast<float*>(b.p[BASE_PARAMS]) + A.off;
  const void* G = static_cast<const char*>(b.p[BASE_GRADS]) + (size_t)A.off * (BF16G ? 2 : 4);
  float* V = state + A.v_off;
  const float lr_s = sc.lr * A.lr_scale;
  const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
#pragma unroll
  for (int rr = 0; rr < 4; ++rr) {
    const int i = i0 + ty * 4 + rr;
    if (i >= m) continue;
    float v_row = 0.f;
    if (A.v_mode == ADAPM_V_BLOCKMEAN) v_row = V[i / A.v_group_rows];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const int j = j0 + tx * 4 + c;
      if (j >= n) continue;
      const int64_t o = (int64_t)i * n + j;
      const float g = gs * load_operand<BF16G>(G, true, o);
      const float mc = sc.cg * g + sc.c0 * p0[rr][c] - sc.c1 * p1[rr][c];
      float v = v_row;
      if (A.v_mode == ADAPM_V_ELEMENT) {
        v = sc.beta2 * V[o] + (1.f - sc.beta2) * (g * g);
        V[o] = v;
      }
      const float w_new = adapm_param_update(W[o], mc, v, sc, lr_s, A.wd);
      W[o] = w_new;
      if (shadow) shadow[o] = (uint16_t)(pack_bf16x2(w_new, 0.f) & 0xffffu);
    }
  }
}

// ---- L_0: Gaussian draws, then modified Gram-Schmidt, one CTA per block ------------------------

__device__ __forceinline__ uint64_t mix64(uint64_t z) {
  z += 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

__device__ __forceinline__ float gaussian_from_counter(uint64_t seed, uint64_t block, uint64_t idx) {
  const uint64_t h = mix64(mix64(seed ^ (block * 0xD1342543DE82EF95ull)) + idx);
  const float u1 = ((uint32_t)(h >> 40) + 1.0f) * (1.0f / 16777217.0f);   // (0, 1)
  const float u2 = (uint32_t)(h & 0xFFFFFFu) * (1.0f / 16777216.0f);       // [0, 1)
  return sqrtf(-2.f * logf(u1)) * cosf(6.283185307179586f * u2);
}

__device__ __forceinline__ float block_sum_1024(float x, float* red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = x;
  __syncthreads();
  float s = 0.f;
  const int nw = blockDim.x >> 5;
  for (int i = 0; i < nw; ++i) s += red[i];
  return s;
}

// (G + delta I)^-1 by Gauss-Jordan elimination without pivoting (the matrix is symmetric positive definite), one
// CTA per matrix, the matrix in global memory, the pivot row and column of a step in shared memory.
constexpr int kInverseMaxRank = 4096;
constexpr float kPrecondFloor = 1e-30f;

__global__ void __launch_bounds__(1024) spd_inverse_kernel(const InverseJob* __restrict__ tab, float* __restrict__ work,
                                                           float damping, const int32_t* __restrict__ status) {
  extern __shared__ float piv[];         // [0, r): column k before the step; [r, 2r): row k after its scaling
  __shared__ float red[32];
  __shared__ int skip;
  if (threadIdx.x == 0) skip = *status != 0;
  __syncthreads();
  if (skip) return;
  const InverseJob J = tab[blockIdx.x];
  const int r = J.r;
  const float* __restrict__ G = work + J.src_off;
  float* __restrict__ S = work + J.dst_off;
  float tr = 0.f;
  for (int i = threadIdx.x; i < r; i += blockDim.x) tr += G[(int64_t)i * r + i];
  tr = block_sum_1024(tr, red);
  const float delta = damping * tr / (float)r + kPrecondFloor;
  const int64_t total = (int64_t)r * r;
  for (int64_t e = threadIdx.x; e < total; e += blockDim.x) {
    const int i = (int)(e / r), j = (int)(e % r);
    S[e] = G[e] + (i == j ? delta : 0.f);
  }
  __syncthreads();
  float* colk = piv;
  float* rowk = piv + r;
  for (int k = 0; k < r; ++k) {
    for (int i = threadIdx.x; i < r; i += blockDim.x) colk[i] = S[(int64_t)i * r + k];
    __syncthreads();
    const float inv_p = 1.f / colk[k];
    for (int j = threadIdx.x; j < r; j += blockDim.x) {
      const float x = (j == k ? 1.f : S[(int64_t)k * r + j]) * inv_p;
      rowk[j] = x;
      S[(int64_t)k * r + j] = x;
    }
    __syncthreads();
    for (int64_t e = threadIdx.x; e < total; e += blockDim.x) {
      const int i = (int)(e / r), j = (int)(e % r);
      if (i == k) continue;
      S[e] = (j == k ? 0.f : S[e]) - colk[i] * rowk[j];
    }
    __syncthreads();
  }
}

// Modified Gram-Schmidt over the columns of L, in order, one CTA per block.  draw = 1: the columns are Gaussian
// draws first (keyed by seed, block, element).  draw = 0: L already holds the matrix to orthonormalise (g Omega of
// the data-driven start); a column that keeps less than kRangeDrop of its squared length becomes zero.
constexpr float kRangeDrop = 1e-8f;

__global__ void __launch_bounds__(1024) init_L0_kernel(const InitJob* __restrict__ tab, float* __restrict__ state,
                                                       uint64_t seed, int draw) {
  __shared__ float red[32];
  const InitJob J = tab[blockIdx.x];
  float* __restrict__ L = state + J.l_off;
  const int rows = J.rows, rank = J.rank;
  const uint64_t block = (uint64_t)J.block_index;
  const int64_t total = (int64_t)rows * rank;
  if (draw)
    for (int64_t e = threadIdx.x; e < total; e += blockDim.x) L[e] = gaussian_from_counter(seed, block, (uint64_t)e);
  __syncthreads();
  for (int j = 0; j < rank; ++j) {
    float n0 = 0.f;
    if (!draw) {
      for (int row = threadIdx.x; row < rows; row += blockDim.x) {
        const float x = L[(int64_t)row * rank + j];
        n0 += x * x;
      }
      n0 = block_sum_1024(n0, red);
    }
    for (int i = 0; i < j; ++i) {
      float d = 0.f;
      for (int row = threadIdx.x; row < rows; row += blockDim.x) d += L[(int64_t)row * rank + i] * L[(int64_t)row * rank + j];
      d = block_sum_1024(d, red);
      for (int row = threadIdx.x; row < rows; row += blockDim.x) L[(int64_t)row * rank + j] -= d * L[(int64_t)row * rank + i];
    }
    float nn = 0.f;
    for (int row = threadIdx.x; row < rows; row += blockDim.x) {
      const float x = L[(int64_t)row * rank + j];
      nn += x * x;
    }
    nn = block_sum_1024(nn, red);
    const float inv = (draw || (n0 > 0.f && nn > kRangeDrop * n0)) ? rsqrtf(nn) : 0.f;
    for (int row = threadIdx.x; row < rows; row += blockDim.x) L[(int64_t)row * rank + j] *= inv;
    __syncthreads();
  }
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

int launch_gemm(const GemmProb* d_tab, int64_t n_prob, int64_t n_tiles, const Bases& b, int grad_dtype,
                cudaStream_t s) {
  if (n_tiles <= 0) return ADAPM_OK;
  if (grad_dtype == ADAPM_GRAD_BF16)
    gemm_kernel<true><<<(unsigned)n_tiles, 256, 0, s>>>(d_tab, (int)n_prob, b);
  else
    gemm_kernel<false><<<(unsigned)n_tiles, 256, 0, s>>>(d_tab, (int)n_prob, b);
  ADAPM_LAUNCH_CHECK();
  return ADAPM_OK;
}

int launch_apply_simt(const ApplyBlk* d_tab, int64_t n_blk, int64_t n_tiles, const Bases& b, const StepScalars& sc,
                      int grad_dtype, cudaStream_t s) {
  if (n_tiles <= 0) return ADAPM_OK;
  if (grad_dtype == ADAPM_GRAD_BF16)
    apply_simt_kernel<true><<<(unsigned)n_tiles, 256, 0, s>>>(d_tab, (int)n_blk, b, sc);
  else
    apply_simt_kernel<false><<<(unsigned)n_tiles, 256, 0, s>>>(d_tab, (int)n_blk, b, sc);
  ADAPM_LAUNCH_CHECK();
  return ADAPM_OK;
}

int launch_spd_inverse(const InverseJob* d_tab, int64_t n_jobs, float* work, float damping, const int32_t* status,
                       cudaStream_t s) {
  if (n_jobs <= 0) return ADAPM_OK;
  spd_inverse_kernel<<<(unsigned)n_jobs, 1024, 2 * kInverseMaxRank * sizeof(float), s>>>(d_tab, work, damping, status);
  ADAPM_LAUNCH_CHECK();
  return ADAPM_OK;
}

int launch_init_L0(const InitJob* d_tab, int64_t n_jobs, float* state, uint64_t seed, int draw, cudaStream_t s) {
  if (n_jobs <= 0) return ADAPM_OK;
  init_L0_kernel<<<(unsigned)n_jobs, 1024, 0, s>>>(d_tab, state, seed, draw);
  ADAPM_LAUNCH_CHECK();
  return ADAPM_OK;
}

}  // namespace adapm
