// Internal declarations shared by the translation units of libadapm.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "adapm.h"

namespace adapm {

// ---------------------------------------------------------------------------------------------
// error plumbing
// ---------------------------------------------------------------------------------------------
void set_cuda_error(cudaError_t e, const char* where);
#define ADAPM_CUDA(call)                                        \
  do {                                                          \
    cudaError_t e__ = (call);                                   \
    if (e__ != cudaSuccess) {                                   \
      ::adapm::set_cuda_error(e__, #call);                      \
      return ADAPM_ECUDA;                                       \
    }                                                           \
  } while (0)

constexpr int64_t kAlignElems = 8;      // block offsets: multiples of 8 elements
constexpr int64_t kStateAlign = 64;     // state sub-buffers: multiples of 64 floats (256 B)

inline int64_t round_up(int64_t x, int64_t a) { return (x + a - 1) / a * a; }

// Which caller buffer an offset is relative to.
enum Base : int32_t { BASE_NONE = -1, BASE_PARAMS = 0, BASE_GRADS = 1, BASE_STATE = 2, BASE_WORK = 3 };

struct Bases {
  void* p[4];             // params (fp32), grads (fp32 | bf16), state (fp32), workspace (bytes; offsets in floats)
  const int32_t* status;  // device status word: a kernel that finds it set writes nothing
  const float* gscale;    // device scalars {s, s^2}: every gradient counts as s g (global norm clipping); null: 1
  uint16_t* shadow;       // bf16 copy of the parameters, written wherever W is written; null: none
};

// ---------------------------------------------------------------------------------------------
// streaming kernel (blocks without momentum and with full momentum)
// ---------------------------------------------------------------------------------------------
constexpr int kTeamChunks = 8;                 // 16-byte gradient chunks a thread keeps in registers
constexpr int kChunkElems = 8;
constexpr int kWarpUnitMax = 32 * kTeamChunks * kChunkElems;    // 2048 elements per warp unit
constexpr int kCtaUnitMax = 256 * kTeamChunks * kChunkElems;    // 16384 elements per CTA unit

enum StreamVMode : int32_t {
  SV_ELEMENT = 0,        // v per element
  SV_GROUP_INLINE = 1,   // one unit == one v group: reduce inside the team
  SV_GROUP_READY = 2     // v of the group was already updated by the reduction kernels
};

struct StreamBlk {
  int64_t off;           // element offset in params / grads
  int64_t m_off;         // float offset of m^f in state, -1 for blocks without momentum
  int64_t v_off;         // float offset of v in state
  int64_t numel;
  int64_t group_elems;   // SV_GROUP_READY: elements per v group
  int32_t unit_elems;    // elements per work unit
  int32_t units_per_group;  // SV_GROUP_READY: units a group is cut into (else 1)
  int64_t n_units;
  int32_t v_mode;        // StreamVMode
  int32_t team;          // 32: one warp per unit (8 units per CTA); 256: one CTA per unit
  int32_t vec_ok;        // units start on 16-byte boundaries
  int32_t pad_;
  float lr_scale, wd;
  int64_t first_cta;     // prefix sum of CTAs
};

// ---------------------------------------------------------------------------------------------
// group sum of squares (v groups too large for one team, and low-rank blocks on the SIMT path)
// ---------------------------------------------------------------------------------------------
struct ReduceJob {
  int64_t g_off;         // element offset in grads
  int64_t group_elems;
  int64_t n_groups;
  int64_t v_off;         // float offset of the group scalars in state
  int64_t part_off;      // float offset of the partial sums in the workspace
  int32_t chunks_per_group;   // chunks of <= 2048 elements
  int32_t pad_;
  int64_t first_unit;    // prefix sum over (group, chunk) pairs
  int64_t first_group;   // prefix sum over groups
};

// ---------------------------------------------------------------------------------------------
// generic batched GEMM on CUDA cores: C = alpha X Y + beta C + c1 Z1 + c2 Z2
// ---------------------------------------------------------------------------------------------
struct GemmProb {
  int64_t x_off, y_off, c_off, z1_off, z2_off;
  int64_t sxi, sxk, syk, syj;     // X(i,k) = X[i*sxi + k*sxk],  Y(k,j) = Y[k*syk + j*syj]
  int32_t M, N, K, ldc;           // C, Z1, Z2: row-major with leading dimension ldc
  int8_t x_base, y_base, c_base, z1_base, z2_base;   // Base; grads operands take the gradient dtype
  int8_t pad_[3];
  float alpha, beta, c1, c2;
  int32_t tiles_n;
  int32_t pad2_;
  int64_t first_tile;
};

// ---------------------------------------------------------------------------------------------
// low-rank apply: m^c = cg g + c0 L0 R0 - c1 L R, then line 9 of Algorithm 1
// ---------------------------------------------------------------------------------------------
struct ApplyBlk {
  int64_t off;                    // params / grads element offset
  int64_t l0_off, r0_off;         // previous factors (state), floats
  int64_t l1_off, r1_off;         // refitted factors, floats
  int64_t v_off;                  // state
  int32_t l1_base, pad0_;         // where the refitted factors live (state when K_eff == 0, else workspace)
  int32_t rows, cols, rank;
  int32_t v_mode;                 // ADAPM_V_ELEMENT | ADAPM_V_BLOCKMEAN (group scalars already updated)
  int32_t v_group_rows;           // rows per group (>= 1)
  int32_t tiles_n;
  float lr_scale, wd;
  int64_t first_tile;
};

// (G + delta I)^-1 of a symmetric r x r matrix, delta = damping * trace(G) / r + floor
struct InverseJob {
  int64_t src_off, dst_off;   // float offsets in the workspace
  int32_t r, pad_;
};

struct InitJob {
  int64_t l_off;        // float offset of L in state
  int64_t block_index;  // keys the random stream
  int32_t rows, rank;
};

struct StepScalars {
  float lr, beta1, beta2, eps, clip;
  float inv_bc1, inv_bc2;         // 1/(1-beta1^t), 1/(1-beta2^t) or 1
  float cg, c0, c1;               // m^c = cg g + c0 P_prev - c1 P
};

// one launch of the static per-step program
enum LaunchKind : int32_t {
  LK_REDUCE_PARTIAL, LK_REDUCE_FINAL, LK_STREAM, LK_GEMM, LK_APPLY_SIMT, LK_COMMIT,
  LK_TC_CONVERT, LK_TC_GRAM, LK_TC_PANEL, LK_TC_APPLY,
  LK_REDUCE_ROWS,       // reduce_final over the row sums of g^2 that the first refit pass left
  LK_GRADNORM,          // global gradient norm and the clip factor
  LK_TC_COPY,           // previous split copy of L -> final set (steps that hold L)
  LK_SPD_INVERSE,       // damped inverses of the r x r Gram matrices (preconditioned passes)
  LK_TC_CONVERT_WORK    // split copy of fp32 arrays that live in the workspace (the transformed factors)
};
// when a launch of the program runs
enum LaunchWhen : int32_t {
  WHEN_ALWAYS = 0,
  WHEN_EVEN, WHEN_ODD   // only in steps of that parity (the factor sets swap roles from step to step)
};
struct Launch {
  LaunchKind kind;
  int64_t table_off;    // byte offset of its descriptor table in the device table blob
  int64_t n_items;      // descriptors
  int64_t grid;         // CTAs
  int64_t aux0 = 0, aux1 = 0, aux2 = 0, aux3 = 0, aux4 = 0, aux5 = 0;
  int32_t when = WHEN_ALWAYS;
  int32_t only_convert = 0;   // 1: only in a step that rebuilds the split copies of the factors
  int32_t phase = 0;          // 0: every step; 1: only steps that refit both factors; 2: only steps that hold L
};

// ---------------------------------------------------------------------------------------------
// kernel launchers (defined in the .cu files)
// ---------------------------------------------------------------------------------------------
// `status` is the device status word: a kernel that finds it set writes nothing (an earlier launch gave up).
int launch_stream(const StreamBlk* d_tab, const int32_t* d_cta_blk, int64_t grid, const Bases& b,
                  const StepScalars& sc, int grad_dtype, cudaStream_t s);
int launch_reduce_partial(const ReduceJob* d_tab, const int32_t* d_cta_job, int64_t n_jobs, int64_t n_units, const void* grads,
                          float* work, int grad_dtype, const int32_t* status, cudaStream_t s);
int launch_reduce_final(const ReduceJob* d_tab, int64_t n_jobs, int64_t n_groups, float* state, const float* work,
                        float beta2, const int32_t* status, const float* gscale, cudaStream_t s);
// global gradient norm: per-chunk sums of g^2 over every block, then {s, s^2} = clip factor into gscale
struct NormRange { int64_t off, numel, first_cta; };
constexpr int kNormChunk = 16384;
int launch_gradnorm(const NormRange* d_tab, const int32_t* d_cta_range, int64_t n_ctas, const void* grads, int grad_dtype,
                    float* partials, float max_norm, int check_finite, float* gscale, int32_t* status, cudaStream_t s);
int launch_gemm(const GemmProb* d_tab, int64_t n_prob, int64_t n_tiles, const Bases& b, int grad_dtype,
                cudaStream_t s);
int launch_apply_simt(const ApplyBlk* d_tab, int64_t n_blk, int64_t n_tiles, const Bases& b, const StepScalars& sc,
                      int grad_dtype, cudaStream_t s);
int launch_spd_inverse(const InverseJob* d_tab, int64_t n_jobs, float* work, float damping, const int32_t* status,
                       cudaStream_t s);
int launch_copy_ranges(const NormRange* d_tab, const int32_t* d_cta_range, int64_t n_ctas, float* dst, const float* src,
                       const int32_t* status, cudaStream_t s);
int launch_meansq_partial(const void* g, int grad_dtype, int64_t n_groups, int64_t group_elems, int chunks_per_group,
                          float* partial, cudaStream_t s);
int launch_meansq_final(const float* partial, int64_t n_groups, int64_t group_elems, int chunks_per_group, float* out,
                        cudaStream_t s);
int launch_init_L0(const InitJob* d_tab, int64_t n_jobs, float* state, uint64_t seed, int draw, cudaStream_t s);

struct TcProgram;   // host side of the tensor-core low-rank path (lowrank_tc.cu)

}  // namespace adapm

// The opaque context.
struct adapm_ctx {
  std::vector<adapm_block> blocks;
  adapm_hparams hp;
  int device = -1;

  // state layout (floats)
  std::vector<int64_t> m_off, l_off, r_off, v_off, v_cnt;
  int64_t state_floats = 0;
  int64_t lr_section_floats = 0;       // L,R of the CUDA-core blocks: the start of the state buffer
  size_t bytes_m = 0, bytes_L = 0, bytes_R = 0, bytes_v = 0;

  // workspace layout (floats)
  int64_t work_floats = 0;
  int64_t ws_lr[2] = {0, 0};           // two copies of the L,R section (ping-pong iterates)
  void* workspace = nullptr;
  size_t workspace_bytes = 0;

  // program
  std::vector<adapm::Launch> program;
  std::vector<unsigned char> h_tables;
  unsigned char* d_tables = nullptr;
  int32_t* d_status = nullptr;
  int64_t init_table_off = 0, n_init_jobs = 0;
  // data-driven L_0: Y = g Omega per low-rank block (one batched GEMM), Omega in a caller buffer laid out by omega_off
  std::vector<int64_t> omega_off;      // float offset of a block's Omega [cols, rank], -1 for other blocks
  int64_t omega_floats = 0;
  int64_t range_table_off = 0, n_range_probs = 0, n_range_tiles = 0;
  int final_lr_buf = -1;               // which workspace copy holds L_t,R_t after the refit (-1: unchanged)
  adapm::TcProgram* tc = nullptr;      // program of the blocks that run on the tensor cores
  int64_t n_tensor_blocks = 0;

  // optional per-launch timing (adapm_set_profiling)
  int profiling = 0, prof_valid = 0;
  std::vector<cudaEvent_t> prof_events;
  std::vector<int32_t> prof_kinds;     // kinds of the launches the last profiled step issued, in order
  int64_t last_step_launches = 0;      // kernels the last adapm_step launched

  float* d_gscale = nullptr;           // device scalars {s, s^2}: the step's clip factor (global norm clipping), or null
  void* shadow = nullptr;              // caller's bf16 copy of the parameters (adapm_set_shadow_params), or null
  int use_gscale = 0;                  // the program starts with the gradient-norm pass
  unsigned char* d_probe = nullptr;    // item table of the expired-wait probe

  size_t step_bytes = 0;
  double step_flops = 0;
};
