/*
 * adapm.h - C ABI of the B200 AdaPM optimizer-step library.
 *
 * One call, adapm_step, performs the loop body of the paper's Algorithm 1 ("Low Rank Update with
 * Correction") for every parameter block of a model on one GPU:
 *   - blocks without momentum (embeddings, attention output; Section 4.1 item 1):  m^c = g
 *   - blocks with full momentum (value blocks; Section 4.1 item 3, Eq. 4):         m^c = m^f
 *   - blocks with low-rank momentum (query, key, MLP; Section 4.1 item 2):
 *       m_t = (1-b1) g + b1 L R;  (L,R) <- K gradient-descent passes of Algorithm 2 on ||L R - m_t||^2;
 *       r_t = L R - m_t (Eq. 2);  m^c = m_t - b1 r_t / (1-b1) (Eq. 3)
 *   - second-order statistic v (Algorithm 1 line 7), per element or one scalar per row group
 *     (the Adam-mini combination of Section 5.1.3: the group average of Adam's statistic)
 *   - W <- W - lr * s_b * ( clamp( m^c / (sqrt(v) + eps), -clip, clip ) + lambda_b W )   (line 9)
 *
 * Conventions
 *   - All matrices are row-major [rows, cols] = [m, n] = [out_features, in_features].
 *   - `params`, `grads`, `state` and the workspace are DEVICE pointers owned by the caller.
 *     params: fp32.  grads: fp32 or bf16 (hparams.grad_dtype), same element offsets as params.
 *     state: fp32, adapm_state_bytes() long, laid out as adapm_state_layout() reports.
 *   - Block offsets are in elements and must be multiples of 8; all device pointers must be
 *     256-byte aligned.
 *   - Every function returns 0 on success or a negative ADAPM_E* code; nothing throws, aborts or
 *     traps.  Invalid descriptors are rejected by adapm_create, never by a kernel.
 *   - adapm_step is asynchronous on `stream`, allocates nothing and never synchronises.  One context
 *     is used from one stream at a time.  The first step that sees a new combination of params /
 *     grads / state / workspace pointers describes the buffers to the TMA unit on the host (a few
 *     hundred microseconds) and copies that description from pageable memory: make that step
 *     outside any stream capture.  Four combinations are remembered.
 *   - Every wait inside a kernel is bounded.  If one runs out (a GPU shared with other work that
 *     keeps this library's CTAs from running together for about a second), the kernel stops, sets a
 *     bit in the device status word, and every later kernel of this context returns without writing
 *     until adapm_get_status has been called.  adapm_get_status then returns ADAPM_EDEVICE: the
 *     factors of some low-rank blocks are a mix of two iterates and the step is incomplete, so
 *     restore params and state from the last checkpoint before stepping again.
 *   - There is no CPU fallback: without a CUDA device every device call returns ADAPM_ECUDA.
 */
#ifndef ADAPM_H_
#define ADAPM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct adapm_ctx adapm_ctx;   /* opaque: host plan + small device descriptor tables */
typedef void* adapm_stream;           /* a cudaStream_t (CUstream); NULL = the default stream */

enum { ADAPM_MOM_NONE = 0, ADAPM_MOM_FULL = 1, ADAPM_MOM_LOWRANK = 2 };
enum { ADAPM_V_ELEMENT = 0, ADAPM_V_BLOCKMEAN = 1 };
enum { ADAPM_GRAD_F32 = 0, ADAPM_GRAD_BF16 = 1 };
enum { ADAPM_PATH_AUTO = 0, ADAPM_PATH_SIMT = 1, ADAPM_PATH_TENSOR = 2 };
enum { ADAPM_STATE_M = 0, ADAPM_STATE_L = 1, ADAPM_STATE_R = 2, ADAPM_STATE_V = 3 };
/* adapm_hparams.flags */
enum {
  ADAPM_FLAG_NO_PANEL_TEAMS = 1,     /* hand the refit's panel items out longest-first: no CTA waits for another
                                        (for callers who share the GPU with long-running kernels)            */
  ADAPM_FLAG_FORCE_PANEL_TEAMS = 2,  /* team schedule even for sets with few blocks (small profiling cases)  */
  ADAPM_FLAG_NO_SUMSQ_FOLD = 4,      /* block-mean v of tensor-path blocks from a pass of its own over g     */
  ADAPM_FLAG_CHECK_FINITE = 8        /* a NaN or Inf anywhere in the gradients: the step writes nothing and
                                        adapm_get_status reports bit 64 (costs one more pass over g)        */
};

/* Tensor roles for the default planner (Section 4.1 names the first six kinds). */
enum {
  ADAPM_ROLE_EMBED = 0, ADAPM_ROLE_Q = 1, ADAPM_ROLE_K = 2, ADAPM_ROLE_V = 3, ADAPM_ROLE_QKV_FUSED = 4,
  ADAPM_ROLE_ATTN_OUT = 5, ADAPM_ROLE_MLP = 6, ADAPM_ROLE_LM_HEAD = 7, ADAPM_ROLE_VECTOR = 8,
  ADAPM_ROLE_OTHER = 9
};

enum {
  ADAPM_OK = 0,
  ADAPM_EINVAL = -1,        /* null pointer, bad enum, bad size                                  */
  ADAPM_EALIGN = -2,        /* offset not a multiple of 8 elements / pointer not 256-B aligned   */
  ADAPM_ERANGE = -3,        /* rank, group or index out of range; output array too small         */
  ADAPM_ECUDA = -4,         /* a CUDA call failed (see adapm_last_cuda_error)                    */
  ADAPM_ENOWORKSPACE = -5,  /* adapm_step before adapm_set_workspace, or workspace too small     */
  ADAPM_EUNSUPPORTED = -6,  /* requested kernel path cannot handle this shape or dtype            */
  ADAPM_EDEVICE = -7        /* a kernel reported a bounded wait that ran out (adapm_get_status)  */
};

typedef struct {
  int32_t role;            /* ADAPM_ROLE_*                                                        */
  int32_t heads;           /* attention heads of Q / K / fused QKV tensors, else 0                */
  int64_t rows, cols;      /* m, n; 1-D tensors: rows = 1                                         */
} adapm_tensor;

typedef struct {
  int64_t offset;          /* element offset of the block in params and grads; multiple of 8      */
  int32_t rows, cols;      /* m, n                                                                */
  int32_t mom_mode;        /* ADAPM_MOM_*                                                         */
  int32_t rank;            /* 1..min(m,n) for LOWRANK, else 0                                     */
  int32_t v_mode;          /* ADAPM_V_*                                                           */
  int32_t v_group_rows;    /* BLOCKMEAN: consecutive rows per group (divides rows); 0 = one group */
  float   lr_scale;        /* s_b: 1, or 0.75 for blocks without momentum (Section 5.1)           */
  float   weight_decay;    /* lambda_b (Algorithm 1 line 9); 0 for 1-D tensors                    */
} adapm_block;

typedef struct {
  float   lr, beta1, beta2, eps;
  float   clip;            /* elementwise bound of line 9 (1 in the paper); +inf disables          */
  int32_t inner_iters;     /* K of Algorithm 2 (5 in Appendix B); 0 freezes the factors            */
  float   inner_lr_scale;  /* multiplies eta_k = 0.5 (1 + cos(pi k / K)); 1 = as printed           */
  int32_t grad_dtype;      /* ADAPM_GRAD_*                                                         */
  int32_t adam_debias;     /* 0 = Algorithm 1 as printed; 1 = divide by 1-beta^t (AdamW check)    */
  int32_t correction;      /* 1 = Eq. 3 on; 0 = ablation, m^c := m_t                               */
  int32_t lowrank_path;    /* ADAPM_PATH_*: which kernels run Algorithm 2's contractions           */
  uint64_t seed;           /* seeds L_0 in adapm_state_init                                        */
  uint32_t flags;          /* ADAPM_FLAG_*; 0 = defaults                                           */
  float   max_grad_norm;   /* global gradient clipping (Section 5.1: threshold 1.0): every gradient is
                              multiplied by min(1, c / ||g||_2), the norm over all blocks; 0 or +inf = off */
  int32_t refresh_period;  /* T of Section 5.1 ("update frequency"; the paper sets 100 and does not define
                              it).  Reading: both factors are refitted by Algorithm 2 at steps 1, T+1,
                              2T+1, ...; in between L is held and only R moves (the R half of Algorithm 2).
                              0 or 1 = Algorithm 1 as printed, every step                          */
  int32_t tune_panels;     /* tensor path: 128-row panels per refit item (1..3); 0 = automatic     */
  int32_t tune_stage_k;    /* tensor path: K per shared-memory stage (64 or 128); 0 = automatic    */
  int32_t inner_precond;   /* 0 = Algorithm 2 as printed.  1 = preconditioned passes (a variant, not in
                              the paper: scaled gradient descent): dl/dL is multiplied from the right
                              by (R R^T + d_R I)^-1 and dl/dR from the left by (L^T L + d_L I)^-1, with
                              d = precond_damping * trace / r + 1e-30; warm start, schedule and the
                              simultaneous update are Algorithm 2's.  On the tensor path the inverses
                              and the transformed factors L (L^T L + d I)^-1 and (R R^T + d I)^-1 R come
                              from CUDA-core kernels before each pass's tensor launches              */
  float   precond_damping; /* >= 0; used when inner_precond = 1                                    */
} adapm_hparams;

/* Library version (major*100 + minor). */
int adapm_version(void);

/* Text for an ADAPM_E* code; never NULL. */
const char* adapm_strerror(int code);

/* Text of the last CUDA error this thread's calls saw ("" if none). */
const char* adapm_last_cuda_error(void);

/*
 * Default block partition (Section 4.1; rank r = max(1, floor(rank_pct * min(m,n) / 100)) with
 * rank_pct = 5 in Section 5.1, or rank_override if > 0; lr_scale 0.75 without momentum).
 * Host only, integer arithmetic only.  Tensors are packed in the given order, each starting at a
 * multiple of 8 elements; a fused [3d, d] QKV tensor becomes three row-range blocks (Q, K, V).
 * 1-D tensors get full momentum, no weight decay and a single v group.
 *   out/out_capacity: caller's array; *n_out receives the number of blocks (also when out == NULL,
 *   to size the array); *total_elems receives the flat buffer length in elements.
 * v_mode: ADAPM_V_ELEMENT or ADAPM_V_BLOCKMEAN (one group per head for Q/K, per row otherwise).
 */
int adapm_plan_default(const adapm_tensor* tensors, int64_t n_tensors, int32_t rank_pct,
                       int32_t rank_override, int32_t v_mode, float weight_decay,
                       adapm_block* out, int64_t out_capacity, int64_t* n_out, int64_t* total_elems);

/*
 * Validate the partition, fix the state and workspace layouts and upload the descriptor tables to
 * the current CUDA device.  `blocks` is copied.  Blocks must not overlap.
 */
int adapm_create(const adapm_block* blocks, int64_t n_blocks, const adapm_hparams* hp, adapm_ctx** out);
void adapm_destroy(adapm_ctx* ctx);

/* Bytes of persistent optimizer state the caller must allocate (momentum, factors, v). */
size_t adapm_state_bytes(const adapm_ctx* ctx);
/* Unpadded byte counts per kind of state (any pointer may be NULL). */
int adapm_state_breakdown(const adapm_ctx* ctx, size_t* full_m, size_t* L, size_t* R, size_t* v);
/* Where block `block` keeps ADAPM_STATE_{M,L,R,V}: offset and count in floats (count 0 if absent).
 * L is [rows, rank] and R is [rank, cols], both row-major and dense. */
int adapm_state_layout(const adapm_ctx* ctx, int64_t block, int which, int64_t* offset, int64_t* count);

/* Transient device memory one step needs (factor iterates, A = g R^T, B = L^T g, partial sums). */
size_t adapm_workspace_bytes(const adapm_ctx* ctx);
int adapm_set_workspace(adapm_ctx* ctx, void* dev_ptr, size_t bytes);

/*
 * Zero the state and give every low-rank block its L_0: orthonormal columns (Gaussian draws from a
 * counter-based generator keyed by (seed, block), then Gram-Schmidt), R_0 = 0.  The paper's
 * L_0 = R_0 = 0 (Algorithm 1 line 1) is a stationary point of Algorithm 2 and would never move.
 */
int adapm_state_init(adapm_ctx* ctx, void* state, adapm_stream stream);

/*
 * Data-driven start (a variant; the paper gives none): zero the state and give every low-rank block
 * L_0 = the columns of g_1 Omega orthonormalised in order by Gram-Schmidt (the randomized range finder),
 * so that L_0 spans what the first gradient spans; R_0 = 0.  A column that keeps less than 1e-8 of its
 * squared length (g_1 has rank below r) becomes zero and the block runs at a lower rank.
 *   grads: device, the first step's gradients, same layout and dtype as for adapm_step (16-B aligned);
 *   omega: device, fp32, adapm_init_omega_floats() floats, 16-B aligned, owned by the caller and only
 *          read: block b's Omega is [cols, rank] row-major at the offset adapm_init_omega_layout
 *          returns (count 0 for blocks without low-rank momentum).  The caller draws it (standard
 *          normal entries): the library draws nothing here.
 * Asynchronous on `stream`.  Errors: ADAPM_EINVAL (null pointers), ADAPM_EALIGN, ADAPM_ECUDA.
 */
int64_t adapm_init_omega_floats(const adapm_ctx* ctx);
int adapm_init_omega_layout(const adapm_ctx* ctx, int64_t block, int64_t* offset, int64_t* count);
int adapm_state_init_from_grads(adapm_ctx* ctx, void* state, const void* grads, const float* omega,
                                adapm_stream stream);

/* Learning rate eta_t of the next steps (Algorithm 1 takes a schedule; the caller owns it). */
int adapm_set_lr(adapm_ctx* ctx, float lr);

/*
 * One optimizer step over all blocks (Algorithm 1, loop body); t is the 1-based step count.
 * The tensor-core path keeps bf16 copies of the factors L, R in the workspace from one step to the
 * next.  It rebuilds them from the state buffer when t is not the successor of the previous call's
 * t, when the state or workspace pointer changed, after adapm_state_init and after
 * adapm_state_changed; a caller who writes L or R in the state buffer between two consecutive steps
 * (importing a checkpoint into the same buffer) must call adapm_state_changed.
 */
int adapm_step(adapm_ctx* ctx, void* params, const void* grads, void* state, int64_t t, adapm_stream stream);
int adapm_state_changed(adapm_ctx* ctx);

/*
 * bf16 copy of the parameters (the weights a mixed-precision forward pass reads): every kernel that
 * writes W also writes bf16(W), rounded to nearest even, at the same element offset of this buffer.
 * bf16_dev_ptr: device, as many bf16 elements as params has floats, 256-B aligned; NULL turns it off.
 * (Not part of Algorithm 1; saves the separate cast pass a training loop would run after the step.)
 */
int adapm_set_shadow_params(adapm_ctx* ctx, void* bf16_dev_ptr);

/* Algorithmic HBM bytes of one step (every operand read once, every result written once). */
size_t adapm_step_bytes(const adapm_ctx* ctx);
/* Algorithmic flops of the low-rank contractions of one step: (4 K_eff + 4) m n r per block. */
double adapm_step_flops(const adapm_ctx* ctx);
/* Kernels adapm_step launched in its last call (before the first call: in a steady-state step). */
int64_t adapm_launch_count(const adapm_ctx* ctx);

/*
 * Measurement aid: with profiling on, adapm_step records a CUDA event on `stream` before its first
 * and after each of its kernels, and wraps each launch in an NVTX range named after its kind.  adapm_get_launch_times waits for the last step's events and
 * returns each kernel's duration in milliseconds and its kind (see adapm_launch_kind_name);
 * with ms == kinds == NULL it only reports the number of launches.
 */
int adapm_set_profiling(adapm_ctx* ctx, int32_t on);
int adapm_get_launch_times(adapm_ctx* ctx, float* ms, int32_t* kinds, int64_t capacity, int64_t* n_out);
const char* adapm_launch_kind_name(int32_t kind);

/* Synchronise `stream`, read the device status word into *status (0 = fine) and clear it.
 * Bits: 1, 2 a shared-memory stage, 4, 8 an accumulator, 16 a parameter tile, 32 a team of CTAs was waited
 * for too long; 64 a gradient was not finite and ADAPM_FLAG_CHECK_FINITE skipped the step (params and state
 * are untouched: step again with good gradients).  Non-zero: returns ADAPM_EDEVICE (see the conventions above). */
int adapm_get_status(adapm_ctx* ctx, adapm_stream stream, int32_t* status);

/*
 * Diagnostic (the paper has no counterpart): launches one CTA of the refit engine whose only work item
 * waits for a team counter that nothing advances, with the wait limit cut to about a millisecond.
 * The kernel must give up, set bit 32 of the status word and return; afterwards adapm_get_status
 * reports ADAPM_EDEVICE once and the context keeps working.  Exercises the give-up path without
 * faulting or hanging anything.
 */
int adapm_selftest_expired_wait(adapm_ctx* ctx, adapm_stream stream);

/*
 * Stand-alone block-mean of g^2 (the reduction behind ADAPM_V_BLOCKMEAN; Adam-mini combination):
 *   out[i] = mean over group i of g^2, groups = consecutive runs of `group_elems` elements of g.
 * g: device, n_groups * group_elems elements of `grad_dtype`; out: device, n_groups floats;
 * scratch: device, at least adapm_group_meansq_scratch_bytes(...) bytes, 256-B aligned.
 */
size_t adapm_group_meansq_scratch_bytes(int64_t n_groups, int64_t group_elems);
int adapm_group_meansq(const void* g, int32_t grad_dtype, int64_t n_groups, int64_t group_elems,
                       float* out, void* scratch, size_t scratch_bytes, adapm_stream stream);

/*
 * adapm_group_meansq without any device allocation (the paper has no counterpart; this is a
 * packaging variant of the call above for callers that must not, or cannot, call cudaMalloc:
 * code running inside a host application whose memory manager owns the whole GPU, plug-ins
 * that are forbidden to allocate in their callback, and loops that cannot afford the implicit
 * device synchronisation an allocation or free may cause).
 *
 * Same arguments and result as adapm_group_meansq, minus the scratch: the partial sums go to a
 * fixed array of ADAPM_STATIC_SCRATCH_FLOATS floats (1 MiB) that is part of the library image;
 * every GPU that loads the library keeps that array until the process exits.
 *   - Limit: n_groups * ceil(group_elems / 2048) <= ADAPM_STATIC_SCRATCH_FLOATS, else ADAPM_ERANGE
 *     (adapm_last_cuda_error() then says so); larger inputs need adapm_group_meansq.
 *   - The call itself allocates and frees nothing.  Its first call on each device looks up the
 *     array's device address (one cudaGetSymbolAddress, with that device current): make that first
 *     call before starting any stream capture.  `stream` must belong to the current device.
 *   - All calls on a device share the one array.  Calls whose kernels may overlap on the GPU
 *     (different streams without an ordering between them) race on it: order them on one stream
 *     or with events.  Nothing has to be cleared between calls: each call overwrites the part of
 *     the array it then reads.
 */
#define ADAPM_STATIC_SCRATCH_FLOATS (1 << 18)
int adapm_group_meansq_static(const void* g, int32_t grad_dtype, int64_t n_groups, int64_t group_elems,
                              float* out, adapm_stream stream);

#ifdef __cplusplus
}
#endif
#endif /* ADAPM_H_ */
