// Tensor-core (tcgen05) low-rank path: the per-step program of Algorithm 2's refit and of the
// corrected update for every low-rank block whose layout the TMA engine can address
// (bf16 gradients, cols a multiple of 8).
//
// Per block the workspace holds three split-bf16 copies ("sets") of the factors, [L hi | L lo]
// (rows x 2 half) and [R^T hi | R^T lo] (cols x 2 half): X and Y side by side in one array of row
// pitch 4 half, Z in an array of its own.  At an even step X holds the factors of step t-1, the
// refit passes write Z, Y, Z, Y, ... so that the last pass ends in Y, and the apply kernel reads
// [X | Y] as one operand; at the next step Y is "previous" and the last pass ends in X.  Nothing is
// converted between steps; the fp32 factors in the state are turned into a split copy only when they
// were written from outside (the first step, adapm_state_changed, a step number that is not the
// successor of the last one).
//
// Per step:
//   (convert  when needed: zero the workspace arrays, (L, R) fp32 -> X)
//   K_eff times:  gram    four r x r products of the current iterate (tensor cores) -> Gs[0..3]
//                         (each stored transposed and twice, one copy under the other: the layout the engine's
//                         N side reads against the [hi | lo] columns of a factor)
//                 panel   row panels update L, column panels update R (tensor cores); fp32 factors
//                         are updated in place in the state, their split copies go to the next set.
//                         The row panels of the first pass also add up g^2 per row (block-mean v).
//   apply     m^c and the parameter write from the previous and the final set
// rp = rank rounded up to 16; padded columns are kept at zero by every writer.
#include <algorithm>
#include <cmath>
#include <cstring>

#include "adapm_internal.h"
#include "tc_apply.cuh"
#include "tc_engine.cuh"
#include "tc_host.h"

namespace adapm {

void set_error_text(const char* text);   // ctx.cu

namespace {

// tensor maps of one block
enum {
  MAP_G = 0,        // g, boxes of 64 x 128 (A operand with K along x)
  MAP_GT = 1,       // g, boxes of 64 x stage_k (A operand with K along y)
  MAP_LC = 2,       // + set: [L hi | L lo] as a matrix, boxes of 64 x 128
  MAP_LCT = 5,      // + set: the same, boxes of 64 x stage_k
  MAP_LCN = 8,      // + set: the same as 64-column chunks (N side)
  MAP_RTC = 11, MAP_RTCT = 14, MAP_RTCN = 17,   // the same three views of [R^T hi | R^T lo]
  MAP_GS = 20,      // + which: Gram operands as chunks
  MAP_W = 24, MAP_G32 = 25, MAP_V = 26,          // W, g, v in quarter-tile boxes (apply)
  MAP_LCAT = 27, MAP_RCAT = 28,                  // X and Y side by side as one matrix (apply)
  MAP_SH = 29,                                   // the bf16 copy of W, boxes like g's (apply; zero without a shadow)
  MAP_LCN_T = 30, MAP_RTCN_T = 31,               // N side of the transformed factors L S_L and (S_R R)^T (preconditioned passes)
  kMapsPerBlock = 32
};

struct ConvertJob {
  int64_t f32_off;          // float offset of the factor in state
  int64_t own_stride, k_stride;
  int64_t dst_off;          // bf16 element offset in the workspace
  int32_t owners, r, rp, half;
  int32_t dst_ld;           // row pitch of the destination, in elements
  int32_t pad_;
  int64_t first_owner;      // prefix sum of owners
};

// fp32 factor -> [owners, 2 half] split bf16 with row pitch dst_ld (hi columns from 0, lo columns from half;
// columns >= r are zero)
__global__ void __launch_bounds__(256) tc_convert_kernel(const ConvertJob* __restrict__ jobs, int n_jobs,
                                                         int64_t total_owners, const float* __restrict__ state,
                                                         uint16_t* __restrict__ work, const int32_t* __restrict__ status) {
  if (*status != 0) return;
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= total_owners) return;
  int lo = 0, hi = n_jobs - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (jobs[mid].first_owner <= gid) lo = mid; else hi = mid - 1;
  }
  const ConvertJob J = jobs[lo];
  const int64_t owner = gid - J.first_owner;
  const float* f = state + J.f32_off + J.own_stride * owner;
  uint16_t* dst = work + J.dst_off + (int64_t)J.dst_ld * owner;
  for (int p = 0; p < J.rp; p += 16) {
    uint32_t h[8], l[8];
#pragma unroll
    for (int e = 0; e < 16; e += 2) {
      const int k = p + e;
      const float x0 = k < J.r ? f[J.k_stride * k] : 0.f;
      const float x1 = k + 1 < J.r ? f[J.k_stride * (k + 1)] : 0.f;
      tc::split_bf16x2(x0, x1, h[e >> 1], l[e >> 1]);
    }
    uint4* dh = reinterpret_cast<uint4*>(dst + p);
    uint4* dl = reinterpret_cast<uint4*>(dst + J.half + p);
    dh[0] = make_uint4(h[0], h[1], h[2], h[3]);
    dh[1] = make_uint4(h[4], h[5], h[6], h[7]);
    dl[0] = make_uint4(l[0], l[1], l[2], l[3]);
    dl[1] = make_uint4(l[4], l[5], l[6], l[7]);
  }
}

struct CopyJob {
  int64_t src_off, dst_off;   // bf16 element offsets in the workspace
  int32_t rows, width;        // width in elements (a multiple of 8)
  int32_t src_ld, dst_ld;
  int64_t first_row;          // prefix sum of rows
};

// rows of `width` bf16 from one split array to another (a step that holds L carries its split copy over)
__global__ void __launch_bounds__(256) tc_copy_kernel(const CopyJob* __restrict__ jobs, int n_jobs, int64_t total_rows,
                                                      uint16_t* __restrict__ work, const int32_t* __restrict__ status) {
  if (*status != 0) return;
  const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= total_rows) return;
  int lo = 0, hi = n_jobs - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (jobs[mid].first_row <= row) lo = mid; else hi = mid - 1;
  }
  const CopyJob J = jobs[lo];
  const int64_t r = row - J.first_row;
  const uint4* src = reinterpret_cast<const uint4*>(work + J.src_off + r * J.src_ld);
  uint4* dst = reinterpret_cast<uint4*>(work + J.dst_off + r * J.dst_ld);
  for (int i = threadIdx.x & 31; i < J.width / 8; i += 32) dst[i] = src[i];
}

}  // namespace

// Host side of the tensor path, owned by the context.
struct TcBlock {
  int64_t id;                      // index into ctx->blocks
  int32_t rp, half;
  int64_t lc[3], rtc[3], gs[4];    // bf16 element offsets in the workspace; sets 0 = X, 1 = Y, 2 = Z
  int32_t ld[3];                   // row pitch of set s of lc / rtc, in elements
  int64_t rowsum;                  // float offset of the row sums of g^2 in the workspace, or -1
  // preconditioned passes: split copies of L S_L and (S_R R)^T (pitch 2 half), and in floats the Gram matrices
  // R R^T, L^T L (gf, gf + r^2), their damped inverses (sf, sf + r^2) and the fp32 products L S_L, S_R R
  int64_t lct = 0, rtct = 0, gf = 0, sf = 0, ltf = 0, rtf = 0;
};

struct MapSet {                     // tensor maps for one combination of caller buffers
  const void* key[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};   // params, grads, state, workspace, shadow
  CUtensorMap* d_maps = nullptr;
  std::vector<CUtensorMap> h_maps;
  uint64_t last_use = 0;
};

struct TcProgram {
  std::vector<TcBlock> blk;
  int64_t n_convert_owners = 0;
  int smem_engine = 0, smem_apply = 0;
  int nb_max = 1, stage_k = 128, rp_max = 16, half_max = 16;
  int64_t work_begin = 0, work_end = 0;   // the tensor path's part of the workspace, in floats
  // shared-memory plan of an engine launch whose segments have up to n_a A operands
  struct EngineConfig { int a_bytes, stage_bytes, n_stages, smem; };
  EngineConfig engine_config(int n_a) const {
    EngineConfig e;
    e.a_bytes = n_a * 256 * stage_k;
    e.stage_bytes = e.a_bytes + stage_k * 128 * nb_max;
    e.n_stages = std::min(8, (224 * 1024) / e.stage_bytes);
    e.smem = std::max(e.n_stages, 1) * e.stage_bytes + 1024;
    return e;
  }
  int apply_r_region = 0, apply_r_stages = 3, apply_w_region = 0, apply_bufs = 2, apply_buf_bytes = 0;
  int apply_s_w_region = 0, apply_s_bufs = 2, smem_apply_s = 0;   // the streaming form of the apply kernel
  int n_sms = 148;
  bool rotate = false;             // sets swap roles from step to step (there is at least one refit pass)
  int32_t* d_team_counters = nullptr;   // pacing counters of the panel launches (see schedule_panels)
  int n_teams = 0;
  MapSet maps[4];
  uint64_t use_clock = 0;
  const CUtensorMap* cur_maps = nullptr;
  // what the split copies in the workspace correspond to
  bool split_valid = false;
  int64_t last_t = 0;
  const void* last_state = nullptr;
  const void* last_work = nullptr;
};

bool tensor_path_block_ok(const adapm_hparams& hp, const adapm_block& b) {
  if (hp.lowrank_path == ADAPM_PATH_SIMT) return false;
  if (hp.grad_dtype != ADAPM_GRAD_BF16) return false;
  if (b.mom_mode != ADAPM_MOM_LOWRANK) return false;
  if (b.cols % 8 != 0 || b.rank > 256) return false;   // 2 rp accumulator columns per panel, 512 in all
  return tc::encode_tiled_fn() != nullptr;
}

void destroy_tensor_program(adapm_ctx* c) {
  TcProgram* p = c->tc;
  if (!p) return;
  for (MapSet& m : p->maps)
    if (m.d_maps) cudaFree(m.d_maps);
  if (p->d_team_counters) cudaFree(p->d_team_counters);
  delete p;
  c->tc = nullptr;
}

void tensor_state_changed(adapm_ctx* c) {
  if (c->tc) c->tc->split_valid = false;
}

// ---------------------------------------------------------------------------------------------------
// program construction
// ---------------------------------------------------------------------------------------------------
namespace {

int round16(int x) { return (x + 15) / 16 * 16; }
int round64(int x) { return (x + 63) / 64 * 64; }

template <typename T>
int64_t append_items(std::vector<unsigned char>& blob, const std::vector<T>& tab) {
  const size_t off = (blob.size() + 15) / 16 * 16;
  blob.resize(off + tab.size() * sizeof(T));
  if (!tab.empty()) std::memcpy(blob.data() + off, tab.data(), tab.size() * sizeof(T));
  return (int64_t)off;
}

struct Geo {
  int stage_k, nb;     // K of a stage; 64-column chunks of every B box of the block
};

// One segment.  A: 2-D map `map_a`, operand p at (ax + dax p, ay + day p), K along x (a_mode 0) or along y
// (a_mode 1).  B: chunked map `map_b`, K rows from 0.  rp2 = 2 rp decides between one MMA of N = 2 rp and two
// of N = rp (the second from the chunk where the lo part starts).
tc::Seg make_seg(const Geo& g, int map_a, int ax, int ay, int a_mode, int n_a, int dax, int day, int map_b, int rp,
                 int half, int k, int d0, int d_step, int first) {
  tc::Seg s;
  std::memset(&s, 0, sizeof(s));
  s.map_a = map_a; s.map_b = map_b;
  for (int p = 0; p < n_a; ++p) { s.ax[p] = ax + dax * p; s.ay[p] = ay + day * p; s.d_col[p] = (int16_t)(d0 + d_step * p); }
  s.a_mode = (int16_t)a_mode; s.n_a = (int16_t)n_a; s.k = round16(k); s.first = (int16_t)first;
  if (2 * rp <= 256) { s.n = (int16_t)(2 * rp); s.n_mma = 1; }
  else { s.n = (int16_t)rp; s.n_mma = 2; s.b2_chunk = (int16_t)(half / 64); s.d_part = (int16_t)rp; }
  s.tx_bytes = (uint32_t)(n_a * 256 * g.stage_k + g.stage_k * 128 * g.nb);
  return s;
}

int item_cost(const tc::Item& it, int stage_k) {
  int c = 0;
  for (int s = 0; s < it.n_seg; ++s) c += (it.seg[s].k + stage_k - 1) / stage_k;
  return c + 2 * 128 / stage_k;   // the epilogue
}

// Hands the items to `grid` CTAs, longest first, each to the CTA with the least work so far.  Afterwards CTA c owns
// v[begin[c] .. begin[c + 1]).
void schedule_items(std::vector<tc::Item>& v, int grid, std::vector<int32_t>& begin, int stage_k) {
  for (auto& it : v) it.cost = item_cost(it, stage_k);
  std::stable_sort(v.begin(), v.end(), [](const tc::Item& a, const tc::Item& b) { return a.cost > b.cost; });
  std::vector<std::vector<tc::Item>> per(grid);
  std::vector<int64_t> load(grid, 0);
  for (const tc::Item& it : v) {
    int best = 0;
    for (int c = 1; c < grid; ++c)
      if (load[c] < load[best]) best = c;
    per[best].push_back(it);
    load[best] += it.cost;
  }
  v.clear();
  begin.assign(grid + 1, 0);
  for (int c = 0; c < grid; ++c) {
    v.insert(v.end(), per[c].begin(), per[c].end());
    begin[c + 1] = (int32_t)v.size();
  }
}

// The panel items of one block: v[first .. first + n_row) work on row panels (K runs over the columns of g),
// the next n_col on column panels (K runs over the rows).
struct BlockSpan {
  size_t first, n_row, n_col;
};

// Team schedule for a panel launch.  The row panels and the column panels of a block each read all of g, and at
// full size the second read finds nothing in L2 unless it follows the first closely.  So a team of CTAs takes one
// block at a time: every item of the kind with the longer K loop gets a CTA of its own, the items of the other kind
// are dealt in order to as many further CTAs as keep pace with them (item j of the short kind covers the j-th
// slice of the long kind's K range, so both kinds sweep g together), and no CTA of the team starts loading the
// next block before all have issued the loads of this one (a counter per team that the items wait on and add to;
// CTAs without work on a block get a filler that only does that).  Blocks go to teams longest first.
// `mode`: 0 = teams when the set has enough blocks to keep them busy, 1 = never, 2 = whenever a team fits.
// Returns the number of teams, or 0 after falling back to schedule_items.
int schedule_panels(std::vector<tc::Item>& v, const std::vector<BlockSpan>& blocks, int grid,
                    std::vector<int32_t>& begin, int stage_k, int mode) {
  for (auto& it : v) it.cost = item_cost(it, stage_k);
  struct Plan { size_t blk; int n_long, n_short_ctas; int64_t duration; bool rows_long; };
  std::vector<Plan> plans;
  int team = 1;
  for (size_t b = 0; b < blocks.size(); ++b) {
    const BlockSpan& B = blocks[b];
    if (B.n_row == 0 || B.n_col == 0) { team = grid + 1; break; }
    const int64_t c_row = v[B.first].cost, c_col = v[B.first + B.n_row].cost;
    Plan p;
    p.blk = b; p.rows_long = c_row >= c_col;
    const int64_t c_long = p.rows_long ? c_row : c_col, c_short = p.rows_long ? c_col : c_row;
    const size_t n_long = p.rows_long ? B.n_row : B.n_col, n_short = p.rows_long ? B.n_col : B.n_row;
    p.n_long = (int)n_long;
    p.n_short_ctas = (int)std::min<int64_t>((int64_t)n_short, ((int64_t)n_short * c_short + c_long - 1) / c_long);
    p.duration = std::max<int64_t>(c_long, ((int64_t)n_short + p.n_short_ctas - 1) / p.n_short_ctas * c_short);
    team = std::max(team, p.n_long + p.n_short_ctas);
    plans.push_back(p);
  }
  const int n_teams = (team <= grid && mode != 1) ? grid / team : 0;
  if (n_teams == 0 || (mode == 0 && (int)blocks.size() < 4 * n_teams)) {
    schedule_items(v, grid, begin, stage_k);
    return 0;
  }
  std::stable_sort(plans.begin(), plans.end(), [](const Plan& a, const Plan& b) { return a.duration > b.duration; });
  std::vector<std::vector<tc::Item>> per(grid);
  std::vector<int64_t> load(n_teams, 0);
  std::vector<int> done(n_teams, 0);      // blocks given to the team so far
  tc::Item filler;
  std::memset(&filler, 0, sizeof(filler));
  filler.epi = tc::EPI_NONE; filler.rp = 16; filler.half = 16; filler.sumsq_off = -1;
  for (const Plan& p : plans) {
    int t = 0;
    for (int q = 1; q < n_teams; ++q)
      if (load[q] < load[t]) t = q;
    load[t] += p.duration;
    const BlockSpan& B = blocks[p.blk];
    const size_t long0 = p.rows_long ? B.first : B.first + B.n_row;
    const size_t short0 = p.rows_long ? B.first + B.n_row : B.first;
    const size_t n_short = p.rows_long ? B.n_col : B.n_row;
    const int cta0 = t * team;
    std::vector<size_t> mark(team);
    for (int q = 0; q < team; ++q) mark[q] = per[cta0 + q].size();
    for (int i = 0; i < p.n_long; ++i) per[cta0 + i].push_back(v[long0 + i]);
    for (size_t j = 0; j < n_short; ++j) per[cta0 + p.n_long + (int)(j % p.n_short_ctas)].push_back(v[short0 + j]);
    for (int q = 0; q < team; ++q) {
      std::vector<tc::Item>& mine = per[cta0 + q];
      if (mine.size() == mark[q]) mine.push_back(filler);
      for (size_t i = mark[q]; i < mine.size(); ++i) { mine[i].team = (int16_t)t; mine[i].signal = 0; mine[i].wait_count = 0; }
      mine[mark[q]].wait_count = team * done[t];      // every member has issued the loads of the block before
      mine.back().signal = 1;
    }
    ++done[t];
  }
  v.clear();
  begin.assign(grid + 1, 0);
  for (int c = 0; c < grid; ++c) {
    v.insert(v.end(), per[c].begin(), per[c].end());
    begin[c + 1] = (int32_t)v.size();
  }
  return n_teams;
}

}  // namespace

int build_tensor_program(adapm_ctx* c, const std::vector<int64_t>& tc_ids, const std::vector<double>& etas,
                         int64_t& work_cursor, std::vector<ReduceJob>& row_jobs, int64_t& row_groups) {
  TcProgram* P = new TcProgram();
  c->tc = P;
  int dev = 0;
  cudaDeviceProp prop;
  if (cudaGetDevice(&dev) == cudaSuccess && cudaGetDeviceProperties(&prop, dev) == cudaSuccess)
    P->n_sms = prop.multiProcessorCount;
  const adapm_hparams& hp = c->hp;
  const float b1 = hp.beta1, a1 = 1.f - hp.beta1;
  const int K_eff = (int)etas.size();
  P->rotate = K_eff > 0;
  const bool fold_sumsq = K_eff > 0 && !(hp.flags & ADAPM_FLAG_NO_SUMSQ_FOLD);

  // ---- workspace arrays (bf16), offsets counted in bf16 elements ------------------------------------
  P->work_begin = work_cursor;
  auto take = [&](int64_t bf16_elems) {
    const int64_t off = work_cursor * 2;
    work_cursor += round_up((bf16_elems + 128 + 1) / 2, kStateAlign);   // +256 B: see encode_bf16_chunked
    return off;
  };
  int rp_max = 16, half_max = 16;
  for (int64_t id : tc_ids) {
    const adapm_block& b = c->blocks[id];
    TcBlock t;
    t.id = id;
    t.rp = round16(b.rank);
    t.half = 2 * t.rp <= 256 ? t.rp : round64(t.rp);
    rp_max = std::max(rp_max, t.rp);
    half_max = std::max(half_max, t.half);
    const int64_t lcat = take((int64_t)b.rows * 4 * t.half), rcat = take((int64_t)b.cols * 4 * t.half);
    t.lc[0] = lcat; t.lc[1] = lcat + 2 * t.half; t.lc[2] = take((int64_t)b.rows * 2 * t.half);
    t.rtc[0] = rcat; t.rtc[1] = rcat + 2 * t.half; t.rtc[2] = take((int64_t)b.cols * 2 * t.half);
    t.ld[0] = t.ld[1] = 4 * t.half; t.ld[2] = 2 * t.half;
    for (int w = 0; w < 4; ++w) t.gs[w] = take((int64_t)2 * t.half * 2 * t.half);
    t.rowsum = -1;
    if (hp.inner_precond) {
      auto take_f = [&](int64_t floats) { const int64_t off = work_cursor; work_cursor += round_up(floats, kStateAlign); return off; };
      t.lct = take((int64_t)b.rows * 2 * t.half);
      t.rtct = take((int64_t)b.cols * 2 * t.half);
      t.gf = take_f(2LL * b.rank * b.rank);
      t.sf = take_f(2LL * b.rank * b.rank);
      t.ltf = take_f((int64_t)b.rows * b.rank);
      t.rtf = take_f((int64_t)b.rank * b.cols);
    }
    P->blk.push_back(t);
  }
  P->work_end = work_cursor;
  // row sums of g^2 of the blocks with group scalars: written by the first refit pass, folded into v by a
  // reduction whose "partial sums" are the rows of a group
  for (TcBlock& t : P->blk) {
    const adapm_block& b = c->blocks[t.id];
    if (!fold_sumsq || b.v_mode != ADAPM_V_BLOCKMEAN) continue;
    t.rowsum = work_cursor;
    work_cursor += round_up(b.rows, kStateAlign);
    const int group_rows = b.v_group_rows == 0 ? b.rows : b.v_group_rows;
    ReduceJob j;
    std::memset(&j, 0, sizeof(j));
    j.g_off = b.offset; j.group_elems = (int64_t)group_rows * b.cols; j.n_groups = b.rows / group_rows;
    j.v_off = c->v_off[t.id]; j.part_off = t.rowsum; j.chunks_per_group = group_rows;
    j.first_unit = 0; j.first_group = row_groups;
    row_groups += j.n_groups;
    row_jobs.push_back(j);
  }
  P->rp_max = rp_max; P->half_max = half_max;
  const int nb_max = (2 * half_max + 63) / 64;
  P->nb_max = nb_max;

  // ---- stage depth and panels per item ---------------------------------------------------------------------------
  // As many panels share a B box as tensor memory has room for accumulators (2 rp columns each) and shared
  // memory for at least two stages; K = 128 stages while two of them fit, else K = 64.
  auto stages_with = [&](int stage_k, int n_a) { return (224 * 1024) / (n_a * 256 * stage_k + stage_k * 128 * nb_max); };
  int n_pan = hp.tune_panels > 0 ? hp.tune_panels : 2;
  n_pan = std::max(1, std::min({n_pan, tc::kMaxA, 512 / (2 * rp_max)}));
  int stage_k = hp.tune_stage_k == 64 || hp.tune_stage_k == 128 ? hp.tune_stage_k : 128;
  if (hp.tune_stage_k == 0 && stages_with(128, std::min(n_pan, 2)) < 2) stage_k = 64;
  while (n_pan > 1 && stages_with(stage_k, n_pan) < 2) --n_pan;
  if (stages_with(stage_k, n_pan) < 2) stage_k = 64;
  if (stages_with(stage_k, n_pan) < 2) { set_error_text("rank too large for the tensor path"); return ADAPM_EUNSUPPORTED; }
  P->stage_k = stage_k;
  const bool gram_small = 4 * rp_max <= 512 && 2 * rp_max <= 256;   // two accumulators of N = 2 rp: hi and lo window
  const int gram_na = (gram_small && stages_with(stage_k, 2) < 2) ? 1 : 2;
  P->smem_engine = std::max(P->engine_config(n_pan).smem, P->engine_config(gram_na).smem);

  auto& prog = c->program;

  // ---- convert -------------------------------------------------------------------------------------------
  // into the set that is "previous" at the step's parity; without refit passes the "final" factors are the
  // previous ones, nothing rotates, and X and Y get the same copy at every step
  for (int parity = 0; parity < (P->rotate ? 2 : 1); ++parity) {
    std::vector<ConvertJob> jobs;
    int64_t owners = 0;
    for (const TcBlock& t : P->blk) {
      const adapm_block& b = c->blocks[t.id];
      ConvertJob j;
      std::memset(&j, 0, sizeof(j));
      j.r = b.rank; j.rp = t.rp; j.half = t.half;
      for (int set = (P->rotate ? parity : 0); set < (P->rotate ? parity + 1 : 2); ++set) {
        j.dst_ld = t.ld[set];
        j.f32_off = c->l_off[t.id]; j.own_stride = b.rank; j.k_stride = 1; j.owners = b.rows; j.dst_off = t.lc[set];
        j.first_owner = owners; owners += j.owners; jobs.push_back(j);
        j.f32_off = c->r_off[t.id]; j.own_stride = 1; j.k_stride = b.cols; j.owners = b.cols; j.dst_off = t.rtc[set];
        j.first_owner = owners; owners += j.owners; jobs.push_back(j);
      }
    }
    P->n_convert_owners = owners;
    Launch L{LK_TC_CONVERT, append_items(c->h_tables, jobs), (int64_t)jobs.size(), (owners + 255) / 256};
    L.aux0 = owners;
    L.only_convert = P->rotate ? 1 : 0;
    L.when = P->rotate ? (parity ? WHEN_ODD : WHEN_EVEN) : WHEN_ALWAYS;
    prog.push_back(L);
  }

  // ---- refit passes, once per parity of the step and per kind of step ------------------------------------------
  // With a refresh period T > 1 a step either refits both factors (phase 1) or holds L and refits R (phase 2:
  // Gram matrices of L only, column panels only, and the split copy of L carried over to the final set).
  int team_mode = (hp.flags & ADAPM_FLAG_NO_PANEL_TEAMS) ? 1 : ((hp.flags & ADAPM_FLAG_FORCE_PANEL_TEAMS) ? 2 : 0);
  {
    // The team pacing lets CTAs of a launch wait for one another, which is only sound when the whole grid (at most
    // one CTA per SM) can be resident at once: ask the runtime whether an SM takes a CTA of this size at all (a
    // device or an MPS share with less shared memory or fewer registers does not), else hand items out longest-first.
    int resident = 0;
    cudaFuncSetAttribute(tc::tc_items_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, P->smem_engine);
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, tc::tc_items_kernel, tc::kEngineThreads,
                                                      (size_t)P->smem_engine) != cudaSuccess || resident < 1)
      team_mode = 1;
    (void)cudaGetLastError();
  }
  const bool with_hold = hp.refresh_period > 1 && K_eff > 0;
  for (int parity = 0; parity < (P->rotate ? 2 : 1); ++parity)
  for (int phase = (with_hold ? 1 : 0); phase <= (with_hold ? 2 : 0); ++phase) {
    const bool hold = phase == 2;
    const int prev = parity, fin = 1 - parity;
    const int when = P->rotate ? (parity ? WHEN_ODD : WHEN_EVEN) : WHEN_ALWAYS;
    if (hold) {
      std::vector<CopyJob> jobs;
      int64_t rows = 0;
      for (const TcBlock& t : P->blk) {
        const adapm_block& b = c->blocks[t.id];
        CopyJob j{t.lc[prev], t.lc[fin], b.rows, 2 * t.half, t.ld[prev], t.ld[fin], rows};
        rows += b.rows;
        jobs.push_back(j);
      }
      Launch CP{LK_TC_COPY, append_items(c->h_tables, jobs), (int64_t)jobs.size(), (rows + 7) / 8};
      CP.aux0 = rows; CP.when = when; CP.phase = phase;
      prog.push_back(CP);
    }
    int src = prev;
    for (int pass = 0; pass < K_eff; ++pass) {
      const int dst = ((K_eff - 1 - pass) % 2 == 0) ? fin : 2;
      const float coef = (float)etas[pass] * a1;
      std::vector<tc::Item> grams, panels;
      std::vector<BlockSpan> spans;
      bool any_sumsq = false;
      // Preconditioned passes: dl/dL (R R^T + d I)^-1 = (L R - m_t) (S_R R)^T and (L^T L + d I)^-1 dl/dR =
      // (L S_L)^T (L R - m_t), so the pass is Algorithm 2's with the transformed factors on the N side of every
      // product.  They are made first, from the fp32 factors in the state (the panels keep those current): the two
      // Gram matrices and the two products by the batched CUDA-core GEMM, the inverses, then the split copies.
      const bool precond = hp.inner_precond != 0;
      if (precond) {
        std::vector<GemmProb> pG, pT;
        std::vector<InverseJob> inv;
        std::vector<ConvertJob> cj;
        int64_t tG = 0, tT = 0, owners = 0;
        auto push = [](std::vector<GemmProb>& v, GemmProb p, int64_t& tiles) {
          p.tiles_n = (p.N + 63) / 64;
          p.first_tile = tiles;
          tiles += (int64_t)((p.M + 63) / 64) * p.tiles_n;
          v.push_back(p);
        };
        for (const TcBlock& t : P->blk) {
          const adapm_block& b = c->blocks[t.id];
          const int m = b.rows, n = b.cols, r = b.rank;
          const int64_t L = c->l_off[t.id], R = c->r_off[t.id];
          const int64_t GR = t.gf, GL = t.gf + (int64_t)r * r, SR = t.sf, SL = t.sf + (int64_t)r * r;
          GemmProb p;
          auto reset = [&]() { std::memset(&p, 0, sizeof(p)); p.z1_base = p.z2_base = BASE_NONE; p.alpha = 1.f; };
          ConvertJob j;
          std::memset(&j, 0, sizeof(j));
          j.r = r; j.rp = t.rp; j.half = t.half; j.dst_ld = 2 * t.half;
          if (!hold) {
            reset(); p.x_base = BASE_STATE; p.x_off = R; p.sxi = n; p.sxk = 1;             // G_R = R R^T
            p.y_base = BASE_STATE; p.y_off = R; p.syk = 1; p.syj = n;
            p.c_base = BASE_WORK; p.c_off = GR; p.M = r; p.N = r; p.K = n; p.ldc = r; push(pG, p, tG);
            inv.push_back({GR, SR, r, 0});
            reset(); p.x_base = BASE_WORK; p.x_off = SR; p.sxi = r; p.sxk = 1;              // S_R R
            p.y_base = BASE_STATE; p.y_off = R; p.syk = n; p.syj = 1;
            p.c_base = BASE_WORK; p.c_off = t.rtf; p.M = r; p.N = n; p.K = r; p.ldc = n; push(pT, p, tT);
            j.f32_off = t.rtf; j.own_stride = 1; j.k_stride = n; j.owners = n; j.dst_off = t.rtct;
            j.first_owner = owners; owners += j.owners; cj.push_back(j);
          }
          reset(); p.x_base = BASE_STATE; p.x_off = L; p.sxi = 1; p.sxk = r;                // G_L = L^T L
          p.y_base = BASE_STATE; p.y_off = L; p.syk = r; p.syj = 1;
          p.c_base = BASE_WORK; p.c_off = GL; p.M = r; p.N = r; p.K = m; p.ldc = r; push(pG, p, tG);
          inv.push_back({GL, SL, r, 0});
          reset(); p.x_base = BASE_STATE; p.x_off = L; p.sxi = r; p.sxk = 1;                // L S_L
          p.y_base = BASE_WORK; p.y_off = SL; p.syk = r; p.syj = 1;
          p.c_base = BASE_WORK; p.c_off = t.ltf; p.M = m; p.N = r; p.K = r; p.ldc = r; push(pT, p, tT);
          j.f32_off = t.ltf; j.own_stride = r; j.k_stride = 1; j.owners = m; j.dst_off = t.lct;
          j.first_owner = owners; owners += j.owners; cj.push_back(j);
        }
        Launch A1{LK_GEMM, append_items(c->h_tables, pG), (int64_t)pG.size(), tG};
        Launch A2{LK_SPD_INVERSE, append_items(c->h_tables, inv), (int64_t)inv.size(), (int64_t)inv.size()};
        Launch A3{LK_GEMM, append_items(c->h_tables, pT), (int64_t)pT.size(), tT};
        Launch A4{LK_TC_CONVERT_WORK, append_items(c->h_tables, cj), (int64_t)cj.size(), (owners + 255) / 256};
        A4.aux0 = owners;
        for (Launch* X : {&A1, &A2, &A3, &A4}) { X->when = when; X->phase = phase; prog.push_back(*X); }
      }
      for (size_t bi = 0; bi < P->blk.size(); ++bi) {
        const TcBlock& t = P->blk[bi];
        const adapm_block& b = c->blocks[t.id];
        const int m = b.rows, n = b.cols, r = b.rank, rp = t.rp, half = t.half;
        const int mb = (int)bi * kMapsPerBlock;
        const Geo geo{stage_k, (2 * half + 63) / 64};
        const bool small = 2 * rp <= 256;
        // Gram item: G[k][j] = sc * sum_x Y[x][k] X[x][j]; Y (the A side, read with K along y in 128-column
        // windows) and X (the N side) are [x, 2 half] arrays.  Up to rank 128 one item makes the whole matrix in
        // two accumulators (the hi and the lo window of Y, four partial sums); above, an item makes 128 rows of
        // it in one accumulator that the hi and the lo window both add to.
        auto gram = [&](int map_y_t, int map_x_n, int kext, int which, float sc) {
          for (int w0 = 0; w0 < rp; w0 += (small ? rp : 128)) {
            tc::Item it;
            std::memset(&it, 0, sizeof(it));
            if (small && gram_na == 2) {
              it.seg[0] = make_seg(geo, map_y_t, 0, 0, 1, 2, half, 0, map_x_n, rp, half, kext, 0, 2 * rp, 1);
              it.n_seg = 1; it.n_sum = 4;
            } else if (small) {
              it.seg[0] = make_seg(geo, map_y_t, 0, 0, 1, 1, 0, 0, map_x_n, rp, half, kext, 0, 0, 1);
              it.seg[1] = make_seg(geo, map_y_t, half, 0, 1, 1, 0, 0, map_x_n, rp, half, kext, 2 * rp, 0, 1);
              it.n_seg = 2; it.n_sum = 4;
            } else {
              it.seg[0] = make_seg(geo, map_y_t, w0, 0, 1, 2, half, 0, map_x_n, rp, half, kext, 0, 0, 1);
              it.seg[0].same_acc = 1;
              it.n_seg = 1; it.n_sum = 2;
            }
            it.epi = tc::EPI_GRAM; it.r = r; it.rp = rp; it.half = half; it.coef = sc; it.own0 = w0;
            it.dst_off = t.gs[which]; it.dst_ld = 2 * half; it.stack_rows = half; it.sumsq_off = -1;
            grams.push_back(it);
          }
        };
        const int srcL = hold ? prev : src;     // a held L stays in the previous set all step long
        // the factor on the N side of every product: itself, or its transformed copy in a preconditioned pass
        const int nR = precond ? mb + MAP_RTCN_T : mb + MAP_RTCN + src;
        const int nL = precond ? mb + MAP_LCN_T : mb + MAP_LCN + srcL;
        if (!hold) {
          gram(mb + MAP_RTCT + src, nR, n, 0, -1.f / a1);  // Bop1[j][k] = -(R R^T)[j][k] / (1-b1), stored as [k][j]
          gram(mb + MAP_RTCT + prev, nR, n, 1, b1 / a1);   // Bop2[j][k] = b1 (R R0^T)[j][k] / (1-b1)
        }
        gram(mb + MAP_LCT + srcL, nL, m, 2, -1.f / a1);    // Bop3[j][k] = -(L^T L)[j][k] / (1-b1)
        gram(mb + MAP_LCT + prev, nL, m, 3, b1 / a1);      // Bop4[j][k] = b1 (L^T L0)[j][k] / (1-b1)

        // one item = up to n_pan adjacent panels of 128 owners that share every B box
        auto panel = [&](bool is_L, int p0, int np) {
          tc::Item it;
          std::memset(&it, 0, sizeof(it));
          const int mS = (is_L ? mb + MAP_LC : mb + MAP_RTC) + src, m0 = (is_L ? mb + MAP_LC : mb + MAP_RTC) + prev;
          const int g1 = mb + MAP_GS + (is_L ? 0 : 2), g2 = g1 + 1;
          if (is_L) it.seg[0] = make_seg(geo, mb + MAP_G, 0, p0, 0, np, 0, 128, nR, rp, half, n, 0, 2 * rp, 1);  // g R^T
          else it.seg[0] = make_seg(geo, mb + MAP_GT, p0, 0, 1, np, 128, 0, nL, rp, half, m, 0, 2 * rp, 1);      // g^T L
          // [hi | lo] of the current and of the previous factor against the stacked Gram operands
          it.seg[1] = make_seg(geo, mS, 0, p0, 0, np, 0, 128, g1, rp, half, half + rp, 0, 2 * rp, 0);
          it.seg[2] = make_seg(geo, m0, 0, p0, 0, np, 0, 128, g2, rp, half, half + rp, 0, 2 * rp, 0);
          it.n_seg = 3;
          it.n_pan = np; it.acc_stride = 2 * rp;
          it.epi = tc::EPI_FACTOR; it.r = r; it.rp = rp; it.half = half; it.coef = coef;
          it.own0 = p0; it.own_count = is_L ? m : n;
          it.f32_off = is_L ? c->l_off[t.id] : c->r_off[t.id];
          it.own_stride = is_L ? r : 1; it.k_stride = is_L ? 1 : n;
          it.dst_off = is_L ? t.lc[dst] : t.rtc[dst]; it.dst_ld = t.ld[dst];
          it.sumsq_off = (is_L && pass == 0 && t.rowsum >= 0) ? t.rowsum + p0 : -1;
          if (it.sumsq_off >= 0) any_sumsq = true;
          panels.push_back(it);
        };
        BlockSpan sp;
        sp.first = panels.size();
        if (!hold)
          for (int p0 = 0; p0 < m; p0 += 128 * n_pan) panel(true, p0, std::min(n_pan, (m - p0 + 127) / 128));
        sp.n_row = panels.size() - sp.first;
        for (int p0 = 0; p0 < n; p0 += 128 * n_pan) panel(false, p0, std::min(n_pan, (n - p0 + 127) / 128));
        sp.n_col = panels.size() - sp.first - sp.n_row;
        spans.push_back(sp);
      }
      const int grid_g = (int)std::min<int64_t>((int64_t)grams.size(), P->n_sms);
      const int grid_p = (int)std::min<int64_t>((int64_t)panels.size(), P->n_sms);
      std::vector<int32_t> begin_g, begin_p;
      schedule_items(grams, grid_g, begin_g, stage_k);
      P->n_teams = std::max(P->n_teams, schedule_panels(panels, spans, grid_p, begin_p, stage_k, team_mode));
      Launch G{LK_TC_GRAM, append_items(c->h_tables, grams), (int64_t)grams.size(), grid_g};
      G.aux0 = gram_small ? 4 * rp_max : 2 * rp_max;
      G.aux1 = 2 * G.aux0 <= 512 ? 2 : 1; G.aux2 = gram_na;
      G.aux3 = append_items(c->h_tables, begin_g);
      G.aux4 = -1; G.aux5 = 0;
      G.when = when; G.phase = phase;
      prog.push_back(G);
      Launch Q{LK_TC_PANEL, append_items(c->h_tables, panels), (int64_t)panels.size(), grid_p};
      Q.aux0 = n_pan * 2 * rp_max; Q.aux1 = 2 * Q.aux0 <= 512 ? 2 : 1;
      Q.aux2 = n_pan;
      Q.aux3 = append_items(c->h_tables, begin_p);
      // one accumulator buffer that leaves room to park the sums D0 + D1 of its panels (rp columns each)
      Q.aux4 = (Q.aux1 == 1 && Q.aux0 + n_pan * rp_max <= 512) ? Q.aux0 : -1;
      Q.aux5 = any_sumsq ? 1 : 0;
      Q.when = when; Q.phase = phase;
      prog.push_back(Q);
      if (pass == 0 && !row_jobs.empty() && !hold) {
        Launch RF{LK_REDUCE_ROWS, 0, 0, 0};       // table filled in by the caller (shared by both parities)
        RF.when = when; RF.phase = phase;
        prog.push_back(RF);
      }
      src = dst;
    }
  }

  // ---- apply ---------------------------------------------------------------------------------------------------
  // Blocks up to rank 128 keep the L panel of an item resident; above that L is streamed like R (second launch).
  {
    std::vector<tc::ApplyItem> items, items_s;
    int nbc_max = 1;
    bool any_element_v = false;
    for (size_t bi = 0; bi < P->blk.size(); ++bi) {
      const TcBlock& t = P->blk[bi];
      const adapm_block& b = c->blocks[t.id];
      const int mb = (int)bi * kMapsPerBlock;
      const bool stream = t.half != t.rp;
      const int nbc1 = (2 * t.rp + 63) / 64, nbc2 = (4 * t.rp + 63) / 64;
      if (!stream) nbc_max = std::max(nbc_max, nbc2);
      if (b.v_mode == ADAPM_V_ELEMENT) any_element_v = true;
      const int tiles = (b.cols + tc::kApplyNT - 1) / tc::kApplyNT;
      const int runs = (tiles + 15) / 16;
      for (int p0 = 0; p0 < b.rows; p0 += 128) {
        for (int q = 0; q < runs; ++q) {
          tc::ApplyItem a;
          std::memset(&a, 0, sizeof(a));
          a.off = b.offset; a.v_off = c->v_off[t.id]; a.rows = b.rows; a.cols = b.cols; a.r = b.rank; a.rp = t.rp;
          a.half = t.half;
          a.map_l = mb + MAP_LCAT; a.map_r = mb + MAP_RCAT;
          a.map_w = mb + MAP_W; a.map_g = mb + MAP_G32; a.map_v = mb + MAP_V; a.map_sh = mb + MAP_SH;
          a.row0 = p0;
          a.tile0 = (int)((int64_t)tiles * q / runs);
          a.n_tiles = (int)((int64_t)tiles * (q + 1) / runs) - a.tile0;
          a.nbc1 = nbc1; a.nbc2 = nbc2; a.v_mode = b.v_mode;
          a.v_group_rows = b.v_group_rows == 0 ? b.rows : b.v_group_rows;
          a.lr_scale = b.lr_scale; a.wd = b.weight_decay;
          (stream ? items_s : items).push_back(a);
        }
      }
    }
    // shared memory: the L panel (both factor sets side by side), a ring of R^T boxes, a ring of g / W quarter
    // tiles.  Three R stages, and whatever is left for g / W: measured, the g / W ring pays more per KB than a
    // deeper R ring, but two R stages leave the MMA warp waiting on every box.
    const int l_region = nbc_max * tc::kBoxBytes;
    P->apply_r_stages = 3;
    P->apply_r_region = l_region;
    P->apply_buf_bytes = tc::kApplyBufBytes + (any_element_v ? tc::kWBoxBytes : 0);
    auto bufs_with = [&](int r_stages) { return (226 * 1024 - l_region - r_stages * tc::kBoxBytes) / P->apply_buf_bytes; };
    if (any_element_v && bufs_with(3) < 3 && bufs_with(1) >= 3) {
      // the larger buffers of a per-element v: a third buffer is worth more than the second and third R stage
      // (measured on the 1.5B shapes: 9.6 ms with three R stages and two buffers, 8.0 ms with one and three)
      P->apply_r_stages = 1;
    } else if (bufs_with(3) < 2) {   // two buffers at least: give up an R stage
      P->apply_r_stages = 2;
    }
    P->apply_w_region = l_region + P->apply_r_stages * tc::kBoxBytes;
    P->apply_bufs = std::max(1, std::min(tc::kApplyMaxBufs, (226 * 1024 - P->apply_w_region) / P->apply_buf_bytes));
    P->smem_apply = P->apply_w_region + P->apply_bufs * P->apply_buf_bytes + 1024;
    // the streaming form: two stages of four boxes, the rest for g / W
    P->apply_s_w_region = 2 * 4 * tc::kBoxBytes;
    P->apply_s_bufs = std::max(1, std::min(tc::kApplyMaxBufs, (226 * 1024 - P->apply_s_w_region) / P->apply_buf_bytes));
    P->smem_apply_s = P->apply_s_w_region + P->apply_s_bufs * P->apply_buf_bytes + 1024;
    if (!items.empty()) {
      Launch A{LK_TC_APPLY, append_items(c->h_tables, items), (int64_t)items.size(),
               std::min<int64_t>((int64_t)items.size(), P->n_sms)};
      prog.push_back(A);
    }
    if (!items_s.empty()) {
      Launch A{LK_TC_APPLY, append_items(c->h_tables, items_s), (int64_t)items_s.size(),
               std::min<int64_t>((int64_t)items_s.size(), P->n_sms)};
      A.aux0 = 1;
      prog.push_back(A);
    }
  }

  // ---- device memory of the path -------------------------------------------------------------------------------
  const size_t map_bytes = P->blk.size() * kMapsPerBlock * sizeof(CUtensorMap);
  cudaError_t e = cudaSuccess;
  for (MapSet& m : P->maps) {
    if (e == cudaSuccess) e = cudaMalloc((void**)&m.d_maps, map_bytes);
    m.h_maps.resize(P->blk.size() * kMapsPerBlock);
  }
  if (e == cudaSuccess && P->n_teams > 0) e = cudaMalloc((void**)&P->d_team_counters, P->n_teams * sizeof(int32_t));
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(tc::tc_items_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, P->smem_engine);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(tc::tc_apply_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, P->smem_apply);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(tc::tc_apply_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, P->smem_apply_s);
  if (e != cudaSuccess) {
    set_cuda_error(e, "build_tensor_program");
    return ADAPM_ECUDA;
  }
  return ADAPM_OK;
}

// ---------------------------------------------------------------------------------------------------
// per-step work
// ---------------------------------------------------------------------------------------------------

// Tensor maps hold absolute addresses.  A small cache keeps the maps of the last four combinations of caller
// buffers (parameters, gradients, state, workspace), each with its own device copy, so that callers who alternate
// between a few buffers encode each combination once.  A new combination is encoded on the host and copied with a
// stream-ordered copy from pageable memory (which the runtime stages before it returns): no wait on the device.
// Also decides whether this step has to rebuild the split copies of the factors, and which parity it runs.
int tensor_prepare_step(adapm_ctx* c, const Bases& b, int64_t t, cudaStream_t s, int* parity, int* convert) {
  TcProgram* P = c->tc;
  *parity = 0; *convert = 0;
  if (!P || P->blk.empty()) return ADAPM_OK;
  // The parity of a step is a function of its number alone, so that a run continued from a checkpoint repeats
  // the uninterrupted run bit for bit (the apply kernel adds the two factor sets in the order they lie in).
  const bool fresh = !P->split_valid || t != P->last_t + 1 || P->last_state != b.p[BASE_STATE] ||
                     P->last_work != b.p[BASE_WORK];
  *convert = (!P->rotate || fresh) ? 1 : 0;
  *parity = P->rotate ? (int)((t - 1) & 1) : 0;
  P->split_valid = true; P->last_t = t; P->last_state = b.p[BASE_STATE]; P->last_work = b.p[BASE_WORK];

  ++P->use_clock;
  MapSet* slot = nullptr;
  for (MapSet& m : P->maps)
    if (m.key[0] == b.p[0] && m.key[1] == b.p[1] && m.key[2] == b.p[2] && m.key[3] == b.p[3] && m.key[4] == b.shadow &&
        m.key[0])
      slot = &m;
  if (slot) {
    slot->last_use = P->use_clock;
    P->cur_maps = slot->d_maps;
    return ADAPM_OK;
  }
  slot = &P->maps[0];
  for (MapSet& m : P->maps)
    if (m.last_use < slot->last_use) slot = &m;
  const char* grads = static_cast<const char*>(b.p[BASE_GRADS]);
  const char* work = static_cast<const char*>(b.p[BASE_WORK]);
  const char* params = static_cast<const char*>(b.p[BASE_PARAMS]);
  const char* state = static_cast<const char*>(b.p[BASE_STATE]);
  const uint32_t sk = (uint32_t)P->stage_k;
  for (size_t bi = 0; bi < P->blk.size(); ++bi) {
    const TcBlock& t2 = P->blk[bi];
    const adapm_block& blk = c->blocks[t2.id];
    CUtensorMap* m = slot->h_maps.data() + bi * kMapsPerBlock;
    const uint64_t rows = blk.rows, cols = blk.cols, half = t2.half;
    const uint32_t nb = (uint32_t)((2 * half + 63) / 64);
    bool ok = tc::encode_bf16_matrix(&m[MAP_G], grads + blk.offset * 2, rows, cols, cols, 128);
    ok = ok && tc::encode_bf16_matrix(&m[MAP_GT], grads + blk.offset * 2, rows, cols, cols, sk);
    ok = ok && tc::encode_panel32(&m[MAP_W], params + blk.offset * 4, rows, cols, true);
    ok = ok && tc::encode_panel32(&m[MAP_G32], grads + blk.offset * 2, rows, cols, false);
    if (blk.v_mode == ADAPM_V_ELEMENT)
      ok = ok && tc::encode_panel32(&m[MAP_V], state + c->v_off[t2.id] * 4, rows, cols, true);
    else
      std::memset(&m[MAP_V], 0, sizeof(CUtensorMap));
    for (int q = 0; q < 3; ++q) {
      const uint64_t ld = (uint64_t)t2.ld[q];
      ok = ok && tc::encode_bf16_matrix(&m[MAP_LC + q], work + t2.lc[q] * 2, rows, 2 * half, ld, 128);
      ok = ok && tc::encode_bf16_matrix(&m[MAP_LCT + q], work + t2.lc[q] * 2, rows, 2 * half, ld, sk);
      ok = ok && tc::encode_bf16_chunked(&m[MAP_LCN + q], work + t2.lc[q] * 2, rows, ld, nb, sk);
      ok = ok && tc::encode_bf16_matrix(&m[MAP_RTC + q], work + t2.rtc[q] * 2, cols, 2 * half, ld, 128);
      ok = ok && tc::encode_bf16_matrix(&m[MAP_RTCT + q], work + t2.rtc[q] * 2, cols, 2 * half, ld, sk);
      ok = ok && tc::encode_bf16_chunked(&m[MAP_RTCN + q], work + t2.rtc[q] * 2, cols, ld, nb, sk);
    }
    ok = ok && tc::encode_bf16_matrix(&m[MAP_LCAT], work + t2.lc[0] * 2, rows, 4 * half, 4 * half, 128);
    ok = ok && tc::encode_bf16_matrix(&m[MAP_RCAT], work + t2.rtc[0] * 2, cols, 4 * half, 4 * half, 128);
    if (c->hp.inner_precond) {
      ok = ok && tc::encode_bf16_chunked(&m[MAP_LCN_T], work + t2.lct * 2, rows, 2 * half, nb, sk);
      ok = ok && tc::encode_bf16_chunked(&m[MAP_RTCN_T], work + t2.rtct * 2, cols, 2 * half, nb, sk);
    } else {
      std::memset(&m[MAP_LCN_T], 0, 2 * sizeof(CUtensorMap));
    }
    if (b.shadow)
      ok = ok && tc::encode_panel32(&m[MAP_SH], reinterpret_cast<const char*>(b.shadow) + blk.offset * 2, rows, cols, false);
    else
      std::memset(&m[MAP_SH], 0, sizeof(CUtensorMap));
    for (int q = 0; q < 4; ++q)
      ok = ok && tc::encode_bf16_chunked(&m[MAP_GS + q], work + t2.gs[q] * 2, 2 * half, 2 * half, nb, sk);
    if (!ok) {
      set_error_text("cuTensorMapEncodeTiled failed for a low-rank block");
      return ADAPM_ECUDA;
    }
  }
  ADAPM_CUDA(cudaMemcpyAsync(slot->d_maps, slot->h_maps.data(), slot->h_maps.size() * sizeof(CUtensorMap),
                             cudaMemcpyHostToDevice, s));
  for (int q = 0; q < 4; ++q) slot->key[q] = b.p[q];
  slot->key[4] = b.shadow;
  slot->last_use = P->use_clock;
  P->cur_maps = slot->d_maps;
  return ADAPM_OK;
}

int run_tensor_launch(adapm_ctx* c, const Launch& L, const Bases& b, const StepScalars& sc, int parity,
                      cudaStream_t s) {
  TcProgram* P = c->tc;
  if (!P) return ADAPM_EUNSUPPORTED;
  const unsigned char* tab = c->d_tables + L.table_off;
  if (L.grid <= 0) return ADAPM_OK;
  switch (L.kind) {
    case LK_TC_CONVERT:
      // arrays are zeroed first: padding columns and rows that no kernel writes must read as zero
      ADAPM_CUDA(cudaMemsetAsync((char*)b.p[BASE_WORK] + P->work_begin * 4, 0, (size_t)(P->work_end - P->work_begin) * 4, s));
      tc_convert_kernel<<<(unsigned)L.grid, 256, 0, s>>>((const ConvertJob*)tab, (int)L.n_items, L.aux0,
                                                        (const float*)b.p[BASE_STATE], (uint16_t*)b.p[BASE_WORK],
                                                        c->d_status);
      break;
    case LK_TC_CONVERT_WORK:
      // the same split copy from fp32 arrays in the workspace (nothing is zeroed: the padding stays as the last
      // full rebuild left it)
      tc_convert_kernel<<<(unsigned)L.grid, 256, 0, s>>>((const ConvertJob*)tab, (int)L.n_items, L.aux0,
                                                        (const float*)b.p[BASE_WORK], (uint16_t*)b.p[BASE_WORK],
                                                        c->d_status);
      break;
    case LK_TC_COPY:
      tc_copy_kernel<<<(unsigned)L.grid, 256, 0, s>>>((const CopyJob*)tab, (int)L.n_items, L.aux0,
                                                     (uint16_t*)b.p[BASE_WORK], c->d_status);
      break;
    case LK_TC_GRAM:
    case LK_TC_PANEL: {
      tc::EngineArgs a;
      std::memset(&a, 0, sizeof(a));
      a.items = (const tc::Item*)tab; a.n_items = (int32_t)L.n_items; a.maps = P->cur_maps;
      a.f32_base = (float*)b.p[BASE_STATE]; a.work_bf16 = (uint16_t*)b.p[BASE_WORK]; a.work_f32 = (float*)b.p[BASE_WORK];
      a.status = c->d_status;
      const TcProgram::EngineConfig e = P->engine_config((int)L.aux2);
      a.stage_k = P->stage_k; a.stage_bytes = e.stage_bytes; a.n_stages = e.n_stages; a.a_bytes = e.a_bytes;
      a.acc_cols = (int32_t)L.aux0; a.n_acc = (int32_t)L.aux1;
      a.cta_begin = (const int32_t*)(c->d_tables + L.aux3);
      a.sum_col = (int32_t)L.aux4; a.sumsq_on = (int32_t)L.aux5;
      a.team_counters = nullptr;
      a.team_spin_limit = tc::kTeamSpinDefault; a.wait_spin_limit = tc::kWaitSpinDefault;
      a.gscale = b.gscale;
      if (L.kind == LK_TC_PANEL && P->d_team_counters) {
        ADAPM_CUDA(cudaMemsetAsync(P->d_team_counters, 0, P->n_teams * sizeof(int32_t), s));
        a.team_counters = P->d_team_counters;
      }
      tc::tc_items_kernel<<<(unsigned)L.grid, tc::kEngineThreads, e.smem, s>>>(a);
      break;
    }
    case LK_TC_APPLY: {
      tc::ApplyArgs a;
      a.items = (const tc::ApplyItem*)tab; a.n_items = (int32_t)L.n_items; a.maps = P->cur_maps;
      a.state = (float*)b.p[BASE_STATE]; a.status = c->d_status; a.sc = sc;
      a.use_new = sc.c1 != 0.f ? 1 : 0;
      a.parity = parity;
      a.buf_bytes = P->apply_buf_bytes;
      a.gscale = b.gscale;
      a.shadow = b.shadow != nullptr;
      if (L.aux0 == 0) {
        a.r_region_off = P->apply_r_region; a.n_rstages = P->apply_r_stages;
        a.w_region_off = P->apply_w_region; a.n_bufs = P->apply_bufs;
        tc::tc_apply_kernel<false><<<(unsigned)L.grid, tc::kApplyThreads, P->smem_apply, s>>>(a);
      } else {
        a.r_region_off = 0; a.n_rstages = 2;
        a.w_region_off = P->apply_s_w_region; a.n_bufs = P->apply_s_bufs;
        tc::tc_apply_kernel<true><<<(unsigned)L.grid, tc::kApplyThreads, P->smem_apply_s, s>>>(a);
      }
      break;
    }
    default:
      return ADAPM_EUNSUPPORTED;
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    set_cuda_error(e, "run_tensor_launch");
    return ADAPM_ECUDA;
  }
  return ADAPM_OK;
}

// Diagnostic: one CTA of the engine whose only item waits for a team counter that nothing advances, with a wait
// limit of about a millisecond.  The kernel must return, leave ST_WAIT_TEAM in the status word and free its
// tensor memory; the context stays usable.
int run_expired_wait_probe(adapm_ctx* c, cudaStream_t s) {
  struct Probe { tc::Item item; int32_t begin[4]; };
  static_assert(sizeof(Probe) % 4 == 0, "probe table");
  if (!c->d_probe) return ADAPM_EUNSUPPORTED;
  tc::EngineArgs a;
  std::memset(&a, 0, sizeof(a));
  a.items = (const tc::Item*)c->d_probe; a.n_items = 1; a.maps = nullptr;
  a.status = c->d_status;
  a.stage_k = 64; a.stage_bytes = 1024; a.a_bytes = 512; a.n_stages = 2; a.acc_cols = 32; a.n_acc = 1;
  a.cta_begin = (const int32_t*)(c->d_probe + sizeof(tc::Item));
  a.sum_col = -1; a.sumsq_on = 0;
  a.team_counters = c->d_status + 16;       // a zeroed word beside the status word that nothing adds to
  a.team_spin_limit = 1u << 12; a.wait_spin_limit = tc::kWaitSpinDefault;
  tc::tc_items_kernel<<<1, tc::kEngineThreads, 4096, s>>>(a);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    set_cuda_error(e, "run_expired_wait_probe");
    return ADAPM_ECUDA;
  }
  return ADAPM_OK;
}

size_t probe_table(std::vector<unsigned char>& out) {
  tc::Item it;
  std::memset(&it, 0, sizeof(it));
  it.epi = tc::EPI_NONE; it.rp = 16; it.half = 16; it.sumsq_off = -1;
  it.team = 0; it.wait_count = 1; it.signal = 0;
  out.resize(sizeof(tc::Item) + 4 * sizeof(int32_t));
  std::memcpy(out.data(), &it, sizeof(it));
  const int32_t begin[4] = {0, 1, 1, 1};
  std::memcpy(out.data() + sizeof(it), begin, sizeof(begin));
  return out.size();
}

}  // namespace adapm
