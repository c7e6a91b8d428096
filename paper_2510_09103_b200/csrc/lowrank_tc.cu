// Tensor-core (tcgen05) low-rank path: the per-step program of Algorithm 2's refit and of the
// corrected update for every low-rank block whose layout the TMA engine can address
// (bf16 gradients, cols a multiple of 8, rank <= 128).
//
// Per step:
//   convert   (L_{t-1}, R_{t-1}) fp32 -> split-bf16 arrays  Lc[0] = [L hi | L lo]  (rows x 2rp)
//                                                           RTc[0] = [R^T hi | R^T lo] (cols x 2rp)
//   K_eff times:  gram    four r x r products of the current iterate (tensor cores) -> Gs[0..3]
//                         (each stored transposed, [rp, 2rp] = [hi | lo], the layout the engine's N side reads)
//                 panel   row panels update L, column panels update R (tensor cores); fp32 factors
//                         are updated in place in the state, their split copies go to the other of
//                         the two iterate sets Lc[1|2], RTc[1|2]
//   apply     m^c and the parameter write from (Lc[0], RTc[0]) and the final iterate set
// rp = rank rounded up to 16; padded columns are kept at zero by every writer.
#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstring>

#include "adapm_internal.h"
#include "tc_apply.cuh"
#include "tc_engine.cuh"
#include "tc_host.h"

namespace adapm {

void set_error_text(const char* text);   // ctx.cu

namespace {

// tensor maps of one block: g; Lc[3] and RTc[3] each as a plain matrix (A side) and as 64-column
// chunks (N side); Gs[4] as chunks; W and g in quarter-tile boxes; the previous and the final set of
// Lc and of RTc side by side as one matrix (the apply kernel's operands); a per-element v like W
constexpr int kMapsPerBlock = 22;
enum { MAP_G = 0, MAP_LC = 1, MAP_LC_N = 4, MAP_RTC = 7, MAP_RTC_N = 10, MAP_GS = 13, MAP_W = 17, MAP_G32 = 18,
       MAP_LCAT = 19, MAP_RCAT = 20, MAP_V = 21 };

struct ConvertJob {
  int64_t f32_off;          // float offset of the factor in state
  int64_t own_stride, k_stride;
  int64_t dst_off;          // bf16 element offset in the workspace
  int32_t owners, r, rp;
  int32_t dst_ld;           // row pitch of the destination, in elements
  int64_t first_owner;      // prefix sum of owners
};

// fp32 factor -> [owners, 2rp] split bf16 with row pitch dst_ld (hi columns, then lo columns; columns >= r are zero)
__global__ void __launch_bounds__(256) tc_convert_kernel(const ConvertJob* __restrict__ jobs, int n_jobs,
                                                         int64_t total_owners, const float* __restrict__ state,
                                                         uint16_t* __restrict__ work) {
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
    uint4* dl = reinterpret_cast<uint4*>(dst + J.rp + p);
    dh[0] = make_uint4(h[0], h[1], h[2], h[3]);
    dh[1] = make_uint4(h[4], h[5], h[6], h[7]);
    dl[0] = make_uint4(l[0], l[1], l[2], l[3]);
    dl[1] = make_uint4(l[4], l[5], l[6], l[7]);
  }
}

}  // namespace

// Host side of the tensor path, owned by the context.
struct TcBlock {
  int64_t id;                      // index into ctx->blocks
  int32_t rp;
  int64_t lc[3], rtc[3], gs[4];    // bf16 element offsets in the workspace
  int32_t ld[3];                   // row pitch of set s of lc / rtc, in elements
};

struct TcProgram {
  std::vector<TcBlock> blk;
  int64_t n_convert_owners = 0;
  int smem_engine = 0, smem_apply = 0;
  int nb_max = 1;
  // shared-memory plan of an engine launch: `wide` = stages with two A operands
  struct EngineConfig { int a_bytes, stage_bytes, n_stages, smem; };
  EngineConfig engine_config(bool wide) const {
    EngineConfig e;
    e.a_bytes = (wide ? 2 : 1) * tc::kStageABytes;
    e.stage_bytes = e.a_bytes + tc::kBoxBytes * nb_max;
    e.n_stages = std::max(2, std::min(8, (224 * 1024) / e.stage_bytes));
    e.smem = e.n_stages * e.stage_bytes + 1024;
    return e;
  }
  int apply_r_region = 0, apply_r_stages = 3, apply_w_region = 0, apply_bufs = 2, apply_buf_bytes = 0;
  int n_sms = 148;
  int final_set = 0;
  // tensor maps: device table + pinned host staging, re-encoded when the buffers move
  CUtensorMap* d_maps = nullptr;
  int32_t* d_team_counters = nullptr;   // pacing counters of the panel launches (see schedule_panels)
  int n_teams = 0;
  CUtensorMap* h_maps = nullptr;
  const void* enc_grads = nullptr;
  const void* enc_work = nullptr;
  const void* enc_params = nullptr;
  const void* enc_state = nullptr;
  cudaEvent_t maps_copied = nullptr;
};

bool tensor_path_block_ok(const adapm_hparams& hp, const adapm_block& b) {
  if (hp.lowrank_path == ADAPM_PATH_SIMT) return false;
  if (hp.grad_dtype != ADAPM_GRAD_BF16) return false;
  if (b.mom_mode != ADAPM_MOM_LOWRANK) return false;
  if (b.cols % 8 != 0 || b.rank > 128) return false;
  return tc::encode_tiled_fn() != nullptr;
}

void destroy_tensor_program(adapm_ctx* c) {
  TcProgram* p = c->tc;
  if (!p) return;
  if (p->d_maps) cudaFree(p->d_maps);
  if (p->d_team_counters) cudaFree(p->d_team_counters);
  if (p->h_maps) cudaFreeHost(p->h_maps);
  if (p->maps_copied) cudaEventDestroy(p->maps_copied);
  delete p;
  c->tc = nullptr;
}

// ---------------------------------------------------------------------------------------------------
// program construction
// ---------------------------------------------------------------------------------------------------
namespace {

int round16(int x) { return (x + 15) / 16 * 16; }

template <typename T>
int64_t append_items(std::vector<unsigned char>& blob, const std::vector<T>& tab) {
  const size_t off = (blob.size() + 15) / 16 * 16;
  blob.resize(off + tab.size() * sizeof(T));
  if (!tab.empty()) std::memcpy(blob.data() + off, tab.data(), tab.size() * sizeof(T));
  return (int64_t)off;
}

// A: 2-D map `map_a`, first box at (ax, ay), K along x (a_mode 0) or along y (a_mode 1).
// B: chunked map `map_b` whose boxes are b_rows x (64 * nb_b), K rows starting at 0.
tc::Seg make_seg(int map_a, int ax, int ay, int a_mode, int map_b, int b_rows, int n, int k, int d_col, int first) {
  tc::Seg s;
  std::memset(&s, 0, sizeof(s));
  const int nb_b = (n + 63) / 64;
  s.map_a = map_a; s.map_b = map_b; s.ax = ax; s.ay = ay; s.by = 0;
  s.a_mode = (int16_t)a_mode; s.n = (int16_t)n; s.k = round16(k); s.d_col = (int16_t)d_col; s.first = (int16_t)first;
  s.b_lbo = 128u * (uint32_t)b_rows;
  s.tx_bytes = (uint32_t)tc::kStageABytes + 128u * (uint32_t)b_rows * (uint32_t)nb_b;
  s.n_a = 1;
  return s;
}

// Adds a second A operand (same map and direction) that accumulates at column d_col2.
void add_second_a(tc::Seg& s, int ax2, int ay2, int d_col2) {
  s.n_a = 2; s.ax2 = ax2; s.ay2 = ay2; s.d_col2 = (int16_t)d_col2;
  s.tx_bytes += (uint32_t)tc::kStageABytes;
}

int item_cost(const tc::Item& it) {
  int c = 0;
  for (int s = 0; s < it.n_seg; ++s) c += (it.seg[s].k + tc::kStageK - 1) / tc::kStageK;
  return c + 2;   // the epilogue
}

// Hands the items to `grid` CTAs, longest first, each to the CTA with the least work so far.  Afterwards CTA c owns
// v[begin[c] .. begin[c + 1]).
void schedule_items(std::vector<tc::Item>& v, int grid, std::vector<int32_t>& begin) {
  for (auto& it : v) it.cost = item_cost(it);
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

// Team schedule for a panel launch.  The row panels and the column panels of a block each read all of g, DRAM is
// what bounds the launch, and at full size the second read finds nothing in L2 unless it follows the first
// closely.  So a team of CTAs takes one block at a time: every item of the kind with the longer K loop gets a CTA
// of its own, the items of the other kind are dealt in order to as many further CTAs as keep pace with them (item
// j of the short kind covers the j-th slice of the long kind's K range, so both kinds sweep g together), and no
// CTA of the team starts loading the next block before all have issued the loads of this one (a counter per team
// that the items wait on and add to; CTAs without work on a block get a filler that only does that).
// Blocks go to teams longest first.  Returns the number of teams, or 0 after falling back to schedule_items when
// the blocks are too few to keep teams busy.
int schedule_panels(std::vector<tc::Item>& v, const std::vector<BlockSpan>& blocks, int grid,
                    std::vector<int32_t>& begin) {
  for (auto& it : v) it.cost = item_cost(it);
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
  // The pacing assumes that the CTAs of the launch run at the same time (one per SM).  A caller who shares the
  // GPU with long-running kernels can turn it off: ADAPM_PANEL_TEAMS=0 in the environment at adapm_create.
  const char* env = std::getenv("ADAPM_PANEL_TEAMS");
  const bool teams_off = env && env[0] == '0';
  const int n_teams = (team <= grid && !teams_off) ? grid / team : 0;
  if (n_teams == 0 || (int)blocks.size() < 4 * n_teams) {
    schedule_items(v, grid, begin);
    return 0;
  }
  std::stable_sort(plans.begin(), plans.end(), [](const Plan& a, const Plan& b) { return a.duration > b.duration; });
  std::vector<std::vector<tc::Item>> per(grid);
  std::vector<int64_t> load(n_teams, 0);
  std::vector<int> done(n_teams, 0);      // blocks given to the team so far
  tc::Item filler;
  std::memset(&filler, 0, sizeof(filler));
  filler.epi = tc::EPI_NONE; filler.own1 = -1; filler.rp = 16;
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
                         int64_t& work_cursor) {
  TcProgram* P = new TcProgram();
  c->tc = P;
  int dev = 0;
  cudaDeviceProp prop;
  if (cudaGetDevice(&dev) == cudaSuccess && cudaGetDeviceProperties(&prop, dev) == cudaSuccess)
    P->n_sms = prop.multiProcessorCount;
  const adapm_hparams& hp = c->hp;
  const float b1 = hp.beta1, a1 = 1.f - hp.beta1;

  // ---- workspace arrays (bf16), offsets counted in bf16 elements ------------------------------------
  auto take = [&](int64_t bf16_elems) {
    const int64_t off = work_cursor * 2;
    work_cursor += round_up((bf16_elems + 128 + 1) / 2, kStateAlign);   // +256 B: see encode_bf16_chunked
    return off;
  };
  // the refit passes alternate between sets 1 and 2, starting from 0.  Without any pass the "final" factors are
  // the previous ones: they are then converted a second time, into set 1, so that the apply kernel's operand
  // layout does not change.
  P->final_set = etas.empty() ? 1 : (etas.size() % 2 ? 1 : 2);
  int rp_max = 16;
  for (int64_t id : tc_ids) {
    const adapm_block& b = c->blocks[id];
    TcBlock t;
    t.id = id;
    t.rp = round16(b.rank);
    rp_max = std::max(rp_max, t.rp);
    // the previous set (0) and the set the last refit pass writes share one array with row pitch 4rp, side by
    // side, so that the apply kernel reads both as one 4rp-wide operand; the third set has an array of its own
    const int64_t lcat = take((int64_t)b.rows * 4 * t.rp), rcat = take((int64_t)b.cols * 4 * t.rp);
    const int other = 3 - P->final_set;
    t.lc[0] = lcat; t.lc[P->final_set] = lcat + 2 * t.rp; t.lc[other] = take((int64_t)b.rows * 2 * t.rp);
    t.rtc[0] = rcat; t.rtc[P->final_set] = rcat + 2 * t.rp; t.rtc[other] = take((int64_t)b.cols * 2 * t.rp);
    for (int s = 0; s < 3; ++s) t.ld[s] = (s == other ? 2 : 4) * t.rp;
    for (int w = 0; w < 4; ++w) t.gs[w] = take((int64_t)2 * t.rp * t.rp);
    P->blk.push_back(t);
  }
  const int nb_max = (2 * rp_max + 63) / 64;
  // Every stage gets two A operands when two such stages still fit: Gram items read the hi and the
  // lo column window of their A side against the same B boxes, panel items take two adjacent panels
  // of a block.  Besides halving the B bytes per flop, consecutive MMAs then alternate between two
  // accumulators instead of forming one dependent chain, which nearly doubles the issue rate.
  const bool two_a = 2 * (2 * tc::kStageABytes + tc::kBoxBytes * nb_max) <= 224 * 1024;
  const bool pair_panels = two_a;
  P->nb_max = nb_max;
  P->smem_engine = 0;
  P->smem_engine = P->engine_config(false).smem;
  if (two_a) P->smem_engine = std::max(P->smem_engine, P->engine_config(true).smem);

  auto& prog = c->program;

  // ---- convert -------------------------------------------------------------------------------------------
  {
    std::vector<ConvertJob> jobs;
    int64_t owners = 0;
    for (const TcBlock& t : P->blk) {
      const adapm_block& b = c->blocks[t.id];
      ConvertJob j;
      std::memset(&j, 0, sizeof(j));
      j.r = b.rank; j.rp = t.rp;
      j.dst_ld = 4 * t.rp;   // sets 0 and (without refit passes) 1 = the final set: the shared array
      for (int set = 0; set < (etas.empty() ? 2 : 1); ++set) {
        j.f32_off = c->l_off[t.id]; j.own_stride = b.rank; j.k_stride = 1; j.owners = b.rows; j.dst_off = t.lc[set];
        j.first_owner = owners; owners += j.owners; jobs.push_back(j);
        j.f32_off = c->r_off[t.id]; j.own_stride = 1; j.k_stride = b.cols; j.owners = b.cols; j.dst_off = t.rtc[set];
        j.first_owner = owners; owners += j.owners; jobs.push_back(j);
      }
    }
    P->n_convert_owners = owners;
    Launch L{LK_TC_CONVERT, append_items(c->h_tables, jobs), (int64_t)jobs.size(), (owners + 255) / 256};
    L.aux0 = owners;
    prog.push_back(L);
  }

  // ---- refit passes ----------------------------------------------------------------------------------------
  int src = 0;
  for (size_t pass = 0; pass < etas.size(); ++pass) {
    const int dst = src == 1 ? 2 : 1;
    const float coef = (float)etas[pass] * a1;
    std::vector<tc::Item> grams, panels;
    std::vector<BlockSpan> spans;
    for (size_t bi = 0; bi < P->blk.size(); ++bi) {
      const TcBlock& t = P->blk[bi];
      const adapm_block& b = c->blocks[t.id];
      const int m = b.rows, n = b.cols, r = b.rank, rp = t.rp;
      const int mb = (int)bi * kMapsPerBlock;
      const int mG = mb + MAP_G, mLs = mb + MAP_LC + src, mL0 = mb + MAP_LC, mRs = mb + MAP_RTC + src,
                mR0 = mb + MAP_RTC, mLsN = mb + MAP_LC_N + src, mRsN = mb + MAP_RTC_N + src;
      // Gram item: dst[k][j] = coef * sum_x Y[x][k] X[x][j]; Y (the A side, read MN-major in two
      // 128-column windows: the hi columns, then the lo columns) and X (the N side) are [x, 2rp] arrays
      auto gram = [&](int map_y, int map_x_n, int kext, int which, float sc) {
        tc::Item it;
        std::memset(&it, 0, sizeof(it));
        it.seg[0] = make_seg(map_y, 0, 0, 1, map_x_n, 128, 2 * rp, kext, 0, 1);
        if (two_a) {
          it.n_seg = 1;
          add_second_a(it.seg[0], rp, 0, 2 * rp);
        } else {
          it.n_seg = 2;
          it.seg[1] = make_seg(map_y, rp, 0, 1, map_x_n, 128, 2 * rp, kext, 2 * rp, 1);
        }
        it.own1 = -1;
        it.epi = tc::EPI_GRAM; it.r = r; it.rp = rp; it.coef = sc;
        it.dst_off = t.gs[which]; it.dst_ld = 2 * rp;
        grams.push_back(it);
      };
      gram(mRs, mRsN, n, 0, -1.f / a1);     // Bop1[j][k] = -(R R^T)[j][k] / (1-b1), stored as [k][j]
      gram(mR0, mRsN, n, 1, b1 / a1);       // Bop2[j][k] = b1 (R R0^T)[j][k] / (1-b1)
      gram(mLs, mLsN, m, 2, -1.f / a1);     // Bop3[j][k] = -(L^T L)[j][k] / (1-b1)
      gram(mL0, mLsN, m, 3, b1 / a1);       // Bop4[j][k] = b1 (L^T L0)[j][k] / (1-b1)

      // one item = one panel of 128 owners, or two adjacent panels that share every B box
      auto panel = [&](bool is_L, int p0, bool pair) {
        tc::Item it;
        std::memset(&it, 0, sizeof(it));
        const int mS = is_L ? mLs : mRs, m0 = is_L ? mL0 : mR0;
        const int g1 = mb + MAP_GS + (is_L ? 0 : 2), g2 = g1 + 1;
        if (is_L) it.seg[0] = make_seg(mG, 0, p0, 0, mRsN, 128, 2 * rp, n, 0, 1);     // g R^T over the columns
        else it.seg[0] = make_seg(mG, p0, 0, 1, mLsN, 128, 2 * rp, m, 0, 1);           // g^T L over the rows
        it.seg[1] = make_seg(mS, 0, p0, 0, g1, rp, 2 * rp, rp, 0, 0);
        it.seg[2] = make_seg(mS, rp, p0, 0, g1, rp, 2 * rp, rp, 0, 0);
        it.seg[3] = make_seg(m0, 0, p0, 0, g2, rp, 2 * rp, rp, 0, 0);
        it.seg[4] = make_seg(m0, rp, p0, 0, g2, rp, 2 * rp, rp, 0, 0);
        it.n_seg = 5;
        it.own1 = -1;
        if (pair) {
          if (is_L) add_second_a(it.seg[0], 0, p0 + 128, 2 * rp);
          else add_second_a(it.seg[0], p0 + 128, 0, 2 * rp);
          for (int q = 1; q < 5; ++q) add_second_a(it.seg[q], it.seg[q].ax, p0 + 128, 2 * rp);
          it.own1 = p0 + 128;
          it.col2 = 2 * rp;
        }
        it.epi = tc::EPI_FACTOR; it.r = r; it.rp = rp; it.coef = coef;
        it.own0 = p0; it.own_count = is_L ? m : n;
        it.f32_off = is_L ? c->l_off[t.id] : c->r_off[t.id];
        it.own_stride = is_L ? r : 1; it.k_stride = is_L ? 1 : n;
        it.dst_off = is_L ? t.lc[dst] : t.rtc[dst]; it.dst_ld = t.ld[dst];
        panels.push_back(it);
      };
      const int step = pair_panels ? 256 : 128;
      BlockSpan sp;
      sp.first = panels.size();
      for (int p0 = 0; p0 < m; p0 += step) panel(true, p0, pair_panels && p0 + 128 < m);
      sp.n_row = panels.size() - sp.first;
      for (int p0 = 0; p0 < n; p0 += step) panel(false, p0, pair_panels && p0 + 128 < n);
      sp.n_col = panels.size() - sp.first - sp.n_row;
      spans.push_back(sp);
    }
    const int grid_g = (int)std::min<int64_t>((int64_t)grams.size(), P->n_sms);
    const int grid_p = (int)std::min<int64_t>((int64_t)panels.size(), P->n_sms);
    std::vector<int32_t> begin_g, begin_p;
    schedule_items(grams, grid_g, begin_g);
    P->n_teams = std::max(P->n_teams, schedule_panels(panels, spans, grid_p, begin_p));
    Launch G{LK_TC_GRAM, append_items(c->h_tables, grams), (int64_t)grams.size(), grid_g};
    G.aux0 = 4 * rp_max; G.aux1 = 8 * rp_max <= 512 ? 2 : 1; G.aux2 = two_a ? 1 : 0;
    G.aux3 = append_items(c->h_tables, begin_g);
    prog.push_back(G);
    Launch Q{LK_TC_PANEL, append_items(c->h_tables, panels), (int64_t)panels.size(), grid_p};
    Q.aux0 = (pair_panels ? 4 : 2) * rp_max; Q.aux1 = (pair_panels ? 8 : 4) * rp_max <= 512 ? 2 : 1;
    Q.aux2 = pair_panels ? 1 : 0;
    Q.aux3 = append_items(c->h_tables, begin_p);
    prog.push_back(Q);
    src = dst;
  }

  // ---- apply ---------------------------------------------------------------------------------------------------
  {
    std::vector<tc::ApplyItem> items;
    int nbc_max = 1;
    bool any_element_v = false;
    for (size_t bi = 0; bi < P->blk.size(); ++bi) {
      const TcBlock& t = P->blk[bi];
      const adapm_block& b = c->blocks[t.id];
      const int mb = (int)bi * kMapsPerBlock;
      const int nbc1 = (2 * t.rp + 63) / 64, nbc2 = (4 * t.rp + 63) / 64;
      nbc_max = std::max(nbc_max, nbc2);
      if (b.v_mode == ADAPM_V_ELEMENT) any_element_v = true;
      const int tiles = (b.cols + tc::kApplyNT - 1) / tc::kApplyNT;
      const int runs = (tiles + 15) / 16;
      for (int p0 = 0; p0 < b.rows; p0 += 128) {
        for (int q = 0; q < runs; ++q) {
          tc::ApplyItem a;
          std::memset(&a, 0, sizeof(a));
          a.off = b.offset; a.v_off = c->v_off[t.id]; a.rows = b.rows; a.cols = b.cols; a.r = b.rank; a.rp = t.rp;
          a.map_l = mb + MAP_LCAT; a.map_r = mb + MAP_RCAT;
          a.map_w = mb + MAP_W; a.map_g = mb + MAP_G32; a.map_v = mb + MAP_V;
          a.row0 = p0;
          a.tile0 = (int)((int64_t)tiles * q / runs);
          a.n_tiles = (int)((int64_t)tiles * (q + 1) / runs) - a.tile0;
          a.nbc1 = nbc1; a.nbc2 = nbc2; a.v_mode = b.v_mode;
          a.v_group_rows = b.v_group_rows == 0 ? b.rows : b.v_group_rows;
          a.lr_scale = b.lr_scale; a.wd = b.weight_decay;
          items.push_back(a);
        }
      }
    }
    // shared memory: the L panel (both factor sets side by side), a ring of R^T boxes, a ring of g / W quarter
    // tiles.  Three R stages, and whatever is left for g / W: measured, the g / W ring pays more per KB than a
    // deeper R ring, but two R stages leave the MMA warp waiting on every box.
    const int l_region = nbc_max * tc::kBoxBytes;
    P->apply_r_stages = 3;
    P->apply_r_region = l_region;
    P->apply_w_region = l_region + P->apply_r_stages * tc::kBoxBytes;
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
    Launch A{LK_TC_APPLY, append_items(c->h_tables, items), (int64_t)items.size(),
             std::min<int64_t>((int64_t)items.size(), P->n_sms)};
    prog.push_back(A);
  }

  // ---- tensor maps -------------------------------------------------------------------------------------------------
  const size_t map_bytes = P->blk.size() * kMapsPerBlock * sizeof(CUtensorMap);
  cudaError_t e = cudaMalloc((void**)&P->d_maps, map_bytes);
  if (e == cudaSuccess && P->n_teams > 0) e = cudaMalloc((void**)&P->d_team_counters, P->n_teams * sizeof(int32_t));
  if (e == cudaSuccess) e = cudaMallocHost((void**)&P->h_maps, map_bytes);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&P->maps_copied, cudaEventDisableTiming);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(tc::tc_items_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, P->smem_engine);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(tc::tc_apply_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, P->smem_apply);
  if (e != cudaSuccess) {
    set_cuda_error(e, "build_tensor_program");
    return ADAPM_ECUDA;
  }
  return ADAPM_OK;
}

// ---------------------------------------------------------------------------------------------------
// per-step work
// ---------------------------------------------------------------------------------------------------

// Tensor maps hold absolute addresses: (re)build them when the parameter, gradient, state or workspace buffer
// moved.
// The copy to the device is asynchronous on `s`; only a second move while that copy is still in
// flight waits for it (the staging buffer is reused).
int tensor_prepare_step(adapm_ctx* c, const Bases& b, cudaStream_t s) {
  TcProgram* P = c->tc;
  if (!P || P->blk.empty()) return ADAPM_OK;
  if (P->enc_grads == b.p[BASE_GRADS] && P->enc_work == b.p[BASE_WORK] && P->enc_params == b.p[BASE_PARAMS] &&
      P->enc_state == b.p[BASE_STATE])
    return ADAPM_OK;
  if (P->enc_grads) ADAPM_CUDA(cudaEventSynchronize(P->maps_copied));
  const char* grads = static_cast<const char*>(b.p[BASE_GRADS]);
  const char* work = static_cast<const char*>(b.p[BASE_WORK]);
  const char* params = static_cast<const char*>(b.p[BASE_PARAMS]);
  const char* state = static_cast<const char*>(b.p[BASE_STATE]);
  for (size_t bi = 0; bi < P->blk.size(); ++bi) {
    const TcBlock& t = P->blk[bi];
    const adapm_block& blk = c->blocks[t.id];
    CUtensorMap* m = P->h_maps + bi * kMapsPerBlock;
    const uint64_t rows = blk.rows, cols = blk.cols, rp = t.rp;
    const uint32_t nb = (uint32_t)((2 * rp + 63) / 64);
    bool ok = tc::encode_bf16_matrix(&m[MAP_G], grads + blk.offset * 2, rows, cols, cols);
    ok = ok && tc::encode_panel32(&m[MAP_W], params + blk.offset * 4, rows, cols, true);
    ok = ok && tc::encode_panel32(&m[MAP_G32], grads + blk.offset * 2, rows, cols, false);
    if (blk.v_mode == ADAPM_V_ELEMENT)
      ok = ok && tc::encode_panel32(&m[MAP_V], state + c->v_off[t.id] * 4, rows, cols, true);
    else
      std::memset(&m[MAP_V], 0, sizeof(CUtensorMap));
    for (int q = 0; q < 3; ++q) {
      const uint64_t ld = (uint64_t)t.ld[q];
      ok = ok && tc::encode_bf16_matrix(&m[MAP_LC + q], work + t.lc[q] * 2, rows, 2 * rp, ld);
      ok = ok && tc::encode_bf16_chunked(&m[MAP_LC_N + q], work + t.lc[q] * 2, rows, ld, nb, 128);
      ok = ok && tc::encode_bf16_matrix(&m[MAP_RTC + q], work + t.rtc[q] * 2, cols, 2 * rp, ld);
      ok = ok && tc::encode_bf16_chunked(&m[MAP_RTC_N + q], work + t.rtc[q] * 2, cols, ld, nb, 128);
    }
    ok = ok && tc::encode_bf16_matrix(&m[MAP_LCAT], work + t.lc[0] * 2, rows, 4 * rp, 4 * rp);
    ok = ok && tc::encode_bf16_matrix(&m[MAP_RCAT], work + t.rtc[0] * 2, cols, 4 * rp, 4 * rp);
    for (int q = 0; q < 4; ++q)
      ok = ok && tc::encode_bf16_chunked(&m[MAP_GS + q], work + t.gs[q] * 2, rp, 2 * rp, nb, (uint32_t)rp);
    if (!ok) {
      set_error_text("cuTensorMapEncodeTiled failed for a low-rank block");
      return ADAPM_ECUDA;
    }
  }
  ADAPM_CUDA(cudaMemcpyAsync(P->d_maps, P->h_maps, P->blk.size() * kMapsPerBlock * sizeof(CUtensorMap),
                             cudaMemcpyHostToDevice, s));
  ADAPM_CUDA(cudaEventRecord(P->maps_copied, s));
  P->enc_grads = b.p[BASE_GRADS];
  P->enc_work = b.p[BASE_WORK];
  P->enc_params = b.p[BASE_PARAMS];
  P->enc_state = b.p[BASE_STATE];
  return ADAPM_OK;
}

int run_tensor_launch(adapm_ctx* c, const Launch& L, const Bases& b, const StepScalars& sc, cudaStream_t s) {
  TcProgram* P = c->tc;
  if (!P) return ADAPM_EUNSUPPORTED;
  const unsigned char* tab = c->d_tables + L.table_off;
  if (L.grid <= 0) return ADAPM_OK;
  switch (L.kind) {
    case LK_TC_CONVERT:
      tc_convert_kernel<<<(unsigned)L.grid, 256, 0, s>>>((const ConvertJob*)tab, (int)L.n_items, L.aux0,
                                                        (const float*)b.p[BASE_STATE], (uint16_t*)b.p[BASE_WORK]);
      break;
    case LK_TC_GRAM:
    case LK_TC_PANEL: {
      tc::EngineArgs a;
      a.items = (const tc::Item*)tab; a.n_items = (int32_t)L.n_items; a.maps = P->d_maps;
      a.f32_base = (float*)b.p[BASE_STATE]; a.work_bf16 = (uint16_t*)b.p[BASE_WORK]; a.status = c->d_status;
      const TcProgram::EngineConfig e = P->engine_config(L.aux2 != 0);
      a.stage_bytes = e.stage_bytes; a.n_stages = e.n_stages; a.a_bytes = e.a_bytes;
      a.acc_cols = (int32_t)L.aux0; a.n_acc = (int32_t)L.aux1;
      a.cta_begin = (const int32_t*)(c->d_tables + L.aux3);
      a.team_counters = nullptr;
      if (L.kind == LK_TC_PANEL && P->d_team_counters) {
        ADAPM_CUDA(cudaMemsetAsync(P->d_team_counters, 0, P->n_teams * sizeof(int32_t), s));
        a.team_counters = P->d_team_counters;
      }
      // one accumulator buffer of paired panels (4 rp_max columns) leaves room to park their sums (2 rp_max)
      a.sum_col = (L.kind == LK_TC_PANEL && L.aux2 != 0 && a.n_acc == 1 && a.acc_cols + a.acc_cols / 2 <= 512)
                      ? a.acc_cols : -1;
      tc::tc_items_kernel<<<(unsigned)L.grid, tc::kEngineThreads, e.smem, s>>>(a);
      break;
    }
    case LK_TC_APPLY: {
      tc::ApplyArgs a;
      a.items = (const tc::ApplyItem*)tab; a.n_items = (int32_t)L.n_items; a.maps = P->d_maps;
      a.state = (float*)b.p[BASE_STATE]; a.status = c->d_status; a.sc = sc;
      a.use_new = sc.c1 != 0.f ? 1 : 0;
      a.r_region_off = P->apply_r_region; a.n_rstages = P->apply_r_stages;
      a.w_region_off = P->apply_w_region; a.n_bufs = P->apply_bufs; a.buf_bytes = P->apply_buf_bytes;
      tc::tc_apply_kernel<<<(unsigned)L.grid, tc::kApplyThreads, P->smem_apply, s>>>(a);
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

}  // namespace adapm
