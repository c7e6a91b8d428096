// Context creation (validation, state / workspace layout, the static per-step launch program) and
// the step driver.  The driver only orders kernels on the caller's stream: it never allocates,
// copies to the host or synchronises.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>

#include <nvtx3/nvToolsExt.h>

#include "adapm_internal.h"

namespace adapm {

static thread_local std::string g_cuda_error;

void set_cuda_error(cudaError_t e, const char* where) {
  g_cuda_error = std::string(cudaGetErrorName(e)) + ": " + cudaGetErrorString(e) + " at " + where;
}

void set_error_text(const char* text) { g_cuda_error = text ? text : ""; }

namespace {

template <typename T>
int64_t append_table(std::vector<unsigned char>& blob, const std::vector<T>& tab) {
  const size_t off = (blob.size() + 15) / 16 * 16;
  blob.resize(off + tab.size() * sizeof(T));
  if (!tab.empty()) std::memcpy(blob.data() + off, tab.data(), tab.size() * sizeof(T));
  return (int64_t)off;
}

double inner_eta(int k, int K) { return 0.5 * (1.0 + std::cos(M_PI * (double)k / (double)K)); }

int validate(const adapm_block* blocks, int64_t n, const adapm_hparams& hp) {
  if (!(hp.beta1 >= 0.f && hp.beta1 < 1.f) || !(hp.beta2 >= 0.f && hp.beta2 < 1.f)) return ADAPM_ERANGE;
  if (!(hp.eps >= 0.f) || !(hp.clip > 0.f) || hp.inner_iters < 0 || hp.inner_iters > 64) return ADAPM_ERANGE;
  if (!std::isfinite(hp.lr) || !std::isfinite(hp.inner_lr_scale)) return ADAPM_EINVAL;
  if (hp.grad_dtype != ADAPM_GRAD_F32 && hp.grad_dtype != ADAPM_GRAD_BF16) return ADAPM_EINVAL;
  if (hp.lowrank_path < ADAPM_PATH_AUTO || hp.lowrank_path > ADAPM_PATH_TENSOR) return ADAPM_EINVAL;
  if (hp.refresh_period < 0) return ADAPM_ERANGE;
  if (!(hp.max_grad_norm >= 0.f)) return ADAPM_ERANGE;      // 0 and +inf both mean "no clipping"; NaN is refused
  if (hp.tune_panels < 0 || hp.tune_panels > 3) return ADAPM_ERANGE;
  if (hp.tune_stage_k != 0 && hp.tune_stage_k != 64 && hp.tune_stage_k != 128) return ADAPM_ERANGE;
  if (hp.inner_precond != 0 && hp.inner_precond != 1) return ADAPM_EINVAL;
  if (hp.inner_precond && !(hp.precond_damping >= 0.f && std::isfinite(hp.precond_damping))) return ADAPM_ERANGE;
  std::vector<std::pair<int64_t, int64_t>> spans;
  spans.reserve((size_t)n);
  for (int64_t i = 0; i < n; ++i) {
    const adapm_block& b = blocks[i];
    if (b.rows < 1 || b.cols < 1 || b.offset < 0) return ADAPM_ERANGE;
    if (b.offset % kAlignElems) return ADAPM_EALIGN;
    if (b.mom_mode < ADAPM_MOM_NONE || b.mom_mode > ADAPM_MOM_LOWRANK) return ADAPM_EINVAL;
    if (b.v_mode != ADAPM_V_ELEMENT && b.v_mode != ADAPM_V_BLOCKMEAN) return ADAPM_EINVAL;
    if (b.mom_mode == ADAPM_MOM_LOWRANK) {
      if (b.rank < 1 || b.rank > std::min(b.rows, b.cols)) return ADAPM_ERANGE;
    } else if (b.rank != 0) {
      return ADAPM_EINVAL;
    }
    if (b.v_mode == ADAPM_V_BLOCKMEAN) {
      if (b.v_group_rows < 0 || b.v_group_rows > b.rows) return ADAPM_ERANGE;
      if (b.v_group_rows > 0 && b.rows % b.v_group_rows) return ADAPM_ERANGE;
    }
    if (!std::isfinite(b.lr_scale) || !std::isfinite(b.weight_decay)) return ADAPM_EINVAL;
    spans.emplace_back(b.offset, b.offset + (int64_t)b.rows * b.cols);
  }
  std::sort(spans.begin(), spans.end());
  for (size_t i = 1; i < spans.size(); ++i)
    if (spans[i].first < spans[i - 1].second) return ADAPM_EINVAL;   // overlapping blocks
  return ADAPM_OK;
}

}  // namespace

// the tensor-core program of the low-rank blocks; defined in lowrank_tc.cu
bool tensor_path_block_ok(const adapm_hparams& hp, const adapm_block& b);
int build_tensor_program(adapm_ctx* c, const std::vector<int64_t>& tc_ids, const std::vector<double>& etas,
                         int64_t& work_cursor, std::vector<ReduceJob>& row_jobs, int64_t& row_groups);
int tensor_prepare_step(adapm_ctx* c, const Bases& b, int64_t t, cudaStream_t s, int* parity, int* convert);
int run_tensor_launch(adapm_ctx* c, const Launch& L, const Bases& b, const StepScalars& sc, int parity,
                      cudaStream_t s);
void destroy_tensor_program(adapm_ctx* c);
void tensor_state_changed(adapm_ctx* c);
int run_expired_wait_probe(adapm_ctx* c, cudaStream_t s);
size_t probe_table(std::vector<unsigned char>& out);

}  // namespace adapm

using namespace adapm;

extern "C" const char* adapm_last_cuda_error(void) { return g_cuda_error.c_str(); }

extern "C" int adapm_create(const adapm_block* blocks, int64_t n_blocks, const adapm_hparams* hp, adapm_ctx** out) {
  if (!blocks || n_blocks <= 0 || !hp || !out) return ADAPM_EINVAL;
  *out = nullptr;
  int rc = validate(blocks, n_blocks, *hp);
  if (rc != ADAPM_OK) return rc;

  adapm_ctx* c = new (std::nothrow) adapm_ctx();
  if (!c) return ADAPM_EINVAL;
  c->blocks.assign(blocks, blocks + n_blocks);
  c->hp = *hp;
  const int n = (int)n_blocks;
  const size_t gsz = hp->grad_dtype == ADAPM_GRAD_BF16 ? 2 : 4;

  // ---- which kernels run each low-rank block ----------------------------------------------------------
  std::vector<int64_t> lowrank_ids, tc_ids;     // lowrank_ids: the blocks of the CUDA-core path
  for (int i = 0; i < n; ++i) {
    const adapm_block& b = c->blocks[i];
    if (b.mom_mode != ADAPM_MOM_LOWRANK) continue;
    if (tensor_path_block_ok(*hp, b)) tc_ids.push_back(i);
    else if (hp->lowrank_path == ADAPM_PATH_TENSOR) { delete c; return ADAPM_EUNSUPPORTED; }
    else if (hp->inner_precond && b.rank > 4096) { delete c; return ADAPM_EUNSUPPORTED; }
    else lowrank_ids.push_back(i);
  }
  c->n_tensor_blocks = (int64_t)tc_ids.size();

  // ---- state layout: [L,R of the CUDA-core low-rank blocks][L,R of the tensor-core ones]
  //                    [m^f of every full block][v of every block] --------------------------------------
  c->m_off.assign(n, -1); c->l_off.assign(n, -1); c->r_off.assign(n, -1); c->v_off.assign(n, -1); c->v_cnt.assign(n, 0);
  int64_t cur = 0;
  auto place_factors = [&](int64_t i) {
    const adapm_block& b = c->blocks[i];
    c->l_off[i] = cur; cur += round_up((int64_t)b.rows * b.rank, kStateAlign);
    c->r_off[i] = cur; cur += round_up((int64_t)b.rank * b.cols, kStateAlign);
    c->bytes_L += (size_t)b.rows * b.rank * 4;
    c->bytes_R += (size_t)b.rank * b.cols * 4;
  };
  for (int64_t i : lowrank_ids) place_factors(i);
  c->lr_section_floats = cur;
  for (int64_t i : tc_ids) place_factors(i);
  for (int i = 0; i < n; ++i) {
    const adapm_block& b = c->blocks[i];
    if (b.mom_mode != ADAPM_MOM_FULL) continue;
    c->m_off[i] = cur; cur += round_up((int64_t)b.rows * b.cols, kStateAlign);
    c->bytes_m += (size_t)b.rows * b.cols * 4;
  }
  for (int i = 0; i < n; ++i) {
    const adapm_block& b = c->blocks[i];
    int64_t cnt;
    if (b.v_mode == ADAPM_V_ELEMENT) cnt = (int64_t)b.rows * b.cols;
    else cnt = b.v_group_rows == 0 ? 1 : b.rows / b.v_group_rows;
    c->v_off[i] = cur; c->v_cnt[i] = cnt; cur += round_up(cnt, kStateAlign);
    c->bytes_v += (size_t)cnt * 4;
  }
  c->state_floats = cur;

  // ---- algorithmic traffic and flops -----------------------------------------------------------
  int K_eff = 0;
  std::vector<double> etas;
  for (int k = 1; k <= hp->inner_iters; ++k) {
    const double e = inner_eta(k, hp->inner_iters) * (double)hp->inner_lr_scale;
    if (std::fabs(e) > 1e-12) { etas.push_back(e); ++K_eff; }
  }
  for (int i = 0; i < n; ++i) {
    const adapm_block& b = c->blocks[i];
    const size_t ne = (size_t)b.rows * b.cols;
    c->step_bytes += ne * (gsz + 8);
    if (b.mom_mode == ADAPM_MOM_FULL) c->step_bytes += ne * 8;
    if (b.mom_mode == ADAPM_MOM_LOWRANK) {
      c->step_bytes += (size_t)b.rank * (b.rows + b.cols) * 8;
      c->step_flops += (4.0 * K_eff + 4.0) * (double)b.rows * b.cols * b.rank;
    }
    c->step_bytes += (size_t)c->v_cnt[i] * 8;
  }

  // ---- streaming blocks and reduction jobs -------------------------------------------------------
  std::vector<StreamBlk> sblk;
  // two-stage group sums of g^2: `rjobs` run every step, `rjobs_hold` only in steps that hold L (there the
  // tensor path has no row panels to take the row sums from)
  struct ReduceSet { std::vector<ReduceJob> jobs; int64_t units = 0, groups = 0; };
  ReduceSet rset_all, rset_hold;
  int64_t cta_cursor = 0, work_cursor = 0;
  auto add_reduce_job = [&](ReduceSet& rs, int i, int64_t group_elems, int64_t n_groups) {
    std::vector<ReduceJob>& rjobs = rs.jobs;
    int64_t& unit_cursor = rs.units;
    int64_t& group_cursor = rs.groups;
    ReduceJob j;
    std::memset(&j, 0, sizeof(j));
    j.g_off = c->blocks[i].offset;
    j.group_elems = group_elems;
    j.n_groups = n_groups;
    j.v_off = c->v_off[i];
    j.chunks_per_group = (int32_t)((group_elems + kWarpUnitMax - 1) / kWarpUnitMax);
    j.part_off = work_cursor;
    work_cursor += round_up(n_groups * j.chunks_per_group, kStateAlign);
    j.first_unit = unit_cursor; unit_cursor += n_groups * j.chunks_per_group;
    j.first_group = group_cursor; group_cursor += n_groups;
    rjobs.push_back(j);
  };
  for (int i = 0; i < n; ++i) {
    const adapm_block& b = c->blocks[i];
    const int64_t numel = (int64_t)b.rows * b.cols;
    const int64_t group_elems = b.v_group_rows == 0 ? numel : (int64_t)b.v_group_rows * b.cols;
    const int64_t n_groups = numel / group_elems;
    if (b.mom_mode == ADAPM_MOM_LOWRANK) continue;
    StreamBlk s;
    std::memset(&s, 0, sizeof(s));
    s.off = b.offset; s.m_off = c->m_off[i]; s.v_off = c->v_off[i]; s.numel = numel;
    s.lr_scale = b.lr_scale; s.wd = b.weight_decay;
    s.units_per_group = 1; s.group_elems = group_elems;
    if (b.v_mode == ADAPM_V_ELEMENT) {
      s.v_mode = SV_ELEMENT; s.team = 32; s.unit_elems = kWarpUnitMax;
      s.n_units = (numel + kWarpUnitMax - 1) / kWarpUnitMax; s.vec_ok = 1;
    } else if (group_elems <= kCtaUnitMax) {
      s.v_mode = SV_GROUP_INLINE; s.team = group_elems <= kWarpUnitMax ? 32 : 256;
      s.unit_elems = (int32_t)group_elems; s.n_units = n_groups;
      s.vec_ok = (group_elems % kChunkElems == 0 || n_groups == 1) ? 1 : 0;
    } else {
      s.v_mode = SV_GROUP_READY; s.team = 32; s.unit_elems = kWarpUnitMax;
      s.units_per_group = (int32_t)((group_elems + kWarpUnitMax - 1) / kWarpUnitMax);
      s.n_units = n_groups * s.units_per_group;
      s.vec_ok = (group_elems % kChunkElems == 0 || n_groups == 1) ? 1 : 0;
      add_reduce_job(rset_all, i, group_elems, n_groups);
    }
    s.first_cta = cta_cursor;
    cta_cursor += s.team == 32 ? (s.n_units + 7) / 8 : s.n_units;
    sblk.push_back(s);
  }

  // Group sums of g^2 of the low-rank blocks come from the reduction kernels, except on the tensor path when
  // there is a refit pass: its row panels read every row of g anyway and leave the row sums behind.
  const bool fold_sumsq = K_eff > 0 && !(hp->flags & ADAPM_FLAG_NO_SUMSQ_FOLD);
  const bool with_hold = hp->refresh_period > 1 && K_eff > 0;
  for (int pass = 0; pass < 2; ++pass) {
    if (pass == 1 && fold_sumsq && !with_hold) break;
    for (int64_t i : (pass == 0 ? lowrank_ids : tc_ids)) {
      const adapm_block& b = c->blocks[i];
      if (b.v_mode != ADAPM_V_BLOCKMEAN) continue;
      const int64_t numel = (int64_t)b.rows * b.cols;
      const int64_t group_elems = b.v_group_rows == 0 ? numel : (int64_t)b.v_group_rows * b.cols;
      add_reduce_job((pass == 1 && fold_sumsq) ? rset_hold : rset_all, (int)i, group_elems, numel / group_elems);
    }
  }

  auto& prog = c->program;
  // Global gradient-norm clipping (and the finite check, which rides on the same reduction) needs the norm of
  // every gradient before anything uses one: a pass of its own over g.
  const bool clip_on = hp->max_grad_norm > 0.f && std::isfinite(hp->max_grad_norm);
  if (clip_on || (hp->flags & ADAPM_FLAG_CHECK_FINITE)) {
    std::vector<NormRange> ranges;
    std::vector<int32_t> cta_range;
    for (int i = 0; i < n; ++i) {
      const adapm_block& b = c->blocks[i];
      NormRange r{b.offset, (int64_t)b.rows * b.cols, (int64_t)cta_range.size()};
      for (int64_t q = 0; q < (r.numel + kNormChunk - 1) / kNormChunk; ++q) cta_range.push_back((int32_t)ranges.size());
      ranges.push_back(r);
    }
    Launch GN{LK_GRADNORM, append_table(c->h_tables, ranges), (int64_t)ranges.size(), (int64_t)cta_range.size()};
    GN.aux0 = append_table(c->h_tables, cta_range);
    GN.aux1 = work_cursor;                                   // per-chunk sums
    work_cursor += round_up((int64_t)cta_range.size(), kStateAlign);
    prog.push_back(GN);
    c->use_gscale = 1;
  }
  for (int which = 0; which < 2; ++which) {
    const ReduceSet& rs = which ? rset_hold : rset_all;
    const std::vector<ReduceJob>& rjobs = rs.jobs;
    if (rjobs.empty()) continue;
    const int64_t off = append_table(c->h_tables, rjobs);
    // CTA index -> job of the CTA's first unit (the job table is sorted by first_unit), so that a warp finds its job
    // with a step or two instead of a binary search
    std::vector<int32_t> cta_job((size_t)((rs.units + 7) / 8));
    for (size_t q = 0, j = 0; q < cta_job.size(); ++q) {
      while (j + 1 < rjobs.size() && rjobs[j + 1].first_unit <= (int64_t)q * 8) ++j;
      cta_job[q] = (int32_t)j;
    }
    Launch RP{LK_REDUCE_PARTIAL, off, (int64_t)rjobs.size(), (rs.units + 7) / 8, rs.units};
    RP.aux1 = append_table(c->h_tables, cta_job);
    RP.phase = which ? 2 : 0;
    prog.push_back(RP);
    Launch RF{LK_REDUCE_FINAL, off, (int64_t)rjobs.size(), (rs.groups + 7) / 8, rs.groups};
    RF.phase = RP.phase;
    prog.push_back(RF);
  }
  if (!sblk.empty()) {
    const int64_t off = append_table(c->h_tables, sblk);
    std::vector<int32_t> cta_blk((size_t)cta_cursor);       // CTA index -> entry of the block table
    for (size_t i = 0; i < sblk.size(); ++i) {
      const int64_t end = i + 1 < sblk.size() ? sblk[i + 1].first_cta : cta_cursor;
      for (int64_t q = sblk[i].first_cta; q < end; ++q) cta_blk[(size_t)q] = (int32_t)i;
    }
    Launch SL{LK_STREAM, off, (int64_t)sblk.size(), cta_cursor};
    SL.aux0 = append_table(c->h_tables, cta_blk);
    prog.push_back(SL);
  }

  // ---- low-rank program --------------------------------------------------------------------------
  if (!lowrank_ids.empty() || !tc_ids.empty()) {
    std::vector<InitJob> ijobs;
    for (int pass = 0; pass < 2; ++pass)
      for (int64_t i : (pass == 0 ? lowrank_ids : tc_ids))
        ijobs.push_back({c->l_off[i], i, c->blocks[i].rows, c->blocks[i].rank});
    c->init_table_off = append_table(c->h_tables, ijobs);
    c->n_init_jobs = (int64_t)ijobs.size();
    // Y = g Omega -> the block's L in the state (data-driven L_0)
    c->omega_off.assign(n, -1);
    std::vector<GemmProb> rp;
    int64_t tiles = 0;
    for (int pass = 0; pass < 2; ++pass)
      for (int64_t i : (pass == 0 ? lowrank_ids : tc_ids)) {
        const adapm_block& b = c->blocks[i];
        c->omega_off[i] = c->omega_floats;
        c->omega_floats += round_up((int64_t)b.cols * b.rank, kStateAlign);
        GemmProb p;
        std::memset(&p, 0, sizeof(p));
        p.z1_base = p.z2_base = BASE_NONE;
        p.alpha = 1.f;
        p.x_base = BASE_GRADS; p.x_off = b.offset; p.sxi = b.cols; p.sxk = 1;
        p.y_base = BASE_WORK; p.y_off = c->omega_off[i]; p.syk = b.rank; p.syj = 1;
        p.c_base = BASE_STATE; p.c_off = c->l_off[i]; p.M = b.rows; p.N = b.rank; p.K = b.cols; p.ldc = b.rank;
        p.tiles_n = (p.N + 63) / 64;
        p.first_tile = tiles;
        tiles += (int64_t)((p.M + 63) / 64) * p.tiles_n;
        rp.push_back(p);
      }
    c->range_table_off = append_table(c->h_tables, rp);
    c->n_range_probs = (int64_t)rp.size();
    c->n_range_tiles = tiles;
  }
  if (!tc_ids.empty()) {
    std::vector<ReduceJob> row_jobs;
    int64_t row_groups = 0;
    rc = build_tensor_program(c, tc_ids, etas, work_cursor, row_jobs, row_groups);
    if (rc != ADAPM_OK) { adapm_destroy(c); return rc; }
    if (!row_jobs.empty()) {
      const int64_t off = append_table(c->h_tables, row_jobs);
      for (Launch& L : prog)
        if (L.kind == LK_REDUCE_ROWS) {
          L.table_off = off; L.n_items = (int64_t)row_jobs.size(); L.grid = (row_groups + 7) / 8; L.aux0 = row_groups;
        }
    }
  }
  if (!lowrank_ids.empty()) {
    // workspace: two copies of the [L,R] section (ping-pong iterates), A/B with the same layout, Gram matrices
    c->ws_lr[0] = work_cursor; work_cursor += c->lr_section_floats;
    c->ws_lr[1] = work_cursor; work_cursor += c->lr_section_floats;
    const int64_t ws_ab = work_cursor; work_cursor += c->lr_section_floats;
    std::vector<int64_t> gram_off(n, 0);
    for (int64_t i : lowrank_ids) {
      gram_off[i] = work_cursor;
      work_cursor += round_up((hp->inner_precond ? 6LL : 4LL) * c->blocks[i].rank * c->blocks[i].rank, kStateAlign);
    }
    const float b1 = hp->beta1, a1 = 1.f - hp->beta1;
    int src_base = BASE_STATE; int64_t src_shift = 0;   // where the current iterate lives
    int dst_buf = 0;
    // with a refresh period the passes exist twice: refitting both factors (phase 1) and holding L (phase 2)
    for (int phase = (with_hold ? 1 : 0); phase <= (with_hold ? 2 : 0); ++phase) {
    const bool hold = phase == 2;
    src_base = BASE_STATE; src_shift = 0; dst_buf = 0;
    for (int it = 0; it < K_eff; ++it) {
      const float se = (float)etas[it];
      const int64_t dst_shift = c->ws_lr[dst_buf];
      std::vector<GemmProb> pAB, pG, pU1, pU2, pU3;
      std::vector<InverseJob> inv;
      int64_t tAB = 0, tG = 0, tU1 = 0, tU2 = 0, tU3 = 0;
      const bool precond = hp->inner_precond != 0;
      auto push = [](std::vector<GemmProb>& v, GemmProb p, int64_t& tiles) {
        p.tiles_n = (p.N + 63) / 64;
        p.first_tile = tiles;
        tiles += (int64_t)((p.M + 63) / 64) * p.tiles_n;
        v.push_back(p);
      };
      for (int64_t i : lowrank_ids) {
        const adapm_block& b = c->blocks[i];
        const int m = b.rows, nn = b.cols, r = b.rank;
        const int64_t Lc = src_shift + c->l_off[i], Rc = src_shift + c->r_off[i];   // current iterate
        const int64_t L0 = c->l_off[i], R0 = c->r_off[i];                             // previous factors (state)
        const int64_t Ld = dst_shift + c->l_off[i], Rd = dst_shift + c->r_off[i];
        const int64_t Aw = ws_ab + c->l_off[i], Bw = ws_ab + c->r_off[i];
        const int64_t G1 = gram_off[i], G2 = G1 + (int64_t)r * r, G3 = G2 + (int64_t)r * r, G4 = G3 + (int64_t)r * r;
        GemmProb p;
        auto reset = [&]() {
          std::memset(&p, 0, sizeof(p));
          p.z1_base = p.z2_base = BASE_NONE;
          p.alpha = 1.f;
        };
        // A = g R^T  (m x r), contraction over n
        reset(); p.x_base = BASE_GRADS; p.x_off = b.offset; p.sxi = nn; p.sxk = 1;
        p.y_base = (int8_t)src_base; p.y_off = Rc; p.syk = 1; p.syj = nn;
        p.c_base = BASE_WORK; p.c_off = Aw; p.M = m; p.N = r; p.K = nn; p.ldc = r; if (!hold) push(pAB, p, tAB);
        // B = L^T g  (r x n), contraction over m
        reset(); p.x_base = (int8_t)src_base; p.x_off = Lc; p.sxi = 1; p.sxk = r;
        p.y_base = BASE_GRADS; p.y_off = b.offset; p.syk = nn; p.syj = 1;
        p.c_base = BASE_WORK; p.c_off = Bw; p.M = r; p.N = nn; p.K = m; p.ldc = nn; push(pAB, p, tAB);
        // G1 = R R^T, G2 = R0 R^T  (contraction over n)
        reset(); p.x_base = (int8_t)src_base; p.x_off = Rc; p.sxi = nn; p.sxk = 1;
        p.y_base = (int8_t)src_base; p.y_off = Rc; p.syk = 1; p.syj = nn;
        p.c_base = BASE_WORK; p.c_off = G1; p.M = r; p.N = r; p.K = nn; p.ldc = r; if (!hold) push(pG, p, tG);
        p.x_base = BASE_STATE; p.x_off = R0; p.c_off = G2; if (!hold) push(pG, p, tG);
        // G3 = L^T L, G4 = L^T L0  (contraction over m)
        reset(); p.x_base = (int8_t)src_base; p.x_off = Lc; p.sxi = 1; p.sxk = r;
        p.y_base = (int8_t)src_base; p.y_off = Lc; p.syk = r; p.syj = 1;
        p.c_base = BASE_WORK; p.c_off = G3; p.M = r; p.N = r; p.K = m; p.ldc = r; push(pG, p, tG);
        p.y_base = BASE_STATE; p.y_off = L0; p.c_off = G4; push(pG, p, tG);
        if (precond) {
          // Preconditioned pass: A <- L G1 - a1 A, A <- A - b1 L0 G2 (= dl/dL), L' = L - se A S1 with
          // S1 = (G1 + d I)^-1; B <- G3 R - a1 B, B <- B - b1 G4 R0 (= dl/dR), R' = R - se S3 B, S3 = (G3 + d I)^-1.
          const int64_t S1 = G4 + (int64_t)r * r, S3 = S1 + (int64_t)r * r;
          if (!hold) inv.push_back({G1, S1, r, 0});
          inv.push_back({G3, S3, r, 0});
          if (!hold) {
            reset(); p.x_base = (int8_t)src_base; p.x_off = Lc; p.sxi = r; p.sxk = 1;
            p.y_base = BASE_WORK; p.y_off = G1; p.syk = r; p.syj = 1;
            p.c_base = BASE_WORK; p.c_off = Aw; p.M = m; p.N = r; p.K = r; p.ldc = r;
            p.z1_base = BASE_WORK; p.z1_off = Aw; p.c1 = -a1; push(pU1, p, tU1);
            reset(); p.x_base = BASE_STATE; p.x_off = L0; p.sxi = r; p.sxk = 1;
            p.y_base = BASE_WORK; p.y_off = G2; p.syk = r; p.syj = 1;
            p.c_base = BASE_WORK; p.c_off = Aw; p.M = m; p.N = r; p.K = r; p.ldc = r;
            p.alpha = -b1; p.beta = 1.f; push(pU2, p, tU2);
          }
          reset(); p.x_base = BASE_WORK; p.x_off = Aw; p.sxi = r; p.sxk = 1;
          p.y_base = BASE_WORK; p.y_off = S1; p.syk = r; p.syj = 1;
          p.c_base = BASE_WORK; p.c_off = Ld; p.M = m; p.N = r; p.K = r; p.ldc = r;
          p.alpha = -se; p.z1_base = (int8_t)src_base; p.z1_off = Lc; p.c1 = 1.f;
          if (hold) { p.K = 0; p.alpha = 0.f; }                                            // L' = L
          push(pU3, p, tU3);
          reset(); p.x_base = BASE_WORK; p.x_off = G3; p.sxi = r; p.sxk = 1;
          p.y_base = (int8_t)src_base; p.y_off = Rc; p.syk = nn; p.syj = 1;
          p.c_base = BASE_WORK; p.c_off = Bw; p.M = r; p.N = nn; p.K = r; p.ldc = nn;
          p.z1_base = BASE_WORK; p.z1_off = Bw; p.c1 = -a1; push(pU1, p, tU1);
          reset(); p.x_base = BASE_WORK; p.x_off = G4; p.sxi = r; p.sxk = 1;
          p.y_base = BASE_STATE; p.y_off = R0; p.syk = nn; p.syj = 1;
          p.c_base = BASE_WORK; p.c_off = Bw; p.M = r; p.N = nn; p.K = r; p.ldc = nn;
          p.alpha = -b1; p.beta = 1.f; push(pU2, p, tU2);
          reset(); p.x_base = BASE_WORK; p.x_off = S3; p.sxi = r; p.sxk = 1;
          p.y_base = BASE_WORK; p.y_off = Bw; p.syk = nn; p.syj = 1;
          p.c_base = BASE_WORK; p.c_off = Rd; p.M = r; p.N = nn; p.K = r; p.ldc = nn;
          p.alpha = -se; p.z1_base = (int8_t)src_base; p.z1_off = Rc; p.c1 = 1.f; push(pU3, p, tU3);
          continue;
        }
        // L' = L - se ( L G1 - b1 L0 G2 - a1 A )
        reset(); p.x_base = (int8_t)src_base; p.x_off = Lc; p.sxi = r; p.sxk = 1;
        p.y_base = BASE_WORK; p.y_off = G1; p.syk = r; p.syj = 1;
        p.c_base = BASE_WORK; p.c_off = Ld; p.M = m; p.N = r; p.K = r; p.ldc = r;
        p.alpha = -se; p.beta = 0.f; p.z1_base = (int8_t)src_base; p.z1_off = Lc; p.c1 = 1.f;
        p.z2_base = BASE_WORK; p.z2_off = Aw; p.c2 = se * a1;
        if (hold) { p.K = 0; p.alpha = 0.f; p.z2_base = BASE_NONE; p.c2 = 0.f; }      // L' = L
        push(pU1, p, tU1);
        reset(); p.x_base = BASE_STATE; p.x_off = L0; p.sxi = r; p.sxk = 1;
        p.y_base = BASE_WORK; p.y_off = G2; p.syk = r; p.syj = 1;
        p.c_base = BASE_WORK; p.c_off = Ld; p.M = m; p.N = r; p.K = r; p.ldc = r;
        p.alpha = se * b1; p.beta = 1.f; if (!hold) push(pU2, p, tU2);
        // R' = R - se ( G3 R - b1 G4 R0 - a1 B )
        reset(); p.x_base = BASE_WORK; p.x_off = G3; p.sxi = r; p.sxk = 1;
        p.y_base = (int8_t)src_base; p.y_off = Rc; p.syk = nn; p.syj = 1;
        p.c_base = BASE_WORK; p.c_off = Rd; p.M = r; p.N = nn; p.K = r; p.ldc = nn;
        p.alpha = -se; p.beta = 0.f; p.z1_base = (int8_t)src_base; p.z1_off = Rc; p.c1 = 1.f;
        p.z2_base = BASE_WORK; p.z2_off = Bw; p.c2 = se * a1; push(pU1, p, tU1);
        reset(); p.x_base = BASE_WORK; p.x_off = G4; p.sxi = r; p.sxk = 1;
        p.y_base = BASE_STATE; p.y_off = R0; p.syk = nn; p.syj = 1;
        p.c_base = BASE_WORK; p.c_off = Rd; p.M = r; p.N = nn; p.K = r; p.ldc = nn;
        p.alpha = se * b1; p.beta = 1.f; push(pU2, p, tU2);
      }
      for (auto* pv : {&pAB, &pG, &pU1, &pU2, &pU3}) {
        if (pv == &pU1 && !inv.empty()) {       // the inverses need the Gram matrices and feed the last update
          Launch IL{LK_SPD_INVERSE, append_table(c->h_tables, inv), (int64_t)inv.size(), (int64_t)inv.size()};
          IL.phase = phase;
          prog.push_back(IL);
        }
        if (pv->empty()) continue;
        const int64_t tiles = pv == &pAB ? tAB : (pv == &pG ? tG : (pv == &pU1 ? tU1 : (pv == &pU2 ? tU2 : tU3)));
        Launch GL{LK_GEMM, append_table(c->h_tables, *pv), (int64_t)pv->size(), tiles};
        GL.phase = phase;
        prog.push_back(GL);
      }
      src_base = BASE_WORK; src_shift = dst_shift;
      c->final_lr_buf = dst_buf;
      dst_buf ^= 1;
    }
    }
    // apply
    std::vector<ApplyBlk> ab;
    int64_t tiles = 0;
    for (int64_t i : lowrank_ids) {
      const adapm_block& b = c->blocks[i];
      ApplyBlk a;
      std::memset(&a, 0, sizeof(a));
      a.off = b.offset; a.l0_off = c->l_off[i]; a.r0_off = c->r_off[i];
      a.l1_base = src_base; a.l1_off = src_shift + c->l_off[i]; a.r1_off = src_shift + c->r_off[i];
      a.v_off = c->v_off[i]; a.rows = b.rows; a.cols = b.cols; a.rank = b.rank; a.v_mode = b.v_mode;
      a.v_group_rows = b.v_group_rows == 0 ? b.rows : b.v_group_rows;
      a.lr_scale = b.lr_scale; a.wd = b.weight_decay;
      a.tiles_n = (b.cols + 63) / 64; a.first_tile = tiles;
      tiles += (int64_t)((b.rows + 63) / 64) * a.tiles_n;
      ab.push_back(a);
    }
    prog.push_back({LK_APPLY_SIMT, append_table(c->h_tables, ab), (int64_t)ab.size(), tiles});
    if (c->final_lr_buf >= 0) {
      // the refitted factors go back to the state, sub-buffer by sub-buffer (the padding between them is not touched)
      std::vector<NormRange> ranges;
      std::vector<int32_t> cta_range;
      for (int64_t i : lowrank_ids) {
        const adapm_block& b = c->blocks[i];
        for (int which = 0; which < 2; ++which) {
          NormRange r{which ? c->r_off[i] : c->l_off[i], (int64_t)b.rank * (which ? b.cols : b.rows), (int64_t)cta_range.size()};
          for (int64_t q = 0; q < (r.numel + kNormChunk - 1) / kNormChunk; ++q) cta_range.push_back((int32_t)ranges.size());
          ranges.push_back(r);
        }
      }
      Launch CM{LK_COMMIT, append_table(c->h_tables, ranges), (int64_t)ranges.size(), (int64_t)cta_range.size()};
      CM.aux0 = append_table(c->h_tables, cta_range);
      prog.push_back(CM);
    }
  }
  c->work_floats = work_cursor;

  // ---- upload ------------------------------------------------------------------------------------
  cudaError_t e = cudaGetDevice(&c->device);
  if (e == cudaSuccess) e = cudaMalloc((void**)&c->d_tables, std::max<size_t>(c->h_tables.size(), 16));
  if (e == cudaSuccess && !c->h_tables.empty())
    e = cudaMemcpy(c->d_tables, c->h_tables.data(), c->h_tables.size(), cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMalloc((void**)&c->d_status, 256);
  if (e == cudaSuccess) e = cudaMemset(c->d_status, 0, 256);
  if (e == cudaSuccess && c->use_gscale) {
    const float ones[2] = {1.f, 1.f};
    e = cudaMalloc((void**)&c->d_gscale, 256);
    if (e == cudaSuccess) e = cudaMemcpy(c->d_gscale, ones, sizeof(ones), cudaMemcpyHostToDevice);
  }
  {
    std::vector<unsigned char> probe;
    const size_t pb = probe_table(probe);
    if (e == cudaSuccess) e = cudaMalloc((void**)&c->d_probe, pb);
    if (e == cudaSuccess) e = cudaMemcpy(c->d_probe, probe.data(), pb, cudaMemcpyHostToDevice);
  }
  if (e != cudaSuccess) {
    set_cuda_error(e, "adapm_create upload");
    adapm_destroy(c);
    return ADAPM_ECUDA;
  }
  *out = c;
  return ADAPM_OK;
}

extern "C" void adapm_destroy(adapm_ctx* c) {
  if (!c) return;
  destroy_tensor_program(c);
  for (auto e : c->prof_events) if (e) cudaEventDestroy(e);
  if (c->d_tables) cudaFree(c->d_tables);
  if (c->d_status) cudaFree(c->d_status);
  if (c->d_probe) cudaFree(c->d_probe);
  if (c->d_gscale) cudaFree(c->d_gscale);
  delete c;
}

extern "C" size_t adapm_state_bytes(const adapm_ctx* c) { return c ? (size_t)c->state_floats * 4 : 0; }

extern "C" int adapm_state_breakdown(const adapm_ctx* c, size_t* full_m, size_t* L, size_t* R, size_t* v) {
  if (!c) return ADAPM_EINVAL;
  if (full_m) *full_m = c->bytes_m;
  if (L) *L = c->bytes_L;
  if (R) *R = c->bytes_R;
  if (v) *v = c->bytes_v;
  return ADAPM_OK;
}

extern "C" int adapm_state_layout(const adapm_ctx* c, int64_t block, int which, int64_t* offset, int64_t* count) {
  if (!c || !offset || !count) return ADAPM_EINVAL;
  if (block < 0 || block >= (int64_t)c->blocks.size()) return ADAPM_ERANGE;
  const adapm_block& b = c->blocks[block];
  int64_t off = -1, cnt = 0;
  switch (which) {
    case ADAPM_STATE_M: off = c->m_off[block]; cnt = off >= 0 ? (int64_t)b.rows * b.cols : 0; break;
    case ADAPM_STATE_L: off = c->l_off[block]; cnt = off >= 0 ? (int64_t)b.rows * b.rank : 0; break;
    case ADAPM_STATE_R: off = c->r_off[block]; cnt = off >= 0 ? (int64_t)b.rank * b.cols : 0; break;
    case ADAPM_STATE_V: off = c->v_off[block]; cnt = c->v_cnt[block]; break;
    default: return ADAPM_EINVAL;
  }
  *offset = off;
  *count = cnt;
  return ADAPM_OK;
}

extern "C" size_t adapm_workspace_bytes(const adapm_ctx* c) { return c ? (size_t)c->work_floats * 4 : 0; }

extern "C" int adapm_set_workspace(adapm_ctx* c, void* dev_ptr, size_t bytes) {
  if (!c) return ADAPM_EINVAL;
  if (c->work_floats > 0) {
    if (!dev_ptr) return ADAPM_EINVAL;
    if ((uintptr_t)dev_ptr % 256) return ADAPM_EALIGN;
    if (bytes < (size_t)c->work_floats * 4) return ADAPM_ENOWORKSPACE;
  }
  c->workspace = dev_ptr;
  c->workspace_bytes = bytes;
  return ADAPM_OK;
}

extern "C" int adapm_state_init(adapm_ctx* c, void* state, adapm_stream stream) {
  if (!c || !state) return ADAPM_EINVAL;
  if ((uintptr_t)state % 256) return ADAPM_EALIGN;
  cudaStream_t s = (cudaStream_t)stream;
  ADAPM_CUDA(cudaMemsetAsync(state, 0, (size_t)c->state_floats * 4, s));
  tensor_state_changed(c);
  if (c->n_init_jobs > 0)
    return launch_init_L0((const InitJob*)(c->d_tables + c->init_table_off), c->n_init_jobs, (float*)state, c->hp.seed, 1, s);
  return ADAPM_OK;
}

extern "C" int64_t adapm_init_omega_floats(const adapm_ctx* c) { return c ? c->omega_floats : 0; }

extern "C" int adapm_init_omega_layout(const adapm_ctx* c, int64_t block, int64_t* offset, int64_t* count) {
  if (!c || !offset || !count) return ADAPM_EINVAL;
  if (block < 0 || block >= (int64_t)c->blocks.size()) return ADAPM_ERANGE;
  const bool lowrank = !c->omega_off.empty() && c->omega_off[(size_t)block] >= 0;
  *offset = lowrank ? c->omega_off[(size_t)block] : 0;
  *count = lowrank ? (int64_t)c->blocks[(size_t)block].cols * c->blocks[(size_t)block].rank : 0;
  return ADAPM_OK;
}

extern "C" int adapm_state_init_from_grads(adapm_ctx* c, void* state, const void* grads, const float* omega,
                                           adapm_stream stream) {
  if (!c || !state || !grads) return ADAPM_EINVAL;
  if (c->n_init_jobs > 0 && !omega) return ADAPM_EINVAL;
  if ((uintptr_t)state % 256 || (uintptr_t)grads % 16 || (uintptr_t)omega % 16) return ADAPM_EALIGN;
  cudaStream_t s = (cudaStream_t)stream;
  ADAPM_CUDA(cudaMemsetAsync(state, 0, (size_t)c->state_floats * 4, s));
  tensor_state_changed(c);
  if (c->n_init_jobs == 0) return ADAPM_OK;
  Bases b;
  b.p[BASE_PARAMS] = nullptr; b.p[BASE_GRADS] = const_cast<void*>(grads); b.p[BASE_STATE] = state;
  b.p[BASE_WORK] = const_cast<float*>(omega);
  b.status = c->d_status; b.gscale = nullptr; b.shadow = nullptr;
  const int rc = launch_gemm((const GemmProb*)(c->d_tables + c->range_table_off), c->n_range_probs, c->n_range_tiles, b,
                             c->hp.grad_dtype, s);
  if (rc != ADAPM_OK) return rc;
  return launch_init_L0((const InitJob*)(c->d_tables + c->init_table_off), c->n_init_jobs, (float*)state, c->hp.seed, 0, s);
}

extern "C" int adapm_set_lr(adapm_ctx* c, float lr) {
  if (!c || !std::isfinite(lr)) return ADAPM_EINVAL;
  c->hp.lr = lr;
  return ADAPM_OK;
}

extern "C" size_t adapm_step_bytes(const adapm_ctx* c) { return c ? c->step_bytes : 0; }
extern "C" double adapm_step_flops(const adapm_ctx* c) { return c ? c->step_flops : 0.0; }
extern "C" int64_t adapm_launch_count(const adapm_ctx* c) {
  if (!c) return 0;
  if (c->last_step_launches > 0) return c->last_step_launches;
  int64_t n = 0;
  for (const Launch& L : c->program)
    if ((L.when == WHEN_ALWAYS || L.when == WHEN_EVEN) && !L.only_convert && L.phase != 2) ++n;
  return n;
}

extern "C" int adapm_set_shadow_params(adapm_ctx* c, void* bf16_dev_ptr) {
  if (!c) return ADAPM_EINVAL;
  if ((uintptr_t)bf16_dev_ptr % 256) return ADAPM_EALIGN;
  c->shadow = bf16_dev_ptr;
  return ADAPM_OK;
}

extern "C" int adapm_state_changed(adapm_ctx* c) {
  if (!c) return ADAPM_EINVAL;
  tensor_state_changed(c);
  return ADAPM_OK;
}

extern "C" int adapm_selftest_expired_wait(adapm_ctx* c, adapm_stream stream) {
  if (!c) return ADAPM_EINVAL;
  return run_expired_wait_probe(c, (cudaStream_t)stream);
}

extern "C" int adapm_step(adapm_ctx* c, void* params, const void* grads, void* state, int64_t t, adapm_stream stream) {
  if (!c || !params || !grads || !state || t < 1) return ADAPM_EINVAL;
  if ((uintptr_t)params % 256 || (uintptr_t)grads % 256 || (uintptr_t)state % 256) return ADAPM_EALIGN;
  if (c->work_floats > 0 && (!c->workspace || c->workspace_bytes < (size_t)c->work_floats * 4)) return ADAPM_ENOWORKSPACE;
  cudaStream_t s = (cudaStream_t)stream;
  const adapm_hparams& hp = c->hp;

  StepScalars sc;
  sc.lr = hp.lr; sc.beta1 = hp.beta1; sc.beta2 = hp.beta2; sc.eps = hp.eps; sc.clip = hp.clip;
  if (hp.adam_debias) {
    sc.inv_bc1 = (float)(1.0 / (1.0 - std::pow((double)hp.beta1, (double)t)));
    sc.inv_bc2 = (float)(1.0 / (1.0 - std::pow((double)hp.beta2, (double)t)));
  } else {
    sc.inv_bc1 = sc.inv_bc2 = 1.f;
  }
  if (hp.correction) {            // m^c = g + c (P_{t-1} - P_t), c = beta1 / (1 - beta1): lines 4, 6, 8 combined
    const float cc = hp.beta1 / (1.f - hp.beta1);
    sc.cg = 1.f; sc.c0 = cc; sc.c1 = cc;
  } else {                        // m^c = m_t = (1-beta1) g + beta1 P_{t-1}
    sc.cg = 1.f - hp.beta1; sc.c0 = hp.beta1; sc.c1 = 0.f;
  }

  Bases b;
  b.p[BASE_PARAMS] = params; b.p[BASE_GRADS] = const_cast<void*>(grads); b.p[BASE_STATE] = state;
  b.p[BASE_WORK] = c->workspace;
  b.status = c->d_status; b.gscale = c->d_gscale; b.shadow = (uint16_t*)c->shadow;
  float* work = (float*)c->workspace;

  // refresh period T: both factors are refitted at steps 1, T+1, 2T+1, ...; the steps in between hold L
  const bool refresh = hp.refresh_period <= 1 || (t - 1) % hp.refresh_period == 0;
  int parity = 0, convert = 0;
  if (c->tc) {
    const int prc = tensor_prepare_step(c, b, t, s, &parity, &convert);
    if (prc != ADAPM_OK) return prc;
  }
  const bool prof = c->profiling && c->prof_events.size() == c->program.size() + 1;
  if (prof) {
    c->prof_kinds.clear();
    ADAPM_CUDA(cudaEventRecord(c->prof_events[0], s));
  }
  size_t li = 0;
  for (const Launch& L : c->program) {
    if ((L.only_convert && !convert) || (L.when == WHEN_EVEN && parity != 0) || (L.when == WHEN_ODD && parity != 1) ||
        (L.phase == 1 && !refresh) || (L.phase == 2 && refresh))
      continue;
    const unsigned char* tab = c->d_tables + L.table_off;
    int rc = ADAPM_OK;
    if (prof) nvtxRangePushA(adapm_launch_kind_name((int32_t)L.kind));   // a named range per launch for timeline tools
    switch (L.kind) {
      case LK_GRADNORM:
        rc = launch_gradnorm((const NormRange*)tab, (const int32_t*)(c->d_tables + L.aux0), L.grid, grads, hp.grad_dtype,
                             work + L.aux1, std::isfinite(hp.max_grad_norm) ? hp.max_grad_norm : 0.f,
                             (hp.flags & ADAPM_FLAG_CHECK_FINITE) ? 1 : 0, c->d_gscale, c->d_status, s);
        break;
      case LK_REDUCE_PARTIAL:
        rc = launch_reduce_partial((const ReduceJob*)tab, (const int32_t*)(c->d_tables + L.aux1), L.n_items, L.aux0, grads,
                                   work, hp.grad_dtype, c->d_status, s);
        break;
      case LK_REDUCE_FINAL:
      case LK_REDUCE_ROWS:
        rc = launch_reduce_final((const ReduceJob*)tab, L.n_items, L.aux0, (float*)state, work, hp.beta2, c->d_status,
                                 c->d_gscale, s);
        break;
      case LK_STREAM:
        rc = launch_stream((const StreamBlk*)tab, (const int32_t*)(c->d_tables + L.aux0), L.grid, b, sc, hp.grad_dtype, s);
        break;
      case LK_SPD_INVERSE:
        rc = launch_spd_inverse((const InverseJob*)tab, L.n_items, work, hp.precond_damping, c->d_status, s); break;
      case LK_GEMM:
        rc = launch_gemm((const GemmProb*)tab, L.n_items, L.grid, b, hp.grad_dtype, s); break;
      case LK_APPLY_SIMT:
        rc = launch_apply_simt((const ApplyBlk*)tab, L.n_items, L.grid, b, sc, hp.grad_dtype, s); break;
      case LK_COMMIT:
        rc = launch_copy_ranges((const NormRange*)tab, (const int32_t*)(c->d_tables + L.aux0), L.grid, (float*)state,
                                work + c->ws_lr[c->final_lr_buf], c->d_status, s);
        break;
      default:
        rc = run_tensor_launch(c, L, b, sc, parity, s); break;
    }
    if (prof) nvtxRangePop();
    if (rc != ADAPM_OK) return rc;
    ++li;
    if (prof) {
      c->prof_kinds.push_back((int32_t)L.kind);
      ADAPM_CUDA(cudaEventRecord(c->prof_events[li], s));
    }
  }
  c->last_step_launches = (int64_t)li;
  if (prof) c->prof_valid = 1;
  return ADAPM_OK;
}

extern "C" int adapm_set_profiling(adapm_ctx* c, int32_t on) {
  if (!c) return ADAPM_EINVAL;
  if (on && c->prof_events.empty()) {
    c->prof_events.resize(c->program.size() + 1, nullptr);
    for (auto& e : c->prof_events) ADAPM_CUDA(cudaEventCreate(&e));
  }
  c->profiling = on ? 1 : 0;
  c->prof_valid = 0;
  return ADAPM_OK;
}

extern "C" int adapm_get_launch_times(adapm_ctx* c, float* ms, int32_t* kinds, int64_t capacity, int64_t* n_out) {
  if (!c || !n_out) return ADAPM_EINVAL;
  // the launches of the last profiled step (a step runs a subset of the program: see LaunchWhen)
  const size_t n = c->prof_valid ? c->prof_kinds.size() : c->program.size();
  *n_out = (int64_t)n;
  if (!ms && !kinds) return ADAPM_OK;
  if (capacity < (int64_t)n) return ADAPM_ERANGE;
  if (!c->prof_valid) return ADAPM_EINVAL;
  ADAPM_CUDA(cudaEventSynchronize(c->prof_events[n]));
  for (size_t i = 0; i < n; ++i) {
    if (ms) ADAPM_CUDA(cudaEventElapsedTime(&ms[i], c->prof_events[i], c->prof_events[i + 1]));
    if (kinds) kinds[i] = c->prof_kinds[i];
  }
  return ADAPM_OK;
}

extern "C" const char* adapm_launch_kind_name(int32_t kind) {
  switch (kind) {
    case LK_REDUCE_PARTIAL: return "reduce_partial";
    case LK_REDUCE_FINAL: return "reduce_final";
    case LK_REDUCE_ROWS: return "reduce_rows";
    case LK_GRADNORM: return "grad_norm";
    case LK_TC_COPY: return "tc_copy";
    case LK_STREAM: return "stream_update";
    case LK_GEMM: return "gemm_simt";
    case LK_SPD_INVERSE: return "spd_inverse";
    case LK_APPLY_SIMT: return "apply_simt";
    case LK_COMMIT: return "commit_copy";
    case LK_TC_CONVERT: return "tc_convert";
    case LK_TC_CONVERT_WORK: return "tc_convert_work";
    case LK_TC_PANEL: return "tc_panel";
    case LK_TC_GRAM: return "tc_gram";
    case LK_TC_APPLY: return "tc_apply";
    default: return "unknown";
  }
}

extern "C" int adapm_get_status(adapm_ctx* c, adapm_stream stream, int32_t* status) {
  if (!c || !status) return ADAPM_EINVAL;
  cudaStream_t s = (cudaStream_t)stream;
  int32_t h = 0;
  ADAPM_CUDA(cudaMemcpyAsync(&h, c->d_status, sizeof(h), cudaMemcpyDeviceToHost, s));
  ADAPM_CUDA(cudaStreamSynchronize(s));
  if (h != 0) {
    ADAPM_CUDA(cudaMemsetAsync(c->d_status, 0, sizeof(h), s));
    // steps issued while the word was set wrote nothing, so the bf16 copies of the factors no longer follow the
    // step numbers the host has counted: rebuild them from the state at the next step
    tensor_state_changed(c);
  }
  *status = h;
  return h == 0 ? ADAPM_OK : ADAPM_EDEVICE;
}

extern "C" size_t adapm_group_meansq_scratch_bytes(int64_t n_groups, int64_t group_elems) {
  if (n_groups <= 0 || group_elems <= 0) return 0;
  const int64_t cpg = (group_elems + kWarpUnitMax - 1) / kWarpUnitMax;
  return (size_t)round_up(n_groups * cpg, kStateAlign) * 4;
}

extern "C" int adapm_group_meansq(const void* g, int32_t grad_dtype, int64_t n_groups, int64_t group_elems, float* out,
                                  void* scratch, size_t scratch_bytes, adapm_stream stream) {
  if (!g || !out || !scratch || n_groups <= 0 || group_elems <= 0) return ADAPM_EINVAL;
  if (grad_dtype != ADAPM_GRAD_F32 && grad_dtype != ADAPM_GRAD_BF16) return ADAPM_EINVAL;
  if ((uintptr_t)g % 16 || (uintptr_t)scratch % 256) return ADAPM_EALIGN;
  if (scratch_bytes < adapm_group_meansq_scratch_bytes(n_groups, group_elems)) return ADAPM_ENOWORKSPACE;
  const int64_t cpg = (group_elems + kWarpUnitMax - 1) / kWarpUnitMax;
  if (cpg > INT32_MAX) return ADAPM_ERANGE;
  cudaStream_t s = (cudaStream_t)stream;
  int rc = launch_meansq_partial(g, grad_dtype, n_groups, group_elems, (int)cpg, (float*)scratch, s);
  if (rc != ADAPM_OK) return rc;
  return launch_meansq_final((const float*)scratch, n_groups, group_elems, (int)cpg, out, s);
}
