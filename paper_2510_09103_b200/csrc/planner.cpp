// Default block-partition planner (host, integers only) and the error-string table.
//
// Section 4.1 of the paper: (1) embedding and attention-output blocks get no momentum, (2) query,
// key and MLP blocks get low-rank momentum with the residual correction, (3) value blocks keep full
// momentum.  Section 5.1: rank = 5% of the full rank, learning rate x0.75 for blocks without momentum.
#include <cstring>

#include "adapm.h"

namespace {

constexpr int64_t kAlign = 8;

int64_t align_up(int64_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

int32_t pick_rank(int64_t rows, int64_t cols, int32_t pct, int32_t override_rank) {
  const int64_t lo = rows < cols ? rows : cols;
  if (override_rank > 0) return (int32_t)(override_rank < lo ? override_rank : lo);
  const int64_t r = (int64_t)pct * lo / 100;
  return (int32_t)(r < 1 ? 1 : r);
}

struct Piece {
  int32_t role;
  int64_t row0, rows;
};

}  // namespace

extern "C" int adapm_plan_default(const adapm_tensor* tensors, int64_t n_tensors, int32_t rank_pct,
                                  int32_t rank_override, int32_t v_mode, float weight_decay, adapm_block* out,
                                  int64_t out_capacity, int64_t* n_out, int64_t* total_elems) {
  if (!tensors || n_tensors <= 0 || !n_out) return ADAPM_EINVAL;
  if (v_mode != ADAPM_V_ELEMENT && v_mode != ADAPM_V_BLOCKMEAN) return ADAPM_EINVAL;
  if (rank_pct < 0 || rank_pct > 100 || rank_override < 0) return ADAPM_ERANGE;
  int64_t cursor = 0, count = 0;
  for (int64_t ti = 0; ti < n_tensors; ++ti) {
    const adapm_tensor& t = tensors[ti];
    if (t.rows < 1 || t.cols < 1 || t.rows > INT32_MAX || t.cols > INT32_MAX) return ADAPM_ERANGE;
    cursor = align_up(cursor);
    Piece pieces[3];
    int np = 1;
    if (t.role == ADAPM_ROLE_QKV_FUSED) {
      if (t.rows % 3) return ADAPM_EINVAL;
      const int64_t d = t.rows / 3;
      pieces[0] = {ADAPM_ROLE_Q, 0, d};
      pieces[1] = {ADAPM_ROLE_K, d, d};
      pieces[2] = {ADAPM_ROLE_V, 2 * d, d};
      np = 3;
    } else {
      pieces[0] = {t.role, 0, t.rows};
    }
    for (int p = 0; p < np; ++p) {
      adapm_block b;
      std::memset(&b, 0, sizeof(b));
      b.offset = cursor + pieces[p].row0 * t.cols;
      if (b.offset % kAlign) return ADAPM_EALIGN;
      b.rows = (int32_t)pieces[p].rows;
      b.cols = (int32_t)t.cols;
      b.lr_scale = 1.0f;
      b.weight_decay = weight_decay;
      int32_t group_rows = 1;
      switch (pieces[p].role) {
        case ADAPM_ROLE_EMBED:
        case ADAPM_ROLE_LM_HEAD:
        case ADAPM_ROLE_ATTN_OUT:
          b.mom_mode = ADAPM_MOM_NONE;
          b.lr_scale = 0.75f;
          break;
        case ADAPM_ROLE_Q:
        case ADAPM_ROLE_K:
          b.mom_mode = ADAPM_MOM_LOWRANK;
          if (t.heads > 0 && b.rows % t.heads == 0) group_rows = b.rows / t.heads;
          break;
        case ADAPM_ROLE_MLP:
          b.mom_mode = ADAPM_MOM_LOWRANK;
          break;
        case ADAPM_ROLE_V:
        case ADAPM_ROLE_OTHER:
          b.mom_mode = ADAPM_MOM_FULL;
          break;
        case ADAPM_ROLE_VECTOR:
          b.mom_mode = ADAPM_MOM_FULL;
          b.weight_decay = 0.0f;
          group_rows = 0;
          break;
        default:
          return ADAPM_EINVAL;
      }
      if (b.mom_mode == ADAPM_MOM_LOWRANK) b.rank = pick_rank(b.rows, b.cols, rank_pct, rank_override);
      b.v_mode = v_mode;
      b.v_group_rows = (v_mode == ADAPM_V_BLOCKMEAN) ? group_rows : 0;
      if (out) {
        if (count >= out_capacity) return ADAPM_ERANGE;
        out[count] = b;
      }
      ++count;
    }
    cursor += t.rows * t.cols;
  }
  *n_out = count;
  if (total_elems) *total_elems = align_up(cursor);
  return ADAPM_OK;
}

extern "C" const char* adapm_strerror(int code) {
  switch (code) {
    case ADAPM_OK: return "ok";
    case ADAPM_EINVAL: return "invalid argument";
    case ADAPM_EALIGN: return "offset or pointer not aligned";
    case ADAPM_ERANGE: return "value out of range";
    case ADAPM_ECUDA: return "CUDA call failed";
    case ADAPM_ENOWORKSPACE: return "workspace missing or too small";
    case ADAPM_EUNSUPPORTED: return "not supported by the requested kernel path";
    case ADAPM_EDEVICE: return "a kernel reported an expired wait";
    default: return "unknown error";
  }
}

extern "C" int adapm_version(void) { return 201; }
