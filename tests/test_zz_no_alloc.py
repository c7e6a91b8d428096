"""adapm_group_meansq_static: the block mean of g^2 for callers that cannot allocate device memory
(hosts whose allocator owns the whole GPU, plug-in callbacks that are not allowed to allocate).

It must give what adapm_group_meansq gives with caller-provided scratch, call after call, although
all calls share one fixed scratch array inside the library.  The file sorts last on purpose: a run
that stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest

import workloads as WL
import paper_2510_09103_b200 as A
from oracle import adapm_oracle as O

pytestmark = pytest.mark.gpu


def _device_grad(x, dtype):
    import torch
    vals, raw = WL.to_grad_dtype(x, dtype)
    return vals, torch.from_numpy(raw.view(np.int16) if dtype == "bf16" else raw).cuda()


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_static_scratch_matches_caller_scratch_on_two_calls_in_a_row(dtype):
    import torch
    gd = A.GRAD_BF16 if dtype == "bf16" else A.GRAD_F32
    rng = np.random.default_rng(11)
    # second call is smaller than the first, so it sees the first call's leftovers in the shared array
    shapes = [(37, 70001), (5, 4100)]
    for n_groups, ge in shapes:
        vals, g = _device_grad((rng.standard_normal(n_groups * ge) * 1e-3).astype(np.float32), dtype)
        want = torch.zeros(n_groups, device="cuda")
        scratch = torch.zeros(max(A.adapm_group_meansq_scratch_bytes(n_groups, ge) // 4, 64), device="cuda")
        A.adapm_group_meansq(g, gd, n_groups, ge, want, scratch)
        got = torch.full((n_groups,), -1.0, device="cuda")
        A.adapm_group_meansq_static(g, gd, n_groups, ge, got)
        torch.cuda.synchronize()
        w, h = want.cpu().numpy().astype(np.float64), got.cpu().numpy().astype(np.float64)
        assert np.isfinite(h).all() and (h > 0).all()
        assert np.abs(h - w).max() <= 1e-5 * np.abs(w).max()
        # and against the definition itself: the group average of g^2 (the oracle's second moment from v = 0)
        blk = O.Block(n_groups, ge, O.MOM_NONE, v_mode=O.V_BLOCKMEAN, v_group_rows=1)
        ref = O.second_moment(np.zeros(n_groups), vals.astype(np.float64).reshape(n_groups, ge), blk, 0.0)
        assert np.abs(h - ref).max() <= 1e-5 * np.abs(ref).max()


def test_static_scratch_rejects_inputs_beyond_its_limit():
    import torch
    g = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(8, device="cuda")
    with pytest.raises(A.AdapmError) as e:
        # would need (1 << 18) + 1 partial sums; rejected on the host before anything is launched
        A.adapm_group_meansq_static(g, A.GRAD_BF16, A.STATIC_SCRATCH_FLOATS + 1, 8, out)
    assert e.value.code == -3 and "ADAPM_STATIC_SCRATCH_FLOATS" in str(e.value)
