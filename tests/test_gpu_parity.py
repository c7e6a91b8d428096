"""GPU-vs-oracle parity through the C ABI: trajectories on the five parameter sets and edge cases.

Tolerances: max relative error <= 1e-5 on the fp32 elementwise / reduction paths
(W, v, m of blocks without or with full momentum; v everywhere) and <= 2e-3 on the contraction paths
(L, R, P = L R and W of low-rank blocks).  The error of a tensor is max|gpu - ref| / max|ref|.
"""
import math

import numpy as np
import pytest

import workloads as WL
import paper_2510_09103_b200 as A
from oracle import adapm_oracle as O

from harness import ParityRun, Tolerances, rel_err, sample_blocks

pytestmark = pytest.mark.gpu

PATHS = [A.PATH_SIMT, A.PATH_AUTO]


def _run(w, blockmean, steps, sel=None, path=A.PATH_AUTO, pooled=False, every=1, hp=None, blocks=None, tol=Tolerances()):
    run = ParityRun(w, blockmean, oracle_blocks=sel, lowrank_path=path, pooled_grads=pooled, hp_overrides=hp,
                    custom_blocks=blocks)
    worst = {}
    try:
        for s in range(1, steps + 1):
            run.step()
            if s % every == 0 or s == steps:
                for k, v in run.compare(tol).items():
                    worst[k] = max(worst.get(k, 0.0), v)
        assert run.ctx.adapm_get_status() == 0
    finally:
        run.close()
    return worst


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("blockmean", [False, True])
def test_tiny_all_blocks_every_step(blockmean, path):
    w = WL.get_workload("tiny")
    _run(w, blockmean, w.steps, path=path)


@pytest.mark.parametrize("path", PATHS)
def test_llama60m_sampled_blocks_20_steps(path):
    w = WL.get_workload("llama60m")
    blocks, _ = A.adapm_plan_default(w.tensors)
    _run(w, True, w.steps, sel=sample_blocks(blocks, 2), path=path)


def test_llama60m_elementwise_v():
    w = WL.get_workload("llama60m")
    blocks, _ = A.adapm_plan_default(w.tensors, v_mode=A.V_ELEMENT)
    _run(w, False, 6, sel=sample_blocks(blocks, 1))


def test_gpt2_124m_sampled_blocks_20_steps():
    w = WL.get_workload("gpt2_124m")
    blocks, _ = A.adapm_plan_default(w.tensors)
    _run(w, True, w.steps, sel=sample_blocks(blocks, 1), every=5)


@pytest.mark.parametrize("rank", [8, 32, 128])
def test_llama350m_rank_sweep_20_steps(rank):
    w = WL.get_workload("llama350m", rank_override=rank)
    blocks, _ = A.adapm_plan_default(w.tensors, rank_override=rank)
    sel = [i for i in sample_blocks(blocks, 1) if blocks[i].rows * blocks[i].cols < 8_000_000]
    _run(w, True, w.steps, sel=sel, pooled=True, every=5)


def test_gpt2_1p5b_sampled_blocks_20_steps():
    """Full-size set in the launch configuration the benchmark times; the oracle follows one block per class."""
    w = WL.get_workload("gpt2_1p5b")
    blocks, _ = A.adapm_plan_default(w.tensors)
    sel = [i for i in sample_blocks(blocks, 1) if blocks[i].rows < 50000]     # wte is checked at 124M size
    _run(w, True, w.steps, sel=sel, pooled=True, every=5)


# ------------------------------------------------------------------------------------ edge cases

def _blk(off, rows, cols, mode, rank=0, vmode=A.V_BLOCKMEAN, gr=1, lr_scale=1.0, wd=0.1):
    return A.adapm_block(off, rows, cols, mode, rank, vmode, gr, lr_scale, wd)


def _pack(specs):
    out, cur = [], 0
    for rows, cols, mode, rank, vmode, gr in specs:
        cur = -(-cur // 8) * 8
        out.append(_blk(cur, rows, cols, mode, rank, vmode, gr, 0.75 if mode == A.MOM_NONE else 1.0))
        cur += rows * cols
    return out


RAGGED = [
    # rows, cols, mode, rank, v_mode, v_group_rows
    (1, 1, A.MOM_FULL, 0, A.V_BLOCKMEAN, 0),            # a single scalar
    (1, 7, A.MOM_FULL, 0, A.V_ELEMENT, 0),              # shorter than one 16-byte chunk
    (1, 4099, A.MOM_FULL, 0, A.V_BLOCKMEAN, 0),         # vector with a ragged tail, CTA-sized group
    (33, 5, A.MOM_NONE, 0, A.V_BLOCKMEAN, 1),           # rows that do not start on 16-byte boundaries
    (12, 1000, A.MOM_FULL, 0, A.V_BLOCKMEAN, 4),        # 4000-element groups: one CTA per group
    (130, 257, A.MOM_NONE, 0, A.V_BLOCKMEAN, 0),        # one 33410-element group: two-stage reduction
    (64, 2056, A.MOM_FULL, 0, A.V_BLOCKMEAN, 32),       # 65792-element groups, not a multiple of 2048
    (100, 77, A.MOM_FULL, 0, A.V_ELEMENT, 0),
    (70, 130, A.MOM_LOWRANK, 1, A.V_BLOCKMEAN, 1),      # rank 1, ragged tiles
    (129, 65, A.MOM_LOWRANK, 3, A.V_BLOCKMEAN, 43),     # groups of 43 rows
    (65, 200, A.MOM_LOWRANK, 8, A.V_ELEMENT, 0),
    (256, 192, A.MOM_LOWRANK, 38, A.V_BLOCKMEAN, 0),    # whole-block group
    (16, 16, A.MOM_LOWRANK, 16, A.V_BLOCKMEAN, 1),      # full rank
]


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_ragged_and_degenerate_blocks(dtype, path):
    w = WL.Workload("ragged", [], dtype, "normal", steps=8)
    _run(w, True, 8, path=path, blocks=_pack(RAGGED))


def test_adam_debias_and_no_clip():
    w = WL.Workload("debias", [], "f32", "normal", steps=6)
    _run(w, True, 6, blocks=_pack(RAGGED[:8]), hp=dict(adam_debias=1, clip=math.inf))


def test_correction_off_and_scaled_inner_steps():
    w = WL.Workload("nocorr", [], "bf16", "normal", steps=6)
    _run(w, True, 6, blocks=_pack(RAGGED[8:]), hp=dict(correction=0, inner_lr_scale=0.5, inner_iters=3))


def test_zero_inner_iterations_freeze_the_factors():
    w = WL.Workload("k0", [], "bf16", "normal", steps=4)
    _run(w, True, 4, blocks=_pack(RAGGED[8:]), hp=dict(inner_iters=0))


# ------------------------------------------------------------------------------------ library behaviour

def test_state_init_gives_orthonormal_L0_and_zero_R0():
    import torch
    blocks = _pack([(300, 64, A.MOM_LOWRANK, 12, A.V_BLOCKMEAN, 1), (64, 500, A.MOM_LOWRANK, 5, A.V_ELEMENT, 0)])
    ctx = A.adapm_create(blocks, A.hparams(seed=7))
    state = torch.full((ctx.adapm_state_bytes() // 4,), 3.0, device="cuda")
    ctx.adapm_state_init(state)
    torch.cuda.synchronize()
    for bi, b in enumerate(blocks):
        off, cnt = ctx.adapm_state_layout(bi, A.STATE_L)
        L = state[off:off + cnt].cpu().numpy().reshape(b.rows, b.rank).astype(np.float64)
        np.testing.assert_allclose(L.T @ L, np.eye(b.rank), atol=2e-5)
        off, cnt = ctx.adapm_state_layout(bi, A.STATE_R)
        assert not state[off:off + cnt].any()
        off, cnt = ctx.adapm_state_layout(bi, A.STATE_V)
        assert not state[off:off + cnt].any()
    ctx.adapm_destroy()


def test_runs_are_bitwise_reproducible_and_resumable():
    import torch
    w = WL.get_workload("tiny")

    def trajectory(split):
        run = ParityRun(w, True, oracle_blocks=[])
        for s in range(1, 7):
            run.step()
            if s == split:          # export everything, rebuild the context, import, continue
                p, st, t = run.params.clone(), run.state.clone(), run.t
                run.close()
                run = ParityRun(w, True, oracle_blocks=[])
                run.params.copy_(p); run.state.copy_(st); run.t = t
        torch.cuda.synchronize()
        out = run.params.clone(), run.state.clone()
        run.close()
        return out

    p1, s1 = trajectory(split=0)
    p2, s2 = trajectory(split=0)
    p3, s3 = trajectory(split=3)
    assert torch.equal(p1, p2) and torch.equal(s1, s2)
    assert torch.equal(p1, p3) and torch.equal(s1, s3)


def test_nan_gradient_propagates_and_does_not_hang():
    import torch
    blocks = _pack([(8, 64, A.MOM_FULL, 0, A.V_ELEMENT, 0), (8, 64, A.MOM_NONE, 0, A.V_BLOCKMEAN, 1)])
    ctx = A.adapm_create(blocks, A.hparams(grad_dtype=A.GRAD_F32))
    n = 1024
    params = torch.ones(n, device="cuda"); grads = torch.full((n,), 1e-3, device="cuda")
    grads[5] = float("nan"); grads[512 + 70] = float("nan")
    state = torch.zeros(ctx.adapm_state_bytes() // 4, device="cuda")
    ctx.adapm_state_init(state)
    ctx.adapm_step(params, grads, state, 1)
    torch.cuda.synchronize()
    p = params.cpu().numpy()
    assert math.isnan(p[5]) and np.isfinite(p[:5]).all() and np.isfinite(p[6:512]).all()
    assert np.isnan(p[512 + 64:512 + 128]).all()          # the whole v group of the poisoned row
    assert np.isfinite(p[512:512 + 64]).all()
    ctx.adapm_destroy()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", [(1, 5), (7, 2048), (3, 70001), (1000, 24), (2, 1 << 20)])
def test_group_meansq_entry_point(shape, dtype):
    import torch
    n_groups, ge = shape
    x = np.random.default_rng(5).standard_normal(n_groups * ge).astype(np.float32) * 1e-3
    vals, raw = WL.to_grad_dtype(x, dtype)
    g = torch.from_numpy(raw.view(np.int16) if dtype == "bf16" else raw).cuda()
    out = torch.zeros(n_groups, device="cuda")
    scratch = torch.zeros(max(A.adapm_group_meansq_scratch_bytes(n_groups, ge) // 4, 64), device="cuda")
    A.adapm_group_meansq(g, A.GRAD_BF16 if dtype == "bf16" else A.GRAD_F32, n_groups, ge, out, scratch)
    torch.cuda.synchronize()
    blk = O.Block(n_groups, ge, O.MOM_NONE, v_mode=O.V_BLOCKMEAN, v_group_rows=1)
    want = O.second_moment(np.zeros(n_groups), vals.astype(np.float64).reshape(n_groups, ge), blk, 0.0)
    assert rel_err(out.cpu().numpy(), want) <= 1e-5


def test_step_requires_workspace_and_aligned_pointers():
    import torch
    blocks = _pack([(64, 64, A.MOM_LOWRANK, 4, A.V_BLOCKMEAN, 1)])
    ctx = A.adapm_create(blocks, A.hparams())
    params = torch.zeros(4096 + 64, device="cuda"); grads = torch.zeros(4096 + 64, dtype=torch.bfloat16, device="cuda")
    state = torch.zeros(ctx.adapm_state_bytes() // 4, device="cuda")
    with pytest.raises(A.AdapmError) as e:
        ctx.adapm_step(params, grads, state, 1)
    assert e.value.code == -5
    with pytest.raises(A.AdapmError) as e:
        ctx.adapm_step(params[1:], grads, state, 1)
    assert e.value.code == -2
    ctx.adapm_destroy()


# ------------------------------------------------------------------------------------ tensor-core path

def test_tensor_path_can_be_forced_and_refuses_what_it_cannot_address():
    blocks = _pack([(256, 192, A.MOM_LOWRANK, 38, A.V_BLOCKMEAN, 0), (384, 128, A.MOM_LOWRANK, 16, A.V_ELEMENT, 0)])
    w = WL.Workload("forced", [], "bf16", "normal", steps=5)
    _run(w, True, 5, path=A.PATH_TENSOR, blocks=blocks)
    # fp32 gradients cannot enter the bf16 tensor cores unchanged: the forced path is refused, AUTO falls back
    with pytest.raises(A.AdapmError) as e:
        A.adapm_create(blocks, A.hparams(grad_dtype=A.GRAD_F32, lowrank_path=A.PATH_TENSOR))
    assert e.value.code == -6
    # a row pitch that is not a multiple of 16 bytes cannot be described to the TMA unit
    odd = _pack([(64, 130, A.MOM_LOWRANK, 4, A.V_BLOCKMEAN, 1)])
    with pytest.raises(A.AdapmError) as e:
        A.adapm_create(odd, A.hparams(lowrank_path=A.PATH_TENSOR))
    assert e.value.code == -6


def test_tensor_path_shallow_rings_partial_tiles_and_every_epilogue_form():
    """Rank 128 next to a per-element v leaves the apply kernel one g / W buffer and two R stages; the other blocks
    add a run of 18 column tiles whose last tile is 24 columns wide (quarters past the edge are not stored), five
    row panels with a ragged last one, and ranks that take the aligned-row, the by-column and the transposing
    form of the refit epilogue."""
    blocks = _pack([(300, 384, A.MOM_LOWRANK, 128, A.V_ELEMENT, 0),
                    (200, 2200, A.MOM_LOWRANK, 24, A.V_BLOCKMEAN, 1),
                    (520, 136, A.MOM_LOWRANK, 40, A.V_ELEMENT, 0),
                    (136, 520, A.MOM_LOWRANK, 13, A.V_BLOCKMEAN, 8)])
    w = WL.Workload("shallow", [], "bf16", "normal", steps=6)
    _run(w, True, 6, path=A.PATH_TENSOR, blocks=blocks)


def test_tensor_path_follows_moving_gradient_buffers():
    """Tensor maps hold absolute addresses; a gradient buffer that moves between steps must be picked up."""
    import torch
    blocks = _pack([(256, 256, A.MOM_LOWRANK, 12, A.V_BLOCKMEAN, 1)])
    w = WL.Workload("moving", [], "bf16", "normal", steps=4)
    run = ParityRun(w, True, lowrank_path=A.PATH_TENSOR, custom_blocks=blocks)
    try:
        first = run.grads
        for s in range(4):
            run.grads = first if s % 2 == 0 else torch.zeros_like(first)     # a second allocation on odd steps
            run.step()
            run.compare()
        assert run.ctx.adapm_get_status() == 0
    finally:
        run.close()


def test_tensor_path_is_bitwise_reproducible():
    import torch
    blocks = _pack([(300, 256, A.MOM_LOWRANK, 20, A.V_BLOCKMEAN, 1), (128, 640, A.MOM_LOWRANK, 6, A.V_BLOCKMEAN, 0)])

    def trajectory():
        w = WL.Workload("repro", [], "bf16", "normal", steps=5)
        run = ParityRun(w, True, oracle_blocks=[], lowrank_path=A.PATH_TENSOR, custom_blocks=blocks)
        for _ in range(5):
            run.step()
        torch.cuda.synchronize()
        out = run.params.clone(), run.state.clone()
        assert run.ctx.adapm_get_status() == 0
        run.close()
        return out

    p1, s1 = trajectory()
    p2, s2 = trajectory()
    assert torch.equal(p1, p2) and torch.equal(s1, s2)


def test_panel_team_schedule_changes_no_bit(monkeypatch):
    """The refit's panel launch hands its items to teams of CTAs kept in step by a counter when the set has enough
    blocks (llama350m has); ADAPM_PANEL_TEAMS=0 hands them out longest-first instead.  Which CTA runs an item, and
    when, must not change any result."""
    import torch

    def trajectory(teams):
        monkeypatch.setenv("ADAPM_PANEL_TEAMS", teams)
        run = ParityRun(WL.get_workload("llama350m"), True, oracle_blocks=[], lowrank_path=A.PATH_TENSOR)
        for _ in range(3):
            run.step()
        torch.cuda.synchronize()
        out = run.params.clone(), run.state.clone()
        assert run.ctx.adapm_get_status() == 0
        run.close()
        return out

    p1, s1 = trajectory("1")
    p0, s0 = trajectory("0")
    assert torch.equal(p1, p0) and torch.equal(s1, s0)


def test_tensor_path_nan_gradient_stays_in_its_block_and_does_not_hang():
    import torch
    blocks = _pack([(256, 128, A.MOM_LOWRANK, 8, A.V_BLOCKMEAN, 1), (128, 128, A.MOM_LOWRANK, 8, A.V_BLOCKMEAN, 1)])
    ctx = A.adapm_create(blocks, A.hparams(lowrank_path=A.PATH_TENSOR))
    n = blocks[1].offset + 128 * 128
    params = torch.ones(n, device="cuda")
    grads = torch.full((n,), 1e-3, device="cuda").bfloat16()
    grads[7] = float("nan")                                  # inside the first block
    state = torch.zeros(ctx.adapm_state_bytes() // 4, device="cuda")
    work = torch.zeros(max(ctx.adapm_workspace_bytes() // 4, 64), device="cuda")
    ctx.adapm_set_workspace(work)
    ctx.adapm_state_init(state)
    ctx.adapm_step(params, grads, state, 1)
    torch.cuda.synchronize()
    assert ctx.adapm_get_status() == 0
    p = params.cpu().numpy()
    assert np.isnan(p[:256 * 128]).any()
    assert np.isfinite(p[blocks[1].offset:]).all()           # the other block never sees it
    ctx.adapm_destroy()
