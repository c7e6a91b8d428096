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


def test_gpt2_1p5b_4layers_elementwise_v():
    """Rank 80 with a per-element v: the apply kernel's three-buffer form (v travels with W), followed by the oracle."""
    w = WL.get_workload("gpt2_1p5b@4")
    blocks, _ = A.adapm_plan_default(w.tensors, v_mode=A.V_ELEMENT)
    sel = [i for i in sample_blocks(blocks, 1) if blocks[i].rows < 50000]
    _run(w, False, 6, sel=sel, pooled=True, every=3)


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


ALIGNED_UNITS = [
    # warp-sized units that start on 16-byte boundaries and hold a multiple of 8 elements ...
    (40, 1600, A.MOM_NONE, 0, A.V_BLOCKMEAN, 1),        # one 1600-element row per unit, no momentum
    (9, 2048, A.MOM_FULL, 0, A.V_BLOCKMEAN, 1),         # units of the largest size
    (300, 8, A.MOM_FULL, 0, A.V_BLOCKMEAN, 1),          # units of the smallest size
    (50, 1000, A.MOM_FULL, 0, A.V_ELEMENT, 0),          # per-element v, an 848-element tail unit
    (3, 24, A.MOM_NONE, 0, A.V_ELEMENT, 0),             # one short unit
    (1, 2040, A.MOM_FULL, 0, A.V_BLOCKMEAN, 0),         # whole-block group in one unit
    (6000, 64, A.MOM_FULL, 0, A.V_BLOCKMEAN, 1),        # many more units than CTAs
    # ... next to blocks whose units are not
    (33, 5, A.MOM_NONE, 0, A.V_BLOCKMEAN, 1),
    (12, 1000, A.MOM_FULL, 0, A.V_BLOCKMEAN, 4),
    (100, 77, A.MOM_FULL, 0, A.V_ELEMENT, 0),
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_streaming_update_unit_shapes(dtype):
    """Blocks without low-rank momentum over the unit shapes the streaming kernel distinguishes (vector and
    guarded chunks, one or several batches per thread, with and without m and per-element v): all blocks against
    the oracle, every step."""
    w = WL.Workload("aligned_units", [], dtype, "normal", steps=6)
    _run(w, True, 6, blocks=_pack(ALIGNED_UNITS))


def test_streaming_update_with_clipping_and_shadow():
    """The same blocks with the gradients scaled by the global clip factor and the bf16 copy of W written."""
    import torch
    w = WL.Workload("aligned_units", [], "bf16", "normal", steps=4)
    run = ParityRun(w, True, custom_blocks=_pack(ALIGNED_UNITS), hp_overrides=dict(max_grad_norm=0.5), shadow=True)
    try:
        for _ in range(4):
            run.step()
            run.compare()
            # padding between blocks is never written: compare the blocks' own ranges
            for blk in run.blocks:
                sl = slice(blk.offset, blk.offset + blk.rows * blk.cols)
                assert torch.equal(run.shadow[sl], run.params[sl].to(torch.bfloat16))
        assert run.ctx.adapm_get_status() == 0
    finally:
        run.close()


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


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_state_init_from_grads_matches_the_range_finder_oracle(dtype):
    """Data-driven L_0 = Gram-Schmidt over the columns of g_1 Omega (a variant, not in the paper): the library's L_0
    against the oracle's, element by element; a gradient of rank 2 under rank 5 leaves three zero columns on both
    sides; R, v and the other blocks' state are zero."""
    import torch
    specs = [(300, 64, A.MOM_LOWRANK, 12, A.V_BLOCKMEAN, 1), (64, 504, A.MOM_LOWRANK, 5, A.V_ELEMENT, 0),
             (40, 16, A.MOM_FULL, 0, A.V_BLOCKMEAN, 1), (640, 384, A.MOM_LOWRANK, 38, A.V_BLOCKMEAN, 1),
             (96, 72, A.MOM_LOWRANK, 5, A.V_BLOCKMEAN, 1)]
    blocks = _pack(specs)
    total = -(-max(b.offset + b.rows * b.cols for b in blocks) // 8) * 8
    rng = np.random.default_rng(5)
    g = np.zeros(total, dtype=np.float32)
    for bi, b in enumerate(blocks):
        x = rng.standard_normal((b.rows, b.cols)) * 1e-3 * np.exp(rng.uniform(-2, 2, size=(b.rows, 1)))
        if bi == 4:     # rank 2, small integers times 2^-10: exact in bf16, so rounding does not fill the rank up
            x = (rng.integers(-3, 4, size=(b.rows, 2)) @ rng.integers(-3, 4, size=(2, b.cols))) * 2.0 ** -10
        g[b.offset:b.offset + b.rows * b.cols] = x.ravel()
    if dtype == "bf16":
        gt = torch.from_numpy(g).to(torch.bfloat16)
        g = gt.to(torch.float32).numpy()
    else:
        gt = torch.from_numpy(g)
    ctx = A.adapm_create(blocks, A.hparams(grad_dtype=A.GRAD_BF16 if dtype == "bf16" else A.GRAD_F32))
    omega = np.zeros(ctx.adapm_init_omega_floats(), dtype=np.float32)
    om_of = {}
    for bi, b in enumerate(blocks):
        off, cnt = ctx.adapm_init_omega_layout(bi)
        assert cnt == (b.cols * b.rank if b.mom_mode == A.MOM_LOWRANK else 0)
        if cnt:
            om_of[bi] = rng.standard_normal((b.cols, b.rank)).astype(np.float32)
            omega[off:off + cnt] = om_of[bi].ravel()
    state = torch.full((ctx.adapm_state_bytes() // 4,), 3.0, device="cuda")
    ctx.adapm_state_init_from_grads(state, gt.cuda(), torch.from_numpy(omega).cuda())
    torch.cuda.synchronize()
    host = state.cpu().numpy()
    seen = np.zeros(host.size, dtype=bool)
    for bi, b in enumerate(blocks):
        if b.mom_mode != A.MOM_LOWRANK:
            continue
        off, cnt = ctx.adapm_state_layout(bi, A.STATE_L)
        L = host[off:off + cnt].reshape(b.rows, b.rank).astype(np.float64)
        seen[off:off + cnt] = True
        ref = O.init_L0_range(g[b.offset:b.offset + b.rows * b.cols].reshape(b.rows, b.cols).astype(np.float64),
                              om_of[bi].astype(np.float64))
        assert rel_err(L, ref) <= 1e-4, (bi, rel_err(L, ref))
        if bi == 4:
            assert np.all(L[:, 2:] == 0.0) and np.all(ref[:, 2:] == 0.0)
            np.testing.assert_allclose(L[:, :2].T @ L[:, :2], np.eye(2), atol=2e-5)
        else:
            np.testing.assert_allclose(L.T @ L, np.eye(b.rank), atol=5e-5)
    assert not host[~seen].any()            # R_0, v, m and the padding: all zero
    assert ctx.adapm_get_status() == 0
    ctx.adapm_destroy()


def test_steps_from_a_data_driven_L0_follow_the_oracle():
    """Three steps started from the library's own range-finder L_0 (handed to the oracle as its L_0), on the CUDA-core
    and on the tensor-core refit."""
    import torch
    for path, dtype in ((A.PATH_SIMT, "f32"), (A.PATH_TENSOR, "bf16")):
        blocks = _pack([(256, 192, A.MOM_LOWRANK, 38, A.V_BLOCKMEAN, 1), (384, 128, A.MOM_LOWRANK, 16, A.V_BLOCKMEAN, 1),
                        (64, 512, A.MOM_FULL, 0, A.V_BLOCKMEAN, 1)])
        run = ParityRun(WL.Workload("range_start", [], dtype, "normal", steps=3), True, lowrank_path=path,
                        custom_blocks=blocks)
        try:
            # the first step's gradients, as the harness will hand them to the step
            np_dt = np.uint16 if dtype == "bf16" else np.float32
            host = np.zeros(run.total, dtype=np_dt)
            for ti in range(len(run.w.tensors)):
                _, raw = run._grad_raw(ti, 1)
                off = run.blocks[run.t2b[ti][0]].offset
                host[off:off + raw.size] = raw
            g1 = torch.from_numpy(host.view(np.int16) if dtype == "bf16" else host).cuda()
            g1 = g1.view(torch.bfloat16) if dtype == "bf16" else g1
            rng = np.random.default_rng(9)
            omega = torch.from_numpy(rng.standard_normal(run.ctx.adapm_init_omega_floats()).astype(np.float32)).cuda()
            canary_state = run.state.clone()
            run.ctx.adapm_state_init_from_grads(run.state, g1, omega)
            torch.cuda.synchronize()
            # keep the harness's canaries in the gaps of the state buffer; take the new sub-buffers
            fresh = run.state.clone()
            run.state.copy_(canary_state)
            for bi, b in enumerate(run.blocks):
                for which in (A.STATE_M, A.STATE_L, A.STATE_R, A.STATE_V):
                    off, cnt = run.ctx.adapm_state_layout(bi, which)
                    if cnt:
                        run.state[off:off + cnt] = fresh[off:off + cnt]
                if b.mom_mode == A.MOM_LOWRANK:
                    off, cnt = run.ctx.adapm_state_layout(bi, A.STATE_L)
                    run.ostate[bi].L = run.state[off:off + cnt].cpu().numpy().reshape(b.rows, b.rank).astype(np.float64)
            run.ctx.adapm_state_changed()
            for _ in range(3):
                run.step()
                run.compare()
            assert run.ctx.adapm_get_status() == 0
        finally:
            run.close()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("damping", [1e-2, 1e-3])
def test_preconditioned_passes_follow_the_oracle(dtype, damping):
    """inner_precond = 1 (scaled gradient descent, a variant that is not in the paper): each derivative of Algorithm 2
    times the damped inverse of the other factor's Gram matrix.  Six steps on the CUDA-core path, every block, every
    step.  (The fp32 inverse of a Gram matrix with condition number k carries about k * 2^-24; with these damped,
    well-conditioned matrices L, R and P agree to 1e-6.)"""
    w = WL.Workload("precond", [], dtype, "normal", steps=6)
    blocks = _pack([(96, 160, A.MOM_LOWRANK, 8, A.V_BLOCKMEAN, 1), (200, 64, A.MOM_LOWRANK, 3, A.V_ELEMENT, 0),
                    (256, 192, A.MOM_LOWRANK, 38, A.V_BLOCKMEAN, 0), (70, 130, A.MOM_LOWRANK, 1, A.V_BLOCKMEAN, 1),
                    (64, 128, A.MOM_FULL, 0, A.V_BLOCKMEAN, 1)])
    worst = _run(w, True, 6, blocks=blocks, hp=dict(inner_precond=1, precond_damping=damping, inner_lr_scale=0.5))
    assert max(worst["L"], worst["R"], worst["P"]) <= 1e-4       # seen: 1e-6


def test_preconditioned_passes_with_a_refresh_period_clipping_and_on_the_tensor_path():
    w = WL.Workload("precond", [], "bf16", "normal", steps=5)
    blocks = _pack([(128, 256, A.MOM_LOWRANK, 12, A.V_BLOCKMEAN, 1), (256, 64, A.MOM_LOWRANK, 5, A.V_BLOCKMEAN, 1)])
    _run(w, True, 5, blocks=blocks, hp=dict(inner_precond=1, precond_damping=1e-2, inner_lr_scale=0.5, refresh_period=3))
    # with the gradients scaled by the global clip factor (the threshold lies far below the norm of these gradients)
    _run(w, True, 3, blocks=blocks, hp=dict(inner_precond=1, precond_damping=1e-2, inner_lr_scale=0.5, max_grad_norm=0.05))
    # forced onto the tensor cores, with a rank above 128 (two MMAs per K step, the wider factor layout) beside them
    blocks = _pack([(128, 256, A.MOM_LOWRANK, 12, A.V_BLOCKMEAN, 1), (256, 64, A.MOM_LOWRANK, 5, A.V_BLOCKMEAN, 1),
                    (512, 384, A.MOM_LOWRANK, 160, A.V_BLOCKMEAN, 1), (1600, 640, A.MOM_LOWRANK, 80, A.V_BLOCKMEAN, 1)])
    worst = _run(w, True, 5, blocks=blocks, path=A.PATH_TENSOR,
                 hp=dict(inner_precond=1, precond_damping=1e-2, inner_lr_scale=0.5))
    print("preconditioned passes on the tensor path, worst errors:", worst)


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
    # the data-driven start: a missing Omega and misaligned buffers are refused on the host
    omega = torch.zeros(ctx.adapm_init_omega_floats() + 4, device="cuda")
    assert ctx.adapm_init_omega_floats() == 64 * 4 and ctx.adapm_init_omega_layout(0) == (0, 64 * 4)
    with pytest.raises(A.AdapmError) as e:
        ctx.adapm_state_init_from_grads(state, grads, None)
    assert e.value.code == -1
    with pytest.raises(A.AdapmError) as e:
        ctx.adapm_state_init_from_grads(state, grads, omega[1:])
    assert e.value.code == -2
    with pytest.raises(A.AdapmError) as e:
        ctx.adapm_state_init_from_grads(state[1:], grads, omega)
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


def test_panel_team_schedule_changes_no_bit():
    """The refit's panel launch hands its items to teams of CTAs kept in step by a counter when the set has enough
    blocks (llama350m has); ADAPM_FLAG_NO_PANEL_TEAMS hands them out longest-first instead.  Which CTA runs an
    item, and when, must not change any result."""
    import torch

    def trajectory(teams):
        run = ParityRun(WL.get_workload("llama350m"), True, oracle_blocks=[], lowrank_path=A.PATH_TENSOR,
                        hp_overrides=dict(flags=0 if teams else A.FLAG_NO_PANEL_TEAMS))
        for _ in range(3):
            run.step()
        torch.cuda.synchronize()
        out = run.params.clone(), run.state.clone()
        assert run.ctx.adapm_get_status() == 0
        run.close()
        return out

    p1, s1 = trajectory(True)
    p0, s0 = trajectory(False)
    assert torch.equal(p1, p0) and torch.equal(s1, s0)


@pytest.mark.parametrize("panels,stage_k", [(1, 128), (2, 64), (3, 64), (3, 128)])
def test_tensor_path_engine_shapes(panels, stage_k):
    """Every shape of the refit engine's pipeline - one to three panels per item, K = 64 or 128 per stage - against
    the oracle, on blocks with ragged last panels and ranks that take each form of the epilogue."""
    blocks = _pack([(700, 392, A.MOM_LOWRANK, 24, A.V_BLOCKMEAN, 1),
                    (392, 1000, A.MOM_LOWRANK, 13, A.V_BLOCKMEAN, 8),
                    (520, 136, A.MOM_LOWRANK, 40, A.V_ELEMENT, 0)])
    w = WL.Workload("shapes", [], "bf16", "normal", steps=5)
    _run(w, True, 5, path=A.PATH_TENSOR, blocks=blocks, hp=dict(tune_panels=panels, tune_stage_k=stage_k))


def test_folded_row_sums_equal_the_separate_reduction_bit_for_bit_in_everything_but_v():
    """The first refit pass adds up g^2 per row while it streams the gradient; ADAPM_FLAG_NO_SUMSQ_FOLD takes the
    sums from a pass of its own instead.  The two add in different orders, so v may differ in the last bits (both
    are checked against the oracle elsewhere); nothing else may change by more than that allows."""
    import torch
    blocks = _pack([(300, 256, A.MOM_LOWRANK, 20, A.V_BLOCKMEAN, 1), (128, 640, A.MOM_LOWRANK, 6, A.V_BLOCKMEAN, 0),
                    (256, 512, A.MOM_LOWRANK, 16, A.V_BLOCKMEAN, 64)])

    def trajectory(flags):
        w = WL.Workload("fold", [], "bf16", "normal", steps=4)
        run = ParityRun(w, True, lowrank_path=A.PATH_TENSOR, custom_blocks=blocks, hp_overrides=dict(flags=flags))
        for _ in range(4):
            run.step()
            run.compare()
        torch.cuda.synchronize()
        out = run.params.clone(), run.state.clone()
        assert run.ctx.adapm_get_status() == 0
        run.close()
        return out

    p1, s1 = trajectory(0)
    p0, s0 = trajectory(A.FLAG_NO_SUMSQ_FOLD)
    assert torch.allclose(p1, p0, rtol=1e-5, atol=1e-9) and torch.allclose(s1, s0, rtol=1e-5, atol=1e-12)


def test_tensor_path_resumes_bit_for_bit_and_follows_a_rewritten_state():
    """The factor copies in the workspace carry over from step to step (the sets swap roles; nothing is converted).
    A run that is exported after 3 steps and continued in a fresh context and workspace must equal an
    uninterrupted one bit for bit, and a state buffer rewritten in place must be picked up after
    adapm_state_changed."""
    import torch
    blocks = _pack([(300, 256, A.MOM_LOWRANK, 20, A.V_BLOCKMEAN, 1), (128, 640, A.MOM_LOWRANK, 6, A.V_ELEMENT, 0)])

    def make():
        return ParityRun(WL.Workload("resume", [], "bf16", "normal", steps=6), True, oracle_blocks=[],
                         lowrank_path=A.PATH_TENSOR, custom_blocks=blocks)

    def trajectory(split, in_place=False):
        run = make()
        for s in range(1, 7):
            run.step()
            if s == split and not in_place:
                p, st, t = run.params.clone(), run.state.clone(), run.t
                run.close()
                run = make()
                run.params.copy_(p); run.state.copy_(st); run.t = t
            elif s == split:
                # overwrite the state with itself through a copy and tell the library: the result must not move
                st = run.state.clone()
                run.state.zero_()
                run.state.copy_(st)
                run.ctx.adapm_state_changed()
        torch.cuda.synchronize()
        out = run.params.clone(), run.state.clone()
        assert run.ctx.adapm_get_status() == 0
        run.close()
        return out

    p1, s1 = trajectory(0)
    p2, s2 = trajectory(3)
    p3, s3 = trajectory(3, in_place=True)
    assert torch.equal(p1, p2) and torch.equal(s1, s2)
    assert torch.equal(p1, p3) and torch.equal(s1, s3)


def test_an_expired_wait_is_reported_and_the_context_keeps_working():
    """A wait inside the refit engine that can never be satisfied (a team counter nothing advances, with the limit
    cut to about a millisecond) must end the kernel with a status bit, make later launches skip until the status
    has been read, and leave the context usable."""
    import torch
    blocks = _pack([(256, 256, A.MOM_LOWRANK, 12, A.V_BLOCKMEAN, 1), (64, 64, A.MOM_FULL, 0, A.V_ELEMENT, 0)])
    w = WL.Workload("expired", [], "bf16", "normal", steps=3)
    run = ParityRun(w, True, lowrank_path=A.PATH_TENSOR, custom_blocks=blocks)
    try:
        run.step()
        run.compare()
        before = run.params.clone(), run.state.clone()
        run.ctx.adapm_selftest_expired_wait()
        # the status word is set: a step issued now must not write anything
        run.ctx.adapm_step(run.params, run.grads, run.state, run.t + 1)
        torch.cuda.synchronize()
        assert torch.equal(before[0], run.params) and torch.equal(before[1], run.state)
        assert run.ctx.adapm_get_status() == A.ST_WAIT_TEAM
        assert run.ctx.adapm_get_status() == 0
        run.step()                      # the same step number again, now for real: parity with the oracle holds
        run.compare()
    finally:
        run.close()


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


# ------------------------------------------------------------------------------------ ranks above 128, Llama3-8B shapes

@pytest.mark.parametrize("rank", [160, 204])
def test_tensor_path_ranks_above_128_20_steps(rank):
    """Above rank 128 the refit takes the hi and the lo half of a factor in separate MMAs and the apply kernel
    streams L as well as R; 20 steps against the oracle."""
    blocks = _pack([(1536, 1024, A.MOM_LOWRANK, rank, A.V_BLOCKMEAN, 1),
                    (640, 2048, A.MOM_LOWRANK, rank, A.V_ELEMENT, 0),
                    (520, 392, A.MOM_LOWRANK, 24, A.V_BLOCKMEAN, 8)])      # a small rank beside them
    w = WL.Workload("bigrank", [], "bf16", "normal", steps=20)
    _run(w, True, 20, path=A.PATH_TENSOR, blocks=blocks, every=4)


def test_llama3_8b_block_shapes_on_the_tensor_path():
    """The four low-rank block shapes of the Llama3-8B-shaped set (Section 5.2: rank 5% of 4096 = 204, 51 for the
    grouped-query key projection) at full size, and the whole set accepted by the tensor path: no block of it
    falls back to the CUDA-core refit."""
    w = WL.get_workload("llama3_8b")
    blocks, _ = A.adapm_plan_default(w.tensors)
    ctx = A.adapm_create(blocks, A.hparams(lowrank_path=A.PATH_TENSOR))       # would raise -6 otherwise
    ctx.adapm_destroy()
    shapes = sorted({(b.rows, b.cols, b.rank, b.v_group_rows) for b in blocks if b.mom_mode == A.MOM_LOWRANK})
    assert shapes == [(1024, 4096, 51, 128), (4096, 4096, 204, 128), (4096, 14336, 204, 1), (14336, 4096, 204, 1)]
    custom = _pack([(r, c, A.MOM_LOWRANK, k, A.V_BLOCKMEAN, g) for r, c, k, g in shapes])
    _run(WL.Workload("llama3_shapes", [], "bf16", "normal", steps=3), True, 3, path=A.PATH_TENSOR, blocks=custom)


@pytest.mark.parametrize("pct", [2, 10, 50])
def test_rank_ratios_of_the_ablation(pct):
    """Section 5.1.2 sweeps the rank over 2, 5, 10 and 50 percent of the full rank; on the LLaMA-350M block shapes
    (d = 1024, FFN 2736) that is 20, 102 and 512.  Up to rank 256 the blocks run on the tensor path, above on the
    CUDA-core path (AUTO).  The ranks come from the planner; the blocks are one of each low-rank shape."""
    w = WL.get_workload("llama350m", rank_pct=pct)
    planned, _ = A.adapm_plan_default(w.tensors, rank_pct=pct)
    shapes = sorted({(b.rows, b.cols, b.rank, b.v_group_rows) for b in planned if b.mom_mode == A.MOM_LOWRANK})
    want = max(1, pct * 1024 // 100)
    assert shapes == [(1024, 1024, want, 64), (1024, 2736, want, 1), (2736, 1024, want, 1)]
    blocks = _pack([(r, c, A.MOM_LOWRANK, k, A.V_BLOCKMEAN, g) for r, c, k, g in shapes])
    _run(WL.Workload(f"ratio{pct}", [], "bf16", "heavyrows", steps=4), True, 4, blocks=blocks)


# ------------------------------------------------------------------------------------ global clipping, bf16 copy, finite check

def _alternating(step):
    return 0.5 if step % 2 else 2.0


@pytest.mark.parametrize("path", [A.PATH_AUTO, A.PATH_SIMT])
def test_llama60m_global_clipping_20_steps(path):
    """Global gradient-norm clipping (Section 5.1, Setups).  The gradients of odd steps are halved and those of even
    steps doubled, and the threshold sits between the two norms, so the clip factor is 1 on odd steps and below 1 on
    even ones; the bf16 copy of the parameters is written along and must be the rounded fp32 parameters."""
    import torch
    w = WL.get_workload("llama60m")
    blocks, _ = A.adapm_plan_default(w.tensors)
    # ||g|| of this set is ~25 (sigma 1e-3, row scales log-uniform in [0.1, 10], 58 M elements)
    run = ParityRun(w, True, oracle_blocks=sample_blocks(blocks, 1), lowrank_path=path, pooled_grads=True,
                    hp_overrides=dict(max_grad_norm=25.0), grad_scale=_alternating, shadow=True)
    seen = []
    try:
        for s in range(1, w.steps + 1):
            run.step()
            seen.append(run.last_gscale)
            if s % 5 == 0 or s <= 2:
                run.compare()
                torch.cuda.synchronize()
                assert torch.equal(run.shadow, run.params.to(torch.bfloat16))
        assert run.ctx.adapm_get_status() == 0
    finally:
        run.close()
    assert all(k == 1.0 for k in seen[0::2]) and all(0.3 < k < 0.9 for k in seen[1::2])


def test_tiny_global_clipping_fp32_gradients():
    w = WL.get_workload("tiny")
    run = ParityRun(w, True, hp_overrides=dict(max_grad_norm=1.0), grad_scale=lambda s: 4.0 if s % 2 else 0.25,
                    shadow=True)
    try:
        for _ in range(6):
            run.step()
            run.compare()
        assert run.ctx.adapm_get_status() == 0
        assert min(run.last_gscale, 1.0) <= 1.0
    finally:
        run.close()


def test_finite_check_skips_the_step_and_reports_it():
    """With ADAPM_FLAG_CHECK_FINITE a NaN or Inf anywhere in the gradients makes the whole step a no-op (parameters
    and state untouched) and sets bit 64 of the status word; the next step with good gradients runs normally."""
    import torch
    blocks = _pack([(256, 128, A.MOM_LOWRANK, 8, A.V_BLOCKMEAN, 1), (64, 64, A.MOM_FULL, 0, A.V_ELEMENT, 0),
                    (32, 64, A.MOM_NONE, 0, A.V_BLOCKMEAN, 1)])
    w = WL.Workload("finite", [], "bf16", "normal", steps=3)
    run = ParityRun(w, True, custom_blocks=blocks, hp_overrides=dict(flags=A.FLAG_CHECK_FINITE))
    try:
        run.step()
        run.compare()
        before = run.params.clone(), run.state.clone()
        bad = run.grads.clone()
        bad[blocks[1].offset + 5] = float("inf")
        run.ctx.adapm_step(run.params, bad, run.state, run.t + 1)
        torch.cuda.synchronize()
        assert torch.equal(before[0], run.params) and torch.equal(before[1], run.state)
        assert run.ctx.adapm_get_status() == A.ST_NONFINITE_GRAD
        run.step()
        run.compare()
        # a caller that counts the skipped step and goes on with the next number must get the same result as one
        # that repeats the number: the library rebuilds its bf16 copies of the factors after a reported skip
        before = run.params.clone(), run.state.clone()
        run.ctx.adapm_step(run.params, bad, run.state, run.t + 1)
        torch.cuda.synchronize()
        assert torch.equal(before[0], run.params) and torch.equal(before[1], run.state)
        assert run.ctx.adapm_get_status() == A.ST_NONFINITE_GRAD
        run.t += 1                      # the skipped step keeps its number
        run.step()
        run.compare()
        assert run.ctx.adapm_get_status() == 0
    finally:
        run.close()


# ------------------------------------------------------------------------------------ refresh period T

@pytest.mark.parametrize("path", [A.PATH_TENSOR, A.PATH_SIMT])
def test_refresh_period_holds_L_between_refreshes(path):
    """refresh_period = 3: Algorithm 2 refits both factors at steps 1, 4, 7, ...; in between L stays as it is (bit
    for bit) and only R is refitted.  Every step is compared with the oracle's reading of T."""
    import torch
    blocks = _pack([(300, 256, A.MOM_LOWRANK, 20, A.V_BLOCKMEAN, 1), (128, 640, A.MOM_LOWRANK, 6, A.V_ELEMENT, 0),
                    (256, 512, A.MOM_LOWRANK, 16, A.V_BLOCKMEAN, 64), (64, 64, A.MOM_FULL, 0, A.V_BLOCKMEAN, 1)])
    w = WL.Workload("refresh", [], "bf16", "normal", steps=8)
    run = ParityRun(w, True, lowrank_path=path, custom_blocks=blocks, hp_overrides=dict(refresh_period=3))
    try:
        for s in range(1, 9):
            off, cnt = run.ctx.adapm_state_layout(0, A.STATE_L)
            before = run.state[off:off + cnt].clone()
            run.step()
            run.compare()
            torch.cuda.synchronize()
            same = torch.equal(before, run.state[off:off + cnt])
            assert same == ((s - 1) % 3 != 0), f"step {s}: L {'did not move' if same else 'moved'}"
        assert run.ctx.adapm_get_status() == 0
    finally:
        run.close()


def test_refresh_period_on_llama60m():
    w = WL.get_workload("llama60m")
    blocks, _ = A.adapm_plan_default(w.tensors)
    _run(w, True, 9, sel=sample_blocks(blocks, 1), pooled=True, every=3, hp=dict(refresh_period=4))
