"""Pins of the fp64 oracle against what the paper and the mathematics fix.

None of these tests compares the oracle with itself: each uses a closed form, a
special case that reduces to a library routine, an identity from the paper's
proof of Theorem 2, or scalar brute force on tiny blocks.
"""
import math
import os

import numpy as np
import pytest

from oracle import adapm_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")
RNG = np.random.default_rng(1234)


def _rand_block(rows, cols, **kw):
    return O.Block(rows=rows, cols=cols, **kw)


# ------------------------------------------------------------------------------------ schedule

def test_inner_schedule_matches_closed_forms():
    want = [float(l) for l in open(os.path.join(GOLD, "inner_schedule_K5.txt")) if l[0] not in "#\n"]
    got = O.inner_schedule(5)
    assert got[4] == 0.0                      # cos(pi) = -1 exactly: the 5th pass is a no-op
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-15)
    s5 = math.sqrt(5.0)
    np.testing.assert_allclose(got[:2], [0.5 * (1 + (1 + s5) / 4), 0.5 * (1 + (s5 - 1) / 4)], atol=1e-15)
    assert all(a > b for a, b in zip(got, got[1:]))      # decreasing


# ------------------------------------------------------------------------------------ P1

def _plain_full_momentum_step(W, g, m, v, lr, b1, b2, eps, lam, clip):
    """Eq. 4 + Algorithm 1 line 7 + line 9, written out on its own."""
    m = b1 * m + (1 - b1) * g
    v = b2 * v + (1 - b2) * g * g
    u = m / (np.sqrt(v) + eps)
    u = np.minimum(np.maximum(u, -clip), clip)
    return W - lr * (u + lam * W), m, v


def test_P1_all_full_equals_plain_routine():
    rows, cols = 7, 5
    blk = _rand_block(rows, cols, mom_mode=O.MOM_FULL, weight_decay=0.1)
    hp = O.HParams(lr=3e-3, beta1=0.9, beta2=0.95)
    st = O.new_state(blk)
    W = RNG.standard_normal((rows, cols)); Wp = W.copy()
    m = np.zeros_like(W); v = np.zeros_like(W)
    for t in range(1, 8):
        g = RNG.standard_normal((rows, cols)) * 1e-2
        W = O.block_step(W, g, st, blk, hp, t)
        Wp, m, v = _plain_full_momentum_step(Wp, g, m, v, 3e-3, 0.9, 0.95, 1e-8, 0.1, 1.0)
        for a, b in ((W, Wp), (st.m, m), (st.v, v)):      # equal up to the order of two roundings
            np.testing.assert_allclose(a, b, rtol=1e-15, atol=0)


def test_P1_debiased_unclipped_full_momentum_is_textbook_adamw():
    torch = pytest.importorskip("torch")
    rows, cols = 6, 4
    W0 = RNG.standard_normal((rows, cols))
    p = torch.nn.Parameter(torch.tensor(W0, dtype=torch.float64))
    opt = torch.optim.AdamW([p], lr=2e-3, betas=(0.9, 0.95), eps=1e-8, weight_decay=0.1)
    blk = _rand_block(rows, cols, mom_mode=O.MOM_FULL, weight_decay=0.1)
    hp = O.HParams(lr=2e-3, beta1=0.9, beta2=0.95, clip=math.inf, adam_debias=True)
    st = O.new_state(blk)
    W = W0.copy()
    for t in range(1, 11):
        g = RNG.standard_normal((rows, cols))
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        W = O.block_step(W, g, st, blk, hp, t)
        np.testing.assert_allclose(W, p.detach().numpy(), rtol=1e-12, atol=1e-14)


# ------------------------------------------------------------------------------------ P2

def test_P2_exact_solver_at_full_rank_is_full_momentum():
    rows, cols = 6, 4
    lr_blk = _rand_block(rows, cols, mom_mode=O.MOM_LOWRANK, rank=4, weight_decay=0.1)
    fm_blk = _rand_block(rows, cols, mom_mode=O.MOM_FULL, weight_decay=0.1)
    hp = O.HParams()
    s1, s2 = O.new_state(lr_blk), O.new_state(fm_blk)
    W1 = RNG.standard_normal((rows, cols)); W2 = W1.copy()
    for t in range(1, 13):
        g = RNG.standard_normal((rows, cols)) * 1e-3
        W1 = O.block_step(W1, g, s1, lr_blk, hp, t, solver="exact", keep=True)
        W2 = O.block_step(W2, g, s2, fm_blk, hp, t)
        assert np.abs(s1.last["r_t"]).max() < 1e-15
        np.testing.assert_allclose(s1.last["m_c"], s2.m, rtol=0, atol=1e-15)
        np.testing.assert_allclose(W1, W2, rtol=0, atol=1e-12)


# ------------------------------------------------------------------------------------ P3

def test_P3_constant_gradient_closed_forms_full_none_and_v():
    rows, cols, b1, b2, eps, lr = 4, 6, 0.9, 0.95, 1e-8, 1e-3
    g = RNG.standard_normal((rows, cols)) * 1e-3
    hp = O.HParams(lr=lr, beta1=b1, beta2=b2, eps=eps)
    full = _rand_block(rows, cols, mom_mode=O.MOM_FULL)
    none = _rand_block(rows, cols, mom_mode=O.MOM_NONE, lr_scale=0.75)
    bm = _rand_block(rows, cols, mom_mode=O.MOM_NONE, v_mode=O.V_BLOCKMEAN, v_group_rows=2)
    sf, sn, sb = O.new_state(full), O.new_state(none), O.new_state(bm)
    Wf = np.zeros((rows, cols)); Wn = Wf.copy(); Wb = Wf.copy()
    acc_f = np.zeros_like(Wf); acc_n = np.zeros_like(Wf); acc_b = np.zeros_like(Wf)
    for t in range(1, 16):
        Wf = O.block_step(Wf, g, sf, full, hp, t)
        Wn = O.block_step(Wn, g, sn, none, hp, t)
        Wb = O.block_step(Wb, g, sb, bm, hp, t)
        np.testing.assert_allclose(sf.m, (1 - b1 ** t) * g, rtol=1e-13)
        np.testing.assert_allclose(sf.v, (1 - b2 ** t) * g * g, rtol=1e-13)
        mean_sq = (g * g).reshape(2, 2 * cols).mean(axis=1)
        np.testing.assert_allclose(sb.v, (1 - b2 ** t) * mean_sq, rtol=1e-13)
        den = math.sqrt(1 - b2 ** t) * np.abs(g) + eps
        acc_f += np.clip((1 - b1 ** t) * g / den, -1, 1)
        acc_n += np.clip(g / den, -1, 1)
        den_b = np.sqrt((1 - b2 ** t) * np.repeat(mean_sq, 2))[:, None] + eps
        acc_b += np.clip(g / den_b, -1, 1)
        np.testing.assert_allclose(Wf, -lr * acc_f, rtol=1e-12, atol=1e-18)     # lambda = 0
        np.testing.assert_allclose(Wn, -lr * 0.75 * acc_n, rtol=1e-12, atol=1e-18)
        np.testing.assert_allclose(Wb, -lr * acc_b, rtol=1e-12, atol=1e-18)


def test_P3_constant_gradient_lowrank_exact_closed_form():
    rows, cols, r, b1 = 7, 5, 2, 0.9
    U, _ = np.linalg.qr(RNG.standard_normal((rows, cols)))
    Vt, _ = np.linalg.qr(RNG.standard_normal((cols, cols)))
    sig = np.array([5.0, 3.0, 1.0, 0.5, 0.25]) * 1e-3
    g = (U * sig) @ Vt.T
    head = (U[:, :r] * sig[:r]) @ Vt[:, :r].T
    tail = g - head
    blk = _rand_block(rows, cols, mom_mode=O.MOM_LOWRANK, rank=r)
    hp = O.HParams(beta1=b1)
    st = O.new_state(blk)
    W = np.zeros((rows, cols))
    for t in range(1, 15):
        W = O.block_step(W, g, st, blk, hp, t, solver="exact", keep=True)
        np.testing.assert_allclose(st.last["P"], (1 - b1 ** t) * head, rtol=0, atol=1e-15)
        np.testing.assert_allclose(st.last["m_t"], (1 - b1 ** t) * head + (1 - b1) * tail, atol=1e-15)
        np.testing.assert_allclose(st.last["r_t"], -(1 - b1) * tail, atol=1e-15)
        np.testing.assert_allclose(st.last["m_c"], (1 - b1 ** t) * head + tail, atol=1e-14)
    # rank(g) <= r: the corrected momentum is the full momentum
    g2 = head
    st = O.new_state(blk)
    for t in range(1, 8):
        O.block_step(W, g2, st, blk, hp, t, solver="exact", keep=True)
        np.testing.assert_allclose(st.last["m_c"], (1 - b1 ** t) * g2, atol=1e-15)


# ------------------------------------------------------------------------------------ P4

@pytest.mark.parametrize("solver", ["gd", "exact"])
def test_P4_proof_identity_along_a_trajectory(solver):
    """m_t - m^f_t = sum_{i=1}^{t-1} beta1^i r_{t-i} and m^c_t = g_t + c (P_{t-1} - P_t), for any solver
    (proof of Theorem 2, first display: m_t - m^f_t = beta1 (m_{t-1} - m^f_{t-1}) + beta1 r_{t-1})."""
    rows, cols, r, b1 = 24, 16, 3, 0.9
    blk = _rand_block(rows, cols, mom_mode=O.MOM_LOWRANK, rank=r)
    hp = O.HParams(beta1=b1)
    st = O.new_state(blk, O.init_L0(rows, r, 0, 0))
    W = RNG.standard_normal((rows, cols)) * 0.02
    mf = np.zeros((rows, cols))
    residuals = []
    c = b1 / (1 - b1)
    for t in range(1, 21):
        g = RNG.standard_normal((rows, cols)) * 1e-3 + 2e-3 * np.outer(np.sin(np.arange(rows)), np.cos(np.arange(cols)))
        W = O.block_step(W, g, st, blk, hp, t, solver=solver, keep=True)
        mf = (1 - b1) * g + b1 * mf
        want = sum(b1 ** i * residuals[t - 1 - i] for i in range(1, t))
        scale = np.abs(mf).max()
        assert np.abs(st.last["m_t"] - mf - want).max() < 1e-13 * scale + 1e-18
        assert np.abs(st.last["m_c"] - (g + c * (st.last["P_prev"] - st.last["P"]))).max() < 1e-12 * scale
        residuals.append(st.last["r_t"])


def test_P4_constant_residual_gives_theorem2_gap():
    """If r_t = r for all t >= 1 then m^c_t - m^f_t = -beta1^t r / (1 - beta1)  (r_0 = 0)."""
    b1, T = 0.9, 12
    r = 0.37
    # scalar recursion of the proof: d_t = beta1 d_{t-1} + beta1 r_{t-1}, d_0 = 0, r_0 = 0
    d = 0.0
    prev_r = 0.0
    for t in range(1, T + 1):
        d = b1 * d + b1 * prev_r
        prev_r = r
        gap = d - b1 * r / (1 - b1)
        assert abs(gap - (-(b1 ** t) * r / (1 - b1))) < 1e-14


# ------------------------------------------------------------------------------------ P5

def _alg2_scalar_rank1(M, l, rho, K):
    """Algorithm 2 for rank 1 with explicit index loops (no matrix products)."""
    m, n = len(l), len(rho)
    l = list(l); rho = list(rho)
    for k in range(1, K + 1):
        eta = 0.5 * (1 + math.cos(math.pi * k / K))
        E = [[l[i] * rho[j] - M[i][j] for j in range(n)] for i in range(m)]
        dl = [sum(E[i][j] * rho[j] for j in range(n)) for i in range(m)]
        dr = [sum(l[i] * E[i][j] for i in range(m)) for j in range(n)]
        l = [l[i] - eta * dl[i] for i in range(m)]
        rho = [rho[j] - eta * dr[j] for j in range(n)]
    return l, rho


@pytest.mark.parametrize("shape", [(2, 2), (3, 2), (2, 3)])
def test_P5_alg2_brute_force_rank1(shape):
    m, n = shape
    M = RNG.standard_normal((m, n))
    l0 = RNG.standard_normal(m) * 0.5
    r0 = RNG.standard_normal(n) * 0.5
    L, R = O.lowrank_refit_gd(M, l0[:, None], r0[None, :], 5)
    l, rho = _alg2_scalar_rank1(M.tolist(), l0.tolist(), r0.tolist(), 5)
    np.testing.assert_allclose(L[:, 0], l, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(R[0, :], rho, rtol=1e-13, atol=1e-15)


def test_P5_alg2_derivatives_by_finite_differences():
    """The printed derivatives are those of l = 0.5 ||L R - m_t||_F^2 (no factor 2)."""
    m, n, r = 4, 3, 2
    M = RNG.standard_normal((m, n)); L = RNG.standard_normal((m, r)); R = RNG.standard_normal((r, n))
    loss = lambda L_, R_: 0.5 * np.sum((L_ @ R_ - M) ** 2)
    h = 1e-6
    # one pass with K=2 has eta_1 = 0.5, eta_2 = 0: the move is -0.5 * derivative
    L1, R1 = O.lowrank_refit_gd(M, L, R, 2)
    dL = (L - L1) / 0.5
    dR = (R - R1) / 0.5
    for i in range(m):
        for k in range(r):
            Lp = L.copy(); Lp[i, k] += h; Lm = L.copy(); Lm[i, k] -= h
            assert abs((loss(Lp, R) - loss(Lm, R)) / (2 * h) - dL[i, k]) < 1e-6
    for k in range(r):
        for j in range(n):
            Rp = R.copy(); Rp[k, j] += h; Rm = R.copy(); Rm[k, j] -= h
            assert abs((loss(L, Rp) - loss(L, Rm)) / (2 * h) - dR[k, j]) < 1e-6


def test_P5_exact_solver_vs_2x2_closed_form_and_power_iteration():
    a, b, c, d = RNG.standard_normal(4)
    M = np.array([[a, b], [c, d]])
    S1 = a * a + b * b + c * c + d * d
    S2 = math.sqrt((a * a + b * b - c * c - d * d) ** 2 + 4 * (a * c + b * d) ** 2)
    s_small = math.sqrt((S1 - S2) / 2)
    L, R = O.lowrank_refit_exact(M, 1)
    assert abs(np.linalg.norm(L @ R - M) - s_small) < 1e-13
    # power iteration for the leading pair on a 5x4 matrix
    A = RNG.standard_normal((5, 4))
    x = np.ones(4)
    for _ in range(2000):
        x = A.T @ (A @ x); x /= np.linalg.norm(x)
    P_pow = np.outer(A @ x, x)
    L, R = O.lowrank_refit_exact(A, 1)
    np.testing.assert_allclose(L @ R, P_pow, atol=1e-10)


def test_alg2_descends_and_tracks_a_low_rank_target():
    rows, cols, r = 40, 30, 3
    M = (RNG.standard_normal((rows, r)) @ RNG.standard_normal((r, cols))) * 0.005   # curvature eta*||R R^T|| << 1
    L = O.init_L0(rows, r, 0, 7); R = np.zeros((r, cols))
    prev = np.linalg.norm(L @ R - M)
    for _ in range(300):
        L, R = O.lowrank_refit_gd(M, L, R, 5)
        cur = np.linalg.norm(L @ R - M)
        assert cur <= prev * (1 + 1e-12)
        prev = cur
    assert prev < 1e-3 * np.linalg.norm(M)


def test_init_L0_is_orthonormal_and_fp32():
    L0 = O.init_L0(200, 12, 3, 5)
    assert np.array_equal(L0, L0.astype(np.float32).astype(np.float64))
    np.testing.assert_allclose(L0.T @ L0, np.eye(12), atol=5e-7)
    assert not np.array_equal(L0, O.init_L0(200, 12, 3, 6))
    assert np.array_equal(L0, O.init_L0(200, 12, 3, 5))


# ------------------------------------------------------------------------------------ P6

def test_P6_blockmean_is_group_average_of_elementwise_v():
    rows, cols = 12, 5
    el = _rand_block(rows, cols, mom_mode=O.MOM_NONE)
    for gr in (0, 1, 3, 12):
        bm = _rand_block(rows, cols, mom_mode=O.MOM_NONE, v_mode=O.V_BLOCKMEAN, v_group_rows=gr)
        se, sb = O.new_state(el), O.new_state(bm)
        hp = O.HParams()
        W = np.zeros((rows, cols))
        for t in range(1, 9):
            g = RNG.standard_normal((rows, cols))
            O.block_step(W, g, se, el, hp, t)
            O.block_step(W, g, sb, bm, hp, t)
            k = rows if gr == 0 else gr
            np.testing.assert_allclose(sb.v, se.v.reshape(rows // k, k * cols).mean(axis=1), rtol=1e-13)


# ------------------------------------------------------------------------------------ P7

def test_P7_no_refit_or_zero_factors_reduce_to_no_momentum():
    rows, cols, r = 9, 6, 2
    none = _rand_block(rows, cols, mom_mode=O.MOM_NONE, weight_decay=0.1)
    lowr = _rand_block(rows, cols, mom_mode=O.MOM_LOWRANK, rank=r, weight_decay=0.1)
    for K, L0 in ((0, O.init_L0(rows, r, 0, 0)), (5, np.zeros((rows, r)))):
        hp = O.HParams(inner_iters=K)
        sn, sl = O.new_state(none), O.new_state(lowr, L0)
        Wn = RNG.standard_normal((rows, cols)) * 0.02; Wl = Wn.copy()
        for t in range(1, 7):
            g = RNG.standard_normal((rows, cols)) * 1e-3
            Wn = O.block_step(Wn, g, sn, none, hp, t)
            Wl = O.block_step(Wl, g, sl, lowr, hp, t)
            np.testing.assert_allclose(Wl, Wn, rtol=0, atol=1e-15)
            assert not sl.R.any()


def test_P7_last_pass_is_a_noop():
    M = RNG.standard_normal((6, 5)) * 0.1
    L = O.init_L0(6, 2, 0, 1); R = RNG.standard_normal((2, 5)) * 0.1
    L5, R5 = O.lowrank_refit_gd(M, L, R, 5)
    # four passes by hand with the K=5 step sizes
    La, Ra = L.copy(), R.copy()
    for k in (1, 2, 3, 4):
        eta = 0.5 * (1 + math.cos(math.pi * k / 5))
        E = La @ Ra - M
        La, Ra = La - eta * (E @ Ra.T), Ra - eta * (La.T @ E)
    assert np.array_equal(L5, La) and np.array_equal(R5, Ra)


# ------------------------------------------------------------------------------------ P8

def test_P8_zero_padded_rank_changes_nothing():
    rows, cols, r, pad = 10, 8, 3, 5
    M = RNG.standard_normal((rows, cols)) * 0.05
    L = O.init_L0(rows, r, 0, 2); R = RNG.standard_normal((r, cols)) * 0.05
    Lp = np.hstack([L, np.zeros((rows, pad - r))]); Rp = np.vstack([R, np.zeros((pad - r, cols))])
    L1, R1 = O.lowrank_refit_gd(M, L, R, 5)
    L2, R2 = O.lowrank_refit_gd(M, Lp, Rp, 5)
    np.testing.assert_allclose(L2[:, :r], L1, rtol=0, atol=1e-16)
    np.testing.assert_allclose(R2[:r], R1, rtol=0, atol=1e-16)
    assert not L2[:, r:].any() and not R2[r:].any()


# ------------------------------------------------------------------------------------ P10

def test_P10_blocks_are_independent():
    blocks = [
        O.Block(6, 4, O.MOM_FULL, weight_decay=0.1),
        O.Block(8, 6, O.MOM_LOWRANK, rank=2, weight_decay=0.1, v_mode=O.V_BLOCKMEAN, v_group_rows=2),
        O.Block(5, 3, O.MOM_NONE, lr_scale=0.75),
    ]
    L0 = {1: O.init_L0(8, 2, 0, 99)}
    a = O.AdaPMOracle(blocks, O.HParams(), L0=L0)
    b = O.AdaPMOracle([blocks[1]], O.HParams(), L0={0: L0[1]})
    Wa = [RNG.standard_normal((x.rows, x.cols)) * 0.02 for x in blocks]
    Wb = [Wa[1].copy()]
    for _ in range(6):
        gs = [RNG.standard_normal((x.rows, x.cols)) * 1e-3 for x in blocks]
        Wa = a.step(Wa, gs)
        Wb = b.step(Wb, [gs[1]])
    assert np.array_equal(Wa[1], Wb[0])
    assert np.array_equal(a.states[1].L, b.states[0].L)


# ------------------------------------------------------------------------------------ weight decay / clip

def test_weight_decay_is_decoupled_and_clip_is_elementwise():
    blk = _rand_block(1, 3, mom_mode=O.MOM_NONE, weight_decay=0.5)
    hp = O.HParams(lr=0.1, beta2=0.0, eps=0.0)       # v = g^2 -> ratio = sign(g)
    st = O.new_state(blk)
    W = np.array([[2.0, -4.0, 8.0]])
    g = np.array([[3.0, -0.5, 0.0]])
    hp.eps = 1e-8
    W1 = O.block_step(W, g, st, blk, hp, 1)
    want = W - 0.1 * (np.array([[1.0, -1.0, 0.0]]) + 0.5 * W)
    np.testing.assert_allclose(W1, want, rtol=1e-7)
    # the clamp acts per element: one large ratio does not shrink the others
    blk2 = _rand_block(1, 2, mom_mode=O.MOM_NONE)
    st2 = O.new_state(blk2); st2.v = np.array([[1.0, 1.0]])
    hp2 = O.HParams(lr=1.0, beta2=1.0, eps=0.0)
    W2 = O.block_step(np.zeros((1, 2)), np.array([[10.0, 0.25]]), st2, blk2, hp2, 1)
    np.testing.assert_allclose(W2, [[-1.0, -0.25]], rtol=1e-15)


# ------------------------------------------------------------------------------------ global gradient-norm clipping

def _three_blocks():
    blks = [O.Block(6, 5, O.MOM_FULL, weight_decay=0.1), O.Block(4, 7, O.MOM_NONE, lr_scale=0.75, weight_decay=0.1),
            O.Block(8, 6, O.MOM_LOWRANK, rank=2, v_mode=O.V_BLOCKMEAN, v_group_rows=2, weight_decay=0.1)]
    return blks


def test_clip_below_threshold_changes_nothing():
    """||g|| <= c gives s = 1: the clipped optimizer is the unclipped one, bit for bit."""
    blks = _three_blocks()
    a = O.AdaPMOracle(blks, O.HParams(max_grad_norm=1.0))
    b = O.AdaPMOracle(blks, O.HParams())
    Wa = [RNG.standard_normal((k.rows, k.cols)) for k in blks]
    Wb = [w.copy() for w in Wa]
    for _ in range(5):
        g = [RNG.standard_normal((k.rows, k.cols)) * 1e-3 for k in blks]      # norm ~ 0.01
        assert O.global_clip_scale(g, 1.0) == 1.0
        Wa, Wb = a.step(Wa, g), b.step(Wb, g)
        for x, y in zip(Wa, Wb):
            assert np.array_equal(x, y)


def test_clip_scale_is_threshold_over_global_norm():
    """Hand numbers: gradients (3, 4) and (12,) have global norm 13; c = 1 gives s = 1/13, c = 26 gives 1."""
    g = [np.array([[3.0, 4.0]]), np.array([[12.0]])]
    assert O.global_clip_scale(g, 1.0) == pytest.approx(1.0 / 13.0, rel=1e-15)
    assert O.global_clip_scale(g, 26.0) == 1.0
    assert O.global_clip_scale(g, math.inf) == 1.0
    assert O.global_clip_scale([np.zeros((2, 2))], 1.0) == 1.0
    # the norm is over all blocks together, not per block
    assert O.global_clip_scale(g[:1], 1.0) == pytest.approx(1.0 / 5.0, rel=1e-15)


def test_clip_constant_gradient_closed_forms_use_the_scaled_gradient():
    """P3 with clipping: a constant gradient g of global norm n > c behaves like the constant gradient (c/n) g."""
    b1, b2, c = 0.9, 0.95, 0.5
    blk = O.Block(4, 6, O.MOM_FULL)
    g = RNG.standard_normal((4, 6))
    s = c / np.linalg.norm(g)
    orc = O.AdaPMOracle([blk], O.HParams(max_grad_norm=c, clip=math.inf, beta1=b1, beta2=b2))
    W = [np.zeros((4, 6))]
    for t in range(1, 9):
        W = orc.step(W, [g])
        np.testing.assert_allclose(orc.states[0].m, (1 - b1 ** t) * s * g, rtol=1e-13)
        np.testing.assert_allclose(orc.states[0].v, (1 - b2 ** t) * (s * g) ** 2, rtol=1e-13)


def test_clip_matches_torch_clip_grad_norm_then_adamw():
    """All blocks FULL, debiased, no elementwise clamp: torch.nn.utils.clip_grad_norm_ followed by
    torch.optim.AdamW.  (torch divides by norm + 1e-6, hence the 2e-6 relative tolerance.)"""
    torch = pytest.importorskip("torch")
    shapes = [(5, 4), (3, 7), (1, 6)]
    W0 = [RNG.standard_normal(sh) for sh in shapes]
    ps = [torch.nn.Parameter(torch.tensor(w, dtype=torch.float64)) for w in W0]
    opt = torch.optim.AdamW(ps, lr=2e-3, betas=(0.9, 0.95), eps=1e-8, weight_decay=0.1)
    blks = [O.Block(r, c, O.MOM_FULL, weight_decay=0.1) for r, c in shapes]
    orc = O.AdaPMOracle(blks, O.HParams(lr=2e-3, clip=math.inf, adam_debias=True, max_grad_norm=1.0))
    W = [w.copy() for w in W0]
    for t in range(1, 9):
        g = [RNG.standard_normal(sh) * (3.0 if t % 2 else 0.05) for sh in shapes]     # above and below the threshold
        for p, gi in zip(ps, g):
            p.grad = torch.tensor(gi, dtype=torch.float64)
        torch.nn.utils.clip_grad_norm_(ps, 1.0)
        opt.step()
        W = orc.step(W, g)
        for w, p in zip(W, ps):
            np.testing.assert_allclose(w, p.detach().numpy(), rtol=2e-6, atol=1e-9)


def test_clip_applies_before_the_lowrank_target_and_the_second_moment():
    """The low-rank block sees s g in line 4 and in line 7: feeding the oracle s g without clipping is the same."""
    blk = O.Block(8, 6, O.MOM_LOWRANK, rank=2, v_mode=O.V_BLOCKMEAN, v_group_rows=2, weight_decay=0.1)
    L0 = O.init_L0(8, 2, 0, 0)
    a, b = O.new_state(blk, L0), O.new_state(blk, L0)
    hp = O.HParams()
    Wa = RNG.standard_normal((8, 6)); Wb = Wa.copy()
    for t in range(1, 6):
        g = RNG.standard_normal((8, 6))
        s = O.global_clip_scale([g], 0.3)
        assert s < 1.0
        Wa = O.block_step(Wa, g, a, blk, hp, t, gscale=s)
        Wb = O.block_step(Wb, s * g, b, blk, hp, t)
        assert np.array_equal(Wa, Wb) and np.array_equal(a.L, b.L) and np.array_equal(a.v, b.v)


# ------------------------------------------------------------------------------------ ablation switches

def test_correction_off_is_the_uncorrected_target_and_the_product_reading_differs_by_the_residual():
    """With Eq. 3 left out the update uses m_t (line 4) as it stands; the other reading of Section 4.2 uses L_t R_t.
    Their difference is the residual r_t of line 6, and with the correction on m^c = m_t - c r_t."""
    blk = O.Block(6, 5, O.MOM_LOWRANK, rank=2)
    L0 = O.init_L0(6, 2, 0, 0)
    W = RNG.standard_normal((6, 5))
    g = RNG.standard_normal((6, 5)) * 1e-2
    outs = {}
    for name, hp in (("on", O.HParams()), ("off", O.HParams(correction=False)),
                     ("product", O.HParams(correction=False, correction_off_uses_product=True))):
        st = O.new_state(blk, L0)
        st.R = RNG.standard_normal((2, 5)) * 1e-2          # a non-trivial previous product
        RNG2 = np.random.default_rng(3)
        st.R = RNG2.standard_normal((2, 5)) * 1e-2
        O.block_step(W, g, st, blk, hp, 1, keep=True)
        outs[name] = st.last
    m_t, r_t = outs["on"]["m_t"], outs["on"]["r_t"]
    b1 = 0.9
    np.testing.assert_allclose(outs["off"]["m_c"], m_t, rtol=0, atol=0)
    np.testing.assert_allclose(outs["product"]["m_c"] - outs["off"]["m_c"], r_t, rtol=1e-12, atol=1e-18)
    np.testing.assert_allclose(outs["on"]["m_c"], m_t - b1 / (1 - b1) * r_t, rtol=1e-12, atol=1e-18)
    # and the uncorrected target itself, from its definition
    P_prev = L0 @ (np.random.default_rng(3).standard_normal((2, 5)) * 1e-2)
    np.testing.assert_allclose(m_t, (1 - b1) * g + b1 * P_prev, rtol=1e-13)


def test_inner_lr_scale_multiplies_every_step_size():
    """inner_lr_scale = s runs Algorithm 2 with s eta_k: the same as the scalar loops of the brute-force pin with
    the schedule scaled, and s = 0 leaves the factors where they were."""
    m, n = 3, 2
    tgt = RNG.standard_normal((m, n))
    L0 = RNG.standard_normal((m, 1)); R0 = RNG.standard_normal((1, n))
    s = 0.37
    L, R = O.lowrank_refit_gd(tgt, L0, R0, 5, s)
    l = [float(x) for x in L0[:, 0]]; r = [float(x) for x in R0[0]]
    for k in range(1, 6):
        eta = s * 0.5 * (1.0 + math.cos(math.pi * k / 5))
        e = [[l[i] * r[j] - tgt[i, j] for j in range(n)] for i in range(m)]
        dl = [sum(e[i][j] * r[j] for j in range(n)) for i in range(m)]
        dr = [sum(l[i] * e[i][j] for i in range(m)) for j in range(n)]
        l = [l[i] - eta * dl[i] for i in range(m)]
        r = [r[j] - eta * dr[j] for j in range(n)]
    np.testing.assert_allclose(L[:, 0], l, rtol=1e-13)
    np.testing.assert_allclose(R[0], r, rtol=1e-13)
    L2, R2 = O.lowrank_refit_gd(tgt, L0, R0, 5, 0.0)
    assert np.array_equal(L2, L0) and np.array_equal(R2, R0)


# ------------------------------------------------------------------------------------ refresh period T

def test_refresh_period_one_is_algorithm_1_as_printed():
    blk = O.Block(8, 6, O.MOM_LOWRANK, rank=2, weight_decay=0.1)
    L0 = O.init_L0(8, 2, 0, 0)
    a, b = O.new_state(blk, L0), O.new_state(blk, L0)
    Wa = RNG.standard_normal((8, 6)); Wb = Wa.copy()
    for t in range(1, 7):
        g = RNG.standard_normal((8, 6)) * 1e-2
        Wa = O.block_step(Wa, g, a, blk, O.HParams(), t)
        Wb = O.block_step(Wb, g, b, blk, O.HParams(refresh_period=1), t)
        assert np.array_equal(Wa, Wb) and np.array_equal(a.L, b.L) and np.array_equal(a.R, b.R)


def test_refresh_period_holds_L_between_refreshes_and_moves_R():
    T = 3
    blk = O.Block(8, 6, O.MOM_LOWRANK, rank=2)
    st = O.new_state(blk, O.init_L0(8, 2, 0, 0))
    W = RNG.standard_normal((8, 6))
    for t in range(1, 9):
        L_before, R_before = st.L.copy(), st.R.copy()
        W = O.block_step(W, RNG.standard_normal((8, 6)) * 1e-2, st, blk, O.HParams(refresh_period=T), t, keep=True)
        if (t - 1) % T == 0:
            assert not np.array_equal(st.L, L_before)
        else:
            assert np.array_equal(st.L, L_before)
        assert not np.array_equal(st.R, R_before)
        # lines 6 and 8 are unchanged: the corrected momentum is g + c (P_{t-1} - P_t) whatever the solver did
        c = 0.9 / (1 - 0.9)
        np.testing.assert_allclose(st.last["m_c"], (st.last["m_t"] - 0.9 * st.last["P_prev"]) / 0.1
                                   + c * (st.last["P_prev"] - st.last["P"]), rtol=1e-10, atol=1e-15)


def test_held_L_passes_equal_scalar_loops_and_hit_least_squares_with_orthonormal_L():
    m, n = 3, 2
    tgt = RNG.standard_normal((m, n))
    L0 = RNG.standard_normal((m, 1)); R0 = RNG.standard_normal((1, n))
    L, R = O.lowrank_refit_gd(tgt, L0, R0, 5, 1.0, update_L=False)
    l = [float(x) for x in L0[:, 0]]; r = [float(x) for x in R0[0]]
    for k in range(1, 6):
        eta = 0.5 * (1.0 + math.cos(math.pi * k / 5))
        dr = [sum(l[i] * (l[i] * r[j] - tgt[i, j]) for i in range(m)) for j in range(n)]
        r = [r[j] - eta * dr[j] for j in range(n)]
    assert np.array_equal(L, L0)
    np.testing.assert_allclose(R[0], r, rtol=1e-13)
    # orthonormal L, one pass with step size exactly 1 (K = 1 would give eta_1 = 0, so use K = 2 scaled to eta_1 = 1):
    # R_1 = R_0 - (L^T L R_0 - L^T m) = L^T m, the least-squares solution for that L
    Q = np.linalg.qr(RNG.standard_normal((7, 3)))[0]
    tgt = RNG.standard_normal((7, 5))
    eta1 = 0.5 * (1.0 + math.cos(math.pi / 2))
    _, R1 = O.lowrank_refit_gd(tgt, Q, RNG.standard_normal((3, 5)), 2, 1.0 / eta1, update_L=False)
    np.testing.assert_allclose(R1, Q.T @ tgt, rtol=1e-12, atol=1e-14)


# ------------------------------------------------------------------------------------------------
# Data-driven L_0 (randomized range finder on the first gradient; not in the paper)
# ------------------------------------------------------------------------------------------------

def test_range_L0_is_orthonormal_and_equals_qr_up_to_column_signs():
    rng = np.random.default_rng(11)
    g = rng.standard_normal((60, 45)); om = rng.standard_normal((45, 7))
    L0 = O.init_L0_range(g, om)
    assert np.array_equal(L0, L0.astype(np.float32).astype(np.float64))
    assert np.abs(L0.T @ L0 - np.eye(7)).max() < 5e-7
    # Gram-Schmidt in column order is the thin QR factorisation with a positive diagonal
    Q, Rq = np.linalg.qr(g @ om)
    Q = Q * np.sign(np.diag(Rq))
    assert np.abs(L0 - Q).max() < 5e-7


def test_range_L0_spans_the_range_of_a_rank_r_gradient_whatever_omega_is():
    rng = np.random.default_rng(12)
    U, _ = np.linalg.qr(rng.standard_normal((50, 4)))
    g = U @ np.diag([3.0, 2.0, 1.0, 0.5]) @ rng.standard_normal((4, 30))
    P = U @ U.T
    for seed in (1, 2):
        L0 = O.init_L0_range(g, np.random.default_rng(seed).standard_normal((30, 4)))
        assert np.abs(L0 @ L0.T - P).max() < 1e-6          # the projector is unique, the basis is not
    # more columns than the gradient has rank: the first four span it, the rest are dropped (zero)
    L0 = O.init_L0_range(g, rng.standard_normal((30, 6)))
    assert np.abs(L0[:, :4] @ L0[:, :4].T - P).max() < 1e-6
    assert np.all(L0[:, 4:] == 0.0)


def test_range_L0_of_a_rank_one_gradient_and_of_a_zero_gradient():
    rng = np.random.default_rng(13)
    u = rng.standard_normal(20); v = rng.standard_normal(9)
    om = rng.standard_normal((9, 3))
    L0 = O.init_L0_range(np.outer(u, v), om)
    s = np.sign((v @ om)[0])
    assert np.abs(L0[:, 0] - s * u / np.linalg.norm(u)).max() < 1e-7
    assert np.all(L0[:, 1:] == 0.0)
    assert np.all(O.init_L0_range(np.zeros((20, 9)), om) == 0.0)


def test_a_dropped_column_of_L0_never_leaves_zero():
    """Algorithm 2 from (L_0, R_0 = 0) with a zero column j in L_0: row j of dl/dR is L[:, j]^T E = 0 and column j of
    dl/dL is E R[j, :]^T = 0, so the pair stays zero: the block simply runs at a lower rank."""
    rng = np.random.default_rng(14)
    g = np.outer(rng.standard_normal(12), rng.standard_normal(8))
    L0 = O.init_L0_range(g, rng.standard_normal((8, 3)))
    L, R = O.lowrank_refit_gd(0.1 * g + 0.01 * rng.standard_normal((12, 8)), L0, np.zeros((3, 8)), 5)
    assert np.all(L[:, 1:] == 0.0) and np.all(R[1:, :] == 0.0)
    assert np.abs(R[0]).max() > 0.0


# ------------------------------------------------------------------------------------------------
# Preconditioned inner passes (scaled gradient descent; not in the paper)
# ------------------------------------------------------------------------------------------------

def _one_pass_schedule(monkeypatch, etas):
    monkeypatch.setattr(O, "inner_schedule", lambda K: list(etas))


def test_scaled_gd_full_step_lands_on_the_two_least_squares_solutions(monkeypatch):
    """One pass with step size 1 and no damping: R' = argmin_R ||L R - m|| and L' = argmin_L ||L R - m||, each with
    the other factor at its old value (both derivatives are taken at the same point)."""
    rng = np.random.default_rng(21)
    m = rng.standard_normal((9, 7)); L = rng.standard_normal((9, 3)); R = rng.standard_normal((3, 7))
    _one_pass_schedule(monkeypatch, [1.0])
    L1, R1 = O.lowrank_refit_scaled_gd(m, L, R, 1, damping=0.0)
    np.testing.assert_allclose(R1, np.linalg.lstsq(L, m, rcond=None)[0], atol=1e-10)
    np.testing.assert_allclose(L1, np.linalg.lstsq(R.T, m.T, rcond=None)[0].T, atol=1e-10)


def test_scaled_gd_does_not_depend_on_how_the_product_is_split():
    """(L, R) -> (L Q, Q^-1 R) leaves L R unchanged; without damping the preconditioned passes then produce the same
    product again (plain gradient descent does not)."""
    rng = np.random.default_rng(22)
    m = rng.standard_normal((10, 8)); L = rng.standard_normal((10, 3)); R = rng.standard_normal((3, 8))
    Q = rng.standard_normal((3, 3)) + 3 * np.eye(3)
    La, Ra = O.lowrank_refit_scaled_gd(m, L, R, 5, scale=0.5, damping=0.0)
    Lb, Rb = O.lowrank_refit_scaled_gd(m, L @ Q, np.linalg.inv(Q) @ R, 5, scale=0.5, damping=0.0)
    np.testing.assert_allclose(La @ Ra, Lb @ Rb, atol=1e-9)
    Lc, Rc = O.lowrank_refit_gd(m, L @ Q, np.linalg.inv(Q) @ R, 5, 0.01)
    Ld, Rd = O.lowrank_refit_gd(m, L, R, 5, 0.01)
    assert np.abs(Lc @ Rc - Ld @ Rd).max() > 1e-4


def test_scaled_gd_rank_one_equals_scalar_loops():
    rng = np.random.default_rng(23)
    m = rng.standard_normal((3, 2)); L = rng.standard_normal((3, 1)); R = rng.standard_normal((1, 2))
    damping = 0.05
    l = [float(x) for x in L[:, 0]]; r = [float(x) for x in R[0]]
    for eta in O.inner_schedule(5):
        rr = sum(x * x for x in r); ll = sum(x * x for x in l)
        sr = 1.0 / (rr + damping * rr + O.PRECOND_FLOOR); sl = 1.0 / (ll + damping * ll + O.PRECOND_FLOOR)
        e = [[l[i] * r[j] - m[i, j] for j in range(2)] for i in range(3)]
        dl = [sum(e[i][j] * r[j] for j in range(2)) * sr for i in range(3)]
        dr = [sum(l[i] * e[i][j] for i in range(3)) * sl for j in range(2)]
        l = [l[i] - eta * dl[i] for i in range(3)]
        r = [r[j] - eta * dr[j] for j in range(2)]
    L5, R5 = O.lowrank_refit_scaled_gd(m, L, R, 5, damping=damping)
    np.testing.assert_allclose(L5[:, 0], l, atol=1e-12)
    np.testing.assert_allclose(R5[0], r, atol=1e-12)


def test_scaled_gd_with_scalar_gram_matrices_is_plain_gd_with_rescaled_steps(monkeypatch):
    """L with orthogonal columns of squared length d and R with orthogonal rows of squared length c: the
    preconditioners are multiples of the identity, so one pass equals Algorithm 2's with the derivatives divided by
    c (1 + damping) and d (1 + damping)."""
    rng = np.random.default_rng(24)
    QL, _ = np.linalg.qr(rng.standard_normal((8, 3))); QR, _ = np.linalg.qr(rng.standard_normal((6, 3)))
    L = 2.0 * QL; R = 0.5 * QR.T
    m = rng.standard_normal((8, 6))
    _one_pass_schedule(monkeypatch, [0.4])
    L1, R1 = O.lowrank_refit_scaled_gd(m, L, R, 1, damping=0.1)
    E = L @ R - m
    np.testing.assert_allclose(L1, L - 0.4 * (E @ R.T) / (0.25 * 1.1), atol=1e-12)
    np.testing.assert_allclose(R1, R - 0.4 * (L.T @ E) / (4.0 * 1.1), atol=1e-12)


def test_scaled_gd_from_R_zero_moves_R_only_and_block_step_uses_it():
    rng = np.random.default_rng(25)
    L0 = O.init_L0(12, 3, 0, 4); m = rng.standard_normal((12, 9)) * 1e-3
    L1, R1 = O.lowrank_refit_scaled_gd(m, L0, np.zeros((3, 9)), 5)
    assert np.all(np.isfinite(L1)) and np.all(np.isfinite(R1)) and np.abs(R1).max() > 0
    blk = O.Block(rows=12, cols=9, mom_mode=O.MOM_LOWRANK, rank=3)
    g = rng.standard_normal((12, 9)) * 1e-3
    outs = []
    for pre in (False, True):
        st = O.new_state(blk, L0)
        O.block_step(rng.standard_normal((12, 9)) * 0 + 0.01, g, st, blk, O.HParams(inner_precond=pre), 1)
        outs.append((st.L.copy(), st.R.copy()))
    Ls, Rs = O.lowrank_refit_scaled_gd(0.1 * g, L0, np.zeros((3, 9)), 5)
    np.testing.assert_allclose(outs[1][0], Ls, atol=1e-14)
    np.testing.assert_allclose(outs[1][1], Rs, atol=1e-14)
    assert np.abs(outs[0][1] - outs[1][1]).max() > 0
