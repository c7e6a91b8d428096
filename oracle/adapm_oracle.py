"""fp64 CPU oracle of the AdaPM optimizer step.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain definition the CUDA library is checked against.
It is written from the paper's Algorithm 1 (low-rank update with correction),
Algorithm 2 (gradient-descent refit of the factors), Eq. 4 (full momentum) and
the Adam-mini combination of Section 5.1.3 / Related Work (one second-moment
scalar per parameter group = the group average of Adam's statistic).  It shares
no code with the CUDA path, imports nothing from it, and only the tests, the
smoke check and the benchmark's CPU-baseline leg may call it.

Everything is float64.  Inputs are the exact values the device receives
(fp32 parameters, fp32 or bf16-rounded gradients) widened to float64.

Readings of the paper taken here (each is a choice; the paper does not settle it):
  * Algorithm 1's last line prints "lambda x_t"; x_t is read as W_t
    (decoupled weight decay).
  * clip(., 1) is the elementwise clamp of the ratio to [-1, 1].
  * No 1/(1-beta^t) debiasing appears in Algorithm 1, so none is applied
    unless `adam_debias` is set (used only to compare with textbook AdamW).
  * Algorithm 2 evaluates both partial derivatives at the same (L, R) and
    then updates both factors (simultaneous, not alternating).
  * The step sizes eta_k = 0.5 (1 + cos(pi k / K)), k = 1..K, are absolute;
    eta_K = 0, so the K-th pass changes nothing.
  * L_0 = R_0 = 0 is a stationary point of Algorithm 2 (both derivatives are
    zero there), so the factors would never move.  R_0 = 0 is kept (L_0 R_0 = 0,
    hence m_1 is unchanged) and L_0 is given orthonormal columns: Gaussian draws
    orthonormalised by modified Gram-Schmidt, rounded to fp32 (`init_L0`).
  * "No momentum" blocks use m^c_t = g_t.
  * "Global gradient clipping at a threshold of 1.0" (Section 5.1, Setups) is the usual clipping by the global
    norm: with n = the 2-norm of all gradients of the step taken together, every gradient is multiplied by
    s = min(1, c / n) before Algorithm 1 sees it (lines 4 and 7 both use the clipped gradient).  n = 0 gives s = 1.
  * The ablation "without bias correction" (Section 5.1.2, Fig. 4a) is read as m^c := m_t, i.e. Eq. 3 left out
    and nothing else changed.  Section 4.2's phrase "directly applying L_t R_t as the momentum" would instead
    give m^c := L_t R_t; the two differ by the residual r_t.  `correction=False` takes the first reading and
    `correction_off_uses_product=True` the second.
  * "Update frequency T" (Section 5.1: T = 100; Section 5.1.2 sweeps it) is set but never defined: Algorithms 1
    and 2 refit both factors at every step.  Reading taken for `refresh_period` = T > 1, PARITY UNPINNED (the
    paper fixes nothing to check it against): the full refit of Algorithm 2 runs at steps 1, T+1, 2T+1, ...; at
    the steps in between L is held and only R moves, by the R half of Algorithm 2 (same schedule, same K).
    Everything else (lines 4, 6-9) is unchanged, so the correction of Eq. 3 still compensates the residual.
    T = 1 is Algorithm 1 as printed.  The function itself is pinned to the mathematics (tests): T = 1 equals
    the default, held-L passes equal scalar loops, and with orthonormal L and step size 1 one pass lands on
    the least-squares R = L^T m_t.
  * A data-driven L_0 (`init_L0_range`; not in the paper, PARITY UNPINNED against it): instead of Gaussian
    draws, L_0 spans what the first gradient spans.  With Omega an n x r Gaussian matrix handed in by the caller,
    L_0 = the columns of g_1 Omega orthonormalised by modified Gram-Schmidt, in order, rounded to fp32 (the
    randomized range finder); R_0 = 0 as before.  A column whose remainder after the projections has less than
    1e-8 of its squared length left (g_1 has rank below r) becomes zero and stays zero under Algorithm 2.
  * Preconditioned inner passes (`inner_precond`, `lowrank_refit_scaled_gd`; not in the paper, PARITY UNPINNED
    against it): each derivative of Algorithm 2 is multiplied by the damped inverse of the other factor's Gram
    matrix (scaled gradient descent), which makes the pass independent of how the product L R is split between
    the factors; everything else of Algorithm 2 (warm start, schedule, simultaneous update) is kept.
Parity with the authors' unreleased code on these readings is unpinned; what is
pinned (tests/test_oracle_pins.py) is this oracle against closed forms, special
cases, a library optimizer, the proof identity of Theorem 2 and brute force.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np

MOM_NONE = 0
MOM_FULL = 1
MOM_LOWRANK = 2
V_ELEMENT = 0
V_BLOCKMEAN = 1


@dataclass
class Block:
    """One parameter block W in R^{rows x cols} and how it is treated."""
    rows: int
    cols: int
    mom_mode: int = MOM_FULL
    rank: int = 0
    v_mode: int = V_ELEMENT
    v_group_rows: int = 0        # BLOCKMEAN: consecutive rows per group; 0 = the whole block
    lr_scale: float = 1.0
    weight_decay: float = 0.0
    offset: int = 0              # element offset in a flat buffer (bookkeeping only)

    def n_groups(self) -> int:
        if self.v_mode == V_ELEMENT:
            return self.rows * self.cols
        return 1 if self.v_group_rows == 0 else self.rows // self.v_group_rows


@dataclass
class HParams:
    lr: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.95
    eps: float = 1e-8
    clip: float = 1.0            # math.inf disables the clamp
    inner_iters: int = 5         # K of Algorithm 2
    inner_lr_scale: float = 1.0  # multiplies every eta_k; 1 = as printed
    adam_debias: bool = False
    correction: bool = True      # Eq. 3 on; off: m^c := m_t
    correction_off_uses_product: bool = False   # with correction off: m^c := L_t R_t instead of m_t
    max_grad_norm: float = math.inf   # global clipping threshold c; inf disables
    refresh_period: int = 1      # T: both factors are refitted at steps 1, T+1, 2T+1, ...; in between only R
    inner_precond: bool = False  # preconditioned passes (ScaledGD) instead of Algorithm 2's plain ones
    precond_damping: float = 1e-3     # delta = damping * trace(Gram) / r is added to the Gram matrix's diagonal


@dataclass
class BlockState:
    m: Optional[np.ndarray] = None   # full momentum m^f (FULL blocks)
    L: Optional[np.ndarray] = None   # rows x rank
    R: Optional[np.ndarray] = None   # rank x cols
    v: Optional[np.ndarray] = None   # rows x cols, or one value per group
    last: Dict[str, np.ndarray] = field(default_factory=dict)   # transients of the last step


# ----------------------------------------------------------------------------------------------
# Algorithm 2 (Appendix B): K gradient-descent passes on || L R - m_t ||_F^2
# ----------------------------------------------------------------------------------------------

def inner_schedule(K: int) -> List[float]:
    """eta_k = 0.5 (1 + cos(pi k / K)) for k = 1..K (Appendix B, text below Algorithm 2)."""
    return [0.5 * (1.0 + math.cos(math.pi * k / K)) for k in range(1, K + 1)]


def lowrank_refit_gd(m_t: np.ndarray, L_prev: np.ndarray, R_prev: np.ndarray, K: int,
                     scale: float = 1.0, update_L: bool = True):
    """Algorithm 2: warm start at (L_{t-1}, R_{t-1}); both derivatives from the same point.
    update_L=False holds L and moves only R (the steps between two refreshes, see `refresh_period`)."""
    L = np.array(L_prev, dtype=np.float64, copy=True)
    R = np.array(R_prev, dtype=np.float64, copy=True)
    if K <= 0:
        return L, R
    for eta in inner_schedule(K):
        E = L @ R - m_t                  # L R - m_t
        dL = E @ R.T                     # dl/dL = (L R - m_t) R^T
        dR = L.T @ E                     # dl/dR = L^T (L R - m_t)
        if update_L:
            L = L - (scale * eta) * dL
        R = R - (scale * eta) * dR
    return L, R


PRECOND_FLOOR = 1e-30    # keeps the damped Gram matrix invertible when the factor is exactly zero (R_0 = 0)


def damped_inverse(G: np.ndarray, damping: float) -> np.ndarray:
    """(G + delta I)^-1 with delta = damping * trace(G) / r + PRECOND_FLOOR, G a symmetric r x r Gram matrix."""
    r = G.shape[0]
    delta = damping * np.trace(G) / r + PRECOND_FLOOR
    return np.linalg.inv(G + delta * np.eye(r))


def lowrank_refit_scaled_gd(m_t: np.ndarray, L_prev: np.ndarray, R_prev: np.ndarray, K: int, scale: float = 1.0,
                            damping: float = 1e-3, update_L: bool = True):
    """Preconditioned passes in place of Algorithm 2's (a variant; not in the paper): the scaled gradient descent
    of Tong, Ma and Chi (2021) for low-rank factorisation, with a damped preconditioner,
        L <- L - eta_k (L R - m_t) R^T (R R^T + delta_R I)^-1,   R <- R - eta_k (L^T L + delta_L I)^-1 L^T (L R - m_t),
    both from the same point, same schedule and warm start as Algorithm 2."""
    L = np.array(L_prev, dtype=np.float64, copy=True)
    R = np.array(R_prev, dtype=np.float64, copy=True)
    if K <= 0:
        return L, R
    for eta in inner_schedule(K):
        E = L @ R - m_t
        dL = (E @ R.T) @ damped_inverse(R @ R.T, damping)
        dR = damped_inverse(L.T @ L, damping) @ (L.T @ E)
        if update_L:
            L = L - (scale * eta) * dL
        R = R - (scale * eta) * dR
    return L, R


def lowrank_refit_exact(m_t: np.ndarray, r: int):
    """A true minimiser of Eq. 1: the rank-r truncated SVD (Eckart-Young).  Used only by pins."""
    U, S, Vt = np.linalg.svd(m_t, full_matrices=False)
    return U[:, :r] * S[:r], Vt[:r, :]


def init_L0(rows: int, rank: int, seed: int, block_index: int) -> np.ndarray:
    """Orthonormal-column L_0: Gaussian draws, modified Gram-Schmidt in fp64, rounded to fp32."""
    key = np.array([(0xAD0A << 32) | (seed & 0xFFFFFFFF), block_index & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64)
    G = np.random.Generator(np.random.Philox(key=key)).standard_normal((rows, rank))
    Q = np.zeros_like(G)
    for j in range(rank):
        q = G[:, j].copy()
        for i in range(j):
            q -= (Q[:, i] @ q) * Q[:, i]
        Q[:, j] = q / math.sqrt(q @ q)
    return Q.astype(np.float32).astype(np.float64)


RANGE_DROP = 1e-8     # a column of g Omega that keeps less than this share of its squared length is dropped


def init_L0_range(g: np.ndarray, omega: np.ndarray) -> np.ndarray:
    """Data-driven L_0: modified Gram-Schmidt over the columns of Y = g Omega, in order (randomized range finder).
    g: [rows, cols], omega: [cols, rank].  Returns [rows, rank] with orthonormal (or zero) columns, rounded to fp32."""
    Y = np.asarray(g, dtype=np.float64) @ np.asarray(omega, dtype=np.float64)
    rows, rank = Y.shape
    Q = np.zeros_like(Y)
    for j in range(rank):
        q = Y[:, j].copy()
        n0 = q @ q
        for i in range(j):
            q -= (Q[:, i] @ q) * Q[:, i]
        n1 = q @ q
        if n0 > 0.0 and n1 > RANGE_DROP * n0:
            Q[:, j] = q / math.sqrt(n1)
    return Q.astype(np.float32).astype(np.float64)


# ----------------------------------------------------------------------------------------------
# Second-order statistic: Algorithm 1 line 7, or its group average (Adam-mini combination)
# ----------------------------------------------------------------------------------------------

def second_moment(v_prev: np.ndarray, g: np.ndarray, blk: Block, beta2: float) -> np.ndarray:
    if blk.v_mode == V_ELEMENT:
        return beta2 * v_prev + (1.0 - beta2) * (g * g)
    gr = blk.rows if blk.v_group_rows == 0 else blk.v_group_rows
    assert blk.rows % gr == 0, "v_group_rows must divide rows"
    mean_sq = (g * g).reshape(blk.rows // gr, gr * blk.cols).mean(axis=1)
    return beta2 * v_prev + (1.0 - beta2) * mean_sq


def _v_per_element(v: np.ndarray, blk: Block) -> np.ndarray:
    if blk.v_mode == V_ELEMENT:
        return v
    gr = blk.rows if blk.v_group_rows == 0 else blk.v_group_rows
    return np.repeat(v, gr)[:, None] * np.ones((1, blk.cols))


# ----------------------------------------------------------------------------------------------
# One step of one block
# ----------------------------------------------------------------------------------------------

def new_state(blk: Block, L0: Optional[np.ndarray] = None) -> BlockState:
    st = BlockState()
    if blk.v_mode == V_ELEMENT:
        st.v = np.zeros((blk.rows, blk.cols))
    else:
        st.v = np.zeros(blk.n_groups())
    if blk.mom_mode == MOM_FULL:
        st.m = np.zeros((blk.rows, blk.cols))
    elif blk.mom_mode == MOM_LOWRANK:
        st.L = np.zeros((blk.rows, blk.rank)) if L0 is None else np.array(L0, dtype=np.float64)
        st.R = np.zeros((blk.rank, blk.cols))
        assert st.L.shape == (blk.rows, blk.rank)
    return st


def global_clip_scale(grads, max_grad_norm: float) -> float:
    """s = min(1, c / ||g||_2) with the norm taken over all gradients of the step (Section 5.1, Setups)."""
    if not math.isfinite(max_grad_norm):
        return 1.0
    total = 0.0
    for g in grads:
        g = np.asarray(g, dtype=np.float64)
        total += float(np.sum(g * g))
    norm = math.sqrt(total)
    if norm == 0.0:
        return 1.0
    return min(1.0, max_grad_norm / norm)


def block_step(W: np.ndarray, g: np.ndarray, st: BlockState, blk: Block, hp: HParams, t: int,
               solver: str = "gd", keep: bool = False, gscale: float = 1.0) -> np.ndarray:
    """Advance one block by one step (t is 1-based).  Returns W_{t+1}; updates `st` in place.
    `gscale` is the step's global clipping factor (global_clip_scale over ALL blocks' gradients)."""
    W = np.asarray(W, dtype=np.float64).reshape(blk.rows, blk.cols)
    g = np.asarray(g, dtype=np.float64).reshape(blk.rows, blk.cols)
    if gscale != 1.0:
        g = gscale * g
    b1 = hp.beta1

    # line 7 (or its group average)
    st.v = second_moment(st.v, g, blk, hp.beta2)

    if blk.mom_mode == MOM_NONE:
        m_c = g
    elif blk.mom_mode == MOM_FULL:
        st.m = (1.0 - b1) * g + b1 * st.m                      # Eq. 4
        m_c = st.m
    elif blk.mom_mode == MOM_LOWRANK:
        P_prev = st.L @ st.R
        m_t = (1.0 - b1) * g + b1 * P_prev                     # line 4
        if solver == "gd":
            refresh = hp.refresh_period <= 1 or (t - 1) % hp.refresh_period == 0
            if hp.inner_precond:
                L, R = lowrank_refit_scaled_gd(m_t, st.L, st.R, hp.inner_iters, hp.inner_lr_scale, hp.precond_damping,
                                               update_L=refresh)
            else:
                L, R = lowrank_refit_gd(m_t, st.L, st.R, hp.inner_iters, hp.inner_lr_scale, update_L=refresh)   # line 5
        elif solver == "exact":
            L, R = lowrank_refit_exact(m_t, blk.rank)
        else:
            raise ValueError(solver)
        r_t = L @ R - m_t                                       # line 6
        if hp.correction:
            m_c = m_t - (b1 * r_t) / (1.0 - b1)                # line 8
        else:
            m_c = L @ R if hp.correction_off_uses_product else m_t
        st.L, st.R = L, R
        if keep:
            st.last = {"m_t": m_t, "r_t": r_t, "P_prev": P_prev, "P": L @ R}
        if not (np.isfinite(L).all() and np.isfinite(R).all()):
            raise FloatingPointError("low-rank factors are not finite")
    else:
        raise ValueError(blk.mom_mode)

    v_el = _v_per_element(st.v, blk)
    if hp.adam_debias:
        m_hat = m_c / (1.0 - b1 ** t)
        v_hat = v_el / (1.0 - hp.beta2 ** t)
    else:
        m_hat, v_hat = m_c, v_el
    ratio = m_hat / (np.sqrt(v_hat) + hp.eps)
    if math.isfinite(hp.clip):
        ratio = np.clip(ratio, -hp.clip, hp.clip)
    if keep:
        st.last["m_c"] = m_c
        st.last["ratio"] = ratio
    # line 9, with x_t read as W_t
    return W - (hp.lr * blk.lr_scale) * (ratio + blk.weight_decay * W)


# ----------------------------------------------------------------------------------------------
# A whole parameter set: blocks are independent of each other
# ----------------------------------------------------------------------------------------------

class AdaPMOracle:
    def __init__(self, blocks: List[Block], hp: HParams, L0: Optional[Dict[int, np.ndarray]] = None,
                 seed: int = 0):
        self.blocks = list(blocks)
        self.hp = hp
        self.t = 0
        self.states: List[BlockState] = []
        for i, b in enumerate(self.blocks):
            l0 = None
            if b.mom_mode == MOM_LOWRANK:
                l0 = L0[i] if (L0 is not None and i in L0) else init_L0(b.rows, b.rank, seed, i)
            self.states.append(new_state(b, l0))

    def step(self, params: List[np.ndarray], grads: List[np.ndarray], solver: str = "gd",
             keep: bool = False) -> List[np.ndarray]:
        self.t += 1
        s = global_clip_scale(grads, self.hp.max_grad_norm)
        return [block_step(W, g, st, b, self.hp, self.t, solver, keep, gscale=s)
                for W, g, st, b in zip(params, grads, self.states, self.blocks)]

    def state_floats(self) -> int:
        """Persistent optimizer-state size in scalars (momentum, factors, second moment)."""
        n = 0
        for b in self.blocks:
            n += b.n_groups()
            if b.mom_mode == MOM_FULL:
                n += b.rows * b.cols
            elif b.mom_mode == MOM_LOWRANK:
                n += b.rank * (b.rows + b.cols)
        return n
