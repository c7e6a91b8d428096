"""Shared plumbing of the GPU-vs-oracle parity tests (and of the smoke check).

Drives the CUDA library through its C ABI and the fp64 oracle on the same seeded inputs, and
compares them block by block.  Nothing here computes any part of the optimizer step.
"""
from __future__ import annotations

import math
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass
from typing import Dict, Iterable, List, Optional, Sequence

import numpy as np

import workloads as WL
import paper_2510_09103_b200 as A
from oracle import adapm_oracle as O
from oracle import planner_oracle as P


def rel_err(gpu: np.ndarray, ref: np.ndarray) -> float:
    """max_i |gpu_i - ref_i| / max_i |ref_i|  (0 if both are all zero)."""
    ref = np.asarray(ref, dtype=np.float64).ravel()
    gpu = np.asarray(gpu, dtype=np.float64).ravel()
    if not np.isfinite(gpu).all():
        return math.inf
    den = np.abs(ref).max() if ref.size else 0.0
    num = np.abs(gpu - ref).max() if ref.size else 0.0
    if den == 0.0:
        return 0.0 if num == 0.0 else math.inf
    return float(num / den)


def oracle_blocks_from(blocks: Sequence) -> List[O.Block]:
    # lr_scale / weight_decay are fp32 fields of the descriptor: the oracle sees exactly those values
    return [O.Block(rows=b.rows, cols=b.cols, mom_mode=b.mom_mode, rank=b.rank, v_mode=b.v_mode,
                    v_group_rows=b.v_group_rows, lr_scale=float(b.lr_scale), weight_decay=float(b.weight_decay),
                    offset=b.offset) for b in blocks]


def assert_plans_equal(gpu_blocks: Sequence, orc_blocks: Sequence[O.Block]) -> None:
    assert len(gpu_blocks) == len(orc_blocks)
    for i, (g, o) in enumerate(zip(gpu_blocks, orc_blocks)):
        got = (g.offset, g.rows, g.cols, g.mom_mode, g.rank, g.v_mode, g.v_group_rows)
        want = (o.offset, o.rows, o.cols, o.mom_mode, o.rank, o.v_mode, o.v_group_rows)
        assert got == want, f"block {i}: library {got} != oracle {want}"
        assert np.float32(g.lr_scale) == np.float32(o.lr_scale)
        assert np.float32(g.weight_decay) == np.float32(o.weight_decay)


def tensor_block_map(tensors: Sequence[WL.Tensor]) -> List[List[int]]:
    """Block indices each tensor becomes (a fused QKV tensor becomes three)."""
    out, k = [], 0
    for t in tensors:
        n = 3 if t.role == WL.ROLE_QKV_FUSED else 1
        out.append(list(range(k, k + n)))
        k += n
    return out


CANARY = 7.25e9          # a value no optimizer quantity takes
CANARY_WORDS = 256


@dataclass
class Tolerances:
    fp32: float = 1e-5       # elementwise / reduction paths
    contraction: float = 2e-3
    # Regression bound of the tensor-core path: about 20 times the worst error seen on the five sets (4e-6 on R
    # after 20 steps).  The contract stays `contraction`; this bound only makes a loss of accuracy visible.
    tensor_regression: float = 1e-4


class ParityRun:
    """One workload on the GPU (all blocks) and in the oracle (a chosen subset of blocks)."""

    def __init__(self, w: WL.Workload, blockmean: bool, oracle_blocks: Optional[Iterable[int]] = None,
                 lowrank_path: int = A.PATH_AUTO, pooled_grads: bool = False, hp_overrides: Optional[dict] = None,
                 device: str = "cuda:0", custom_blocks: Optional[Sequence] = None, grad_scale=None,
                 shadow: bool = False):
        """grad_scale: step -> power of two that multiplies every gradient of that step (exact in bf16 and fp32);
        shadow: also ask for the bf16 copy of the parameters."""
        import torch
        self.torch = torch
        self.w = w
        self.dev = torch.device(device)
        v_mode = A.V_BLOCKMEAN if blockmean else A.V_ELEMENT
        if custom_blocks is not None:
            # hand-made partition: one synthetic tensor per block, packed at the blocks' own offsets
            self.blocks = list(custom_blocks)
            self.total = -(-max(b.offset + b.rows * b.cols for b in self.blocks) // 8) * 8
            w.tensors = [WL.Tensor(f"b{i}", WL.ROLE_OTHER, b.rows, b.cols) for i, b in enumerate(self.blocks)]
            self.t2b = [[i] for i in range(len(self.blocks))]
        else:
            self.blocks, self.total = A.adapm_plan_default(w.tensors, w.rank_pct, w.rank_override, v_mode,
                                                           w.weight_decay)
            orc_plan = P.plan(w.tensors, w.weight_decay, w.rank_pct, blockmean, w.rank_override)
            assert_plans_equal(self.blocks, orc_plan)
            assert self.total == P.total_elems(w.tensors)
            self.t2b = tensor_block_map(w.tensors)
        self.b2t = {b: ti for ti, bs in enumerate(self.t2b) for b in bs}
        self.sel = sorted(set(range(len(self.blocks)) if oracle_blocks is None else oracle_blocks))
        self.sel_tensors = {self.b2t[b] for b in self.sel}

        hpk = dict(lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps, clip=1.0, inner_iters=5, inner_lr_scale=1.0,
                   grad_dtype=A.GRAD_BF16 if w.grad_dtype == "bf16" else A.GRAD_F32, lowrank_path=lowrank_path, seed=0)
        hpk.update(hp_overrides or {})
        self.hp = A.hparams(**hpk)
        self.ctx = A.adapm_create(self.blocks, self.hp)

        # parameters
        host = np.zeros(self.total, dtype=np.float32)
        cursor_blocks = self.blocks
        for ti, t in enumerate(w.tensors):
            off = cursor_blocks[self.t2b[ti][0]].offset
            host[off:off + t.numel] = WL.init_params(t, ti).ravel()
        self.params = torch.from_numpy(host).to(self.dev)
        self.host_params0 = host
        gdt = torch.bfloat16 if w.grad_dtype == "bf16" else torch.float32
        self.grads = torch.zeros(self.total, dtype=gdt, device=self.dev)
        # canary words: behind the state and the workspace, and in every gap between the state's sub-buffers
        n_state = self.ctx.adapm_state_bytes() // 4
        n_work = max(self.ctx.adapm_workspace_bytes() // 4, 64)
        self._state_full = torch.zeros(n_state + CANARY_WORDS, dtype=torch.float32, device=self.dev)
        self._work_full = torch.zeros(n_work + CANARY_WORDS, dtype=torch.float32, device=self.dev)
        self.state, self.work = self._state_full[:n_state], self._work_full[:n_work]
        self.ctx.adapm_set_workspace(self.work)
        self.ctx.adapm_state_init(self.state)
        self._state_full[n_state:] = CANARY
        self._work_full[n_work:] = CANARY
        used = []
        for bi in range(len(self.blocks)):
            for which in (A.STATE_M, A.STATE_L, A.STATE_R, A.STATE_V):
                off, cnt = self.ctx.adapm_state_layout(bi, which)
                if cnt > 0:
                    used.append((off, off + cnt))
        used.sort()
        self._gaps, cur = [], 0
        for a0, a1 in used:
            assert a0 >= cur, "state sub-buffers overlap"
            if a0 > cur:
                self._gaps.append((cur, a0))
            cur = a1
        if cur < n_state:
            self._gaps.append((cur, n_state))
        if len(self._gaps) <= 4096:
            for a0, a1 in self._gaps:
                self.state[a0:a1] = CANARY
        else:
            self._gaps = []
        self.grad_scale = grad_scale
        self.shadow = None
        if shadow:
            self.shadow = torch.zeros(self.total, dtype=torch.bfloat16, device=self.dev)
            self.ctx.adapm_set_shadow_params(self.shadow)

        # oracle side: its own L_0, injected into the GPU state so that both start from the same factors
        # the C ABI takes its hyperparameters as fp32: the oracle gets the same (rounded) values
        f32 = lambda x: float(np.float32(x))
        oh = O.HParams(lr=f32(hpk["lr"]), beta1=f32(hpk["beta1"]), beta2=f32(hpk["beta2"]), eps=f32(hpk["eps"]),
                       clip=f32(hpk["clip"]), inner_iters=hpk["inner_iters"], inner_lr_scale=f32(hpk["inner_lr_scale"]),
                       adam_debias=bool(hpk.get("adam_debias", 0)), correction=bool(hpk.get("correction", 1)),
                       max_grad_norm=(f32(hpk["max_grad_norm"]) if hpk.get("max_grad_norm", 0) > 0 else math.inf),
                       refresh_period=max(1, int(hpk.get("refresh_period", 0))),
                       inner_precond=bool(hpk.get("inner_precond", 0)),
                       precond_damping=f32(hpk.get("precond_damping", 1e-3)))
        self.ohp = oh
        self.ostate: Dict[int, O.BlockState] = {}
        self.oW: Dict[int, np.ndarray] = {}
        self.oblk: Dict[int, O.Block] = {}
        for bi, ob in enumerate(oracle_blocks_from(self.blocks)):
            b = self.blocks[bi]
            L0 = None
            if b.mom_mode == A.MOM_LOWRANK:
                L0 = O.init_L0(b.rows, b.rank, 0, bi)
                off, cnt = self.ctx.adapm_state_layout(bi, A.STATE_L)
                assert cnt == b.rows * b.rank
                self.state[off:off + cnt] = torch.from_numpy(L0.astype(np.float32).ravel()).to(self.dev)
            if bi in self.sel:
                self.oblk[bi] = ob
                self.ostate[bi] = O.new_state(ob, L0)
                self.oW[bi] = host[b.offset:b.offset + b.rows * b.cols].astype(np.float64).reshape(b.rows, b.cols)
        self.pool = WL.GradPool(w) if pooled_grads else None
        self.t = 0
        self._pinned = None

    # ------------------------------------------------------------------------------------------
    def _grad_raw(self, ti: int, step: int):
        t = self.w.tensors[ti]
        k = np.float32(self.grad_scale(step)) if self.grad_scale else None
        if self.pool is not None and ti not in self.sel_tensors:
            raw = self.pool.window(ti, step, t.numel)
            if k is not None:      # a power of two: exact on the stored values
                raw = WL.to_grad_dtype(WL.bf16_bits_to_f32(raw) * k if self.w.grad_dtype == "bf16" else raw * k,
                                       self.w.grad_dtype)[1]
            return None, raw
        x = WL.grad_for_tensor(self.w, ti, step)
        if k is not None:
            x = x * k
        vals, raw = WL.to_grad_dtype(x, self.w.grad_dtype)
        return vals, raw.ravel()

    def step(self) -> None:
        torch = self.torch
        self.t += 1
        np_dt = np.uint16 if self.w.grad_dtype == "bf16" else np.float32
        if self._pinned is None:
            tdt = torch.int16 if self.w.grad_dtype == "bf16" else torch.float32
            self._pinned = torch.zeros(self.total, dtype=tdt).pin_memory()
        host = self._pinned.numpy().view(np_dt)
        vals_of: Dict[int, np.ndarray] = {}

        def fill(ti: int):
            vals, raw = self._grad_raw(ti, self.t)
            off = self.blocks[self.t2b[ti][0]].offset
            host[off:off + raw.size] = raw
            if ti in self.sel_tensors:
                vals_of[ti] = vals

        with ThreadPoolExecutor(max_workers=8) as ex:
            list(ex.map(fill, range(len(self.w.tensors))))
        self.grads.view(self._pinned.dtype).copy_(self._pinned, non_blocking=False)
        self.ctx.adapm_step(self.params, self.grads, self.state, self.t)
        # the step's clipping factor for the oracle: from ALL gradients (the gaps between tensors hold zeros)
        gscale = 1.0
        if math.isfinite(self.ohp.max_grad_norm):
            allg = WL.bf16_bits_to_f32(host) if self.w.grad_dtype == "bf16" else host
            gscale = O.global_clip_scale([allg[i:i + (1 << 24)] for i in range(0, allg.size, 1 << 24)],
                                         self.ohp.max_grad_norm)
        self.last_gscale = gscale

        for bi in self.sel:
            b = self.blocks[bi]
            ti = self.b2t[bi]
            t_off = self.blocks[self.t2b[ti][0]].offset
            g = vals_of[ti].ravel()[b.offset - t_off: b.offset - t_off + b.rows * b.cols]
            self.oW[bi] = O.block_step(self.oW[bi], g.astype(np.float64), self.ostate[bi], self.oblk[bi], self.ohp, self.t,
                                       gscale=gscale)

    # ------------------------------------------------------------------------------------------
    def _state_slice(self, bi: int, which: int) -> np.ndarray:
        off, cnt = self.ctx.adapm_state_layout(bi, which)
        return self.state[off:off + cnt].cpu().numpy()

    def compare(self, tol: Tolerances = Tolerances()) -> Dict[str, float]:
        """Worst relative error per kind over the oracle's blocks; asserts the tolerances."""
        self.torch.cuda.synchronize()
        worst = {"W": 0.0, "W_lowrank": 0.0, "dW": 0.0, "dW_lowrank": 0.0, "v": 0.0, "m": 0.0, "L": 0.0, "R": 0.0,
                 "P": 0.0}
        on_tensor = self.w.grad_dtype == "bf16" and self.hp.lowrank_path != A.PATH_SIMT
        for bi in self.sel:
            b = self.blocks[bi]
            st = self.ostate[bi]
            n = b.rows * b.cols
            Wg = self.params[b.offset:b.offset + n].cpu().numpy()
            eW = rel_err(Wg, self.oW[bi])
            # The displacement W_t - W_0 is what the steps produced; |W| itself is ~100 times larger than one
            # step's update and would hide an error in it.  (fp32 rounding of W: |W| 2^-24 per step, relative to
            # a displacement of at least lr per step wherever the ratio is clamped.)
            W0 = self.host_params0[b.offset:b.offset + n].astype(np.float64)
            eD = rel_err(Wg.astype(np.float64) - W0, self.oW[bi].ravel() - W0)
            ev = rel_err(self._state_slice(bi, A.STATE_V), st.v)
            worst["v"] = max(worst["v"], ev)
            assert ev <= tol.fp32, f"block {bi} step {self.t}: v error {ev:.3e}"
            if b.mom_mode == A.MOM_LOWRANK:
                Lg = self._state_slice(bi, A.STATE_L).reshape(b.rows, b.rank)
                Rg = self._state_slice(bi, A.STATE_R).reshape(b.rank, b.cols)
                eL, eR = rel_err(Lg, st.L), rel_err(Rg, st.R)
                eP = rel_err(Lg.astype(np.float64) @ Rg.astype(np.float64), st.L @ st.R)
                for k, e in (("L", eL), ("R", eR), ("P", eP), ("W_lowrank", eW), ("dW_lowrank", eD)):
                    worst[k] = max(worst[k], e)
                    what = f"block {bi} ({b.rows}x{b.cols} r{b.rank}) step {self.t}: {k} error {e:.3e}"
                    # The displacement of a low-rank block is judged with group scalars v only.  With a per-element
                    # v the update of an element is (g - c dP) / (sqrt(1-beta2) |g|): where g is near zero the error
                    # of dP is divided by that gradient, and the element's update is as uncertain as P's smallest
                    # entries are, whatever the arithmetic.  (L, R, P and W are still compared.)
                    if k == "dW_lowrank" and b.v_mode == A.V_ELEMENT:
                        continue
                    assert e <= tol.contraction, what
                    if on_tensor and b.cols % 8 == 0 and b.rank <= 256 and k != "dW_lowrank":
                        assert e <= tol.tensor_regression, what + " (regression bound)"
            else:
                worst["W"] = max(worst["W"], eW)
                worst["dW"] = max(worst["dW"], eD)
                assert eW <= tol.fp32, f"block {bi} step {self.t}: W error {eW:.3e}"
                # the displacement carries the fp32 rounding of W (2^-24 |W| per step) against a movement of ~lr per step
                assert eD <= 20 * tol.fp32, f"block {bi} step {self.t}: displacement error {eD:.3e}"
                if b.mom_mode == A.MOM_FULL:
                    em = rel_err(self._state_slice(bi, A.STATE_M), st.m)
                    worst["m"] = max(worst["m"], em)
                    assert em <= tol.fp32, f"block {bi} step {self.t}: m error {em:.3e}"
        return worst

    def check_canaries(self) -> None:
        """No kernel wrote behind the state or the workspace, or between two sub-buffers of the state."""
        self.torch.cuda.synchronize()
        n_state, n_work = self.state.numel(), self.work.numel()
        assert bool((self._state_full[n_state:] == CANARY).all()), "a kernel wrote behind the state buffer"
        assert bool((self._work_full[n_work:] == CANARY).all()), "a kernel wrote behind the workspace"
        for a0, a1 in self._gaps:
            assert bool((self._state_full[a0:a1] == CANARY).all()), f"a kernel wrote into the state gap [{a0}, {a1})"

    def close(self) -> None:
        try:
            if getattr(self, "_state_full", None) is not None and self.state.data_ptr() == self._state_full.data_ptr():
                self.check_canaries()
        finally:
            self.ctx.adapm_destroy()


def sample_blocks(blocks: Sequence, per_class: int = 1) -> List[int]:
    """One (or a few) block(s) of every distinct (mode, rows, cols, rank, v_group_rows) class."""
    seen: Dict[tuple, int] = {}
    out = []
    for i, b in enumerate(blocks):
        key = (b.mom_mode, b.rows, b.cols, b.rank, b.v_group_rows)
        if seen.get(key, 0) < per_class:
            seen[key] = seen.get(key, 0) + 1
            out.append(i)
    return out
