"""ctypes binding of libadapm.so: argument marshalling only.

Every function here has the name of the C entry point it calls (include/adapm.h).  All arithmetic
of the optimizer step runs in the library's CUDA kernels; there is no Python or CPU fallback, and
loading fails loudly when the shared library is missing.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence, Tuple

from . import build as _build

MOM_NONE, MOM_FULL, MOM_LOWRANK = 0, 1, 2
V_ELEMENT, V_BLOCKMEAN = 0, 1
GRAD_F32, GRAD_BF16 = 0, 1
PATH_AUTO, PATH_SIMT, PATH_TENSOR = 0, 1, 2
STATE_M, STATE_L, STATE_R, STATE_V = 0, 1, 2, 3
FLAG_NO_PANEL_TEAMS, FLAG_FORCE_PANEL_TEAMS, FLAG_NO_SUMSQ_FOLD, FLAG_CHECK_FINITE = 1, 2, 4, 8
ST_WAIT_TEAM, ST_NONFINITE_GRAD = 32, 64

EXPORTS = (
    "adapm_version", "adapm_strerror", "adapm_last_cuda_error", "adapm_plan_default", "adapm_create",
    "adapm_destroy", "adapm_state_bytes", "adapm_state_breakdown", "adapm_state_layout",
    "adapm_workspace_bytes", "adapm_set_workspace", "adapm_state_init", "adapm_set_lr", "adapm_step",
    "adapm_step_bytes", "adapm_step_flops", "adapm_launch_count", "adapm_get_status",
    "adapm_group_meansq_scratch_bytes", "adapm_group_meansq", "adapm_set_profiling", "adapm_get_launch_times",
    "adapm_launch_kind_name", "adapm_group_meansq_static", "adapm_state_changed", "adapm_selftest_expired_wait", "adapm_set_shadow_params",
    "adapm_init_omega_floats", "adapm_init_omega_layout", "adapm_state_init_from_grads",
)


class adapm_tensor(C.Structure):
    _fields_ = [("role", C.c_int32), ("heads", C.c_int32), ("rows", C.c_int64), ("cols", C.c_int64)]


class adapm_block(C.Structure):
    _fields_ = [("offset", C.c_int64), ("rows", C.c_int32), ("cols", C.c_int32), ("mom_mode", C.c_int32),
                ("rank", C.c_int32), ("v_mode", C.c_int32), ("v_group_rows", C.c_int32),
                ("lr_scale", C.c_float), ("weight_decay", C.c_float)]

    def numel(self) -> int:
        return self.rows * self.cols

    def as_tuple(self) -> tuple:
        return (self.offset, self.rows, self.cols, self.mom_mode, self.rank, self.v_mode, self.v_group_rows,
                self.lr_scale, self.weight_decay)


class adapm_hparams(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("clip", C.c_float), ("inner_iters", C.c_int32), ("inner_lr_scale", C.c_float),
                ("grad_dtype", C.c_int32), ("adam_debias", C.c_int32), ("correction", C.c_int32),
                ("lowrank_path", C.c_int32), ("seed", C.c_uint64), ("flags", C.c_uint32),
                ("max_grad_norm", C.c_float), ("refresh_period", C.c_int32), ("tune_panels", C.c_int32),
                ("tune_stage_k", C.c_int32), ("inner_precond", C.c_int32), ("precond_damping", C.c_float)]


def hparams(lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, clip=1.0, inner_iters=5, inner_lr_scale=1.0,
            grad_dtype=GRAD_BF16, adam_debias=0, correction=1, lowrank_path=PATH_AUTO, seed=0, flags=0,
            max_grad_norm=0.0, refresh_period=0, tune_panels=0, tune_stage_k=0, inner_precond=0,
            precond_damping=1e-3) -> adapm_hparams:
    return adapm_hparams(lr, beta1, beta2, eps, clip, inner_iters, inner_lr_scale, grad_dtype, adam_debias,
                         correction, lowrank_path, seed, flags, max_grad_norm, refresh_period, tune_panels,
                         tune_stage_k, inner_precond, precond_damping)


class AdapmError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {strerror(code)} ({code}) {last_cuda_error()}".strip())


_lib: Optional[C.CDLL] = None


def lib_path() -> str:
    return _build.LIB_PATH


def load(build_if_missing: bool = True) -> C.CDLL:
    """Load libadapm.so (building it with nvcc first if it is absent or stale)."""
    global _lib
    if _lib is not None:
        return _lib
    if build_if_missing and _build.needs_build():
        _build.build()
    if not os.path.exists(_build.LIB_PATH):
        raise RuntimeError(f"{_build.LIB_PATH} is missing: the CUDA library was not built; there is no fallback")
    lib = C.CDLL(_build.LIB_PATH)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    sig = {
        "adapm_version": (C.c_int, []),
        "adapm_strerror": (C.c_char_p, [C.c_int]),
        "adapm_last_cuda_error": (C.c_char_p, []),
        "adapm_plan_default": (C.c_int, [C.POINTER(adapm_tensor), i64, i32, i32, i32, C.c_float,
                                         C.POINTER(adapm_block), i64, C.POINTER(i64), C.POINTER(i64)]),
        "adapm_create": (C.c_int, [C.POINTER(adapm_block), i64, C.POINTER(adapm_hparams), C.POINTER(vp)]),
        "adapm_destroy": (None, [vp]),
        "adapm_state_bytes": (sz, [vp]),
        "adapm_state_breakdown": (C.c_int, [vp, C.POINTER(sz), C.POINTER(sz), C.POINTER(sz), C.POINTER(sz)]),
        "adapm_state_layout": (C.c_int, [vp, i64, C.c_int, C.POINTER(i64), C.POINTER(i64)]),
        "adapm_workspace_bytes": (sz, [vp]),
        "adapm_set_workspace": (C.c_int, [vp, vp, sz]),
        "adapm_state_init": (C.c_int, [vp, vp, vp]),
        "adapm_set_lr": (C.c_int, [vp, C.c_float]),
        "adapm_step": (C.c_int, [vp, vp, vp, vp, i64, vp]),
        "adapm_step_bytes": (sz, [vp]),
        "adapm_step_flops": (C.c_double, [vp]),
        "adapm_launch_count": (i64, [vp]),
        "adapm_get_status": (C.c_int, [vp, vp, C.POINTER(i32)]),
        "adapm_group_meansq_scratch_bytes": (sz, [i64, i64]),
        "adapm_group_meansq": (C.c_int, [vp, i32, i64, i64, vp, vp, sz, vp]),
        "adapm_group_meansq_static": (C.c_int, [vp, i32, i64, i64, vp, vp]),
        "adapm_set_profiling": (C.c_int, [vp, i32]),
        "adapm_get_launch_times": (C.c_int, [vp, C.POINTER(C.c_float), C.POINTER(i32), i64, C.POINTER(i64)]),
        "adapm_launch_kind_name": (C.c_char_p, [i32]),
        "adapm_state_changed": (C.c_int, [vp]),
        "adapm_selftest_expired_wait": (C.c_int, [vp, vp]),
        "adapm_set_shadow_params": (C.c_int, [vp, vp]),
        "adapm_init_omega_floats": (i64, [vp]),
        "adapm_init_omega_layout": (C.c_int, [vp, i64, C.POINTER(i64), C.POINTER(i64)]),
        "adapm_state_init_from_grads": (C.c_int, [vp, vp, vp, vp, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load().adapm_strerror(code).decode()


def last_cuda_error() -> str:
    return load().adapm_last_cuda_error().decode()


def _check(code: int, what: str) -> None:
    if code != 0:
        raise AdapmError(code, what)


def adapm_version() -> int:
    return load().adapm_version()


def adapm_plan_default(tensors: Sequence, rank_pct: int = 5, rank_override: int = 0, v_mode: int = V_BLOCKMEAN,
                       weight_decay: float = 0.1) -> Tuple[List[adapm_block], int]:
    """tensors: objects with .role .heads .rows .cols.  Returns (blocks, total_elems)."""
    lib = load()
    n = len(tensors)
    arr = (adapm_tensor * n)(*[adapm_tensor(t.role, t.heads, t.rows, t.cols) for t in tensors])
    n_out, total = C.c_int64(0), C.c_int64(0)
    _check(lib.adapm_plan_default(arr, n, rank_pct, rank_override, v_mode, weight_decay, None, 0,
                                  C.byref(n_out), C.byref(total)), "adapm_plan_default(size)")
    out = (adapm_block * n_out.value)()
    _check(lib.adapm_plan_default(arr, n, rank_pct, rank_override, v_mode, weight_decay, out, n_out.value,
                                  C.byref(n_out), C.byref(total)), "adapm_plan_default")
    return list(out), total.value


def _ptr(x) -> int:
    """Device (or host) address of a torch tensor, an int address, or None."""
    if x is None:
        return 0
    if isinstance(x, int):
        return x
    return x.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


class Context:
    """Owns one adapm_ctx.  Methods are named after the C calls they forward to."""

    def __init__(self, blocks: Sequence[adapm_block], hp: adapm_hparams):
        self._lib = load()
        self.blocks = list(blocks)
        self.hp = hp
        arr = (adapm_block * len(self.blocks))(*self.blocks)
        h = C.c_void_p()
        _check(self._lib.adapm_create(arr, len(self.blocks), C.byref(hp), C.byref(h)), "adapm_create")
        self._h = h
        self._workspace = None

    def adapm_destroy(self) -> None:
        if getattr(self, "_h", None):
            self._lib.adapm_destroy(self._h)
            self._h = None

    close = adapm_destroy

    def __del__(self):
        try:
            self.adapm_destroy()
        except Exception:
            pass

    def adapm_state_bytes(self) -> int:
        return self._lib.adapm_state_bytes(self._h)

    def adapm_state_breakdown(self) -> dict:
        a, b, c, d = C.c_size_t(), C.c_size_t(), C.c_size_t(), C.c_size_t()
        _check(self._lib.adapm_state_breakdown(self._h, C.byref(a), C.byref(b), C.byref(c), C.byref(d)),
               "adapm_state_breakdown")
        return {"full_m": a.value, "L": b.value, "R": c.value, "v": d.value}

    def adapm_state_layout(self, block: int, which: int) -> Tuple[int, int]:
        off, cnt = C.c_int64(), C.c_int64()
        _check(self._lib.adapm_state_layout(self._h, block, which, C.byref(off), C.byref(cnt)), "adapm_state_layout")
        return off.value, cnt.value

    def adapm_workspace_bytes(self) -> int:
        return self._lib.adapm_workspace_bytes(self._h)

    def adapm_set_workspace(self, buf, nbytes: Optional[int] = None) -> None:
        if nbytes is None:
            nbytes = buf.numel() * buf.element_size() if buf is not None else 0
        _check(self._lib.adapm_set_workspace(self._h, _ptr(buf), nbytes), "adapm_set_workspace")
        self._workspace = buf          # keep the caller's buffer alive

    def adapm_state_init(self, state, stream=None) -> None:
        _check(self._lib.adapm_state_init(self._h, _ptr(state), _stream(stream)), "adapm_state_init")

    def adapm_init_omega_floats(self) -> int:
        return self._lib.adapm_init_omega_floats(self._h)

    def adapm_init_omega_layout(self, block: int) -> Tuple[int, int]:
        off, cnt = C.c_int64(), C.c_int64()
        _check(self._lib.adapm_init_omega_layout(self._h, block, C.byref(off), C.byref(cnt)), "adapm_init_omega_layout")
        return off.value, cnt.value

    def adapm_state_init_from_grads(self, state, grads, omega, stream=None) -> None:
        _check(self._lib.adapm_state_init_from_grads(self._h, _ptr(state), _ptr(grads), _ptr(omega), _stream(stream)),
               "adapm_state_init_from_grads")

    def adapm_set_lr(self, lr: float) -> None:
        _check(self._lib.adapm_set_lr(self._h, lr), "adapm_set_lr")

    def adapm_step(self, params, grads, state, t: int, stream=None) -> None:
        _check(self._lib.adapm_step(self._h, _ptr(params), _ptr(grads), _ptr(state), t, _stream(stream)),
               "adapm_step")

    def adapm_set_shadow_params(self, buf) -> None:
        _check(self._lib.adapm_set_shadow_params(self._h, _ptr(buf)), "adapm_set_shadow_params")
        self._shadow = buf             # keep the caller's buffer alive

    def adapm_state_changed(self) -> None:
        _check(self._lib.adapm_state_changed(self._h), "adapm_state_changed")

    def adapm_selftest_expired_wait(self, stream=None) -> None:
        _check(self._lib.adapm_selftest_expired_wait(self._h, _stream(stream)), "adapm_selftest_expired_wait")

    def adapm_step_bytes(self) -> int:
        return self._lib.adapm_step_bytes(self._h)

    def adapm_step_flops(self) -> float:
        return self._lib.adapm_step_flops(self._h)

    def adapm_launch_count(self) -> int:
        return self._lib.adapm_launch_count(self._h)

    def adapm_set_profiling(self, on: bool) -> None:
        _check(self._lib.adapm_set_profiling(self._h, 1 if on else 0), "adapm_set_profiling")

    def adapm_get_launch_times(self) -> List[Tuple[str, float]]:
        """[(kernel kind, milliseconds)] of the last profiled step, in launch order."""
        n = C.c_int64()
        _check(self._lib.adapm_get_launch_times(self._h, None, None, 0, C.byref(n)), "adapm_get_launch_times(size)")
        ms = (C.c_float * n.value)()
        kinds = (C.c_int32 * n.value)()
        _check(self._lib.adapm_get_launch_times(self._h, ms, kinds, n.value, C.byref(n)), "adapm_get_launch_times")
        return [(self._lib.adapm_launch_kind_name(k).decode(), float(t)) for k, t in zip(kinds, ms)]

    def adapm_get_status(self, stream=None) -> int:
        st = C.c_int32(0)
        rc = self._lib.adapm_get_status(self._h, _stream(stream), C.byref(st))
        if rc not in (0, -7):
            _check(rc, "adapm_get_status")
        return st.value


def adapm_create(blocks: Sequence[adapm_block], hp: adapm_hparams) -> Context:
    return Context(blocks, hp)


def adapm_group_meansq_scratch_bytes(n_groups: int, group_elems: int) -> int:
    return load().adapm_group_meansq_scratch_bytes(n_groups, group_elems)


def adapm_group_meansq(g, grad_dtype: int, n_groups: int, group_elems: int, out, scratch, stream=None) -> None:
    nbytes = scratch.numel() * scratch.element_size()
    _check(load().adapm_group_meansq(_ptr(g), grad_dtype, n_groups, group_elems, _ptr(out), _ptr(scratch), nbytes,
                                     _stream(stream)), "adapm_group_meansq")


STATIC_SCRATCH_FLOATS = 1 << 18


def adapm_group_meansq_static(g, grad_dtype: int, n_groups: int, group_elems: int, out, stream=None) -> None:
    """Block mean of g^2 with the library's built-in scratch: for callers that must not allocate device
    memory.  Limit: n_groups * ceil(group_elems / 2048) <= STATIC_SCRATCH_FLOATS.  Calls that may overlap
    on the GPU share the scratch and race; keep them on one stream."""
    _check(load().adapm_group_meansq_static(_ptr(g), grad_dtype, n_groups, group_elems, _ptr(out), _stream(stream)),
           "adapm_group_meansq_static")
