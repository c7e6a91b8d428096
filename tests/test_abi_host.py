"""Host-side checks that need no GPU: the library loads, exports what the header declares, the C
planner equals the oracle's planner bit for bit, and bad descriptors are rejected before any kernel."""
import ctypes
import os
import re

import pytest

import workloads as WL
import paper_2510_09103_b200 as A
from oracle import planner_oracle as P

from harness import assert_plans_equal

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "adapm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(adapm_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = A.load()
    declared = _declared_functions()
    assert set(A.EXPORTS) <= set(declared)
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in adapm.h but not exported by libadapm.so"
    assert A.adapm_version() >= 100
    assert A.strerror(-2) and A.strerror(-99) == "unknown error"


@pytest.mark.parametrize("name", WL.WORKLOAD_NAMES)
@pytest.mark.parametrize("blockmean", [True, False])
def test_c_planner_equals_oracle_planner(name, blockmean):
    w = WL.get_workload(name)
    blocks, total = A.adapm_plan_default(w.tensors, w.rank_pct, 0, A.V_BLOCKMEAN if blockmean else A.V_ELEMENT,
                                         w.weight_decay)
    assert_plans_equal(blocks, P.plan(w.tensors, w.weight_decay, w.rank_pct, blockmean))
    assert total == P.total_elems(w.tensors)


@pytest.mark.parametrize("rank", [8, 32, 128])
def test_c_planner_rank_override(rank):
    w = WL.get_workload("llama350m")
    blocks, _ = A.adapm_plan_default(w.tensors, 5, rank)
    assert_plans_equal(blocks, P.plan(w.tensors, w.weight_decay, 5, True, rank))


def _create_code(blocks, **hp):
    lib = A.load()
    arr = (A.adapm_block * len(blocks))(*blocks) if blocks else None
    h = ctypes.c_void_p()
    hpar = A.hparams(**hp)
    rc = lib.adapm_create(arr, len(blocks), ctypes.byref(hpar), ctypes.byref(h))
    if rc == 0:
        lib.adapm_destroy(h)
    return rc


def test_create_rejects_bad_descriptors_on_the_host():
    ok = A.adapm_block(0, 16, 16, A.MOM_LOWRANK, 4, A.V_BLOCKMEAN, 4, 1.0, 0.1)
    bad = lambda **kw: A.adapm_block(*[kw.get(f, getattr(ok, f)) for f, _ in A.adapm_block._fields_])
    assert _create_code([]) == -1                                    # empty partition
    assert _create_code([bad(offset=4)]) == -2                       # offset not a multiple of 8
    assert _create_code([bad(rank=0)]) == -3
    assert _create_code([bad(rank=17)]) == -3                        # rank above min(m, n)
    assert _create_code([bad(v_group_rows=5)]) == -3                 # does not divide rows
    assert _create_code([bad(mom_mode=7)]) == -1
    assert _create_code([bad(rows=0)]) == -3
    assert _create_code([ok, bad(offset=128)]) == -1                 # overlapping blocks
    assert _create_code([ok], beta1=1.0) == -3
    assert _create_code([ok], grad_dtype=9) == -1
    assert _create_code([ok], inner_iters=-1) == -3
    assert _create_code([ok], refresh_period=-1) == -3
    assert _create_code([ok], max_grad_norm=-1.0) == -3
    assert _create_code([ok], max_grad_norm=float("nan")) == -3
    assert _create_code([ok], tune_stage_k=32) == -3
    assert _create_code([ok], tune_panels=4) == -3
    assert _create_code([ok], inner_precond=2) == -1
    assert _create_code([ok], inner_precond=1, precond_damping=-1.0) == -3
    assert _create_code([ok], inner_precond=1, precond_damping=float("nan")) == -3


def test_hparams_struct_matches_the_header():
    """The ctypes mirror of adapm_hparams lists the header's fields in the header's order."""
    text = open(os.path.join(ROOT, "include", "adapm.h")).read()
    body = text[text.index("typedef struct {\n  float   lr, beta1"):text.index("} adapm_hparams;")]
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    names = []
    for decl in body.split(";"):
        decl = decl.replace("typedef struct {", "").strip()
        if not decl:
            continue
        first, *rest = decl.split(",")
        names.append(first.split()[-1])
        names += [r.strip() for r in rest]
    assert names == [f for f, _ in A.adapm_hparams._fields_]


def test_planner_rejects_bad_input():
    lib = A.load()
    t = (A.adapm_tensor * 1)(A.adapm_tensor(WL.ROLE_QKV_FUSED, 4, 10, 8))   # rows not a multiple of 3
    n, tot = ctypes.c_int64(), ctypes.c_int64()
    assert lib.adapm_plan_default(t, 1, 5, 0, 1, 0.1, None, 0, ctypes.byref(n), ctypes.byref(tot)) == -1
    t = (A.adapm_tensor * 1)(A.adapm_tensor(WL.ROLE_MLP, 0, 8, 8))
    out = (A.adapm_block * 1)()
    assert lib.adapm_plan_default(t, 1, 5, 0, 1, 0.1, out, 0, ctypes.byref(n), ctypes.byref(tot)) == -3   # no room
    assert lib.adapm_plan_default(t, 1, 5, 0, 3, 0.1, None, 0, ctypes.byref(n), ctypes.byref(tot)) == -1  # bad v_mode


def test_no_cpu_fallback_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    ok = A.adapm_block(0, 16, 16, A.MOM_FULL, 0, A.V_ELEMENT, 0, 1.0, 0.1)
    assert _create_code([ok]) == -4            # ADAPM_ECUDA: the library refuses, nothing runs on the CPU
    assert "cuda" in A.last_cuda_error().lower()
