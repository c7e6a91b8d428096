"""B200-native AdaPM optimizer step: a C-ABI CUDA library (csrc/, include/adapm.h) and its ctypes binding."""
from .binding import (  # noqa: F401
    MOM_NONE, MOM_FULL, MOM_LOWRANK, V_ELEMENT, V_BLOCKMEAN, GRAD_F32, GRAD_BF16, PATH_AUTO, PATH_SIMT,
    PATH_TENSOR, FLAG_NO_PANEL_TEAMS, FLAG_FORCE_PANEL_TEAMS, FLAG_NO_SUMSQ_FOLD, FLAG_CHECK_FINITE, ST_WAIT_TEAM, ST_NONFINITE_GRAD, STATE_M, STATE_L, STATE_R, STATE_V, EXPORTS, AdapmError, Context, adapm_block, adapm_hparams,
    adapm_tensor, adapm_create, adapm_plan_default, adapm_version, adapm_group_meansq,
    adapm_group_meansq_scratch_bytes, adapm_group_meansq_static, STATIC_SCRATCH_FLOATS, hparams, lib_path, load, strerror, last_cuda_error,
)
