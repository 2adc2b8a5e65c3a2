"""B200-native (sm_100a) Based sequence mixers: Taylor linear attention prefill and
decode, and sliding-window softmax attention, behind the C ABI of include/based.h."""
from . import workloads  # noqa: F401
from .binding import (  # noqa: F401
    BASED_BF16, BASED_F32, BASED_OK, BASED_NUMERATOR_ONLY, BASED_STATE_CONTINUE, BASED_STATE_SYM, BASED_STATE_ZERO_INIT, D_EXPANDED, D_FEAT, D_SYM, BasedError,
    baseconv_gate_forward, baseconv_gate_step, based_decode_step, based_decode_step_flags, based_decode_step_sym, based_generation_step, based_state_from_sym, based_state_to_sym, based_poll_error, based_prefill, based_prefill_backward, based_prefill_state, based_prefill_static_scratch, based_prefill_workspace_bytes,
    based_static_scratch_bytes, based_selftest_bounded_wait, launch_count, lib,
    new_state, status_string, swa_decode_step, swa_decode_step_ragged, swa_forward, version,
)
