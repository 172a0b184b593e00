"""fsmguide: FSM vocabulary indexing and masked greedy / sampled decoding on NVIDIA B200.

The work is done by hand-written CUDA kernels behind a C ABI
(``include/fsmguide.h``, built into ``libfsmguide.so``); this package is the thin
Python binding.  There is no CPU fallback: importing the binding without the
built library raises.
"""
from .batching import stack_automata
from .binding import (FSM_INDEX_BITMASK, FSM_INDEX_CSR, FSM_INDEX_DENSE, FSM_LOGITS_BF16, FSM_LOGITS_F32,
                      FSM_STATE_I32, FSM_STATE_U16, FsmError, GuidedIndex, IndexDesc, fsm_checksum64,
                      fsm_debug_set, fsm_device_check, fsm_index_build, fsm_index_build_csr,
                      fsm_index_build_rows, fsm_index_build_static, fsm_index_input_digest,
                      fsm_index_load, fsm_index_peek, fsm_index_row_alias, fsm_index_save, fsm_index_serialized_bytes,
                      fsm_index_workspace_bytes, fsm_profile_read, fsm_row_alias_workspace_bytes, fsm_sha256, fsm_status_string,
                      guided_mask_step, guided_sample_step, guided_step_csr, index_desc, lib,
                      library_path)

__all__ = [
    "FSM_INDEX_BITMASK", "FSM_INDEX_CSR", "FSM_INDEX_DENSE", "IndexDesc", "fsm_checksum64",
    "fsm_index_input_digest", "fsm_index_load", "fsm_index_peek", "fsm_index_save",
    "fsm_index_serialized_bytes", "fsm_sha256", "index_desc", "fsm_index_row_alias",
    "fsm_row_alias_workspace_bytes",
    "FSM_LOGITS_BF16", "FSM_LOGITS_F32", "FSM_STATE_I32", "FSM_STATE_U16", "FsmError",
    "GuidedIndex", "fsm_debug_set", "fsm_device_check", "fsm_index_build",
    "fsm_index_build_csr", "fsm_index_build_rows", "fsm_index_build_static", "fsm_index_workspace_bytes", "fsm_profile_read", "fsm_status_string",
    "guided_mask_step", "guided_sample_step", "guided_step_csr", "lib", "library_path", "stack_automata",
]
