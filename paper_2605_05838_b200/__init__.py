"""B200-native chunkwise forward of the MDN stepwise-momentum delta-rule recurrence.

The work is done by hand-written sm_100a CUDA kernels behind the C ABI of
include/mdn.h (libmdn.so, built in-tree by `python -m paper_2605_05838_b200.build`);
the functions here only marshal torch tensors into that ABI.
"""
from .binding import (MdnError, MdnParams, MdnWsLayout, MdnLayerOps, make_layer_ops, chunk_bwd, chunk_fwd, chunk_fwd_host, coeff_scan, unpack_chunk_states, unpack_chunk_vt, bwd_state_chain, chunk_attention,  # noqa: F401
                      host_arena_bytes, intra_chunk, last_launch_count, lib, make_params, read_status,
                      status_string, workspace_bytes, workspace_layout, set_stage_events, resolved_path, chunk_fwd_static_scratch, decode_step,
                      STATIC_SCRATCH_BYTES,
                      LIB_PATH, NUM_COEF, CHUNK, NUM_STAGE_EVENTS, STAGE_NAMES, PATH_NAMES)
