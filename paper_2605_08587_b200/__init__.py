"""B200-native (sm_100a) Kaczmarz Linear Attention hot path: chunkwise forward and decode step.

`binding` wraps the C ABI of include/kla.h; `workloads` draws the seeded synthetic inputs;
`build` compiles the CUDA library in-tree.
"""
from .binding import (KlaError, check, kla_chunk_fwd, kla_chunk_fwd_static_scratch, kla_chunk_span_map, kla_state_chain, kla_decode_step,  # noqa: F401
                      kla_dg_fwd, kla_dg_decode_step, kla_bwd,
                      kla_decode_steps, launch_count,
                      KLA_F32, KLA_BF16, KLA_FLAG_NONE, KLA_FLAG_FORCE_SIMT, KLA_FLAG_NO_SEGMENTS, KLA_FLAG_SEGMENTS, KLA_FLAG_COEFF_ETA, KLA_FLAG_QNORM, KLA_FLAG_NO_PAIR, KLA_FLAG_WY_FORM, KLA_FLAG_EXACT_SEGMENTS)
