"""Prefix-shared attention (forward + backward) and the DPO log-prob gather for
B200, behind a small C ABI (include/psa.h).  See binding.py for the Python calls."""
from .binding import (Plan, PsaError, dpo_logp, dpo_logp_bwd, dpo_loss, load_library, psa_pack_ffd, psa_position_ids, psa_rope, psa_bwd, psa_bwd_static_scratch, psa_bwd_f32, psa_check_device_status, psa_selftest_wait_expiry, psa_pack_ffd_emit, psa_logp_labels, psa_fwd, psa_step_host, psa_step_host_arena_bytes, simpo_loss, orpo_loss,
                      psa_plan)  # noqa: F401
from .labels import logp_labels  # noqa: F401
