"""B200-native verification step of Calibrated Speculative Decoding.

`libcsd.so` (CUDA, sm_100a, C ABI declared in include/csd.h) does all the work;
this package is its thin Python binding and the build script.
The library is loaded on first use and there is no other code path: without
the built library every call raises.
"""

from .binding import (CSD_BF16, CSD_F32, CSD_MAX_K, CsdError, HostStep, Ocm, StepBuffers, csd_host_staging_bytes,
                      csd_launch_shape, csd_scg_threshold, csd_set_overlap, csd_set_tuning, csd_step, csd_verify, csd_verify_static,
                      csd_workspace_bytes, lib, SampledBuffers, csd_step_sampled, csd_verify_sampled, sampled_launches_per_step, LmheadBuffers, csd_lmhead_shape, csd_step_lmhead, csd_verify_lmhead, EarlyExitBuffers, csd_step_early_exit, csd_lmhead_set_tuning, csd_lmhead_set_pairing, csd_sampled_set_rounds)

__all__ = ["CSD_BF16", "CSD_F32", "CSD_MAX_K", "CsdError", "HostStep", "Ocm", "StepBuffers", "csd_host_staging_bytes",
           "csd_launch_shape", "csd_scg_threshold", "csd_set_overlap", "csd_set_tuning", "csd_step", "csd_verify", "csd_verify_static", "csd_workspace_bytes",
           "lib", "SampledBuffers", "csd_step_sampled", "csd_verify_sampled", "sampled_launches_per_step", "LmheadBuffers", "csd_lmhead_shape", "csd_step_lmhead", "csd_verify_lmhead", "EarlyExitBuffers", "csd_step_early_exit", "csd_lmhead_set_tuning", "csd_lmhead_set_pairing", "csd_sampled_set_rounds"]
