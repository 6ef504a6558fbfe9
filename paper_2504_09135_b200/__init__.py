"""B200 (sm_100a) implementation of the DISC + PPV constrained-decoding hot path.

The work is done by the CUDA library built from csrc/ (C ABI: include/disc.h); this package is
its Python binding plus a small decode-loop helper.  Nothing here falls back to the CPU.
"""
from .binding import (DISC_BF16, DISC_F32, ROW_DEAD, ROW_DONE, ROW_NOMASS, ROW_NONFINITE, DiscError,
                      DiscSet, DiscState, StepOutputs, disc_accept, disc_accept_resample, disc_build_set, disc_build_set_eok, disc_mask,
                      disc_mask_static, disc_project_check, disc_project_scratch, disc_project_step, disc_resample, disc_sampling_uniforms, disc_set_rows, disc_state_init, disc_step, disc_step_topm, disc_topm, disc_verify,
                      lib)
from .decoder import DiscDecoder

__all__ = ["DISC_BF16", "DISC_F32", "ROW_DEAD", "ROW_DONE", "ROW_NOMASS", "ROW_NONFINITE", "DiscError",
           "DiscSet", "DiscState", "StepOutputs", "disc_accept", "disc_accept_resample", "disc_build_set", "disc_build_set_eok", "disc_mask",
           "disc_mask_static", "disc_project_check", "disc_project_scratch", "disc_project_step", "disc_resample", "disc_sampling_uniforms", "disc_set_rows", "disc_state_init", "disc_step", "disc_step_topm", "disc_topm", "disc_verify",
           "lib", "DiscDecoder"]
