"""SpecKV speculation-step hot path for B200 (sm_100a): draft signals, gamma controller and
draft verification from one pass over vocabulary-sized logits, behind a C ABI (libspeckv)."""
from .binding import (ROW_INFO_BYTES, Batch, Mlp, StepOutputs, SpeckvError, load_library, shard_workspace,
                      speckv_sample_draft, speckv_select_gamma, speckv_shard_draw_pick, speckv_shard_draw_sums,
                      speckv_shard_finish, speckv_shard_sweep, speckv_signals, speckv_signals_static, speckv_step,
                      speckv_verify, status_string, version, workspace_size)

__all__ = ["ROW_INFO_BYTES", "Batch", "Mlp", "StepOutputs", "SpeckvError", "load_library", "shard_workspace",
           "speckv_sample_draft", "speckv_select_gamma", "speckv_shard_draw_pick", "speckv_shard_draw_sums",
           "speckv_shard_finish", "speckv_shard_sweep", "speckv_signals", "speckv_signals_static", "speckv_step",
           "speckv_verify", "status_string", "version", "workspace_size"]
