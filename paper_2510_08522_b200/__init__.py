"""B200-native gradient step for batch-size-controlled data-parallel training (DYNAMIX hot path).

`binding` mirrors the C ABI of include/dmx.h; `workload` holds the seeded synthetic inputs;
`build` compiles the CUDA sources in-tree.
"""
from .binding import (BF16, F32, ctl_decide, dmx_ctl_decide, dmx_ctl_num_features, dmx_ctl_num_weights, dmx_plan_chunks, ShardedDmx, dmx_shard_range, dmx_shard_segments, dmx_partials_len,
                      dmx_step_partial, dmx_step_adam_partial, dmx_finalize_partials, dmx_agg_create, dmx_agg_destroy, dmx_agg_push, Dmx, DmxError, dmx_create, dmx_destroy, dmx_get_profile,  # noqa: F401
                      dmx_last_cuda_error, dmx_launches_per_step, dmx_set_profiling, dmx_state_len, dmx_step,
                      dmx_step_adam, dmx_step_host, dmx_step_static, strerror)
