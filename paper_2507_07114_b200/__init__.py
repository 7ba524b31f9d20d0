"""B200-native lossy data-parallel step: CUDA library (csrc/) + its ctypes binding."""
from . import build  # noqa: F401
from .binding import *  # noqa: F401,F403
from .binding import (EXPORTS, LossyError, drift_norms, drift_norms_static, drift_pairwise, load_library, lossy_aggregate, lossy_aggregate_alg1, lossy_broadcast, lossy_closed_loop_grads,
                      lossy_config, lossy_describe_plan, lossy_destroy, lossy_device_status, lossy_fused_step, lossy_fused_step_alg1, lossy_fused_step_host, lossy_fused_step_prepared, lossy_hash_u32,
                      lossy_init, lossy_kernel_launches, lossy_last_error, lossy_mask, lossy_mask_grid, lossy_num_packets,
                      lossy_packet_sqnorms, lossy_replica_elems, lossy_reset_status, lossy_selftest_wait_expiry, lossy_has_device_checks, lossy_selftest_shrink_checks, lossy_set_bursty, lossy_set_lr, lossy_set_reliable, lossy_step)
from .sharding import packet_range_config, shard_range  # noqa: F401
