"""Batched InferLine Estimator for NVIDIA B200: thin Python binding over the
C ABI in ``include/il_estimator.h``.  All computation happens in the CUDA
library; this package only marshals arguments."""
from .estimator import (  # noqa: F401
    Estimator, ILError, StageConfig, il_estimate, il_estimate_device, il_estimate_device_static, il_estimate_latencies, il_feasible, il_feasible_device,
    il_estimator_create,
    il_estimator_create_dag,
    il_estimator_destroy, il_get_stats, il_kernel_name, il_measure_int_issue, il_set_stream, il_set_test_knob, il_set_variant, il_set_workspace,
    il_stage_visits, il_traffic_envelope, il_strerror, il_workspace_bytes, il_workspace_min_bytes, library_path,
    load_library,
)
from .sharded import ShardedEstimator, shard_range  # noqa: F401,E402
