"""CPU checker for batched replica placement -- test infrastructure only.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
package. The CUDA library and its Python binding never do.
"""
from .placement import (  # noqa: F401
    KEY_IDLE_FIRST,
    KEY_SR_FIRST,
    REQUIRE_IDLE_GPUS,
    autoscale,
    build,
    cluster_limit,
    cluster_sums,
    compare_sr_after,
    feasible,
    place,
    place_sequential,
    place_workload,
    ranks_before,
    scale_out_deficit,
    select_executors,
    subscription_ratio,
)
