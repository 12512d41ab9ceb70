"""B200-native parameter-server step with backup workers (arXiv 1604.00981, Algorithm 4).

`paper_1604_00981_b200.binding` wraps the C ABI of `libsgdb.so` (include/sgdb.h);
`paper_1604_00981_b200.workload` draws the seeded synthetic inputs;
`paper_1604_00981_b200.build` compiles the CUDA library for sm_100a.

The binding is imported on first use of one of its names, and raises if the
CUDA library has not been built: there is no CPU fallback.
"""
from __future__ import annotations

import importlib

__all__ = ["binding", "workload", "build"]

_BINDING_NAMES = (
    "sgdb_select", "sgdb_aggregate", "sgdb_update", "sgdb_step", "sgdb_step_segmented", "sgdb_select_deadline", "sgdb_step_deadline", "sgdb_step_ema", "sgdb_ema", "sgdb_learning_rate",
    "sgdb_accumulate_arrival", "sgdb_accumulate_arrival_ema", "sgdb_step_host", "sgdb_step_host_workspace_bytes", "sgdb_step_host_static",
    "sgdb_select_grouped", "sgdb_step_grouped", "sgdb_step_segmented_ema", "sgdb_step_segmented_deadline", "sgdb_accumulate_arrival_deadline", "sgdb_accumulate_close", "sgdb_set_tuning", "sgdb_set_arrival_tuning", "sgdb_strerror", "sgdb_version", "Opt", "SgdbError",
    "sgdb_step_rows", "sgdb_step_rows_ordered", "sgdb_shard_range", "sgdb_enable_peer_access", "sgdb_selftest_bounded_wait", "sgdb_set_wait_limit_ns",
    "make_address_table",
)


def __getattr__(name):
    if name in ("binding", "workload", "build"):
        return importlib.import_module("." + name, __name__)
    if name in _BINDING_NAMES:
        return getattr(importlib.import_module(".binding", __name__), name)
    raise AttributeError(name)
