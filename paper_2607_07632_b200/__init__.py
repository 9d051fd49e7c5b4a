"""sjq: fused star-join query pipeline for B200 (thin binding over libsjq.so)."""
from .sjq import (Result, SjqError, Table, build_dim, lib, run, run_workload, build_workload_tables,  # noqa: F401
                  strerror, version, RunOpts, run_host, run_workload_host, staging_bytes, build_launches,
                  HostResult, alloc_result, run_hashed_static, STATIC_MAX_GROUPS, TableBuilder,
                  workload_builders, build_tables, jit_log, host_transfer_plan, layout_bytes, DimLayout, merge_groups, sample_preds, PredSampler, unfused_scratch, release)
