"""Python binding of libhx.so: batched placement scoring and workflow horizons
for workflow-aware scheduling on heterogeneous prefill/decode clusters.

The binding only marshals arguments; every step runs in the CUDA library.  It
raises at import if the library has not been built (python -m
paper_2605_16637_b200.build); there is no CPU fallback.
"""
from .api import (CALL_DTYPE, INSTANCE_DTYPE, HX_FLAG_NO_DAG, HX_FLAG_NO_TAIL, HX_FLAG_UNLOADED, HX_FLAG_ONE_PASS,
                  HX_MODE_COMPLETION, HX_MODE_RATIO, HX_MODE_SLACK, HxError, Cluster,
                  hx_cluster_create, hx_cluster_destroy, hx_cluster_read_loads, hx_set_kv_free_restore,
                  hx_cluster_update_loads, hx_critical_path, hx_enable_kernel_timing,
                  hx_read_kernel_timing, hx_dag_upload, hx_dag_update_costs, hx_dag_update_elapsed, hx_get_dag_results,
                  hx_dag_append, hx_earliest_start, hx_get_earliest_results,
                  hx_get_status, hx_get_topk, hx_last_error, hx_launch_count, hx_schedule_batch,
                  hx_schedule_batch_host, hx_schedule_batch_host_async, hx_schedule_sweep_host, hx_set_attention_flops, hx_schedule_batch_static, hx_schedule_greedy, hx_schedule_greedy_plan, hx_replay, hx_replay_lifecycle, hx_measure_fp32_rates, hx_dag_append_workflows, hx_estimate_calls,
                  hx_decode_set_running, hx_schedule_decode, KV_INTERVAL_DTYPE, hx_set_options, lib_path)

__all__ = [n for n in dir() if n.startswith(("hx_", "HX_", "Hx")) or n in
           ("CALL_DTYPE", "INSTANCE_DTYPE", "KV_INTERVAL_DTYPE", "Cluster", "lib_path")]
