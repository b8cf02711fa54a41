"""B200-native cloud verification step of Synera (arxiv 2511.07423): thin Python binding
over the C ABI of libsynera.so.  All computation runs in the library's CUDA kernels."""
from .binding import (SynError, Model, KVCache, Plan, StepStats, lib_path, load_library,  # noqa: F401
                      syn_op_linear, plan_host, Scheduler, SchedStats, Sampling, verify_batch_sampled,
                      syn_op_sample_verify, gemm_plan_host, gemm_work_host, debug_set_spin_limit,
                      debug_linear_counter, debug_set_schedule, debug_set_attention, gemm2_plan_host, gemm2_work_host)
