"""B200 (sm_100a) library for batched greedy RNN-T decoding with windowed non-blank detection.

The product is ``libwind_b200.so`` (C ABI declared in ``include/wind.h``); this
package is its thin Python binding.  Importing the package does not load the
library; the first call does, and raises if it has not been built.
"""
from .binding import *  # noqa: F401,F403
from .binding import (WindModel, WindError, alloc_workspace, decode, decode_refill, decode_dataset, wind_plan_batches, wind_beam_search, load_library, to_device_enc,  # noqa: F401
                      wind_decode_greedy, wind_decode_window_greedy, wind_decode_greedy_host, wind_eval_joint_window, wind_window_first_output, wind_eval_joint_window_static, wind_profile_decode, wind_read_stats,
                      wind_set_kernels, wind_set_loop_options, wind_debug_plan, wind_bench_joint, wind_debug_stall_barrier, wind_set_trace, wind_read_trace, wind_status_string, wind_workspace_bytes, wind_host_staging_bytes)
