"""B200-native fused operator chains: Python binding over the C ABI declared in include/fc.h."""
from .binding import (FcError, PreparedRun, fc_run, fc_run_host, fc_run_softmax_static_scratch, fc_staging_size, fc_workspace_size, fc_set_workspace,  # noqa: F401
                      fc_get_async_status, fc_launch_count, fc_version, fc_last_error, fc_last_plan, make_spec,
                      run_chain, run_chain_host, lib, to_device, LIB_PATH)
