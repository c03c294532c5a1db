"""Early-exit head decision and DSSD verify step on B200: Python binding over the C-ABI library."""
from .api import (  # noqa: F401
    EE_PATH_AUTO,
    EE_PATH_STREAM,
    EE_PATH_TCGEN05,
    EExitError,
    dssd_accept,
    ee_compact,
    ee_exit_head,
    ee_exit_head_host,
    ee_exit_head_launches,
    ee_exit_head_static,
    EE_STATIC_MAX_ROWS,
    ee_exit_head_workspace_bytes,
    ee_query_async_error,
    ee_workspace_init,
    new_outputs,
    new_workspace,
)
