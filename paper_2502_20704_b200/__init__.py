"""B200 (sm_100a) verification step of Fuzzy Speculative Decoding: Python binding of the C ABI."""

from .binding import (  # noqa: F401
    FsdOpts,
    FsdError,
    fsd_accept_labels,
    fsd_calibrate_threshold,
    fsd_debug_checks,
    fsd_default_opts,
    fsd_host_staging_bytes,
    fsd_set_stage_event,
    fsd_set_group_size,
    fsd_set_timeout_injection,
    fsd_status_string,
    fsd_threshold_sweep,
    fsd_verify_chain,
    fsd_verify_chain_host,
    fsd_verify_chain_static,
    fsd_verify_tree,
    fsd_version,
    fsd_workspace_bytes,
    library_path,
    make_opts,
)
