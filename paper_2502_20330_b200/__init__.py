"""RAPID verify step on B200: thin Python binding over the C-ABI library.

Every step of the path runs in the CUDA kernels of ``librapid.so``; this package
only marshals arguments (torch tensors -> device pointers).  There is no CPU
fallback: calls raise if the library cannot be loaded or a call fails.
"""
from .binding import (  # noqa: F401
    RapidError,
    AcceptParams,
    AttnParams,
    accept_workspace_bytes,
    attention_workspace_bytes,
    kernel_launch_count,
    kernel_launch_count_reset,
    last_error,
    lib_path,
    load_library,
    new_workspace,
    rapid_accept,
    rapid_accept_static,
    rapid_draft_sample,
    rapid_kv_append,
    rapid_retrieval_select,
    retrieval_budget_chunks,
    rapid_merge_partials,
    rapid_kv_append_paged,
    rapid_step_commit,
    rapid_verify_attention,
    rapid_verify_attention_paged,
    rapid_verify_step,
    rapid_verify_step_host,
    verify_step_host_arena_bytes,
    version,
    workspace_init,
    workspace_status,
    STATUS_BAD_CTX_LEN,
    STATUS_BAD_DRAFT_TOKEN,
    STATUS_RESIDUAL_FALLBACK,
    STATUS_PIPELINE_TIMEOUT,
    STATUS_BAD_BLOCK_TABLE,
    RESIDUAL_PAPER,
    RESIDUAL_PHAT,
)
