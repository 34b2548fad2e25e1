"""B200-native Gated DeltaNet tail-replay: thin Python binding over the C-ABI CUDA library.

The binding only marshals arguments (pointers, sizes, the CUDA stream); every step of the
path runs in the library's kernels.  PyTorch is used for device memory and streams only.
There is no CPU fallback: if the CUDA library is missing, loading fails loudly.
"""
from ._binding import (  # noqa: F401
    GdnDesc, GDN_OK, GDN_F32, GDN_BF16, GDN_MEM_DEVICE, GDN_MEM_HOST,
    GDN_KERNEL_AUTO, GDN_KERNEL_FP32_SIMT, GDN_KERNEL_TCGEN05,
    GdnError, library_path, load_library, status_string, tail_select, workspace_size,
    gdn_tail_replay, gdn_full_prefill, gdn_tail_replay_static_scratch, gdn_decode_step, last_launch_count, Workspace,
    test_hooks,
)

__all__ = [
    "GdnDesc", "GdnError", "library_path", "load_library", "status_string", "tail_select",
    "workspace_size", "gdn_tail_replay", "gdn_full_prefill", "gdn_tail_replay_static_scratch", "gdn_decode_step",
    "last_launch_count", "Workspace",
]
