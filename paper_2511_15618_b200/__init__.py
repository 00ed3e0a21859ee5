"""B200-native speculative decode step of an hourglass mesh transformer (FlashMesh).

The product is `libflashmesh.so` (CUDA, sm_100a, C ABI declared in include/flashmesh.h);
this package is the thin ctypes binding over it.  PyTorch is used only for device memory
and streams.  There is no CPU fallback: importing the binding without the built library,
or running it without a CUDA device, raises.
"""
from .binding import (FlashMesh, FmConfig, FmError, fm_workspace_bytes, fm_create, fm_destroy, fm_prefill,
                      fm_set_max_faces, fm_draft, fm_draft_labels, fm_correct, fm_correct_ex, fm_verify, fm_verify_static_scratch, fm_accept, fm_step_host, fm_generate, fm_verify_bytes,
                      fm_launch_count, fm_profile_begin, fm_profile_end, fm_profile_class, fm_strerror, fm_device_status, fm_selftest_wait_timeout, fm_attention_layout, load_library, library_path)

__all__ = ["FlashMesh", "FmConfig", "FmError", "fm_workspace_bytes", "fm_create", "fm_destroy", "fm_prefill",
           "fm_set_max_faces", "fm_draft", "fm_draft_labels", "fm_correct", "fm_correct_ex", "fm_verify", "fm_verify_static_scratch", "fm_accept", "fm_step_host", "fm_generate", "fm_verify_bytes",
           "fm_launch_count", "fm_profile_begin", "fm_profile_end", "fm_profile_class", "fm_strerror", "fm_device_status", "fm_selftest_wait_timeout", "fm_attention_layout", "load_library", "library_path"]
