"""B200-native coalesced attention engine (the rank-local attention path of Zellige,
paper Section IV-D): a C-ABI CUDA library for sm_100a plus this thin Python binding.

The binding only marshals arguments; every step of the path runs in the library's
kernels.  PyTorch is used for device memory and streams.  There is no CPU fallback: if
``libzellige.so`` has not been built, the first use of any binding name raises.

The names of :mod:`.binding` are resolved on first access, so that
``python -m paper_2608_01150_b200.build`` can run before the library exists.
"""
_BINDING_NAMES = ("ZlError", "TaskHandle", "ShardDesc", "WholeDesc", "HeadRange", "TasksInfo", "build_tasks",
                  "build_tasks_heads", "coalesced_attn_fwd", "lse_merge", "coalesced_attn_bwd",
                  "coalesced_attn_bwd_noalloc", "coalesced_attn_fwd_packed", "coalesced_attn_bwd_packed",
                  "coalesced_attn_fwd_phase", "coalesced_attn_bwd_phase", "MAX_PHASES",
                  "NOALLOC_SCRATCH_BYTES", "BUILD_FUSE_LOCAL_CHUNKS", "launch_count", "library_path", "STATUS_NAMES")


def __getattr__(name):
    if name in _BINDING_NAMES:
        from . import binding
        return getattr(binding, name)
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")


def __dir__():
    return sorted(list(globals()) + list(_BINDING_NAMES))
