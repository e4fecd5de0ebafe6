"""B200-native coalesced attention engine (the rank-local attention path of Zellige,
paper Section IV-D): a C-ABI CUDA library for sm_100a plus this thin Python binding.

The binding only marshals arguments; every step of the path runs in the library's
kernels.  PyTorch is used for device memory and streams.  There is no CPU fallback: if
``libzellige.so`` has not been built, importing :mod:`.binding` raises.
"""
from .binding import (ZlError, TaskHandle, ShardDesc, TasksInfo, build_tasks,  # noqa: F401
                      coalesced_attn_fwd, lse_merge, coalesced_attn_bwd, coalesced_attn_bwd_noalloc,
                      coalesced_attn_fwd_packed, coalesced_attn_bwd_packed,
                      NOALLOC_SCRATCH_BYTES, BUILD_FUSE_LOCAL_CHUNKS, launch_count,
                      library_path, STATUS_NAMES)
