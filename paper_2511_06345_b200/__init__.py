"""Fused GEMM + epilogue + row-reduce for NVIDIA B200 (sm_100a).

The product is the CUDA library ``libfgr.so`` behind the C ABI of ``include/fgr.h``; this package
is its ctypes binding plus a small torch-based convenience wrapper (device memory and streams only).
"""
from .binding import *  # noqa: F401,F403
from .binding import EXPORTS, FgrError, fgr_desc, fgr_plan_info, fgr_reduce_desc, fgr_shard_desc, lib, make_desc  # noqa: F401
from .op import FusedGemmReduce  # noqa: F401
from .sharded import NShardedFusedGemmReduce, gather_pairs, local_reduce_kind, shard_range  # noqa: F401
