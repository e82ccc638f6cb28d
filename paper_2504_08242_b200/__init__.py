"""B200 (sm_100a) KV-cache attention library: chunked-prefill attention, shared-prefix
branch attention and KV append, behind the C ABI declared in ``include/jupiter.h``.

Importing the package loads ``libjupiter.so`` (building it with nvcc if its sources are
newer); there is no other implementation behind these names.
"""
from .binding import (branch_attn_noalloc, plan_sequence_partition, Context, JupiterError, cache_desc, jupiter_kv_cache, lib, library_path, EXPORTS,
                      STATUS_NAMES, OK, ERR_INVALID_ARG, ERR_OUT_OF_RANGE, ERR_UNSUPPORTED, ERR_ALIGNMENT,
                      ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, BRANCH_AUTO, BRANCH_STREAM, BRANCH_SPLIT_KV,
                      BRANCH_TENSOR_CORE)

__all__ = ["branch_attn_noalloc", "plan_sequence_partition", "Context", "JupiterError", "cache_desc", "jupiter_kv_cache", "lib", "library_path", "EXPORTS",
           "STATUS_NAMES", "OK", "ERR_INVALID_ARG", "ERR_OUT_OF_RANGE", "ERR_UNSUPPORTED", "ERR_ALIGNMENT",
           "ERR_WORKSPACE", "ERR_CUDA", "ERR_TIMEOUT", "BRANCH_AUTO", "BRANCH_STREAM", "BRANCH_SPLIT_KV",
           "BRANCH_TENSOR_CORE"]
