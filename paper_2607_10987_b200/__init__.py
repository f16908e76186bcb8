"""B200-native paged-KV operator data path (after AAFLOW+, arxiv 2607.10987).

The product is the C-ABI library ``libaafkv.so`` (sources under ``csrc/``, declarations in
``include/aaf_kv.h``).  ``binding`` exposes the same entry points to Python through ctypes and
does argument marshalling only; PyTorch supplies device memory and streams.
"""
from . import binding  # noqa: F401
from .binding import KVPool  # noqa: F401
