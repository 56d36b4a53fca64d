"""B200-native tree-verification kernels for EAGLE-2-style speculative decoding of
LLaVA-class VLMs (the target-side verify step of SpecVLM): tree-masked split-KV
attention, vocabulary argmax, lossless temperature-0 acceptance and KV compaction.

The product is the C-ABI library `lib/libspecvlm.so` (see include/specvlm.h); this
package is its thin ctypes binding. Build with `python -m paper_2509_11815_b200.build`.
"""

from .binding import *  # noqa: F401,F403
from .binding import (  # noqa: F401
    AttnDesc,
    KvDesc,
    SpecvlmError,
    EXPORTS,
    LIB_PATH,
    alloc_attn_workspace,
    load_library,
    make_attn_desc,
    make_kv_desc,
)
