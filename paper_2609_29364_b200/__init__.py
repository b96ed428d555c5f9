"""B200 verification round for M-for-N speculative decoding (thin binding).

`libnsd.so` (built in-tree from `csrc/` by `build.py`) does all the work; this
package only marshals arguments.  There is no CPU fallback: importing the
binding without the built library raises.
"""
from .api import (  # noqa: F401
    NsdConfig,
    NsdError,
    RoundArgs,
    VerifyContext,
    lib_path,
    load_library,
    nsd_schedule_batch,
    nsd_verify_attn_static,
    STATUS,
    NSD_FLAG_ATTN_CP_ASYNC,
    NSD_FLAG_ATTN_TCGEN05,
    NSD_FLAG_ATTN_NO_TCGEN05,
    NSD_FLAG_LOGITS_DIRECT,
    NSD_FLAG_ROUND_SPLIT_ALWAYS,
    NSD_FLAG_ROUND_SPLIT_NEVER,
    NSD_FLAG_NO_DEPENDENT_LAUNCH,
    NSD_FLAG_TEST_STARVE_GATHER,
)
