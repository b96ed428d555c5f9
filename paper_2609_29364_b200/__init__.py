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
)
