"""B200-native GRAFT draft-tree builder: hand-written sm_100a kernels behind a C ABI (include/graft.h),
with a thin ctypes binding.  PyTorch is used by callers only for device memory and streams."""
from .binding import (  # noqa: F401
    Graft, GraftError, TreeOut, BF16, F32, ST_BAD_LOGITS, ST_TAU_CLAMPED, ST_FRONTIER_EMPTY, ST_INTERNAL,
    load_library, library_path, vocab_pass_static, VOCAB_PARTIAL_BYTES,
)
from .shard import shard_range  # noqa: F401
from .vocab_parallel import vocab_range, gather_partials, vocab_pass_parallel  # noqa: F401
from .pipeline import MicroBatch, run_rounds, join  # noqa: F401
