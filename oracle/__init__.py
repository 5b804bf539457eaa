"""Independent CPU oracle for asynchronous-thread decode attention.  TEST INFRASTRUCTURE.

Plain Python for the integer bookkeeping, NumPy float64 for the attention.  Imported only by the
test-suite, the smoke check and the benchmark's CPU-baseline / reference legs; never by the product
path, which must fail loudly when its CUDA library is missing.
"""
from .pool_model import (PoolModel, PoolError, OK, INVALID_ARG, OUT_OF_PAGES, BAD_STATE, CAPACITY,  # noqa: F401
                         ACTIVE, FINISHED, MERGED)
from .attention import KVStore, attend, decode_attention  # noqa: F401
from .replay import OracleReplay  # noqa: F401
from .rope import rope, rope_bf16  # noqa: F401
from .interpreter_model import paper_timeline  # noqa: F401
