"""B200-native (sm_100a) MONA optimizer step: thin Python binding over the C-ABI library libmona.so.

All arithmetic runs in the CUDA library; this package only marshals pointers.  PyTorch is used for
device memory and streams.  There is no CPU fallback: loading fails loudly when the library has not
been built (run `python -m paper_2605_26842_b200.build`)."""
from .binding import (MONA_STATE_COMBINED, Hparams, Options, default_options, MatrixDesc, MonaError, MonaOptimizer, default_hparams, lib, prologue_noalloc, query_sizes,  # noqa: F401
                      set_chunk_budget, set_chunk_overlap, STATUS_NAMES)
