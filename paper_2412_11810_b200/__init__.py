"""B200 (sm_100a) BPTT training step for sparse recurrent / spiking networks under the
gradient-checkpointing strategies of arXiv 2412.11810.  The CUDA library sits behind the C ABI
of include/snn.h; `binding` mirrors it, `session` owns the torch buffers and streams."""
from . import binding  # noqa: F401  (fails loudly if the CUDA library is missing)
from .session import Session  # noqa: F401
