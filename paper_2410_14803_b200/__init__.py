"""B200 (sm_100a) learner hot path of DistRL's A-RIDE algorithm (arXiv 2410.14803).

The product is the C-ABI CUDA library under ``csrc/`` (declared in
``include/distrl.h``).  ``binding`` marshals torch CUDA tensors into it;
``synth`` generates the seeded synthetic trajectory buffers used by tests and
benchmarks.  There is no CPU path.
"""
from .binding import *  # noqa: F401,F403
from .binding import (DistrlError, Replay, Sampler, alloc_workspace, distrl_batch, distrl_prio_cfg, library_path,
                      make_batch, make_prio_cfg)
