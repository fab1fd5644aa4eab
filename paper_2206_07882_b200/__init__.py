"""INT4 RNN-T inference with density-ratio LM fusion: CUDA library binding.

`synth` draws the seeded synthetic workloads; `binding` (loaded on first use)
wraps the C-ABI shared library built from `csrc/`.  There is no CPU fallback:
every call into `binding` raises if the CUDA library is missing.
"""
from . import synth  # noqa: F401
