"""B200-native batched suffix-automaton draft retrieval (the retrieval path of SAM-Decoding).

`binding` exposes the C ABI of libsamdraft.so one to one; `StaticSam` and `Batch` are thin owners
of the handles and of the torch tensors that back them.
"""
from .binding import (Batch, BatchOpts, SamError, StaticSam, StepOutputs, lib)  # noqa: F401
from . import binding  # noqa: F401
