"""CPU oracle for MoFQ format selection.  Test infrastructure only.

Only tests, the smoke check and the bench's CPU-baseline leg may import this package; the CUDA
library never does.  ``oracle.build()`` compiles ``mofq_oracle.c`` with gcc; ``oracle.api`` is
the numpy-facing wrapper.
"""
from .build import build  # noqa: F401
