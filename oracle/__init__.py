"""fp64 CPU oracle for the BiGLA forward pass, its gradient and the locality injection.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the CPU-baseline / reference legs of the
benchmark may import this package.  It shares no code with the CUDA path.
"""
from .oracle import (  # noqa: F401
    bigla_fwd,
    bigla_fwd_directions,
    build_oracle,
    gate_prep,
)
from .backward import bigla_bwd, gate_prep_bwd  # noqa: F401
from .locality import dwconv3x3, gate_blend  # noqa: F401
from .quadratic import bigla_quadratic  # noqa: F401
