"""fp64 CPU oracle for the partially linear FFN forward.  Test infrastructure only:
the product (the CUDA library and its Python binding) never imports this package."""
from .tardis_oracle import *  # noqa: F401,F403
from . import tardis_oracle  # noqa: F401
