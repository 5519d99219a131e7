"""B200-native fast-slow flow serving: Python binding of the C-ABI CUDA library.

`binding` mirrors include/serveflow.h call for call; `harness` holds the small
amount of host glue (moving numpy planes into torch device tensors, building the
library's handles from generated models) that tests and the benchmark share.
"""
from . import binding
from .binding import *  # noqa: F401,F403
