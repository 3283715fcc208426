"""B200-native (sm_100a) hot path of SASQ: the static-scale activation quantizer
(fake-quant forward, straight-through backward with a reduced scale gradient) and
the static W8A8 linear, behind a C-ABI library.  This package is only the thin
Python binding: argument marshalling, no arithmetic, no fallback."""
from .binding import *  # noqa: F401,F403
from .binding import __all__  # noqa: F401
