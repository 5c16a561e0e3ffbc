"""qv2: B200-native local-metric sensitivity sweep (calibrate -> fake-quantize -> MSE/SQNR -> rank).

The product is ``libqv2.so`` (CUDA, C ABI, see include/qv2.h); this package builds it, loads it
and marshals arguments.  It has no CPU implementation of any step."""
from .binding import *  # noqa: F401,F403
from .binding import Context, lib  # noqa: F401
from .model import model_descs, ModelDescs  # noqa: F401
