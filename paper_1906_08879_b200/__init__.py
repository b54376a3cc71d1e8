"""B200 (sm_100a) implementation of the Placeto policy forward.

The CUDA library ``libplaceto.so`` (sources under ``csrc/``, C ABI in
``include/placeto.h``) does all the work; ``binding`` marshals arguments.
"""
from .binding import *  # noqa: F401,F403
from .binding import (CALL_EMBED, CALL_EMBED_ROUNDS, CALL_EPISODE, CALL_GRADIENT, CALL_FORWARD, CALL_FORWARD_HOST, CALL_LOGITS, EXPORTS, Graph,
                      PlacetoError, Weights, workspace)  # noqa: F401
