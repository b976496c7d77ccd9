"""B200-native batched rollout decoding for multi-turn self-play (the response-generation step of
Algorithm 1).  The work is done by libspiral.so (hand-written CUDA for sm_100a, C ABI in
include/spiral.h); this package only marshals arguments.  There is no CPU fallback: importing
`binding` raises if the library has not been built."""
from . import binding  # noqa: F401
from .binding import *  # noqa: F401,F403
