"""GPU-resident LLM serving loop for B200 (sm_100a): Python binding of libblink.so."""
from .binding import *  # noqa: F401,F403
from .binding import Blink, lib, parse_trace, tokens_by_ticket  # noqa: F401
