"""B200-native (sm_100a) hot path of HiLoRe's GRPO actor update, behind the C ABI of include/hilore.h.

``paper_2609_33570_b200.api`` is the thin binding of that ABI; ``paper_2609_33570_b200.synth``
draws the seeded synthetic workloads; ``paper_2609_33570_b200.build`` compiles the library.
"""
from . import api, build, synth  # noqa: F401
from .api import *  # noqa: F401,F403
