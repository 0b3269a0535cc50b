"""B200-native (sm_100a) hot path of RepQuant's reparameterized quantized inference.

`binding` exposes the C-ABI entry points of librepq.so under the same names; `engine` prepares
parameters (fold + pack through the library's host entry points) and drives a whole block.
"""
from . import binding  # noqa: F401
