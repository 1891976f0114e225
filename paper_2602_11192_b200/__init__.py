"""B200-native cached Mixture-of-Experts layer: thin Python binding over the C ABI.

All computation happens in the CUDA library (csrc/, built into libmelinoe_moe.so); this
package only marshals arguments.  Importing it never falls back to a CPU path: a missing
library raises.
"""
from .binding import *  # noqa: F401,F403
