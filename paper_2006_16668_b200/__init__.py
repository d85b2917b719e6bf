"""B200-native top-2 gated Mixture-of-Experts FFN layer (GShard, Algorithm 1 and 2).

The compute path is a C-ABI CUDA library (``include/gshard_moe.h``); this package
is its thin Python binding plus the seeded input generators.  Importing the
package does not load the library; the first call through ``binding`` does and
fails loudly when it is missing.
"""
from .inputs import CONFIGS, MoEConfig, make_inputs  # noqa: F401
