"""forgestep: a B200-native (sm_100a) training step for Llama-style dense decoders behind a C ABI.

`binding` loads the CUDA library lazily; importing this package needs neither a GPU nor the built library,
using it does.
"""
from . import flops  # noqa: F401
