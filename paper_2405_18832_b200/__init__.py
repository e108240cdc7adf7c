"""B200-native MoE FFN layer forward with a load-aware hot/cold expert split.

The compute lives in a C-ABI CUDA library (``libmonde.so``, sources under
``csrc/``); ``binding`` marshals arguments to it and ``synthetic`` draws seeded
inputs.  Nothing is loaded at import time: the first call into ``binding``
loads the library and raises if it has not been built.
"""
__all__ = ["binding", "synthetic", "build"]
