"""Elastic (masked) backward pass of a stack of dense layers on B200: Python binding of libet.so.

The binding only marshals arguments (torch tensors -> device pointers, numpy -> host
pointers); every computation runs in the library's CUDA kernels.  There is no CPU or
PyTorch fallback: importing this package without the built library raises.
"""
from .binding import *  # noqa: F401,F403
from .binding import __all__  # noqa: F401
