"""B200-native paged-KV GQA decode attention (split-KV partial + LSE combine) behind a C ABI.

`binding` mirrors include/concur_attn.h one to one; `DecodeAttention` is a small
convenience holder of a handle for torch tensors.  Importing the package requires the
built shared library (see build.py); nothing here computes on the CPU.
"""
from . import binding
from .binding import *  # noqa: F401,F403
from .runner import DecodeAttention  # noqa: F401
