"""Exact softmax attention forward/backward for B200 (sm_100a) behind a C ABI.

``inputs`` (seeded synthetic inputs) imports without the compiled library; the
binding (``attn_fwd``, ``attn_bwd`` and friends) loads ``libattn_b200.so`` on first
use and raises if it is missing -- there is no CPU fallback.
"""
from . import inputs  # noqa: F401

_BINDING_NAMES = None


def __getattr__(name):
    # The binding is imported lazily so that input generation works on machines
    # where the CUDA library has not been built.
    from . import binding
    if hasattr(binding, name):
        return getattr(binding, name)
    raise AttributeError(name)
