"""B200-native paged-KV GQA decode attention (split-KV partial + LSE combine) behind a C ABI.

`binding` mirrors include/concur_attn.h one to one; `DecodeAttention` is a small
convenience holder of a handle for torch tensors.  Using anything but `build` requires the
built shared library (see build.py); nothing here computes on the CPU.

The binding is loaded on first use, so that `paper_2510_07356_b200.build` can be imported
(and run with `python -m`) in a fresh checkout that has no shared library yet.  Any other
attribute access without the library raises ImportError: there is no fallback.
"""
import importlib

_LAZY_MODULES = ("binding", "runner", "build", "bench_probe")


def _load_all():
    binding = importlib.import_module(".binding", __name__)
    runner = importlib.import_module(".runner", __name__)
    g = globals()
    for k in dir(binding):
        if not k.startswith("_"):
            g.setdefault(k, getattr(binding, k))
    g["DecodeAttention"] = runner.DecodeAttention
    g["_loaded"] = True


def __getattr__(name):
    if name in _LAZY_MODULES:
        return importlib.import_module("." + name, __name__)
    if name.startswith("__") or globals().get("_loaded"):
        raise AttributeError(name)
    _load_all()
    try:
        return globals()[name]
    except KeyError:
        raise AttributeError(name) from None
