"""B200-native batched rollout decoding for multi-turn self-play (the response-generation step of
Algorithm 1).  The work is done by libspiral.so (hand-written CUDA for sm_100a, C ABI in
include/spiral.h); this package only marshals arguments.  There is no CPU fallback: the first use
of any entry point loads `binding`, which raises if the library has not been built
(`python -m paper_2506_24119_b200.build` builds it; that submodule imports without the library)."""
import importlib

_SUBMODULES = ("build", "binding")


def __getattr__(name):
    if name in _SUBMODULES or name.startswith("__"):
        raise AttributeError(name)
    binding = importlib.import_module(".binding", __name__)
    try:
        return getattr(binding, name)
    except AttributeError:
        raise AttributeError(f"module {__name__!r} has no attribute {name!r}") from None


def __dir__():
    binding = importlib.import_module(".binding", __name__)
    return sorted(set(list(globals()) + list(binding.__all__)))
