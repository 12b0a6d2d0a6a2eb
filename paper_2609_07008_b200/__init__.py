"""B200-native MLA-Online step (RedKnot-MLA, Algorithm 2): C-ABI CUDA library + thin binding.

`synth` draws seeded inputs; `binding` (imported lazily) loads the sm_100a shared library and
raises if it is missing -- there is no CPU or eager fallback for any step of the path.
"""
__all__ = ["synth"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
