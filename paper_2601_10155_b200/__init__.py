"""B200 (sm_100a) implementation of LOOKAT decode attention over product-quantised keys.

    from paper_2601_10155_b200 import Lookat      # binding of the C-ABI library (needs a GPU)
    from paper_2601_10155_b200 import synth        # seeded synthetic inputs (numpy only)

Importing the package loads nothing native; the library is loaded when a
context is created and its absence is an error, never a fallback.
"""


def __getattr__(name):
    if name in ("Lookat", "LookatError", "load_library"):
        from . import binding
        return getattr(binding, name)
    raise AttributeError(name)
