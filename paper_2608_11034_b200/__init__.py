"""B200-native sign+vote hot path of Consensus Collective Communication (C3).

``binding`` exposes the C-ABI library (``scout_*`` calls, hand-written sm_100a
CUDA); ``inputs`` generates the seeded synthetic replica sets.  Importing the
package does not load the CUDA library; the first ``scout_*`` call does, and it
raises if the library has not been built.
"""
from . import inputs  # noqa: F401

__all__ = ["inputs", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
