"""B200-native lightning indexer, causal top-k and IndexCache layer schedule.

``paper_2603_12201_b200.binding`` wraps the C-ABI library (``libidxc.so``, built
from ``csrc/`` by ``build.py``); ``synth`` draws seeded synthetic inputs. The
binding is imported on first use so that ``synth`` stays usable on machines
without the compiled library; using any indexer call without the library raises.
"""

__all__ = ["binding", "synth", "build"]


def __getattr__(name):
    if name in __all__:
        import importlib
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
