"""B200-native unified-memory-pool hot path: producer scatter into GVA-addressed pages, the dynamic
packing plan, and packed-microbatch assembly.  Everything runs in hand-written CUDA kernels behind the
C ABI of include/flowpool.h; this package only builds and binds it."""
from .build import build  # noqa: F401


def __getattr__(name):
    # the binding (and with it the shared library) loads on first use, so importing the package
    # for a build check needs no CUDA device
    if name in ("binding", "Pool", "Plan", "PoolConfig", "PlanConfig", "FlowpoolError", "lib"):
        import importlib
        mod = importlib.import_module(".binding", __name__)
        return mod if name == "binding" else getattr(mod, name)
    raise AttributeError(name)
