"""TopoEP planning step for one B200: hand-written CUDA behind a C boundary.

`binding` mirrors include/topoep.h one to one; `Planner` holds a handle with its
torch-allocated workspace.  The CUDA library is the only implementation.
"""
from . import binding  # noqa: F401
from .binding import CostParams, Summary, TopoEPError  # noqa: F401


def __getattr__(name):
    if name == "Planner" or name == "PlanOutputs":
        from . import planner
        return getattr(planner, name)
    raise AttributeError(name)
