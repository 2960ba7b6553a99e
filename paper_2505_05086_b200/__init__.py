"""B200-native ASI (Activation Subspace Iteration) hot path: a C-ABI CUDA library plus this thin binding."""
from .binding import (AsiError, LayerDesc, Plan, PlanInfo, lib, status_string)  # noqa: F401
