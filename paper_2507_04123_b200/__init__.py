"""B200-native data bridge and dispatch of EMC2 (arXiv 2507.04123): CUDA library + thin binding."""
from .bridge import (ABI_SYMBOLS, LIB_PATH, Bridge, Emc2Config, Emc2Error, Emc2Grid, config_from_workload,
                     load_library, make_config, route_dispatch_static)

__all__ = ["ABI_SYMBOLS", "LIB_PATH", "Bridge", "Emc2Config", "Emc2Error", "Emc2Grid",
           "config_from_workload", "load_library", "make_config", "route_dispatch_static"]
