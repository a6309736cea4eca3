"""B200-native routed structured-sparse causal prefill attention (RouteSparse hot path).

The product is the C-ABI library built from csrc/ (see include/routesparse.h); this package is the thin
Python binding over it.  PyTorch is used for device memory and streams only.
"""
from .binding import *  # noqa: F401,F403
from .pipeline import (GraphedPrefill, RoutedPrefillLayer, RouteConfig, StreamedPrefill, default_library, dense_flops, probe_flops,
                       prefill_from_host)  # noqa: F401,E402
