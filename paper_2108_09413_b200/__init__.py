"""isc: integer randomized smoothing PREDICT / CERTIFY on one B200.

Thin ctypes binding of ``libisc.so`` (see ``include/isc.h``).  Every step of the path runs in
the library's CUDA kernels; this module only marshals arguments.  Importing it needs the
compiled library (``python -m paper_2108_09413_b200.build``); there is no CPU fallback.
"""
from .binding import (IscError, Model, certify_decide, certify_integer_decide, certified_metrics, noise_table, predict_decide, radius_integer, plan_resident, residual_form, lib,  # noqa: F401
                      EXPORTS)
