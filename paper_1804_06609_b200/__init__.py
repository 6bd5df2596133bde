"""B200-native Dynamic Beam Allocation step (Post & Vilar 2018) -- thin Python binding over libdba.so."""
from .binding import (DbaError, DbaStepper, F32, BF16, FLAG_ADJUST_OFF, FLAG_HOST_STAGING, FLAG_LENGTH_NORM,  # noqa: F401
                      FLAG_FUSED_PROJECTION, FLAG_PRUNE_NORMALISED, lib, project_scan, row_scan, row_scan_static)
