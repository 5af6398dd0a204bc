"""B200-native rollout library for RPO (arXiv 2601.19404): Python binding of the C ABI.

`paper_2601_19404_b200.binding` loads `librpo.so` (built in-tree by `build.py`) and
exposes the same calls as `include/rpo.h`; it only marshals arguments.  There is no
CPU path: importing works anywhere, computing needs a CUDA device.
"""
from .binding import (Context, Sampler, Group, ObjectiveCfg, shape_preset, load_library, RpoError, EXPORTED_SYMBOLS,
                      sample_rows_noalloc)  # noqa: F401
