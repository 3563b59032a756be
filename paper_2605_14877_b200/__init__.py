"""B200-native HeatKV hot path: Python binding over the C ABI in include/heatkv.h.

Importing the package loads libheatkv.so (built in-tree by `build.build_library()` or
`__graft_entry__.build()`); there is no fallback of any kind when it is missing.
"""
from .heatkv import *  # noqa: F401,F403
from .heatkv import __all__  # noqa: F401
