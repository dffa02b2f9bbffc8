"""B200-native two-dimensional KV-cache migration (section 3.4 of the ReMP paper) behind a C ABI.

`api` mirrors include/remp.h; `synth` holds the seeded input generators; `build` compiles libremp.so.
"""
from .api import *  # noqa: F401,F403
from .api import RempError  # noqa: F401
