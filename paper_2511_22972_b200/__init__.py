"""B200-native (sm_100a) FLy loose-verification step.

`binding` wraps the C ABI of libfly_verify.so (include/fly_verify.h);
`synthetic` draws the benchmark inputs; `build` compiles the library.
"""
from . import binding, build, synthetic  # noqa: F401
from .binding import FlyError, FlyVerify, VerifyBuffers, verify, verify_fused  # noqa: F401
