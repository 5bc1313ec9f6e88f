"""B200-native residual-binary linear layer (RaBiT inference hot path).

The product is ``librabit.so`` (hand-written CUDA for sm_100a behind a C ABI, declared in
``include/rabit.h``).  This package is the thin binding: it marshals arguments and owns
nothing but the descriptor handle.  There is no CPU fallback: if the library is missing the
import fails.
"""
from .binding import (  # noqa: F401
    RabitError,
    RabitLayer,
    layout_version,
    lib_path,
    packed_bytes,
    pack_host,
    unpack_host,
    rabit_pack,
    rabit_derive_pack,
    rabit_linear,
    rabit_linear_group,
    rabit_linear_group_host,
    PreparedGroupHost,
    rabit_linear_host,
    rabit_linear_static_scratch,
    rabit_free,
    last_error,
)
