"""DeltaLog recurrent-state decode for linear attention on B200 (sm_100a).

``binding``  ctypes binding of the C ABI in ``include/deltalog.h`` (the CUDA kernels live in ``csrc/``)
``traffic``  the algorithmic-byte model of one decode cycle (Eq. 7-9 adapted to the split merge)
``build``    compiles ``csrc/*.cu`` into ``libdeltalog.so``
"""
from . import traffic  # noqa: F401
from .binding import (  # noqa: F401
    BF16, F32, GDN, GLA, HINT_BASE_UNTOUCHED, HINT_SLOTS_STABLE, HINT_WALK_DOWN, KDA, LINATTN, RETNET, RWKV6, STATUS_BAD_SLOT, STATUS_LOG_FULL, STATUS_TIMEOUT, DeltalogError, Desc,
    HostLane, HostStaging, State, decode_merge_step, decode_step, decode_steps, decode_step_host_overlapped, decode_step_host, decode_step_host_static, eager_step, build_id, launch_count, load_library, merge, packed_host_tokens, reset_slots,
    status_string, version,
)
