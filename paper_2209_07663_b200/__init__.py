"""B200-native collisionless embedding table (the hot path of Monolith, arXiv 2209.07663).

`binding` is the thin ctypes layer over the C ABI of include/mono.h;
`workload` draws seeded synthetic ID streams; `build` compiles the CUDA library.
"""
from . import workload  # noqa: F401
from .binding import (  # noqa: F401
    MonoError, MonoTable, load_library, mono_apply_grads, mono_apply_grads_host, mono_audit,
    mono_expire, mono_expire_slice, mono_export, mono_prepare_push, mono_group_lookup_pool, mono_group_apply_grads, mono_export_touched, mono_import, mono_lookup_pool, mono_lookup_pool_host,
    mono_lookup_pool_noalloc, mono_probe, mono_rehash,
    mono_read_rows, mono_reserve, mono_status, mono_table_create, mono_table_destroy, mono_timing_enable,
    mono_timing_read,
)
