"""B200 (sm_100a) delta-rule linear-attention prefill: GDN and KDA, chunkwise, behind a C ABI.

`binding` marshals torch CUDA tensors into the C struct of include/ha_la.h and calls
libha_la.so; `synth` draws the seeded synthetic workloads; `build` compiles the library.
Importing the package loads nothing native; the first call does, and raises if the
library has not been built.
"""
from .binding import (  # noqa: F401
    HaLaError,
    ha_la_debug_wait_timeout,
    ha_la_decode,
    ha_la_decode_args,
    ha_la_decode_raw,
    ha_la_prefill,
    ha_la_prefill_args,
    ha_la_prefill_launch_plan,
    ha_la_prefill_num_launches,
    ha_la_prefill_num_segments,
    ha_la_prefill_path,
    ha_la_prefill_noalloc,
    ha_la_prefill_noalloc_scratch_bytes,
    ha_la_prefill_raw,
    ha_la_prefill_timed,
    ha_la_prefill_workspace_bytes,
    ha_la_version,
    load_library,
    make_args,
    prepare_args,
    prepare_decode_args,
    status_string,
)
