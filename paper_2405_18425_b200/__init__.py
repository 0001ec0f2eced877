"""B200-native forward pass of ViG's bidirectional gated linear attention (BiGLA) token mixer.

The compute lives in hand-written sm_100a CUDA kernels behind a C ABI (include/vig_bigla.h,
libvig_bigla.so); `binding` marshals torch tensors into those calls and `synth` draws the seeded
synthetic inputs of the benchmark configurations.  Importing the package does not load the CUDA
library; the first binding call does and raises if it has not been built.
"""
from . import synth  # noqa: F401
from .binding import (  # noqa: F401
    VIG_DTYPE_BF16,
    VIG_DTYPE_F32,
    VigError,
    load,
    status_string,
    vig_bigla_fwd,
    vig_bigla_fwd_bf16,
    vig_bigla_fwd_f32,
    vig_bigla_fwd_gates_bf16,
    vig_bigla_fwd_blend_bf16,
    vig_bigla_bwd,
    vig_gate_prep_bwd,
    vig_dwconv3x3,
    vig_gate_blend,
    vig_bigla_fwd_host,
    vig_bigla_fwd_static_bf16,
    vig_bigla_fwd_ws_bf16,
    vig_bigla_workspace_bytes,
    vig_gate_prep_bf16,
    vig_gate_prep_f32,
    vig_kernel_launch_count,
    vig_last_device_status,
    vig_test_set_kernel_preference,
    vig_test_take_fallback_count,
    vig_test_expire_next_wait,
    VIG_TEST_KERNEL_AUTO,
    VIG_TEST_KERNEL_SIMT,
    VIG_TEST_KERNEL_CHUNK_TASKS,
    VIG_TEST_KERNEL_SEGMENTS,
)
