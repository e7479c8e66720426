"""QSGD gradient codec for NVIDIA B200: hand-written sm_100a kernels behind a C ABI
(include/qsgd.h), with a thin ctypes binding. The library is loaded on first use."""
from .binding import (CODE_ELIAS, CODE_ELIAS_DENSE, CODE_FIXED, NORM_L2, NORM_MAX,  # noqa: F401
                      QsgdError, encode_alloc, new_status, qsgd_decode_accumulate,
                      qsgd_decode_sgd_step, qsgd_decode_accumulate_packed, qsgd_decode_sgd_step_packed, qsgd_encode, qsgd_encode_elias_static, qsgd_fixed_layout, qsgd_launch_count,
                      qsgd_message_capacity, qsgd_profile_collect, qsgd_profile_enable,
                      qsgd_sgd_step, qsgd_static_scratch_bytes, qsgd_workspace_bytes,
                      Policy, qsgd_policy_decode_accumulate, qsgd_policy_decode_sgd_step,
                      qsgd_policy_encode, qsgd_policy_message_capacity, qsgd_policy_workspace_bytes,
                      qsgd_test_default_wait_polls, qsgd_test_set_wait_polls, qsgd_set_launch_chaining)
