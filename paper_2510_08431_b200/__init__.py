"""B200 (sm_100a) attention-JVP library: Python binding of the C ABI in include/attn_jvp.h."""
from . import synth  # noqa: F401
from .layers import AttentionCoreJVP, TensorWithT  # noqa: F401
from .ulysses import UlyssesAttentionJVP  # noqa: F401
from .attn_jvp import (  # noqa: F401
    FWD_ONLY, KV_TANGENT_FREE, AttnJvpError, attention_jvp, attention_jvp_host, attn_jvp_device_status,
    attn_jvp_fwd, attn_jvp_fwd_host, attn_jvp_fwd_mu, attn_jvp_host_workspace_bytes, attn_jvp_fwd_splitkv, attn_jvp_fwd_splitkv_static, attn_jvp_fwd_stream, attn_jvp_qknorm_fwd, attn_jvp_selftest_bounded_wait, attn_jvp_set_stream, attn_jvp_set_tuning,
    attn_jvp_splitkv_workspace_bytes, attn_jvp_suggest_splits, attn_jvp_strerror, attn_jvp_version, load, qknorm_jvp)
