"""PHOTON decode-step library for B200 (sm_100a): ctypes binding over libphoton.so.

`workloads` (seeded inputs) is importable without the shared library; every
photon_* call loads it on first use and raises if it is missing.
"""
from . import workloads  # noqa: F401
from .binding import (  # noqa: F401
    PHOTON_DEV_BAD_INDEX, PHOTON_DEV_CAPACITY, PHOTON_DEV_TIMEOUT, PHOTON_ERR_CUDA,
    PHOTON_ERR_INVALID_ARG, PHOTON_ERR_UNSUPPORTED, PHOTON_ERR_WORKSPACE, PHOTON_OK,
    PHOTON_W_IN_MAJOR, PHOTON_W_OUT_MAJOR, HostIO, PhotonError, load, make_kv, make_layer, make_layer_scratch, make_step_args,
    photon_chunk_attn, photon_chunk_causal_attn, photon_coarse_attn, photon_coarse_attn_noalloc, photon_config, photon_converter, photon_create,
    photon_decode_step, photon_decode_step_host, photon_destroy, photon_device_status, photon_flat_attn, photon_kv,
    photon_decoder_prefill, photon_decoder_step, photon_encoder_step, photon_kv_append, photon_launch_count, photon_layer, photon_layer_scratch, photon_linear,
    photon_read_probe, photon_wait_probe, photon_rmsnorm, photon_rope_split, photon_swiglu, photon_set_attention_ctas, photon_set_host_step_tuning, photon_status_str, photon_step_args,
)
