"""B200-native Interlaced-Mask attention of GsiT (arXiv 2505.01068): thin Python access to libgsit.so.

The C ABI is declared in include/gsit.h (test and timing hooks in include/gsit_test.h); `binding` marshals torch tensors into it.  Nothing here computes:
all arithmetic runs in the library's CUDA kernels, and a missing library raises.
"""
from .binding import (CALL_ATTENTION, CALL_LAYER, CALL_QKV_PROJ, DEVFLAG_CLAMPED, DEVFLAG_TIMEOUT, DTYPE_BF16,
                      DTYPE_F32, EXPORTS, PHASE_CUSTOM, PHASE_INTER_BWD, PHASE_INTER_FWD, PHASE_INTRA, GsitError,
                      im_attention_fwd, im_layer_fwd, im_layer_pair_fwd, plan_rows, pack_rows, unpack_rows, im_layer_fwd_static, im_qkv_proj, STATIC_SCRATCH_BYTES, last_device_status, load, make_shape, stack_head_fwd,
                      status_string, trace_enable, trace_launches, trace_read, tune_attention, version, workspace_bytes,
                      KERNEL_ATTENTION, KERNEL_LINEAR, KERNEL_LAYERNORM, ATTN_DEFAULT, ATTN_UNFUSED, ATTN_LEGACY, ATTN_TMEM,
                      expire_wait_selftest)
from .stack import GsitStack
from .hostio import HostPipeline

__all__ = [n for n in dir() if not n.startswith("_")]
