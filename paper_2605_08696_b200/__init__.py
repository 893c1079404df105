"""B200-native (sm_100a) Structured Recurrent Mixer decode path.

`binding` is a thin ctypes layer over the C-ABI library libsrm.so (include/srm.h): it marshals
torch device buffers and streams into the calls, nothing else. All arithmetic of the path runs
in the CUDA kernels under csrc/.
"""
from .binding import (SRM, SRMState, Sampling, SRMError, load_library, lib_path,  # noqa: F401
                      k_wait_probe, k_ffn_plan, k_mixer_combined_step, k_mixer_kernel_step, k_mixer_combined_scan, k_mixer_kernel_scan,
                      EPI_BIAS_GELU, EPI_BIAS_RESIDUAL, EPI_PLAIN, FLAG_NO_GRAPH, FLAG_GRAPH, FLAG_NO_SPLITK, FLAG_NO_FUSED_TOPK, FLAG_NO_SMALL_BATCH, FLAG_NO_TAIL_SPLIT, FLAG_NO_FUSED_FFN, FLAG_NO_KSLICE, FLAG_SIMT_GEMM, FLAG_HEAD_PROJ,
                      ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_BUFFER_TOO_SMALL, ERR_CTX_OVERFLOW,
                      ERR_CUDA, ERR_DEVICE_STATUS, ERR_STATIC_SCRATCH)
