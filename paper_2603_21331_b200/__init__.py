"""B200-native row-reduction kernels: RMSNorm, LayerNorm, last-dim softmax, fused
cross-entropy and row-sum forward over bf16 [rows, D] tensors, exported from the C-ABI
library ``libak.so`` (``include/ak.h``) and bound here with ctypes.  No CPU or PyTorch
fallback exists."""
from .binding import (  # noqa: F401
    AK_OK, AK_PATH_AUTO, AK_PATH_CLUSTER, AK_PATH_CTA, AK_PATH_GENERIC, AK_PATH_SMEM, AK_PATH_WARP,
    AK_XENT_AUTO, AK_XENT_ROW, AK_XENT_SPLIT, AkError, LIB_PATH,
    AK_DTYPE_BF16, AK_DTYPE_F16, AK_DTYPE_F32, ak_choose_path_dt, ak_rmsnorm_fwd_dt, ak_softmax_fwd_dt,
    ak_xent_fwd_dt, ak_launch_count, ak_sm_count, ak_wait_timeouts, ak_layernorm_choose_path, ak_layernorm_fwd, ak_layernorm_fwd_dt, ak_rowsum_fwd_dt, ak_rmsnorm_choose_path,
    ak_rmsnorm_fwd, ak_rmsnorm_fwd_host, ak_rope_fwd, ak_rowsum_fwd,
    ak_softmax_choose_path, ak_softmax_fwd, ak_softmax_fwd_host, ak_status_string, ak_version,
    ak_xent_choose_path, ak_xent_fwd, ak_xent_fwd_host, ak_xent_fwd_static, ak_xent_fwd_ws,
    ak_xent_mean_merge, ak_xent_sum_count,
    ak_xent_vp_merge, ak_xent_vp_nsplit, ak_xent_vp_partial, ak_xent_workspace_bytes, lib,
)
