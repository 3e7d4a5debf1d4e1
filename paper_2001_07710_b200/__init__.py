"""Pattern-based sparse 3x3 convolution for B200 (sm_100a): C-ABI CUDA library + thin Python binding."""
from .binding import (PAT_F16, PAT_F32, PAT_PRUNED, PatError, load, pat_blob_layout, pat_conv3x3, pat_conv3x3_workspace,  # noqa: F401
                      pat_conv3x3_dense, pat_debug_set, pat_launch_count, pat_measure_fma_peak, pat_library_builtin, pat_pack, pat_pack_size, pat_project,
                      pat_project_static, pat_project_static_max_kernels, pat_project_workspace, pat_query_status,
                      pat_unpack, pat_simplex_project, pat_argmax_binarize, pat_extract_library, pat_relu_maxpool)
