"""B200-native XFP decode path: a C-ABI CUDA library (libxfp.so) and its thin Python binding."""
from .binding import (XfpDesc, XfpError, PackedMatrix, library_path, load_library, xfp_packed_size, xfp_pack,
                      xfp_gemv_v2, xfp_gemv_v2a, xfp_gemv_grouped, xfp_gemv_host, xfp_dequant, xfp_status_str,
                      pack_tensors, xfp_gemv_v2_noalloc, xfp_gemv_grouped_epilogue, XFP_EPI_NONE, XFP_EPI_SWIGLU,
                      XFP_EPI_COMBINE, xfp_gemv_typed, xfp_gemv_grouped_typed, XFP_T_F32, XFP_T_F16, XFP_T_BF16, xfp_gemm, xfp_gemm_workspace_size,
                      xfp_gemm_typed, xfp_gemm_typed_workspace_size)

__all__ = ["XfpDesc", "XfpError", "PackedMatrix", "library_path", "load_library", "xfp_packed_size", "xfp_pack",
           "xfp_gemv_v2", "xfp_gemv_v2a", "xfp_gemv_grouped", "xfp_gemv_host", "xfp_dequant", "xfp_status_str",
           "pack_tensors", "xfp_gemv_v2_noalloc", "xfp_gemv_grouped_epilogue", "XFP_EPI_NONE", "XFP_EPI_SWIGLU",
           "XFP_EPI_COMBINE", "xfp_gemv_typed", "xfp_gemv_grouped_typed", "XFP_T_F32", "XFP_T_F16", "XFP_T_BF16", "xfp_gemm",
           "xfp_gemm_workspace_size", "xfp_gemm_typed", "xfp_gemm_typed_workspace_size"]
