"""B200 library for unaligned block-wise pruned (UBP) layers -- Python binding.

Thin ctypes layer over ``libubp_b200.so`` (C ABI declared in ``include/ubp.h``).
Every function here only marshals arguments: packing runs in the library's
host code, every product runs in its CUDA kernels. PyTorch is used for
device memory and streams. There is no CPU fallback: if the shared library
is missing or a call fails, an exception is raised.
"""
from .binding import (UbpError, Plan, pack_ubp, unpack_ubp, blob_view, plan_size, plan_image, variants,
                      ubp_pack, ubp_unpack, ubp_spmm, ubp_conv1x1, ubp_conv3x3_implicit, ubp_spmm_static,
                      static_plan_capacity, lib_path, load, BedSelector, ubp_block_scores, ubp_bed_select,
                      ubp_pack_kmajor, ubp_kmajor_to_plan_blob)

__all__ = ["UbpError", "Plan", "pack_ubp", "unpack_ubp", "blob_view", "plan_size", "plan_image", "variants",
           "ubp_pack", "ubp_unpack", "ubp_spmm", "ubp_conv1x1", "ubp_conv3x3_implicit", "ubp_spmm_static",
           "static_plan_capacity", "lib_path", "load", "BedSelector", "ubp_block_scores", "ubp_bed_select",
           "ubp_pack_kmajor", "ubp_kmajor_to_plan_blob"]
