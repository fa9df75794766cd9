"""Few-Bit Backward hot path for NVIDIA B200: Python binding of the C ABI.

Every step of the path runs in the CUDA library ``libfewbit.so`` (built
in-tree by ``paper_2202_00441_b200.build``); this package only marshals
arguments.  PyTorch supplies device memory and streams.  There is no CPU
fallback: if the library is missing, every call raises.
"""
from .binding import (  # noqa: F401
    ACTS, FewbitError, Table, fewbit_table_create, fewbit_table_create_ex, fewbit_table_create_folded, fewbit_table_create_opt, fewbit_table_from_arrays,
    fewbit_packed_bytes, fewbit_fwd, fewbit_fwd_bias, fewbit_bwd, fewbit_fwd_host, fewbit_bwd_host,
    fewbit_host_workspace_bytes, fewbit_launch_count, library_path, load_library,
    fewbit_fwd_host_static, fewbit_static_max_elements, fewbit_f32_activation_scan,
    fewbit_set_option, fewbit_get_option, fewbit_tail_warp_count,
)
from . import workloads  # noqa: F401
from .autograd import FewBitActivation, fewbit_activation  # noqa: F401
