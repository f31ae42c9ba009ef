"""Sub-bit binary 3x3 convolution for B200 (sm_100a): thin Python binding over
the C-ABI CUDA library `libsnnconv.so`.  See include/snn_conv.h for the
contract; every step of the forward pass runs in the library's kernels."""
from .binding import (  # noqa: F401
    ACT_BIN, ACT_F16, OUT_F32, OUT_I32, OUT_BITS, PATH_AUTO, PATH_REUSE, PATH_DECODED, PATH_DECODED_TC, PATH_NAMES,
    SnnConv, SnnConvGroup, SnnConvStack, SnnError, forward_static, kernel_launches, library_path, load_library, microbench, version,
)
