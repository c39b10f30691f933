"""B200-native FlexiQ hot path: channel-wise mixed 4/8-bit quantized GEMM / conv.

The product is the C-ABI CUDA library ``libflexiq.so`` (declared in ``include/flexiq.h``);
``binding`` is a thin ctypes layer with the same entry-point names.  PyTorch is used only
for device memory and streams.  There is no CPU fallback: loading fails loudly when the
library has not been built.
"""
from . import binding  # noqa: F401
from .binding import (  # noqa: F401
    DTYPE_BF16, DTYPE_F16, DTYPE_F32, DTYPE_I8, LOWBIT_MASKED_I8, LOWBIT_PACKED_U4,
    OUT_ACC_I32, OUT_DEQUANT_BF16, OUT_DEQUANT_F16, OUT_DEQUANT_F32, OUT_REQUANT_I8, FlexiqError, Layer,
)
