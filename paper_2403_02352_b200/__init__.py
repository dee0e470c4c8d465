"""ATP prefill hot path for B200: thin Python binding over the C-ABI library libatp.so.

Every step of the path runs in the CUDA library; this package only marshals arguments
(torch tensors provide device memory and streams). There is no CPU or PyTorch fallback:
importing the binding without a built libatp.so raises.
"""
from .binding import (  # noqa: F401
    Context, AtpError, atp_principal_basis, atp_attention, atp_lowrank_linear, atp_input_norm,
    library_path, exported_symbols, atp_lowrank_linear_static, atp_alternating_basis, atp_svd_entropy,
)
