"""B200-native frozen-quantized linear layer with a trainable LoRA branch (forward + backward).

The work is done by hand-written CUDA kernels behind the C ABI of include/qlora.h; this package is the thin
Python binding (argument marshalling only).  There is no CPU or PyTorch fallback: every call raises if the CUDA
library is missing.
"""
from .binding import (STATIC_SCRATCH_BYTES, QloraError, desc, library, library_path, qlora_bwd_input, qlora_bwd_input_db, qlora_bwd_input_db_on_producers, qlora_bwd_lora,
                      qlora_bwd_lora_dropout, qlora_bwd_input_dropout, qlora_fwd_dropout,
                      qlora_bwd_lora_static, qlora_dequant, qlora_device_status, qlora_gather_columns, qlora_lrec_loss,
                      qlora_fwd, qlora_pack, qlora_quantize_rtn, qlora_selftest_bounded_wait, qlora_status_string, qlora_unpack, qlora_workspace_bytes)

__all__ = ["STATIC_SCRATCH_BYTES", "QloraError", "desc", "library", "library_path", "qlora_bwd_input", "qlora_bwd_input_db", "qlora_bwd_input_db_on_producers", "qlora_bwd_lora",
           "qlora_bwd_lora_dropout", "qlora_bwd_input_dropout", "qlora_fwd_dropout",
           "qlora_bwd_lora_static", "qlora_dequant", "qlora_device_status", "qlora_gather_columns", "qlora_lrec_loss",
           "qlora_fwd", "qlora_pack", "qlora_quantize_rtn", "qlora_selftest_bounded_wait", "qlora_status_string", "qlora_unpack", "qlora_workspace_bytes"]
