"""CPU float64 oracle for the LoRDBA adapter forward -- test infrastructure only.

Nothing in the product package imports this; see ``oracle/lordba_oracle.c``.
"""
from .oracle import (  # noqa: F401
    build,
    num_threads,
    adapter_forward,
    adapter_forward_ell,
    packed_words,
    pack_signs,
    unpack_signs,
    adapter_bits,
    lora_fp16_bits,
    bpw_tot,
    bandwidth_ratio,
    widen_bf16,
)
