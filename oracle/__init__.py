"""CPU oracle package (test infrastructure; see tilefuse_oracle.py for who may import it)."""
from .tilefuse_oracle import (  # noqa: F401
    unpack_awq, bf16_bits_to_f64, dequant_w4, dequant_w8, linear,
    linear_w4a16, linear_w8a16, solve,
)
