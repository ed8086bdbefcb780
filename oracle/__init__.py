"""CPU oracle (test infrastructure only; never imported by the product path)."""
from .dst_oracle import (  # noqa: F401
    OracleResult,
    build_oracle_library,
    bytes_report,
    densify,
    round_bf16,
    widen_bf16,
)
