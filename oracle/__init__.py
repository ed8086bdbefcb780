"""CPU oracle (test infrastructure only; never imported by the product path)."""
from .dst_oracle import (  # noqa: F401
    OracleResult,
    SgdResult,
    apply_sgd,
    build_oracle_library,
    bytes_report,
    densify,
    round_bf16,
    widen_bf16,
)
from .cpu_threads import build_cpu_threads_library, densify_threads, host_cores  # noqa: F401,E402
