"""CPU oracle for the HGEMM hot path -- TEST INFRASTRUCTURE, not product code.

Only ``tests/``, ``__graft_entry__.smoke()`` and the CPU legs of ``bench.py`` may
import this package.  It shares no code with the CUDA library and imports nothing
from it.
"""
from .hgemm_oracle import (  # noqa: F401
    build,
    f16_bits_to_f64,
    f64_to_f16_bits,
    hgemm_full,
    hgemm_f16acc_full,
    f16acc_envelope,
    f16_spacing,
    hgemm_scaled_full,
    hgemm_sampled,
    max_threads,
)
from .acceptance import (  # noqa: F401
    contract_bound,
    check_contract,
    check_scale_aware,
    canonical_bits,
)
