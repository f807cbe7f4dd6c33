"""CPU oracle of the lazy update (Algorithm 1) in dynamic fixed-point.

Test infrastructure only: imported by the tests, the smoke check and the CPU
baseline leg of the benchmark.  The CUDA library never imports it.
"""
from .kahan_oracle import (  # noqa: F401
    OracleElem,
    OracleTensor,
    OracleState,
    oracle_element,
    oracle_increment,
    oracle_rne_shift,
    oracle_next_exponent,
    oracle_next_exponent_velocity,
    oracle_step_tensor,
    oracle_step,
    oracle_fit_exponent,
    OracleAdamElem,
    oracle_adam_element,
    oracle_adam_step_tensor,
    oracle_adam_step,
    oracle_dequantize_gradient,
    OracleStrictElem,
    oracle_strict_element,
    oracle_strict_step_tensor,
    oracle_strict_step,
    oracle_next_exponent_acc,
    oracle_step_qgrad,
    oracle_quantize,
    oracle_dequantize,
    OracleMomElem,
    oracle_momentum_element,
    oracle_momentum_step_tensor,
    oracle_momentum_step,
    oracle_max_threads,
    EXP_FIXED,
    EXP_AMAX,
)
