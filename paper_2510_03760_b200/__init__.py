"""B200-native candidate evaluation: seeded test inputs, batched correctness check and
median-of-trials fitness of the EvoEngineer evaluation step, as CUDA kernels behind a C ABI
(include/evo.h).  This package is the thin Python binding; it needs the compiled library
(paper_2510_03760_b200/libevo.so, built by build.py) and a CUDA device, and has no fallback."""
from . import binding  # noqa: F401
from .binding import (  # noqa: F401
    EVO_U32, EVO_F32, EVO_F16, EVO_BF16, EVO_FLAG_INCOMPLETE, RESULT_DTYPE, FIT_DTYPE, EvoError, Context, Prepared, plan_inspect,
    evo_gen_inputs, evo_validate, evo_validate_host, evo_validate_static, evo_fitness, evo_fitness_host,
    default_context, load_library, results_to_numpy, fits_to_numpy, dtype_code, evo_summary, summary_to_numpy, evo_select_elite, evo_mismatch_sample, OFFENDER_DTYPE,
    evo_validate_exact, evo_validate_generated, exact_to_numpy, EXACT_DTYPE, EVO_I32, EVO_I64, EVO_U8,
    evo_validate_f64, results64_to_numpy, RESULT64_DTYPE, EVO_F64,
    SUMMARY_DTYPE, EVO_STAT_MEDIAN, EVO_STAT_MEAN, EVO_STAT_MIN, EVO_STAT_TRIMMED_MEAN,
)
