"""B200 (sm_100a) pixel-adaptive dictionary regression: Python binding of the C-ABI CUDA library.

The work happens in `libsr.so` (hand-written CUDA under `csrc/`, ABI in `include/sr.h`); this package
only marshals arguments. Build the library with `python -m paper_2303_08999_b200.build`.
"""
from .api import (SR_CLAMP01, SR_COEF_COMPACT, SR_F16, SR_F32, SR_IDX_GLOBAL, SR_LUMA_ONLY, SR_OUT_F16, SR_OUT_U8, SR_UPSAMPLE_BILINEAR, SrError,  # noqa: F401
                  load_library, sr_bicubic_upsample, sr_bilinear_upsample, sr_device_status, sr_dict_regress_dense, sr_dict_regress_selected,
                  sr_dict_select, sr_launch_count, sr_probe_rate, sr_producer_fold, sr_producer_regress, sr_selection_gram, sr_selection_search, sr_set_wait_limit, sr_test_force_kernel, sr_test_lose_arrival, sr_tune_dense, sr_tune_reset, sr_tune_selected,
                  status_string)
