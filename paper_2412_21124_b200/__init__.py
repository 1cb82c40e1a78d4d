"""B200-native norm-test + AdamW step for adaptive batch-size training.

The product is the CUDA shared library behind ``include/abs_normtest.h``; this package
is its thin Python binding plus the seeded synthetic-input generators.
"""
from .binding import (ABS_BF16, ABS_F32, ABS_FLAG_DEGENERATE, ABS_FLAG_NONFINITE,  # noqa: F401
                      ABS_FLAG_VIOLATED, AbsError, FusedStep, abs_adamw_hparams, abs_adamw_step, abs_adamw_step_clipped,
                      abs_adamw_step_mixed, abs_normtest_adamw_mixed,
                      abs_decide, abs_combine_sums, abs_noalloc_fits,
                      abs_norm_test, abs_normtest_adamw, abs_normtest_adamw_noalloc,
                      abs_norm_test_coordwise, abs_normtest_adamw_coordwise, abs_norm_test_q,
                      abs_norm_test_accumulate, abs_norm_test_accumulate_adamw,
                      abs_normtest_adamw_clip_prev, abs_selftest_bounded_wait,
                      abs_persample_norm_test, abs_persample_norm_test_coordwise,
                      abs_persample_stats_bytes, abs_round_batch, abs_schedule_advance,
                      abs_schedule_init, abs_schedule_test_due, abs_stats_bytes,
                      alloc_persample_stats, alloc_stats, read_stats)
