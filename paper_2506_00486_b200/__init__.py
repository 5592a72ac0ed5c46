"""B200-native generalized-Gaussian (GG) pass: moments, fit, penalty gradient, symbol histogram
and entropy, and GG sampling, as hand-written sm_100a CUDA behind a small C interface.

`binding` marshals torch tensors into that interface; `build` compiles the library in-tree.
Nothing here computes on the CPU.
"""
from .binding import (BETA_HI, BETA_LO, FLAG_BETA_CLAMPED_HI, FLAG_BETA_CLAMPED_LO,  # noqa: F401
                      FLAG_CLAMPED_SYMBOLS, FLAG_DEGENERATE, FLAG_NONFINITE, GG_BF16, GG_F32,
                      GG_MEAN, GG_PARAMS_FITTED, GG_PARAMS_GIVEN, GG_RATE_EG, GG_STEP_FROM_ALPHA,
                      GG_STEP_GIVEN, GG_SUM, Context, GGError, Segments, gg_alpha_from_std, gg_compression_ratio, gg_fit_noalloc,
                      gg_diff_entropy_bits, gg_init_alpha)
