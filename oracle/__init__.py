"""Float64 CPU oracle of the PPOW window-scoring pass.  Test infrastructure, not the product."""
from .ppow_oracle import (BF16, F16, F32, GREEDY, STOCHASTIC, build, decode, diagnostics, group_advantage,  # noqa: F401
                          reference_logprob,
                          sample_start, sample_start_mixed, score_windows, select_windows, sliding_scores, tau_cumprod)
