"""Float64 CPU oracle of the PPOW window-scoring pass.  Test infrastructure, not the product."""
from .ppow_oracle import (BF16, F32, GREEDY, STOCHASTIC, build, score_windows, select_windows,  # noqa: F401
                          tau_cumprod)
