"""CPU oracle (test infrastructure): see mate_oracle.c.  Never imported by the CUDA package."""
from .mate_oracle import (fwd, bwd, mask, mask_sat, cell_mean, plan, useful_pairs, num_threads)  # noqa: F401
