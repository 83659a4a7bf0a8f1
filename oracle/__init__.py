"""fp64 CPU oracle of the filtered convolution backward pass.

TEST INFRASTRUCTURE, NOT THE PRODUCT: imported only by tests, the smoke check
and the benchmark's CPU-baseline leg.
"""
from .gf_oracle import (act_stash_forward, activation, activation_fast, backward, exact_backward, expand, grid, kernel_sum,  # noqa: F401
                        literal_backward, num_threads, patch_mean, patch_sum,
                        reduced_gw, reduced_gx, stash_forward, stash_num_values)
from .gf_diagnostics import dcac_ratio, filter_snr_terms, snr_terms, snr_terms_fast  # noqa: F401,E402
from .gf_strided import (exact_backward_strided, kernel_phase_sums, strided_backward,  # noqa: F401,E402
                         strided_stash_forward)
from . import gf_int8 as int8  # noqa: F401,E402
