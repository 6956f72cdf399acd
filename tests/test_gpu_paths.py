"""GPU parity of the alternative kernel paths.  Shapes that the tensor-core far-field, summary and
cluster-resident retrieval kernels do not cover fall back to other kernels of the library; a
test hook of the library forces each of those paths at shapes where the default would be the tensor-core
one, so that both are held to the same oracle and the same tolerances (2e-2 relative max-abs in
bf16 mode) on identical inputs."""
import pytest

from tests.test_gpu_cluster import CASES
from tests.test_gpu_forward import _forward_parity
from tests.test_gpu_backward import _backward_parity

pytestmark = pytest.mark.gpu

# test-hook bit (muse_test_force_paths) -> (which pass it affects, a kernel that must then run)
SWITCHES = {
    "summaries_simt": (1, "fwd", "k_summarize"),            # summaries without the tensor-core kernel
    "far_simt": (2, "both", "k_far_fwd"),                   # far field (forward and backward) without the tensor-core kernels
    "summ_bwd_simt": (4, "bwd", "k_summ_bwd"),              # key-side pass through the summaries without the tensor-core kernel
    "ret_fwd_stream": (8, "fwd", "k_ret_fwd_tc"),           # retrieval forward: one CTA per (cluster, plane) group
    "ret_bwd_split": (16, "bwd", "k_ret_bwd_dq_tc"),        # retrieval backward: separate dQ and dK/dV kernels
}


@pytest.mark.parametrize("switch", list(SWITCHES))
def test_alternative_path_matches_oracle(switch):
    from paper_2509_10406_b200 import binding as mb
    bit, which, kernel = SWITCHES[switch]
    w = CASES["d128"]
    mb.muse_test_force_paths(bit)
    try:
        if which in ("fwd", "both"):
            _forward_parity(w, 128.0, expect_kernels=[kernel] if which == "fwd" or kernel.startswith("k_far_fwd") else [])
        if which in ("bwd", "both"):
            _backward_parity(w, 128.0, expect_kernels=[kernel] if which == "bwd" else [])
    finally:
        mb.muse_test_force_paths(0)
