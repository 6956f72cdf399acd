"""GPU parity of the alternative kernel paths.  Shapes that the tensor-core far-field, summary and
cluster-resident retrieval kernels do not cover fall back to other kernels of the library; an
environment switch forces each of those paths at shapes where the default would be the tensor-core
one, so that both are held to the same oracle and the same tolerances (2e-2 relative max-abs in
bf16 mode) on identical inputs."""
import os

import pytest

from tests.test_gpu_cluster import CASES
from tests.test_gpu_forward import _forward_parity
from tests.test_gpu_backward import _backward_parity

pytestmark = pytest.mark.gpu

# switch -> which pass it affects
SWITCHES = {
    "MUSE_SUMM_FWD_SIMT": "fwd",     # summaries without the tensor-core kernel
    "MUSE_FAR_SIMT": "both",         # far field (forward and backward) without the tensor-core kernels
    "MUSE_SUMM_SIMT": "bwd",         # key-side pass through the summaries without the tensor-core kernel
    "MUSE_RET_FWD_STREAM": "fwd",    # retrieval forward: one CTA per (cluster, plane) group instead of per cluster
    "MUSE_RET_BWD_SPLIT": "bwd",     # retrieval backward: separate dQ and dK/dV kernels instead of the fused one
}


@pytest.mark.parametrize("switch", list(SWITCHES))
def test_alternative_path_matches_oracle(switch):
    w = CASES["d128"]
    old = os.environ.get(switch)
    os.environ[switch] = "1"
    try:
        if SWITCHES[switch] in ("fwd", "both"):
            _forward_parity(w, 128.0)
        if SWITCHES[switch] in ("bwd", "both"):
            _backward_parity(w, 128.0)
    finally:
        if old is None:
            del os.environ[switch]
        else:
            os.environ[switch] = old
