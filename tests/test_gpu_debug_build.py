"""The bounds-checked build of the library (the same sources with -DMUSE_DEBUG): every data-derived index of
the kernels passes a range check that records a violation and skips the access.  A child process loads that build
and runs the smoke cases (tiny fp32 and the bf16 D = 128 tensor-core case, forward and backward against the
oracle) plus a two-level retrieval forward; no check may fire.  A second child hands the backward pass
a bucket permutation with one entry past N: the checks must name the two kernels that read it, and the process
must end normally."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CLEAN = """
import numpy as np, torch
import __graft_entry__ as g
from paper_2509_10406_b200 import binding as mb
assert mb.LIB_PATH.endswith("libmuse_debug.so"), mb.LIB_PATH
g.smoke()
from tests.gpu_util import Case, to_dev
from tests.test_gpu_cluster import CASES
c = Case(CASES["d128"], gain=128.0)
qbar = to_dev(c.qbar.astype(np.float32), "f32")
p = c.params(k2=1)
buf = mb.MuseBuffers(p, backward=False)
Q, K, V, _ = c.dev()
mb.muse_summarize(p, K, V, to_dev(c.a_k, "i"), qbar, buf.off_k, buf.perm_k, buf.summaries, buf.ws)
mb.muse_attn_fwd(p, Q, K, V, to_dev(c.a_q, "i"), qbar, buf.off_k, buf.perm_k, buf.summaries, None, buf.O, buf.LSE,
                 buf.sel, buf.ws, bsel_out=buf.bsel)
torch.cuda.synchronize()
assert mb.muse_status(buf.ws) == 0
n, text = mb.muse_debug_report()
assert n == 0, text
print("DEBUG-BUILD-CLEAN")
"""

BAD_PERM = """
import numpy as np, torch
from paper_2509_10406_b200 import binding as mb
from tests.gpu_util import Case, to_dev
from tests.test_gpu_cluster import CASES
c = Case(CASES["d128"], gain=128.0)
w = c.w
qbar = to_dev(c.qbar.astype(np.float32), "f32")
p = c.params()
buf = mb.MuseBuffers(p, backward=True)
Q, K, V, dO = c.dev()
aq = to_dev(c.a_q, "i")
mb.muse_summarize(p, K, V, to_dev(c.a_k, "i"), qbar, buf.off_k, buf.perm_k, buf.summaries, buf.ws)
mb.muse_attn_fwd(p, Q, K, V, aq, qbar, buf.off_k, buf.perm_k, buf.summaries, None, buf.O, buf.LSE, buf.sel, buf.ws)
torch.cuda.synchronize()
assert mb.muse_debug_report()[0] == 0
buf.perm_k.view(-1)[7] = w.N + 5                     # one bucketed position names a key that does not exist
# the backward pass that rebuilds the summaries reads the permutation twice: in the row gather of the bucketed K, V
# copies and when it returns dK, dV to token order; both checks fire, both accesses are skipped
ws = torch.empty(buf.sizes[5], dtype=torch.uint8, device="cuda")
mb.muse_attn_bwd(p, Q, K, V, buf.O, buf.LSE, dO, aq, qbar, buf.off_k, buf.perm_k, None, buf.sel, buf.dQ, buf.dK, buf.dV, ws)
torch.cuda.synchronize()
n, text = mb.muse_debug_report()
assert n == 2 and "summarize.cu" in text and "attn_bwd.cu" in text and str(w.N + 5) in text, (n, text)
assert mb.muse_debug_report()[0] == 0                # the report cleared the records
print("DEBUG-BUILD-CAUGHT", text)
"""


def _child(code):
    lib = os.path.join(ROOT, "paper_2509_10406_b200", "libmuse_debug.so")
    if not os.path.exists(lib):
        from paper_2509_10406_b200 import build as b
        b.build(debug=True)
    env = dict(os.environ, MUSE_LIBRARY="libmuse_debug.so", PYTHONPATH=ROOT)
    return subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)


def test_bounds_checked_build_runs_clean():
    r = _child(CLEAN)
    assert r.returncode == 0 and "DEBUG-BUILD-CLEAN" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]


def test_bounds_checked_build_records_a_bad_permutation():
    r = _child(BAD_PERM)
    assert r.returncode == 0 and "DEBUG-BUILD-CAUGHT" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]


def test_product_build_has_no_checks():
    from paper_2509_10406_b200 import binding as mb
    if "debug" in os.path.basename(mb.LIB_PATH):
        pytest.skip("suite is running against the bounds-checked build")
    assert mb.muse_debug_report()[0] == -2            # MUSE_ERR_UNSUPPORTED
