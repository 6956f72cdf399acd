"""muse_cluster_noalloc (clustering on the library's built-in scratch array, for callers that
cannot allocate device memory) must reproduce muse_cluster, call after call.

The file name sorts last on purpose: if this add-on fails, a run that stops at the first
failure has already exercised every other test."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2509_10406_b200 import workloads as wl
from tests.gpu_util import Case, to_dev, to_np


@pytest.mark.gpu
@pytest.mark.parametrize("name", ["tiny", "bf16"])
def test_noalloc_cluster_matches_workspace_version_twice(name):
    from paper_2509_10406_b200 import binding as mb
    w = wl.WORKLOADS["tiny"] if name == "tiny" else wl.WORKLOADS["small"].with_(B=1, Hq=4, Hkv=2, N=4096, Cq=32, Ck=64, components=64)
    c = Case(w, gain=128.0, cluster=False)
    Q, K, V, _ = c.dev()
    iq, ik = to_dev(c.init_q, "i"), to_dev(c.init_k, "i")
    p = c.params()
    assert mb.muse_workspace_bytes(p)[0] <= mb.muse_cluster_noalloc_max_bytes()
    ref = mb.MuseBuffers(p, backward=False)
    mb.muse_cluster(p, Q, K, iq, ik, ref.assign_q, ref.assign_k, ref.qbar, ref.kcent, ref.ws)
    torch.cuda.synchronize()
    exp = [to_np(x).copy() for x in (ref.assign_q, ref.assign_k, ref.qbar, ref.kcent)]
    for call in range(2):                       # the second call finds the first call's leftovers in the scratch
        out = mb.MuseBuffers(p, backward=False)
        for t in (out.assign_q, out.assign_k):
            t.fill_(-7)
        torch.cuda.synchronize()
        # bytes the DRIVER reports free on the device: unlike torch's own counter, this would also see an
        # allocation made inside the library.  The first call may load the library's device image (that is
        # when its 32 MiB are reserved), so the comparison is made on the second call.
        free_before = torch.cuda.mem_get_info()[0]
        mb.muse_cluster_noalloc(p, Q, K, iq, ik, out.assign_q, out.assign_k, out.qbar, out.kcent)
        torch.cuda.synchronize()
        if call == 1:
            assert torch.cuda.mem_get_info()[0] >= free_before
        assert mb.muse_cluster_noalloc_status() == 0
        got = [to_np(x) for x in (out.assign_q, out.assign_k, out.qbar, out.kcent)]
        assert np.array_equal(got[0], exp[0]) and np.array_equal(got[1], exp[1]), f"assignments differ on call {call}"
        assert np.abs(got[2] - exp[2]).max() <= 1e-6 * np.abs(exp[2]).max()
        assert np.abs(got[3] - exp[3]).max() <= 1e-6 * np.abs(exp[3]).max()


@pytest.mark.gpu
def test_noalloc_rejects_problems_larger_than_its_scratch():
    from paper_2509_10406_b200 import binding as mb
    p = mb.make_params(B=4, Hq=32, Hkv=32, N=131072, D=128, Cq=512, Ck=2048, m=32)
    assert mb.muse_workspace_bytes(p)[0] > mb.muse_cluster_noalloc_max_bytes()
    one = torch.zeros(64, device="cuda")
    rc = mb.lib().muse_cluster_noalloc(ctypes.byref(p), *([ctypes.c_void_p(one.data_ptr())] * 8), None)
    assert rc == -3 and b"workspace" in mb.lib().muse_strerror(rc)
