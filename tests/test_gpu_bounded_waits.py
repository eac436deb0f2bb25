"""Every barrier wait of the tensor-core kernels is bounded: when it runs out the kernel records a
code, drains and returns, and the host sees ROCS_ERR_TIMEOUT.  The self-test entry (exported by the
library, not declared in the public header) waits on a barrier nothing ever arrives on, through the
same wait routines, with a limit of one millisecond, so the expiry path runs without any kernel
hanging; afterwards the library must work as before."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import rocs_ref as ref
from paper_2607_27744_b200 import binding as rocs, workloads as wl
from _util import rel_err, to_dev, to_host_f64, tol_for

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("flavour,code", [(0, 0x701), (1, 0x702), (2, 0x703)])
def test_a_wait_that_runs_out_reports_timeout_and_leaves_the_context_usable(flavour, code):
    lib = rocs.lib()
    fn = lib.rocs_selftest_wait_expires
    fn.argtypes = [ctypes.c_int, ctypes.c_uint32, ctypes.c_void_p, ctypes.c_void_p]
    rocs.last_device_status()                      # start from a clear status word
    gave_up = torch.zeros(1, dtype=torch.int32, device="cuda")
    assert fn(flavour, 1000, gave_up.data_ptr(), None) == 0
    with pytest.raises(rocs.RocsError) as e:       # synchronises: the kernel has returned
        rocs.last_device_status()
    assert e.value.code == -7 and f"0x{code:08x}" in str(e.value)
    assert int(gave_up.item()) == 64               # all waiting threads left through the abort path
    assert rocs.last_device_status() == 0          # reading the word cleared it
    # the next ordinary call is unaffected
    cfg = wl.CONFIGS[2].with_(R=3, d_req=128, d_cand=64, d_out=128)
    co = wl.offsets_from_counts([300, 5, 260])
    d = wl.linear_inputs(cfg, co)
    W = to_dev(d["W"])
    Y = rocs.ikbo_linear(rocs.plan_create(to_dev(co), co), to_dev(d["XR"]), to_dev(d["XC"]), W[:, :128], W[:, 128:])
    assert rel_err(to_host_f64(Y), ref.ikbo_linear(co, d["XR"], d["XC"], d["W"])) <= tol_for("bf16")
    assert rocs.last_device_status() == 0


def test_self_test_rejects_bad_arguments():
    fn = rocs.lib().rocs_selftest_wait_expires
    fn.argtypes = [ctypes.c_int, ctypes.c_uint32, ctypes.c_void_p, ctypes.c_void_p]
    assert fn(5, 1000, None, None) == -1
    gave_up = torch.zeros(1, dtype=torch.int32, device="cuda")
    assert fn(0, 0, gave_up.data_ptr(), None) == -1 and fn(0, 2000000, gave_up.data_ptr(), None) == -1
