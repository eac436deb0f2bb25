"""rocs_ikbo_linear_static: the split linear layer for hosts that cannot allocate while scoring
(frozen allocator, foreign memory budget, no tolerance for an allocation's synchronisation).

Collected last on purpose.  The entry point keeps its scratch in a fixed array inside the library,
so it must give the same answer as the regular plan + workspace entry point, also on a second
call that finds the first call's leftovers in the array, and must refuse sizes beyond its limits.
"""
import numpy as np
import pytest
import torch

from oracle import rocs_ref as ref
from paper_2607_27744_b200 import binding as rocs, workloads as wl
from _util import rel_err, to_dev, to_host_f64, tol_for

pytestmark = pytest.mark.gpu


def _case(cfg, counts):
    co = wl.offsets_from_counts(counts)
    d = wl.linear_inputs(cfg.with_(R=len(counts)), co, bias=True)
    W = to_dev(d["W"])
    return co, to_dev(co), to_dev(d["XR"]), to_dev(d["XC"]), W[:, :cfg.d_req], W[:, cfg.d_req:], to_dev(d["bias"])


@pytest.mark.parametrize("cfg_id,dtype", [(2, "bf16"), (1, "f32")])
def test_static_entry_matches_regular_entry_on_two_calls_in_a_row(cfg_id, dtype):
    cfg = wl.CONFIGS[cfg_id].with_(dtype=dtype, d_req=64, d_cand=32, d_out=64) if cfg_id == 1 else \
        wl.CONFIGS[2].with_(d_req=192, d_cand=128, d_out=320)
    # second call: fewer requests, other segment boundaries, so stale Z rows and map entries
    # of the first call are still sitting in the array beyond what the second call rewrites
    for counts in ([130, 1, 0, 257, 64, 9], [3, 200, 31]):
        co, co_d, XR, XC, W_CR, W_CC, bias = _case(cfg, counts)
        plan = rocs.plan_create(co_d, co)
        want = rocs.ikbo_linear(plan, XR, XC, W_CR, W_CC, bias=bias, relu=True)
        got = torch.full_like(want, float("nan"))
        rocs.ikbo_linear_static(co_d, XR, XC, W_CR, W_CC, got, bias=bias, relu=True)
        torch.cuda.synchronize()
        assert rel_err(to_host_f64(got), to_host_f64(want)) <= tol_for(dtype)
    rocs.last_device_status()


def test_static_entry_on_the_batch_sizes_real_callers_send():
    """Batches large enough for the tensor-core candidate kernel (request rows fetched by TMA from
    the fixed array, segments that change inside 32-row slabs), two calls in a row with different
    request counts; checked against the regular entry point AND the CPU oracle; after a warm-up
    call the device's free memory must not move across a call."""
    cfg = wl.CONFIGS[2].with_(d_req=256, d_cand=128, d_out=192)
    first = True
    for counts in ([700, 3, 41, 0, 520, 17, 300], [33, 1290, 5]):
        c = cfg.with_(R=len(counts))
        co = wl.offsets_from_counts(counts)
        d = wl.linear_inputs(c, co, bias=True)
        W = to_dev(d["W"])
        co_d, XR, XC, bias = to_dev(co), to_dev(d["XR"]), to_dev(d["XC"]), to_dev(d["bias"])
        W_CR, W_CC = W[:, :c.d_req], W[:, c.d_req:]
        plan = rocs.plan_create(co_d, co)
        want = rocs.ikbo_linear(plan, XR, XC, W_CR, W_CC, bias=bias, relu=True)
        got = torch.full_like(want, float("nan"))
        if first:  # warm-up: first use of the kernels loads their code
            rocs.ikbo_linear_static(co_d, XR, XC, W_CR, W_CC, got, bias=bias, relu=True)
            torch.cuda.synchronize()
            got.fill_(float("nan"))
            first = False
        free_before = torch.cuda.mem_get_info()[0]
        rocs.ikbo_linear_static(co_d, XR, XC, W_CR, W_CC, got, bias=bias, relu=True)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the device's free memory"
        assert rel_err(to_host_f64(got), to_host_f64(want)) <= tol_for("bf16")
        oracle = ref.ikbo_linear(co, d["XR"], d["XC"], d["W"], bias=d["bias"], relu=True)
        assert rel_err(to_host_f64(got), oracle) <= tol_for("bf16")
    rocs.last_device_status()


def test_static_entry_rejects_sizes_beyond_its_scratch():
    lib = rocs.lib()
    max_z, max_n = int(lib.rocs_ikbo_linear_static_max_z_elems()), int(lib.rocs_ikbo_linear_static_max_candidates())
    assert max_z == 1 << 20 and max_n == 1 << 18
    co = wl.offsets_from_counts([4, 4])
    XR = torch.zeros((2, 64), dtype=torch.bfloat16, device="cuda")
    XC = torch.zeros((8, 64), dtype=torch.bfloat16, device="cuda")
    d_out = max_z // 2 + 8                       # R * d_out just over the limit
    W = torch.zeros((d_out, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((8, d_out), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(rocs.RocsError) as e:
        rocs.ikbo_linear_static(to_dev(co), XR, XC, W[:, :64], W[:, 64:], out)
    assert e.value.code == -8 and "scratch" in str(e.value)
    big = np.array([0, max_n + 1], np.int32)      # too many candidates
    XCb = torch.zeros((max_n + 1, 64), dtype=torch.bfloat16, device="cuda")
    Wb = torch.zeros((16, 128), dtype=torch.bfloat16, device="cuda")
    outb = torch.zeros((max_n + 1, 16), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(rocs.RocsError) as e:
        rocs.ikbo_linear_static(to_dev(big), XR[:1], XCb, Wb[:, :64], Wb[:, 64:], outb)
    assert e.value.code == -8
