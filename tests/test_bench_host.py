"""Host-side logic of bench.py that needs no GPU: the multi-GPU relaunch and the clock summary."""
import os
import sys
import types

import bench


def test_gpus_flag_starts_that_many_ranks_on_the_loopback_address(monkeypatch):
    seen = {}
    monkeypatch.setattr(os, "execv", lambda exe, argv: seen.update(exe=exe, argv=argv))
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "4", "--steps", "7", "--warmup", "3"])
    bench.relaunch_under_torchrun(types.SimpleNamespace(gpus=4))
    argv = seen["argv"]
    assert seen["exe"] == sys.executable and argv[1:3] == ["-m", "torch.distributed.run"]
    assert "--nproc-per-node=4" in argv and "--nnodes=1" in argv
    assert argv[argv.index("--master-addr") + 1] == "127.0.0.1"
    assert 1024 < int(argv[argv.index("--master-port") + 1]) < 65536
    script = argv.index(os.path.abspath(bench.__file__))
    assert argv[script + 1:] == ["--gpus", "4", "--steps", "7", "--warmup", "3"]


def test_clock_summary_keeps_only_samples_inside_the_timed_region():
    s = bench.ClockSampler(0)
    row = lambda mhz, cap: [str(mhz), "1965", "700.0", "Not Active", "Not Active", "Not Active", cap]
    s.rows = [(10.0, row(1965, "Not Active")), (11.0, row(1500, "Active")), (11.5, row(1470, "Active")),
              (12.0, row(1480, "Active")), (13.0, row(1965, "Not Active"))]
    inside = s.summary(10.9, 12.1)
    assert inside["samples"] == 3 and inside["sm_mhz"] == 1480.0 and inside["reasons"] == ["sw_power_cap"]
    assert s.summary()["samples"] == 5 and s.summary(20.0, 30.0)["samples"] == 0
