"""Host-side checks of the seeded input generators."""
import numpy as np

from paper_2607_27744_b200 import workloads as wl


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.0 + 2**-8, 1.0 + 3 * 2**-8, 1.0 + 2**-7, -(1.0 + 2**-8 + 2**-12)], np.float32)
    got = wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(x))
    want = np.array([1.0, 1.0, 1.0 + 2**-6, 1.0 + 2**-7, -(1.0 + 2**-7)], np.float32)
    assert np.array_equal(got, want)


def test_generators_are_deterministic_and_chunk_independent():
    a = wl.normal((70000, 3), 9, 1, "bf16")
    b = wl.normal((70000, 3), 9, 1, "bf16")
    assert np.array_equal(a, b)
    c = wl.normal((65536, 3), 9, 1, "bf16")
    assert np.array_equal(a[:65536], c)
    assert abs(wl.to_f64(a).std() - 1.0) < 0.02


def test_config_structure():
    for cid, cfg in wl.CONFIGS.items():
        co = wl.cand_offsets(cfg)
        assert co[0] == 0 and co.size == cfg.R + 1 and np.all(np.diff(co) >= 1)
    assert int(wl.cand_offsets(wl.CONFIGS[2])[-1]) == 131072
    assert int(wl.cand_offsets(wl.CONFIGS[4])[-1]) == 131072
    n3 = np.diff(wl.cand_offsets(wl.CONFIGS[3]))
    assert n3.max() <= 4096 and 30000 < n3.sum() < 90000
    n5 = np.diff(wl.cand_offsets(wl.CONFIGS[5]))
    assert n5.max() == 8192 and n5.min() == 1 and np.median(n5) < 64
    L5 = np.diff(wl.seq_offsets(wl.CONFIGS[5]))
    assert L5.min() >= 256 and L5.max() <= 1024


def test_stratified_sample_covers_segment_ends():
    co = np.array([0, 3, 3, 10, 11], np.int32)
    s = wl.stratified_sample(co, n_uniform=4, n_small_requests=1)
    for i in (0, 2, 3, 9, 10):
        assert i in s
    assert s.min() >= 0 and s.max() < 11 and np.all(np.diff(s) > 0)
