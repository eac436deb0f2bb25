"""GPU parity: the CUDA kernels, called through the C ABI, against the fp64 CPU oracle.

Error metric for every output tensor: max_i |gpu_i - ref_i| / max_i |ref_i|, which must be
<= 1e-2 for bf16 storage and <= 1e-4 for the fp32 path.  Small cases compare every element;
the full-size configurations compare a stratified sample of candidates (segment ends, the
smallest requests, uniform draws) because the oracle is slow by design.
"""
import numpy as np
import pytest
import torch

from oracle import rocs_ref as ref
from paper_2607_27744_b200 import binding as rocs, workloads as wl
from _util import rel_err, to_dev, to_host_f64, tol_for

pytestmark = pytest.mark.gpu

PATHS = [rocs.PATH_AUTO, rocs.PATH_GENERAL]


@pytest.fixture(autouse=True)
def _reset_path():
    yield
    rocs.set_path(rocs.PATH_AUTO)
    rocs.last_device_status()


def _plan(co):
    return rocs.plan_create(to_dev(co), co)


# ------------------------------------------------------------------ linear ------------------
def _run_linear(cfg, co, bias=False, relu=False, sample=None, path=rocs.PATH_AUTO):
    rocs.set_path(path)
    d = wl.linear_inputs(cfg, co, bias=bias)
    plan = _plan(co)
    W = to_dev(d["W"])
    XR = to_dev(d["XR"]) if cfg.d_req else None
    Y = rocs.ikbo_linear(plan, XR, to_dev(d["XC"]), W[:, :cfg.d_req] if cfg.d_req else None,
                         W[:, cfg.d_req:], bias=to_dev(d["bias"]), relu=relu)
    want = ref.ikbo_linear(co, d["XR"] if cfg.d_req else None, d["XC"], d["W"], bias=d["bias"], relu=relu,
                           sample=sample)
    got = to_host_f64(Y)
    return rel_err(got if sample is None else got[sample], want)


def test_linear_config1_fp32_every_element():
    cfg = wl.CONFIGS[1]
    assert _run_linear(cfg, wl.cand_offsets(cfg), bias=True, relu=True) <= tol_for("f32")


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("relu,bias", [(False, False), (True, True)])
def test_linear_bf16_ragged_segments_several_tiles(path, relu, bias):
    # counts straddle the 128-row tiles, include empty and single-candidate requests
    co = wl.offsets_from_counts([1, 0, 127, 129, 300, 0, 2, 513, 64])
    cfg = wl.CONFIGS[2].with_(R=len(co) - 1, d_req=192, d_cand=128, d_out=320)
    assert _run_linear(cfg, co, bias=bias, relu=relu, path=path) <= tol_for("bf16")


@pytest.mark.parametrize("relu,bias", [(False, False), (True, True)])
def test_linear_bf16_narrow_input_many_short_segments(relu, bias):
    # N >= 512 with d_cand <= 256 takes the weight-stationary kernel; segments of 0..40 rows put
    # several requests into every 32-row slab, so both the shared-memory and the global request
    # rows are exercised; d_out = 328 leaves a ragged last column slice
    counts = [(i * 7) % 41 for i in range(70)]
    co = wl.offsets_from_counts(counts)
    cfg = wl.CONFIGS[5].with_(R=len(counts), d_req=64, d_cand=200, d_out=328)
    assert _run_linear(cfg, co, bias=bias, relu=relu) <= tol_for("bf16")


@pytest.mark.parametrize("path", PATHS)
def test_linear_bf16_odd_widths(path):
    co = wl.offsets_from_counts([5, 77, 1])
    cfg = wl.CONFIGS[2].with_(R=3, d_req=72, d_cand=40, d_out=24)
    assert _run_linear(cfg, co, relu=True, path=path) <= tol_for("bf16")


@pytest.mark.parametrize("path", PATHS)
def test_linear_bf16_no_request_half(path):
    co = wl.offsets_from_counts([200, 56])
    cfg = wl.CONFIGS[2].with_(R=2, d_req=0, d_cand=256, d_out=256)
    assert _run_linear(cfg, co, bias=True, relu=True, path=path) <= tol_for("bf16")


@pytest.mark.parametrize("relu,bias", [(False, True), (True, False)])
def test_plain_linear_bf16_wide_many_rows(relu, bias):
    # M >= 2048 rows, wide K and d_out >= 256 take the CTA-pair K-ring GEMM; M is not a multiple of the
    # 256-row super-tile and d_out = 328 leaves a ragged last column tile
    g = np.random.default_rng(17)
    M, d_in, d_out = 2500, 712, 328
    X = wl.store(g.standard_normal((M, d_in), dtype=np.float32), "bf16")
    W = wl.store(g.standard_normal((d_out, d_in), dtype=np.float32) * d_in ** -0.5, "bf16")
    b = g.standard_normal(d_out).astype(np.float32) if bias else None
    y = rocs.linear(to_dev(X), to_dev(W), bias=to_dev(b), relu=relu)
    want = ref.ikbo_linear(wl.offsets_from_counts([M]), None, X, W, bias=b, relu=relu)
    assert rel_err(to_host_f64(y), want) <= tol_for("bf16")


def test_linear_empty_batch():
    co = np.zeros(3, np.int32)
    cfg = wl.CONFIGS[2].with_(R=2, d_req=64, d_cand=64, d_out=64)
    plan = _plan(co)
    d = wl.linear_inputs(cfg, co)
    W = to_dev(d["W"])
    Y = rocs.ikbo_linear(plan, to_dev(d["XR"]), torch.empty((0, 64), dtype=torch.bfloat16, device="cuda"),
                         W[:, :64], W[:, 64:])
    assert Y.shape == (0, 64)


def test_linear_config2_shapes_reduced_rows():
    # full widths of config 2 (512 | 256 -> 1024), fewer requests so the oracle finishes in seconds
    cfg = wl.CONFIGS[2].with_(R=5, count_const=150)
    assert _run_linear(cfg, wl.cand_offsets(cfg), relu=True) <= tol_for("bf16")


def test_mlp_config2_three_layers_reduced_rows():
    cfg = wl.CONFIGS[2].with_(R=3, count_const=100)
    co = wl.cand_offsets(cfg)
    d = wl.linear_inputs(cfg, co)
    ws = wl.mlp_weights(cfg)
    plan = _plan(co)
    W = to_dev(d["W"])
    h = rocs.ikbo_linear(plan, to_dev(d["XR"]), to_dev(d["XC"]), W[:, :cfg.d_req], W[:, cfg.d_req:], relu=True)
    h = rocs.linear(h, to_dev(ws[0]), relu=True)
    y = rocs.linear(h, to_dev(ws[1]))
    r = ref.ikbo_linear(co, d["XR"], d["XC"], d["W"], relu=True)
    one = wl.offsets_from_counts([r.shape[0]])
    r = ref.ikbo_linear(one, None, r, wl.to_f64(ws[0]), relu=True)
    r = ref.ikbo_linear(one, None, r, wl.to_f64(ws[1]))
    assert rel_err(to_host_f64(y), r) <= tol_for("bf16")


def test_mlp_config2_full_size_sampled():
    # the whole benchmark step (plan, split layer, two plain layers) at full size; the oracle follows
    # the sampled candidates through all three layers in fp64
    cfg = wl.CONFIGS[2]
    co = wl.cand_offsets(cfg)
    d = wl.linear_inputs(cfg, co)
    ws = wl.mlp_weights(cfg)
    sample = wl.stratified_sample(co, n_uniform=128, n_small_requests=0, cfg_id=2)
    plan = _plan(co)
    W = to_dev(d["W"])
    h = rocs.ikbo_linear(plan, to_dev(d["XR"]), to_dev(d["XC"]), W[:, :cfg.d_req], W[:, cfg.d_req:], relu=True)
    h = rocs.linear(h, to_dev(ws[0]), relu=True)
    y = rocs.linear(h, to_dev(ws[1]))
    r = ref.ikbo_linear(co, d["XR"], d["XC"], d["W"], relu=True, sample=sample)
    one = wl.offsets_from_counts([r.shape[0]])
    r = ref.ikbo_linear(one, None, r, wl.to_f64(ws[0]), relu=True)
    r = ref.ikbo_linear(one, None, r, wl.to_f64(ws[1]))
    assert rel_err(to_host_f64(y)[sample], r) <= tol_for("bf16")


def test_isolation_config2_full_size_is_bit_exact():
    # Eq. 1 at the size and launch configuration the benchmark times: one candidate changes, every
    # other output row of the split layer keeps its bits
    cfg = wl.CONFIGS[2]
    co = wl.cand_offsets(cfg)
    d = wl.linear_inputs(cfg, co)
    plan = _plan(co)
    W, XR, XC = to_dev(d["W"]), to_dev(d["XR"]), to_dev(d["XC"])
    base = rocs.ikbo_linear(plan, XR, XC, W[:, :cfg.d_req], W[:, cfg.d_req:], relu=True)
    j = 77_777
    XC2 = XC.clone()
    XC2[j] += 1.0
    pert = rocs.ikbo_linear(plan, XR, XC2, W[:, :cfg.d_req], W[:, cfg.d_req:], relu=True)
    same = (base.view(torch.int16) == pert.view(torch.int16)).all(dim=1)
    assert not bool(same[j])
    same[j] = True
    assert bool(same.all())


def test_linear_config2_full_size_sampled():
    cfg = wl.CONFIGS[2]
    co = wl.cand_offsets(cfg)
    sample = wl.stratified_sample(co, n_uniform=256, n_small_requests=0, cfg_id=2)
    assert _run_linear(cfg, co, relu=True, sample=sample) <= tol_for("bf16")


def test_linear_config5_full_size_sampled():
    cfg = wl.CONFIGS[5]
    co = wl.cand_offsets(cfg)
    sample = wl.stratified_sample(co, n_uniform=256, n_small_requests=8, cfg_id=5)
    assert _run_linear(cfg, co, sample=sample) <= tol_for("bf16")


# ------------------------------------------------------------------ attention ---------------
def _run_dca(cfg, co, so, sample=None, path=rocs.PATH_AUTO, scale=0.0):
    rocs.set_path(path)
    d = wl.dca_inputs(cfg, co, so)
    plan = _plan(co)
    O = rocs.dca_attention(plan, to_dev(d["Q"]), to_dev(d["K"]), to_dev(d["V"]), to_dev(so), scale=scale)
    want = ref.dca_attention(co, so, d["Q"], d["K"], d["V"], scale=scale if scale > 0 else None, sample=sample)
    got = to_host_f64(O)
    return rel_err(got if sample is None else got[sample], want)


def test_dca_config1_fp32_every_element():
    cfg = wl.CONFIGS[1]
    assert _run_dca(cfg, wl.cand_offsets(cfg), wl.seq_offsets(cfg)) <= tol_for("f32")


@pytest.mark.parametrize("path", PATHS)
def test_dca_bf16_ragged(path):
    # segments around the 128-row tile, empty request, empty sequence, lengths around the key tile
    co = wl.offsets_from_counts([1, 130, 0, 128, 17, 255])
    so = wl.offsets_from_counts([5, 128, 64, 129, 0, 300])
    cfg = wl.CONFIGS[3].with_(R=6, H=2, dh=64)
    assert _run_dca(cfg, co, so, path=path) <= tol_for("bf16")


@pytest.mark.parametrize("path", PATHS)
def test_dca_bf16_several_query_tokens_and_scale(path):
    co = wl.offsets_from_counts([3, 50, 9])
    so = wl.offsets_from_counts([70, 33, 257])
    cfg = wl.CONFIGS[3].with_(R=3, H=3, dh=64, n_q=5)
    assert _run_dca(cfg, co, so, path=path, scale=0.2) <= tol_for("bf16")


def test_dca_bf16_32_query_tokens_per_candidate():
    # the paper's typical candidate-side query length (Section 4.3): four candidates fill a 128-row tile
    co = wl.offsets_from_counts([9, 1, 30])
    so = wl.offsets_from_counts([200, 64, 130])
    cfg = wl.CONFIGS[3].with_(R=3, H=2, dh=64, n_q=32)
    assert _run_dca(cfg, co, so) <= tol_for("bf16")


def test_dca_request_side_query_group():
    # A^R of Eq. 13 (first line) through the same kernel: one query group per request, i.e. a plan
    # whose "candidates" are the requests themselves
    R = 5
    co = np.arange(R + 1, dtype=np.int32)
    so = wl.offsets_from_counts([300, 17, 0, 128, 65])
    cfg = wl.CONFIGS[3].with_(R=R, H=4, dh=64, n_q=16)
    assert _run_dca(cfg, co, so) <= tol_for("bf16")


@pytest.mark.parametrize("dh", [32, 128])
def test_dca_bf16_other_head_dims(dh):
    co = wl.offsets_from_counts([40, 2])
    so = wl.offsets_from_counts([100, 31])
    cfg = wl.CONFIGS[3].with_(R=2, H=2, dh=dh)
    assert _run_dca(cfg, co, so) <= tol_for("bf16")


@pytest.mark.parametrize("dh", [32, 128])
def test_dca_bf16_head_dim_32_and_128_ragged_on_tensor_cores(dh):
    # dh = 128 runs on the tensor-core kernel with 64-key blocks, dh = 32 with 64-byte operand rows:
    # segments around the 128-row tile, empty request / sequence, lengths around the key block, several
    # query tokens
    co = wl.offsets_from_counts([1, 130, 0, 128, 17, 255])
    so = wl.offsets_from_counts([5, 128, 64, 129, 0, 300])
    cfg = wl.CONFIGS[3].with_(R=6, H=2, dh=dh)
    assert _run_dca(cfg, co, so) <= tol_for("bf16")
    cfg = wl.CONFIGS[3].with_(R=3, H=3, dh=dh, n_q=5)
    assert _run_dca(cfg, wl.offsets_from_counts([3, 50, 9]), wl.offsets_from_counts([70, 33, 257]), scale=0.1) <= tol_for("bf16")


@pytest.mark.parametrize("dh", [32, 128])
def test_dca_bf16_head_dim_32_and_128_many_tiles_sampled(dh):
    # enough tiles that every SM runs several items on both of its streams (L = 700: 11 or 6 key blocks)
    cfg = wl.CONFIGS[3].with_(R=48, H=4, dh=dh, L_const=700)
    co, so = wl.cand_offsets(cfg), wl.seq_offsets(cfg)
    sample = wl.stratified_sample(co, n_uniform=128, n_small_requests=2, cfg_id=3)
    assert _run_dca(cfg, co, so, sample=sample) <= tol_for("bf16")


@pytest.mark.parametrize("dh", [32, 64, 128])
def test_dca_bf16_scores_that_outgrow_the_first_key_block(dh):
    # The tensor-core kernel fixes a row's softmax reference from its first key block.  Keys far
    # down the sequence that are large multiples of a query row push that row's (and, through
    # chance alignment, other rows') scores hundreds of nats above the reference, beyond what
    # fp32 exponentials can hold: such rows must come out of the kernel's plain-fp32 recomputation,
    # and every other row must be untouched by it.
    co = wl.offsets_from_counts([200, 100])
    so = wl.offsets_from_counts([600, 300])
    cfg = wl.CONFIGS[5].with_(R=2, dh=dh)
    d = wl.dca_inputs(cfg, co, so)
    Q, K = wl.bf16_bits_to_f32(d["Q"]), wl.bf16_bits_to_f32(d["K"])
    K[300] = Q[5, 0] * 60.0      # request 0, third key block: +60 |q|^2 for query row 5
    K[450] = Q[140, 0] * 3.0
    K[258] = Q[7, 0] * 60.0
    K[130] = Q[150, 0] * -80.0   # second key block: huge negative for row 150, +-hundreds for the rest
    K[700] = Q[250, 0] * 40.0    # request 1, second key block
    d["K"] = wl.f32_to_bf16_bits(K)
    plan = _plan(co)
    O = rocs.dca_attention(plan, to_dev(d["Q"]), to_dev(d["K"]), to_dev(d["V"]), to_dev(so))
    want = ref.dca_attention(co, so, d["Q"], d["K"], d["V"])
    assert rel_err(to_host_f64(O), want) <= tol_for("bf16")
    assert rocs.last_device_status() == 0


def test_dca_bf16_64_query_tokens_per_candidate():
    # two candidates fill a 128-row tile (Section 4.3.2 names query tiles of 32 and 64 tokens)
    co = wl.offsets_from_counts([5, 1, 12, 2])
    so = wl.offsets_from_counts([200, 64, 130, 513])
    cfg = wl.CONFIGS[3].with_(R=4, H=2, dh=64, n_q=64)
    assert _run_dca(cfg, co, so) <= tol_for("bf16")


def test_dca_config3_shapes_reduced_requests():
    cfg = wl.CONFIGS[3].with_(R=2)
    co = wl.offsets_from_counts([140, 9])
    assert _run_dca(cfg, co, wl.seq_offsets(cfg)) <= tol_for("bf16")


def test_dca_stack_config3_two_layers_reduced():
    # h_0 = x^C; Q_l = W_Q,l h_{l-1}; A_l = DCA(Q_l, K_l, V_l); h_l = [h_{l-1}, A_l]
    cfg = wl.CONFIGS[3].with_(R=2, L_const=200)
    co = wl.offsets_from_counts([70, 3])
    so = wl.seq_offsets(cfg)
    d = wl.dca_stack_inputs(cfg, co, so)
    plan = _plan(co)
    N = int(co[-1])
    h = to_dev(d["XC"])
    hr = wl.to_f64(d["XC"])
    one = wl.offsets_from_counts([N])
    for lay in d["layers"]:
        q = rocs.linear(h, to_dev(lay["WQ"]))
        a = rocs.dca_attention(plan, q.view(N, 1, cfg.H, cfg.dh), to_dev(lay["K"]), to_dev(lay["V"]), to_dev(so))
        h = torch.cat([h, a.view(N, -1)], dim=1).contiguous()
        qr = ref.ikbo_linear(one, None, hr, wl.to_f64(lay["WQ"]))
        ar = ref.dca_attention(co, so, qr.reshape(N, 1, cfg.H, cfg.dh), wl.to_f64(lay["K"]), wl.to_f64(lay["V"]))
        hr = np.concatenate([hr, ar.reshape(N, -1)], axis=1)
    assert rel_err(to_host_f64(h), hr) <= tol_for("bf16")


def test_dca_stack_config3_full_size_sampled():
    # two stacked DCA layers at full size: Q_l = W_Q,l h_{l-1}, A_l = DCA(Q_l, K_l, V_l), h_l = [h_{l-1}, A_l];
    # the oracle follows a sample of candidates through both layers
    cfg = wl.CONFIGS[3]
    co, so = wl.cand_offsets(cfg), wl.seq_offsets(cfg)
    d = wl.dca_stack_inputs(cfg, co, so)
    plan = _plan(co)
    N = int(co[-1])
    sample = wl.stratified_sample(co, n_uniform=24, n_small_requests=0, cfg_id=3)[::4]
    h = to_dev(d["XC"])
    hr = wl.to_f64(d["XC"])[sample]
    one = wl.offsets_from_counts([sample.size])
    for lay in d["layers"]:
        q = rocs.linear(h, to_dev(lay["WQ"]))
        a = rocs.dca_attention(plan, q.view(N, 1, cfg.H, cfg.dh), to_dev(lay["K"]), to_dev(lay["V"]), to_dev(so))
        h = torch.cat([h, a.view(N, -1)], dim=1).contiguous()
        qr = ref.ikbo_linear(one, None, hr, wl.to_f64(lay["WQ"]))
        # the oracle attends the sampled rows against their own requests: scatter them into a full-size Q
        Qf = np.zeros((N, 1, cfg.H, cfg.dh))
        Qf[sample] = qr.reshape(-1, 1, cfg.H, cfg.dh)
        ar = ref.dca_attention(co, so, Qf, wl.to_f64(lay["K"]), wl.to_f64(lay["V"]), sample=sample)
        hr = np.concatenate([hr, ar.reshape(sample.size, -1)], axis=1)
    assert rel_err(to_host_f64(h)[sample], hr) <= tol_for("bf16")


def test_dca_config3_full_size_sampled():
    cfg = wl.CONFIGS[3]
    co, so = wl.cand_offsets(cfg), wl.seq_offsets(cfg)
    sample = wl.stratified_sample(co, n_uniform=64, n_small_requests=1, cfg_id=3)
    assert _run_dca(cfg, co, so, sample=sample) <= tol_for("bf16")


def test_dca_config5_full_size_sampled():
    cfg = wl.CONFIGS[5]
    co, so = wl.cand_offsets(cfg), wl.seq_offsets(cfg)
    sample = wl.stratified_sample(co, n_uniform=128, n_small_requests=4, cfg_id=5)
    assert _run_dca(cfg, co, so, sample=sample) <= tol_for("bf16")


# ------------------------------------------------------------------ interaction -------------
def _run_glm(cfg, co, sample=None, path=rocs.PATH_AUTO):
    rocs.set_path(path)
    d = wl.glm_inputs(cfg, co)
    plan = _plan(co)
    outs = rocs.glm_interaction(plan, to_dev(d["XR"]), to_dev(d["XC"]), to_dev(d["W"]), cfg.n_ro, cfg.n_co)
    G, O = ref.glm_interaction(co, d["XR"], d["XC"], d["W"], cfg.n_ro, cfg.n_co, sample=sample)
    m = np.repeat(np.arange(cfg.R), np.diff(co))
    sel = (lambda a: a) if sample is None else (lambda a: a[sample])
    errs = []
    if G.shape[0]:
        errs.append(rel_err(sel(to_host_f64(outs["YC"])), G[:, cfg.n_r:]))
        errs.append(rel_err(sel(to_host_f64(outs["YR"])[m]), G[:, :cfg.n_r]))
        if O is not None:
            errs.append(rel_err(sel(to_host_f64(outs["OC"])), O[:, cfg.n_ro:]))
            errs.append(rel_err(sel(to_host_f64(outs["OR"])[m]), O[:, :cfg.n_ro]))
    return max(errs) if errs else 0.0


def test_glm_config1_fp32_every_element():
    cfg = wl.CONFIGS[1].with_(n_ro=3, n_co=2)
    assert _run_glm(cfg, wl.cand_offsets(cfg)) <= tol_for("f32")


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("which", [4, 5])
def test_glm_bf16_ragged(path, which):
    co = wl.offsets_from_counts([1, 0, 9, 8, 33, 7, 130])
    cfg = wl.CONFIGS[which].with_(R=len(co) - 1)
    if which == 5:
        cfg = cfg.with_(n_ro=0, n_co=0)
    assert _run_glm(cfg, co, path=path) <= tol_for("bf16")


@pytest.mark.parametrize("path", PATHS)
def test_glm_bf16_other_split(path):
    co = wl.offsets_from_counts([20, 3])
    cfg = wl.CONFIGS[4].with_(R=2, n_r=16, n_c=16, d_emb=64, n_ro=4, n_co=12)
    assert _run_glm(cfg, co, path=path) <= tol_for("bf16")


def test_glm_config4_full_size_sampled():
    cfg = wl.CONFIGS[4]
    co = wl.cand_offsets(cfg)
    sample = wl.stratified_sample(co, n_uniform=512, n_small_requests=0, cfg_id=4)
    assert _run_glm(cfg, co, sample=sample) <= tol_for("bf16")


def test_glm_config5_full_size_sampled():
    cfg = wl.CONFIGS[5]
    co = wl.cand_offsets(cfg)
    sample = wl.stratified_sample(co, n_uniform=512, n_small_requests=8, cfg_id=5)
    assert _run_glm(cfg, co, sample=sample) <= tol_for("bf16")


# ------------------------------------------------------------------ isolation ---------------
def _bits(t):
    return t.contiguous().view(torch.uint8).cpu().numpy().reshape(t.shape[0], -1)


@pytest.mark.parametrize("path", PATHS)
def test_candidate_isolation_is_bit_exact(path):
    """Eq. 1 on the GPU: perturb one candidate, every other candidate's output bits stay put;
    perturb one request, only its own segment moves.  Also run-to-run determinism."""
    rocs.set_path(path)
    co = wl.offsets_from_counts([130, 1, 64, 300, 5, 150])
    so = wl.offsets_from_counts([150, 20, 128, 260, 64, 33])
    cfg = wl.CONFIGS[5].with_(R=6, d_req=128, d_cand=128, d_out=256, n_ro=4, n_co=4)
    plan = _plan(co)
    N = int(co[-1])
    j = int(co[3]) + 77           # a candidate in the middle of a tile
    seg = slice(int(co[2]), int(co[3]))

    lin = wl.linear_inputs(cfg, co)
    W, XR, XC = to_dev(lin["W"]), to_dev(lin["XR"]), to_dev(lin["XC"])
    att = wl.dca_inputs(cfg, co, so)
    Q, K, V, sod = to_dev(att["Q"]), to_dev(att["K"]), to_dev(att["V"]), to_dev(so)
    g = wl.glm_inputs(cfg, co)
    GR, GC, GW = to_dev(g["XR"]), to_dev(g["XC"]), to_dev(g["W"])

    def run_all(XR, XC, Q, K, GR, GC):
        y = rocs.ikbo_linear(plan, XR, XC, W[:, :cfg.d_req], W[:, cfg.d_req:], relu=True)
        o = rocs.dca_attention(plan, Q, K, V, sod)
        gi = rocs.glm_interaction(plan, GR, GC, GW, cfg.n_ro, cfg.n_co)
        return [_bits(y), _bits(o), _bits(gi["YC"]), _bits(gi["OC"])]

    base = run_all(XR, XC, Q, K, GR, GC)
    again = run_all(XR, XC, Q, K, GR, GC)
    for a, b in zip(base, again):
        assert np.array_equal(a, b), "not run-to-run deterministic"

    XC2, Q2, GC2 = XC.clone(), Q.clone(), GC.clone()
    XC2[j] += 1.0
    Q2[j] *= 1.5
    GC2[j] += 0.5
    pert = run_all(XR, XC2, Q2, K, GR, GC2)
    others = np.ones(N, bool)
    others[j] = False
    for a, b in zip(base, pert):
        assert np.array_equal(a[others], b[others]), "another candidate's output changed"
        assert not np.array_equal(a[j], b[j])

    XR2, K2, GR2 = XR.clone(), K.clone(), GR.clone()
    XR2[2] += 1.0
    K2[int(so[2]):int(so[3])] *= 0.5
    GR2[2] += 0.5
    pert = run_all(XR2, XC, Q, K2, GR2, GC)
    outside = np.ones(N, bool)
    outside[seg] = False
    for a, b in zip(base, pert):
        assert np.array_equal(a[outside], b[outside]), "a request leaked into another segment"
        assert np.all(np.any(a[seg] != b[seg], axis=1))


# ------------------------------------------------------------------ ABI errors --------------
def test_error_codes_on_bad_arguments():
    co = wl.offsets_from_counts([4, 4])
    d_co = to_dev(co)
    with pytest.raises(rocs.RocsError) as e:
        rocs.plan_create(d_co, np.array([0, 5, 4], np.int32))
    assert e.value.code == -4
    with pytest.raises(rocs.RocsError) as e:
        rocs.plan_create(d_co, np.array([1, 4, 8], np.int32))
    assert e.value.code == -4
    plan = rocs.plan_create(d_co)                # host copy omitted: read back from the device
    assert plan.N == 8
    X = torch.zeros((8, 72), dtype=torch.bfloat16, device="cuda")
    XR = torch.zeros((2, 64), dtype=torch.bfloat16, device="cuda")
    W = torch.zeros((16, 136), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(rocs.RocsError) as e:     # misaligned view: column offset of 2 bytes
        rocs.ikbo_linear(plan, XR, X[:, 1:65], W[:, :64], W[:, 64:128])
    assert e.value.code == -2
    with pytest.raises(rocs.RocsError) as e:     # workspace too small
        rocs.ikbo_linear(plan, XR, X[:, :64], W[:, :64], W[:, 64:128],
                         workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert e.value.code == -5
    Q = torch.zeros((8, 1, 2, 36), dtype=torch.bfloat16, device="cuda")
    KV = torch.zeros((6, 2, 36), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(rocs.RocsError) as e:     # dh * 2 bytes not a multiple of 16
        rocs.dca_attention(plan, Q, KV, KV, to_dev(np.array([0, 3, 6], np.int32)))
    assert e.value.code == -2
