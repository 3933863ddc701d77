"""slim_linear_fwd against the oracle, element by element (small and ragged
cases, every kernel family) and on sampled token rows at the full sizes of the
five workload configurations."""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_09615_b200 import binding, inputs, parity
from helpers import cached_weights, run_case, to_dev

pytestmark = pytest.mark.gpu

K = binding


def assert_ok(res):
    assert res["ok"], res


# ---- small cases, all elements, every kernel family ------------------------
SMALL = [  # d_in, d_out, r, b
    (512, 512, 64, 8),       # configuration 0
    (256, 16, 0, 1),         # one tile, one k-block, no adapters
    (256, 16, 16, 1),
    (768, 48, 16, 3),        # ragged batch, three k-blocks
    (2304, 272, 112, 13),    # nine k-blocks (two k-slices), ragged rank and batch
    (4352, 1040, 208, 16),   # 17 k-blocks, 65 row tiles
    (1024, 4096, 48, 9),
]


@pytest.mark.parametrize("d_in,d_out,r,b", SMALL)
def test_small_simple_kernel(d_in, d_out, r, b):
    assert_ok(run_case(d_in, d_out, r, b, seed=11, kernel=K.KERNEL_SIMPLE))


@pytest.mark.parametrize("d_in,d_out,r,b", SMALL)
def test_small_decode_kernel(d_in, d_out, r, b):
    res = run_case(d_in, d_out, r, b, seed=12, kernel=K.KERNEL_DECODE)
    assert_ok(res)
    assert res["launches"] == 1


@pytest.mark.parametrize("b", [1, 2, 7, 8, 9, 15, 16])
def test_decode_every_batch_size(b):
    assert_ok(run_case(1024, 256, 32, b, seed=20 + b, kernel=K.KERNEL_DECODE))


def test_dispatcher_choices():
    assert K.slim_select_kernel(1, 4096, 4096, 416) == K.KERNEL_DECODE
    assert K.slim_select_kernel(16, 4096, 11008, 416) == K.KERNEL_DECODE
    assert K.slim_select_kernel(8, 512, 512, 64) == K.KERNEL_DECODE
    assert K.slim_select_kernel(4, 64, 64, 16) != K.KERNEL_DECODE      # d_in not a multiple of 256
    assert K.slim_select_kernel(17, 4096, 4096, 416) == K.KERNEL_PREFILL
    assert K.slim_select_kernel(2048, 4096, 11008, 416) == K.KERNEL_PREFILL
    assert K.slim_select_kernel(64, 48, 4096, 16) == K.KERNEL_SIMPLE        # d_out not a multiple of 128
    assert K.slim_select_kernel(50, 128, 704, 32) == K.KERNEL_SIMPLE        # d_in not a multiple of 128


def test_shapes_outside_the_fast_kernels_still_work():
    assert_ok(run_case(64, 16, 16, 2, seed=31))          # d_in = 64: simple kernel
    assert_ok(run_case(320, 32, 0, 40, seed=32))         # b > 16, no adapters
    assert_ok(run_case(704, 128, 32, 50, seed=33))       # b > 16, d_in % 128 != 0: not the prefill kernel


# ---- tcgen05 prefill kernel, small cases, all elements ----------------------
PREFILL_SMALL = [  # d_in, d_out, r, b
    (128, 128, 0, 17),       # one stage, no adapters
    (256, 128, 16, 40),
    (512, 256, 112, 200),    # ragged token tile, ragged rank, two row tiles
    (1024, 384, 64, 128),    # more stages than the ring holds
    (640, 128, 48, 8),       # a batch the dispatcher would give to the decode kernel
    (2048, 512, 208, 300),
    (1408, 128, 32, 50),     # 22 stages: the K slices of the T' launch are uneven
    (384, 256, 16, 600),     # more token tiles than stages per slice
]


@pytest.mark.parametrize("d_in,d_out,r,b", PREFILL_SMALL)
def test_small_prefill_kernel(d_in, d_out, r, b):
    res = run_case(d_in, d_out, r, b, seed=13, kernel=K.KERNEL_PREFILL)
    assert_ok(res)
    # main launch; with adapters also the T' launch and, when that one is split along K, its reduction
    assert res["launches"] in ((2, 3) if r else (1,))


# The wide variant (128 rows x 256 tokens per CTA) is what the dispatcher runs on every full-size
# prefill configuration; it is chosen when (d_out / 128) * ceil(b / 256) >= the SM count, so these
# shapes have many row tiles and a short contraction axis (the oracle stays cheap).
PREFILL_WIDE = [  # d_in, d_out, r, b
    (384, 4864, 48, 1000),   # ragged last token tile, d_in = 128 mod 256 (no rotated walk), ragged 32-column adapter stage
    (256, 19072, 0, 130),    # two token tiles, the second almost empty; no adapters
    (512, 9600, 112, 512),   # whole token tiles, ragged rank
]


@pytest.mark.parametrize("d_in,d_out,r,b", PREFILL_WIDE)
def test_wide_prefill_kernel_all_elements(d_in, d_out, r, b):
    res = run_case(d_in, d_out, r, b, seed=16, kernel=K.KERNEL_PREFILL)
    assert res["token_tile"] == 256, "this shape must run the 256-token variant"
    assert_ok(res)


def test_narrow_prefill_kernel_reports_its_tile():
    res = run_case(256, 128, 16, 40, seed=13, kernel=K.KERNEL_PREFILL)
    assert res["token_tile"] == 64 and res["ok"]


def test_wide_prefill_integer_inputs_are_exact_and_one_hot_reads_columns():
    rng = np.random.default_rng(17)
    d_in, d_out, r, b = 256, 19072, 16, 300
    codes = rng.integers(-8, 8, size=(d_out, d_in)).astype(np.int8)
    mask = inputs.top2_mask(rng.standard_normal((d_out, d_in)).astype(np.float32))
    Xi = rng.integers(-1, 2, size=(b, d_in))
    Li = rng.integers(-1, 2, size=(d_out, r))
    Ri = (rng.random((r, d_in)) < 0.05).astype(np.int64) * rng.integers(-1, 2, size=(r, d_in))
    vals, meta = K.slim_pack(to_dev(codes), to_dev(mask))
    Y = K.slim_linear_fwd(K.bf16_from_bits(bf(Xi)), vals, meta, 1.0, K.bf16_from_bits(bf(Li)),
                          K.bf16_from_bits(bf(Ri)), kernel=K.KERNEL_PREFILL)
    assert K.slim_last_token_tile() == 256
    exact = Xi @ (codes.astype(np.int64) * mask).T + (Xi @ Ri.T) @ Li.T
    assert np.abs(exact).max() <= 256
    assert np.array_equal(inputs.bf16_bits_to_f64(K.bits_from_bf16(Y)), exact.astype(np.float64))
    # one-hot activations: token m reads back column ks[m] of the weight
    ks = rng.integers(0, d_in, size=b)
    X = np.zeros((b, d_in), np.float32)
    X[np.arange(b), ks] = 1.0
    Y = K.slim_linear_fwd(K.bf16_from_bits(bf(X)), vals, meta, 0.5, None, None, kernel=K.KERNEL_PREFILL)
    assert K.slim_last_token_tile() == 256
    assert np.array_equal(inputs.bf16_bits_to_f64(K.bits_from_bf16(Y)), 0.5 * (codes.astype(np.float64) * mask)[:, ks].T)


PREFILL_PAIR = [  # d_in, d_out, r, b: even numbers of 128-row tiles
    (256, 256, 16, 40),
    (1024, 512, 112, 300),   # ragged token tile and rank, more stages than the ring holds
    (2048, 256, 0, 520),     # no adapters, three token tiles
    (1408, 256, 48, 50),     # uneven K slices of the T' launch, ragged 32-column adapter stages
]


@pytest.mark.parametrize("d_in,d_out,r,b", PREFILL_PAIR)
def test_small_prefill_pair_kernel(d_in, d_out, r, b):
    assert_ok(run_case(d_in, d_out, r, b, seed=14, kernel=K.KERNEL_PREFILL_PAIR))


def test_prefill_pair_needs_an_even_number_of_row_tiles():
    with pytest.raises(K.SlimError):
        run_case(256, 384, 16, 40, seed=14, kernel=K.KERNEL_PREFILL_PAIR)


def test_prefill_integer_inputs_are_exact():
    rng = np.random.default_rng(15)
    d_in, d_out, r, b = 256, 128, 16, 48
    codes = rng.integers(-8, 8, size=(d_out, d_in)).astype(np.int8)
    mask = inputs.top2_mask(rng.standard_normal((d_out, d_in)).astype(np.float32))
    Xi = rng.integers(-1, 2, size=(b, d_in))
    Li = rng.integers(-1, 2, size=(d_out, r))
    Ri = (rng.random((r, d_in)) < 0.05).astype(np.int64) * rng.integers(-1, 2, size=(r, d_in))
    vals, meta = K.slim_pack(to_dev(codes), to_dev(mask))
    Y = K.slim_linear_fwd(K.bf16_from_bits(bf(Xi)), vals, meta, 1.0, K.bf16_from_bits(bf(Li)),
                          K.bf16_from_bits(bf(Ri)), kernel=K.KERNEL_PREFILL)
    exact = Xi @ (codes.astype(np.int64) * mask).T + (Xi @ Ri.T) @ Li.T
    assert np.abs(exact).max() <= 256
    got = inputs.bf16_bits_to_f64(K.bits_from_bf16(Y))
    assert np.array_equal(got, exact.astype(np.float64))


def test_prefill_one_hot_tokens_read_back_weight_columns():
    rng = np.random.default_rng(16)
    d_in, d_out, b = 512, 256, 64
    codes = rng.integers(-8, 8, size=(d_out, d_in)).astype(np.int8)
    mask = inputs.top2_mask(rng.standard_normal((d_out, d_in)).astype(np.float32))
    vals, meta = K.slim_pack(to_dev(codes), to_dev(mask))
    for base in (0, 61, 300):
        ks = [(base + 7 * m) % d_in for m in range(b)]
        X = np.zeros((b, d_in), np.float32)
        X[np.arange(b), ks] = 1.0
        Y = K.slim_linear_fwd(K.bf16_from_bits(bf(X)), vals, meta, 0.5, None, None, kernel=K.KERNEL_PREFILL)
        got = inputs.bf16_bits_to_f64(K.bits_from_bf16(Y))
        want = 0.5 * (codes.astype(np.float64) * mask)[:, ks].T
        assert np.array_equal(got, want)


def test_prefill_zero_scale_keeps_the_adapter_term():
    ly = inputs.make_layer(256, 128, 32, 20, seed=17)
    vals, meta = K.slim_pack(to_dev(ly.codes), to_dev(ly.mask))
    X, L, R = K.bf16_from_bits(ly.X), K.bf16_from_bits(ly.L), K.bf16_from_bits(ly.R)
    Y = K.slim_linear_fwd(X, vals, meta, 0.0, L, R, kernel=K.KERNEL_PREFILL)
    ov, om = oracle.pack(ly.codes, ly.mask)
    ref = oracle.linear_fwd(ly.X, ov, om, 0.0, ly.L, ly.R)
    assert parity.compare(inputs.bf16_bits_to_f64(K.bits_from_bf16(Y)), ref)["ok"]
    Y0 = K.slim_linear_fwd(X, vals, meta, 0.0, None, None, kernel=K.KERNEL_PREFILL)
    assert float(Y0.float().abs().max()) == 0.0


# ---- exact cases ------------------------------------------------------------
def bf(x):
    return inputs.f32_to_bf16_bits(np.asarray(x, np.float32))


@pytest.mark.parametrize("kernel", [K.KERNEL_SIMPLE, K.KERNEL_DECODE])
def test_integer_inputs_are_exact(kernel):
    """Small integers: every partial sum is exactly representable, so the
    result must equal the integer arithmetic bit for bit."""
    rng = np.random.default_rng(5)
    d_in, d_out, r, b = 256, 64, 16, 16
    codes = rng.integers(-8, 8, size=(d_out, d_in)).astype(np.int8)
    mask = inputs.top2_mask(rng.standard_normal((d_out, d_in)).astype(np.float32))
    Xi = rng.integers(-1, 2, size=(b, d_in))
    Li = rng.integers(-1, 2, size=(d_out, r))
    Ri = (rng.random((r, d_in)) < 0.05).astype(np.int64) * rng.integers(-1, 2, size=(r, d_in))
    vals, meta = K.slim_pack(to_dev(codes), to_dev(mask))
    Y = K.slim_linear_fwd(K.bf16_from_bits(bf(Xi)), vals, meta, 1.0, K.bf16_from_bits(bf(Li)),
                          K.bf16_from_bits(bf(Ri)), kernel=kernel)
    exact = Xi @ (codes.astype(np.int64) * mask).T + (Xi @ Ri.T) @ Li.T
    assert np.abs(exact).max() <= 256          # representable in bf16
    got = inputs.bf16_bits_to_f64(K.bits_from_bf16(Y))
    assert np.array_equal(got, exact.astype(np.float64))


@pytest.mark.parametrize("kernel", [K.KERNEL_SIMPLE, K.KERNEL_DECODE])
def test_one_hot_tokens_read_back_weight_columns(kernel):
    """Token m is the unit vector e_{k(m)}: row m of Y is column k(m) of the
    weight, so any layout or index slip shows up at a known position."""
    rng = np.random.default_rng(6)
    d_in, d_out, b = 512, 48, 16
    codes = rng.integers(-8, 8, size=(d_out, d_in)).astype(np.int8)
    mask = inputs.top2_mask(rng.standard_normal((d_out, d_in)).astype(np.float32))
    vals, meta = K.slim_pack(to_dev(codes), to_dev(mask))
    for base in (0, 37, 255, 496):
        ks = [(base + 17 * m) % d_in for m in range(b)]
        X = np.zeros((b, d_in), np.float32)
        X[np.arange(b), ks] = 1.0
        Y = K.slim_linear_fwd(K.bf16_from_bits(bf(X)), vals, meta, 0.5, None, None, kernel=kernel)
        got = inputs.bf16_bits_to_f64(K.bits_from_bf16(Y))
        want = 0.5 * (codes.astype(np.float64) * mask)[:, ks].T
        assert np.array_equal(got, want)


def test_decode_is_deterministic_and_reuses_its_workspace():
    d_in, d_out, r, b = 2048, 512, 64, 16
    s, codes, mask, _, _ = cached_weights(d_out, d_in, 77)
    ly = inputs.make_layer(d_in, d_out, r, b, 77, weights=(s, codes, mask))
    vals, meta = K.slim_pack(to_dev(codes), to_dev(mask))
    X, L, R = K.bf16_from_bits(ly.X), K.bf16_from_bits(ly.L), K.bf16_from_bits(ly.R)
    ws = K.new_workspace(b, d_out, d_in, r)
    outs = [K.slim_linear_fwd(X, vals, meta, s, L, R, workspace=ws, kernel=K.KERNEL_DECODE).clone()
            for _ in range(5)]
    torch.cuda.synchronize()
    for o in outs[1:]:
        assert torch.equal(o.view(torch.int16), outs[0].view(torch.int16))


def test_forward_argument_errors():
    X = torch.zeros((2, 256), dtype=torch.bfloat16, device="cuda")
    vals = torch.zeros((16, 64), dtype=torch.uint8, device="cuda")
    meta = torch.full((16, 32), 0x44, dtype=torch.uint8, device="cuda")
    tiny = torch.zeros(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(K.SlimError) as e:
        K.slim_linear_fwd(X, vals, meta, 1.0, None, None, workspace=tiny[:128])
    assert e.value.code == K.SLIM_ERR_WORKSPACE
    with pytest.raises(K.SlimError) as e:   # decode kernel forced on a batch it does not take
        K.slim_linear_fwd(torch.zeros((17, 256), dtype=torch.bfloat16, device="cuda"), vals, meta, 1.0, None, None,
                          kernel=K.KERNEL_DECODE)
    assert e.value.code == K.SLIM_ERR_UNSUPPORTED_SHAPE
    Y = K.slim_linear_fwd(X, vals, meta, 1.0, None, None)
    assert float(Y.float().abs().max()) == 0.0


def test_host_buffer_entry_point_matches_device_call():
    d_in, d_out, r, b = 1024, 256, 32, 16
    s, codes, mask, _, _ = cached_weights(d_out, d_in, 78)
    ly = inputs.make_layer(d_in, d_out, r, b, 78, weights=(s, codes, mask))
    vals, meta = K.slim_pack(to_dev(codes), to_dev(mask))
    L, R = K.bf16_from_bits(ly.L), K.bf16_from_bits(ly.R)
    Xh = K.bf16_from_bits(ly.X, device="cpu").pin_memory()
    Yh = torch.empty((b, d_out), dtype=torch.bfloat16).pin_memory()
    x_dev, y_dev = torch.empty_like(Xh, device="cuda"), torch.empty_like(Yh, device="cuda")
    ws = K.new_workspace(b, d_out, d_in, r)
    K.slim_linear_fwd_host(Xh, vals, meta, s, L, R, Yh, x_dev, y_dev, ws)
    Y = K.slim_linear_fwd(Xh.cuda(), vals, meta, s, L, R, workspace=ws)
    assert torch.equal(Yh.view(torch.int16), Y.cpu().view(torch.int16))


# ---- the five workload configurations at full size --------------------------
def full_cases(cfgs, max_b=16):
    out = []
    for cfg in cfgs:
        for name, d_in, d_out, r, b, seed, wseed in inputs.config_cases(cfg):
            if b <= max_b:
                out.append(pytest.param(d_in, d_out, r, b, seed, wseed, id=f"cfg{cfg}-{name}-b{b}-r{r}"))
    return out


@pytest.mark.parametrize("d_in,d_out,r,b,seed,wseed", full_cases([0, 1, 3, 4]))
def test_full_size_decode_configs(d_in, d_out, r, b, seed, wseed):
    """Batch 1-16 cases of configurations 0, 1, 3 and 4 in the launch the
    benchmark times (dispatcher's choice); all tokens compared."""
    assert K.slim_select_kernel(b, d_out, d_in, r) == K.KERNEL_DECODE
    assert_ok(run_case(d_in, d_out, r, b, seed, wseed))


def prefill_cases(cfgs):
    out = []
    for cfg in cfgs:
        for name, d_in, d_out, r, b, seed, wseed in inputs.config_cases(cfg):
            if b > 16:
                out.append(pytest.param(d_in, d_out, r, b, seed, wseed, id=f"cfg{cfg}-{name}-b{b}-r{r}"))
    return out


@pytest.mark.parametrize("d_in,d_out,r,b,seed,wseed", prefill_cases([2, 3, 4]))
def test_full_size_prefill_configs(d_in, d_out, r, b, seed, wseed):
    """2048- and 4096-token cases of configurations 2, 3 and 4 in the launch the
    dispatcher picks; compared on sampled token rows (first, middle and last
    rows of the edge tiles plus one seeded row in every other 128-token tile)."""
    assert K.slim_select_kernel(b, d_out, d_in, r) == K.KERNEL_PREFILL
    # every row of the first and of the last 128-token tile for the square attention layers (the oracle
    # needs a few seconds per 100 rows of the largest layers, so those keep three rows per edge tile)
    dense = d_in == d_out
    rows = inputs.sample_rows(b, tile=128, seed=seed, dense_edges=dense)
    res = run_case(d_in, d_out, r, b, seed, wseed, rows=rows)
    # the wide token tile is taken when it gives a quarter of the SMs or more an output tile (include/slim.h)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    assert res["token_tile"] == (256 if (d_out // 128) * ((b + 255) // 256) * 4 >= sms else 64)
    assert_ok(res)


def test_prefill_chain_replays_from_a_cuda_graph():
    """The prefill call's launches depend on one another programmatically (the main launch starts before the
    dense-only launch has ended): captured in a CUDA graph and replayed, the call gives the same bits."""
    d_in, d_out, r, b = 1024, 512, 64, 600
    s, codes, mask, ovals, ometa = cached_weights(d_out, d_in, 91)
    ly = inputs.make_layer(d_in, d_out, r, b, 91, weights=(s, codes, mask))
    vals, meta = binding.slim_pack(to_dev(codes), to_dev(mask))
    X, L, R = binding.bf16_from_bits(ly.X), binding.bf16_from_bits(ly.L), binding.bf16_from_bits(ly.R)
    ws = binding.new_workspace(b, d_out, d_in, r)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Y = torch.empty((b, d_out), dtype=torch.bfloat16, device="cuda")
    assert binding.slim_select_kernel(b, d_out, d_in, r) == binding.KERNEL_PREFILL
    binding.slim_linear_fwd(X, vals, meta, s, L, R, Y=Y, workspace=ws, status=status)
    torch.cuda.synchronize()
    direct = Y.clone()
    stream = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(g, stream=stream):
            binding.slim_linear_fwd(X, vals, meta, s, L, R, Y=Y, workspace=ws, status=status)
        for _ in range(3):
            Y.zero_()
            g.replay()
            stream.synchronize()
            assert torch.equal(Y.view(torch.int16), direct.view(torch.int16))
    assert binding.read_status(status) == 0
    res = parity.compare(inputs.bf16_bits_to_f64(binding.bits_from_bf16(direct)), oracle.linear_fwd(ly.X, ovals, ometa, s, ly.L, ly.R))
    assert res["ok"], res
