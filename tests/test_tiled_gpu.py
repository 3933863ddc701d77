"""The decode-tiled path: slim_repack_tiled byte for byte against the oracle's layout, and
slim_linear_fwd_tiled against the oracle's forward, element by element (small and ragged cases,
every batch size, the workload configurations at full size, workspace sharing)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_09615_b200 import binding, inputs, parity
from helpers import cached_weights, to_dev

pytestmark = pytest.mark.gpu

K = binding


def run_tiled(d_in, d_out, r, b, seed, wseed=None, check_repack=True, ws=None):
    """One case through slim_pack -> slim_repack_tiled -> slim_linear_fwd_tiled, compared with the oracle."""
    wseed = seed if wseed is None else wseed
    s, codes, mask, ovals, ometa = cached_weights(d_out, d_in, wseed)
    ly = inputs.make_layer(d_in, d_out, r, b, seed, weights=(s, codes, mask))
    vals, meta = K.slim_pack(to_dev(codes), to_dev(mask))
    tiled = K.slim_repack_tiled(vals, meta)
    assert K.slim_last_launch_count() == 1
    if check_repack:
        assert np.array_equal(tiled.cpu().numpy(), oracle.repack_tiled(ovals, ometa)), "tiled bytes differ from the oracle's"
    X = K.bf16_from_bits(ly.X)
    L = K.bf16_from_bits(ly.L) if r else None
    R = K.bf16_from_bits(ly.R) if r else None
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    if ws is None:
        ws = K.new_workspace(b, d_out, d_in, r)
    Y = K.slim_linear_fwd_tiled(X, tiled, d_out, s, L, R, workspace=ws, status=status)
    assert K.slim_last_launch_count() == 1
    torch.cuda.synchronize()
    assert K.read_status(status) == 0, f"device status {K.read_status(status):#x}"
    # the workspace is left ready for the next call: same inputs, same bits
    Y2 = K.slim_linear_fwd_tiled(X, tiled, d_out, s, L, R, workspace=ws, status=status)
    torch.cuda.synchronize()
    assert K.read_status(status) == 0 and torch.equal(Y2.view(torch.int16), Y.view(torch.int16))
    y_ref = oracle.linear_fwd(ly.X, ovals, ometa, s, ly.L, ly.R)
    return parity.compare(inputs.bf16_bits_to_f64(K.bits_from_bf16(Y)), y_ref)


SMALL = [  # d_in, d_out, r, b
    (512, 512, 64, 8),       # configuration 0
    (256, 16, 0, 1),         # one tile, one block, no adapters
    (256, 16, 16, 1),
    (768, 48, 16, 3),        # ragged batch, three blocks
    (2304, 272, 112, 13),    # nine blocks, ragged rank (one adapter slot, mostly past r), 17 row tiles
    (4352, 1040, 208, 16),   # 17 blocks: two k-slices at batch 16; 65 row tiles
    (1024, 4096, 48, 9),
    (256, 2064, 400, 5),     # many row tiles on one block; four adapter slots, the last one ragged
]


@pytest.mark.parametrize("d_in,d_out,r,b", SMALL)
def test_small_tiled(d_in, d_out, r, b):
    res = run_tiled(d_in, d_out, r, b, seed=41)
    assert res["ok"], res


@pytest.mark.parametrize("b", list(range(1, 17)))
def test_tiled_every_batch_size(b):
    res = run_tiled(1024, 256, 32, b, seed=60 + b, wseed=60)
    assert res["ok"], res


@pytest.mark.parametrize("d_in,d_out,r,b", [(9472, 4096, 64, 16), (9472, 4096, 64, 8), (1536, 16384, 0, 16)])
def test_tiled_wide_slots(d_in, d_out, r, b):
    """Shapes large enough for the plans that put two and four row tiles in a weight slot, small
    enough for the oracle to check every element (9472 columns: 37 blocks, several k-slices at batch 16)."""
    res = run_tiled(d_in, d_out, r, b, seed=43)
    assert res["ok"], res


def test_tiled_integer_inputs_are_exact():
    """Integer-valued activations, adapters and codes over the whole range [-8, 7], s = 1: every
    partial sum is an integer below 2^24 and |Y| <= 256, so the result must equal int64 arithmetic."""
    rng = np.random.default_rng(44)
    d_in, d_out, r, b = 512, 96, 16, 11
    codes = rng.integers(-8, 8, size=(d_out, d_in)).astype(np.int8)
    mask = inputs.top2_mask(rng.standard_normal((d_out, d_in)).astype(np.float32))
    Xi = rng.integers(-1, 2, size=(b, d_in))
    Li = rng.integers(-1, 2, size=(d_out, r))
    Ri = (rng.random((r, d_in)) < 0.05).astype(np.int64) * rng.integers(-1, 2, size=(r, d_in))
    bf = lambda a: inputs.f32_to_bf16_bits(np.asarray(a, np.float32))
    vals, meta = K.slim_pack(to_dev(codes), to_dev(mask))
    tiled = K.slim_repack_tiled(vals, meta)
    Y = K.slim_linear_fwd_tiled(K.bf16_from_bits(bf(Xi)), tiled, d_out, 1.0, K.bf16_from_bits(bf(Li)), K.bf16_from_bits(bf(Ri)))
    exact = Xi @ (codes.astype(np.int64) * mask).T + (Xi @ Ri.T) @ Li.T
    assert np.abs(exact).max() <= 256
    assert np.array_equal(inputs.bf16_bits_to_f64(K.bits_from_bf16(Y)), exact.astype(np.float64))


def test_tiled_one_hot_activations_read_back_single_columns():
    rng = np.random.default_rng(45)
    d_in, d_out = 768, 64
    codes = rng.integers(-8, 8, size=(d_out, d_in)).astype(np.int8)
    mask = inputs.top2_mask(rng.standard_normal((d_out, d_in)).astype(np.float32))
    vals, meta = K.slim_pack(to_dev(codes), to_dev(mask))
    tiled = K.slim_repack_tiled(vals, meta)
    for b, ks in [(16, rng.choice(d_in, 16, replace=False)), (7, np.array([0, 3, 255, 256, 511, 700, 767]))]:
        X = np.zeros((b, d_in), np.float32)
        X[np.arange(b), ks] = 1.0
        Y = K.slim_linear_fwd_tiled(K.bf16_from_bits(inputs.f32_to_bf16_bits(X)), tiled, d_out, 0.5, None, None)
        got = inputs.bf16_bits_to_f64(K.bits_from_bf16(Y))
        want = 0.5 * (codes.astype(np.float64) * mask)[:, ks].T
        assert np.array_equal(got, want)


def test_tiled_zero_scale_and_zero_rank():
    res = run_tiled(512, 64, 0, 4, seed=46)
    assert res["ok"], res
    s, codes, mask, ovals, ometa = cached_weights(64, 512, 46)
    ly = inputs.make_layer(512, 64, 32, 4, 46, weights=(s, codes, mask))
    vals, meta = K.slim_pack(to_dev(codes), to_dev(mask))
    tiled = K.slim_repack_tiled(vals, meta)
    Y = K.slim_linear_fwd_tiled(K.bf16_from_bits(ly.X), tiled, 64, 0.0, K.bf16_from_bits(ly.L), K.bf16_from_bits(ly.R))
    y_ref = oracle.linear_fwd(ly.X, ovals, ometa, 0.0, ly.L, ly.R)
    assert parity.compare(inputs.bf16_bits_to_f64(K.bits_from_bf16(Y)), y_ref)["ok"]


@pytest.mark.parametrize("d_in,d_out,r,b", [
    (8192, 8192, 1648, 16),     # two ring slots per warp, four k-slices
    (8192, 8192, 832, 16),
    (4096, 11008, 416, 3),
    (8192, 1024, 112, 16),
    (2048, 2064, 3072, 16),     # the largest rank
])
def test_tiled_calls_repeat_bit_for_bit(d_in, d_out, r, b):
    """Every partial sum is added in list order, so a call's bits do not depend on which warp was
    first: forty calls back to back on one workspace (random weight bytes, nothing to compare but
    the calls with one another) give one result."""
    g = torch.Generator(device="cuda")
    g.manual_seed(5)
    tiled = torch.randint(0, 256, (K.slim_tiled_bytes(d_out, d_in),), dtype=torch.uint8, device="cuda", generator=g)
    tiled.view(-1, 1536)[:, 1024:] = 0x44        # index bytes must name two different positions per group
    L = torch.randn(d_out, r, device="cuda", generator=g).mul_(0.02).bfloat16()
    R = torch.randn(r, d_in, device="cuda", generator=g).mul_(0.02).bfloat16()
    X = torch.randn(b, d_in, device="cuda", generator=g).bfloat16()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = K.new_workspace(b, d_out, d_in, r)
    first = K.slim_linear_fwd_tiled(X, tiled, d_out, 0.01, L, R, workspace=ws, status=status).clone()
    assert torch.isfinite(first.float()).all()
    differ = 0
    for _ in range(40):
        Y = K.slim_linear_fwd_tiled(X, tiled, d_out, 0.01, L, R, workspace=ws, status=status)
        differ += int(not torch.equal(Y.view(torch.int16), first.view(torch.int16)))
    torch.cuda.synchronize()
    assert K.read_status(status) == 0 and differ == 0, (differ, K.read_status(status))


def test_one_workspace_serves_every_kernel_and_shape_in_turn():
    """Decode calls of different shapes and batch sizes (both tiled and packed-format kernels), a
    prefill call and a CUDA-core call share one workspace; every result is checked against the
    oracle.  A kernel that left the hand-over slots of another in a used state would show here."""
    shapes = [(1024, 256, 32, 16), (768, 48, 16, 3), (2304, 272, 112, 13), (512, 512, 0, 1), (4352, 1040, 208, 9)]
    big = max(K.slim_workspace_bytes(b, d_out, d_in, r) for d_in, d_out, r, b in shapes)
    big = max(big, K.slim_workspace_bytes(300, 256, 512, 112), K.slim_workspace_bytes(50, 128, 704, 32))
    ws = torch.empty(big, dtype=torch.uint8, device="cuda")
    K.slim_workspace_reset(ws)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def packed_call(d_in, d_out, r, b, seed, kernel):
        s, codes, mask, ovals, ometa = cached_weights(d_out, d_in, seed)
        ly = inputs.make_layer(d_in, d_out, r, b, seed, weights=(s, codes, mask))
        vals, meta = K.slim_pack(to_dev(codes), to_dev(mask))
        L = K.bf16_from_bits(ly.L) if r else None
        R = K.bf16_from_bits(ly.R) if r else None
        Y = K.slim_linear_fwd(K.bf16_from_bits(ly.X), vals, meta, s, L, R, workspace=ws, status=status, kernel=kernel)
        torch.cuda.synchronize()
        assert K.read_status(status) == 0
        y_ref = oracle.linear_fwd(ly.X, ovals, ometa, s, ly.L, ly.R)
        res = parity.compare(inputs.bf16_bits_to_f64(K.bits_from_bf16(Y)), y_ref)
        assert res["ok"], (d_in, d_out, r, b, kernel, res)

    for rnd in range(2):
        for i, (d_in, d_out, r, b) in enumerate(shapes):
            res = run_tiled(d_in, d_out, r, b, seed=70 + i, ws=ws, check_repack=False)
            assert res["ok"], (rnd, d_in, d_out, r, b, res)
            packed_call(d_in, d_out, r, b, 70 + i, K.KERNEL_DECODE)
        packed_call(512, 256, 112, 300, 80, K.KERNEL_PREFILL)      # writes T' where the decode slots live
        packed_call(704, 128, 32, 50, 81, K.KERNEL_SIMPLE)         # writes T (fp32) there


def test_tiled_argument_errors():
    X = torch.zeros((2, 256), dtype=torch.bfloat16, device="cuda")
    tiled = torch.zeros(K.slim_tiled_bytes(16, 256), dtype=torch.uint8, device="cuda")
    lib = K.lib()
    ws = K.new_workspace(2, 16, 256, 0)
    P = lambda t: t.data_ptr()
    Y = torch.empty((2, 16), dtype=torch.bfloat16, device="cuda")
    call = lambda b, layout, s, d_out, d_in, wsz: lib.slim_linear_fwd_tiled(P(X), b, P(tiled), layout, s, None, None, 0, d_out, d_in,
                                                                             P(Y), P(ws), wsz, None, None)
    assert call(2, K.LAYOUT_DECODE_TILED, 1.0, 16, 256, ws.numel()) == K.SLIM_OK
    assert call(17, K.LAYOUT_DECODE_TILED, 1.0, 16, 256, ws.numel()) == K.SLIM_ERR_UNSUPPORTED_SHAPE
    assert call(2, 7, 1.0, 16, 256, ws.numel()) == K.SLIM_ERR_UNSUPPORTED_SHAPE
    assert call(2, K.LAYOUT_DECODE_TILED, float("nan"), 16, 256, ws.numel()) == K.SLIM_ERR_INVALID_ARG
    assert call(2, K.LAYOUT_DECODE_TILED, 1.0, 16, 320, ws.numel()) == K.SLIM_ERR_UNSUPPORTED_SHAPE
    assert call(2, K.LAYOUT_DECODE_TILED, 1.0, 16, 256, 128) == K.SLIM_ERR_WORKSPACE
    torch.cuda.synchronize()


def full_cases(cfgs):
    out = []
    for cfg in cfgs:
        for name, d_in, d_out, r, b, seed, wseed in inputs.config_cases(cfg):
            if b <= 16:
                out.append(pytest.param(d_in, d_out, r, b, seed, wseed, id=f"cfg{cfg}-{name}-b{b}-r{r}"))
    return out


@pytest.mark.parametrize("d_in,d_out,r,b,seed,wseed", full_cases([0, 1, 3, 4]))
def test_full_size_tiled_decode_configs(d_in, d_out, r, b, seed, wseed):
    """Batch 1-16 cases of configurations 0, 1, 3 and 4 at full size through the tiled path (the launch
    the benchmark times); all tokens and all output columns compared."""
    res = run_tiled(d_in, d_out, r, b, seed, wseed, check_repack=(d_out * d_in <= 5120 * 13824))
    assert res["ok"], res


def test_layout_hint_follows_the_stated_rule():
    """Tiled when the packed weight has 64 MiB or more and b <= 4 (b <= 2 when d_out < d_in); packed otherwise."""
    T = K.LAYOUT_DECODE_TILED
    assert K.slim_decode_layout_hint(1, 28672, 8192, 832) == T
    assert K.slim_decode_layout_hint(4, 28672, 8192, 832) == T
    assert K.slim_decode_layout_hint(5, 28672, 8192, 832) == 0
    assert K.slim_decode_layout_hint(2, 8192, 28672, 832) == T
    assert K.slim_decode_layout_hint(4, 8192, 28672, 832) == 0
    assert K.slim_decode_layout_hint(16, 28672, 8192, 832) == 0
    assert K.slim_decode_layout_hint(1, 8192, 8192, 832) == 0          # 24 MiB of packed weight
    assert K.slim_decode_layout_hint(1, 28672, 8192, 8) == 0           # not a legal rank
    assert K.slim_decode_layout_hint(0, 28672, 8192, 832) == 0
