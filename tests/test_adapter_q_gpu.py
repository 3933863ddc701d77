"""Quantized adapters on the GPU (Sec. 3.3 of the paper): slim_pack_adapter byte for byte against the
oracle, slim_unpack_adapter against the values the storage stands for, and the layer forward on
quantized adapters against oracle.linear_fwd_q, all through the C-ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_09615_b200 import binding as K, inputs, parity
from helpers import cached_weights, to_dev

pytestmark = pytest.mark.gpu


def long_tailed(rows, cols, seed):
    rng = np.random.default_rng([seed, 7])
    a = rng.standard_t(3, (rows, cols)).astype(np.float32) * 0.02
    a[rng.random((rows, cols)) < 0.01] = 0.0
    return inputs.f32_to_bf16_bits(a)


@pytest.mark.parametrize("rows,cols,seed", [
    (1, 2, 1), (3, 16, 2), (5, 128, 3), (7, 144, 4), (16, 1000, 5), (33, 4096, 6), (416, 4096, 7), (4096, 416, 8),
    (832, 28672, 9),
])
def test_pack_adapter_is_bit_exact(rows, cols, seed):
    A = long_tailed(rows, cols, seed)
    if rows >= 3:
        A[1, :] = 0                                            # a row of all-zero groups
        A[2, : min(cols, 128)] = inputs.f32_to_bf16_bits(-np.abs(inputs.bf16_bits_to_f64(A[2, : min(cols, 128)])).astype(np.float32))
    codes, scales = K.slim_pack_adapter(K.bf16_from_bits(A))
    assert K.slim_last_launch_count() == 1
    ocodes, oscales = oracle.quant_adapter(A)
    assert np.array_equal(codes.cpu().numpy(), ocodes), "codes differ from the oracle's bytes"
    assert np.array_equal(K.bits_from_bf16(scales), oscales), "scales differ from the oracle's"
    assert codes.numel() == K.lib().slim_adapter_code_bytes(rows, cols)
    assert scales.numel() * 2 == K.lib().slim_adapter_scale_bytes(rows, cols)
    # the bf16 expansion is the stored value rounded once
    back = inputs.bf16_bits_to_f64(K.bits_from_bf16(K.slim_unpack_adapter(codes, scales)))
    want = oracle.dequant_adapter(ocodes, oscales)
    assert np.all(np.abs(back - want) <= np.abs(want) * 2.0 ** -8)
    exact = inputs.bf16_bits_to_f64(inputs.f32_to_bf16_bits(want.astype(np.float32)))
    assert np.array_equal(back, exact)


def test_unpack_adapter_decodes_every_nibble():
    codes = np.array([[0x10 * h + l for l in range(16)] for h in range(16)], np.uint8).reshape(2, 128)
    scales = inputs.f32_to_bf16_bits(np.array([[0.5, 2.0], [1.0, 0.25]], np.float32))
    got = K.slim_unpack_adapter(to_dev(codes), K.bf16_from_bits(scales))
    assert np.array_equal(inputs.bf16_bits_to_f64(K.bits_from_bf16(got)), oracle.dequant_adapter(codes, scales))


def run_q(d_in, d_out, r, b, seed, wseed=None, rows=None):
    wseed = seed if wseed is None else wseed
    s, codes, mask, ovals, ometa = cached_weights(d_out, d_in, wseed)
    ly = inputs.make_layer(d_in, d_out, r, b, seed, weights=(s, codes, mask))
    vals, meta = K.slim_pack(to_dev(codes), to_dev(mask))
    Lq, Ls = K.slim_pack_adapter(K.bf16_from_bits(ly.L))
    Rq, Rs = K.slim_pack_adapter(K.bf16_from_bits(ly.R))
    oLq, oLs = oracle.quant_adapter(ly.L)
    oRq, oRs = oracle.quant_adapter(ly.R)
    assert np.array_equal(Lq.cpu().numpy(), oLq) and np.array_equal(Rq.cpu().numpy(), oRq)
    assert np.array_equal(K.bits_from_bf16(Ls), oLs) and np.array_equal(K.bits_from_bf16(Rs), oRs)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(K.slim_workspace_bytes_q(b, d_out, d_in, r), dtype=torch.uint8, device="cuda")
    K.slim_workspace_reset(ws)
    X = K.bf16_from_bits(ly.X)
    Y = K.slim_linear_fwd_q(X, vals, meta, s, Lq, Ls, Rq, Rs, workspace=ws, status=status)
    launches = K.slim_last_launch_count()
    Y2 = K.slim_linear_fwd_q(X, vals, meta, s, Lq, Ls, Rq, Rs, workspace=ws, status=status)
    torch.cuda.synchronize()
    assert K.read_status(status) == 0 and torch.equal(Y2.view(torch.int16), Y.view(torch.int16))
    y = inputs.bf16_bits_to_f64(K.bits_from_bf16(Y))
    if rows is not None:
        y = y[np.asarray(rows)]
    res = parity.compare(y, oracle.linear_fwd_q(ly.X, ovals, ometa, s, oLq, oLs, oRq, oRs, rows=rows))
    res["launches"] = launches
    return res


@pytest.mark.parametrize("d_in,d_out,r,b", [
    # decode kernel reading codes and scales as they are: short last group, two chunk widths, several
    # k-slices, both token-tile counts; ranks whose rows of L codes are no 16-byte multiples (plain loads)
    (256, 64, 32, 1), (512, 512, 64, 8), (768, 208, 96, 16), (1024, 384, 160, 5), (2304, 128, 416, 16), (4352, 96, 544, 3),
    (1280, 1040, 1056, 9),
    (256, 64, 16, 1), (768, 208, 48, 16), (1024, 384, 144, 5), (8192, 1024, 112, 16), (2048, 160, 1040, 2),
    # adapters expanded first: CUDA-core kernel, prefill kernel
    (320, 48, 32, 3),
    (512, 256, 64, 200), (640, 384, 144, 70),
])
def test_forward_on_quantized_adapters_small(d_in, d_out, r, b):
    res = run_q(d_in, d_out, r, b, seed=300 + r + b)
    assert res["ok"], res
    fused = b <= 16 and d_in % 256 == 0
    assert res["launches"] == 1 if fused else res["launches"] >= 3      # else two expansions and the forward launches


def test_quantized_adapter_codes_reach_the_right_rows_and_columns():
    """One non-zero code at a time in R and in L (scales a power of two): the output is one product, exactly."""
    d_in, d_out, r, b = 1024, 64, 160, 4
    s, codes, mask, ovals, ometa = cached_weights(d_out, d_in, 77)
    vals, meta = K.slim_pack(to_dev(codes), to_dev(mask))
    rng = np.random.default_rng(77)
    X = inputs.f32_to_bf16_bits(rng.integers(-3, 4, (b, d_in)).astype(np.float32))
    for (j, k, n) in [(0, 0, 0), (159, 1023, 63), (37, 515, 9), (128, 300, 40), (95, 64, 17)]:
        R = np.zeros((r, d_in), np.float32); L = np.zeros((d_out, r), np.float32)
        R[j, k] = -1.75                  # code -7 at scale 0.25
        L[n, j] = 3.5                    # code 7 at scale 0.5
        Rq, Rs = K.slim_pack_adapter(K.bf16_from_bits(inputs.f32_to_bf16_bits(R)))
        Lq, Ls = K.slim_pack_adapter(K.bf16_from_bits(inputs.f32_to_bf16_bits(L)))
        Y = K.slim_linear_fwd_q(K.bf16_from_bits(X), vals, meta, 0.0, Lq, Ls, Rq, Rs)
        assert K.slim_last_launch_count() == 1
        y = inputs.bf16_bits_to_f64(K.bits_from_bf16(Y))
        want = np.zeros((b, d_out)); want[:, n] = inputs.bf16_bits_to_f64(X)[:, k] * -1.75 * 3.5
        assert np.array_equal(y, want), (j, k, n)


def full_q_cases():
    out = []
    for cfg in (1, 3, 4):
        for name, d_in, d_out, r, b, seed, wseed in inputs.config_cases(cfg):
            if b == 16 and r > 0 and abs(r - inputs.rank_for_ratio(0.1, d_in, d_out)) == 0:
                out.append(pytest.param(d_in, d_out, r, b, seed, wseed, id=f"cfg{cfg}-{name}-b{b}-r{r}"))
    return out


@pytest.mark.parametrize("d_in,d_out,r,b,seed,wseed", full_q_cases())
def test_forward_on_quantized_adapters_full_size(d_in, d_out, r, b, seed, wseed):
    assert run_q(d_in, d_out, r, b, seed, wseed)["ok"]


def test_forward_on_quantized_adapters_prefill_full_size():
    d_in, d_out, r, b = 4096, 4096, 416, 2048
    rows = inputs.sample_rows(b, tile=128, seed=5, dense_edges=False)
    res = run_q(d_in, d_out, r, b, seed=1000, wseed=1000, rows=rows)
    assert res["ok"], res


def test_quantized_adapter_argument_errors():
    A = torch.zeros((4, 7), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(K.SlimError):
        K.slim_pack_adapter(A)
    assert K.slim_workspace_bytes_q(4, 64, 256, 0) == 0
    s, codes, mask, ovals, ometa = cached_weights(64, 256, 1)
    vals, meta = K.slim_pack(to_dev(codes), to_dev(mask))
    L = torch.zeros((64, 16), dtype=torch.bfloat16, device="cuda")
    R = torch.zeros((16, 256), dtype=torch.bfloat16, device="cuda")
    Lq, Ls = K.slim_pack_adapter(L)
    Rq, Rs = K.slim_pack_adapter(R)
    X = torch.zeros((2, 256), dtype=torch.bfloat16, device="cuda")
    small = K.new_workspace(2, 64, 256, 16)                       # the ordinary size: too small for the expansion
    with pytest.raises(K.SlimError) as e:
        K.slim_linear_fwd_q(X, vals, meta, s, Lq, Ls, Rq, Rs, workspace=small)
    assert e.value.code == K.SLIM_ERR_WORKSPACE
    Y = K.slim_linear_fwd_q(X, vals, meta, s, Lq, Ls, Rq, Rs)     # zero adapters, zero activations
    assert not Y.float().abs().any()
