"""SLiM-Quant on the GPU (Sec. 3.1, Algorithm 1 of the paper): slim_quant against oracle.slim_quant, bit for
bit (codes, scale, alpha*, the table of candidates and their errors), through the C-ABI; and the
step in its place: float32 weights -> slim_quant -> top-2 mask -> slim_pack -> slim_linear_fwd."""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_09615_b200 import binding as K, inputs, parity
from helpers import to_dev

pytestmark = pytest.mark.gpu


def weights(kind, shape, seed):
    rng = np.random.default_rng([seed, 11])
    if kind == "normal":
        w = rng.standard_normal(shape)
    elif kind == "laplace":
        w = rng.laplace(size=shape)
    elif kind == "student":
        w = rng.standard_t(4, shape)
    else:
        w = rng.uniform(-1, 1, shape)
    return (w * 0.02).astype(np.float32)


@pytest.mark.parametrize("kind,shape,seed", [
    ("normal", (16, 32), 1),                 # 512 bins, hardly any weights
    ("laplace", (300, 400), 2),
    ("student", (700, 900), 3),              # 630 bins
    ("uniform", (512, 512), 4),              # no clipping pays: alpha* near M
    ("normal", (4096, 4096), 5),             # 16777 bins
    ("normal", (4096, 11008), 6),            # the cap of 20000 bins
])
def test_slim_quant_matches_the_oracle_bit_for_bit(kind, shape, seed):
    W = weights(kind, shape, seed)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    codes, sa, table, alpha = K.slim_quant(to_dev(W), status=status)
    assert K.slim_last_launch_count() == 4
    torch.cuda.synchronize()
    assert K.read_status(status) == 0
    ocodes, oscale, oalpha, otable = oracle.slim_quant(W)
    assert float(alpha) == oalpha
    assert np.array_equal(table.cpu().numpy().view(np.uint64), otable.view(np.uint64)), "candidate table differs"
    s, a32 = sa.cpu().numpy()
    assert s == oscale and a32 == np.float32(oalpha)
    assert np.array_equal(codes.cpu().numpy(), ocodes)


def test_slim_quant_degenerate_inputs():
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    codes, sa, table, alpha = K.slim_quant(torch.zeros((8, 64), dtype=torch.float32, device="cuda"), status=status)
    torch.cuda.synchronize()
    assert not codes.any() and sa[0] == 0 and float(alpha) == 0 and K.read_status(status) == 0
    W = torch.ones((8, 64), dtype=torch.float32, device="cuda")
    W[3, 5] = float("nan")
    codes, sa, table, alpha = K.slim_quant(W, status=status)
    torch.cuda.synchronize()
    assert K.read_status(status) & (1 << K.SLIM_ERR_INVALID_ARG) and sa[0] == 0 and not codes.any()
    assert K.lib().slim_quant(None, 8, 64, None, None, None, 0, None, None) == K.SLIM_ERR_INVALID_ARG


def test_quantize_then_pack_then_forward():
    """The producer in its place: float32 weights -> SLiM-Quant codes and scale -> magnitude 2:4 mask ->
    slim_pack -> the layer, against the oracle fed with the oracle's own quantization."""
    d_in, d_out, r, b = 1024, 256, 32, 8
    W = weights("normal", (d_out, d_in), 21)
    codes, sa, _, _ = K.slim_quant(to_dev(W))
    s = float(sa[0])
    ocodes, oscale, _, _ = oracle.slim_quant(W)
    assert s == float(oscale) and np.array_equal(codes.cpu().numpy(), ocodes)
    rng = np.random.default_rng(21)
    xbar = (np.abs(rng.standard_normal(d_in)) + 0.1).astype(np.float32)          # synthetic average input magnitudes
    mask_d = K.slim_mask_top2(codes, to_dev(xbar))
    mask = oracle.mask_top2(ocodes, xbar)
    assert np.array_equal(mask_d.cpu().numpy(), mask)
    vals, meta = K.slim_pack(codes, mask_d)
    ovals, ometa = oracle.pack(ocodes, mask)
    assert np.array_equal(vals.cpu().numpy(), ovals) and np.array_equal(meta.cpu().numpy(), ometa)
    L, R = inputs.make_adapters(d_out, d_in, r, 21)
    X = inputs.make_activations(b, d_in, 21)
    Y = K.slim_linear_fwd(K.bf16_from_bits(X), vals, meta, s, K.bf16_from_bits(L), K.bf16_from_bits(R))
    res = parity.compare(inputs.bf16_bits_to_f64(K.bits_from_bf16(Y)), oracle.linear_fwd(X, ovals, ometa, oscale, L, R))
    assert res["ok"], res


@pytest.mark.parametrize("d_out,d_in,seed,with_x", [(3, 8, 1, False), (64, 1000, 2, True), (4096, 4096, 3, True), (1000, 11008, 4, False)])
def test_mask_top2_is_bit_exact(d_out, d_in, seed, with_x):
    rng = np.random.default_rng([seed, 13])
    codes = rng.integers(-8, 8, (d_out, d_in)).astype(np.int8)
    xbar = rng.random(d_in).astype(np.float32) if with_x else None
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = K.slim_mask_top2(to_dev(codes), None if xbar is None else to_dev(xbar), status=status)
    assert K.slim_last_launch_count() == 1
    assert np.array_equal(got.cpu().numpy(), oracle.mask_top2(codes, xbar))
    assert K.read_status(status) == 0
    if with_x:
        bad = xbar.copy(); bad[5] = -1.0
        K.slim_mask_top2(to_dev(codes), to_dev(bad), status=status)
        torch.cuda.synchronize()
        assert K.read_status(status) & (1 << K.SLIM_ERR_INVALID_ARG)
