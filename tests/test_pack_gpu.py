"""slim_pack / slim_unpack against the oracle: byte-identical."""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_09615_b200 import binding, inputs
from helpers import to_dev

pytestmark = pytest.mark.gpu


def random_codes_mask(rng, d_out, d_in):
    """Groups with 0, 1 and 2 kept positions, codes over the full [-8, 7] range."""
    codes = rng.integers(-8, 8, size=(d_out, d_in)).astype(np.int8)
    pri = rng.random((d_out, d_in // 4, 4))
    kept = rng.integers(0, 3, size=(d_out, d_in // 4, 1))
    rank = np.argsort(np.argsort(pri, -1), -1)
    mask = (rank < kept).astype(np.uint8).reshape(d_out, d_in)
    return codes, mask


@pytest.mark.parametrize("d_out,d_in", [(16, 64), (48, 192), (512, 512), (1040, 2112)])
def test_pack_random_bit_exact(d_out, d_in):
    rng = np.random.default_rng(d_out + d_in)
    codes, mask = random_codes_mask(rng, d_out, d_in)
    # garbage at pruned positions must be ignored
    codes = np.where(mask > 0, codes, rng.integers(-128, 128, size=codes.shape)).astype(np.int8)
    ovals, ometa = oracle.pack(codes, mask)
    vals, meta = binding.slim_pack(to_dev(codes), to_dev(mask))
    assert np.array_equal(vals.cpu().numpy(), ovals)
    assert np.array_equal(meta.cpu().numpy(), ometa)
    c2, m2 = binding.slim_unpack(vals, meta)
    oc, om = oracle.unpack(ovals, ometa)
    assert np.array_equal(c2.cpu().numpy(), oc)
    assert np.array_equal(m2.cpu().numpy(), om)
    c3, none = binding.slim_unpack(vals, meta, want_mask=False)
    assert none is None and torch.equal(c3, c2)


def test_pack_generated_layer_bit_exact():
    ly = inputs.make_layer(4096, 4096, 0, 1, seed=1000)
    ovals, ometa = oracle.pack(ly.codes, ly.mask)
    vals, meta = binding.slim_pack(to_dev(ly.codes), to_dev(ly.mask))
    assert np.array_equal(vals.cpu().numpy(), ovals)
    assert np.array_equal(meta.cpu().numpy(), ometa)


def test_pack_flags_bad_groups_without_trapping():
    codes = np.zeros((16, 64), np.int8)
    mask = np.zeros((16, 64), np.uint8)
    mask[3, 8:11] = 1                     # three kept in one group
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    vals, meta = binding.slim_pack(to_dev(codes), to_dev(mask), status=status, check=False)
    assert binding.read_status(status) == 1 << binding.SLIM_ERR_BAD_MASK
    assert int(vals.sum()) == 0 and bool((meta == 0x44).all())
    with pytest.raises(binding.SlimError) as e:
        binding.slim_pack(to_dev(codes), to_dev(mask))
    assert e.value.code == binding.SLIM_ERR_BAD_MASK
    mask[:] = 0
    mask[5, 1] = 1
    codes[5, 1] = 8                       # out of range at a kept position
    with pytest.raises(binding.SlimError) as e:
        binding.slim_pack(to_dev(codes), to_dev(mask))
    assert e.value.code == binding.SLIM_ERR_CODE_RANGE
    # the context is still usable
    mask[:] = 0
    vals, meta = binding.slim_pack(to_dev(codes), to_dev(mask))
    assert int(vals.sum()) == 0


def test_pack_rejects_bad_arguments():
    good = torch.zeros((16, 64), dtype=torch.int8, device="cuda")
    with pytest.raises(binding.SlimError) as e:
        binding.slim_pack(torch.zeros((16, 32), dtype=torch.int8, device="cuda"),
                          torch.zeros((16, 32), dtype=torch.uint8, device="cuda"))
    assert e.value.code == binding.SLIM_ERR_UNSUPPORTED_SHAPE
    with pytest.raises(TypeError):
        binding.slim_pack(good, good)     # mask has the wrong dtype
