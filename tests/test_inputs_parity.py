"""Host logic: the seeded generator recipe and the acceptance rule."""
import numpy as np

from paper_2410_09615_b200 import inputs, parity


def test_bf16_rounding_is_nearest_even():
    # 1 + 2^-8 is halfway between two bf16 values -> rounds to even (1.0);
    # 1 + 3*2^-8 is halfway -> rounds up to 1 + 2^-6
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -2.5, 0.0], np.float32)
    bits = inputs.f32_to_bf16_bits(x)
    assert bits.tolist() == [0x3F80, 0x3F80, 0x3F82, 0xC020, 0x0000]
    assert inputs.bf16_bits_to_f64(bits).tolist() == [1.0, 1.0, 1.015625, -2.5, 0.0]


def test_ranks_follow_the_config_rule():
    assert inputs.default_rank(4096, 4096) == 416
    assert inputs.default_rank(4096, 11008) == 416
    assert inputs.default_rank(5120, 13824) == 512
    assert inputs.default_rank(8192, 1024) == 112
    assert inputs.default_rank(8192, 28672) == 832
    assert [inputs.rank_for_ratio(x, 8192, 28672) for x in (0, 0.05, 0.1, 0.2)] == [0, 416, 832, 1648]
    assert [inputs.rank_for_ratio(x, 8192, 1024) for x in (0, 0.05, 0.1, 0.2)] == [0, 64, 112, 208]


def test_layer_recipe():
    ly = inputs.make_layer(512, 512, 64, 8, seed=0)
    again = inputs.make_layer(512, 512, 64, 8, seed=0)
    assert (ly.codes == again.codes).all() and (ly.X == again.X).all() and ly.s == again.s
    assert ly.codes.dtype == np.int8 and ly.codes.min() >= -7 and ly.codes.max() <= 7
    assert (ly.mask.reshape(512, 128, 4).sum(-1) == 2).all()
    assert ly.L.shape == (512, 64) and ly.R.shape == (64, 512) and ly.X.shape == (8, 512)
    assert abs(inputs.bf16_bits_to_f64(ly.X).std() - 1.0) < 0.05
    assert abs(inputs.bf16_bits_to_f64(ly.L).std() - 0.02) < 0.002


def test_top2_mask_ties_take_lower_index():
    W = np.array([[1, 1, 1, 1, 0.5, -2, 2, 0.1]], np.float32)
    assert inputs.top2_mask(W).tolist() == [[1, 1, 0, 0, 0, 1, 1, 0]]


def test_config_table_covers_all_five():
    n = {c: len(list(inputs.config_cases(c))) for c in range(5)}
    assert n == {0: 1, 1: 6, 2: 3, 3: 9, 4: 48}
    assert ("single", 512, 512, 64, 8, 0, 0) in list(inputs.config_cases(0))


def test_sample_rows():
    rows = inputs.sample_rows(2048)
    assert rows[0] == 0 and rows[-1] == 2047 and len(set(rows.tolist())) == len(rows)
    assert set(range(128)) <= set(rows.tolist()) and set(range(1920, 2048)) <= set(rows.tolist())
    tiles = set((rows // 128).tolist())
    assert tiles == set(range(16))
    assert inputs.sample_rows(16).tolist() == list(range(16))
    few = inputs.sample_rows(4096, dense_edges=False)
    assert few[0] == 0 and few[-1] == 4095 and len(few) < 40
    assert set((few // 128).tolist()) == set(range(32))


def test_parity_rule():
    ref = np.array([[1.0, -2.0], [0.0, 4.0]])
    rms = np.sqrt((1 + 4 + 0 + 16) / 4)
    assert parity.compare(ref, ref)["ok"]
    ok = ref.copy()
    ok[1, 0] = 0.009 * rms            # inside 1e-2*rms at a zero reference
    assert parity.compare(ok, ref)["ok"]
    bad = ref.copy()
    bad[1, 0] = 0.011 * rms
    res = parity.compare(bad, ref)
    assert not res["ok"] and tuple(res["worst_index"]) == (1, 0)
    # a uniform 2 % error fails the Frobenius bound even if element-wise terms were loose
    assert not parity.compare(ref * 1.02, ref)["ok"]
    nan = ref.copy()
    nan[0, 0] = np.nan
    assert not parity.compare(nan, ref)["ok"]
