"""Pins for the CPU oracle: every expected value here comes from outside
oracle/ (hand arithmetic, numpy's own float64 matmul, integer arithmetic, the
paper's printed table, invariants)."""
import os

import numpy as np
import pytest

import oracle
from paper_2410_09615_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf(x):
    return inputs.f32_to_bf16_bits(np.asarray(x, np.float32))


# ---------------------------------------------------------------- P4: by hand
HAND_CODES = np.array([[3, -2, 0, 5, -8, 7, 1, 0],
                       [-1, -8, 4, 2, 6, 0, 0, -3]], np.int8)
HAND_MASK = np.array([[1, 0, 0, 1, 0, 1, 1, 0],
                      [0, 1, 1, 0, 0, 0, 0, 1]], np.uint8)


def test_pack_bytes_by_hand():
    vals, meta = oracle.pack(HAND_CODES, HAND_MASK)
    # row 0: group 0 keeps positions (0,3) codes (3,5)   -> 0x53, index nibble 0|3<<2 = 0xC
    #        group 1 keeps positions (1,2) codes (7,1)   -> 0x17, index nibble 1|2<<2 = 0x9
    # row 1: group 0 keeps positions (1,2) codes (-8,4)  -> 0x48, 0x9
    #        group 1 keeps only position 3 (code -3): completed with position 0 (value 0)
    #                 -> positions (0,3) codes (0,-3)    -> 0xD0, 0xC
    assert vals.tolist() == [[0x53, 0x17], [0x48, 0xD0]]
    assert meta.tolist() == [[0x9C], [0xC9]]


def test_unpack_by_hand():
    vals = np.array([[0x53, 0x17], [0x48, 0xD0]], np.uint8)
    meta = np.array([[0x9C], [0xC9]], np.uint8)
    codes, mask = oracle.unpack(vals, meta)
    assert codes.tolist() == [[3, 0, 0, 5, 0, 7, 1, 0], [0, -8, 4, 0, 0, 0, 0, -3]]
    assert mask.tolist() == [[1, 0, 0, 1, 0, 1, 1, 0], [0, 1, 1, 0, 1, 0, 0, 1]]


def test_forward_by_hand():
    vals, meta = oracle.pack(HAND_CODES, HAND_MASK)
    X = bf([[1, 2, -1, 0.5, 3, -2, 4, 1]])
    R = bf([[0.5, 0, 0, 1, 0, 0, 0.25, 2]])
    L = bf([[1.5], [-0.5]])
    # row 0 of the kept weight: [3,0,0,5,0,7,1,0] . x = 3 + 2.5 - 14 + 4 = -4.5 ; * 0.5 = -2.25
    # row 1:                    [0,-8,4,0,0,0,0,-3] . x = -16 - 4 - 3 = -23    ; * 0.5 = -11.5
    # t = R . x = 0.5 + 0.5 + 1 + 2 = 4 ; adapters add 1.5*4 = 6 and -0.5*4 = -2
    Y = oracle.linear_fwd(X, vals, meta, 0.5, L, R)
    assert Y.tolist() == [[3.75, -13.5]]
    Yd = oracle.linear_fwd_dense(X, vals, meta, 0.5, L, R)
    assert Yd.tolist() == [[3.75, -13.5]]
    # without adapters only the sparse term remains
    assert oracle.linear_fwd(X, vals, meta, 0.5, None, None).tolist() == [[-2.25, -11.5]]


# ------------------------------------------------------- P1/P2: structure
def random_codes_mask(rng, d_out, d_in, kept_choices=(0, 1, 2)):
    codes = rng.integers(-8, 8, size=(d_out, d_in)).astype(np.int8)
    mask = np.zeros((d_out, d_in // 4, 4), np.uint8)
    kept = rng.choice(kept_choices, size=(d_out, d_in // 4))
    for n in range(d_out):
        for g in range(d_in // 4):
            pos = rng.permutation(4)[: kept[n, g]]
            mask[n, g, pos] = 1
    return codes, mask.reshape(d_out, d_in)


def test_round_trip_and_invariants():
    rng = np.random.default_rng(1)
    codes, mask = random_codes_mask(rng, 24, 64)
    # make sure -8, 0-at-kept-slot and every group population occur
    codes[0, :4] = [-8, 0, -8, 0]
    mask[0, :4] = [1, 1, 0, 0]
    vals, meta = oracle.pack(codes, mask)
    assert vals.shape == (24, 16) and meta.shape == (24, 8)
    c2, m2 = oracle.unpack(vals, meta)
    kept = mask.astype(bool)
    # stored positions are a superset of the kept ones, exactly two per group
    assert (m2.reshape(24, 16, 4).sum(-1) == 2).all()
    assert (m2.astype(bool) | ~kept).all()
    assert (c2 == np.where(kept, codes, 0)).all()
    # 2:4 invariant on the decoded weight
    assert ((c2.reshape(24, 16, 4) != 0).sum(-1) <= 2).all()
    # every index nibble is an ascending pair i0 < i1
    nib = np.stack([meta & 0xF, meta >> 4], -1).reshape(24, 16)
    assert set(np.unique(nib).tolist()) <= {0x4, 0x8, 0xC, 0x9, 0xD, 0xE}
    assert ((nib & 3) < (nib >> 2)).all()
    # packing is idempotent on its own output
    v3, t3 = oracle.pack(c2, m2)
    assert (v3 == vals).all() and (t3 == meta).all()


def test_pack_layout_one_hot():
    """A single kept weight lands in exactly one nibble whose place follows the format."""
    d_out, d_in = 3, 32
    for n, k, code in [(0, 0, 5), (1, 7, -8), (2, 30, -1), (1, 17, 7)]:
        codes = np.zeros((d_out, d_in), np.int8)
        mask = np.zeros((d_out, d_in), np.uint8)
        codes[n, k] = code
        mask[n, k] = 1
        vals, meta = oracle.pack(codes, mask)
        g, i = divmod(k, 4)
        # the group is completed with the lowest other position
        other = 0 if i != 0 else 1
        p0, p1 = sorted((i, other))
        exp_v = np.zeros_like(vals)
        exp_v[n, g] = (code & 0xF) << (0 if p0 == i else 4)
        assert (vals == exp_v).all()
        got = (int(meta[n, g // 2]) >> (4 * (g % 2))) & 0xF
        assert got == (p0 | (p1 << 2))
        # all other groups hold the default pair (0,1) = 0x4
        m_all = np.stack([meta & 0xF, meta >> 4], -1).reshape(d_out, d_in // 4)
        m_all[n, g] = 0x4
        assert (m_all == 0x4).all()


def test_pack_errors():
    codes = np.zeros((2, 8), np.int8)
    mask = np.zeros((2, 8), np.uint8)
    mask[1, 4:7] = 1
    with pytest.raises(oracle.OracleError) as e:
        oracle.pack(codes, mask)
    assert e.value.code == oracle.BAD_MASK and (e.value.row, e.value.group) == (1, 1)
    mask[:] = 0
    mask[0, 2] = 1
    codes[0, 2] = 9
    with pytest.raises(oracle.OracleError) as e:
        oracle.pack(codes, mask)
    assert e.value.code == oracle.CODE_RANGE and (e.value.row, e.value.group) == (0, 0)
    # out-of-range codes at pruned positions are ignored
    mask[:] = 0
    vals, meta = oracle.pack(codes, mask)
    assert (vals == 0).all()


# ------------------------------------- P3/P5: identity and independent matmul
@pytest.mark.parametrize("d_in,d_out,r,b", [(64, 48, 16, 5), (128, 32, 48, 3), (32, 80, 0, 4)])
def test_forward_matches_numpy_float64(d_in, d_out, r, b):
    ly = inputs.make_layer(d_in, d_out, r, b, seed=7)
    vals, meta = oracle.pack(ly.codes, ly.mask)
    Y = oracle.linear_fwd(ly.X, vals, meta, ly.s, ly.L, ly.R)
    # independent restatement with numpy's float64 matmul from the *unpacked inputs*
    Wc = np.float64(np.float32(ly.s)) * (ly.codes.astype(np.float64) * ly.mask)
    Xf = inputs.bf16_bits_to_f64(ly.X)
    if r:
        W_eff = Wc + inputs.bf16_bits_to_f64(ly.L) @ inputs.bf16_bits_to_f64(ly.R)
    else:
        W_eff = Wc
    Yn = Xf @ W_eff.T
    scale = np.abs(Yn).max()
    assert np.abs(Y - Yn).max() <= 1e-12 * scale
    Yd, We = oracle.linear_fwd_dense(ly.X, vals, meta, ly.s, ly.L, ly.R, return_weight=True)
    assert np.abs(Yd - Yn).max() <= 1e-12 * scale
    assert np.abs(We - W_eff).max() <= 1e-15
    # a row subset equals the same rows of the full result, in list order
    rows = [b - 1, 0]
    Ys = oracle.linear_fwd(ly.X, vals, meta, ly.s, ly.L, ly.R, rows=rows)
    assert (Ys == Y[rows]).all()


# ----------------------------------------------------- P6: integer-exact case
def test_forward_integer_exact():
    rng = np.random.default_rng(3)
    d_in, d_out, r, b = 96, 40, 16, 6
    codes, mask = random_codes_mask(rng, d_out, d_in)
    vals, meta = oracle.pack(codes, mask)
    Xi = rng.integers(-4, 5, size=(b, d_in))
    Li = rng.integers(-2, 3, size=(d_out, r))
    Ri = rng.integers(-2, 3, size=(r, d_in))
    Y = oracle.linear_fwd(bf(Xi), vals, meta, 1.0, bf(Li), bf(Ri))
    Wi = codes.astype(np.int64) * mask
    exact = Xi @ Wi.T + (Xi @ Ri.T) @ Li.T       # int64 arithmetic
    assert (Y == exact.astype(np.float64)).all()


def test_one_hot_activations_read_weight_columns():
    rng = np.random.default_rng(4)
    d_in, d_out = 32, 24
    codes, mask = random_codes_mask(rng, d_out, d_in, kept_choices=(2,))
    vals, meta = oracle.pack(codes, mask)
    X = np.eye(d_in, dtype=np.float32)
    Y = oracle.linear_fwd(bf(X), vals, meta, 0.25, None, None)
    assert (Y == 0.25 * (codes.astype(np.float64) * mask).T).all()


# ------------------------------------------------- P8: degenerate reductions
def test_degenerate_cases():
    ly = inputs.make_layer(64, 32, 16, 4, seed=11)
    vals, meta = oracle.pack(ly.codes, ly.mask)
    Xf = inputs.bf16_bits_to_f64(ly.X)
    Lf, Rf = inputs.bf16_bits_to_f64(ly.L), inputs.bf16_bits_to_f64(ly.R)
    full = oracle.linear_fwd(ly.X, vals, meta, ly.s, ly.L, ly.R)
    sparse_only = oracle.linear_fwd(ly.X, vals, meta, ly.s, None, None)
    # zero weight -> pure low-rank term
    zv, zm = oracle.pack(np.zeros_like(ly.codes), np.zeros_like(ly.mask))
    lowrank = oracle.linear_fwd(ly.X, zv, zm, ly.s, ly.L, ly.R)
    assert np.abs(lowrank - (Xf @ Rf.T) @ Lf.T).max() <= 1e-13
    assert np.abs(full - (sparse_only + lowrank)).max() <= 1e-12
    # doubling s doubles only the sparse term (2*s is exact in fp32)
    doubled = oracle.linear_fwd(ly.X, vals, meta, 2 * ly.s, ly.L, ly.R)
    assert np.abs(doubled - (2 * sparse_only + lowrank)).max() <= 1e-12
    # zero adapters equal no adapters
    z = oracle.linear_fwd(ly.X, vals, meta, ly.s, np.zeros_like(ly.L), np.zeros_like(ly.R))
    assert (z == sparse_only).all()


# ---------------------------------------- P7: the paper's printed FLOP table
def test_flop_reduction_matches_printed_table():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "flop_reduction_table.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 4
    for _name, d, n, dff, V, rr, printed in rows:
        d, n, dff, V, rr, printed = int(d), int(n), int(dff), int(V), float(rr), float(printed)
        got = oracle.flop_reduction(d, n, dff / d, V, rr)
        assert abs(got - printed) <= 0.005 + 1e-9, (got, printed)


# ---------------------------------------------------------------- decode-tiled copy
def test_repack_tiled_bytes_by_hand():
    """One value byte and one index byte placed by hand arithmetic.
    Row 9 = lane row g = 1, upper half of the tile; group 5 of the row = step 0,
    second half of the step (4 + t with t = 1): value word of lane 4*1 + 1 = 5, step 0,
    slot i = 3 (upper row, second half): low nibble at bits 12-15, high nibble at bits 28-31.
    Index byte 2 of row 9 = columns 16-23 of step 0: second half of the step, so the
    word of lane (g = 1, t = 1) for step 0, upper row in bits 16-31."""
    vals = np.zeros((16, 64), np.uint8)
    meta = np.zeros((16, 32), np.uint8)
    vals[9, 5] = 0xA3
    meta[9, 2] = 0xE4
    out = oracle.repack_tiled(vals, meta)
    assert out.size == 4 * 1536              # one group of four pieces: the tile and three padding pieces
    assert not out[1536:].reshape(3, 1536)[:, :1024].any() and (out[1536:].reshape(3, 1536)[:, 1024:] == 0x44).all()
    out = out[:1536]
    expect = np.zeros(1536, np.uint8)
    expect[5 * 16 + 0: 5 * 16 + 4] = [0x00, 0x30, 0x00, 0xA0]           # 0xA0003000 little-endian
    expect[1024 + 5 * 16 + 0: 1024 + 5 * 16 + 4] = [0x00, 0x00, 0xE4, 0x00]
    assert np.array_equal(out, expect)
    # a byte of the second half of the block (step 6 -> second 512 bytes, word 2 of the lane),
    # lower row, first half of the step (t = 2): slot i = 0
    vals[:] = 0
    meta[:] = 0
    vals[3, 8 * 6 + 2] = 0x7C
    meta[3, 4 * 6 + 1] = 0x9D        # columns 8-15 of step 6: first half -> lane t even of steps 4-7: t = 2
    out = oracle.repack_tiled(vals, meta)[:1536]
    expect = np.zeros(1536, np.uint8)
    lane = 3 * 4 + 2
    expect[512 + lane * 16 + 2 * 4: 512 + lane * 16 + 2 * 4 + 4] = [0x0C, 0x00, 0x07, 0x00]
    expect[1024 + lane * 16 + 2 * 4: 1024 + lane * 16 + 2 * 4 + 4] = [0x00, 0x9D, 0x00, 0x00]
    assert np.array_equal(out, expect)


def dense_from_tiled(buf, d_out, d_in):
    """Read a decode-tiled buffer the way its consumer does (per lane and step: four
    value slots, index half-words from the lane that holds them) and rebuild the dense
    code matrix.  Written from the layout's description, not from the oracle's loops."""
    nblk, tiles = d_in // 256, d_out // 16
    tiles4 = (tiles + 3) // 4 * 4
    pieces = buf.view("<u4").reshape(tiles4 * nblk, 384)        # 1536-byte pieces in storage order
    dense = np.zeros((16 * tiles4, d_in), np.int64)
    sext = lambda n: n - 16 if n >= 8 else n
    # storage order: groups of four tiles; in a group block after block; in a block the group's four tiles
    order = [(g4 + t, blk) for g4 in range(0, tiles4, 4) for blk in range(nblk) for t in range(4)]
    assert len(order) == tiles4 * nblk
    for piece, (tile, blk) in enumerate(order):
        if True:
            wv = pieces[piece, :256].reshape(2, 32, 4)          # [half of the steps][lane][word]
            wm = pieces[piece, 256:].reshape(32, 4)             # [lane][word]
            for j in range(8):
                for lane in range(32):
                    g, t = divmod(lane, 4)
                    w = int(wv[j // 4, lane, j % 4])
                    for i in range(4):
                        up, second = i % 2, i // 2
                        lo, hi = (w >> (4 * i)) & 15, (w >> (16 + 4 * i)) & 15
                        # the index half-word of this half of the step lives in lane (g, 2 * (j // 4) + second)
                        e = int(wm[g * 4 + 2 * (j // 4) + second, j % 4])
                        half = (e >> (16 * up)) & 0xFFFF
                        nib = (half >> (4 * t)) & 15
                        p0, p1 = nib & 3, nib >> 2
                        col = 256 * blk + 32 * j + 16 * second + 4 * t
                        row = 16 * tile + g + 8 * up
                        dense[row, col + p0] += sext(lo)
                        dense[row, col + p1] += sext(hi)
    return dense


def test_repack_tiled_keeps_every_code_and_position():
    rng = np.random.default_rng(5)
    d_out, d_in = 112, 768      # seven tiles: one full group of four and a group of three
    codes = rng.integers(-8, 8, size=(d_out, d_in)).astype(np.int8)
    mask = inputs.top2_mask(rng.standard_normal((d_out, d_in)).astype(np.float32))
    vals, meta = oracle.pack(codes, mask)
    tiled = oracle.repack_tiled(vals, meta)
    assert tiled.size == 128 * d_in * 3 // 8                     # seven tiles are stored as two groups of four
    dense = dense_from_tiled(tiled, d_out, d_in)
    assert np.array_equal(dense[:d_out], codes.astype(np.int64) * mask)
    assert not dense[d_out:].any()                               # the padding tile holds stored zeros
    # a permutation of the input bits plus the padding tile's index nibbles (one set bit each)
    pad_bits = 16 * d_in // 4
    assert int(np.unpackbits(tiled).sum()) == int(np.unpackbits(vals).sum() + np.unpackbits(meta).sum()) + pad_bits


def test_repack_tiled_group_order_by_hand():
    """Where whole pieces go: 6 tiles x 2 blocks.  Group 0 (tiles 0-3) holds block 0 of tiles 0..3, then
    block 1 of tiles 0..3; group 1 (tiles 4, 5 and two padding tiles) holds block 0 of its four tiles, then block 1."""
    d_out, d_in = 96, 512
    vals = np.zeros((d_out, d_in // 4), np.uint8)
    meta = np.zeros((d_out, d_in // 8), np.uint8)
    for tile in range(6):
        for blk in range(2):
            vals[16 * tile, 64 * blk] = 0x10 * tile + blk + 1      # row g = 0, group 0 of the block: lane 0, step 0, slot 0
    out = oracle.repack_tiled(vals, meta).reshape(16, 1536)
    where = {(0, 0): 0, (1, 0): 1, (2, 0): 2, (3, 0): 3, (0, 1): 4, (1, 1): 5, (2, 1): 6, (3, 1): 7,
             (4, 0): 8, (5, 0): 9, (4, 1): 12, (5, 1): 13}
    for piece in (10, 11, 14, 15):                               # padding: stored zeros at positions (0, 1)
        assert not out[piece, :1024].any() and (out[piece, 1024:] == 0x44).all()
    for (tile, blk), piece in where.items():
        B = 0x10 * tile + blk + 1
        w = int(out[piece, :4].view("<u4")[0])
        assert w == (B & 15) | ((B >> 4) << 16), (tile, blk, piece, hex(w))
        assert not out[piece, 4:].any()


def test_repack_tiled_rejects_shapes_it_cannot_tile():
    with pytest.raises(oracle.OracleError):
        oracle.repack_tiled(np.zeros((8, 64), np.uint8), np.zeros((8, 32), np.uint8))
    with pytest.raises(oracle.OracleError):
        oracle.repack_tiled(np.zeros((16, 32), np.uint8), np.zeros((16, 16), np.uint8))


# ---------------------------------------------------------------- quantized adapters (Sec. 3.3)
def np_dequant(codes, scales):
    """Reader-side decode of the adapter storage, written with numpy bit operations only."""
    lo = (codes & 0xF).astype(np.int16)
    hi = (codes >> 4).astype(np.int16)
    q = np.stack([lo, hi], axis=-1).reshape(codes.shape[0], -1)
    q = np.where(q > 7, q - 16, q).astype(np.float64)
    sc = inputs.bf16_bits_to_f64(scales)
    return q * np.repeat(sc, 128, axis=1)[:, :q.shape[1]]


def test_quant_adapter_groups_by_hand():
    cols = 128 + 16                      # a full group and a short one per row
    A = np.zeros((3, cols), np.float32)
    # row 0, group 0: absmax 1.75 -> scale 0.25 exactly; 0.3 -> bf16 0.30078 / 0.25 = 1.203 -> 1;
    #   ties go to even: 0.375 / 0.25 = 1.5 -> 2, 0.625 / 0.25 = 2.5 -> 2, -0.375 -> -2 (= -1.5 to even)
    A[0, :8] = [0.5, -1.75, 0.25, 0.0, 0.3, 0.375, 0.625, -0.375]
    # row 0, group 1 (16 elements): its largest magnitude is negative: -3.5 -> scale 0.5, code -7
    A[0, 128:132] = [-3.5, 1.0, 0.26, -0.74]       # 2, 0.26 -> bf16 0.2598 / 0.5 = 0.52 -> 1, -0.74 -> -1.48 -> -1
    # row 1: all zeros -> scale 0, codes 0
    # row 2, group 0: absmax 1 -> 1/7 = 0.142857 -> bf16 0x3E12 = 0.142578125; 1 / 0.142578125 = 7.01 -> 7
    A[2, :4] = [1.0, -1.0, 0.5, 0.07]               # 0.5 / 0.142578 = 3.507 -> 4 ; 0.07 -> bf16 0.06982 / 0.142578 = 0.49 -> 0
    codes, scales = oracle.quant_adapter(bf(A))
    assert codes.shape == (3, cols // 2) and scales.shape == (3, 2)
    assert scales.tolist() == [[0x3E80, 0x3F00], [0, 0], [0x3E12, 0]]
    # two codes per byte, the even column in the low nibble, two's complement
    assert codes[0, :4].tolist() == [0x92, 0x01, 0x21, 0xE2]          # (2,-7) (1,0) (1,2) (2,-2)
    assert codes[0, 64:66].tolist() == [0x29, 0xF1]                    # (-7,2) (1,-1)
    assert not codes[0, 4:64].any() and not codes[0, 66:].any() and not codes[1].any()
    assert codes[2, :2].tolist() == [0x97, 0x04] and not codes[2, 2:].any()   # (7,-7) (4,0)
    # the values they stand for
    val = oracle.dequant_adapter(codes, scales)
    assert val[0, :8].tolist() == [0.5, -1.75, 0.25, 0.0, 0.25, 0.5, 0.5, -0.5]
    assert val[0, 128:132].tolist() == [-3.5, 1.0, 0.5, -0.5]
    assert val[2, :4].tolist() == [7 * 0.142578125, -7 * 0.142578125, 4 * 0.142578125, 0.0]
    assert not val[1].any()


def test_dequant_adapter_decodes_minus_eight_and_every_nibble():
    codes = np.array([[0x10 * h + l for l in range(16)] for h in range(16)], np.uint8).reshape(2, 128)
    scales = bf(np.array([[0.5, 2.0], [1.0, 0.25]], np.float32))
    val = oracle.dequant_adapter(codes, scales)
    assert np.array_equal(val, np_dequant(codes, scales))
    assert val[0, 16] == -8 * 0.5 and val[0, 17] == 0.0           # byte 0x08: nibble 8 is -8, even column low
    assert val.min() == -8 * 2.0 and val.max() == 7 * 2.0


@pytest.mark.parametrize("rows,cols,seed", [(5, 256, 1), (7, 144, 2), (3, 16, 3), (2, 1000, 4)])
def test_quant_adapter_round_trip_bound_and_invariants(rows, cols, seed):
    rng = np.random.default_rng(seed)
    A = bf(rng.standard_t(3, (rows, cols)).astype(np.float32) * 0.02)        # long-tailed, like adapters
    a = inputs.bf16_bits_to_f64(A)
    codes, scales = oracle.quant_adapter(A)
    val = oracle.dequant_adapter(codes, scales)
    assert np.array_equal(val, np_dequant(codes, scales))
    sc = np.repeat(inputs.bf16_bits_to_f64(scales), 128, axis=1)[:, :cols]
    # AbsMax: the scale is the group's largest magnitude over 7, to bf16 precision
    for i in range(rows):
        for g in range((cols + 127) // 128):
            m = np.abs(a[i, g * 128:(g + 1) * 128]).max()
            assert abs(sc[i, g * 128] - m / 7) <= m / 7 * 2.0 ** -8
    # nearest code: the error is at most half a step (a hair more where the rounded scale makes 7.0x -> 7)
    assert np.all(np.abs(val - a) <= sc * (0.5 + 2.0 ** -6))
    q = np.rint(val / np.where(sc > 0, sc, 1))
    assert q.min() >= -7 and q.max() <= 7
    # the element with the group's largest magnitude gets code +-7
    for i in range(rows):
        k = np.abs(a[i, :min(cols, 128)]).argmax()
        assert abs(q[i, k]) == 7


def test_quant_adapter_rejects_bad_shapes():
    with pytest.raises(oracle.OracleError):
        oracle.quant_adapter(np.zeros((2, 7), np.uint16))


def test_linear_fwd_q_matches_numpy_float64_from_decoded_storage():
    d_in, d_out, r, b = 272, 24, 48, 5                 # short last groups on both adapters
    s, codes, mask = inputs.make_weights(d_out, d_in, 71)
    vals, meta = oracle.pack(codes, mask)
    L, R = inputs.make_adapters(d_out, d_in, r, 71)
    X = inputs.make_activations(b, d_in, 71)
    Lq, Ls = oracle.quant_adapter(L)
    Rq, Rs = oracle.quant_adapter(R)
    got = oracle.linear_fwd_q(X, vals, meta, s, Lq, Ls, Rq, Rs)
    x = inputs.bf16_bits_to_f64(X)
    W = np.float64(np.float32(s)) * (codes.astype(np.float64) * mask)
    want = x @ W.T + (x @ np_dequant(Rq, Rs).T) @ np_dequant(Lq, Ls).T
    assert got.shape == (b, d_out)
    assert np.abs(got - want).max() <= 1e-12 * np.abs(want).max()
    # it is not the unquantized layer: the adapters' rounding shows
    plain = oracle.linear_fwd(X, vals, meta, s, L, R)
    assert np.abs(got - plain).max() > 1e-6
    # rows subset
    sub = oracle.linear_fwd_q(X, vals, meta, s, Lq, Ls, Rq, Rs, rows=[4, 0])
    assert np.array_equal(sub, got[[4, 0]])


def test_linear_fwd_q_reduces_to_the_plain_layer_for_adapters_on_the_grid():
    """Adapters whose entries are already code x power-of-two scale survive quantization unchanged,
    so the quantized layer equals the pinned bf16-adapter layer."""
    d_in, d_out, r, b = 256, 16, 32, 3
    rng = np.random.default_rng(9)
    s, codes, mask = inputs.make_weights(d_out, d_in, 72)
    vals, meta = oracle.pack(codes, mask)
    def on_grid(rows, cols):
        q = rng.integers(-7, 8, (rows, cols)).astype(np.float32)
        q[:, ::128] = 7                                  # every group reaches +7, so its scale is what was meant
        sc = 2.0 ** rng.integers(-9, -3, (rows, (cols + 127) // 128)).astype(np.float32)
        return bf(q * np.repeat(sc, 128, axis=1)[:, :cols])
    L, R = on_grid(d_out, r), on_grid(r, d_in)
    X = inputs.make_activations(b, d_in, 72)
    Lq, Ls = oracle.quant_adapter(L)
    Rq, Rs = oracle.quant_adapter(R)
    assert np.array_equal(oracle.dequant_adapter(Lq, Ls), inputs.bf16_bits_to_f64(L))
    assert np.array_equal(oracle.dequant_adapter(Rq, Rs), inputs.bf16_bits_to_f64(R))
    assert np.array_equal(oracle.linear_fwd_q(X, vals, meta, s, Lq, Ls, Rq, Rs), oracle.linear_fwd(X, vals, meta, s, L, R))


# ---------------------------------------------------------------- SLiM-Quant scale search (Sec. 3.1, Alg. 1)
def true_mse(W, alpha):
    """Eq. 3 on the weights themselves: mean |Q^-1(Q(w)) - w|^2 with the symmetric 4-bit grid of Eq. 2 / Eq. 5."""
    w = W.astype(np.float64)
    q = np.rint(np.clip(w / alpha, -1.0, 1.0) * 8.0)
    return float(np.mean((q * alpha / 8.0 - w) ** 2))


def bell(kind, shape, seed):
    rng = np.random.default_rng(seed)
    if kind == "normal":
        w = rng.standard_normal(shape)
    elif kind == "laplace":
        w = rng.laplace(size=shape)
    else:
        w = rng.standard_t(4, shape)
    return (w * 0.02).astype(np.float32)


@pytest.mark.parametrize("kind,shape,seed", [("normal", (300, 400), 0), ("laplace", (64, 1000), 1), ("student", (700, 900), 2),
                                              ("normal", (16, 32), 3)])
def test_slim_quant_error_model_and_search(kind, shape, seed):
    W = bell(kind, shape, seed)
    M = float(np.abs(W).max())
    codes, scale, alpha, table = oracle.slim_quant(W)
    # the grid of Algorithm 1 as read: ten uniform samples of (0, M], then nineteen steps of a tenth around the best
    assert np.allclose(table[:10, 0], M * np.arange(1, 11) / 10, rtol=1e-15)
    k_low = int(np.argmin(table[:10, 1]))
    a_low, eta = table[k_low, 0], M / 10
    assert np.allclose(table[10:, 0], np.minimum(a_low - eta + np.arange(1, 20) * eta / 10, M), rtol=1e-12, atol=1e-18)
    # the histogram integral follows the error of the definition, candidate by candidate
    n_bins = max(512, min(W.size // 1000, 20000))
    for a, e in table:
        assert abs(e - true_mse(W, a)) <= 0.02 * true_mse(W, a) + (M / n_bins) ** 2, (a, e, true_mse(W, a))
    # alpha* is the first minimiser of the table, and (to the accuracy of the integral) of the true error
    i_best = int(np.argmin(table[:, 1]))
    assert alpha == table[i_best, 0] and 0 < alpha <= M
    best_true = min(true_mse(W, a) for a in table[:, 0])
    assert true_mse(W, alpha) <= 1.02 * best_true
    # clipping pays on bell-shaped weights: better than AbsMax (alpha = M), which is candidate 10
    if W.size > 1000:
        assert alpha < M and true_mse(W, alpha) < 0.8 * true_mse(W, M)
    # codes and scale of the quantization step at alpha*
    assert scale == np.float32(np.float32(alpha) * np.float32(0.125))
    want = np.clip(np.rint(W.astype(np.float64) / np.float64(np.float32(alpha)) * 8.0), -8, 7)
    assert np.mean(codes != want) < 1e-4 and np.abs(codes - want).max() <= 1          # binary32 decisions at ties only
    assert codes.min() >= -8 and codes.max() <= 7


def test_slim_quant_single_magnitude_by_hand():
    # every |w| = c: all weights sit in the last bin (centre c (1 - 1/1024)); among alpha = k c / 10 only
    # alpha = c avoids clipping it (error (c/1024)^2, level 8); the fine steps below c clip it again, so
    # alpha* = c, the scale is c / 8 and the codes are +8 -> 7 (int4) and -8
    c = np.float32(0.75)
    W = np.full((6, 10), c, np.float32)
    W[::2] *= -1
    codes, scale, alpha, table = oracle.slim_quant(W)
    assert alpha == 0.75 and scale == np.float32(0.09375)
    assert np.array_equal(codes, np.where(W > 0, 7, -8))
    assert table[9, 0] == 0.75 and abs(table[9, 1] - (0.75 / 1024) ** 2) < 1e-15
    assert abs(table[8, 1] - (0.75 * (0.9 - (1 - 1 / 1024))) ** 2) < 1e-12     # alpha = 0.9 c clips the bin centre


def test_slim_quant_scales_with_powers_of_two_and_handles_degenerate_input():
    W = bell("normal", (128, 256), 5)
    codes, scale, alpha, table = oracle.slim_quant(W)
    codes4, scale4, alpha4, table4 = oracle.slim_quant(W * np.float32(4))
    assert np.array_equal(codes, codes4) and scale4 == scale * 4 and alpha4 == alpha * 4
    assert np.array_equal(table4[:, 0], table[:, 0] * 4) and np.allclose(table4[:, 1], table[:, 1] * 16, rtol=1e-12)
    z = oracle.slim_quant(np.zeros((4, 8), np.float32))
    assert not z[0].any() and z[1] == 0 and z[2] == 0
    bad = np.zeros((4, 8), np.float32)
    bad[1, 2] = np.nan
    with pytest.raises(oracle.OracleError):
        oracle.slim_quant(bad)


# ---------------------------------------------------------------- 2:4 mask producer (pipeline step 2)
def test_mask_top2_by_hand():
    codes = np.array([[3, -3, 3, 1,   0, 0, 0, 0,   -8, 7, -7, 8 - 16,   1, 2, 3, 4]], np.int8)
    # group 0: |3| three times: the two lowest indices win the tie; group 1: all zero -> positions 0, 1;
    # group 2: magnitudes 8, 7, 7, 8 -> positions 0 and 3; group 3: 3 and 4
    assert oracle.mask_top2(codes).tolist() == [[1, 1, 0, 0,  1, 1, 0, 0,  1, 0, 0, 1,  0, 0, 1, 1]]
    # input magnitudes re-rank the entries: |q| * xbar = (3, 0.75, 6, 2 | ... | 8, 14, 3.5, 8 | 0.5, 2, 0, 8)
    xbar = np.array([1, 0.25, 2, 2,  5, 0, 1, 1,  1, 2, 0.5, 1,  0.5, 1, 0, 2], np.float32)
    # group 1: metrics all zero whatever xbar says: positions 0, 1 again
    assert oracle.mask_top2(codes, xbar).tolist() == [[1, 0, 1, 0,  1, 1, 0, 0,  1, 1, 0, 0,  0, 1, 0, 1]]


@pytest.mark.parametrize("d_out,d_in,seed", [(7, 64, 1), (33, 1000, 2)])
def test_mask_top2_agrees_with_the_generators_mask_and_keeps_two_per_group(d_out, d_in, seed):
    rng = np.random.default_rng(seed)
    codes = rng.integers(-8, 8, (d_out, d_in)).astype(np.int8)
    m = oracle.mask_top2(codes)
    assert np.array_equal(m, inputs.top2_mask(codes.astype(np.float32)))      # numpy's own statement of the rule
    xbar = rng.random(d_in).astype(np.float32)
    mx = oracle.mask_top2(codes, xbar)
    assert np.array_equal(mx, inputs.top2_mask(np.abs(codes).astype(np.float32) * xbar[None, :]))
    for mask in (m, mx):
        assert np.all(mask.reshape(d_out, d_in // 4, 4).sum(-1) == 2)
    with pytest.raises(oracle.OracleError):
        oracle.mask_top2(codes, np.full(d_in, np.nan, np.float32))
