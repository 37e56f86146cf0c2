"""Pins for the CPU oracle: each test fixes it to something other than itself - a closed form, an
invariant, a library routine, brute force, or a hand-worked example under tests/golden/.  The paper
(Section 4) prints no numeric example of the LUT path, so none of the pins is a paper-printed value."""
import itertools
import os

import numpy as np
import pytest

from oracle import lcd_oracle as O

HERE = os.path.dirname(os.path.abspath(__file__))


def rnd_case(seed, N, K, C, M):
    rng = np.random.default_rng(seed)
    idx = rng.integers(0, C, size=(N, K), dtype=np.uint8)
    cb = (rng.standard_normal((N, C)) * 0.1).astype(np.float16)
    q = rng.integers(-8, 8, size=(M, K), dtype=np.int8)
    s_q = (rng.random(M) + 0.1).astype(np.float32)
    return idx, cb, q, s_q


# ---------------------------------------------------------------- linear forms (Section 4.2)
@pytest.mark.parametrize("bits", [2, 3])
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_four_forms_and_loops_agree(bits, seed):
    C = 1 << bits
    idx, cb, q, s_q = rnd_case(seed, N=7, K=61, C=C, M=3)
    ref = O.lut_linear_loops(idx, cb, q, s_q)
    scale = (np.abs(q.astype(float)).sum(axis=1)[:, None] * np.abs(cb.astype(float)).max(axis=1)[None, :]
             * s_q[:, None].astype(float))
    for f in (O.lut_linear_dequant, O.lut_linear_product, O.lut_linear_signfold, O.lut_linear_bucket):
        y = f(idx, cb, q, s_q)
        assert np.all(np.abs(y - ref) <= 1e-12 * scale + 1e-300), f.__name__


def test_matches_library_matmul_on_dequantised_matrix():
    idx, cb, q, s_q = rnd_case(5, N=33, K=200, C=8, M=4)
    Wq = np.empty((33, 200))
    for n in range(33):
        for k in range(200):
            Wq[n, k] = float(cb[n, idx[n, k]])
    xq = s_q[:, None].astype(np.float64) * q.astype(np.float64)
    ref = np.matmul(xq, Wq.T)
    y = O.lut_linear_bucket(idx, cb, q, s_q)
    assert np.allclose(y, ref, rtol=1e-12, atol=1e-12)
    assert np.allclose(O.lut_linear_dequant(idx, cb, q, s_q), ref, rtol=1e-12, atol=1e-12)


def test_one_centroid_codebook_gives_c_times_sum_x():
    rng = np.random.default_rng(3)
    N, K, M = 5, 40, 2
    idx = np.zeros((N, K), dtype=np.uint8)
    cb = (rng.standard_normal((N, 1))).astype(np.float16)
    q = rng.integers(-8, 8, size=(M, K), dtype=np.int8)
    s_q = np.array([0.25, 1.5], dtype=np.float32)
    expect = (s_q.astype(float)[:, None] * q.astype(float).sum(axis=1)[:, None]) * cb.astype(float)[:, 0][None, :]
    for f in (O.lut_linear_dequant, O.lut_linear_product, O.lut_linear_signfold, O.lut_linear_bucket):
        assert np.allclose(f(idx, cb, q, s_q), expect, rtol=1e-13, atol=0), f.__name__


def test_affine_codebook_closed_form_hand_case():
    # hand-worked example, see tests/golden/affine_k4.txt
    g = [l for l in open(os.path.join(HERE, "golden", "affine_k4.txt")) if not l.startswith("#")]
    vals = [float(v) for v in g[0].split()]
    idx = np.array([[0, 3, 1, 2]], dtype=np.uint8)
    cb = np.array([[0.5 * w - 0.25 for w in range(4)]], dtype=np.float16)        # alpha=.5, beta=-.25
    q = np.array([[3, -2, 7, -8]], dtype=np.int8)
    s_q = np.array([0.5], dtype=np.float32)
    # sum q*idx = 0 - 6 + 7 - 16 = -15 ; sum q = 0 ; y = 0.5 * (0.5 * -15 + -0.25 * 0) = -3.75
    for f in (O.lut_linear_dequant, O.lut_linear_product, O.lut_linear_signfold, O.lut_linear_bucket,
              O.lut_linear_loops):
        assert f(idx, cb, q, s_q)[0, 0] == vals[0] == -3.75


@pytest.mark.parametrize("seed", [0, 1])
def test_affine_codebook_closed_form_random(seed):
    rng = np.random.default_rng(seed)
    N, K, M, C = 6, 50, 3, 8
    idx = rng.integers(0, C, size=(N, K), dtype=np.uint8)
    alpha = rng.integers(-4, 5, size=N) / 8.0
    beta = rng.integers(-8, 9, size=N) / 16.0
    cb = (alpha[:, None] * np.arange(C)[None, :] + beta[:, None]).astype(np.float16)   # exact in fp16
    q = rng.integers(-8, 8, size=(M, K), dtype=np.int8)
    s_q = np.array([0.5, 2.0, 0.125], dtype=np.float32)
    sqi = (q.astype(np.int64) @ idx.astype(np.int64).T)
    sq = q.astype(np.int64).sum(axis=1)
    expect = s_q.astype(float)[:, None] * (alpha[None, :] * sqi + beta[None, :] * sq[:, None])
    for f in (O.lut_linear_dequant, O.lut_linear_bucket, O.lut_linear_product, O.lut_linear_signfold):
        assert np.allclose(f(idx, cb, q, s_q), expect, rtol=1e-13, atol=1e-13)


def test_brute_force_all_index_patterns_k6_c2():
    K = 6
    cb = np.array([[-0.75, 1.25]], dtype=np.float16)
    acts = np.array([[1, -2, 3, -4, 5, -6], [7, 7, -8, 0, 0, 1]], dtype=np.int8)
    s_q = np.array([1.0, 0.5], dtype=np.float32)
    for pattern in itertools.product([0, 1], repeat=K):
        idx = np.array([pattern], dtype=np.uint8)
        expect = [[s * sum(int(a[k]) * (1.25 if pattern[k] else -0.75) for k in range(K))] for a, s in
                  zip(acts, [1.0, 0.5])]
        for f in (O.lut_linear_dequant, O.lut_linear_bucket, O.lut_linear_product, O.lut_linear_signfold):
            assert np.array_equal(f(idx, cb, acts, s_q), np.array(expect))


def test_bucket_sums_partition_the_activation_sum():
    idx, cb, q, s_q = rnd_case(9, N=4, K=97, C=4, M=2)
    S = O.bucket_sums(idx, q, 4)
    assert np.array_equal(S.sum(axis=2), np.repeat(q.astype(np.int64).sum(axis=1)[:, None], 4, axis=1))
    # a transposed operand or swapped index would break this one-hot case
    idx1 = np.zeros((2, 5), dtype=np.uint8); idx1[1, 3] = 2
    q1 = np.array([[1, 2, 3, 4, 5]], dtype=np.int8)
    S1 = O.bucket_sums(idx1, q1, 4)
    assert S1.tolist() == [[[15, 0, 0, 0], [11, 0, 4, 0]]]


# ---------------------------------------------------------------- quantiser (Section 4.1)
def test_quantiser_hand_example():
    # x = [7, -3.5, 0.5, 1.5, 2.5, -7] with inv_s = 1: A = 7, s_q = 1, r = 1 -> ties go to even
    x = np.array([[7, -3.5, 0.5, 1.5, 2.5, -7]], dtype=np.float16)
    q, s = O.smooth_quantize(x, None)
    assert q.tolist() == [[7, -4, 0, 2, 2, -7]] and s[0] == 1.0
    # smoothing is a multiply by 1/s_k: halving channel 0 moves the max to channel 5
    q2, s2 = O.smooth_quantize(x, np.array([0.5, 1, 1, 1, 1, 1], dtype=np.float32))
    assert q2.tolist() == [[4, -4, 0, 2, 2, -7]] and s2[0] == 1.0   # 3.5 -> 4 (even), A still 7


def test_quantiser_max_maps_to_pm7_and_sign_symmetry():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((5, 300)).astype(np.float16)
    inv_s = (rng.random(300) + 0.5).astype(np.float32)
    q, s = O.smooth_quantize(x, inv_s)
    assert np.all(np.abs(q).max(axis=1) == 7) and q.min() >= -7
    qn, sn = O.smooth_quantize(-x, inv_s)
    assert np.array_equal(qn, -q) and np.array_equal(sn, s)


def test_quantiser_power_of_two_scale_invariance():
    rng = np.random.default_rng(1)
    x = (rng.standard_normal((3, 128))).astype(np.float16)
    inv_s = (rng.random(128) + 0.5).astype(np.float32)
    q, s = O.smooth_quantize(x, inv_s)
    for j in (-3, 2, 5):
        q2, s2 = O.smooth_quantize((x.astype(np.float32) * 2.0 ** j).astype(np.float16), inv_s)
        assert np.array_equal(q2, q)
        assert np.array_equal(s2, (s * np.float32(2.0 ** j)).astype(np.float32))


def test_quantiser_monotone_and_zero_row_and_static_mode():
    xs = np.linspace(-3, 3, 193).astype(np.float16)
    x = np.concatenate([xs, [4.0]]).astype(np.float16)[None, :]        # fixed maximum 4 -> fixed scale
    q, s = O.smooth_quantize(x, None)
    assert np.all(np.diff(q[0, :-1].astype(int)) >= 0)
    z, sz = O.smooth_quantize(np.zeros((2, 8), dtype=np.float16), None)
    assert not z.any() and np.all(sz == 1.0)
    # static mode: f = 1/(s*s_q) and every level -8..7 is reachable, values beyond are clipped
    xv = np.arange(-10, 10, dtype=np.float16)[None, :]
    qs, ss = O.smooth_quantize(xv, np.full(20, 1.0, dtype=np.float32), static_scale=1.0)
    assert qs.tolist() == [[-8, -8, -8, -7, -6, -5, -4, -3, -2, -1, 0, 1, 2, 3, 4, 5, 6, 7, 7, 7]]
    qt, _ = O.smooth_quantize(np.array([[0.5, 1.5, 2.5, -0.5, -1.5, 6.5, -6.5]], dtype=np.float16),
                              np.ones(7, dtype=np.float32), static_scale=1.0)
    assert qt.tolist() == [[0, 2, 2, 0, -2, 6, -6]]


def test_quantiser_is_binary32_arithmetic():
    # the double-with-casts sequence must equal native float32 arithmetic step by step
    rng = np.random.default_rng(2)
    x = (rng.standard_normal((4, 512)) * 3).astype(np.float16)
    inv_s = (rng.random(512) * 3 + 0.01).astype(np.float32)
    q, s = O.smooth_quantize(x, inv_s)
    t = x.astype(np.float32) * inv_s[None, :]
    A = np.abs(t).max(axis=1)
    s32 = A / np.float32(7.0)
    r = np.float32(7.0) / A
    u = t * r[:, None]
    q32 = np.clip(np.rint(u), -8, 7).astype(np.int8)
    assert np.array_equal(q, q32) and np.array_equal(s, s32.astype(np.float32))
    ideal = O.smooth_quantize_ideal(x, inv_s)
    assert (ideal != q).mean() < 1e-3


def test_quantisation_error_bound():
    # |x/s - s_q*q| <= s_q/2 (+ rounding slack): the encoding is a uniform quantiser of step s_q
    rng = np.random.default_rng(4)
    x = rng.standard_normal((3, 256)).astype(np.float16)
    q, s = O.smooth_quantize(x, None)
    err = np.abs(x.astype(np.float64) - s.astype(np.float64)[:, None] * q)
    assert np.all(err <= 0.5 * s[:, None] * (1 + 1e-5))


def test_act_pack_roundtrip_and_padding():
    rng = np.random.default_rng(0)
    q = rng.integers(-8, 8, size=(3, 300), dtype=np.int8)
    p = O.pack_act(q)
    assert p.shape == (3, 256) and np.array_equal(O.unpack_act(p, 300), q)
    assert np.all(p[:, 150:] == 0x88)
    assert p[0, 0] == ((int(q[0, 0]) + 8) | ((int(q[0, 1]) + 8) << 4))


# ---------------------------------------------------------------- packing
@pytest.mark.parametrize("bits,C", [(2, 4), (3, 8), (3, 5), (2, 3), (4, 16), (4, 10)])
def test_pack_roundtrip_random(bits, C):
    rng = np.random.default_rng(bits * 10 + C)
    N, K = 19, 300
    idx = rng.integers(0, C, size=(N, K), dtype=np.uint8)
    cb = rng.standard_normal((N, C)).astype(np.float16)
    blob = O.pack_weights(idx, cb, bits, C)
    assert blob.size == O.packed_weights_bytes(N, K, bits)
    N_pad, K_pad = 32, 512
    assert blob.size == 256 + N_pad * K_pad * bits // 8 + ((N_pad * (1 << bits) * 2 + 255) // 256) * 256
    i2, c2, b2, C2 = O.unpack_weights(blob)
    assert np.array_equal(i2, idx) and np.array_equal(c2.view(np.uint16), cb.view(np.uint16)) and (b2, C2) == (bits, C)


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_pack_one_hot_positions_hit_distinct_bits(bits):
    # each (row, column) of one tile maps to its own bit field: one-hot inputs give disjoint blobs whose
    # union is the all-ones blob, and every payload bit is covered exactly once (exactly `bits` bits/weight)
    C = 1 << bits
    N, K = 8, 256
    cb = np.zeros((N, C), dtype=np.float16)
    full = O.pack_weights(np.full((N, K), C - 1, dtype=np.uint8), cb, bits)
    body = slice(256, 256 + N * K * bits // 8)
    assert np.all(full[body] == 0xFF)
    acc = np.zeros(N * K * bits // 8, dtype=np.uint16)
    for n in (0, 3, 7):
        for k in range(K):
            idx = np.zeros((N, K), dtype=np.uint8)
            idx[n, k] = C - 1
            b = O.pack_weights(idx, cb, bits)[body]
            assert int(np.unpackbits(b).sum()) == bits
            assert not np.any(acc.astype(np.uint8) & b)
            acc |= b
    assert int(np.unpackbits(acc.astype(np.uint8)).sum()) == 3 * K * bits


def test_pack_2bit_layout_spot_bytes():
    # written out by hand from the layout text: item 0 = tile of rows 0-7 (512 bytes) then tile of rows 8-15;
    # in a tile, lane l = 4g+t, byte p of k-block h holds columns 128h + 32t + 4p + i at bits [2i,2i+2)
    N, K = 16, 256
    idx = np.zeros((N, K), dtype=np.uint8)
    idx[0, 0] = 3          # g=0,t=0,h=0,p=0,i=0            -> byte 0,                  value 0b11
    idx[1, 5] = 2          # g=1,t=0,h=0,p=1,i=1            -> byte 16*4 + 1,           value 2<<2
    idx[2, 128 + 37] = 1   # g=2,h=1,r=37: t=1,p=1,i=1      -> byte 16*(8+1) + 8 + 1,   value 1<<2
    idx[7, 255] = 3        # g=7,h=1,r=127: t=3,p=7,i=3     -> byte 16*31 + 8 + 7,      value 3<<6
    idx[9, 4] = 1          # second tile, g=1,t=0,h=0,p=1,i=0 -> byte 512 + 16*4 + 1,   value 1
    blob = O.pack_weights(idx, np.zeros((N, 4), dtype=np.float16), 2)
    body = blob[256:256 + 1024]
    expect = np.zeros(1024, dtype=np.uint8)
    expect[0] = 3
    expect[16 * 4 + 1] = 2 << 2
    expect[16 * 9 + 8 + 1] = 1 << 2
    expect[16 * 31 + 8 + 7] = 3 << 6
    expect[512 + 16 * 4 + 1] = 1
    assert np.array_equal(body, expect)


def test_pack_item_order_two_row_groups_two_column_tiles():
    # item (rp, kt) sits at 256 + (rp * n_kt + kt) * 1024 (2 bit): rows 16..31, columns 256..511 -> item 3
    N, K = 32, 512
    idx = np.zeros((N, K), dtype=np.uint8)
    idx[16, 256] = 2       # rp=1, kt=1, first tile, g=0,t=0,h=0,p=0,i=0
    idx[31, 0] = 1         # rp=1, kt=0, second tile, g=7,t=0,h=0,p=0,i=0 -> lane 28
    blob = O.pack_weights(idx, np.zeros((N, 4), dtype=np.float16), 2)
    body = blob[256:256 + 4 * 1024]
    expect = np.zeros(4 * 1024, dtype=np.uint8)
    expect[3 * 1024] = 2
    expect[2 * 1024 + 512 + 16 * 28] = 1
    assert np.array_equal(body, expect)


def test_pack_3bit_layout_spot_bytes():
    N, K = 8, 256
    idx = np.zeros((N, K), dtype=np.uint8)
    idx[0, 0] = 5            # g=0,t=0,h=0,m=0  -> word0 bits[0,3) = 5        -> plane0 byte 0 = 5
    idx[0, 9] = 7            # m=9 -> word1, j=1 -> bits [4,7)                 -> plane1 byte 0 = 0x70
    idx[0, 24] = 6           # m=24 (j=0): bit1 -> word1 bit3, bit2 -> word2 bit3
    idx[3, 128 + 32 * 2 + 31] = 1   # g=3,t=2,h=1,m=31 (j=7): bit0 -> word0 bit 31 -> lane 14, byte offset 8*14+4+3
    blob = O.pack_weights(idx, np.zeros((N, 8), dtype=np.float16), 3)
    body = blob[256:256 + 768]
    expect = np.zeros(768, dtype=np.uint8)
    expect[0] = 5
    expect[256 + 0] = 0x70 | 0x08
    expect[512 + 0] = 0x08
    expect[8 * 14 + 4 + 3] = 0x80
    assert np.array_equal(body, expect)


def test_pack_4bit_layout_spot_bytes():
    # by hand from the layout text: a 4-bit tile is two 512-byte planes (k-block h = 0, 1); in plane h lane l = 4g+t
    # has 16 bytes at 16*l, byte p = the columns 128h + 32t + 2p (low nibble) and 2p + 1 (high nibble); an item is
    # the tile of rows 0-7 (1024 bytes) followed by the tile of rows 8-15
    N, K = 16, 256
    idx = np.zeros((N, K), dtype=np.uint8)
    idx[0, 0] = 9            # g=0,t=0,h=0,m=0            -> plane 0, byte 0, low nibble
    idx[0, 1] = 12           # m=1                        -> the same byte, high nibble
    idx[2, 37] = 15          # g=2,h=0,t=1,m=5: p=2,i=1   -> byte 16*(8+1) + 2, high nibble
    idx[7, 255] = 10         # g=7,h=1,t=3,m=31: p=15,i=1 -> byte 512 + 16*31 + 15, high nibble
    idx[9, 130] = 3          # second tile, g=1,h=1,t=0,m=2: p=1,i=0 -> byte 1024 + 512 + 16*4 + 1, low nibble
    blob = O.pack_weights(idx, np.zeros((N, 16), dtype=np.float16), 4)
    body = blob[256:256 + 2048]
    expect = np.zeros(2048, dtype=np.uint8)
    expect[0] = 9 | (12 << 4)
    expect[16 * 9 + 2] = 15 << 4
    expect[512 + 16 * 31 + 15] = 10 << 4
    expect[1024 + 512 + 16 * 4 + 1] = 3
    assert np.array_equal(body, expect)
    # the codebook area follows the index area: 16 rows of 16 fp16 values, 256-byte aligned
    assert blob.size == 256 + 2048 + 512


def test_pack_rejects_bad_indices_and_corruption():
    cb = np.zeros((2, 3), dtype=np.float16)
    with pytest.raises(ValueError):
        O.pack_weights(np.full((2, 4), 3, dtype=np.uint8), cb, 2, 3)
    blob = O.pack_weights(np.zeros((2, 4), dtype=np.uint8), cb, 2, 3)
    bad = blob.copy(); bad[300] ^= 1
    with pytest.raises(ValueError):
        O.unpack_weights(bad)
    bad = blob.copy(); bad[0] ^= 1
    with pytest.raises(ValueError):
        O.unpack_weights(bad)


# ---------------------------------------------------------------- 8-bit activations (the paper's b = 8, Section 4.1)
def test_quantiser_8bit_hand_example_and_static_levels():
    # A = 127 with inv_s = 1: s_q = 1 and r = 1 exactly, so q = round-half-even(x)
    x = np.array([[127, -63.5, 0.5, 1.5, 2.5, -127, 100.25, -0.75]], dtype=np.float16)
    q, s = O.smooth_quantize(x, None, act_bits=8)
    assert q.tolist() == [[127, -64, 0, 2, 2, -127, 100, -1]] and s[0] == 1.0
    # static mode: every level of [-128, 127] is reachable, values beyond are clipped
    xv = np.arange(-130, 131, dtype=np.float16)[None, :]
    qs, ss = O.smooth_quantize(xv, np.ones(261, dtype=np.float32), static_scale=0.25, act_bits=8)
    assert qs[0].tolist() == [max(-128, min(127, v)) for v in range(-130, 131)] and np.all(ss == np.float32(0.25))


def test_quantiser_8bit_is_binary32_arithmetic_symmetric_and_bounded():
    rng = np.random.default_rng(12)
    x = (rng.standard_normal((4, 512)) * 3).astype(np.float16)
    inv_s = (rng.random(512) * 3 + 0.01).astype(np.float32)
    q, s = O.smooth_quantize(x, inv_s, act_bits=8)
    t = x.astype(np.float32) * inv_s[None, :]
    A = np.abs(t).max(axis=1)
    s32 = A / np.float32(127.0)
    u = t * (np.float32(127.0) / A)[:, None]
    assert np.array_equal(q, np.clip(np.rint(u), -128, 127).astype(np.int8)) and np.array_equal(s, s32)
    assert np.all(np.abs(q.astype(int)).max(axis=1) == 127) and q.min() >= -127
    qn, sn = O.smooth_quantize(-x, inv_s, act_bits=8)
    assert np.array_equal(qn, -q) and np.array_equal(sn, s)
    # uniform quantiser of step s_q: |t - s_q q| <= s_q / 2
    err = np.abs(t.astype(np.float64) - s.astype(np.float64)[:, None] * q)
    assert np.all(err <= 0.5 * s[:, None] * (1 + 1e-4))
    assert (O.smooth_quantize_ideal(x, inv_s, act_bits=8) != q).mean() < 2e-3
    # sixteen times finer than the 4-bit grid of the same row: q4 is q8 rescaled and re-rounded, up to ties
    q4, s4 = O.smooth_quantize(x, inv_s)
    assert np.abs(q4.astype(np.float64) - q.astype(np.float64) * 7.0 / 127.0).max() <= 0.5 + 7.0 / 127.0


def test_lookup_forms_agree_for_8bit_levels_and_known_values():
    rng = np.random.default_rng(13)
    N, K, C, M = 6, 40, 4, 3
    idx = rng.integers(0, C, size=(N, K), dtype=np.uint8)
    cb = rng.standard_normal((N, C)).astype(np.float16)
    q = rng.integers(-128, 128, size=(M, K)).astype(np.int8)
    q[0, :3] = (-128, 127, 0)
    s_q = (rng.random(M) + 0.1).astype(np.float32)
    ref = (q.astype(np.float64) @ cb.astype(np.float64)[np.arange(N)[:, None], idx].T) * s_q.astype(np.float64)[:, None]
    for f in (O.lut_linear_dequant, O.lut_linear_loops, O.lut_linear_bucket):
        np.testing.assert_allclose(f(idx, cb, q, s_q), ref, rtol=1e-12, atol=1e-12)
    for f in (O.lut_linear_product, O.lut_linear_signfold):      # 256 x C and 129 x C tables
        np.testing.assert_allclose(f(idx, cb, q, s_q, act_bits=8), ref, rtol=1e-12, atol=1e-12)
    # a 4-bit-sized table cannot hold these levels: the width is part of the definition
    with pytest.raises(IndexError):
        O.lut_linear_signfold(idx, cb, q, s_q, act_bits=4)
    # one weight, one column: y = s_q * q * cb
    y = O.lut_linear_product(np.array([[1]], dtype=np.uint8), np.array([[0.5, -2.0]], dtype=np.float16),
                             np.array([[-128]], dtype=np.int8), np.array([0.5], dtype=np.float32), act_bits=8)
    assert y[0, 0] == 0.5 * -128 * -2.0


def test_act8_padding():
    q = np.arange(-128, 128, dtype=np.int8).reshape(1, 256)[:, :200]
    p = O.pad_act8(q)
    assert p.shape == (1, 256) and p.dtype == np.int8 and np.array_equal(p[:, :200], q) and not p[:, 200:].any()


# ---------------------------------------------------------------- adaptive smoothing search (Section 3.4)
def test_smoothing_factors_closed_forms_and_clamps():
    xmax = np.array([4.0, 9.0, 0.0, 1e12, 1e-12, 2.0])
    wmax = np.array([1.0, 4.0, 3.0, 1e-12, 1e12, 0.0])
    s0 = O.smoothing_factors(xmax, wmax, 0.0)       # alpha = 0: 1 / wmax
    s1 = O.smoothing_factors(xmax, wmax, 1.0)       # alpha = 1: xmax
    sh = O.smoothing_factors(xmax, wmax, 0.5)       # alpha = 1/2: sqrt(xmax / wmax)
    assert s0[:2].tolist() == [1.0, 0.25] and s1[:2].tolist() == [4.0, 9.0] and sh[:2].tolist() == [2.0, 1.5]
    assert sh[2] == 1.0 and sh[5] == 1.0            # a zero maximum leaves the channel alone
    assert sh[3] == np.float32(1e5) and sh[4] == np.float32(1e-5)


def test_smoothing_mse_zero_when_representable_and_matches_loops():
    # integers up to 127 with a 127 in every row are their own 8-bit levels: no error at s = 1 ...
    rng = np.random.default_rng(21)
    x = rng.integers(-127, 128, size=(5, 64)).astype(np.float16)
    x[:, 0] = 127
    assert O.smoothing_mse(x, np.ones(64, dtype=np.float32)) == 0.0
    # ... and at any power-of-two s (division and multiplication are exact)
    assert O.smoothing_mse(x, np.full(64, 4.0, dtype=np.float32)) == 0.0
    # brute force on a small case
    x = (rng.standard_normal((3, 10)) * 5).astype(np.float16)
    s = (rng.random(10) + 0.5).astype(np.float32)
    tot = 0.0
    for t in range(3):
        tv = [np.float32(x[t, k]) * (np.float32(1.0) / s[k]) for k in range(10)]
        A = max(abs(v) for v in tv)
        for k in range(10):
            lev = float(np.clip(np.rint(np.float32(tv[k] * (np.float32(127.0) / A))), -128, 127))
            rec = lev * float(np.float32(A / np.float32(127.0))) * float(s[k])
            tot += (float(x[t, k]) - rec) ** 2
    assert abs(O.smoothing_mse(x, s) - tot / 30) <= 1e-15 * max(1.0, tot)


def test_smoothing_search_prefers_taming_outlier_channels():
    # a few channels 50x larger than the rest: without smoothing (alpha = 0, equal weights) the 8-bit step is set by
    # the outliers and the small channels lose their resolution; alpha = 1 equalises the channels completely
    rng = np.random.default_rng(22)
    T, K = 64, 256
    x = rng.standard_normal((T, K))
    x[:, ::32] *= 50.0
    x = x.astype(np.float16)
    wmax = np.ones(K)
    alphas = [0.0, 0.25, 0.5, 0.75, 1.0]
    best, mse = O.smoothing_search(x, wmax, alphas)
    assert best >= 2 and mse[best] < 0.5 * mse[0]
    # uniform 8-bit quantiser noise of step d is about d^2 / 12: at alpha = 0 (s = 1) the step of a token is A / 127
    A = np.abs(x.astype(np.float64)).max(axis=1)
    expect = ((A / 127.0) ** 2 / 12.0).mean()
    assert 0.8 * expect < mse[0] < 1.2 * expect
    # scaling X and the factors by a power of two scales the error by its square
    s = O.smoothing_factors(np.abs(x.astype(np.float64)).max(axis=0), wmax, 0.5)
    m1 = O.smoothing_mse(x, s)
    m2 = O.smoothing_mse((x.astype(np.float32) * 4).astype(np.float16), s)
    assert abs(m2 - 16 * m1) <= 1e-12 * m2


# ---------------------------------------------------------------- reclassification + centroid update (Section 3.2)
def test_reclassify_hand_example():
    # centroids -1, 0, 2: half-gaps 0.5 and 1
    cb = np.array([[-1.0, 0.0, 2.0]], dtype=np.float16)
    idx = np.array([[1, 1, 1, 1, 0, 0, 2, 2]], dtype=np.uint8)
    dw = np.array([[0.25, -0.5, -0.75, 1.5, -3.0, 0.75, 0.5, -1.25]], dtype=np.float32)
    new_idx, dC, cnt = O.reclassify(idx, cb, dw)
    #  0.25 stays in 1; -0.5 is not beyond -0.5: stays; -0.75 crosses to 0; 1.5 > 1 crosses to 2;
    #  -3 in the leftmost cluster has no left side: stays; 0.75 > 0.5 crosses to 1; 0.5 in the rightmost: stays;
    #  -1.25 < -1 crosses to 1
    assert new_idx.tolist() == [[1, 1, 0, 2, 0, 1, 2, 1]]
    assert cnt.tolist() == [[2, 4, 2]]
    # cluster 0: stays -3, arrival from 1: (0 - -1) + -0.75 = 0.25             -> -2.75
    # cluster 1: stays 0.25 - 0.5, from 0: (-1 - 0) + 0.75, from 2: (2 - 0) - 1.25 -> -0.25 - 0.25 + 0.75 = 0.25
    # cluster 2: stays 0.5, arrival from 1: (0 - 2) + 1.5 = -0.5                -> 0.0
    assert dC.tolist() == [[-2.75, 0.25, 0.0]]


def test_reclassify_invariants_and_brute_force():
    rng = np.random.default_rng(31)
    N, K, C = 7, 300, 5
    cb = np.sort(rng.standard_normal((N, C)), axis=1).astype(np.float16)
    idx = rng.integers(0, C, size=(N, K), dtype=np.uint8)
    dw = (rng.standard_normal((N, K)) * 0.4).astype(np.float32)
    new_idx, dC, cnt = O.reclassify(idx, cb, dw)
    assert np.all(np.abs(new_idx.astype(int) - idx.astype(int)) <= 1) and new_idx.max() < C
    assert np.all(cnt.sum(axis=1) == K)
    # zero updates change nothing
    z_idx, z_dC, z_cnt = O.reclassify(idx, cb, np.zeros_like(dw))
    assert np.array_equal(z_idx, idx) and not z_dC.any()
    # the offsets of a row add up to: sum of updates + sum over moved weights of (old centroid - new centroid)
    cbd = cb.astype(np.float64)
    for n in range(N):
        moved = cbd[n][idx[n]] - cbd[n][new_idx[n]]
        assert abs(dC[n].sum() - (dw[n].astype(np.float64).sum() + moved.sum())) < 1e-9
    # triple loop
    bf = np.zeros((N, C))
    for n in range(N):
        for k in range(K):
            i, j = int(idx[n, k]), int(new_idx[n, k])
            if i > 0 and dw[n, k] < -np.float32((np.float32(cb[n, i]) - np.float32(cb[n, i - 1])) * np.float32(0.5)):
                assert j == i - 1
            elif i < C - 1 and dw[n, k] > np.float32((np.float32(cb[n, i + 1]) - np.float32(cb[n, i])) * np.float32(0.5)):
                assert j == i + 1
            else:
                assert j == i
            bf[n, j] += float(dw[n, k]) + (float(cb[n, i]) - float(cb[n, j]))
    np.testing.assert_allclose(dC, bf, rtol=1e-12, atol=1e-12)
    with pytest.raises(ValueError):
        O.reclassify(idx, cb[:, ::-1], dw)
    # one cluster: no neighbour, nothing moves, the offset is the sum of the updates
    one_idx, one_dC, one_cnt = O.reclassify(np.zeros((1, 5), dtype=np.uint8), np.array([[0.5]], dtype=np.float16),
                                            np.array([[1, -2, 3, 0.5, 0.25]], dtype=np.float32))
    assert not one_idx.any() and one_dC.tolist() == [[2.75]] and one_cnt.tolist() == [[5]]


# ---------------------------------------------------------------- density-based centroid initialisation (Section 3.1)
def _dbscan_brute(y, eps, min_pts):
    """Textbook DBSCAN (region queries by full scans, breadth-first expansion) on a small 1-D array."""
    m = len(y)
    nbrs = [[j for j in range(m) if abs(y[j] - y[i]) <= eps] for i in range(m)]
    core = [len(nb) >= min_pts for nb in nbrs]
    lab = [None] * m
    c = 0
    for i in range(m):
        if lab[i] is not None or not core[i]:
            continue
        lab[i] = c
        queue = list(nbrs[i])
        while queue:
            j = queue.pop()
            if lab[j] is None or lab[j] == -1:
                lab[j] = c
                if core[j]:
                    queue.extend(nbrs[j])
        c += 1
    return core, [(-1 if v is None else v) for v in lab]


def test_dbci_sigma_of_a_gaussian_and_hand_example():
    # half-normal percentiles at 68.27 / 95.44 / 99.74 % are 1, 2, 3 sigma: six of them sum to 12 sigma
    rng = np.random.default_rng(41)
    w = (rng.standard_normal(200000) * 0.02).astype(np.float32)
    r = O.dbci_scan(w)         # 200000 weights: the n log n form (checked against the plain one below)
    assert abs(r["sigma"] / 0.02 - 1.0) < 0.02
    assert r["min_pts"] == min(r["left"], r["right"]) and r["eps"] == r["sigma"] / r["min_pts"]
    assert np.all(np.diff(r["centroids"]) > 0) and np.all(np.isin(r["centroids"].astype(np.float32), r["sorted"]))
    # hand example: two tight groups, two far outliers
    w = np.array([-10.0, -1.0, -0.9, -1.1, 1.0, 1.1, 0.9, 1.05, 12.0], dtype=np.float32)
    r = O.dbci(w)
    # positives 0.9 1 1.05 1.1 12 -> ranks ceil(p * 5) = 4, 5, 5 -> 1.1, 12, 12; negatives (magnitudes) 0.9 1 1.1 10
    # -> ranks 3, 4, 4 -> 1.1, 10, 10; sigma = 46.2 / 12 = 3.85
    assert abs(r["sigma"] - 46.2 / 12) < 1e-6
    assert r["left"] == 1 and r["right"] == 1 and r["min_pts"] == 1     # nothing within 3.85 of -10 or of 12
    # MinPts 1: every point is a core point, eps = sigma: the seven middle points chain into one cluster
    assert r["labels"].tolist() == [0, 1, 1, 1, 1, 1, 1, 1, 2]
    assert r["centroids"].tolist() == [-10.0, float(np.float32(0.9)), 12.0]


def test_dbci_middle_matches_textbook_dbscan():
    rng = np.random.default_rng(42)
    for trial in range(6):
        body = rng.standard_normal(300) * 0.02
        clumps = np.concatenate([0.1 + rng.standard_normal(25) * 0.001, -0.08 + rng.standard_normal(15) * 0.001])
        outl = np.array([-0.5, -0.49, -0.495, 0.6, 0.61, 0.6050])
        w = np.concatenate([body, clumps, outl, rng.uniform(-0.3, 0.3, 12)]).astype(np.float32)
        r = O.dbci(w)
        x = r["sorted"].astype(np.float64)
        L, R = r["left"], len(x) - r["right"]
        core, lab = _dbscan_brute(x[L:R], r["eps"], r["min_pts"])
        mine = r["labels"][L:R]
        core_idx = [i for i in range(R - L) if core[i]]
        # core points: same partition (cluster numbers may be permuted)
        pairs = {(lab[i], int(mine[i])) for i in core_idx}
        assert len(pairs) == len({a for a, _ in pairs}) == len({b for _, b in pairs})
        assert all(mine[i] >= 1 for i in core_idx)
        # the rest: noise exactly where the textbook says noise; a border point sits within eps of a core of its cluster
        for i in range(R - L):
            if core[i]:
                continue
            assert (mine[i] == -1) == (lab[i] == -1)
            if mine[i] != -1:
                assert any(core[j] and mine[j] == mine[i] and abs(x[L + j] - x[L + i]) <= r["eps"] for j in range(R - L))
        # clusters are contiguous in sorted order and every centroid is the lower median of its members
        labs = r["labels"]
        for c in range(int(labs.max()) + 1):
            mem = np.flatnonzero(labs == c)
            if mem.size:
                assert not np.any((labs[mem[0]:mem[-1] + 1] != c) & (labs[mem[0]:mem[-1] + 1] != -1))
        assert r["centroids"].size == len({int(v) for v in labs if v >= 0})


def test_dbci_border_point_rule_by_hand():
    # Four outliers on either side seed the two outer clusters; positives 0.95 1.05 1.15 1.25 7.97 7.98 7.99 8 ->
    # nearest ranks ceil(p * 8) = 6, 8, 8 -> 7.98 + 8 + 8, the same for the negative magnitudes:
    # sigma = 47.96 / 12 = 3.99667; each seed takes its four outliers (nothing else within sigma of -8 or 8), so
    # MinPts = 4 and eps = sigma / 4 = 0.99917.  Both groups of four are core points (four points within 0.3);
    # the point 0 sees only -0.95, itself and 0.95 (three points), so it is not a core point, and it lies
    # exactly 0.95 from the rightmost core of the left group and from the leftmost core of the right group:
    # the left cluster takes it.
    w = np.array([-8, -7.99, -7.98, -7.97, -1.25, -1.15, -1.05, -0.95, 0, 0.95, 1.05, 1.15, 1.25, 7.97, 7.98, 7.99, 8],
                 dtype=np.float32)
    for f in (O.dbci, O.dbci_scan):
        r = f(w)
        assert abs(r["sigma"] - 47.96 / 12) < 1e-6 and r["min_pts"] == 4 and abs(r["eps"] - 47.96 / 48) < 1e-6
        assert (r["left"], r["right"]) == (4, 4)
        assert r["labels"].tolist() == [0] * 4 + [1] * 5 + [2] * 4 + [3] * 4
        # lower medians: member 1 of four, member 2 of five
        assert r["centroids"].astype(np.float32).tolist() == [np.float32(v) for v in (-7.99, -1.05, 1.05, 7.98)]
    # the same with the lonely point at 0.02: nine positives, ranks ceil(p * 9) = 7, 9, 9 -> the same three values,
    # so sigma and eps are unchanged; 0.02 is 0.97 from -0.95 and 0.93 from 0.95, both within eps: the nearer,
    # right cluster takes it
    w2 = np.sort(np.where(w == 0, np.float32(0.02), w))
    for f in (O.dbci, O.dbci_scan):
        r = f(w2)
        assert r["labels"].tolist() == [0] * 4 + [1] * 4 + [2] * 5 + [3] * 4
        assert r["centroids"].astype(np.float32).tolist() == [np.float32(v) for v in (-7.99, -1.15, 1.05, 7.98)]
    # ... and a point no core point reaches is noise: 0 moved out to 3.0 (more than eps from 1.25 and from 7.97)
    w3 = np.sort(np.where(w == 0, np.float32(3.0), w))
    r = O.dbci(w3)        # nine positives again: ranks 7, 9, 9 -> 7.98 + 8 + 8, sigma and eps as before
    assert abs(r["sigma"] - 47.96 / 12) < 1e-6
    assert r["labels"].tolist() == [0] * 4 + [1] * 4 + [2] * 4 + [-1] + [3] * 4


def test_dbci_seed_clusters_by_hand():
    # every weight within sigma of the smallest one: positives 1.0 1.1 1.2, ranks ceil(p * 3) = 3, 3, 3 ->
    # sigma = 3.6 / 12 = 0.3; the left seed takes all three, the right one gives way completely, so MinPts is
    # the left count and nothing is left for DBSCAN
    for f in (O.dbci, O.dbci_scan):
        r = f(np.array([1.0, 1.1, 1.2], dtype=np.float32))
        assert abs(r["sigma"] - 0.3) < 1e-6 and (r["left"], r["right"], r["min_pts"]) == (3, 0, 3)
        assert abs(r["eps"] - 0.1) < 1e-6 and r["labels"].tolist() == [0, 0, 0]
        assert r["centroids"].astype(np.float32).tolist() == [np.float32(1.1)]
        # partial overlap: 10 12.5 13.5 16 -> ranks 3, 4, 4 -> sigma = (13.5 + 16 + 16) / 12 = 3.79167; the left seed
        # reaches 13.79 (three weights), the right one 12.21 (three weights): 12.5 and 13.5 stay with the left
        r = f(np.array([10, 12.5, 13.5, 16], dtype=np.float32))
        assert abs(r["sigma"] - 45.5 / 12) < 1e-9 and (r["left"], r["right"], r["min_pts"]) == (3, 1, 1)
        assert r["labels"].tolist() == [0, 0, 0, 1] and r["centroids"].tolist() == [12.5, 16.0]
        # a single weight
        r = f(np.array([0.25], dtype=np.float32))
        assert (r["left"], r["right"], r["min_pts"]) == (1, 0, 1) and r["labels"].tolist() == [0]


def test_dbci_scan_form_equals_plain_form():
    # the n log n form used for large inputs against the plain one, on inputs with many exact ties (values on a
    # grid), clumps, one-sided data and uniform noise
    rng = np.random.default_rng(7)
    for trial in range(40):
        kind = trial % 4
        if kind == 0:
            w = np.round(rng.standard_normal(400) * 0.02, 3)
            w = np.concatenate([w, [-0.5, -0.499, 0.6, 0.601, 0.602]])
        elif kind == 1:
            w = np.concatenate([rng.standard_normal(300) * 0.02, 0.1 + rng.standard_normal(25) * 0.001,
                                rng.uniform(-0.3, 0.3, 20), [-0.5, -0.49, -0.495, 0.6, 0.61, 0.605]])
        elif kind == 2:
            w = np.abs(np.round(rng.standard_normal(300) * 0.02, 3)) + 0.001
        else:
            w = np.round(rng.uniform(-1, 1, 200), 2)
        a, b = O.dbci(w.astype(np.float32)), O.dbci_scan(w.astype(np.float32))
        assert (a["sigma"], a["eps"], a["min_pts"], a["left"], a["right"]) == (b["sigma"], b["eps"], b["min_pts"], b["left"], b["right"])
        assert np.array_equal(a["labels"], b["labels"]) and np.array_equal(a["centroids"], b["centroids"])
