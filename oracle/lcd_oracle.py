"""CPU oracle for the LUT-based inference matmul of the LCD paper (Section 4,
"Inference with Table Lookup").

TEST INFRASTRUCTURE ONLY.  Plain, slow, double-precision numpy written from the paper;
it shares no code with the CUDA path and must never be imported by the product package.
Only the tests, the smoke check and the benchmark's CPU-baseline leg may call it.

What is implemented, and which passage each part follows:

* ``smooth_quantize``      Section 4.1 "Input Transformation Stage", both equations:
                           smoothing and uniform symmetric quantisation fused into a single
                           multiply, round to nearest, clip.  (An *encoding*: taken step by
                           step in a fixed binary32 operation order, see the function.)
* ``lut_linear_dequant``   the plain definition the method reaches exactly: dequantise the
                           clustered weights and the quantised activations and multiply
                           (Section 4.2: the looked-up values are "pre-computed" products
                           that are then summed; no dequantisation pass changes the value).
* ``lut_linear_product``   Section 4.2 first paragraph: a table of pre-computed
                           (activation level x weight centroid) products, read by index pair
                           and accumulated.
* ``lut_linear_signfold``  Section 4.2 third paragraph, last sentence: only non-negative
                           activation levels are stored, the sign is applied when accumulating.
* ``lut_linear_bucket``    Section 4.2 third paragraph: centroid-stationary buckets - per
                           weight centroid, gather what belongs to it, then combine with the
                           centroid values.
* ``pack_weights`` / ``unpack_weights``  Section 4.2 last paragraph (fewer than 16
                           centroids => low-bit index representation); the byte layout is this
                           library's own and is specified in the function docstrings.

Parity pins (tests/test_oracle_pins.py): the four linear forms agree with each other and
with a brute-force triple loop, with a float64 library matmul on the dequantised matrix,
with closed forms for one-centroid and affine codebooks and with exhaustive enumeration on
tiny inputs.  The paper prints no numeric example of this path, so the quantiser's tie rule
(half to even) and the absmax/7 scale are pinned by invariants only (sign symmetry,
power-of-two scale invariance, monotonicity, exact ties): "parity unpinned" against paper
values for those two choices of ``smooth_quantize``.
"""
from __future__ import annotations

import struct
import numpy as np

QMIN, QMAX = -8, 7            # 4-bit symmetric range [-2^(b-1), 2^(b-1)-1], b = 4
LEVELS = 16


def act_range(act_bits: int):
    """(qmin, qmax) = (-2^(b-1), 2^(b-1)-1) of Section 4.1's clip for b-bit activations (b = 4 or 8)."""
    if act_bits not in (4, 8):
        raise ValueError("act_bits must be 4 or 8")
    return -(1 << (act_bits - 1)), (1 << (act_bits - 1)) - 1
MAGIC = 0x5744434C            # "LCDW"
VERSION = 1
LAYOUT_PAIR16X256 = 2
HEADER_BYTES = 64
INDEX_OFFSET = 256
TILE_ROWS = 8              # rows of one tile
PAIR_ROWS = 16             # two tiles (rows 0-7, rows 8-15) form one 16-row item
TILE_K = 256
KBLOCK = 128


def _f32(v):
    """Round a float64 array to binary32 and return it as float64 (one IEEE rounding)."""
    return np.asarray(v, dtype=np.float64).astype(np.float32).astype(np.float64)


def round_up(v: int, m: int) -> int:
    return (v + m - 1) // m * m


# --------------------------------------------------------------------------------------
# Section 4.1 - input transformation
# --------------------------------------------------------------------------------------
def smooth_quantize(x_fp16: np.ndarray, inv_s: np.ndarray | None, static_scale: float | None = None,
                    act_bits: int = 4):
    """Activation index assignment, Section 4.1.

    q = Clip(round(X / (s_m * s_q))): the smoothing divide and the quantisation divide are one
    multiply.  Per token m (dynamic mode, static_scale is None):
        t_k = fl32(x_k * inv_s_k)            inv_s_k = 1/s_k given as binary32
        A   = max_k |t_k|
        A == 0:  s_q = 1, q = 0
        else     s_q = fl32(A / 7),  r = fl32(7 / A),  u_k = fl32(t_k * r)
        q_k = clip(round_half_even(u_k), -8, 7)
    Static mode (the paper's literal form: s_q fixed offline): the caller passes
    f_k = 1/(s_k*s_q) as ``inv_s`` and s_q as ``static_scale``;  q_k = clip(rhe(fl32(x_k*f_k))).
    Every product of two binary32 values is exact in binary64 and a binary32 quotient obtained
    through one binary64 division rounds identically (53 >= 2*24+2), so casting to binary32 after
    each step reproduces IEEE binary32 arithmetic exactly.

    With act_bits = 8 (the paper's b = 8) the same steps run with 127 in place of 7 and the clip range
    [-128, 127].

    Returns (q int8 [M,K], s_q float32 [M]).
    """
    qmin, qmax = act_range(act_bits)
    top = float(qmax)
    x = np.asarray(x_fp16, dtype=np.float16).astype(np.float64)
    M, K = x.shape
    f = np.ones(K) if inv_s is None else np.asarray(inv_s, dtype=np.float32).astype(np.float64)
    t = _f32(x * f[None, :])
    if static_scale is not None:
        q = np.clip(np.rint(t), qmin, qmax).astype(np.int8)
        return q, np.full(M, np.float32(static_scale), dtype=np.float32)
    A = np.abs(t).max(axis=1) if K else np.zeros(M)
    s_q = np.ones(M, dtype=np.float64)
    r = np.zeros(M, dtype=np.float64)
    nz = A > 0
    s_q[nz] = _f32(A[nz] / top)
    r[nz] = _f32(top / A[nz])
    u = _f32(t * r[:, None])
    q = np.clip(np.rint(u), qmin, qmax).astype(np.int8)   # np.rint rounds half to even
    return q, s_q.astype(np.float32)


def smooth_quantize_ideal(x_fp16, inv_s, act_bits: int = 4):
    """The same assignment in unrounded real arithmetic (binary64): x/(s_k*s_q) with s_q = A/7.
    Differs from ``smooth_quantize`` only where the pre-rounding value sits within a few binary32
    ulps of a half-integer; used to count such positions, never as an expected value."""
    x = np.asarray(x_fp16, dtype=np.float16).astype(np.float64)
    f = np.ones(x.shape[1]) if inv_s is None else np.asarray(inv_s, dtype=np.float32).astype(np.float64)
    t = x * f[None, :]
    A = np.abs(t).max(axis=1)
    qmin, qmax = act_range(act_bits)
    u = np.where(A[:, None] > 0, t * float(qmax) / np.where(A > 0, A, 1.0)[:, None], 0.0)
    return np.clip(np.rint(u), qmin, qmax).astype(np.int8)


def pack_act(q: np.ndarray, K_pad: int | None = None) -> np.ndarray:
    """Activation indices a = q + 8 in [0,15], two per byte (even k in the low nibble), row padded
    to K_pad (multiple of 256) with a = 8 (q = 0)."""
    M, K = q.shape
    K_pad = round_up(K, TILE_K) if K_pad is None else K_pad
    a = np.full((M, K_pad), 8, dtype=np.uint8)
    a[:, :K] = (q.astype(np.int16) + 8).astype(np.uint8)
    return (a[:, 0::2] | (a[:, 1::2] << 4)).astype(np.uint8)


def pad_act8(q: np.ndarray, K_pad: int | None = None) -> np.ndarray:
    """8-bit activation levels as stored for the lookup: one signed byte per column, row padded to K_pad
    (multiple of 256) with zeros."""
    M, K = q.shape
    K_pad = round_up(K, TILE_K) if K_pad is None else K_pad
    out = np.zeros((M, K_pad), dtype=np.int8)
    out[:, :K] = q
    return out


def unpack_act(packed: np.ndarray, K: int) -> np.ndarray:
    M = packed.shape[0]
    a = np.empty((M, packed.shape[1] * 2), dtype=np.int16)
    a[:, 0::2] = packed & 0xF
    a[:, 1::2] = packed >> 4
    return (a[:, :K] - 8).astype(np.int8)


# --------------------------------------------------------------------------------------
# Section 4.2 - lookup and accumulation, four equivalent statements
# --------------------------------------------------------------------------------------
def dequantize(idx: np.ndarray, codebook_fp16: np.ndarray) -> np.ndarray:
    """W_q[n][k] = codebook[n][idx[n][k]] as float64."""
    cb = np.asarray(codebook_fp16, dtype=np.float16).astype(np.float64)
    return np.take_along_axis(cb, idx.astype(np.int64), axis=1)


def lut_linear_dequant(idx, codebook_fp16, q, s_q) -> np.ndarray:
    """y[m][n] = s_q[m] * sum_k q[m][k] * cb[n][idx[n][k]]   (float64, library matmul as the sum)."""
    Wq = dequantize(idx, codebook_fp16)
    acc = q.astype(np.float64) @ Wq.T
    return np.asarray(s_q, dtype=np.float64)[:, None] * acc


def lut_linear_loops(idx, codebook_fp16, q, s_q) -> np.ndarray:
    """The same definition as an explicit triple loop, k ascending (tiny inputs only)."""
    cb = np.asarray(codebook_fp16, dtype=np.float16).astype(np.float64)
    M, K = q.shape
    N = idx.shape[0]
    y = np.zeros((M, N))
    for m in range(M):
        for n in range(N):
            acc = 0.0
            for k in range(K):
                acc += float(q[m, k]) * cb[n, idx[n, k]]
            y[m, n] = float(s_q[m]) * acc
    return y


def lut_linear_product(idx, codebook_fp16, q, s_q, act_bits: int = 4) -> np.ndarray:
    """Product table: T_{m,n}[a][w] = ((a + qmin) * s_q[m]) * cb[n][w];  y[m][n] = sum_k T[a_k][idx_k], with the
    activation index a = q - qmin in [0, 2^b) (16 rows for b = 4, 256 for b = 8)."""
    cb = np.asarray(codebook_fp16, dtype=np.float16).astype(np.float64)
    M, K = q.shape
    N, C = cb.shape
    qmin, _ = act_range(act_bits)
    a = q.astype(np.int64) - qmin
    levels = np.arange(1 << act_bits, dtype=np.float64) + float(qmin)
    y = np.zeros((M, N))
    ii = idx.astype(np.int64)
    for m in range(M):
        act_val = levels * float(s_q[m])                  # 16 activation values of this token
        for n in range(N):
            T = act_val[:, None] * cb[n][None, :]         # 16 x C table
            y[m, n] = T[a[m], ii[n]].sum()
    return y


def lut_linear_signfold(idx, codebook_fp16, q, s_q, act_bits: int = 4) -> np.ndarray:
    """Only |q| in [0, 2^(b-1)] is tabulated (9 rows for b = 4, 129 for b = 8):
    T+[|q|][w] = (|q| * s_q) * cb[w]; y = sum_k sgn(q_k) * T+[|q_k|][idx_k]."""
    cb = np.asarray(codebook_fp16, dtype=np.float16).astype(np.float64)
    M, K = q.shape
    N, C = cb.shape
    mag = np.abs(q.astype(np.int64))
    sgn = np.sign(q.astype(np.int64)).astype(np.float64)
    y = np.zeros((M, N))
    ii = idx.astype(np.int64)
    for m in range(M):
        lev = np.arange((1 << (act_bits - 1)) + 1, dtype=np.float64) * float(s_q[m])
        for n in range(N):
            Tp = lev[:, None] * cb[n][None, :]            # 9 x C
            y[m, n] = (sgn[m] * Tp[mag[m], ii[n]]).sum()
    return y


def bucket_sums(idx, q, C: int) -> np.ndarray:
    """S[m][n][w] = sum over {k : idx[n][k] == w} of q[m][k]   (exact int64)."""
    M, K = q.shape
    N = idx.shape[0]
    S = np.zeros((M, N, C), dtype=np.int64)
    q64 = q.astype(np.int64)
    for w in range(C):
        mask = (idx == w).astype(np.int64)                # N x K
        S[:, :, w] = q64 @ mask.T
    return S


def lut_linear_bucket(idx, codebook_fp16, q, s_q) -> np.ndarray:
    """Centroid-stationary form: y[m][n] = s_q[m] * sum_w cb[n][w] * S[m][n][w]."""
    cb = np.asarray(codebook_fp16, dtype=np.float16).astype(np.float64)
    S = bucket_sums(idx, q, cb.shape[1]).astype(np.float64)
    return np.asarray(s_q, dtype=np.float64)[:, None] * np.einsum("mnw,nw->mn", S, cb)


def lut_linear_rows(idx, codebook_fp16, q, s_q, rows: np.ndarray) -> np.ndarray:
    """Dequant form restricted to a sample of output rows (for spot checks at full size)."""
    return lut_linear_dequant(idx[rows], np.asarray(codebook_fp16)[rows], q, s_q)


# --------------------------------------------------------------------------------------
# Packed-weight blob (layout id 2, "pair16x256")
# --------------------------------------------------------------------------------------
def packed_weights_bytes(N: int, K: int, bits: int) -> int:
    N_pad, K_pad = round_up(N, PAIR_ROWS), round_up(K, TILE_K)
    idx_bytes = N_pad * K_pad * bits // 8
    cb_off = round_up(INDEX_OFFSET + idx_bytes, 256)
    return cb_off + round_up(N_pad * (1 << bits) * 2, 256)


def _tile_lane_bytes_2bit(rows_idx: np.ndarray, g: int, t: int) -> np.ndarray:
    """16 bytes of lane (g,t) of one 2-bit tile.  rows_idx: [8][256] indices of the tile."""
    out = np.zeros(16, dtype=np.uint8)
    for half in range(2):                 # k-block 0 / 1 of the tile
        for p in range(8):                # byte position inside the 8-byte quarter record
            G = 8 * t + p                 # k-group (4 consecutive k) inside the k-block
            b = 0
            for i in range(4):
                k = KBLOCK * half + 4 * G + i
                b |= int(rows_idx[g, k]) << (2 * i)
            out[8 * half + p] = b
    return out


def _record_3bit(v32: np.ndarray) -> np.ndarray:
    """12-byte record of 32 three-bit indices v32[0..31]: words 0..2 carry indices 8i+j in bits
    [4j,4j+3); index 24+j has bit b stored at bit 4j+3 of word b."""
    words = [0, 0, 0]
    for i in range(3):
        for j in range(8):
            words[i] |= int(v32[8 * i + j]) << (4 * j)
    for j in range(8):
        v = int(v32[24 + j])
        for b in range(3):
            words[b] |= ((v >> b) & 1) << (4 * j + 3)
    return np.frombuffer(struct.pack("<3I", *words), dtype=np.uint8)


def pack_weights(idx: np.ndarray, codebook_fp16: np.ndarray, bits: int, C: int | None = None) -> np.ndarray:
    """Build the blob (uint8 array).

    Header, 64 bytes little-endian:  u32 magic "LCDW", u32 version=1, u64 N, u64 K, u64 K_pad,
    u32 bits, u32 C, u32 layout=2, u32 checksum (sum of all payload bytes mod 2^32),
    u64 index_offset (=256), u64 codebook_offset.  Bytes 64..255 are zero.

    Index area: rows padded to N_pad = 16*ceil(N/16), columns to K_pad = 256*ceil(K/256), padding
    index 0.  Tiles of 8 rows x 256 columns of T = 512 (2 bit), 768 (3 bit) or 1024 bytes (4 bit); the two
    tiles of a 16-row group rp (rows 16rp..16rp+7, then 16rp+8..16rp+15) are adjacent and form one
    item: tile (rg, kt), rg = 2*rp + u, is at index_offset + (rp*(K_pad/256) + kt)*2T + u*T.
    Lane l = 4*g + t (g = 0..7 row inside the tile, t = 0..3 quarter) owns, for each of the tile's
    two 128-column k-blocks h, the 32 columns 128*h + 32*t .. +31 of row g.
      2 bit: lane record = 16 bytes at tile + 16*l: bytes [8h, 8h+8) are k-block h.  Byte p of those
             holds columns 128h + 32t + 4p + i at bits [2i, 2i+2) (plain little-endian packing).
      3 bit: the tile is three 256-byte planes; plane b holds, at plane + 8*l, word b of the lane's
             record for k-block 0 then word b of its record for k-block 1.  A record packs the 32
             columns 128h + 32t + m: m = 8i+j (i<3) in bits [4j,4j+3) of word i; m = 24+j has its bit b
             at bit 4j+3 of word b.
      4 bit: the tile is two 512-byte planes, one per k-block h; plane h holds, at plane + 16*l, the lane's
             16 bytes, byte p of which packs the columns 128h + 32t + 2p (low nibble) and 128h + 32t + 2p + 1.
    Codebook area: N_pad rows of 2^bits fp16 values (entries >= C and padded rows are zero).
    """
    idx = np.asarray(idx, dtype=np.uint8)
    N, K = idx.shape
    C = (1 << bits) if C is None else C
    if bits not in (2, 3, 4) or not (1 <= C <= (1 << bits)):
        raise ValueError("bits/C")
    if idx.size and int(idx.max()) >= C:
        raise ValueError("index out of range")
    cb = np.asarray(codebook_fp16, dtype=np.float16)
    assert cb.shape == (N, C)
    N_pad, K_pad = round_up(N, PAIR_ROWS), round_up(K, TILE_K)
    total = packed_weights_bytes(N, K, bits)
    blob = np.zeros(total, dtype=np.uint8)
    P = np.zeros((N_pad, K_pad), dtype=np.uint8)
    P[:N, :K] = idx
    tile_bytes = TILE_ROWS * TILE_K * bits // 8
    n_kt = K_pad // TILE_K
    for rg in range(N_pad // TILE_ROWS):
        for kt in range(n_kt):
            sub = P[rg * 8:(rg + 1) * 8, kt * TILE_K:(kt + 1) * TILE_K]
            base = INDEX_OFFSET + ((rg // 2) * n_kt + kt) * 2 * tile_bytes + (rg % 2) * tile_bytes
            for g in range(8):
                for t in range(4):
                    lane = 4 * g + t
                    if bits == 2:
                        blob[base + 16 * lane: base + 16 * lane + 16] = _tile_lane_bytes_2bit(sub, g, t)
                    elif bits == 4:
                        for h in range(2):
                            for p in range(16):
                                k = KBLOCK * h + 32 * t + 2 * p
                                blob[base + 512 * h + 16 * lane + p] = int(sub[g, k]) | (int(sub[g, k + 1]) << 4)
                    else:
                        for h in range(2):
                            rec = _record_3bit(sub[g, KBLOCK * h + 32 * t: KBLOCK * h + 32 * t + 32])
                            for b in range(3):
                                o = base + 256 * b + 8 * lane + 4 * h
                                blob[o:o + 4] = rec[4 * b:4 * b + 4]
    cb_off = round_up(INDEX_OFFSET + N_pad * K_pad * bits // 8, 256)
    cbp = np.zeros((N_pad, 1 << bits), dtype=np.float16)
    cbp[:N, :C] = cb
    blob[cb_off:cb_off + cbp.size * 2] = cbp.view(np.uint8).reshape(-1)
    checksum = int(blob[HEADER_BYTES:].astype(np.uint64).sum()) & 0xFFFFFFFF
    hdr = struct.pack("<IIQQQIIIIQQ", MAGIC, VERSION, N, K, K_pad, bits, C, LAYOUT_PAIR16X256, checksum,
                      INDEX_OFFSET, cb_off)
    assert len(hdr) == HEADER_BYTES
    blob[:HEADER_BYTES] = np.frombuffer(hdr, dtype=np.uint8)
    return blob


def parse_header(blob: np.ndarray) -> dict:
    f = struct.unpack("<IIQQQIIIIQQ", bytes(blob[:HEADER_BYTES]))
    keys = ("magic", "version", "N", "K", "K_pad", "bits", "C", "layout", "checksum", "index_offset",
            "codebook_offset")
    return dict(zip(keys, f))


def unpack_weights(blob: np.ndarray):
    """Exact inverse of ``pack_weights``: returns (idx uint8 [N,K], codebook fp16 [N,C], bits, C)."""
    h = parse_header(blob)
    if h["magic"] != MAGIC or h["version"] != VERSION or h["layout"] != LAYOUT_PAIR16X256:
        raise ValueError("bad blob header")
    if (int(blob[HEADER_BYTES:].astype(np.uint64).sum()) & 0xFFFFFFFF) != h["checksum"]:
        raise ValueError("bad blob checksum")
    N, K, K_pad, bits, C = h["N"], h["K"], h["K_pad"], h["bits"], h["C"]
    N_pad = round_up(N, PAIR_ROWS)
    tile_bytes = TILE_ROWS * TILE_K * bits // 8
    n_kt = K_pad // TILE_K
    P = np.zeros((N_pad, K_pad), dtype=np.uint8)
    for rg in range(N_pad // TILE_ROWS):
        for kt in range(n_kt):
            base = h["index_offset"] + ((rg // 2) * n_kt + kt) * 2 * tile_bytes + (rg % 2) * tile_bytes
            for g in range(8):
                for t in range(4):
                    lane = 4 * g + t
                    for hb in range(2):
                        k0 = kt * TILE_K + KBLOCK * hb
                        if bits == 2:
                            for p in range(8):
                                G = 8 * t + p
                                b = int(blob[base + 16 * lane + 8 * hb + p])
                                for i in range(4):
                                    P[rg * 8 + g, k0 + 4 * G + i] = (b >> (2 * i)) & 3
                        elif bits == 4:
                            for p in range(16):
                                b = int(blob[base + 512 * hb + 16 * lane + p])
                                P[rg * 8 + g, k0 + 32 * t + 2 * p] = b & 15
                                P[rg * 8 + g, k0 + 32 * t + 2 * p + 1] = b >> 4
                        else:
                            words = []
                            for b in range(3):
                                o = base + 256 * b + 8 * lane + 4 * hb
                                words.append(struct.unpack("<I", bytes(blob[o:o + 4]))[0])
                            for m in range(32):
                                if m < 24:
                                    v = (words[m // 8] >> (4 * (m % 8))) & 7
                                else:
                                    j = m - 24
                                    v = sum(((words[b] >> (4 * j + 3)) & 1) << b for b in range(3))
                                P[rg * 8 + g, k0 + 32 * t + m] = v
    cbp = blob[h["codebook_offset"]:h["codebook_offset"] + N_pad * (1 << bits) * 2].view(np.float16)
    cbp = cbp.reshape(N_pad, 1 << bits)
    return P[:N, :K].copy(), cbp[:N, :C].copy(), bits, C


# --------------------------------------------------------------------------------------
# Section 3.4 - adaptive smoothing search (offline; needs only a calibration batch)
# --------------------------------------------------------------------------------------
def smoothing_factors(xmax, wmax, alpha: float) -> np.ndarray:
    """Per-input-channel smoothing factors for migration strength alpha:
    s_k = xmax_k^alpha / wmax_k^(1-alpha), clamped to [1e-5, 1e5]; a channel whose activation or weight maximum
    is zero keeps s_k = 1.  Computed in binary64 and rounded once to binary32 (what the kernels consume)."""
    xm = np.asarray(xmax, dtype=np.float64)
    wm = np.asarray(wmax, dtype=np.float64)
    ok = (xm > 0) & (wm > 0)
    s = np.ones_like(xm)
    s[ok] = np.power(xm[ok], alpha) / np.power(wm[ok], 1.0 - alpha)
    return np.clip(s, 1e-5, 1e5).astype(np.float32)


def smoothing_mse(x_fp16, s) -> float:
    """The objective of Section 3.4 for one candidate: MSE(X, Q_INT8(X / s) * s) over a calibration batch X [T,K],
    with Q_INT8 the symmetric per-token 8-bit quantiser of Section 4.1 (scale A/127, round half to even).
    The level decision is taken in binary32 exactly as ``smooth_quantize`` does (t = x * fl32(1/s)); the
    reconstruction and the mean are binary64."""
    x = np.asarray(x_fp16, dtype=np.float16)
    s32 = np.asarray(s, dtype=np.float32)
    inv = (np.float32(1.0) / s32).astype(np.float32)
    q, s_q = smooth_quantize(x, inv, act_bits=8)
    rec = q.astype(np.float64) * s_q.astype(np.float64)[:, None] * s32.astype(np.float64)[None, :]
    d = x.astype(np.float64) - rec
    return float((d * d).mean())


def smoothing_search(x_fp16, wmax, alphas):
    """Grid search of Section 3.4: the activation maxima are taken over the calibration batch itself; returns
    (index of the best alpha, the MSE of every candidate).  Ties go to the first candidate."""
    x = np.asarray(x_fp16, dtype=np.float16)
    xmax = np.abs(x.astype(np.float64)).max(axis=0)
    mse = np.array([smoothing_mse(x, smoothing_factors(xmax, wmax, float(a))) for a in alphas])
    return int(np.argmin(mse)), mse


# --------------------------------------------------------------------------------------
# Section 3.2 - reclassification of weights and centroid update (offline; mechanics only)
# --------------------------------------------------------------------------------------
def reclassify(idx, codebook_fp16, delta_w):
    """One round of Section 3.2's bookkeeping for per-row codebooks sorted in ascending order.

    For a weight in cluster i with update dw:  d_left = (C_i - C_{i-1}) / 2,  d_right = (C_{i+1} - C_i) / 2
    (binary32: one subtraction, one halving); it moves to cluster i - 1 when dw < -d_left (the update carries it
    across the half-way point to the left neighbour), to i + 1 when dw > d_right, edge clusters have one side only.
    Centroid offset, as printed:  dC_i = sum over weights that stay in i of dw
                                      + sum over weights that arrive from i + 1 of ((C_{i+1} - C_i) + dw)
                                      + sum over weights that arrive from i - 1 of ((C_{i-1} - C_i) + dw).
    Returns (new_idx uint8 [N,K], dC float64 [N,C], count int64 [N,C] = members after the move)."""
    idx = np.asarray(idx, dtype=np.uint8)
    cb32 = np.asarray(codebook_fp16, dtype=np.float16).astype(np.float32)
    dw = np.asarray(delta_w, dtype=np.float32)
    N, K = idx.shape
    C = cb32.shape[1]
    if np.any(np.diff(cb32.astype(np.float64), axis=1) < 0):
        raise ValueError("codebook rows must be sorted in ascending order")
    half = ((cb32[:, 1:] - cb32[:, :-1]).astype(np.float32) * np.float32(0.5)).astype(np.float32)   # [N, C-1]
    new_idx = idx.copy()
    dC = np.zeros((N, C))
    cnt = np.zeros((N, C), dtype=np.int64)
    cb = cb32.astype(np.float64)
    for n in range(N):
        i = idx[n].astype(np.int64)
        hp = np.concatenate([half[n], np.array([np.inf], dtype=np.float32)])   # a single cluster has no half-gap
        d_left = np.where(i > 0, hp[np.maximum(i - 1, 0)], np.float32(np.inf)).astype(np.float32)
        d_right = np.where(i < C - 1, hp[np.minimum(i, max(C - 2, 0))], np.float32(np.inf)).astype(np.float32)
        go_left = dw[n] < -d_left
        go_right = (dw[n] > d_right) & ~go_left
        j = i - go_left.astype(np.int64) + go_right.astype(np.int64)
        new_idx[n] = j.astype(np.uint8)
        contrib = dw[n].astype(np.float64) + (cb[n][i] - cb[n][j])
        dC[n] = np.bincount(j, weights=contrib, minlength=C)
        cnt[n] = np.bincount(j, minlength=C)
    return new_idx, dC, cnt


# --------------------------------------------------------------------------------------
# Section 3.1 - density-based centroid initialisation (DBCI), offline
# --------------------------------------------------------------------------------------
DBCI_PERCENTILES = (0.6827, 0.9544, 0.9974)      # the 1, 2 and 3 sigma ranges of a half-normal


def _nearest_rank(sorted_vals: np.ndarray, p: float) -> float:
    """Value at percentile p of an ascending array by the nearest-rank rule, 0 for an empty array."""
    if sorted_vals.size == 0:
        return 0.0
    k = int(np.ceil(p * sorted_vals.size)) - 1
    return float(sorted_vals[min(max(k, 0), sorted_vals.size - 1)])


def _dbci_seeds(xd: np.ndarray):
    """Steps 2-4 on the sorted binary64 copy of the weights: sigma, the two seed clusters as index ranges
    [0, L) and [R, n), MinPts and eps."""
    n = xd.size
    pos = xd[xd > 0]
    neg = -xd[xd < 0][::-1]
    sigma = sum(_nearest_rank(pos, p) + _nearest_rank(neg, p) for p in DBCI_PERCENTILES) / 12.0
    L = int(np.count_nonzero(xd <= xd[0] + sigma))            # sorted: these are the first L points
    R = n - int(np.count_nonzero(xd >= xd[-1] - sigma))       # and these the points from R on
    R = max(R, L)                          # a weight both seeds reach stays with the left one
    n_right = n - R
    min_pts = min(L, n_right) if n_right > 0 else L      # an empty right cluster cannot set MinPts to zero
    return sigma, L, R, int(min_pts), sigma / min_pts


def _dbci_finish(x, xd, sigma, L, R, min_pts, eps, mid):
    """Labels of all points from the labels `mid` of the middle points (0.. = DBSCAN clusters from left to
    right, -1 noise) and step 6: the centroid of a cluster is its lower median (an L1 minimiser)."""
    n = xd.size
    labels = np.full(n, -1, dtype=np.int64)
    labels[:L] = 0
    n_mid = int(mid.max()) + 1 if mid.size and mid.max() >= 0 else 0
    labels[L:R] = np.where(mid >= 0, mid + 1, -1)
    if n - R > 0:
        labels[R:] = n_mid + 1
    cents = []
    for c in range(n_mid + 2):
        members = np.flatnonzero(labels == c)
        if members.size:
            cents.append(xd[members[(members.size - 1) // 2]])
    return {"sigma": sigma, "min_pts": int(min_pts), "eps": eps, "left": L, "right": n - R, "labels": labels,
            "centroids": np.array(cents), "sorted": x}


def dbci(weights):
    """Density-based centroid initialisation, the six steps of Section 3.1, on a flat array of binary32 weights,
    written out plainly (quadratic in the number of weights: for small inputs).  All comparisons and the few
    scalar operations are binary64 on the binary32 data.

    1. sort;  2. sigma = (sum over the 68.27 / 95.44 / 99.74 % nearest-rank percentiles of the positive weights and
    of the magnitudes of the negative weights) / 12;  3. the smallest and the largest weight seed two clusters that
    take every point within sigma of them (the right one gives way if they overlap);  4. MinPts = the smaller of the
    two counts, eps = sigma / MinPts;  5. DBSCAN on the remaining points alone: the eps-neighbourhood of a point is
    found by a scan over all of them (the point itself counts); a point with at least MinPts neighbours is a core
    point; clusters grow breadth-first from core point to core point; another point within eps of a core point
    joins the cluster of its nearest core point, found by explicit search (the left one on a tie: textbook DBSCAN
    leaves this to the visiting order), the rest is noise;  6. the centroid of a cluster is its lower median.

    Returns a dict: sigma, min_pts, eps, left (count), right (count), labels (int64 per sorted point: cluster number
    in ascending order of position, -1 noise), centroids (float64, ascending), sorted (the sorted weights)."""
    x = np.sort(np.asarray(weights, dtype=np.float32).ravel())
    xd = x.astype(np.float64)
    if xd.size == 0:
        raise ValueError("no weights")
    sigma, L, R, min_pts, eps = _dbci_seeds(xd)
    y = xd[L:R]
    m = y.size
    neighbours = [np.flatnonzero(np.abs(y - y[i]) <= eps) for i in range(m)]         # region query: full scan
    core = np.array([nb.size >= min_pts for nb in neighbours], dtype=bool)
    mid = np.full(m, -1, dtype=np.int64)
    n_clusters = 0
    for i in range(m):                     # ascending position, so clusters are numbered from left to right
        if not core[i] or mid[i] >= 0:
            continue
        mid[i] = n_clusters
        queue = [i]
        while queue:                       # breadth-first over core points
            a = queue.pop(0)
            for b in neighbours[a]:
                if core[b] and mid[b] < 0:
                    mid[b] = n_clusters
                    queue.append(int(b))
        n_clusters += 1
    cores = np.flatnonzero(core)
    for i in np.flatnonzero(~core):        # border points and noise
        best, best_d = -1, np.inf
        for c in cores:                    # ascending position: a strict comparison keeps the left one on a tie
            d = abs(y[c] - y[i])
            if d <= eps and d < best_d:
                best, best_d = int(c), d
        if best >= 0:
            mid[i] = mid[best]
    return _dbci_finish(x, xd, sigma, L, R, min_pts, eps, mid)


def dbci_scan(weights):
    """The result of ``dbci`` for large inputs, computed on the sorted array with searches and running
    extrema instead of scans over all pairs (n log n).  tests/test_oracle_pins.py checks it against ``dbci``
    on small inputs with many ties; it is used where the plain form would take hours."""
    x = np.sort(np.asarray(weights, dtype=np.float32).ravel())
    xd = x.astype(np.float64)
    n = xd.size
    if n == 0:
        raise ValueError("no weights")
    sigma, L, R, min_pts, eps = _dbci_seeds(xd)
    y = xd[L:R]
    m = y.size
    mid = np.full(m, -1, dtype=np.int64)
    if m:
        lo = np.searchsorted(y, y - eps, side="left")
        hi = np.searchsorted(y, y + eps, side="right")
        core = (hi - lo) >= min_pts
        idx = np.arange(m)
        prev_core = np.maximum.accumulate(np.where(core, idx, -1))                   # nearest core at or before i
        next_core = np.minimum.accumulate(np.where(core, idx, m)[::-1])[::-1]        # nearest core at or after i
        prev_before = np.concatenate([[-1], prev_core[:-1]])                         # nearest core strictly before i
        start = core & ((prev_before < 0) | ((y - y[np.maximum(prev_before, 0)]) > eps))
        cid = np.cumsum(start) - 1                                                   # cluster of a core point
        mid[core] = cid[core]
        nc = np.flatnonzero(~core)
        if nc.size:
            pc, nx = prev_core[nc], next_core[nc]
            dl = np.where(pc >= 0, y[nc] - y[np.maximum(pc, 0)], np.inf)
            dr = np.where(nx < m, y[np.minimum(nx, m - 1)] - y[nc], np.inf)
            take_left = (dl <= eps) & (dl <= dr)
            take_right = (dr <= eps) & ~take_left
            mid[nc[take_left]] = cid[pc[take_left]]
            mid[nc[take_right]] = cid[nx[take_right]]
    return _dbci_finish(x, xd, sigma, L, R, min_pts, eps, mid)
