"""Pins for the CPU oracle's block-based GEMM and for its packed formats (CPU only)."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2012_00596_b200 import inputs

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def brute_force_linear(x, w, rk, ck, Bo, Bi, bias=None, relu=False):
    """Block-stationary form written independently: per block, the kept sub-matrix only."""
    M, I = x.shape
    O = w.shape[0]
    y = np.zeros((M, O))
    for bo in range(O // Bo):
        for bi in range(I // Bi):
            rows = [r for r in range(Bo) if (int(rk[bo, bi]) >> r) & 1]
            cols = [c for c in range(Bi) if (int(ck[bo, bi]) >> c) & 1]
            for r in rows:
                for c in cols:
                    for m in range(M):
                        y[m, bo * Bo + r] += float(x[m, bi * Bi + c]) * float(w[bo * Bo + r, bi * Bi + c])
    if bias is not None:
        y += np.asarray(bias, dtype=np.float64)
    return np.maximum(y, 0) if relu else y


def test_linear_against_brute_force_and_matmul():
    c = inputs.linear_case(M=5, I=12, O=8, Bo=4, Bi=6, keep_rows=lambda a, b: (a + b) % 5,
                           keep_cols=lambda a, b: (2 * a + b) % 7, dtype="f32", w_sigma=1.0, seed=31)
    y = oracle.linear_bb(c.x, c.w, c.row_keep, c.col_keep, Bo=4, Bi=6, bias=c.bias, relu=True)
    yb = brute_force_linear(c.x, c.w, c.row_keep, c.col_keep, 4, 6, c.bias, True)
    np.testing.assert_allclose(y, yb, rtol=1e-12, atol=1e-12)
    m = oracle.bb_element_mask(c.row_keep, c.col_keep, 8, 12, 4, 6)
    ym = np.maximum(c.x.astype(np.float64) @ (c.w.astype(np.float64) * m).T + c.bias, 0)
    np.testing.assert_allclose(y, ym, rtol=1e-12, atol=1e-12)


def test_linear_residual_is_added_before_the_activation():
    """Shortcut epilogue: act(b + X Wm^T + res); pinned against the library matrix product, with a
    residual chosen so that adding it after the ReLU would give a different answer."""
    c = inputs.linear_case(M=7, I=12, O=8, Bo=4, Bi=6, keep_rows=3, keep_cols=4, dtype="f32", w_sigma=1.0, seed=33)
    res = -np.abs(inputs.rng_for(34).standard_normal((7, 8)))          # negative: flips signs before the ReLU
    m = oracle.bb_element_mask(c.row_keep, c.col_keep, 8, 12, 4, 6)
    pre = c.x.astype(np.float64) @ (c.w.astype(np.float64) * m).T + c.bias
    want = np.maximum(pre + res, 0)
    assert not np.allclose(want, np.maximum(pre, 0) + res)
    y = oracle.linear_bb(c.x, c.w, c.row_keep, c.col_keep, Bo=4, Bi=6, bias=c.bias, residual=res, relu=True)
    np.testing.assert_allclose(y, want, rtol=1e-12, atol=1e-12)
    pts = np.array([[0, 0], [6, 7], [3, 2]], dtype=np.int32)
    yp = oracle.linear_bb(c.x, c.w, c.row_keep, c.col_keep, Bo=4, Bi=6, bias=c.bias, residual=res, relu=True, points=pts)
    np.testing.assert_allclose(yp, want[pts[:, 0], pts[:, 1]], rtol=1e-12, atol=1e-12)
    y0 = oracle.linear_bb(c.x, c.w, c.row_keep, c.col_keep, Bo=4, Bi=6, bias=c.bias, relu=False)
    np.testing.assert_allclose(y0, pre, rtol=1e-12, atol=1e-12)


def test_bb_mask_is_outer_product_per_block():
    """Inside each block the support is (kept rows) x (kept cols) (paper Sec. 3)."""
    rng = inputs.rng_for(32)
    rk = inputs.draw_keep_sets(rng, 3, 2, 8, lambda a, b: (a * 3 + b) % 9)
    ck = inputs.draw_keep_sets(rng, 3, 2, 8, 3)
    m = oracle.bb_element_mask(rk, ck, 24, 16, 8, 8)
    for bo in range(3):
        for bi in range(2):
            blk = m[bo * 8:(bo + 1) * 8, bi * 8:(bi + 1) * 8]
            r = np.array([(int(rk[bo, bi]) >> i) & 1 for i in range(8)])
            c = np.array([(int(ck[bo, bi]) >> i) & 1 for i in range(8)])
            assert np.array_equal(blk, np.outer(r, c))


def test_linear_single_block_is_submatrix_gemm():
    c = inputs.linear_case(M=4, I=8, O=8, Bo=8, Bi=8, keep_rows=3, keep_cols=5, dtype="f32",
                           w_sigma=1.0, bias=False, relu=False, seed=33)
    y = oracle.linear_bb(c.x, c.w, c.row_keep, c.col_keep, Bo=8, Bi=8)
    rows = [r for r in range(8) if (int(c.row_keep[0, 0]) >> r) & 1]
    cols = [r for r in range(8) if (int(c.col_keep[0, 0]) >> r) & 1]
    expect = np.zeros((4, 8))
    expect[:, rows] = c.x[:, cols].astype(np.float64) @ c.w[np.ix_(rows, cols)].astype(np.float64).T
    np.testing.assert_allclose(y, expect, rtol=1e-13, atol=1e-13)
    pts = np.array([[0, rows[0]], [3, 7], [2, rows[-1]]], dtype=np.int32)
    yp = oracle.linear_bb(c.x, c.w, c.row_keep, c.col_keep, Bo=8, Bi=8, points=pts)
    assert np.array_equal(yp, y[pts[:, 0], pts[:, 1]])


def test_config3_pruning_rate():
    c = inputs.config3(M=4)
    m = oracle.bb_element_mask(c.row_keep, c.col_keep, c.O, c.I, 64, 64)
    assert int(m.sum()) * 16 == c.O * c.I
    assert c.kept_macs() == 4 * int(m.sum())


# ---------------------------------------------------------------- bf16 rounding -----------

def test_bf16_rounding_matches_torch_and_special_values():
    rng = inputs.rng_for(41)
    a = np.concatenate([
        rng.standard_normal(20000).astype(np.float32),
        (rng.standard_normal(2000) * 1e-39).astype(np.float32),       # subnormals
        np.array([0.0, -0.0, np.inf, -np.inf, 1.0, 65504.0, 3.3895314e38, -3.4e38], np.float32),
        np.array([0x3F808000, 0x3F818000, 0x3F807FFF, 0x3F808001, 0x7F7FFFFF], np.uint32).view(np.float32),
    ])
    got = oracle.f32_to_bf16_bits(a)
    ref = torch.from_numpy(a).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(got, ref)
    # ties to even, written out: 1.00390625 (0x3F808000) -> 0x3F80 ; 0x3F818000 -> 0x3F82
    assert oracle.f32_to_bf16_bits(np.array([0x3F808000], np.uint32).view(np.float32))[0] == 0x3F80
    assert oracle.f32_to_bf16_bits(np.array([0x3F818000], np.uint32).view(np.float32))[0] == 0x3F82
    nan = np.array([0x7F800001, 0xFFC12345], np.uint32).view(np.float32)
    nb = oracle.f32_to_bf16_bits(nan)
    assert nb[0] == 0x7FC0 and nb[1] == 0xFFC1


# ---------------------------------------------------------------- block-punched blob ------

@pytest.mark.parametrize("Mb,Nb,dtype", [(8, 4, "f32"), (16, 8, "bf16"), (16, 16, "bf16"), (4, 32, "bf16"), (1, 1, "f32")])
def test_pack_bp_round_trip_and_structure(Mb, Nb, dtype):
    K, C = 2 * Mb, 3 * Nb
    c = inputs.conv_case(N=1, H=4, W=4, C=C, K=K, Mb=Mb, Nb=Nb, keep=lambda fb, cb: (4 * fb + 3 * cb) % 10,
                         dtype=dtype, act="normal", w_sigma=1.0, seed=51)
    blob = oracle.pack_bp(c.w, c.tap_mask, Mb, Nb, dtype)
    dense, tm = oracle.unpack_bp(blob)
    assert np.array_equal(tm, c.tap_mask)
    m = oracle.bp_element_mask(c.tap_mask, K, C, 3, 3, Mb, Nb)
    if dtype == "f32":
        assert np.array_equal(dense.view(np.uint32), (c.w * m).astype(np.float32).view(np.uint32) * m)
    else:
        assert np.array_equal(dense, oracle.f32_to_bf16_bits(c.w).reshape(c.w.shape) * m)
    hdr = blob[:128].view(np.uint32)
    nP = int(hdr[11])
    assert nP == sum(bin(int(v)).count("1") for v in c.tap_mask.ravel())
    assert blob.size == int(hdr[15]) and all(int(hdr[i]) % 128 == 0 for i in (12, 13, 14, 15))
    blk_off = blob[int(hdr[12]):int(hdr[12]) + 4 * (tm.size + 1)].view(np.uint32)
    pw = blob[int(hdr[13]):int(hdr[13]) + 4 * nP].view(np.uint32)
    assert blk_off[0] == 0 and blk_off[-1] == nP and np.all(np.diff(blk_off.astype(np.int64)) >= 0)
    nCB = C // Nb
    for b in range(tm.size):
        seg = pw[blk_off[b]:blk_off[b + 1]]
        assert np.all((seg & 0xFFFF) == b % nCB)
        assert np.all(np.diff((seg >> 16).astype(np.int64)) > 0)          # taps strictly ascending
    # idempotence: pack(unpack(blob)) == blob
    if dtype == "f32":
        again = oracle.pack_bp(dense, tm, Mb, Nb, dtype)
    else:
        again = oracle.pack_bp(inputs.bf16_bits_to_f32(dense), tm, Mb, Nb, dtype)
    assert np.array_equal(again, blob)
    # operand image and tap unions (bf16, C % 16 == 0 only): checked element by element against the
    # matrix that unpacking the canonical sections gives back
    off_image, off_tapu, GI = int(hdr[17]), int(hdr[18]), int(hdr[19])
    if dtype == "bf16" and C % 16 == 0:
        assert GI == K and off_image % 2048 == 0 and off_tapu % 128 == 0      # K = 2 * Mb <= 128 is a power of two here
        img = blob[off_image:off_image + K * 9 * C * 2].view(np.uint16)
        tapu = blob[off_tapu:off_tapu + (K // GI) * (C // 16) * 4].view(np.uint32).reshape(K // GI, C // 16)
        for k in range(K):
            for t in range(9):
                for ch in range(C):
                    e = (((((k // GI) * (C // 16) + ch // 16) * 9 + t) * 2 + (ch % 16) // 8) * GI + k % GI) * 8 + ch % 8
                    assert img[e] == dense[k, t // 3, t % 3, ch]
        for chunk in range(C // 16):
            want = 0
            for fb in range(K // Mb):
                for cb in range(C // Nb):
                    if cb * Nb < (chunk + 1) * 16 and (cb + 1) * Nb > chunk * 16:
                        want |= int(c.tap_mask[fb, cb])
            assert int(tapu[0, chunk]) == want
    else:
        assert off_image == 0 and off_tapu == 0


def test_pack_bp_value_placement_literal():
    """Nb = 16 uses channel groups of 8: element ((j*2 + c//8)*Mb + f)*8 + c%8."""
    Mb, Nb = 2, 16
    w = np.zeros((2, 1, 2, 16), dtype=np.float32)
    for f in range(2):
        for s in range(2):
            for ch in range(16):
                w[f, 0, s, ch] = 100 * f + 1000 * s + ch
    tm = np.array([[0b10]], dtype=np.uint64)               # keep tap 1 only
    blob = oracle.pack_bp(w, tm, Mb, Nb, "f32")
    hdr = blob[:128].view(np.uint32)
    assert [int(v) for v in hdr[20:24]] == [0, 0, 0, 0]                      # no tile section for f32
    assert [int(v) for v in hdr[:20]] == [0x5042504E, 4, 0, 2, 16, 1, 2, 2, 16, 1, 1, 1, 128, 256, 384, 512, 8, 0, 0, 2]
    vals = blob[384:384 + 32 * 4].view(np.float32)
    expect = [1000 + 100 * f + 8 * g + c for g in range(2) for f in range(2) for c in range(8)]
    assert vals.tolist() == [float(v) for v in expect]
    assert blob[256:260].view(np.uint32)[0] == (0 | (1 << 16))


def _kt_views(blob):
    hdr = blob[:128].view(np.uint32)
    K, C, R, S, Mb, Nb = [int(v) for v in hdr[3:9]]
    off_ktoff, off_kt, GS, nKt = [int(v) for v in hdr[20:24]]
    nCh, nGrp = C // 16, (K // Mb) // GS
    kt_off = blob[off_ktoff:off_ktoff + 4 * (nCh * nGrp + 1)].view(np.uint32).astype(np.int64)
    kt = blob[off_kt:off_kt + nKt * Mb * 32].view(np.uint16).reshape(nKt, Mb * 16)
    return K, C, R, S, Mb, Nb, GS, nKt, nCh, nGrp, kt_off, kt


@pytest.mark.parametrize("K,C,Mb,Nb", [(64, 32, 16, 16), (64, 64, 32, 32), (512, 16, 16, 16), (96, 32, 16, 16), (128, 64, 64, 32)])
def test_pack_bp_tile_section_element_by_element(K, C, Mb, Nb):
    """The (chunk, group, tap, block) ordered tiles hold exactly the kept weights: every stored
    element is looked up by its index formula and compared with the canonical content."""
    c = inputs.conv_case(N=1, H=4, W=4, C=C, K=K, Mb=Mb, Nb=Nb, keep=lambda fb, cb: (3 * fb + 5 * cb + 1) % 10,
                         dtype="bf16", act="normal", w_sigma=1.0, seed=53)
    blob = oracle.pack_bp(c.w, c.tap_mask, Mb, Nb, "bf16")
    dense, tm = oracle.unpack_bp(blob)
    K_, C_, R, S, Mb_, Nb_, GS, nKt, nCh, nGrp, kt_off, kt = _kt_views(blob)
    FGW = max(f for f in (256, 128, 64, 32, 16) if K % f == 0)
    assert (K_, C_, Mb_, Nb_) == (K, C, Mb, Nb) and GS == FGW // Mb
    assert nKt == int(blob[:128].view(np.uint32)[11]) * (Nb // 16)
    assert kt_off[0] == 0 and kt_off[-1] == nKt and np.all(np.diff(kt_off) >= 0)
    seen = 0
    for ch in range(nCh):
        cb = ch * 16 // Nb
        for g in range(nGrp):
            j = int(kt_off[ch * nGrp + g])
            for t in range(R * S):
                for fb in range(g * GS, (g + 1) * GS):
                    if not (int(tm[fb, cb]) >> t) & 1:
                        continue
                    for f in range(Mb):
                        for cc in range(16):
                            e = (((f // 8) * 2 + cc // 8) * 8 + f % 8) * 8 + cc % 8
                            assert kt[j, e] == dense[fb * Mb + f, t // S, t % S, ch * 16 + cc]
                    j += 1
                    seen += 1
            assert j == int(kt_off[ch * nGrp + g + 1])
    assert seen == nKt


def test_pack_bp_tile_section_literal():
    """Hand-made case: 32 filters in two blocks of 16, 16 channels, two taps.  Block 0 keeps tap 1,
    block 1 keeps taps 0 and 1.  One chunk, one group (FGW = 32, GS = 2), so the tile order is
    (tap 0, block 1), (tap 1, block 0), (tap 1, block 1).  Two probes whose values are small integers
    (exact in bf16): one numbers (tap, filter), the other (tap, channel)."""
    tm = np.array([[0b10], [0b11]], dtype=np.uint64)

    def tiles(fn):
        w = np.zeros((32, 1, 2, 16), dtype=np.float32)
        for k in range(32):
            for t in range(2):
                for ch in range(16):
                    w[k, 0, t, ch] = fn(t, k, ch)
        blob = oracle.pack_bp(w, tm, 16, 16, "bf16")
        hdr = blob[:128].view(np.uint32)
        off_ktoff, off_kt, GS, nKt = [int(v) for v in hdr[20:24]]
        assert (GS, nKt) == (2, 3) and off_ktoff % 128 == 0 and off_kt % 128 == 0
        assert blob[off_ktoff:off_ktoff + 8].view(np.uint32).tolist() == [0, 3]
        assert int(hdr[15]) == blob.size == off_kt + 3 * 512
        return inputs.bf16_bits_to_f32(blob[off_kt:off_kt + 3 * 512].view(np.uint16)).reshape(3, 2, 2, 8, 8)

    kf = tiles(lambda t, k, ch: 64 * t + k)          # [tile][filter octet][channel octet][filter][channel]
    assert kf[0, 1, 1, 2, 3] == 26                    # (tap 0, block 1): filter 16 + 8 + 2
    assert kf[1, 0, 0, 0, 0] == 64 and kf[1, 1, 0, 7, 5] == 64 + 15      # (tap 1, block 0)
    assert kf[2, 0, 1, 4, 0] == 64 + 20               # (tap 1, block 1): filter 16 + 4
    kc = tiles(lambda t, k, ch: 32 * t + ch + 1)
    assert kc[0, 1, 1, 2, 3] == 12 and kc[0, 0, 0, 5, 0] == 1            # channel 8 + 3; channel 0
    assert kc[1, 1, 0, 7, 5] == 32 + 6 and kc[2, 0, 1, 4, 7] == 32 + 16  # channel 5; channel 15


def test_pack_bp_tile_section_absent_when_not_applicable():
    for (Mb, Nb, dtype) in [(8, 8, "bf16"), (16, 8, "bf16"), (16, 16, "f32"), (4, 4, "bf16")]:
        c = inputs.conv_case(N=1, H=4, W=4, C=2 * max(Nb, 8), K=2 * Mb, Mb=Mb, Nb=Nb, keep=3, dtype=dtype, seed=54)
        hdr = oracle.pack_bp(c.w, c.tap_mask, Mb, Nb, dtype)[:128].view(np.uint32)
        assert [int(v) for v in hdr[20:24]] == [0, 0, 0, 0]


# ---------------------------------------------------------------- block-based blob --------

@pytest.mark.parametrize("Bo,Bi,dtype", [(64, 64, "bf16"), (8, 16, "f32"), (4, 4, "bf16")])
def test_pack_bb_round_trip_and_structure(Bo, Bi, dtype):
    O, I = 3 * Bo, 2 * Bi
    c = inputs.linear_case(M=2, I=I, O=O, Bo=Bo, Bi=Bi, keep_rows=lambda a, b: (5 * a + b) % (Bo + 1),
                           keep_cols=lambda a, b: (a + 3 * b + 1) % (Bi + 1), dtype=dtype, w_sigma=1.0, seed=61)
    blob = oracle.pack_bb(c.w, c.row_keep, c.col_keep, Bo, Bi, dtype)
    dense, rk, ck = oracle.unpack_bb(blob)
    assert np.array_equal(rk, c.row_keep) and np.array_equal(ck, c.col_keep)
    m = oracle.bb_element_mask(c.row_keep, c.col_keep, O, I, Bo, Bi)
    if dtype == "f32":
        assert np.array_equal(dense.view(np.uint32), c.w.view(np.uint32) * m)
    else:
        assert np.array_equal(dense, oracle.f32_to_bf16_bits(c.w).reshape(O, I) * m)
    hdr = blob[:128].view(np.uint32)
    nBlk = 6
    rows = blob[int(hdr[11]):int(hdr[11]) + Bo * nBlk].reshape(nBlk, Bo)
    cnt = blob[int(hdr[10]):int(hdr[10]) + 2 * nBlk].reshape(nBlk, 2)
    voff = blob[int(hdr[13]):int(hdr[13]) + 4 * (nBlk + 1)].view(np.uint32)
    for b in range(nBlk):
        nr = int(cnt[b, 0])
        assert np.all(np.diff(rows[b, :nr].astype(np.int64)) > 0) and np.all(rows[b, nr:] == 0xFF)
        assert voff[b] % 8 == 0 and voff[b + 1] >= voff[b] + nr * int(cnt[b, 1])
    src = dense if dtype == "f32" else inputs.bf16_bits_to_f32(dense)
    assert np.array_equal(oracle.pack_bb(src, rk, ck, Bo, Bi, dtype), blob)
    # operand-image section: tiles[b][c // 8][row][c % 8] holds the masked dense weight of (row, cols[c])
    Kp, off_tiles = int(hdr[16]), int(hdr[17])
    cols = blob[int(hdr[12]):int(hdr[12]) + Bi * nBlk].reshape(nBlk, Bi)
    assert Kp % 16 == 0 and Kp >= max(16, int(cnt[:, 1].max()))
    es = 4 if dtype == "f32" else 2
    tiles = blob[off_tiles:off_tiles + nBlk * Kp * Bo * es].view(np.float32 if dtype == "f32" else np.uint16)
    tiles = tiles.reshape(nBlk, Kp // 8, Bo, 8)
    for b in range(nBlk):
        bo, bi = divmod(b, 2)
        expect = np.zeros((Kp // 8, Bo, 8), dtype=tiles.dtype)
        for c in range(int(cnt[b, 1])):
            expect[c // 8, :, c % 8] = dense[bo * Bo:(bo + 1) * Bo, bi * Bi + int(cols[b, c])]
        assert np.array_equal(tiles[b], expect)
    # masked dense section: the matrix that unpacking the compact sections gives back
    off_dense = int(hdr[18])
    assert off_dense == int(hdr[13]) + -(-4 * (nBlk + 1) // 128) * 128 and int(hdr[15]) == blob.size
    assert int(hdr[14]) == off_dense + -(-dense.size * es // 128) * 128      # values follow the dense image
    img = blob[off_dense:off_dense + dense.size * es].view(dense.dtype).reshape(dense.shape)
    assert np.array_equal(img, dense)
