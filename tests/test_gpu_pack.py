"""GPU packers vs the oracle's packers: blobs byte-identical, round trips exact."""
import numpy as np
import pytest
import torch

import oracle
import paper_2012_00596_b200 as npas
from paper_2012_00596_b200 import inputs
from util import dev

pytestmark = pytest.mark.gpu


def _blob_np(b):
    return b.data.cpu().numpy()


@pytest.mark.parametrize("Mb,Nb,dtype,keep", [
    (8, 4, "f32", 3), (16, 8, "bf16", 3), (16, 16, "bf16", 5), (32, 32, "bf16", 9), (4, 4, "bf16", 1),
    (1, 1, "f32", lambda fb, cb: (fb * 5 + cb) % 10), (16, 8, "bf16", lambda fb, cb: (fb + 3 * cb) % 10),
    (8, 24, "bf16", 2), (16, 32, "bf16", lambda fb, cb: (2 * fb + cb) % 10), (64, 16, "bf16", 4),
])
def test_pack_bp_bit_exact_and_round_trip(Mb, Nb, dtype, keep):
    K, C = 3 * Mb, 5 * Nb
    c = inputs.conv_case(N=1, H=4, W=4, C=C, K=K, Mb=Mb, Nb=Nb, keep=keep, dtype="f32", act="normal",
                         w_sigma=1.0, seed=101)
    ref = oracle.pack_bp(c.w, c.tap_mask, Mb, Nb, dtype)
    w = dev(c.w)
    blob = npas.pack_bp(w, c.tap_mask, Mb, Nb, torch.float32 if dtype == "f32" else torch.bfloat16)
    assert np.array_equal(_blob_np(blob), ref)
    npas.blob_check(blob)
    wd, tm = npas.unpack_bp(blob)
    dense_ref, tm_ref = oracle.unpack_bp(ref)
    assert np.array_equal(npas.mask_to_numpy(tm), tm_ref)
    got = wd.view(torch.int16).cpu().numpy().view(np.uint16) if dtype == "bf16" else wd.cpu().numpy()
    assert np.array_equal(got.view(np.uint16 if dtype == "bf16" else np.uint32),
                          dense_ref.view(np.uint16 if dtype == "bf16" else np.uint32))
    # idempotence: packing the unpacked weights reproduces the blob
    again = npas.pack_bp(wd, tm, Mb, Nb)
    assert np.array_equal(_blob_np(again), ref)


def test_pack_bp_special_values_and_rounding_ties():
    w = np.zeros((16, 1, 1, 8), dtype=np.float32)
    bits = np.array([0x3F808000, 0x3F818000, 0x3F807FFF, 0x3F808001, 0x7F7FFFFF, 0x7F800000, 0xFF800000,
                     0x7F800001, 0xFFC12345, 0x00000001, 0x80000000, 0x00400000], dtype=np.uint32)
    w.reshape(-1)[:bits.size] = bits.view(np.float32)
    tm = np.ones((1, 1), dtype=np.uint64)
    ref = oracle.pack_bp(w, tm, 16, 8, "bf16")
    blob = npas.pack_bp(torch.from_numpy(w).cuda(), tm, 16, 8, torch.bfloat16)
    assert np.array_equal(_blob_np(blob), ref)


def test_pack_bp_config2_and_config5_sizes():
    for c in (inputs.config2(N=1), inputs.config5(16, 16, 3, N=1), inputs.config5(4, 4, 2, N=1), inputs.config5(32, 32, 5, N=1)):
        ref = oracle.pack_bp(c.w, c.tap_mask, c.Mb, c.Nb, "bf16")
        blob = npas.pack_bp(dev(c.w, "bf16"), c.tap_mask, c.Mb, c.Nb)
        assert np.array_equal(_blob_np(blob), ref)


@pytest.mark.parametrize("Bo,Bi,dtype,kr,kc", [
    (64, 64, "bf16", 16, 16), (64, 64, "bf16", 32, 32), (16, 32, "f32", lambda a, b: (3 * a + b) % 17, 5),
    (64, 64, "bf16", lambda a, b: (a * 7 + b * 3) % 65, lambda a, b: (a + b * 11) % 65), (8, 8, "bf16", 3, 0),
])
def test_pack_bb_bit_exact_and_round_trip(Bo, Bi, dtype, kr, kc):
    O, I = 3 * Bo, 4 * Bi
    c = inputs.linear_case(M=1, I=I, O=O, Bo=Bo, Bi=Bi, keep_rows=kr, keep_cols=kc, dtype="f32", w_sigma=1.0, seed=102)
    ref = oracle.pack_bb(c.w, c.row_keep, c.col_keep, Bo, Bi, dtype)
    blob = npas.pack_bb(dev(c.w), c.row_keep, c.col_keep, Bo, Bi, torch.float32 if dtype == "f32" else torch.bfloat16)
    assert np.array_equal(_blob_np(blob), ref)
    npas.blob_check(blob)
    wd, rk, ck = npas.unpack_bb(blob)
    dense_ref, rk_ref, ck_ref = oracle.unpack_bb(ref)
    assert np.array_equal(npas.mask_to_numpy(rk), rk_ref) and np.array_equal(npas.mask_to_numpy(ck), ck_ref)
    got = wd.view(torch.int16).cpu().numpy().view(np.uint16) if dtype == "bf16" else wd.cpu().numpy().view(np.uint32)
    assert np.array_equal(got, dense_ref.view(np.uint16 if dtype == "bf16" else np.uint32))
    again = npas.pack_bb(wd, rk, ck, Bo, Bi)
    assert np.array_equal(_blob_np(again), ref)


def test_mask_from_dense_and_structure_violation():
    c = inputs.conv_case(N=1, H=4, W=4, C=16, K=16, Mb=8, Nb=4, keep=lambda fb, cb: (fb + cb) % 10, seed=103)
    m = oracle.bp_element_mask(c.tap_mask, 16, 16, 3, 3, 8, 4)
    tm = npas.mask_bp_from_dense(torch.from_numpy(m).cuda(), 8, 4)
    assert np.array_equal(npas.mask_to_numpy(tm), c.tap_mask)
    bad = m.copy()
    bad[3, 1, 1, 2] ^= 1                                   # one kernel of one block disagrees
    with pytest.raises(npas.NpasError) as e:
        npas.mask_bp_from_dense(torch.from_numpy(bad).cuda(), 8, 4)
    assert e.value.code == 5
    l = inputs.linear_case(M=1, I=32, O=48, Bo=16, Bi=16, keep_rows=5, keep_cols=7, seed=104)
    mb = oracle.bb_element_mask(l.row_keep, l.col_keep, 48, 32, 16, 16)
    rk, ck = npas.mask_bb_from_dense(torch.from_numpy(mb).cuda(), 16, 16)
    assert np.array_equal(npas.mask_to_numpy(rk), l.row_keep) and np.array_equal(npas.mask_to_numpy(ck), l.col_keep)
    badb = mb.copy()
    r, cc = np.argwhere(mb == 1)[0]
    badb[r, cc] = 0                                        # hole inside a rows x cols product
    with pytest.raises(npas.NpasError) as e:
        npas.mask_bb_from_dense(torch.from_numpy(badb).cuda(), 16, 16)
    assert e.value.code == 5


def test_blob_check_rejects_foreign_blob():
    c = inputs.conv_case(N=1, H=4, W=4, C=16, K=16, Mb=8, Nb=8, keep=3, seed=105)
    blob = npas.pack_bp(dev(c.w, "bf16"), c.tap_mask, 8, 8)
    wrong = npas.BpBlob(blob.data, npas.binding.BpDesc(16, 16, 3, 3, 16, 8, 1, 1))
    with pytest.raises(npas.NpasError) as e:
        npas.blob_check(wrong)
    assert e.value.code == 6
    corrupted = npas.BpBlob(blob.data.clone(), blob.desc)
    corrupted.data[0] = 0
    with pytest.raises(npas.NpasError):
        npas.blob_check(corrupted)


def test_pack_reports_a_buffer_that_the_device_masks_overflow():
    """The size call sees host masks; if the masks on the device keep more, the blob does not fit.
    The pack call must say so, leave a header nobody can mistake for a blob (magic 0, offsets 0,
    needed size in word 15), and the header check must reject it."""
    import ctypes
    from paper_2012_00596_b200 import binding as B
    lib = npas.load()
    c = inputs.conv_case(N=1, H=4, W=4, C=32, K=32, Mb=16, Nb=16, keep=2, seed=106)
    w = dev(c.w, "bf16")
    d = B.BpDesc(32, 32, 3, 3, 16, 16, B.BF16, B.BF16, 9)
    size = ctypes.c_size_t(0)
    assert lib.npas_pack_bp_size(ctypes.byref(d), c.tap_mask.ctypes.data_as(ctypes.c_void_p), ctypes.byref(size)) == 0
    more = np.full_like(c.tap_mask, 0x1FF)                                   # every tap kept on the device
    full = ctypes.c_size_t(0)
    assert lib.npas_pack_bp_size(ctypes.byref(d), more.ctypes.data_as(ctypes.c_void_p), ctypes.byref(full)) == 0
    blob = torch.full((size.value,), 0xAB, dtype=torch.uint8, device="cuda")
    rc = lib.npas_pack_bp(ctypes.byref(d), B._p(w), B._p(B._mask_to_device(more, w.device)), B._p(blob),
                          ctypes.c_size_t(size.value), B._stream())
    assert rc == 7                                                           # NPAS_ERR_BUFFER_TOO_SMALL
    hdr = blob[:128].cpu().numpy().view(np.uint32)
    assert hdr[0] == 0 and int(hdr[15]) == full.value and not hdr[12:15].any() and not hdr[16:24].any()
    with pytest.raises(npas.NpasError) as e:
        npas.blob_check(npas.BpBlob(blob, d))
    assert e.value.code == 6
    # block-based: same contract
    l = inputs.linear_case(M=1, I=64, O=64, Bo=32, Bi=32, keep_rows=4, keep_cols=4, seed=107)
    db = B.BbDesc(64, 64, 32, 32, B.BF16, B.BF16, 32)
    assert lib.npas_pack_bb_size(ctypes.byref(db), l.row_keep.ctypes.data_as(ctypes.c_void_p),
                                 l.col_keep.ctypes.data_as(ctypes.c_void_p), ctypes.byref(size)) == 0
    allk = np.full_like(l.row_keep, 0xFFFFFFFF)
    bb = torch.zeros(size.value, dtype=torch.uint8, device="cuda")
    rc = lib.npas_pack_bb(ctypes.byref(db), B._p(dev(l.w, "bf16")), B._p(B._mask_to_device(allk, "cuda")),
                          B._p(B._mask_to_device(allk, "cuda")), B._p(bb), ctypes.c_size_t(size.value), B._stream())
    assert rc == 7
    assert bb[:4].cpu().numpy().view(np.uint32)[0] == 0
    with pytest.raises(npas.NpasError):
        npas.blob_check(npas.BbBlob(bb, db))
