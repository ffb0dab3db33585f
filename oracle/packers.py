"""numpy restatement of the packed-weight formats (test infrastructure; see package docstring).

The paper (Sec. 3) fixes only the STRUCTURE of the two sparsity schemes; it does not describe a
storage format.  The format below is this library's own, restated here independently of the CUDA
packer so that "bit-exact" means byte-for-byte equality of two separately written encoders.

Block-punched blob, version 4 (little endian, every section starts on a 128-byte boundary,
padding = 0):
  header   32 x uint32: magic 'NPBP', version 4, dtype (0 = f32, 1 = bf16), K, C, R, S, Mb, Nb,
           nFB = K/Mb, nCB = C/Nb, nPairs, off_blk_off, off_pairs, off_values, total_bytes,
           G (channel-group width: 8 when Nb is a multiple of 8, else Nb), off_image, off_tapu, GI,
           off_kt_off, off_kt, GS, nKt, zeros.
  blk_off  uint32[nFB*nCB + 1]: exclusive prefix sum of the kept-tap counts over blocks in
           (fb major, cb minor) order; block (fb,cb) owns pairs blk_off[fb*nCB+cb] ..
  pairs    uint32[nPairs] = cb | tap << 16, block order, taps ascending inside a block.
  values   for pair j, filter f < Mb, channel c < Nb the weight W[fb*Mb+f, tap/S, tap%S, cb*Nb+c]
           sits at element ((j*(Nb/G) + c/G)*Mb + f)*G + c%G.
  These three sections are the canonical content (what unpack reads).  The remaining sections are
  compile-time expansions of it for particular kernels, written by the same call:
  image    (bf16, C % 16 == 0; else off_image = 0) the masked dense weights, pruned = +0, as
           [K/GI][C/16][tap][2 channel octets][GI filters][8 channels], GI = largest power of two
           <= 128 dividing K.  The section starts on a multiple of 2048 bytes (every other
           section on a multiple of 128).
  tapu     uint32[K/GI][C/16]: union of the kept-tap bitsets of the blocks touching the (filter
           group, 16-channel chunk); all ones when R*S > 32.
  kt_off, kt  (bf16, Mb % 16 == 0, Nb % 16 == 0, R*S <= 16 and Mb dividing FGW, the largest power
           of two <= 256 that divides K; else off_kt = 0)  the kept weights once more, cut into
           tiles of Mb filters x 16 channels and ordered so that everything one group of
           GS = FGW/Mb filter blocks needs for one 16-channel chunk is a contiguous run in which
           the tiles of one tap are neighbours: order (chunk ch = c/16, group g = fb/GS, tap,
           fb ascending, kept only).  kt_off uint32[(C/16)*(K/FGW) + 1] is the exclusive prefix
           sum of the tile counts per (chunk, group), chunk major; nKt = nPairs * Nb/16 tiles.
           A tile is [Mb/8 filter octets][2 channel octets][8 filters][8 channels] (Mb*32 bytes).

Block-based blob, version 3:
  header   32 x uint32: magic 'NPBB', version 3, dtype, O, I, Bo, Bi, nBo, nBi, nVals,
           off_cnt, off_rows, off_cols, off_val_off, off_values, total_bytes, Kp, off_tiles,
           off_dense, zeros (Kp = largest kept-column count of any block rounded up to 16, at
           least 16).
  cnt      uint8[nBlk][2] = (kept rows, kept cols), blocks in (bo major, bi minor) order.
  rows     uint8[nBlk][Bo] kept row indices ascending, unused slots 0xFF.
  cols     uint8[nBlk][Bi] kept column indices ascending, unused slots 0xFF.
  val_off  uint32[nBlk + 1]: element offset of each block's values, every start rounded up to a
           multiple of 8 elements; val_off[nBlk] = nVals.
  dense    the masked weight matrix [O][I], row major, pruned = +0 (placed before the values so
           that its offset follows from O, I, Bo, Bi alone).
  values   per block, kept rows x kept cols, row major: W[bo*Bo + rows[r], bi*Bi + cols[c]].
  tiles    per block a [Kp/8][Bo][8] tensor-core operand image of the same weights: element
           (c // 8, rows[r], c % 8) = W[bo*Bo + rows[r], bi*Bi + cols[c]], everything else zero
           (pruned rows stay zero rows, columns past the block's kept count are zero).
  cnt, rows, cols, val_off, values are the canonical content; dense and tiles are expansions.

fp32 -> bf16 is round-to-nearest-even on the bit pattern; NaN keeps its sign and upper payload
and gets the quiet bit; infinities, zeros and subnormals follow the same integer rule.
"""
from __future__ import annotations

import numpy as np

MAGIC_BP = 0x5042504E
MAGIC_BB = 0x4242504E


def _up(x: int, a: int) -> int:
    return (x + a - 1) // a * a


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    bits = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    is_nan = ((bits & 0x7F800000) == 0x7F800000) & ((bits & 0x007FFFFF) != 0)
    lsb = (bits >> 16) & 1
    rounded = ((bits + 0x7FFF + lsb) >> 16) & 0xFFFF
    nan_bits = ((bits >> 16) | 0x0040) & 0xFFFF
    return np.where(is_nan, nan_bits, rounded).astype(np.uint16)


def _bits(v: int, n: int):
    return [t for t in range(n) if (int(v) >> t) & 1]


def bp_element_mask(tap_mask, K, C, R, S, Mb, Nb) -> np.ndarray:
    """m[k,r,s,c] = 1 iff tap r*S+s is kept in block (k // Mb, c // Nb)."""
    m = np.zeros((K, R, S, C), dtype=np.uint8)
    for fb in range(K // Mb):
        for cb in range(C // Nb):
            for t in _bits(tap_mask[fb, cb], R * S):
                m[fb * Mb:(fb + 1) * Mb, t // S, t % S, cb * Nb:(cb + 1) * Nb] = 1
    return m


def bb_element_mask(row_keep, col_keep, O, I, Bo, Bi) -> np.ndarray:
    """m[o,i] = 1 iff row o%Bo and column i%Bi are both kept in block (o // Bo, i // Bi)."""
    m = np.zeros((O, I), dtype=np.uint8)
    for bo in range(O // Bo):
        for bi in range(I // Bi):
            r = np.array(_bits(row_keep[bo, bi], Bo), dtype=np.int64)
            c = np.array(_bits(col_keep[bo, bi], Bi), dtype=np.int64)
            if r.size and c.size:
                m[np.ix_(bo * Bo + r, bi * Bi + c)] = 1
    return m


def _encode(vals_f32: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "f32":
        return np.ascontiguousarray(vals_f32, dtype=np.float32).view(np.uint8)
    return f32_to_bf16_bits(vals_f32).view(np.uint8)


def pack_bp(w: np.ndarray, tap_mask: np.ndarray, Mb: int, Nb: int, dtype: str = "bf16") -> np.ndarray:
    """Dense KRSC fp32 weights + per-block tap bitsets -> blob (uint8 array)."""
    K, R, S, C = w.shape
    nFB, nCB = K // Mb, C // Nb
    G = 8 if Nb % 8 == 0 else Nb
    es = 4 if dtype == "f32" else 2
    blk_off = [0]
    pairs = []
    for fb in range(nFB):
        for cb in range(nCB):
            taps = _bits(tap_mask[fb, cb], R * S)
            pairs += [(cb, t, fb) for t in taps]
            blk_off.append(len(pairs))
    nP = len(pairs)
    vals = np.zeros((nP, Nb // G, Mb, G), dtype=np.float32)
    for j, (cb, t, fb) in enumerate(pairs):
        blk = w[fb * Mb:(fb + 1) * Mb, t // S, t % S, cb * Nb:(cb + 1) * Nb]      # [Mb, Nb]
        vals[j] = blk.reshape(Mb, Nb // G, G).transpose(1, 0, 2)
    off_blk = 128
    off_pairs = _up(off_blk + 4 * (nFB * nCB + 1), 128)
    off_vals = _up(off_pairs + 4 * nP, 128)
    total = off_vals + _up(nP * Mb * Nb * es, 128)
    # operand image of the masked dense weights (bf16 blobs with C % 16 == 0) and, per (group of GI
    # filters, 16-channel chunk), the union of the taps kept by the blocks that touch it
    GI = 128
    while K % GI:
        GI //= 2
    off_image = off_tapu = 0
    if dtype == "bf16" and C % 16 == 0:
        off_image = _up(total, 2048)          # the image starts on a multiple of 2048 bytes
        off_tapu = off_image + _up(K * R * S * C * 2, 128)
        total = off_tapu + _up((K // GI) * (C // 16) * 4, 128)
    # kept weights as 16-channel tiles grouped by (chunk, filter group, tap)
    FGW = 256
    while K % FGW:
        FGW //= 2
    off_ktoff = off_kt = GS = nKt = 0
    if dtype == "bf16" and Mb % 16 == 0 and Nb % 16 == 0 and R * S <= 16 and FGW % Mb == 0:
        GS = FGW // Mb
        nKt = nP * (Nb // 16)
        off_ktoff = total
        off_kt = off_ktoff + _up(4 * ((C // 16) * (K // FGW) + 1), 128)
        total = off_kt + _up(nKt * Mb * 32, 128)
    blob = np.zeros(total, dtype=np.uint8)
    hdr = np.zeros(32, dtype=np.uint32)
    hdr[:24] = [MAGIC_BP, 4, 0 if dtype == "f32" else 1, K, C, R, S, Mb, Nb, nFB, nCB, nP,
                off_blk, off_pairs, off_vals, total, G, off_image, off_tapu, GI,
                off_ktoff, off_kt, GS, nKt]
    blob[:128] = hdr.view(np.uint8)
    blob[off_blk:off_blk + 4 * len(blk_off)] = np.array(blk_off, dtype=np.uint32).view(np.uint8)
    if nP:
        pw = np.array([cb | (t << 16) for cb, t, _ in pairs], dtype=np.uint32)
        blob[off_pairs:off_pairs + 4 * nP] = pw.view(np.uint8)
        enc = _encode(vals.ravel(), dtype)
        blob[off_vals:off_vals + enc.size] = enc
    if off_image:
        RS, nCh = R * S, C // 16
        m = bp_element_mask(tap_mask, K, C, R, S, Mb, Nb)
        masked = np.where(m != 0, np.asarray(w, dtype=np.float32), np.float32(0.0))     # [K,R,S,C]
        # image[k // GI][c // 16][tap][(c % 16) // 8][k % GI][c % 8]
        img = masked.reshape(K // GI, GI, RS, nCh, 2, 8).transpose(0, 3, 2, 4, 1, 5)
        enc = _encode(np.ascontiguousarray(img).ravel(), dtype)
        blob[off_image:off_image + enc.size] = enc
        tapu = np.zeros((K // GI, nCh), dtype=np.uint32)
        for fb in range(nFB):
            for cb in range(nCB):
                bits = int(tap_mask[fb, cb]) & ((1 << RS) - 1)
                if not bits:
                    continue
                lo32 = 0xFFFFFFFF if RS > 32 else bits
                for gi in range(fb * Mb // GI, ((fb + 1) * Mb - 1) // GI + 1):
                    for ch in range(cb * Nb // 16, ((cb + 1) * Nb - 1) // 16 + 1):
                        tapu[gi, ch] |= lo32
        blob[off_tapu:off_tapu + tapu.size * 4] = tapu.view(np.uint8).ravel()
    if off_kt:
        RS = R * S
        kt_off = []
        tiles = []
        for ch in range(C // 16):
            cb = ch * 16 // Nb
            for g in range(K // FGW):
                kt_off.append(len(tiles))
                for t in range(RS):
                    for fb in range(g * GS, (g + 1) * GS):
                        if (int(tap_mask[fb, cb]) >> t) & 1:
                            tile = w[fb * Mb:(fb + 1) * Mb, t // S, t % S, ch * 16:(ch + 1) * 16]   # [Mb, 16]
                            tiles.append(np.asarray(tile, dtype=np.float32).reshape(Mb // 8, 8, 2, 8).transpose(0, 2, 1, 3))
        kt_off.append(len(tiles))
        assert len(tiles) == nKt
        blob[off_ktoff:off_ktoff + 4 * len(kt_off)] = np.array(kt_off, dtype=np.uint32).view(np.uint8)
        if tiles:
            enc = _encode(np.ascontiguousarray(np.stack(tiles)).ravel(), dtype)
            blob[off_kt:off_kt + enc.size] = enc
    return blob


def unpack_bp(blob: np.ndarray):
    """blob -> (masked dense weights [K,R,S,C] as uint16 bf16 bits or float32, tap_mask)."""
    hdr = blob[:128].view(np.uint32)
    assert hdr[0] == MAGIC_BP and hdr[1] == 4
    dt, K, C, R, S, Mb, Nb, nFB, nCB, nP, off_blk, off_pairs, off_vals, total, G = \
        [int(v) for v in hdr[2:17]]
    es = 4 if dt == 0 else 2
    blk_off = blob[off_blk:off_blk + 4 * (nFB * nCB + 1)].view(np.uint32)
    pw = blob[off_pairs:off_pairs + 4 * nP].view(np.uint32)
    raw = blob[off_vals:off_vals + nP * Mb * Nb * es]
    vals = raw.view(np.float32 if dt == 0 else np.uint16).reshape(nP, Nb // G, Mb, G)
    dense = np.zeros((K, R, S, C), dtype=vals.dtype)
    tap_mask = np.zeros((nFB, nCB), dtype=np.uint64)
    for fb in range(nFB):
        for cb in range(nCB):
            for j in range(int(blk_off[fb * nCB + cb]), int(blk_off[fb * nCB + cb + 1])):
                t = int(pw[j]) >> 16
                assert (int(pw[j]) & 0xFFFF) == cb
                tap_mask[fb, cb] |= np.uint64(1 << t)
                dense[fb * Mb:(fb + 1) * Mb, t // S, t % S, cb * Nb:(cb + 1) * Nb] = \
                    vals[j].transpose(1, 0, 2).reshape(Mb, Nb)
    return dense, tap_mask


def pack_bb(w: np.ndarray, row_keep: np.ndarray, col_keep: np.ndarray, Bo: int, Bi: int,
            dtype: str = "bf16") -> np.ndarray:
    """Dense [O,I] fp32 weights + per-block kept-row / kept-column bitsets -> blob."""
    O, I = w.shape
    nBo, nBi = O // Bo, I // Bi
    nBlk = nBo * nBi
    es = 4 if dtype == "f32" else 2
    cnt = np.zeros((nBlk, 2), dtype=np.uint8)
    rows = np.full((nBlk, Bo), 0xFF, dtype=np.uint8)
    cols = np.full((nBlk, Bi), 0xFF, dtype=np.uint8)
    val_off = np.zeros(nBlk + 1, dtype=np.uint32)
    chunks = []
    pos = 0
    for bo in range(nBo):
        for bi in range(nBi):
            b = bo * nBi + bi
            r = _bits(row_keep[bo, bi], Bo)
            c = _bits(col_keep[bo, bi], Bi)
            cnt[b] = (len(r), len(c))
            rows[b, :len(r)] = r
            cols[b, :len(c)] = c
            val_off[b] = pos
            sub = w[np.ix_(bo * Bo + np.array(r, dtype=np.int64), bi * Bi + np.array(c, dtype=np.int64))] \
                if r and c else np.zeros((0,), np.float32)
            chunks.append((pos, np.ascontiguousarray(sub, dtype=np.float32).ravel()))
            pos = _up(pos + len(r) * len(c), 8)
    val_off[nBlk] = pos
    Kp = max(16, _up(int(cnt[:, 1].max()) if nBlk else 0, 16))
    off_cnt = 128
    off_rows = _up(off_cnt + 2 * nBlk, 128)
    off_cols = _up(off_rows + Bo * nBlk, 128)
    off_voff = _up(off_cols + Bi * nBlk, 128)
    off_dense = _up(off_voff + 4 * (nBlk + 1), 128)
    off_vals = off_dense + _up(O * I * es, 128)
    off_tiles = off_vals + _up(pos * es, 128)
    total = off_tiles + _up(nBlk * Kp * Bo * es, 128)
    blob = np.zeros(total, dtype=np.uint8)
    hdr = np.zeros(32, dtype=np.uint32)
    hdr[:19] = [MAGIC_BB, 3, 0 if dtype == "f32" else 1, O, I, Bo, Bi, nBo, nBi, pos,
                off_cnt, off_rows, off_cols, off_voff, off_vals, total, Kp, off_tiles, off_dense]
    blob[:128] = hdr.view(np.uint8)
    blob[off_cnt:off_cnt + cnt.size] = cnt.ravel()
    blob[off_rows:off_rows + rows.size] = rows.ravel()
    blob[off_cols:off_cols + cols.size] = cols.ravel()
    blob[off_voff:off_voff + 4 * (nBlk + 1)] = val_off.view(np.uint8)
    tiles = np.zeros((nBlk, Kp // 8, Bo, 8), dtype=np.float32)
    for b, (p0, v) in enumerate(chunks):
        if v.size:
            enc = _encode(v, dtype)
            blob[off_vals + p0 * es: off_vals + p0 * es + enc.size] = enc
            nr, nc = int(cnt[b, 0]), int(cnt[b, 1])
            sub = v.reshape(nr, nc)
            for c in range(nc):
                tiles[b, c // 8, rows[b, :nr].astype(np.int64), c % 8] = sub[:, c]
    enc = _encode(tiles.ravel(), dtype)
    blob[off_tiles:off_tiles + enc.size] = enc
    # the masked dense [O][I] matrix (what the zero-skipping forms above encode), row major
    masked = np.where(bb_element_mask(row_keep, col_keep, O, I, Bo, Bi) != 0, np.asarray(w, dtype=np.float32),
                      np.float32(0.0))
    enc = _encode(masked.ravel(), dtype)
    blob[off_dense:off_dense + enc.size] = enc
    return blob


def unpack_bb(blob: np.ndarray):
    """blob -> (masked dense weights [O,I] as uint16 bf16 bits or float32, row_keep, col_keep)."""
    hdr = blob[:128].view(np.uint32)
    assert hdr[0] == MAGIC_BB and hdr[1] == 3
    dt, O, I, Bo, Bi, nBo, nBi, nVals, off_cnt, off_rows, off_cols, off_voff, off_vals, total = \
        [int(v) for v in hdr[2:16]]
    nBlk = nBo * nBi
    es = 4 if dt == 0 else 2
    cnt = blob[off_cnt:off_cnt + 2 * nBlk].reshape(nBlk, 2)
    rows = blob[off_rows:off_rows + Bo * nBlk].reshape(nBlk, Bo)
    cols = blob[off_cols:off_cols + Bi * nBlk].reshape(nBlk, Bi)
    val_off = blob[off_voff:off_voff + 4 * (nBlk + 1)].view(np.uint32)
    vals = blob[off_vals:off_vals + nVals * es].view(np.float32 if dt == 0 else np.uint16)
    dense = np.zeros((O, I), dtype=vals.dtype)
    rk = np.zeros((nBo, nBi), dtype=np.uint64)
    ck = np.zeros((nBo, nBi), dtype=np.uint64)
    for bo in range(nBo):
        for bi in range(nBi):
            b = bo * nBi + bi
            nr, nc = int(cnt[b, 0]), int(cnt[b, 1])
            r = rows[b, :nr].astype(np.int64)
            c = cols[b, :nc].astype(np.int64)
            for v in r:
                rk[bo, bi] |= np.uint64(1 << int(v))
            for v in c:
                ck[bo, bi] |= np.uint64(1 << int(v))
            if nr and nc:
                p0 = int(val_off[b])
                dense[np.ix_(bo * Bo + r, bi * Bi + c)] = vals[p0:p0 + nr * nc].reshape(nr, nc)
    return dense, rk, ck
