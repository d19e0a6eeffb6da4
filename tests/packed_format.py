"""Reader and writer of the byte format that include/mwu.h documents for mwu_pack.

This is a FORMAT-CONFORMANCE helper, not part of the CPU checker: it restates the file format
of the header comment (records, class lists, entry order, byte offsets inside a record's tile)
so that tests can (a) read a packed buffer back into a weight matrix and (b) notice when the
bytes mwu_pack writes drift from what the header promises.  Whether the packed weights are the
RIGHT weights is judged elsewhere, against oracle.decoded_weights; nothing here is evidence of
parity with the paper.
"""
from __future__ import annotations

import struct

import numpy as np

from oracle import mwu_oracle as O

TILE_ROWS = 128          # rows of W per record
STAGE_K = 64             # reduction-axis extent per record
HEADER_BYTES = 256
SECTION_ALIGN = 256
MAGIC = b"MWUPACK1"
VERSION = 4

HEADER_FIELDS = ["magic", "version", "N", "K", "b", "n_pad", "n_tiles", "n_stages", "n_pruned",
                 "n_unified", "n_dense", "n_plist", "off_rec", "off_ulist", "off_dpos", "off_dpay",
                 "off_ppos", "total"]


def _align(x: int, a: int = SECTION_ALIGN) -> int:
    return (x + a - 1) // a * a


def packed_layout(N: int, K: int, b: int, n_unified: int, n_dense: int, n_pruned: int) -> dict:
    assert K % STAGE_K == 0 and STAGE_K % b == 0
    n_pad = _align(N, TILE_ROWS)
    n_tiles = n_pad // TILE_ROWS
    n_stages = K // STAGE_K
    n_plist = n_pruned + (n_pad - N) * (K // b)          # padding rows count as pruned
    off_rec = HEADER_BYTES
    off_ulist = _align(off_rec + 16 * (n_tiles * n_stages + 1))
    off_dpos = _align(off_ulist + 8 * n_unified)
    off_dpay = _align(off_dpos + 2 * n_dense)
    off_ppos = _align(off_dpay + 2 * b * n_dense)
    total = _align(off_ppos + 2 * n_plist)
    return dict(n_pad=n_pad, n_tiles=n_tiles, n_stages=n_stages, n_plist=n_plist, off_rec=off_rec,
                off_ulist=off_ulist, off_dpos=off_dpos, off_dpay=off_dpay, off_ppos=off_ppos,
                total=total)


def tile_offset(pos: np.ndarray, b: int) -> np.ndarray:
    """Byte offset of block slot `pos` in a record's 128 x 64 bf16 tile: row r = pos // (64/b)
    starts at (r // 8) * 1024 + (r % 8) * 128; the row's 16-byte chunk c is stored at chunk
    position c XOR (r % 8); inside a chunk bytes keep their order."""
    pos = np.asarray(pos, dtype=np.int64)
    nb = STAGE_K // b
    r, i = pos // nb, pos % nb
    byte_in_row = i * 2 * b
    c, within = byte_in_row // 16, byte_in_row % 16
    return (r // 8) * 1024 + (r % 8) * 128 + ((c ^ (r % 8)) * 16) + within


def tile_offset_inverse(off: int, b: int):
    r = (off >> 10) * 8 + ((off >> 7) & 7)
    c = ((off >> 4) & 7) ^ (r & 7)
    byte_in_row = c * 16 + (off & 15)
    return r, byte_in_row // (2 * b)


def entry_order(off: np.ndarray, b: int) -> np.ndarray:
    """Order of a class list: entries (given in ascending pos order) are dealt round-robin over
    the values of (off % 128) // min(2*b, 16): sort by (rank inside that value, value)."""
    off = np.asarray(off, dtype=np.int64)
    g = min(2 * b, 16)
    lane = (off % 128) // g
    rank = np.zeros(off.shape[0], dtype=np.int64)
    seen = {}
    for e, sl in enumerate(lane.tolist()):
        rank[e] = seen.get(sl, 0)
        seen[sl] = rank[e] + 1
    return np.lexsort((lane, rank))


def write(p: "O.Projection", b: int) -> np.ndarray:
    """The bytes mwu_pack must produce for this projection (1-dim blocks of width b)."""
    N, K = p.V.shape
    nb = STAGE_K // b
    n_unified = int(p.unified.sum())
    n_pruned = int(p.pruned.sum())
    n_dense = p.unified.shape[0] - n_unified - n_pruned
    L = packed_layout(N, K, b, n_unified, n_dense, n_pruned)
    n_pad, n_tiles, n_stages = L["n_pad"], L["n_tiles"], L["n_stages"]
    buf = np.zeros(L["total"], dtype=np.uint8)

    hdr = [int.from_bytes(MAGIC, "little"), VERSION, N, K, b, n_pad, n_tiles, n_stages,
           n_pruned, n_unified, n_dense, L["n_plist"], L["off_rec"], L["off_ulist"],
           L["off_dpos"], L["off_dpay"], L["off_ppos"], L["total"]]
    buf[:8 * len(hdr)] = np.frombuffer(struct.pack("<%dQ" % len(hdr), *hdr), dtype=np.uint8)

    pruned = np.ones((n_pad, K // b), dtype=bool)
    unified = np.zeros((n_pad, K // b), dtype=bool)
    pruned[:N] = p.pruned.reshape(N, K // b)
    unified[:N] = p.unified.reshape(N, K // b)
    sign = np.zeros((n_pad, K), dtype=bool)
    sign[:N] = p.sign
    u = np.zeros((n_pad, K // b), dtype=np.float32)
    u[:N] = p.u.reshape(N, K // b)
    vbf = np.zeros((n_pad, K), dtype=np.uint16)
    vbf[:N] = O.bf16_bits_rne(p.V)

    n_rec = n_tiles * n_stages
    rec = np.zeros((n_rec + 1, 4), dtype=np.uint32)
    ulist_w0, ulist_u, dpos, dpay, ppos = [], [], [], [], []
    n_u = n_d = n_p = 0
    ell = np.arange(b, dtype=np.uint32)
    bitw = (np.uint32(1) << (ell // 2 + 16 * (ell % 2)))           # spread sign bit of weight l
    ubf = O.bf16_bits_rne(u.reshape(-1)).reshape(u.shape).astype(np.uint32)
    for t in range(n_tiles):
        r0 = t * TILE_ROWS
        for s in range(n_stages):
            ri = t * n_stages + s
            P = pruned[r0:r0 + TILE_ROWS, s * nb:(s + 1) * nb]
            Uf = unified[r0:r0 + TILE_ROWS, s * nb:(s + 1) * nb]
            D = ~P & ~Uf
            live = 0
            for sl in range(4):                      # 16-wide slices of the stage
                lo = (sl * 16) // b
                hi = max(lo + 1, ((sl + 1) * 16) // b)
                if (~P[:, lo:hi]).any():
                    live |= 1 << sl
            rec[ri] = (n_u, n_d, n_p, live)
            pos_u = np.flatnonzero(Uf.reshape(-1)).astype(np.uint32)      # ascending pos
            pos_d = np.flatnonzero(D.reshape(-1)).astype(np.uint16)
            pos_p = np.flatnonzero(P.reshape(-1)).astype(np.uint16)
            pos_u = pos_u[entry_order(tile_offset(pos_u, b), b)]
            pos_d = pos_d[entry_order(tile_offset(pos_d, b), b)]
            pos_p = pos_p[entry_order(tile_offset(pos_p, b), b)]
            sg = sign[r0:r0 + TILE_ROWS, s * STAGE_K:(s + 1) * STAGE_K].reshape(TILE_ROWS * nb, b)
            sbits = (sg.astype(np.uint32) * bitw).sum(axis=1).astype(np.uint32)
            ulist_w0.append(sbits[pos_u])
            ub = ubf[r0:r0 + TILE_ROWS, s * nb:(s + 1) * nb].reshape(-1)[pos_u]
            ulist_u.append(tile_offset(pos_u, b).astype(np.uint32) | (ub << np.uint32(16)))
            dpos.append(tile_offset(pos_d, b).astype(np.uint16))
            vb = vbf[r0:r0 + TILE_ROWS, s * STAGE_K:(s + 1) * STAGE_K].reshape(TILE_ROWS * nb, b)
            dpay.append(vb[pos_d].reshape(-1))
            ppos.append(tile_offset(pos_p, b).astype(np.uint16))
            n_u += pos_u.shape[0]
            n_d += pos_d.shape[0]
            n_p += pos_p.shape[0]
    assert n_u == n_unified and n_d == n_dense and n_p == L["n_plist"]
    rec[n_rec] = (n_u, n_d, n_p, 0)

    def put(off, arr):
        raw = np.ascontiguousarray(arr).view(np.uint8).reshape(-1)
        buf[off:off + raw.shape[0]] = raw

    put(L["off_rec"], rec)
    if n_unified:
        ul = np.zeros((n_unified, 2), dtype=np.uint32)
        ul[:, 0] = np.concatenate(ulist_w0)
        ul[:, 1] = np.concatenate(ulist_u)
        put(L["off_ulist"], ul)
    if n_dense:
        put(L["off_dpos"], np.concatenate(dpos).astype(np.uint16))
        put(L["off_dpay"], np.concatenate(dpay).astype(np.uint16))
    if L["n_plist"]:
        put(L["off_ppos"], np.concatenate(ppos).astype(np.uint16))
    return buf


def parse_header(buf: np.ndarray) -> dict:
    vals = struct.unpack("<%dQ" % len(HEADER_FIELDS), bytes(buf[:8 * len(HEADER_FIELDS)]))
    h = dict(zip(HEADER_FIELDS, vals))
    assert h["magic"] == int.from_bytes(MAGIC, "little") and h["version"] == VERSION
    return h


def records(buf: np.ndarray) -> np.ndarray:
    """The record table, uint32 [n_records + 1][4]: ubase, dbase, pbase, live."""
    h = parse_header(buf)
    n_rec = h["n_tiles"] * h["n_stages"]
    return buf[h["off_rec"]:h["off_rec"] + 16 * (n_rec + 1)].view(np.uint32).reshape(-1, 4)


def read(buf: np.ndarray) -> np.ndarray:
    """Packed bytes -> the weights they stand for, fp64 [N][K]; every block slot must be listed
    exactly once."""
    h = parse_header(buf)
    N, K, b = h["N"], h["K"], h["b"]
    n_tiles, n_stages = h["n_tiles"], h["n_stages"]
    rec = records(buf)
    ulist = buf[h["off_ulist"]:h["off_ulist"] + 8 * h["n_unified"]].view(np.uint32).reshape(-1, 2)
    dpos = buf[h["off_dpos"]:h["off_dpos"] + 2 * h["n_dense"]].view(np.uint16)
    dpay = buf[h["off_dpay"]:h["off_dpay"] + 2 * b * h["n_dense"]].view(np.uint16)
    ppos = buf[h["off_ppos"]:h["off_ppos"] + 2 * h["n_plist"]].view(np.uint16)
    What = np.full((h["n_pad"], K), np.nan, dtype=np.float64)
    seen = np.zeros((h["n_pad"], K // b), dtype=np.int32)
    for t in range(n_tiles):
        for s in range(n_stages):
            ri = t * n_stages + s
            for e in range(int(rec[ri, 0]), int(rec[ri + 1, 0])):
                sbits, w1 = int(ulist[e, 0]), int(ulist[e, 1])
                uval = float(O.bf16_bits_to_f64(np.array([w1 >> 16], dtype=np.uint16))[0])
                r, i = tile_offset_inverse(w1 & 0xFFFF, b)
                seen[t * TILE_ROWS + r, s * (STAGE_K // b) + i] += 1
                for l in range(b):
                    neg = (sbits >> (l // 2 + 16 * (l % 2))) & 1
                    What[t * TILE_ROWS + r, s * STAGE_K + i * b + l] = -uval if neg else uval
            for e in range(int(rec[ri, 1]), int(rec[ri + 1, 1])):
                r, i = tile_offset_inverse(int(dpos[e]), b)
                k0 = s * STAGE_K + i * b
                seen[t * TILE_ROWS + r, s * (STAGE_K // b) + i] += 1
                What[t * TILE_ROWS + r, k0:k0 + b] = O.bf16_bits_to_f64(dpay[e * b:(e + 1) * b])
            for e in range(int(rec[ri, 2]), int(rec[ri + 1, 2])):
                r, i = tile_offset_inverse(int(ppos[e]), b)
                k0 = s * STAGE_K + i * b
                seen[t * TILE_ROWS + r, s * (STAGE_K // b) + i] += 1
                What[t * TILE_ROWS + r, k0:k0 + b] = 0.0
    assert np.all(seen == 1) and not np.isnan(What).any()
    return What[:N]
