"""CPU checker for micro-structured weight unification / pruning (arXiv 2106.08301).

TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, fp64 restatement of what
the paper defines; it exists so that the CUDA library can be checked against
something that is not itself.  It shares no code with the CUDA path, is never
imported by the library, and must not be tuned for speed.

What follows the paper directly
  * block partition of a weight tensor               -- Section 3.1, first paragraph
  * unified value q = mean |w| of the block          -- Section 3.1, text after Eq. (2)
  * sign rule  v = +q if w >= 0 else -q              -- Eq. (2)
  * pruning = the special case q = 0                 -- Section 3.1, "special situation"
  * Q-step is a Euclidean projection                 -- Eq. (7) and the sentence after it
  * Unify(W + U) is what ADMM calls                  -- Algorithm 1
  * pruned blocks are skipped, unified blocks share
    one multiplication per output                    -- Section 3.2, Fig. 2 text, Table 1

Readings where the paper is silent (each is also pinned stage-wise by tests)
  * unification loss of a block  L_u = sum (|v| - q)^2   (squared distance to its
    unified image; the paper only says "Euclidean projection")
  * prune loss of a block        L_p = sum v^2           (squared distance to zero);
    the L1 norm the Fig. 1 walk-through mentions is available as prune_key="l1"
  * for a ratio below 100 % the blocks with the smallest loss are chosen
  * mixed mode: prune first (k_p smallest prune keys over all blocks), then unify
    the k_u - k_p smallest L_u among the blocks that were not pruned
  * ties go to the lower block index
  * sign bit = (v < 0), so -0.0 and +0.0 both count as ">= 0"
  * fp64 arithmetic, every operation rounded on its own, block sums taken as a
    balanced pairwise tree (l with l^1, then l^2, ...)

Parity status: every function below is pinned by tests/test_oracle_*.py against
closed forms, brute force or a library routine.  The mixed-mode rule is a reading,
pinned only stage by stage (each stage is an exact projection for its own count).
"""
from __future__ import annotations

import dataclasses
import struct
from typing import Optional, Tuple

import numpy as np

# ----------------------------------------------------------------------------
# packed format constants (a file format shared by specification, not by code)
# ----------------------------------------------------------------------------
TILE_ROWS = 128          # rows of W per record
STAGE_K = 64             # reduction-axis extent per record
HEADER_BYTES = 256
SECTION_ALIGN = 256
MAGIC = b"MWUPACK1"
VERSION = 4


def count_from_permille(n_blocks: int, permille: int) -> int:
    """Integer count for a ratio given in 1/1000: round half up, integers only."""
    return (int(permille) * int(n_blocks) + 500) // 1000


# ----------------------------------------------------------------------------
# Section 3.1: block statistics
# ----------------------------------------------------------------------------
def combine_dual(W: np.ndarray, U: Optional[np.ndarray]) -> np.ndarray:
    """Input of Unify(): W, or W + U rounded once to fp32 (Algorithm 1, Q-step)."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    if U is None:
        return W
    U = np.ascontiguousarray(U, dtype=np.float32)
    return (W + U).astype(np.float32)      # fp32 + fp32 -> one fp32 rounding


def tree_sum(x: np.ndarray) -> np.ndarray:
    """Balanced pairwise sum over the last axis (length a power of two)."""
    n = x.shape[-1]
    assert n >= 1 and (n & (n - 1)) == 0, "block width must be a power of two"
    while x.shape[-1] > 1:
        x = x[..., 0::2] + x[..., 1::2]
    return x[..., 0]


@dataclasses.dataclass
class BlockStats:
    S: np.ndarray      # sum |v|           (L1 norm of the block), fp64 [Mb]
    q: np.ndarray      # S / b             (unified value),        fp64 [Mb]
    L_u: np.ndarray    # sum (|v| - q)^2   (unification loss),     fp64 [Mb]
    L_p: np.ndarray    # sum v^2           (prune loss),           fp64 [Mb]


def block_stats(V: np.ndarray, b: int) -> BlockStats:
    """Per-block statistics of V[N][K] with blocks of b consecutive entries of a row."""
    V = np.ascontiguousarray(V, dtype=np.float32)
    N, K = V.shape
    assert K % b == 0
    assert np.all(np.isfinite(V)), "non-finite weights are outside the method's domain"
    a = np.abs(V.astype(np.float64)).reshape(N * (K // b), b)
    S = tree_sum(a)
    q = S / float(b)                       # text after Eq. (2): average of |w|
    d = a - q[:, None]
    L_u = tree_sum(d * d)                  # distance^2 to the unified block (Eq. 7 projection)
    L_p = tree_sum(a * a)                  # distance^2 to the zero block (q = 0 special case)
    return BlockStats(S=S, q=q, L_u=L_u, L_p=L_p)


# ----------------------------------------------------------------------------
# selection by ratio (Section 3.1 example; Section 4.3 "threshold is applied to each block")
# ----------------------------------------------------------------------------
def select_blocks(stats: BlockStats, k_unify: int, k_prune: int,
                  prune_key: str = "l2sq") -> Tuple[np.ndarray, np.ndarray]:
    """Return boolean masks (pruned, unified) over the Mb blocks.

    k_unify counts unified and pruned blocks together; k_prune <= k_unify.
    Order of blocks: key ascending, then block index ascending.
    """
    Mb = stats.S.shape[0]
    assert 0 <= k_prune <= k_unify <= Mb
    kp = stats.L_p if prune_key == "l2sq" else stats.S
    order_p = np.argsort(kp, kind="stable")          # stable: ties keep index order
    pruned = np.zeros(Mb, dtype=bool)
    pruned[order_p[:k_prune]] = True
    rest = np.flatnonzero(~pruned)                   # ascending block index
    order_u = rest[np.argsort(stats.L_u[rest], kind="stable")]
    unified = np.zeros(Mb, dtype=bool)
    unified[order_u[:k_unify - k_prune]] = True
    return pruned, unified


# ----------------------------------------------------------------------------
# Eq. (2) and the q = 0 special case: the projected tensor
# ----------------------------------------------------------------------------
@dataclasses.dataclass
class Projection:
    Q: np.ndarray          # fp32 [N][K]
    u: np.ndarray          # fp32 [Mb]: fp32(q) on unified blocks, +0 elsewhere
    pruned: np.ndarray     # bool [Mb]
    unified: np.ndarray    # bool [Mb]
    sign: np.ndarray       # bool [N][K]: v < 0
    stats: BlockStats
    V: np.ndarray          # fp32 [N][K]: the tensor that was projected


def project(W: np.ndarray, b: int, k_unify: int, k_prune: int,
            U: Optional[np.ndarray] = None, prune_key: str = "l2sq") -> Projection:
    V = combine_dual(W, U)
    N, K = V.shape
    stats = block_stats(V, b)
    pruned, unified = select_blocks(stats, k_unify, k_prune, prune_key)
    q32 = stats.q.astype(np.float32)
    Vb = V.reshape(-1, b)
    Qb = Vb.copy()
    sign = Vb < 0                                    # -0.0 < 0 is False
    uni_vals = np.where(sign, -q32[:, None], q32[:, None]).astype(np.float32)
    Qb[unified] = uni_vals[unified]
    Qb[pruned] = np.float32(0.0)
    u = np.where(unified, q32, np.float32(0.0)).astype(np.float32)
    return Projection(Q=Qb.reshape(N, K), u=u, pruned=pruned, unified=unified,
                      sign=sign.reshape(N, K), stats=stats, V=V)


@dataclasses.dataclass
class DualUpdate:
    U_next: np.ndarray     # fp32 [N][K]
    residual_sq: float     # ||V - Q||_F^2 with unrounded unified magnitudes, fp64


def dual_update(p: Projection, b: int) -> DualUpdate:
    """Dual step of ADMM (Algorithm 1, last assignment of the loop; third ADMM step of Section
    3.3): U_{k+1} = U_k + W_{k+1} - Q_{k+1}.  With V = fp32(W_{k+1} + U_k), the tensor that was
    projected, this is V - Q: one fp32 subtraction per entry.  residual_sq is the quadratic term
    ||W - Q + U||_F^2 of the augmented Lagrangian of Section 3.3 (without rho/2) after the Q-step,
    summed per block from the fp64 block statistics: sum v^2 for a pruned block, the unification
    loss for a unified block, nothing for a block that keeps its values."""
    U_next = (p.V - p.Q).astype(np.float32)                 # fp32 - fp32, rounded once
    Vb = p.V.reshape(-1, b).astype(np.float64)
    sumsq = tree_sum(Vb * Vb)
    residual = float(np.sum(sumsq[p.pruned]) + np.sum(p.stats.L_u[p.unified]))
    return DualUpdate(U_next=U_next, residual_sq=residual)


def bitmap_words(mask: np.ndarray) -> np.ndarray:
    """bool[n] -> uint32[ceil(n/32)], bit (j % 32) of word (j // 32)."""
    n = mask.shape[0]
    padded = np.zeros(((n + 31) // 32) * 32, dtype=np.uint8)
    padded[:n] = mask.astype(np.uint8)
    bits = padded.reshape(-1, 32).astype(np.uint64)
    weights = (np.uint64(1) << np.arange(32, dtype=np.uint64))
    return (bits * weights).sum(axis=1).astype(np.uint32)


# ----------------------------------------------------------------------------
# bf16 (1 sign, 8 exponent, 7 fraction bits), round to nearest even
# ----------------------------------------------------------------------------
def bf16_bits_rne(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round-to-nearest-even, finite inputs."""
    bits = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    lsb = (bits >> np.uint64(16)) & np.uint64(1)
    rounded = (bits + np.uint64(0x7FFF) + lsb) >> np.uint64(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f64(h: np.ndarray) -> np.ndarray:
    return (h.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


# ----------------------------------------------------------------------------
# packed format (storage model of Section 3.1 / Table 1: one magnitude per
# unified block, one sign bit per weight, nothing for pruned blocks)
# ----------------------------------------------------------------------------
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
    """Byte offset of block slot `pos` in a decoded 128 x 64 bf16 tile: row r = pos // (64/b)
    starts at (r // 8) * 1024 + (r % 8) * 128; the row's 16-byte chunk c is stored at chunk
    position c XOR (r % 8); inside a chunk bytes keep their order."""
    pos = np.asarray(pos, dtype=np.int64)
    nb = STAGE_K // b
    r, i = pos // nb, pos % nb
    byte_in_row = i * 2 * b
    c, within = byte_in_row // 16, byte_in_row % 16
    return (r // 8) * 1024 + (r % 8) * 128 + ((c ^ (r % 8)) * 16) + within


def slot_order(off: np.ndarray, b: int) -> np.ndarray:
    """Permutation that deals entries (given in ascending pos order) round-robin over their
    store slots: sort by (rank inside the slot, slot)."""
    off = np.asarray(off, dtype=np.int64)
    g = min(2 * b, 16)
    slot = (off % 128) // g
    rank = np.zeros(off.shape[0], dtype=np.int64)
    seen = {}
    for e, sl in enumerate(slot.tolist()):
        rank[e] = seen.get(sl, 0)
        seen[sl] = rank[e] + 1
    return np.lexsort((slot, rank))


def tile_offset_inverse(off: int, b: int):
    r = (off >> 10) * 8 + ((off >> 7) & 7)
    c = ((off >> 4) & 7) ^ (r & 7)
    byte_in_row = c * 16 + (off & 15)
    return r, byte_in_row // (2 * b)


HEADER_FIELDS = ["magic", "version", "N", "K", "b", "n_pad", "n_tiles", "n_stages", "n_pruned",
                 "n_unified", "n_dense", "n_plist", "off_rec", "off_ulist", "off_dpos", "off_dpay",
                 "off_ppos", "total"]


def pack(p: Projection, b: int) -> np.ndarray:
    """Serialise a projection into the packed byte format (uint8 array).

    A record is (row tile of 128 rows) x (64 reduction-axis entries) and holds 128 * 64/b
    block slots; slot number pos = row_in_tile * (64/b) + block_in_stage.  A block is addressed
    by the byte offset `off` of its first value inside the record's decoded tile (bf16, rows of
    128 bytes, 16-byte chunks of a row XOR-permuted by the row number mod 8 -- the layout the
    tensor-core instruction reads; see tile_offset).  Per record the blocks are listed by
    class.  Inside a class list the entries are dealt round-robin over the store slots
    slot = (off % 128) // g, g = min(2*b, 16): entries with the same slot keep ascending pos
    order, and the list takes the first entry of every slot (ascending slot), then the second of
    every slot that has one, and so on (so that neighbouring entries fall into different
    shared-memory banks when the GEMM writes them):
      ulist  8 B per unified block: u32 spread sign bits (weight l -> bit l//2 + 16*(l%2)),
             u16 off, u16 bf16(unified value)
      dpos   u16 off per dense block;  dpay  its b values as bf16 (round to nearest even)
      ppos   u16 off per pruned block (rows beyond N are padding and count as pruned)
    rec[i] = (u32 ubase, dbase, pbase, live) gives where record i starts in each list; rec has
    one extra entry holding the totals.  live bit s = some row of the record has a non-pruned
    block overlapping columns [16s, 16s+16).
    """
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
    vbf[:N] = bf16_bits_rne(p.V)

    n_rec = n_tiles * n_stages
    rec = np.zeros((n_rec + 1, 4), dtype=np.uint32)
    ulist_w0, ulist_u, dpos, dpay, ppos = [], [], [], [], []
    n_u = n_d = n_p = 0
    ell = np.arange(b, dtype=np.uint32)
    bitw = (np.uint32(1) << (ell // 2 + 16 * (ell % 2)))           # spread sign bit of weight l
    ubf = bf16_bits_rne(u.reshape(-1)).reshape(u.shape).astype(np.uint32)
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
            pos_u = pos_u[slot_order(tile_offset(pos_u, b), b)]
            pos_d = pos_d[slot_order(tile_offset(pos_d, b), b)]
            pos_p = pos_p[slot_order(tile_offset(pos_p, b), b)]
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


def decode(buf: np.ndarray) -> np.ndarray:
    """Packed bytes -> decoded weights W_hat[N][K] in fp64.

    pruned block -> 0; unified block -> +-bf16(u) by sign bit; dense block ->
    its stored bf16 values.  This is what the GEMM multiplies with.
    """
    h = parse_header(buf)
    N, K, b = h["N"], h["K"], h["b"]
    nb = STAGE_K // b
    n_tiles, n_stages = h["n_tiles"], h["n_stages"]
    n_rec = n_tiles * n_stages
    rec = buf[h["off_rec"]:h["off_rec"] + 16 * (n_rec + 1)].view(np.uint32).reshape(-1, 4)
    ulist = buf[h["off_ulist"]:h["off_ulist"] + 8 * h["n_unified"]].view(np.uint32).reshape(-1, 2)
    dpos = buf[h["off_dpos"]:h["off_dpos"] + 2 * h["n_dense"]].view(np.uint16)
    dpay = buf[h["off_dpay"]:h["off_dpay"] + 2 * b * h["n_dense"]].view(np.uint16)
    ppos = buf[h["off_ppos"]:h["off_ppos"] + 2 * h["n_plist"]].view(np.uint16)
    What = np.full((h["n_pad"], K), np.nan, dtype=np.float64)     # every slot must be listed once
    for t in range(n_tiles):
        for s in range(n_stages):
            ri = t * n_stages + s
            for e in range(int(rec[ri, 0]), int(rec[ri + 1, 0])):
                sbits, w1 = int(ulist[e, 0]), int(ulist[e, 1])
                uval = float(bf16_bits_to_f64(np.array([w1 >> 16], dtype=np.uint16))[0])
                r, i = tile_offset_inverse(w1 & 0xFFFF, b)
                for l in range(b):
                    neg = (sbits >> (l // 2 + 16 * (l % 2))) & 1
                    What[t * TILE_ROWS + r, s * STAGE_K + i * b + l] = -uval if neg else uval
            for e in range(int(rec[ri, 1]), int(rec[ri + 1, 1])):
                r, i = tile_offset_inverse(int(dpos[e]), b)
                k0 = s * STAGE_K + i * b
                What[t * TILE_ROWS + r, k0:k0 + b] = bf16_bits_to_f64(dpay[e * b:(e + 1) * b])
            for e in range(int(rec[ri, 2]), int(rec[ri + 1, 2])):
                r, i = tile_offset_inverse(int(ppos[e]), b)
                k0 = s * STAGE_K + i * b
                What[t * TILE_ROWS + r, k0:k0 + b] = 0.0
    assert not np.isnan(What).any()
    return What[:N]


def decoded_weights(p: Projection, b: int) -> np.ndarray:
    """W_hat straight from a projection (no byte format involved), fp64 [N][K]."""
    N, K = p.V.shape
    u_bf = bf16_bits_to_f64(bf16_bits_rne(p.u))
    v_bf = bf16_bits_to_f64(bf16_bits_rne(p.V)).reshape(-1, b)
    out = v_bf.copy()
    uni = np.where(p.sign.reshape(-1, b), -u_bf[:, None], u_bf[:, None])
    out[p.unified] = uni[p.unified]
    out[p.pruned] = 0.0
    return out.reshape(N, K)


# ----------------------------------------------------------------------------
# Section 3.2: the layer forward on compressed weights
# ----------------------------------------------------------------------------
def gemm(X: np.ndarray, What: np.ndarray) -> np.ndarray:
    """Y[m][n] = sum_k X[m][k] * W_hat[n][k] in fp64 (X holds bf16-representable values)."""
    return np.asarray(X, dtype=np.float64) @ np.asarray(What, dtype=np.float64).T


def gemm_shared_partial(X: np.ndarray, p: Projection, b: int) -> np.ndarray:
    """The paper's form (Fig. 2 text): pruned blocks are skipped; a unified block costs one
    multiplication per output: u * (signed sum of its inputs).  Dense blocks as usual."""
    X = np.asarray(X, dtype=np.float64)
    M = X.shape[0]
    N, K = p.V.shape
    nbr = K // b
    u_bf = bf16_bits_to_f64(bf16_bits_rne(p.u)).reshape(N, nbr)
    v_bf = bf16_bits_to_f64(bf16_bits_rne(p.V)).reshape(N, nbr, b)
    sgn = np.where(p.sign.reshape(N, nbr, b), -1.0, 1.0)
    pr = p.pruned.reshape(N, nbr)
    un = p.unified.reshape(N, nbr)
    Xb = X.reshape(M, nbr, b)
    Y = np.zeros((M, N), dtype=np.float64)
    for n in range(N):
        for j in range(nbr):
            if pr[n, j]:
                continue                                  # skipped entirely
            if un[n, j]:
                Y[:, n] += u_bf[n, j] * (Xb[:, j, :] * sgn[n, j]).sum(axis=1)
            else:
                Y[:, n] += Xb[:, j, :] @ v_bf[n, j]
    return Y


def conv2d_direct(x: np.ndarray, What: np.ndarray, kh: int, kw: int, stride: int,
                  pad: int) -> np.ndarray:
    """Direct convolution, NCHW, zero padding, fp64.  W_hat is [cout][cin*kh*kw] in
    [cout, cin, kh, kw] order.  y[n][o][oh][ow] = sum_{c,i,j} x[n][c][oh*s+i-p][ow*s+j-p] w[o][c][i][j]."""
    x = np.asarray(x, dtype=np.float64)
    B, C, H, Wd = x.shape
    O = What.shape[0]
    w4 = np.asarray(What, dtype=np.float64).reshape(O, C, kh, kw)
    OH = (H + 2 * pad - kh) // stride + 1
    OW = (Wd + 2 * pad - kw) // stride + 1
    xp = np.zeros((B, C, H + 2 * pad, Wd + 2 * pad), dtype=np.float64)
    xp[:, :, pad:pad + H, pad:pad + Wd] = x
    y = np.zeros((B, O, OH, OW), dtype=np.float64)
    for i in range(kh):
        for j in range(kw):
            patch = xp[:, :, i:i + stride * (OH - 1) + 1:stride, j:j + stride * (OW - 1) + 1:stride]
            y += np.einsum("bchw,oc->bohw", patch, w4[:, :, i, j])
    return y


# ----------------------------------------------------------------------------
# Table 1 accounting: multipliers and storage of one unified block
# ----------------------------------------------------------------------------
def multiplies_per_block(shape: Tuple[int, ...]) -> Tuple[int, int]:
    """(dense multiplies, unified multiplies) of one block for one column of the other operand.

    Dense: one multiply per weight.  Unified: along the block's first axis the signed inputs
    are added first and the shared magnitude multiplies the sum once, so the multiplies drop
    by the extent of that axis; the remaining axes index different partial results (Section
    3.2: a 2x2 block needs 4 multipliers instead of 8 for two columns, i.e. 2 instead of 4
    per column).  This reading reproduces every row of Table 1.
    """
    n = int(np.prod(shape))
    return n, n // int(shape[0])


def multiplier_reduction(shape: Tuple[int, ...]) -> float:
    dense, unified = multiplies_per_block(shape)
    return dense / unified


def storage_reduction(shape: Tuple[int, ...], include_sign_bits: bool = False,
                      value_bits: int = 32) -> float:
    n = int(np.prod(shape))
    dense_bits = n * value_bits
    unified_bits = value_bits + (n if include_sign_bits else 0)
    return dense_bits / unified_bits
