"""CPU checker for micro-structured weight unification / pruning (arXiv 2106.08301).

TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, fp64 restatement of what
the paper defines; it exists so that the CUDA library can be checked against
something that is not itself.  It shares no code with the CUDA path, is never
imported by the library, knows nothing about how the CUDA kernels lay their data
out, and must not be tuned for speed.

What follows the paper directly
  * block partition of a weight tensor by a block shape -- Section 3.1, first paragraph
    (1-dim, 2-dim and 3-dim shapes; Table 1 lists [2,2], [4,1], [8,1], [2,2,2])
  * unified value q = mean |w| of the block          -- Section 3.1, text after Eq. (2)
  * sign rule  v = +q if w >= 0 else -q              -- Eq. (2)
  * pruning = the special case q = 0                 -- Section 3.1, "special situation"
  * Q-step is a Euclidean projection                 -- Eq. (7) and the sentence after it
  * Unify(W + U) is what ADMM calls                  -- Algorithm 1
  * pruned blocks are skipped, unified blocks share
    one multiplication per output                    -- Section 3.2, Fig. 2 text, Table 1
  * keeping 2 of every 4 consecutive weights         -- Section 4.7 (the pruning half of the
                                                        combination test)

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
  * axes of a block shape [D1, D2(, D3)] on a weight viewed as W[rows][cin * taps]
    (taps = kh*kw, reduction index = cin*taps + tap): D1 runs along the input channels
    (the reduction axis whose signed inputs are added before the one multiplication, the
    only axis Table 1's multiplier column counts), D2 along the output rows, D3 along the
    kernel taps; a tap count that D3 does not divide leaves a shorter last block
  * grouped pruning (not in the paper; a constraint set of this library that lets a
    tile-based GEMM skip work): the prune decision is taken for whole groups of
    group_rows x group_cols weights, the group's key being the sum of its blocks' prune keys

Parity status: every function below is pinned by tests/test_oracle_*.py against
closed forms, brute force or a library routine.  The mixed-mode rule is a reading,
pinned only stage by stage (each stage is an exact projection for its own count).
"""
from __future__ import annotations

import dataclasses
import struct
from typing import Optional, Tuple

import numpy as np


def count_from_permille(n_blocks: int, permille: int) -> int:
    """Integer count for a ratio given in 1/1000: round half up, integers only."""
    return (int(permille) * int(n_blocks) + 500) // 1000


# ----------------------------------------------------------------------------
# Section 3.1: the block partition
# ----------------------------------------------------------------------------
@dataclasses.dataclass(frozen=True)
class BlockShape:
    """Block shape [D1, D2, D3] on W[rows][cin * taps]: dk input channels x dr output rows x
    dt kernel taps.  The 1-dim blocks of b consecutive reduction-axis entries are (b, 1, 1)
    with taps = 1."""
    dk: int
    dr: int = 1
    dt: int = 1
    taps: int = 1


def as_shape(b) -> BlockShape:
    return b if isinstance(b, BlockShape) else BlockShape(int(b))


@dataclasses.dataclass
class Partition:
    idx: np.ndarray        # int64 [Mb][n_max]: flat indices of each block's weights, -1 = none
    size: np.ndarray       # int64 [Mb]: weights in the block
    n_max: int
    row_runs: bool = False  # blocks are consecutive runs of one row: idx == arange(N*K).reshape(Mb, n_max)


def partition(N: int, K: int, shape) -> Partition:
    """Blocks of W[N][K] in index order j = (row group, channel group, tap group); inside a
    block the weights are ordered (row, channel, tap)."""
    s = as_shape(shape)
    assert K % s.taps == 0
    cin = K // s.taps
    assert cin % s.dk == 0 and N % s.dr == 0, "block shape must tile rows and input channels"
    ntg = (s.taps + s.dt - 1) // s.dt
    n_max = s.dk * s.dr * s.dt
    assert n_max & (n_max - 1) == 0, "block size must be a power of two"
    gi, gc, gt = np.meshgrid(np.arange(N // s.dr), np.arange(cin // s.dk), np.arange(ntg), indexing="ij")
    r, c, t = np.meshgrid(np.arange(s.dr), np.arange(s.dk), np.arange(s.dt), indexing="ij")
    # first weight of block j, and the offset of member (r, c, t) from it
    first = (gi.reshape(-1) * s.dr) * K + (gc.reshape(-1) * s.dk) * s.taps + gt.reshape(-1) * s.dt
    offs = r.reshape(-1) * K + c.reshape(-1) * s.taps + t.reshape(-1)
    idx = (first[:, None] + offs[None, :]).astype(np.int64)
    if s.taps % s.dt == 0:
        return Partition(idx=idx, size=np.full(idx.shape[0], n_max, dtype=np.int64), n_max=n_max,
                         row_runs=(s.dr == 1 and s.dt == 1 and s.taps == 1))
    ok = (gt.reshape(-1) * s.dt)[:, None] + t.reshape(-1)[None, :] < s.taps
    idx = np.where(ok, idx, -1)
    size = ok.sum(axis=1).astype(np.int64)
    assert np.all(size & (size - 1) == 0), "a short last block must still hold a power of two"
    # members first, holes last, member order kept
    order = np.argsort(~ok, axis=1, kind="stable")
    idx = np.take_along_axis(idx, order, axis=1)
    return Partition(idx=idx, size=size, n_max=n_max)


def gather_blocks(V: np.ndarray, part: Partition) -> np.ndarray:
    """fp32 [Mb][n_max]: the blocks' values (0 in the holes of short blocks)."""
    flat = np.ascontiguousarray(V, dtype=np.float32).reshape(-1)
    if part.row_runs:
        return flat.reshape(-1, part.n_max).copy()
    out = flat[np.maximum(part.idx, 0)]
    out[part.idx < 0] = np.float32(0.0)
    return out


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
    q: np.ndarray      # S / n             (unified value),        fp64 [Mb]
    L_u: np.ndarray    # sum (|v| - q)^2   (unification loss),     fp64 [Mb]
    L_p: np.ndarray    # sum v^2           (prune loss),           fp64 [Mb]


def block_stats(V: np.ndarray, b, part: Optional[Partition] = None) -> BlockStats:
    """Per-block statistics of V[N][K]; b is a width (blocks of b consecutive entries of a row)
    or a BlockShape."""
    V = np.ascontiguousarray(V, dtype=np.float32)
    N, K = V.shape
    assert np.all(np.isfinite(V)), "non-finite weights are outside the method's domain"
    if part is None:
        part = partition(N, K, b)
    a = np.abs(gather_blocks(V, part).astype(np.float64))
    S = tree_sum(a)
    q = S / part.size.astype(np.float64)   # text after Eq. (2): average of |w|
    d = a - q[:, None]
    if int(part.size.min()) < part.n_max:
        d[part.idx < 0] = 0.0              # the holes of short blocks are not weights
    L_u = tree_sum(d * d)                  # distance^2 to the unified block (Eq. 7 projection)
    L_p = tree_sum(a * a)                  # distance^2 to the zero block (q = 0 special case)
    return BlockStats(S=S, q=q, L_u=L_u, L_p=L_p)


# ----------------------------------------------------------------------------
# selection by ratio (Section 3.1's example; Section 4.3: a threshold per block after training)
# ----------------------------------------------------------------------------
def group_prune_keys(prune_key: np.ndarray, N: int, K: int, b: int, group_rows: int,
                     group_cols: int) -> np.ndarray:
    """Key of every prune group of a 1-dim partition, fp64 [N/group_rows][K/group_cols]: the
    blocks of one row inside the group are summed first (pairwise tree in column order), then
    the rows of the group (pairwise tree in row order)."""
    assert N % group_rows == 0 and K % group_cols == 0 and group_cols % b == 0
    k4 = prune_key.reshape(N // group_rows, group_rows, K // group_cols, group_cols // b)
    per_row = tree_sum(k4)                                     # [tile][row][slice]
    return tree_sum(np.moveaxis(per_row, 1, -1))               # [tile][slice]


def select_blocks(stats: BlockStats, k_unify: int, k_prune: int,
                  prune_key: str = "l2sq", groups=None) -> Tuple[np.ndarray, np.ndarray]:
    """Return boolean masks (pruned, unified) over the Mb blocks.

    k_unify counts unified and pruned blocks together; k_prune <= k_unify.
    Order of blocks: key ascending, then block index ascending.
    groups = (N, K, b, group_rows, group_cols): blocks are pruned by whole groups (k_prune must
    be a multiple of the blocks per group); order of groups: key ascending, then group index
    (row tile, then column slice) ascending.
    """
    Mb = stats.S.shape[0]
    assert 0 <= k_prune <= k_unify <= Mb
    kp = stats.L_p if prune_key == "l2sq" else stats.S
    pruned = np.zeros(Mb, dtype=bool)
    if groups is None:
        order_p = np.argsort(kp, kind="stable")          # stable: ties keep index order
        pruned[order_p[:k_prune]] = True
    else:
        N, K, b, gr, gc = groups
        per_group = gr * gc // b
        assert k_prune % per_group == 0, "grouped pruning takes whole groups"
        gk = group_prune_keys(kp, N, K, b, gr, gc)
        order_g = np.argsort(gk.reshape(-1), kind="stable")[:k_prune // per_group]
        gmask = np.zeros(gk.size, dtype=bool)
        gmask[order_g] = True
        gmask = gmask.reshape(gk.shape)                   # [tile][slice]
        full = np.repeat(np.repeat(gmask, gr, axis=0), gc // b, axis=1)   # [N][K/b]
        pruned = full.reshape(-1).copy()
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
    part: Partition        # which weights each block holds


def project(W: np.ndarray, b, k_unify: int, k_prune: int,
            U: Optional[np.ndarray] = None, prune_key: str = "l2sq",
            prune_group: Optional[Tuple[int, int]] = None) -> Projection:
    V = combine_dual(W, U)
    N, K = V.shape
    part = partition(N, K, b)
    stats = block_stats(V, b, part)
    groups = None
    if prune_group is not None:
        s = as_shape(b)
        assert s.dr == 1 and s.dt == 1 and s.taps == 1, "grouped pruning is defined for 1-dim blocks"
        groups = (N, K, s.dk, prune_group[0], prune_group[1])
    pruned, unified = select_blocks(stats, k_unify, k_prune, prune_key, groups)
    q32 = stats.q.astype(np.float32)
    sign = V < 0                                     # -0.0 < 0 is False
    Qf = V.reshape(-1).copy()
    for cls, is_unified in ((unified, True), (pruned, False)):
        rows = np.flatnonzero(cls)
        if rows.size == 0:
            continue
        ii = part.idx[rows]
        mm = ii >= 0                                 # the holes of short blocks are not weights
        if is_unified:
            vals = np.where(sign.reshape(-1)[np.maximum(ii, 0)], -q32[rows, None], q32[rows, None])
        else:
            vals = np.zeros(ii.shape, dtype=np.float32)
        Qf[ii[mm]] = vals[mm].astype(np.float32)
    u = np.where(unified, q32, np.float32(0.0)).astype(np.float32)
    return Projection(Q=Qf.reshape(N, K), u=u, pruned=pruned, unified=unified,
                      sign=sign, stats=stats, V=V, part=part)


@dataclasses.dataclass
class DualUpdate:
    U_next: np.ndarray     # fp32 [N][K]
    residual_sq: float     # ||V - Q||_F^2 with unrounded unified magnitudes, fp64


def dual_update(p: Projection, b=None) -> DualUpdate:
    """Dual step of ADMM (Algorithm 1, last assignment of the loop; third ADMM step of Section
    3.3): U_{k+1} = U_k + W_{k+1} - Q_{k+1}.  With V = fp32(W_{k+1} + U_k), the tensor that was
    projected, this is V - Q: one fp32 subtraction per entry.  residual_sq is the quadratic term
    ||W - Q + U||_F^2 of the augmented Lagrangian of Section 3.3 (without rho/2) after the Q-step,
    summed per block from the fp64 block statistics: sum v^2 for a pruned block, the unification
    loss for a unified block, nothing for a block that keeps its values."""
    U_next = (p.V - p.Q).astype(np.float32)                 # fp32 - fp32, rounded once
    Vb = gather_blocks(p.V, p.part).astype(np.float64)
    sumsq = tree_sum(Vb * Vb)
    residual = float(np.sum(sumsq[p.pruned]) + np.sum(p.stats.L_u[p.unified]))
    return DualUpdate(U_next=U_next, residual_sq=residual)


# ----------------------------------------------------------------------------
# Section 4.7: "1x4 blocks with 50 % prune ratio in each block" -- keep n of every m
# ----------------------------------------------------------------------------
@dataclasses.dataclass
class KeepNofM:
    Q: np.ndarray          # fp32 [N][K]: kept weights copied, the others +0
    keep: np.ndarray       # bool [N][K]
    V: np.ndarray


def project_n_of_m(W: np.ndarray, n: int = 2, m: int = 4,
                   U: Optional[np.ndarray] = None) -> KeepNofM:
    """Euclidean projection onto "at most n non-zeros in every m consecutive entries of a row":
    the n entries of largest magnitude stay (equal magnitudes: the lower index stays)."""
    V = combine_dual(W, U)
    N, K = V.shape
    assert K % m == 0 and 0 <= n <= m
    a = np.abs(V.astype(np.float64)).reshape(-1, m)
    order = np.argsort(-a, axis=1, kind="stable")           # descending |v|, ties by index
    keep = np.zeros(a.shape, dtype=bool)
    np.put_along_axis(keep, order[:, :n], True, axis=1)
    Q = np.where(keep, V.reshape(-1, m), np.float32(0.0)).astype(np.float32)
    return KeepNofM(Q=Q.reshape(N, K), keep=keep.reshape(N, K), V=V)


def bitmap_words(mask: np.ndarray) -> np.ndarray:
    """bool[n] -> uint32[ceil(n/32)], bit (j % 32) of word (j // 32)."""
    n = mask.shape[0]
    padded = np.zeros(((n + 31) // 32) * 32, dtype=np.uint8)
    padded[:n] = mask.astype(np.uint8)
    bits = padded.reshape(-1, 32).astype(np.uint64)
    weights = (np.uint64(1) << np.arange(32, dtype=np.uint64))
    return (bits * weights).sum(axis=1).astype(np.uint32)


def bitmap_bools(words: np.ndarray, n: int) -> np.ndarray:
    w = np.ascontiguousarray(words, dtype=np.uint32)
    bits = (w[:, None] >> np.arange(32, dtype=np.uint32)[None, :]) & np.uint32(1)
    return bits.reshape(-1)[:n].astype(bool)


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
# storage form (Section 3.1 / Table 1: one magnitude per unified block, one sign bit
# per weight of a unified block, nothing for a pruned block, the values of the rest)
# ----------------------------------------------------------------------------
STORE_MAGIC = b"MWUSTORE"
STORE_FIELDS = ["magic", "N", "K", "n_blocks", "n_pruned", "n_unified", "n_dense",
                "n_unified_weights", "n_dense_weights"]


def storage_bits(p: Projection, value_bits: int = 32, dense_bits: int = 16) -> dict:
    """What the storage model costs for this projection, in bits, class by class."""
    size = p.part.size
    n_uw = int(size[p.unified].sum())
    dense = ~(p.pruned | p.unified)
    n_dw = int(size[dense].sum())
    return {"class_bits": 2 * int(size.shape[0]),           # which of the three classes a block has
            "unified_values": value_bits * int(p.unified.sum()),
            "unified_signs": n_uw,
            "dense_values": dense_bits * n_dw,
            "pruned": 0}


def pack(p: Projection) -> np.ndarray:
    """The storage form as one byte string: header, the two class bitmaps, then in ascending
    block order the fp32 magnitude of every unified block, the sign bits of the weights of the
    unified blocks (block after block, member order) and the bf16 values of the blocks that
    keep their values.  A pruned block contributes nothing but its bitmap bit."""
    N, K = p.V.shape
    dense = ~(p.pruned | p.unified)
    member = p.part.idx >= 0
    uni_idx = p.part.idx[p.unified][member[p.unified]]      # member order, block after block
    den_idx = p.part.idx[dense][member[dense]]
    hdr = [int.from_bytes(STORE_MAGIC, "little"), N, K, int(p.pruned.shape[0]), int(p.pruned.sum()),
           int(p.unified.sum()), int(dense.sum()), int(uni_idx.size), int(den_idx.size)]
    parts = [np.frombuffer(struct.pack("<%dQ" % len(hdr), *hdr), dtype=np.uint8),
             bitmap_words(p.pruned).view(np.uint8), bitmap_words(p.unified).view(np.uint8),
             p.u[p.unified].astype(np.float32).view(np.uint8),
             bitmap_words(p.sign.reshape(-1)[uni_idx]).view(np.uint8),
             bf16_bits_rne(p.V.reshape(-1)[den_idx]).view(np.uint8)]
    return np.concatenate(parts)


def unpack(buf: np.ndarray, b) -> np.ndarray:
    """Storage form -> the weights the layer multiplies with, fp64 [N][K]: 0 for a pruned block,
    +-bf16(u) by sign bit for a unified block, the stored bf16 value otherwise."""
    nh = 8 * len(STORE_FIELDS)
    h = dict(zip(STORE_FIELDS, struct.unpack("<%dQ" % len(STORE_FIELDS), bytes(buf[:nh]))))
    assert h["magic"] == int.from_bytes(STORE_MAGIC, "little")
    N, K, Mb = h["N"], h["K"], h["n_blocks"]
    part = partition(N, K, b)
    assert part.idx.shape[0] == Mb
    nw = (Mb + 31) // 32 * 4
    o = nh
    pruned = bitmap_bools(buf[o:o + nw].view(np.uint32), Mb); o += nw
    unified = bitmap_bools(buf[o:o + nw].view(np.uint32), Mb); o += nw
    u = buf[o:o + 4 * h["n_unified"]].view(np.float32); o += 4 * h["n_unified"]
    ns = (h["n_unified_weights"] + 31) // 32 * 4
    signs = bitmap_bools(buf[o:o + ns].view(np.uint32), h["n_unified_weights"]); o += ns
    vals = buf[o:o + 2 * h["n_dense_weights"]].view(np.uint16); o += 2 * h["n_dense_weights"]
    assert o == buf.shape[0]
    assert int(pruned.sum()) == h["n_pruned"] and int(unified.sum()) == h["n_unified"]
    member = part.idx >= 0
    dense = ~(pruned | unified)
    out = np.zeros(N * K, dtype=np.float64)
    uni_idx = part.idx[unified][member[unified]]
    u_bf = bf16_bits_to_f64(bf16_bits_rne(u))
    per_weight_u = np.repeat(u_bf, part.size[unified])
    out[uni_idx] = np.where(signs, -per_weight_u, per_weight_u)
    out[part.idx[dense][member[dense]]] = bf16_bits_to_f64(vals)
    return out.reshape(N, K)


def decoded_weights(p: Projection, b=None) -> np.ndarray:
    """W_hat straight from a projection (no byte format involved), fp64 [N][K]."""
    N, K = p.V.shape
    u_bf = bf16_bits_to_f64(bf16_bits_rne(p.u))
    out = bf16_bits_to_f64(bf16_bits_rne(p.V)).reshape(-1)
    member = p.part.idx >= 0
    sign = p.sign.reshape(-1)
    rows = np.flatnonzero(p.unified)
    ii, mm = p.part.idx[rows], member[rows]
    vals = np.where(sign[np.maximum(ii, 0)], -u_bf[rows, None], u_bf[rows, None])
    out[ii[mm]] = vals[mm]
    rows = np.flatnonzero(p.pruned)
    ii, mm = p.part.idx[rows], member[rows]
    out[ii[mm]] = 0.0
    return out.reshape(N, K)


# ----------------------------------------------------------------------------
# Section 3.2: the layer forward on compressed weights
# ----------------------------------------------------------------------------
def gemm(X: np.ndarray, What: np.ndarray) -> np.ndarray:
    """Y[m][n] = sum_k X[m][k] * W_hat[n][k] in fp64 (X holds bf16-representable values)."""
    return np.asarray(X, dtype=np.float64) @ np.asarray(What, dtype=np.float64).T


def gemm_shared_partial(X: np.ndarray, p: Projection, b: int) -> np.ndarray:
    """The paper's form (Fig. 2 text) for 1-dim blocks: pruned blocks are skipped; a unified
    block costs one multiplication per output: u * (signed sum of its inputs).  Dense blocks as
    usual."""
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
