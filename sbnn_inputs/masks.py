"""Group masks: which (output-channel group, input channel) units a layer keeps.

A unit is the G weights (1x1) or 9*G weights (3x3) that connect one input
channel to one group of G consecutive output channels.  The functions here
return a boolean unit mask of shape [Cout/G][Cin] (True = kept) and
`expand_mask` broadcasts it to the full weight shape.
"""
from __future__ import annotations

import numpy as np

from .rng import u64_stream


def removed_units(units: int, sparsity_pct: int) -> int:
    """Number of units to remove for an integer sparsity percentage, rounding halves up."""
    if not 0 <= sparsity_pct <= 100:
        raise ValueError("sparsity_pct must be in [0, 100]")
    return (sparsity_pct * units + 50) // 100


def _ranks(keys: np.ndarray) -> np.ndarray:
    """Rank of every key along the last axis (stable: equal keys keep index order)."""
    order = np.argsort(keys, axis=-1, kind="stable")
    ranks = np.empty_like(order)
    np.put_along_axis(ranks, order, np.broadcast_to(np.arange(keys.shape[-1]), keys.shape), axis=-1)
    return ranks


def group_mask_balanced(seed: int, stream: int, ngroups: int, cin: int, sparsity_pct: int, gi: int = 1) -> np.ndarray:
    """Per group, a uniform-random subset of input channels is removed.

    The layer removes removed_units(ngroups*cin/gi, pct) blocks of gi aligned
    input channels in total; every group removes the same number, except that
    the first (total mod ngroups) groups remove one more.  Within a group the
    blocks with the smallest random keys go.
    """
    if cin % gi:
        raise ValueError("cin must be a multiple of gi")
    nblk = cin // gi
    total = removed_units(ngroups * nblk, sparsity_pct)
    base, extra = divmod(total, ngroups)
    per_group = np.full(ngroups, base, dtype=np.int64)
    per_group[:extra] += 1
    keys = u64_stream(seed, stream, ngroups * nblk).reshape(ngroups, nblk)
    kept_blk = _ranks(keys) >= per_group[:, None]
    return np.repeat(kept_blk, gi, axis=1)


def group_mask_layer_global(seed: int, stream: int, ngroups: int, cin: int, sparsity_pct: int) -> np.ndarray:
    """The removed units are a uniform-random subset of the whole layer, so the kept count varies by group."""
    units = ngroups * cin
    total = removed_units(units, sparsity_pct)
    keys = u64_stream(seed, stream, units)
    return (_ranks(keys) >= total).reshape(ngroups, cin)


def group_mask_magnitude(w: np.ndarray, g: int, sparsity_pct: int) -> np.ndarray:
    """Units ranked by the l1 norm of their weights over the whole layer; the smallest are removed.

    w has shape [Cout][KH][KW][Cin].
    """
    cout, kh, kw, cin = w.shape
    ngroups = cout // g
    l1 = np.abs(w.astype(np.float64)).reshape(ngroups, g * kh * kw, cin).sum(axis=1)
    total = removed_units(ngroups * cin, sparsity_pct)
    return (_ranks(l1.reshape(-1)) >= total).reshape(ngroups, cin)


def expand_mask(unit_mask: np.ndarray, g: int, kh: int, kw: int) -> np.ndarray:
    """Broadcast a [ngroups][Cin] unit mask to a uint8 mask of shape [ngroups*g][kh][kw][Cin]."""
    ngroups, cin = unit_mask.shape
    m = np.broadcast_to(unit_mask[:, None, None, None, :], (ngroups, g, kh, kw, cin))
    return np.ascontiguousarray(m.reshape(ngroups * g, kh, kw, cin)).astype(np.uint8)


def tap_pattern_mask(seed: int, stream: int, unit_mask: np.ndarray, g: int, kept_taps: int = 4) -> np.ndarray:
    """3x3 kernel patterns on top of a unit mask: every kept unit keeps the centre tap and `kept_taps - 1` of the
    other eight (those with the largest random keys), the same pattern for the g filters of the group.

    With kept_taps = 4 these are the C(8,3) = 56 four-entry patterns of pattern-based pruning.  Returns a uint8
    mask of shape [ngroups*g][3][3][Cin].
    """
    if not 1 <= kept_taps <= 9:
        raise ValueError("kept_taps must be in [1, 9]")
    ngroups, cin = unit_mask.shape
    keys = u64_stream(seed, stream, ngroups * cin * 8).reshape(ngroups, cin, 8)
    others = _ranks(keys) >= 8 - (kept_taps - 1)                      # [ngroups][cin][8]: taps 0-3 and 5-8
    taps = np.ones((ngroups, cin, 9), dtype=bool)
    taps[:, :, [0, 1, 2, 3, 5, 6, 7, 8]] = others
    taps &= unit_mask[:, :, None]
    m = np.broadcast_to(taps.transpose(0, 2, 1).reshape(ngroups, 1, 3, 3, cin), (ngroups, g, 3, 3, cin))
    return np.ascontiguousarray(m.reshape(ngroups * g, 3, 3, cin)).astype(np.uint8)


def dw_pattern_mask(seed: int, stream: int, c: int, go: int, w: np.ndarray | None = None) -> np.ndarray:
    """3:9 patterns for depthwise 3x3 weights [3][3][C]: in every kernel row the middle weight stays and either the
    first or the third column goes, one choice per row and per block of `go` consecutive channels.

    With w given, a block keeps in each row the side whose weights have the larger l1 norm over the block (the
    pattern that maximises the remaining l1 norm); otherwise the side is drawn at random.  Returns uint8 [3][3][C].
    """
    if c % go:
        raise ValueError("C must be a multiple of go")
    nblk = c // go
    if w is None:
        drop_third = (u64_stream(seed, stream, 3 * nblk).reshape(3, nblk) >> np.uint64(63)).astype(bool)
    else:
        l1 = np.abs(np.asarray(w, dtype=np.float64)).reshape(3, 3, nblk, go).sum(axis=3)   # [kh][kw][blk]
        drop_third = l1[:, 0, :] >= l1[:, 2, :]
    m = np.ones((3, 3, nblk, go), dtype=np.uint8)
    m[:, 2][drop_third] = 0
    m[:, 0][~drop_third] = 0
    return m.reshape(3, 3, c)
