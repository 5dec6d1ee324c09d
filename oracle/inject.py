"""Seeded soft-error injection into worker outputs (test oracle; numpy).

Error Model 2 of the paper (Section V-B) corrupts the entire output of an erroneous
node with additive continuous noise; the workloads also ask for single-bit flips and
for additive errors on a random subset of entries.  All draws come from one
counter-based generator, SplitMix64 (Steele, Lea, Flood 2014) used statelessly:

    mix64(z)        = SplitMix64 output function applied to z + GAMMA
    draw(key, ctr)  = mix64(key + ctr * GAMMA)      (the (ctr+1)-th output of a SplitMix64 seeded with key)
    key(seed,tag,p) = mix64(mix64(seed ^ (tag * TAGMUL)) + p)

so that any entry's error can be computed independently of all others.  The CUDA
library implements the same published generator on its own; no code is shared.

Modes
    bitflip : `count` distinct nodes, one entry each, one bit each; a bit is redrawn
              until the change is at least 2^-6 * scale in magnitude or non-finite
              (smaller changes are below the arithmetic's own noise and not the
              subject of the method).
    additive: each selected node gets errors on a random subset of entries (one
              guaranteed entry plus Bernoulli(phi_p) on the rest, phi_p ~ U(0,1]);
              magnitude (1+f) * 2^k * scale, k uniform in {-4..7}, f uniform in [0,1),
              random sign.
    gauss   : each selected node gets scale * N(0,1) added to every entry
              (Error Model 2 verbatim; Box-Muller in FP64).
Nodes are selected independently with probability `prob`, or given explicitly.
"""

from __future__ import annotations

from typing import Optional, Sequence

import numpy as np

U64 = np.uint64
GAMMA = U64(0x9E3779B97F4A7C15)
M1 = U64(0xBF58476D1CE4E5B9)
M2 = U64(0x94D049BB133111EB)
TAGMUL = U64(0xD6E8FEB86659FD93)

TAG_NODE, TAG_PHI, TAG_ENTRY, TAG_MAG, TAG_FIRST, TAG_BITFLIP, TAG_GAUSS = 1, 2, 3, 4, 5, 6, 7

def mix64(z):
    with np.errstate(over="ignore"):          # arithmetic is modulo 2^64 by design
        z = (np.asarray(z, dtype=U64) + GAMMA).astype(U64)
        z = ((z ^ (z >> U64(30))) * M1).astype(U64)
        z = ((z ^ (z >> U64(27))) * M2).astype(U64)
        return (z ^ (z >> U64(31))).astype(U64)


def draw(key, ctr):
    with np.errstate(over="ignore"):
        return mix64((np.asarray(key, dtype=U64) + np.asarray(ctr, dtype=U64) * GAMMA).astype(U64))


def make_key(seed: int, tag: int, p=0):
    with np.errstate(over="ignore"):
        s = U64(seed & 0xFFFFFFFFFFFFFFFF) ^ (U64(tag) * TAGMUL)
        return mix64((mix64(s) + np.asarray(p, dtype=U64)).astype(U64))


def unit(r):
    """Uniform double in [0,1) from the top 53 bits."""
    return (np.asarray(r, dtype=U64) >> U64(11)).astype(np.float64) * 2.0 ** -53


def select_nodes(seed: int, P: int, prob: float) -> np.ndarray:
    """Node p is erroneous iff its uniform draw is below prob."""
    u = unit(draw(make_key(seed, TAG_NODE), np.arange(P, dtype=U64)))
    return u < prob


def inject_bitflip(outputs: np.ndarray, seed: int, count: int, scale: float) -> np.ndarray:
    """In place on outputs [P, ...] (float32 or float64).  Returns bool[P] of corrupted nodes."""
    P = outputs.shape[0]
    flat = outputs.reshape(P, -1)
    L = flat.shape[1]
    nbits = flat.dtype.itemsize * 8
    itype = np.uint32 if nbits == 32 else np.uint64
    key = make_key(seed, TAG_BITFLIP)
    ctr = 0
    hit = np.zeros(P, dtype=bool)
    done = 0
    while done < min(count, P):
        p = int(draw(key, ctr) % U64(P)); ctr += 1
        if hit[p]:
            continue
        l = int(draw(key, ctr) % U64(L)); ctr += 1
        old = flat[p, l]
        for _ in range(4096):
            b = int(draw(key, ctr) % U64(nbits)); ctr += 1
            word = np.array([old]).view(itype)
            new = (word ^ itype(1 << b)).view(flat.dtype)[0]
            if (not np.isfinite(new)) or abs(float(new) - float(old)) >= 2.0 ** -6 * scale:
                break
        flat[p, l] = new
        hit[p] = True
        done += 1
    return hit


def _entry_errors(seed: int, p: int, L: int, scale: float):
    """Additive error of every entry of node p (zero where the entry is not hit)."""
    idx = np.arange(L, dtype=U64)
    phi = 1.0 - float(unit(draw(make_key(seed, TAG_PHI), p)))
    first = int(draw(make_key(seed, TAG_FIRST), p) % U64(L))
    hit = unit(draw(make_key(seed, TAG_ENTRY, p), idx)) < phi
    hit[first] = True
    r = draw(make_key(seed, TAG_MAG, p), idx)
    k = -4 + ((r >> U64(53)) % U64(12)).astype(np.int64)
    f = (r & U64((1 << 52) - 1)).astype(np.float64) * 2.0 ** -52
    neg = ((r >> U64(52)) & U64(1)).astype(bool)
    mag = np.ldexp(1.0 + f, k) * scale
    return np.where(hit, np.where(neg, -mag, mag), 0.0)


def inject_additive(outputs: np.ndarray, seed: int, scale: float, prob: float = 0.0,
                    nodes: Optional[Sequence[bool]] = None) -> np.ndarray:
    P = outputs.shape[0]
    flat = outputs.reshape(P, -1)
    sel = select_nodes(seed, P, prob) if nodes is None else np.asarray(nodes, dtype=bool)
    for p in np.flatnonzero(sel):
        e = _entry_errors(seed, int(p), flat.shape[1], scale)
        flat[p] = (flat[p].astype(np.float64) + e).astype(flat.dtype)
    return sel


def inject_gauss(outputs: np.ndarray, seed: int, scale: float, prob: float = 0.0,
                 nodes: Optional[Sequence[bool]] = None) -> np.ndarray:
    P = outputs.shape[0]
    flat = outputs.reshape(P, -1)
    L = flat.shape[1]
    sel = select_nodes(seed, P, prob) if nodes is None else np.asarray(nodes, dtype=bool)
    idx = np.arange(L, dtype=U64)
    for p in np.flatnonzero(sel):
        key = make_key(seed, TAG_GAUSS, int(p))
        u1 = ((draw(key, idx * U64(2)) >> U64(11)).astype(np.float64) + 1.0) * 2.0 ** -53
        u2 = unit(draw(key, idx * U64(2) + U64(1)))
        g = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
        flat[p] = (flat[p].astype(np.float64) + scale * g).astype(flat.dtype)
    return sel
