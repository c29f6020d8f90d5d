"""Oracle of the local halves of the Ulysses all-to-all (Section 3.5: the all-to-all transposes that
partition the attention heads across the ranks of a group; Eq. (ulysses) counts their volume).

TEST INFRASTRUCTURE ONLY. Nothing in the product path imports this module.

A group of P ranks holds a sequence by tokens: rank r owns n tokens with all h heads, [n, h, d]. Attention
wants the opposite split: all tokens, h / P heads per rank. The exchange is an all-to-all of P equal
blocks per rank; what runs on a rank before and after it is a pure permutation of 2-byte elements:

  pack    send[j, t, b, :] = x[t, j * (h / P) + b, :]      block j goes to rank j
  (all-to-all: recv[i] on rank r = send[r] of rank i, so recv is [P * n, h / P, d], tokens in rank order)
  unpack  y[t, j * (h / P) + b, :] = recv[j, t, b, :]       the way back, after attention

Both are written here element by element over the indices of the definition (plain Python loops over
(j, t, b); a row of d elements is copied as one slice), so that they can be checked against the text by
eye. The elements are opaque 16-bit patterns (numpy uint16): the result is exact.
"""
import numpy as np


def ulysses_pack(x: np.ndarray, cp_u: int) -> np.ndarray:
    """[n, h, d] -> [cp_u, n, h / cp_u, d]; cp_u must divide h."""
    n, h, d = x.shape
    if cp_u < 1 or h % cp_u:
        raise ValueError("the Ulysses degree must divide the head count")
    hg = h // cp_u
    send = np.empty((cp_u, n, hg, d), dtype=x.dtype)
    for j in range(cp_u):
        for t in range(n):
            for b in range(hg):
                send[j, t, b, :] = x[t, j * hg + b, :]
    return send


def ulysses_unpack(recv: np.ndarray) -> np.ndarray:
    """[cp_u, n, h / cp_u, d] -> [n, h, d]: the inverse of ulysses_pack."""
    cp_u, n, hg, d = recv.shape
    y = np.empty((n, cp_u * hg, d), dtype=recv.dtype)
    for j in range(cp_u):
        for t in range(n):
            for b in range(hg):
                y[t, j * hg + b, :] = recv[j, t, b, :]
    return y


def all_to_all(send_of_rank):
    """The exchange itself, on a list of per-rank send buffers [P, n, hg, d]: rank r receives block r of
    every rank, in rank order."""
    world = len(send_of_rank)
    return [np.stack([send_of_rank[i][r] for i in range(world)]) for r in range(world)]
