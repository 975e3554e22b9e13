"""fp64 numpy algebra shared by the tests: the leaf weights that the binary Adasum tree assigns,
derived from the Gram matrix of the leaves alone (every tree node is a linear combination of the
leaves).  Pinned against the literal-tree oracle in test_oracle_pins.py."""
import numpy as np


def leaf_weights_from_gram(gram):
    n = gram.shape[0]
    c = np.ones(n)
    blocks = [([i], gram[i, i]) for i in range(n)]
    while len(blocks) > 1:
        nxt = []
        for i in range(0, len(blocks) - 1, 2):
            (left, na), (right, nb) = blocks[i], blocks[i + 1]
            d = sum(c[p] * c[q] * gram[p, q] for p in left for q in right)
            ca = 1.0 if na == 0 else 1.0 - d / (2 * na)
            cb = 1.0 if nb == 0 else 1.0 - d / (2 * nb)
            c[left] *= ca
            c[right] *= cb
            nxt.append((left + right, ca * ca * na + cb * cb * nb + 2 * ca * cb * d))
        if len(blocks) % 2:
            nxt.append(blocks[-1])
        blocks = nxt
    return c
