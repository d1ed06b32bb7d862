"""Small random corpora for tests (inputs only; no scoring arithmetic)."""
import numpy as np


def unit_rows(rng, n, d):
    x = rng.standard_normal((n, d)).astype(np.float32)
    x /= np.linalg.norm(x, axis=1, keepdims=True)
    return x.astype(np.float32)


def random_corpus(seed, n_docs, n_centroids, dim, nbits, len_lo=1, len_hi=12):
    """Random unit centroids, random centroid ids, random code bytes, random lengths."""
    rng = np.random.default_rng(seed)
    cent = unit_rows(rng, n_centroids, dim)
    doclens = rng.integers(len_lo, len_hi + 1, size=n_docs).astype(np.int32)
    T = int(doclens.sum())
    cids = rng.integers(0, n_centroids, size=T).astype(np.int32)
    codes = rng.integers(0, 256, size=(T, dim * nbits // 8)).astype(np.uint8)
    return cent, cids, codes, doclens


def unpack_codes(codes, dim, nbits):
    """[T, D] integer bucket indices from packed bytes, written straight from the packing rule:
    2-bit: dimension 4g+t in bits [2t, 2t+1] of byte g; 1-bit: dimension 8g+t in bit t of byte g."""
    T = codes.shape[0]
    u = np.zeros((T, dim), dtype=np.int64)
    for x in range(dim):
        if nbits == 2:
            u[:, x] = (codes[:, x // 4].astype(np.int64) >> (2 * (x % 4))) & 3
        else:
            u[:, x] = (codes[:, x // 8].astype(np.int64) >> (x % 8)) & 1
    return u


def levels(nbits, lo=-0.25, hi=0.25):
    n = 1 << nbits
    delta = (hi - lo) / n
    return np.array([lo + (u + 0.5) * delta for u in range(n)], dtype=np.float64)
