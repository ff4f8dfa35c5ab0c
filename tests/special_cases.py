"""Hand-built matrices that reach corner cases of the device packer (used by CPU and GPU tests)."""
import numpy as np


def clustered_surplus_tile(seed=0):
    """One 128 x 128 tile whose surplus elements sit in two far-apart clusters of the bank-major slot
    order (the windows held by word 0 and by word 31 of every 128-byte row of the value image)
    while its empty slots are spread over the whole tile.  Consecutive pairs then straddle the gap
    between the clusters, which is more than 255 dummy bytes wide: the packer has to cut that chain
    and send the rest to the Residual list."""
    rng = np.random.default_rng(seed)
    W = np.zeros((128, 128), dtype=np.float16)

    def fill(r, q, n):                     # non-zeros at positions 0..n-1 of window q in row r: n = 3 leaves one surplus
        vals = (rng.standard_normal(n) * 0.05).astype(np.float16)
        vals[vals == 0] = np.float16(0.01)
        W[r, 4 * q:4 * q + n] = vals

    for r in range(128):
        q0 = (r & 7) << 2                  # window stored in word (bank) 0 of row r
        q31 = ((7 ^ (r & 7)) << 2) | 3     # window stored in word (bank) 31
        if r >= 4:
            fill(r, q0, 3)                 # 124 surplus elements in the first cluster (with 124 the
        fill(r, q31, 3)                    # cluster boundary falls inside a chain), 128 in the second
    return W
