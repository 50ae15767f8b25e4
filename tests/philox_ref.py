"""Host restatement of the library's Gaussian generator, for tests only: Philox-4x32 with 10
rounds (Salmon, Moraes, Dror, Shaw, SC'11) keyed by the seed, counter = (pair index, vector
index), Box-Muller in float64.  Written from the published algorithm with numpy integers."""
import numpy as np


def philox4x32_10(c, k):
    M0, M1, W0, W1 = 0xD2511F53, 0xCD9E8D57, 0x9E3779B9, 0xBB67AE85
    c = [np.asarray(x, dtype=np.uint64) for x in c]
    k0, k1 = np.uint64(k[0]), np.uint64(k[1])
    mask = np.uint64(0xFFFFFFFF)
    for _ in range(10):
        p0 = np.uint64(M0) * c[0]
        p1 = np.uint64(M1) * c[2]
        c = [((p1 >> np.uint64(32)) ^ c[1] ^ k0) & mask, p1 & mask, ((p0 >> np.uint64(32)) ^ c[3] ^ k1) & mask, p0 & mask]
        k0 = (k0 + np.uint64(W0)) & mask
        k1 = (k1 + np.uint64(W1)) & mask
    return c


def omega_reference(seed, n, nvec, first=0):
    npairs = (n + 1) // 2
    q, j = np.meshgrid(np.arange(npairs, dtype=np.uint64), np.arange(first, first + nvec, dtype=np.uint64))
    c = philox4x32_10([q & np.uint64(0xFFFFFFFF), q >> np.uint64(32), j & np.uint64(0xFFFFFFFF), j >> np.uint64(32)],
                       [seed & 0xFFFFFFFF, seed >> 32])
    a = (c[1] << np.uint64(32)) | c[0]
    bb = (c[3] << np.uint64(32)) | c[2]
    u1 = ((a >> np.uint64(12)).astype(np.float64) + 0.5) / 4503599627370496.0
    u2 = ((bb >> np.uint64(12)).astype(np.float64) + 0.5) / 4503599627370496.0
    rad = np.sqrt(-2.0 * np.log(u1))
    out = np.empty((nvec, 2 * npairs))
    out[:, 0::2] = rad * np.cos(2 * np.pi * u2)
    out[:, 1::2] = rad * np.sin(2 * np.pi * u2)
    return out[:, :n]


