"""Print the 24 Q63 constants floor(2^63 * 2^(-2^-i)) used by the device-side 2^(-z).

Method: a chain of big-integer square roots carried with 256 guard bits,
r_1 = isqrt(2^(2W) / 2), r_i = isqrt(r_{i-1} * 2^W) with W = 63 + 256, then r_i >> 256.
"""
from math import isqrt

GUARD = 256
W = 63 + GUARD


def consts():
    out = []
    r = isqrt((1 << (2 * W)) >> 1)          # 2^W * 2^(-1/2)
    out.append(r >> GUARD)
    for _ in range(2, 25):
        r = isqrt(r << W)                   # sqrt(r/2^W) * 2^W
        out.append(r >> GUARD)
    return out


if __name__ == "__main__":
    v = consts()
    for i in range(0, 24, 3):
        print("    " + " ".join("0x%016XULL," % x for x in v[i:i + 3]))
