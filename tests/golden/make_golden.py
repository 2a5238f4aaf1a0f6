"""Writes tests/golden/digest_zero_sequences.json from big-integer arithmetic only.

Facts stored (all follow from the digest's definition, h <- (h*B + t + 1) mod (2^61 - 1)):
  * all_zero: the digest of n zero tokens is the geometric sum (B^n - 1)/(B - 1) mod p;
  * zero_digest: per lane, three tokens whose digest is exactly 0, i.e.
    (t0+1)*B^2 + (t1+1)*B + (t2+1) = 0 mod p, found with a reduced 2-D lattice basis.
Run: python tests/golden/make_golden.py
"""
import json
import os

P = (1 << 61) - 1
BASE = (0x0B4E0EF37BC32127, 0x16A09E667F3BCC90)


def reduced_basis(b):
    """Gauss-reduced basis of the lattice {(x, y): x*b + y = 0 mod p} (exact integers)."""
    u, v = (1, (-b) % P), (0, P)
    n2 = lambda w: w[0] * w[0] + w[1] * w[1]
    while True:
        if n2(u) > n2(v):
            u, v = v, u
        d, n = u[0] * v[0] + u[1] * v[1], n2(u)
        m = (2 * d + n) // (2 * n)
        if m == 0:
            return u, v
        v = (v[0] - m * u[0], v[1] - m * u[1])


def zero_sequence(b):
    """Three tokens (t0, t1, t2) with (t0+1)*b^2 + (t1+1)*b + (t2+1) = 0 mod p: fix a small
    t0, then pick the lattice point nearest the middle of the token box for the other two."""
    u, v = reduced_basis(b)
    det = u[0] * v[1] - u[1] * v[0]
    for x0 in range(1, 10000):
        tx, ty = (1 << 31) - 0, (1 << 31) - (-x0 * b * b) % P      # centre - particular
        a0 = (tx * v[1] - ty * v[0]) // det                          # Cramer, floored
        c0 = (u[0] * ty - u[1] * tx) // det
        for a in (a0 - 1, a0, a0 + 1, a0 + 2):
            for c in (c0 - 1, c0, c0 + 1, c0 + 2):
                x1 = a * u[0] + c * v[0]
                x2 = (-x0 * b * b) % P + a * u[1] + c * v[1]
                if 0 < x1 <= 2**32 and 0 < x2 <= 2**32:
                    assert (x0 * b * b + x1 * b + x2) % P == 0
                    return [x0 - 1, x1 - 1, x2 - 1]
    raise SystemExit("no zero sequence found")


def main():
    out = {"all_zero": [], "zero_digest": [zero_sequence(b) for b in BASE]}
    for lane, b in enumerate(BASE):
        for n in (1, 16, 64, 4096, 131072):
            d = (pow(b, n, P) - 1) * pow(b - 1, P - 2, P) % P
            out["all_zero"].append({"lane": lane, "n": n, "digest": hex(d)})
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)),
                        "digest_zero_sequences.json")
    with open(path, "w") as f:
        json.dump(out, f, indent=1)
        f.write("\n")


if __name__ == "__main__":
    main()
