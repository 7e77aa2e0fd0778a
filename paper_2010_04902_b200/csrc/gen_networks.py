"""Generator of the comparator networks the CUDA kernels keep in registers.

Writes csrc/sort_networks.inc with
  * MedianNet<N>::run  - a network that leaves the element of rank (N-1)/2 on wire (N-1)/2,
    obtained from Batcher's odd-even merge sort for N inputs by deleting every comparator (or
    comparator half) the middle output does not depend on;
  * SortNet<N>::run    - the full odd-even merge sort, for the trimmed mean.

The sizes are those of the coordinate-wise median over f = l*l files (l = 3, 5, 7) and of Bulyan's
selection sets theta = f - 2c for every c with f >= 4c + 3.

Run `python gen_networks.py` to rewrite the .inc file, `python gen_networks.py --check` to verify
that the committed file is current and that every network is correct (0-1 principle: exhaustively
for N <= 25, on random 0/1 and integer inputs above).
"""
import os
import random
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
OUT = os.path.join(HERE, "sort_networks.inc")

MEDIAN_SIZES = [9, 25, 49]
SORT_SIZES = sorted(set([f - 2 * c for f in (25, 49) for c in range(0, (f - 3) // 4 + 1)] + [5, 7, 9]))


def batcher(n):
    """Comparators (lo_wire, hi_wire) of Batcher's odd-even merge sort for any n."""
    ces = []
    p = 1
    while p < n:
        k = p
        while k >= 1:
            j = k % p
            while j + k < n:
                for i in range(min(k, n - j - k)):
                    if (i + j) // (2 * p) == (i + j + k) // (2 * p):
                        ces.append((i + j, i + j + k))
                j += 2 * k
            k //= 2
        p *= 2
    return ces


def prune(ces, outputs):
    """Keep only what `outputs` depend on.  Returns (a, b, need_lo, need_hi) tuples."""
    need = set(outputs)
    keep = []
    for a, b in reversed(ces):
        na, nb = a in need, b in need
        if na or nb:
            keep.append((a, b, na, nb))
            need.add(a)
            need.add(b)
    keep.reverse()
    return keep


def run_network(net, v):
    v = list(v)
    for a, b, na, nb in net:
        lo, hi = min(v[a], v[b]), max(v[a], v[b])
        if na:
            v[a] = lo
        if nb:
            v[b] = hi
    return v


def _packed_wires(n):
    """Wire w as a bit-vector over all 2^n 0/1 inputs (input x has bit w of x on wire w), packed
    64 inputs per word."""
    words = max(1, (1 << n) >> 6)
    idx = np.arange(words, dtype=np.uint64)
    wires = []
    low = [0xAAAAAAAAAAAAAAAA, 0xCCCCCCCCCCCCCCCC, 0xF0F0F0F0F0F0F0F0, 0xFF00FF00FF00FF00, 0xFFFF0000FFFF0000,
           0xFFFFFFFF00000000]
    for w in range(n):
        if w < 6:
            wires.append(np.full(words, low[w], dtype=np.uint64))
        else:
            bit = (idx >> np.uint64(w - 6)) & np.uint64(1)
            wires.append(np.where(bit == 1, np.uint64(0xFFFFFFFFFFFFFFFF), np.uint64(0)))
    return wires


def verify_median(net, n):
    mid = (n - 1) // 2
    if 6 <= n <= 25:
        # 0-1 principle over all 2^n inputs: the middle output must be 1 exactly when at least
        # n - mid inputs are 1; the number of ones is counted independently of the network.
        wires = _packed_wires(n)
        ref = _packed_wires(n)
        for a, b, na, nb in net:
            lo, hi = wires[a] & wires[b], wires[a] | wires[b]
            if na:
                wires[a] = lo
            if nb:
                wires[b] = hi
        # reference by counting ones with bit-sliced adders (5 planes are enough for n <= 31)
        planes = [np.zeros_like(ref[0]) for _ in range(5)]
        for w in ref:
            carry = w
            for p in range(5):
                planes[p], carry = planes[p] ^ carry, planes[p] & carry
        need = n - mid  # the element of rank mid is 1 iff at least n - mid inputs are 1
        ge = np.zeros_like(ref[0])
        eq = ~np.zeros_like(ref[0])
        for p in reversed(range(5)):  # ones >= need, compared plane by plane from the top
            if (need >> p) & 1:
                eq &= planes[p]
            else:
                ge |= eq & planes[p]
                eq &= ~planes[p]
        ge |= eq
        assert np.array_equal(wires[mid], ge), "median network for n=%d is wrong" % n
    rng = random.Random(n)
    for _ in range(3000):
        kind = rng.random()
        if kind < 0.4:
            ones = rng.randint(0, n)
            v = [1] * ones + [0] * (n - ones)
            rng.shuffle(v)
        elif kind < 0.7:
            v = [rng.randint(0, 6) for _ in range(n)]
        else:
            v = [rng.randint(-10**6, 10**6) for _ in range(n)]
        assert run_network(net, v)[mid] == sorted(v)[mid], "median network for n=%d is wrong" % n


def verify_sort(ces, n):
    net = [(a, b, True, True) for a, b in ces]
    if 6 <= n <= 20:
        wires = _packed_wires(n)
        for a, b in ces:
            wires[a], wires[b] = wires[a] & wires[b], wires[a] | wires[b]
        for w in range(n - 1):
            assert not (wires[w] & ~wires[w + 1]).any(), "sorting network for n=%d is wrong" % n
    rng = random.Random(1000 + n)
    for _ in range(2000):
        v = [rng.randint(0, 8) for _ in range(n)] if rng.random() < 0.5 else [rng.random() for _ in range(n)]
        assert run_network(net, v) == sorted(v), "sorting network for n=%d is wrong" % n


def emit():
    lines = [
        "// GENERATED by gen_networks.py - do not edit.  Comparator networks on register arrays:",
        "// BZ_CE(a,b) orders wires a <= b; BZ_LO / BZ_HI keep only the min on a / the max on b.",
        "// BZ_CM is a BZ_CE that run<true> computes on the multiply-add pipe (two of three full comparators).",
        "",
    ]
    for n in MEDIAN_SIZES:
        net = prune(batcher(n), [(n - 1) // 2])
        verify_median(net, n)
        ops = sum(int(x) + int(y) for _, _, x, y in net)
        lines.append("// median of %d: %d comparators, %d min/max operations" % (n, len(net), ops))
        lines.append("template <> struct MedianNet<%d> {" % n)
        lines.append("    template <bool MIX = false, typename T> __device__ __forceinline__ static T run(T (&k)[%d]) {" % n)
        body = []
        full = 0
        for a, b, na, nb in net:
            if na and nb:
                full += 1
                body.append(("BZ_CM(%d,%d)" if full % 3 else "BZ_CE(%d,%d)") % (a, b))
            else:
                body.append(("BZ_LO(%d,%d)" if na else "BZ_HI(%d,%d)") % (a, b))
        for i in range(0, len(body), 8):
            lines.append("        " + " ".join(body[i:i + 8]))
        lines.append("        return k[%d];" % ((n - 1) // 2))
        lines.append("    }")
        lines.append("};")
        lines.append("")
    for n in SORT_SIZES:
        ces = batcher(n)
        verify_sort(ces, n)
        lines.append("// sort of %d: %d comparators" % (n, len(ces)))
        lines.append("template <> struct SortNet<%d> {" % n)
        lines.append("    template <bool MIX = false, typename T> __device__ __forceinline__ static void run(T (&k)[%d]) {" % n)
        body = [("BZ_CM(%d,%d)" if i % 3 else "BZ_CE(%d,%d)") % (a, b) for i, (a, b) in enumerate(ces)]
        for i in range(0, len(body), 8):
            lines.append("        " + " ".join(body[i:i + 8]))
        lines.append("    }")
        lines.append("};")
        lines.append("")
    return "\n".join(lines)


def main():
    text = emit()
    if "--check" in sys.argv:
        with open(OUT) as fh:
            if fh.read() != text:
                print("sort_networks.inc is stale: run gen_networks.py")
                return 1
        print("sort_networks.inc is current; all networks verified")
        return 0
    with open(OUT, "w") as fh:
        fh.write(text)
    print("wrote", OUT)
    return 0


if __name__ == "__main__":
    sys.exit(main())
