"""Generator of the comparator networks the CUDA kernels keep in registers.

Writes csrc/sort_networks.inc with
  * MedianNet<N>::run  - a network that leaves the element of rank (N-1)/2 on wire (N-1)/2,
    obtained from an odd-even merge sort of N inputs by deleting every comparator (or comparator
    half) the middle output does not depend on;
  * SortNet<N>::run    - the full merge sort, for the trimmed mean.

The sizes are those of the coordinate-wise median over f = l*l files (l = 3, 5, 7) and of Bulyan's
selection sets theta = f - 2c for every c with f >= 4c + 3.

Run `python gen_networks.py` to rewrite the .inc file, `python gen_networks.py --check` to verify
that the committed file is current and that every network is correct (0-1 principle: exhaustively
for N <= 25, on random 0/1 and integer inputs above).
"""
import functools
import os
import random
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
OUT = os.path.join(HERE, "sort_networks.inc")

MEDIAN_SIZES = [9, 25, 49]
SORT_SIZES = sorted(set([f - 2 * c for f in (25, 49) for c in range(0, (f - 3) // 4 + 1)] + [5, 7, 9]))


def odd_even_merge(a, b):
    """Batcher's odd-even merge of two sorted runs of any lengths.  a, b: the wires holding each run in
    ascending order.  Returns (comparators, wires of the merged run in ascending order): the elements at
    even and at odd positions of both runs are merged recursively, then neighbours are exchanged."""
    if not a:
        return [], list(b)
    if not b:
        return [], list(a)
    if len(a) == 1 and len(b) == 1:
        return [(a[0], b[0])], [a[0], b[0]]
    ces_v, v = odd_even_merge(a[0::2], b[0::2])
    ces_w, w = odd_even_merge(a[1::2], b[1::2])
    ces = ces_v + ces_w
    out = [v[0]]
    pairs = min(len(w), len(v) - 1)
    for i in range(pairs):
        ces.append((w[i], v[i + 1]))
        out += [w[i], v[i + 1]]
    out += w[pairs:] + v[pairs + 1:]
    return ces, out


@functools.lru_cache(None)
def merge_count(m, n):
    return len(odd_even_merge(list(range(m)), list(range(m, m + n)))[0])


@functools.lru_cache(None)
def best_split(n):
    """(comparators, size of the first part) of the cheapest merge sort of n wires."""
    if n <= 1:
        return 0, 0
    return min((best_split(a)[0] + best_split(n - a)[0] + merge_count(a, n - a), a) for a in range(1, n // 2 + 1))


def merge_sort_wires(wires):
    n = len(wires)
    if n <= 1:
        return [], list(wires)
    a = best_split(n)[1]
    ces_a, run_a = merge_sort_wires(wires[:a])
    ces_b, run_b = merge_sort_wires(wires[a:])
    ces_m, run = odd_even_merge(run_a, run_b)
    return ces_a + ces_b + ces_m, run


def by_layers(ces):
    """The same comparators, earliest layer first (a comparator's layer is one more than the later layer of its
    two wires' previous comparators): independent comparators end up next to each other."""
    depth, keyed = {}, []
    for pos, (a, b) in enumerate(ces):
        layer = 1 + max(depth.get(a, 0), depth.get(b, 0))
        depth[a] = depth[b] = layer
        keyed.append((layer, pos, (a, b)))
    return [ce for _, _, ce in sorted(keyed)]


def merge_sort(n):
    """Comparators (wire of the min, wire of the max) of a merge sort of n wires whose splits minimise the
    comparator count (Batcher's network when n is a power of two; for other n it saves up to 16 % on padding
    to the next power).  Wires are renamed so that wire i ends with the element of rank i; a comparator may
    therefore put its min on the higher-numbered wire."""
    ces, run = merge_sort_wires(list(range(n)))
    name = {w: i for i, w in enumerate(run)}
    return by_layers([(name[a], name[b]) for a, b in ces])


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
        "// BZ_CE(a,b,i) leaves the min on wire a and the max on wire b; BZ_LO / BZ_HI keep only the min on a / the max",
        "// on b.  i numbers the full comparators: run<NUM, DEN> computes the max of those with i % DEN < NUM on the",
        "// multiply-add pipe.",
        "",
    ]
    for n in MEDIAN_SIZES:
        net = prune(merge_sort(n), [(n - 1) // 2])
        verify_median(net, n)
        ops = sum(int(x) + int(y) for _, _, x, y in net)
        lines.append("// median of %d: %d comparators, %d min/max operations" % (n, len(net), ops))
        lines.append("template <> struct MedianNet<%d> {" % n)
        lines.append("    template <int NUM = 0, int DEN = 1, typename T> __device__ __forceinline__ static T run(T (&k)[%d]) {" % n)
        body = []
        full = 0
        for a, b, na, nb in net:
            if na and nb:
                body.append("BZ_CE(%d,%d,%d)" % (a, b, full))
                full += 1
            else:
                body.append(("BZ_LO(%d,%d)" if na else "BZ_HI(%d,%d)") % (a, b))
        for i in range(0, len(body), 8):
            lines.append("        " + " ".join(body[i:i + 8]))
        lines.append("        return k[%d];" % ((n - 1) // 2))
        lines.append("    }")
        lines.append("};")
        lines.append("")
    for n in SORT_SIZES:
        ces = merge_sort(n)
        verify_sort(ces, n)
        lines.append("// sort of %d: %d comparators" % (n, len(ces)))
        lines.append("template <> struct SortNet<%d> {" % n)
        lines.append("    template <int NUM = 0, int DEN = 1, typename T> __device__ __forceinline__ static void run(T (&k)[%d]) {" % n)
        body = ["BZ_CE(%d,%d,%d)" % (a, b, i) for i, (a, b) in enumerate(ces)]
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
