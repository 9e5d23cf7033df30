"""Writes closed_forms.txt: activation, logsumexp and softmax values evaluated with 40-digit
arithmetic (mpmath), independent of the oracle and of the CUDA path.

The formulas are the definitions of the operators named by the benchmark
configurations (GELU in its tanh form, SiLU = z * sigmoid(z), logsumexp, softmax); the
paper itself prints no worked value for any of them, so these closed forms are
the fixed points the oracle is pinned to.

Run:  python tests/golden/make_closed_forms.py
"""
import os

import mpmath as mp

mp.mp.dps = 40
POINTS = ["-6", "-3", "-2", "-1", "-0.5", "-0.125", "0", "0.125", "0.5", "1", "2", "3", "6"]
LSE_CASES = [[0, 0, 0, 0], [1, 2, 3, 4], [-1, 0, 1, 2], [1000, 1000], [-1000, -1000.5, -999], [0.25]]
SOFTMAX_CASES = [[1, 2, 3, 4], [-1, 0, 1, 2], [0.5, -1.25, 3, 0.125, -7], [1000, 999.5, 990], [-20, 0, 20]]


def gelu_tanh(z):
    return 0.5 * z * (1 + mp.tanh(mp.sqrt(2 / mp.pi) * (z + mp.mpf("0.044715") * z ** 3)))


def silu(z):
    return z / (1 + mp.exp(-z))


def lse(v):
    m = max(v)
    return m + mp.log(sum(mp.exp(x - m) for x in v))


def main():
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "closed_forms.txt")
    with open(out, "w") as f:
        f.write("# kind  argument(s)  value   (40-digit mpmath evaluation, printed to 20 digits)\n")
        for p in POINTS:
            z = mp.mpf(p)
            f.write("gelu_tanh %s %s\n" % (p, mp.nstr(gelu_tanh(z), 20)))
            f.write("silu %s %s\n" % (p, mp.nstr(silu(z), 20)))
            f.write("relu %s %s\n" % (p, mp.nstr(max(z, mp.mpf(0)), 20)))
        for case in LSE_CASES:
            v = [mp.mpf(str(x)) for x in case]
            f.write("lse %s %s\n" % (",".join(str(x) for x in case), mp.nstr(lse(v), 20)))
        for case in SOFTMAX_CASES:      # one line per element: "softmax <logits>|<index> <probability>"
            v = [mp.mpf(str(x)) for x in case]
            total = lse(v)
            for i, x in enumerate(v):
                f.write("softmax %s|%d %s\n" % (",".join(str(c) for c in case), i, mp.nstr(mp.exp(x - total), 20)))


if __name__ == "__main__":
    main()
