"""Writes tracegen/quantile_tables.json: the integer quantile tables the trace generator draws from.

Run once (`python -m tracegen.make_tables`); the JSON file is committed and is the definition of
the tables, so a trace is the same on every machine whatever its libm does in the last bit.

Every table has N+1 = 4097 knots at probabilities p_i = (i + 0.5) / (N + 1), i = 0..N, and holds
round(q(p_i) * 2**16):

  normal   q = standard normal quantile z(p)
  expo     q = -ln(1 - p)                       (unit-mean exponential)
  logn01   q = exp(0.1 * z(p))                  (lognormal, sigma 0.1, median 1)
  logn10   q = exp(1.0 * z(p))                  (lognormal, sigma 1.0, median 1)
"""
import json
import math
import os
from statistics import NormalDist

N = 4096
FRAC_BITS = 16


def build():
    nd = NormalDist()
    one = 1 << FRAC_BITS
    ps = [(i + 0.5) / (N + 1) for i in range(N + 1)]
    zs = [nd.inv_cdf(p) for p in ps]
    return {
        "n_intervals": N,
        "frac_bits": FRAC_BITS,
        "normal": [round(z * one) for z in zs],
        "expo": [round(-math.log1p(-p) * one) for p in ps],
        "logn01": [round(math.exp(0.1 * z) * one) for z in zs],
        "logn10": [round(math.exp(z) * one) for z in zs],
    }


if __name__ == "__main__":
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "quantile_tables.json")
    with open(out, "w") as f:
        json.dump(build(), f, separators=(",", ":"))
    print("wrote", out)
