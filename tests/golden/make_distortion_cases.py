"""Writes distortion_cases.json: Eq. (Delta_def) and the regulariser of Algorithm 2 step 9 evaluated in
binary64 for inputs whose quotient is exactly representable.  Uses only the Python math module: no
oracle, no CUDA library."""
import json
import math
import os

cases = []


def case(G, w, ap, a, mu, note):
    delta = (G - w * ap) / (w * a)
    m = math.tanh(abs(1 + delta) / mu)
    cases.append(dict(g_prev=G, omega=w, a_prev=ap, a_now=a, mu=mu, delta=delta,
                      regulariser=float(f"{m:.12g}"), note=note))


case(1.0, 0.5, 1.0, 0.25, 4.0, "others contribute as much as this worker did; accumulator shrank 4x: Delta = 4")
case(0.75, 0.5, 0.5, 1.0, 4.0, "Delta = 1")
case(0.5, 0.5, 1.0, 1.0, 4.0, "only this worker sent the entry: Delta = 0, regulariser tanh(1/mu)")
case(0.5, 0.5, 1.0, 1.0, 1.0, "same with mu = 1")
case(0.0, 0.5, 2.0, 2.0, 4.0, "cancelled at the server: Delta = -1, regulariser 0")
case(-1.0, 0.25, 4.0, 2.0, 2.0, "aggregate opposes the worker: Delta = -4, |1+Delta| = 3")
case(3.0, 0.25, 4.0, -2.0, 2.0, "accumulator changed sign: Delta = -4")
case(2.0, 0.125, 8.0, 0.5, 8.0, "N = 8 weights; Delta = 16")
case(1.0, 0.5, -1.0, 0.5, 10.0, "previous value negative: numerator 1.5, Delta = 6")

out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "distortion_cases.json")
json.dump(dict(source="Eq. (Delta_def) and Algorithm 2 step 9, closed forms for exactly representable inputs",
               cases=cases), open(out, "w"), indent=1)
