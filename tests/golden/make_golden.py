"""Writes two_key_softmax.json from the logistic closed form (no oracle, no kernel)."""
import json
import math
import os

D = 128
cases = []
for q, a, b, w in [(1.0, 2.0, -1.0, 1), (0.5, 4.0, 4.0, 3), (-2.0, 1.0, 3.0, 2), (8.0, 0.25, -0.5, 4)]:
    # one query row (q, 0, ..., 0) repeated w times, keys (a, 0, ...) and (b, 0, ...)
    u0 = w / (1.0 + math.exp((b - a) * q / math.sqrt(D)))
    cases.append({"q": q, "a": a, "b": b, "w": w, "d": D, "u": [u0, w - u0]})
with open(os.path.join(os.path.dirname(__file__), "two_key_softmax.json"), "w") as f:
    json.dump({"_rule": "Section 4.5: softmax over two keys is the logistic function", "cases": cases}, f, indent=1)
