"""Reader for the hand-worked fixtures in tests/golden/."""
import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _vals(tokens, n):
    if tokens == ["iota"]:
        return np.arange(n, dtype=np.float64)
    if tokens == ["ones"]:
        return np.ones(n, dtype=np.float64)
    v = np.array([float(t) for t in tokens], dtype=np.float64)
    assert v.size == n, (v.size, n)
    return v


def load_case(name):
    fields = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, rest = line.split(":", 1)
            fields[key.strip()] = rest.split()
    xs = tuple(int(t) for t in fields["x_shape"])
    ws = tuple(int(t) for t in fields["w_shape"])
    ys = tuple(int(t) for t in fields["y_shape"])
    p = fields["params"]
    params = {p[i]: int(p[i + 1]) for i in range(0, len(p), 2)}
    x = _vals(fields["x"], int(np.prod(xs))).reshape(xs).astype(np.float32)
    w = _vals(fields["w"], int(np.prod(ws))).reshape(ws).astype(np.float32)
    y = _vals(fields["y"], int(np.prod(ys))).reshape(ys)
    return x, w, params, y


def load_numbers(name, key):
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            if line.startswith(key + ":"):
                return [float(t) for t in line.split(":", 1)[1].split()]
    raise KeyError(key)
