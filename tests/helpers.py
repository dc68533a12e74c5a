"""Shared test helpers (no method arithmetic)."""
import os


def paper_values():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_values.txt")
    out = {}
    with open(path) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            k, v = (s.strip() for s in line.split("=", 1))
            out[k] = float(v)
    return out
