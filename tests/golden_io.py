"""Reader for tests/golden/mxint_worked_blocks.txt (plain text, '|' separated fields)."""
import os

_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "mxint_worked_blocks.txt")


def _kv(field):
    out = {}
    for tok in field.split():
        k, v = tok.split("=", 1)
        out[k] = v
    return out


def load():
    rows = []
    with open(_PATH) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            parts = [p.strip() for p in line.split("|")]
            rec = {"kind": parts[0]}
            for p in parts[1:]:
                rec.update(_kv(p))
            rows.append(rec)
    return rows


def floats(s):
    return [float(t) for t in s.split(",")]


def ints(s):
    return [int(t) for t in s.split(",")]
