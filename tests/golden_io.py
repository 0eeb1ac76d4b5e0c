"""Parser for tests/golden/hand_vectors.txt (format described in that file)."""
import os
import re

import numpy as np

_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "hand_vectors.txt")


def _expand(tokens: str):
    out = []
    for m in re.finditer(r"(\d+)\*\(([^)]*)\)|([0-9a-fA-F]+)", tokens):
        if m.group(1):
            out.extend(m.group(2).split() * int(m.group(1)))
        else:
            out.append(m.group(3))
    return out


def _words(s: str) -> np.ndarray:
    return np.array([int(t, 16) for t in s.split()], dtype=np.uint32)


def load():
    recs = {"pack": [], "vote": [], "momentum": [], "apply": []}
    with open(_PATH) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            parts = [p.strip() for p in line.split("|")]
            kind = parts[0]
            if kind == "pack":
                toks = _expand(parts[2])
                if parts[1] == "f32":
                    arr = np.array([int(t, 16) for t in toks], dtype=np.uint32).view(np.float32)
                else:
                    arr = np.array([int(t, 16) for t in toks], dtype=np.uint16)
                recs["pack"].append((parts[1], arr, _words(parts[3])))
            elif kind == "vote":
                workers = [_words(w) for w in parts[3].split(";")]
                recs["vote"].append((int(parts[1]), int(parts[2], 16), workers, _words(parts[4])))
            elif kind == "momentum":
                recs["momentum"].append(tuple(float(x) for x in parts[1:5]) + (int(parts[5]),))
            elif kind == "apply":
                recs["apply"].append((float(parts[1]), int(parts[2]), float(parts[3]),
                                      float(parts[4]), float(parts[5])))
            else:
                raise ValueError("unknown record kind %r" % kind)
    return recs
