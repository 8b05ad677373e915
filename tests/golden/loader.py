"""Parser for the small hand-written text fixtures in this folder."""
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
SCALARS = ("K", "N", "group_size")
SECTIONS = ("qweight", "q", "qzeros", "z", "scales", "g_idx", "x")


def load_fixture(name):
    """Return {scalar: int, section: list of token rows}."""
    out = {}
    section = None
    with open(os.path.join(HERE, name)) as f:
        for line in f:
            tok = line.split("#", 1)[0].split()
            if not tok:
                continue
            if tok[0] in SCALARS and len(tok) == 2:
                out[tok[0]] = int(tok[1])
            elif tok[0] in SECTIONS and len(tok) == 1:
                section = tok[0]
                out[section] = []
            else:
                out[section].append(tok)
    return out


def hex_words(rows):
    return np.array([[int(t, 16) for t in r] for r in rows], dtype=np.uint32).view(np.int32)


def numbers(rows, dtype):
    return np.array([[float(t) for t in r] for r in rows]).astype(dtype)
